"""PuzzleKV decode hot path for B200 (sm_100a): mixed dense/factor paged-KV
attention and batched per-page truncated SVD behind a small C ABI.

`paper_2608_23843_b200.pkv` is the Python binding of that ABI (argument
marshalling only); `paper_2608_23843_b200.synth` draws seeded synthetic inputs.
Importing this package does not load the CUDA library; the binding loads it on
first use and raises if it has not been built.
"""
__all__ = ["pkv", "synth"]
