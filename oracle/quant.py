"""ORACLE — TEST INFRASTRUCTURE ONLY.

INT4 quantization of the page factors (Section 4.3, "Quantization Compatibility").

The singular values are split evenly between the two factors,
    L~ = U_r Sigma_r^{1/2}   (P x r),      R~ = Sigma_r^{1/2} W_r^T   (r x d),
and each factor matrix gets symmetric INT4 quantization: column-wise for L~_K and R~_K, row-wise for
L~_V, column-wise for R~_V.

Readings (the paper says only "symmetric INT4"): one scale per column (or row), scale = max|x| / 7
stored in bf16, code = round-half-even(x / stored scale) clipped to [-7, 7] (no -8: symmetric),
a zero column gets scale 0 and codes 0.  The value attention reads is the stored factor dequantised
to the storage/compute type of the dense cache: bf16(code * scale), one rounding.
"""
import numpy as np

from .bf16 import round_to_bf16

QMAX = 7


def balanced_factors(A: np.ndarray, B: np.ndarray):
    """A: [P, r] orthonormal columns, B: [r, d] = Sigma W^T  ->  (L~, R~, sigma) with L~ R~ = A B."""
    sigma = np.linalg.norm(B, axis=1)
    root = np.sqrt(sigma)
    inv = np.where(root > 0, 1.0 / np.where(root > 0, root, 1.0), 0.0)
    return A * root[None, :], B * inv[:, None], sigma


def quantize(x: np.ndarray, axis: int):
    """Symmetric INT4 along `axis` groups: axis=0 -> one scale per column, axis=1 -> one per row.
    Returns (codes int8 in [-7, 7], stored scales fp64 holding bf16 values)."""
    amax = np.abs(x).max(axis=axis, keepdims=True)
    scale = round_to_bf16(amax / QMAX)
    safe = np.where(scale > 0, scale, 1.0)
    codes = np.clip(np.rint(x / safe), -QMAX, QMAX)
    codes = np.where(scale > 0, codes, 0.0).astype(np.int8)
    return codes, scale


def dequantize(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """bf16(code * scale) as fp64."""
    return round_to_bf16(codes.astype(np.float64) * scale)


def quantized_page_factors(A_k, B_k, A_v, B_v):
    """The four stored matrices of one page after INT4 quantization, dequantised:
    (A_k^, B_k^, A_v^, B_v^) with A^ B^ ~= A B.  Column-wise: L~_K, R~_K, R~_V; row-wise: L~_V."""
    Lk, Rk, _ = balanced_factors(A_k, B_k)
    Lv, Rv, _ = balanced_factors(A_v, B_v)
    out = []
    for x, axis in ((Lk, 0), (Rk, 0), (Lv, 1), (Rv, 0)):
        out.append(dequantize(*quantize(x, axis)))
    return tuple(out)


def int4_page_storage_ratio(r_k: int, r_v: int, P: int, d: int, scale_bytes: int = 2, dense_bytes: int = 2) -> float:
    """Stored bytes of an INT4 factor page pair over the dense bf16 pair: half a byte per factor element
    plus one scale per column of L~_K (r_k), of R~_K (d), per row of L~_V (P) and per column of R~_V (d)."""
    codes = (r_k + r_v) * (P + d) / 2.0
    scales = scale_bytes * (r_k + d + P + d)
    return (codes + scales) / (2.0 * P * d * dense_bytes)
