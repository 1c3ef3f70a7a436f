"""Host-side logic of the N > 1 benchmark path, on CPU with the gloo backend (world size 2):
the max-over-ranks reduction, and the reference arm under torchrun (rank 0 alone prints)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    vals = bench.max_over_ranks([10.0 + rank, 5.0 - rank, 7.0], world)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = vals


def test_max_over_ranks_gloo_world2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    assert out[0] == out[1] == [11.0, 5.0, 7.0]


def test_reference_arm_under_torchrun_prints_once():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29612", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--workload", "tiny", "--steps", "1", "--warmup", "0"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["unit"] == "us" and d["higher_is_better"] is False
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["config"]["workload"] == "tiny" and d["value"] > 0


def test_plain_launch_with_gpus_2_starts_two_ranks_itself():
    """`python bench.py --gpus 2` without a launcher around it must start one rank per GPU on its own (here the
    reference arm, which needs no GPU): one JSON line, n_gpus 2, and both ranks ran (rank 1 leaves a marker)."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload", "tiny",
           "--steps", "1", "--warmup", "0"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    env.update(OMP_NUM_THREADS="2", PKV_BENCH_RANK_MARKER="1")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["impl"] == "reference"
    assert "rank 1 of 2 present" in r.stderr


def _shard_worker(rank, world, port, out):
    """Each rank owns a token range of one sequence, computes its softmax state with the oracle, and gathers the
    states with the package's helper (gloo, CPU tensors)."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import attention as att
    from paper_2608_23843_b200 import sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(7)                        # the same stream on both ranks
    T, d, Hq = 90, 128, 4
    K, V, q = rng.standard_normal((T, d)), rng.standard_normal((T, d)), rng.standard_normal((1, Hq, d))
    lo, hi = (0, 53) if rank == 0 else (53, T)
    state = torch.zeros((1, Hq, d + 2), dtype=torch.float64)
    for h in range(Hq):
        m, l, o = att.page_state_dense(q[0, h], K[lo:hi], V[lo:hi], d ** -0.5)
        state[0, h, :d] = torch.from_numpy(o)
        state[0, h, d], state[0, h, d + 1] = m, l
    gathered = sharded.gather_states(state)
    dist.barrier()
    dist.destroy_process_group()
    merged = []
    for h in range(Hq):
        sts = [(float(gathered[r, 0, h, d]), float(gathered[r, 0, h, d + 1]), gathered[r, 0, h, :d].numpy()) for r in range(world)]
        merged.append(att.merge_page_states(sts))
    ref = [att.attention_plain(q[0, h], K, V, d ** -0.5) for h in range(Hq)]
    out[rank] = (tuple(gathered.shape), float(max(np.abs(a - b).max() for a, b in zip(merged, ref))),
                 float(gathered[rank, 0, 0, d + 1] - state[0, 0, d + 1]))


def test_gathered_shard_states_merge_to_full_attention_gloo_world2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(2, 29613, out), nprocs=2, join=True)
    for rank in (0, 1):
        shape, err, own = out[rank]
        assert shape == (2, 1, 4, 130) and err <= 1e-13 and own == 0.0     # slot `rank` of the result is the rank's own state
