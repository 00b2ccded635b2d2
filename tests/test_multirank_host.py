"""World-size-2 gloo test of the benchmark's multi-rank host logic (no GPU).

The path shards along tokens with no data-path collective: every rank runs its own batch and only the
timing is combined -- MAX of the elapsed time, SUM of the tokens.  The reference arm runs on rank 0 only.
"""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        elapsed, tokens = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 8192 * 3, dist, torch.device("cpu"))
        out.put((rank, elapsed, tokens))
    finally:
        dist.destroy_process_group()


def test_timing_is_max_over_ranks_and_tokens_are_summed():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == [0, 1]
    for _, elapsed, tokens in results:
        assert elapsed == 15.0                 # the slower rank decides
        assert tokens == 2 * 8192 * 3          # weak scaling: every rank brings its own batch


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 100) == (3.5, 100)
    fl = bench.layer_flops(8192, 4096, 11008, 64)
    assert fl["fwd"] == 2.0 * 8192 * 4096 * 11008 and fl["dw"] == 2.0 * 8192 * 11008 * 64 + 11008 * 4096


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    import oracle
    import velora_inputs as vi
    from paper_2405_17991_b200.distributed import allreduce_sum_
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        N, D, O, Dsub = 96, 80, 12, 16
        case = vi.small_case(77, N, D, O, dtype="bf16", mean_offset=0.2)
        X, dY = case["X"].f64(), case["dY"].f64()
        lo, hi = (0, 37) if rank == 0 else (37, N)            # uneven shards of the token dimension
        # the stand-in for this rank's kernels is the oracle: what is tested is the exchange
        _, s_local, _ = oracle.init_v(X[lo:hi], Dsub, return_sum=True)
        s = allreduce_sum_(torch.from_numpy(s_local.copy()))
        v = s.numpy() / np.linalg.norm(s.numpy())
        Z_local = oracle.compress(X[lo:hi], v)
        _, P_local = oracle.weight_grad(dY[lo:hi], Z_local, v, D, factored=True, return_P=True)
        P = allreduce_sum_(torch.from_numpy(P_local.copy())).numpy()
        dW = np.einsum("om,j->omj", P, v).reshape(O, -1)[:, :D]
        v_full = oracle.init_v(X, Dsub)
        dW_full = oracle.weight_grad(dY, oracle.compress(X, v_full), v_full, D)
        out.put((rank, float(np.abs(v - v_full).max()), float(np.abs(dW - dW_full).max() / np.abs(dW_full).max())))
    finally:
        dist.destroy_process_group()


def test_sharded_batches_reproduce_the_single_process_result():
    """Two ranks, each with its rows: all-reducing s (Dsub floats) and P (O*M floats) gives every rank the
    v and the dW of the undivided batch."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, dv, dw in results:
        assert dv < 1e-12 and dw < 1e-12
