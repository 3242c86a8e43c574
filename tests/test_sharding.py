"""Parameter-range sharding for one rank per GPU: the range rule, the exchange protocol on two
gloo ranks (CPU tensors; each rank's owned ranges are updated by the CPU oracle, standing in for
the kernel that a rank would run on its GPU), the sharded step on one GPU with the ranks taken
one after the other, and the whole path as it runs with one process per rank -- two processes
that share one GPU, map each other's gradient buffers through CUDA IPC, run the library's kernels
on their own ranges over local and peer memory and pull the updated ranges back."""
import os
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from paper_2503_17469_b200 import binding as B

ROOT = Path(__file__).resolve().parents[1]
UNIT = 64


@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_ranges_tile_the_bucket_in_order_on_unit_boundaries(world):
    for n in list(range(0, 5 * UNIT + 3)) + [1000, 4095, 4097, 25_557_032, 102_760_448]:
        pos, counts = 0, []
        for rank in range(world):
            b, c = B.shard_range(n, world, rank)
            assert b == pos and (b % UNIT == 0 or b == n)
            pos += c
            counts.append(c)
        assert pos == n
        units = [-(-c // UNIT) for c in counts]
        assert max(units) - min(units) <= 1                      # balanced to one unit
        nonempty = [c for c in counts if c]
        assert all(c % UNIT == 0 for c in nonempty[:-1])           # only the range holding the tail is ragged


def test_range_arguments_are_validated():
    L = B.lib()
    import ctypes as C

    b, c = C.c_uint64(), C.c_uint64()
    assert L.omni_shard_range(10, 0, 0, C.byref(b), C.byref(c)) == B.ERR_BAD_CONFIG
    assert L.omni_shard_range(10, 2, 2, C.byref(b), C.byref(c)) == B.ERR_BAD_CONFIG
    assert L.omni_shard_range(10, 2, -1, C.byref(b), C.byref(c)) == B.ERR_BAD_CONFIG
    assert L.omni_shard_range(10, 2, 0, None, C.byref(c)) == B.ERR_NULL


def _inputs(K, sizes, seed):
    rng = np.random.default_rng(seed)
    theta = [rng.normal(0, 0.05, n).astype(np.float32) for n in sizes]
    v = [np.zeros(n, np.float32) for n in sizes]
    g = [[rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(K)] for n in sizes]
    return theta, v, g


def _gloo_rank(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, str(ROOT))
    import torch.distributed as dist

    from oracle import oracle as O
    from paper_2503_17469_b200 import sharded as S

    dist.init_process_group("gloo")
    K, sizes, b = 3, [1000, 4097, 70], [3, 10, 19]
    theta, v, g = _inputs(K, sizes, 11)                      # every rank draws the same inputs
    t_theta = [torch.from_numpy(t) for t in theta]           # share memory with the numpy arrays
    t_v = [torch.from_numpy(x) for x in v]
    local_sq = 0.0
    for i, (lo, cnt) in enumerate(S.owned_ranges(sizes, world, rank)):
        if cnt:
            sl = slice(lo, lo + cnt)
            th, vv = theta[i][sl].copy(), v[i][sl].copy()
            local_sq += O.bsp_step_f32([np.ascontiguousarray(x[sl]) for x in g[i]], b, th, vv, 0.1, 0.9, 0.0)
            theta[i][sl], v[i][sl] = th, vv
    S.all_gather_ranges(t_theta, world, rank, dist)          # one all-gather per tensor over padded ranges
    S.exchange(t_v, world, dist)                             # one broadcast per (tensor, owner)
    total = S.total_sqnorm(local_sq, dist)
    np.savez(Path(out_dir, f"rank{rank}.npz"), total=total, **{f"theta{i}": t for i, t in enumerate(theta)},
             **{f"v{i}": x for i, x in enumerate(v)})
    dist.destroy_process_group()


def test_two_ranks_exchange_their_ranges_and_add_their_norms(tmp_path):
    from oracle import oracle as O

    world = 2
    port = 31500 + os.getpid() % 2000
    mp.spawn(_gloo_rank, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    K, sizes, b = 3, [1000, 4097, 70], [3, 10, 19]
    theta, v, g = _inputs(K, sizes, 11)
    want_sq = sum(O.bsp_step_f32(g[i], b, theta[i], v[i], 0.1, 0.9, 0.0) for i in range(len(sizes)))
    for rank in range(world):
        got = np.load(tmp_path / f"rank{rank}.npz")
        for i in range(len(sizes)):
            assert np.array_equal(got[f"theta{i}"], theta[i]) and np.array_equal(got[f"v{i}"], v[i])
        assert abs(float(got["total"]) - want_sq) <= 1e-12 * want_sq


@pytest.mark.gpu
@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("world", [2, 4, 7])
def test_sharded_step_on_one_gpu_rank_after_rank(world, kind):
    """The ranks' sub-range steps run one after the other on one GPU (the K gradient buffers stand
    for the peer-mapped ones): together they are the full step, bit for bit, and their squared
    norms add up to the aggregate's."""
    from oracle import oracle as O
    from paper_2503_17469_b200 import sharded as S

    from parity_util import SQNORM_RTOL, to_np

    dev = "cuda:0"
    K, sizes, b = 8, [3 * 8192 + 17, 50, 100_003], [4, 8, 12, 16, 20, 24, 28, 144]
    gen = torch.Generator(device=dev).manual_seed(99)
    gdt = torch.bfloat16 if kind == "bf16" else torch.float32
    theta = [torch.empty(n, device=dev).normal_(0, 0.05, generator=gen) for n in sizes]
    v = [torch.zeros(n, device=dev) for n in sizes]
    grads = [[torch.empty(n, device=dev).normal_(0, 1e-3, generator=gen).to(gdt) for _ in range(K)] for n in sizes]
    th_o, v_o = [to_np(t) for t in theta], [to_np(x) for x in v]
    g_o = [[to_np(x) for x in row] for row in grads]
    sq = 0.0
    for rank in range(world):
        o = B.Omni(K, 256, 4, 200, 0.1)
        o.aggregate_bsp(S.shard_buckets(theta, grads, v, None, world, rank), b, 0.1, 0.9, 1e-4)
        sq += o.stats().grad_sqnorm
    want = sum(O.bsp_step_f32(g_o[i], b, th_o[i], v_o[i], 0.1, 0.9, 1e-4) for i in range(len(sizes)))
    for i in range(len(sizes)):
        assert np.array_equal(to_np(theta[i]), th_o[i]) and np.array_equal(to_np(v[i]), v_o[i])
    assert abs(sq - want) <= SQNORM_RTOL * want


# ------------------------------------------------------------------------------------------------
# one process per rank, two ranks on one GPU, peers' buffers mapped through CUDA IPC
# ------------------------------------------------------------------------------------------------
IPC_K, IPC_SIZES, IPC_B, IPC_STEPS = 4, [3 * 8192 + 17, 50, 100_003], [8, 24, 40, 56], 2


def _ipc_inputs(kind):
    rng = np.random.default_rng(2024)
    theta = [rng.normal(0, 0.05, n).astype(np.float32) for n in IPC_SIZES]
    g32 = [[rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(IPC_K)] for n in IPC_SIZES]
    if kind == "bf16":      # both sides consume the same rounded bits (rounding by torch, as in the workloads)
        g = [[torch.from_numpy(x).to(torch.bfloat16) for x in row] for row in g32]
    else:
        g = [[torch.from_numpy(x) for x in row] for row in g32]
    return theta, g


def _ipc_rank(rank, world, port, out_dir, flags, kind):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, str(ROOT))
    import torch.distributed as dist

    from paper_2503_17469_b200 import binding as Bc
    from paper_2503_17469_b200 import sharded as S

    dist.init_process_group("gloo")
    torch.cuda.set_device(0)
    dev = "cuda:0"
    Bc.DEFAULT_FLAGS = flags
    theta_np, g_cpu = _ipc_inputs(kind)
    nb = len(IPC_SIZES)
    theta = [torch.from_numpy(t).to(dev) for t in theta_np]            # every rank keeps a full replica
    v = [torch.zeros(n, device=dev) for n in IPC_SIZES]
    mine = [k for k in range(IPC_K) if k % world == rank]               # worker k computes on rank k mod world
    own_g = {(i, k): g_cpu[i][k].to(dev) for i in range(nb) for k in mine}
    keys = sorted(own_g)
    torch.cuda.synchronize()
    views = S.map_peers([own_g[key] for key in keys] + theta + v, dist)
    ng = len(keys)
    # grads[i][k]: the local buffer for this rank's workers, the peer mapping for the others
    grads = []
    for i in range(nb):
        row = []
        for k in range(IPC_K):
            owner = k % world
            peers_keys = sorted((ii, kk) for ii in range(nb) for kk in range(IPC_K) if kk % world == owner)
            row.append(views[owner][peers_keys.index((i, k))])
        grads.append(row)
    state_views = [vw[ng:] for vw in views]                            # every rank's theta and v buckets
    o = Bc.Omni(IPC_K, sum(IPC_B), 1, sum(IPC_B), 0.1)
    totals = []
    for _ in range(IPC_STEPS):
        dist.barrier()                                                  # all gradients are in place
        o.aggregate_bsp(S.shard_buckets(theta, grads, v, None, world, rank), IPC_B, 0.1, 0.9, 1e-4)
        local_sq = o.stats().grad_sqnorm                                # synchronises the stream
        dist.barrier()                                                  # every owner has updated its ranges
        S.pull_ranges(theta + v, state_views, world, rank)
        torch.cuda.synchronize()
        totals.append(S.total_sqnorm(local_sq, dist))
    np.savez(Path(out_dir, f"rank{rank}.npz"), totals=np.array(totals),
             **{f"theta{i}": t.cpu().numpy() for i, t in enumerate(theta)},
             **{f"v{i}": x.cpu().numpy() for i, x in enumerate(v)})
    del views, grads, state_views                                       # unmap before the owners free
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.gpu
@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("family", ["bulk", "registers"])
def test_two_processes_on_one_gpu_read_each_others_gradients_through_ipc(tmp_path, family, kind):
    """Algorithm 1's AllReduce + update as it runs with one process per rank: worker k's gradient
    lives in the process of rank k mod 2, each rank runs the fused step on its ranges reading two
    gradients from its own memory and two through IPC mappings of the other process's memory, then
    pulls the other rank's updated ranges.  Both replicas must equal the oracle's full step bit
    for bit after two steps, and the ranks' squared norms must add up to the aggregate's."""
    from oracle import oracle as O

    from parity_util import SQNORM_RTOL

    world = 2
    port = 33500 + os.getpid() % 2000
    flags = {"bulk": B.BULK_COPY, "registers": B.NO_BULK_COPY}[family]
    mp.spawn(_ipc_rank, args=(world, port, str(tmp_path), flags, kind), nprocs=world, join=True)
    theta, g = _ipc_inputs(kind)
    v = [np.zeros(n, np.float32) for n in IPC_SIZES]
    as_np = lambda t: t.view(torch.int16).numpy().view(np.uint16).copy() if t.dtype == torch.bfloat16 else t.numpy()
    want = []
    for _ in range(IPC_STEPS):
        want.append(sum(O.bsp_step_f32([as_np(x) for x in g[i]], IPC_B, theta[i], v[i], 0.1, 0.9, 1e-4)
                        for i in range(len(IPC_SIZES))))
    for rank in range(world):
        got = np.load(tmp_path / f"rank{rank}.npz")
        for i in range(len(IPC_SIZES)):
            assert np.array_equal(got[f"theta{i}"], theta[i]), (rank, i)
            assert np.array_equal(got[f"v{i}"], v[i]), (rank, i)
        for a, w in zip(got["totals"], want):
            assert abs(float(a) - w) <= SQNORM_RTOL * w


@pytest.mark.gpu
def test_bench_sharded_leg_with_two_ranks_on_one_gpu():
    """`bench.py --extras sharded --sharded-exchange ipc` under torchrun with two ranks that share
    the GPU: the headline configuration stepped by both ranks together (8 workers' gradients per
    rank, the other 8 read through IPC mappings) must equal the unsharded step bit for bit."""
    import json
    import subprocess

    port = 35500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), "bench.py", "--gpus", "2", "--steps", "5",
           "--warmup", "3", "--extras", "sharded", "--sharded-exchange", "ipc", "--no-cpu-baseline"]
    r = subprocess.run(cmd, cwd=str(ROOT), capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][-1])
    sh = line["extras"]["resnet50_bf16+sharded"]
    assert line["n_gpus"] == 2 and sh["ranks"] == 2 and sh["exchange"] == "ipc"
    assert sh["matches_unsharded_step_bit_for_bit"] is True
