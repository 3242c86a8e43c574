"""Parameter-range sharding for one rank per GPU: the range rule, the exchange protocol on two
gloo ranks (CPU tensors; each rank's owned ranges are updated by the CPU oracle, standing in for
the kernel that a rank would run on its GPU), and the sharded step on one GPU with the ranks taken
one after the other."""
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
    S.exchange(t_theta + t_v, world, dist)
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
