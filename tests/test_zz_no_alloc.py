"""The allocation-free entry point against the regular one.

``omni_aggregate_bsp_noalloc`` exists for callers that cannot allocate device memory while they
step: code running inside another framework's allocator callback or under its allocator lock,
processes whose device memory is entirely owned by a pool, and loops that forbid calls which
may synchronise the device.  It keeps its scratch in a fixed array of the library image instead
of a workspace allocated on first use.  The file name makes pytest collect it last, so a run that
stops at the first failure has already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2503_17469_b200 import binding as B

from parity_util import TOL, SQNORM_RTOL, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(K, n, kind, seed):
    gen = torch.Generator(device=DEV).manual_seed(seed)
    gdt = torch.bfloat16 if kind == "bf16" else torch.float32
    theta = torch.empty(n, device=DEV).normal_(0, 0.05, generator=gen)
    grads = [torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen).to(gdt) for _ in range(K)]
    return theta, grads


@pytest.mark.parametrize("kind,K,n", [("bf16", 16, 3 * 12288 * 7 + 11), ("f32", 8, 200_003), ("f32", 3, 77)])
def test_noalloc_matches_regular_entry_point_twice_in_a_row(kind, K, n):
    """Two calls in a row through the C ABI on the same state; parameters, momentum, the bf16
    copy and the squared norm must agree with omni_aggregate_bsp within the tolerance the parity
    tests use.  The second call also shows that the shared scratch is cleaned between calls."""
    theta0, grads = _inputs(K, n, kind, 4242 + K)
    b = [int(x) for x in np.random.default_rng(K).integers(1, 97, K)]
    # regular path (context, workspace allocated on first launch)
    th_a, v_a = theta0.clone(), torch.zeros(n, device=DEV)
    lp_a = torch.zeros(n, device=DEV, dtype=torch.bfloat16)
    ctx = B.Omni(K, sum(b), 1, sum(b), 0.1)
    bs_a = B.BucketSet([th_a], [grads], [v_a], [lp_a])
    # allocation-free path
    th_b, v_b = theta0.clone(), torch.zeros(n, device=DEV)
    lp_b = torch.zeros(n, device=DEV, dtype=torch.bfloat16)
    bs_b = B.BucketSet([th_b], [grads], [v_b], [lp_b])
    sq_dev = torch.full((1,), -1.0, device=DEV, dtype=torch.float64)
    for call in range(2):
        ctx.aggregate_bsp(bs_a, b, 0.1, 0.9, 1e-4)
        sq_a = ctx.stats().grad_sqnorm
        B.aggregate_bsp_noalloc(bs_b, b, 0.1, 0.9, 1e-4, grad_sqnorm_out=sq_dev)
        torch.cuda.synchronize()
        np.testing.assert_allclose(to_np(th_b), to_np(th_a), **TOL[kind])
        np.testing.assert_allclose(to_np(v_b), to_np(v_a), **TOL[kind])
        assert np.array_equal(to_np(lp_b), to_np(lp_a))
        assert abs(float(sq_dev.item()) - sq_a) <= SQNORM_RTOL * sq_a, (call, float(sq_dev.item()), sq_a)
    assert sq_a > 0


def test_noalloc_rejects_what_it_cannot_hold():
    K = 2
    theta, grads = _inputs(K, 1024, "f32", 1)
    L = B.lib()
    tab = (C.c_void_p * K)(*[g.data_ptr() for g in grads])
    def bucket(n):
        return B.omni_bucket(theta.data_ptr(), None, None, C.cast(tab, C.POINTER(C.c_void_p)), n)
    b = (C.c_int32 * K)(3, 5)
    call = lambda arr, nb: L.omni_aggregate_bsp_noalloc(K, arr, nb, B.F32, b, 0, 0.1, 0.0, 0.0, None, None)
    before = to_np(theta)
    # more live buckets than the limit
    many = (B.omni_bucket * (B.NOALLOC_MAX_BUCKETS + 1))(*[bucket(16)] * (B.NOALLOC_MAX_BUCKETS + 1))
    assert call(many, B.NOALLOC_MAX_BUCKETS + 1) == B.ERR_TOO_LARGE
    # more elements than the limit (rejected on the size alone: nothing is launched)
    huge = (B.omni_bucket * 1)(bucket(B.NOALLOC_MAX_ELEMENTS + 1))
    assert call(huge, 1) == B.ERR_TOO_LARGE
    assert L.omni_aggregate_bsp_noalloc(0, huge, 1, B.F32, b, 0, 0.1, 0.0, 0.0, None, None) == B.ERR_BAD_K
    assert L.omni_aggregate_bsp_noalloc(K, huge, 1, B.F32, (C.c_int32 * K)(0, 5), 0, 0.1, 0.0, 0.0, None, None) == B.ERR_BAD_BATCH
    torch.cuda.synchronize()
    assert np.array_equal(to_np(theta), before)
    # empty buckets do not count against the limit
    ok = (B.omni_bucket * 10)(*([bucket(0)] * 9 + [bucket(1024)]))
    assert call(ok, 10) == B.OK
    torch.cuda.synchronize()
    assert not np.array_equal(to_np(theta), before)
