"""The allocation-free entry point against the regular one and against the CPU oracle.

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

from oracle import oracle as O
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
    # the CPU oracle on the same inputs: both entry points are the same ordered chain of
    # correctly rounded FMAs as the oracle's, so the bits must agree
    th_o, v_o, lp_o = to_np(theta0), np.zeros(n, np.float32), np.zeros(n, np.uint16)
    g_np = [to_np(g) for g in grads]
    for call in range(2):
        ctx.aggregate_bsp(bs_a, b, 0.1, 0.9, 1e-4)
        sq_a = ctx.stats().grad_sqnorm
        B.aggregate_bsp_noalloc(bs_b, b, 0.1, 0.9, 1e-4, grad_sqnorm_out=sq_dev)
        torch.cuda.synchronize()
        sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 1e-4, theta_lp=lp_o)
        np.testing.assert_allclose(to_np(th_b), to_np(th_a), **TOL[kind])
        np.testing.assert_allclose(to_np(v_b), to_np(v_a), **TOL[kind])
        assert np.array_equal(to_np(lp_b), to_np(lp_a))
        assert abs(float(sq_dev.item()) - sq_a) <= SQNORM_RTOL * sq_a, (call, float(sq_dev.item()), sq_a)
        assert np.array_equal(to_np(th_b), th_o) and np.array_equal(to_np(v_b), v_o), call
        assert np.array_equal(to_np(lp_b), lp_o), call
        assert abs(float(sq_dev.item()) - sq_o) <= SQNORM_RTOL * sq_o, (call, float(sq_dev.item()), sq_o)
    assert sq_a > 0


def _ragged_buckets(K, kind, sizes, seed, shift):
    """Several buckets of ragged sizes cut out of flat buffers; with ``shift`` every buffer starts
    16 bytes past a 32-byte boundary, which sends the call to the 128-bit instantiation."""
    gdt = torch.bfloat16 if kind == "bf16" else torch.float32
    gen = torch.Generator(device=DEV).manual_seed(seed)
    pad = lambda m: (m + 63) // 64 * 64
    total = sum(pad(m) for m in sizes) + 64
    theta = torch.empty(total, device=DEV).normal_(0, 0.05, generator=gen)
    v = torch.empty(total, device=DEV).normal_(0, 1e-3, generator=gen)
    lp = torch.zeros(total, device=DEV, dtype=torch.bfloat16)
    grads = [torch.empty(total, device=DEV).normal_(0, 1e-3, generator=gen).to(gdt) for _ in range(K)]
    off = lambda t: (16 // t.element_size()) if shift else 0
    views, start = [], 0
    for m in sizes:
        cut = lambda t: t[start + off(t):start + off(t) + m]
        views.append((cut(theta), cut(v), cut(lp), [cut(g) for g in grads]))
        start += pad(m)
    want = 16 if shift else 0
    assert all(t.data_ptr() % 32 == want for vw in views for t in (vw[0], vw[1], vw[2], *vw[3]))
    return views


@pytest.mark.parametrize("kind,K", [("f32", 5), ("bf16", 16), ("f32", 32)])
@pytest.mark.parametrize("shift", [False, True], ids=["aligned32", "aligned16"])
def test_noalloc_ragged_buckets_both_vector_widths_against_oracle(kind, K, shift):
    """Three to eight ragged buckets in one call (their tiles are numbered across buckets), with
    32-byte and with only 16-byte aligned buffers, bit for bit against the oracle, squared norm
    included; then a small call after the large one, whose norm must not see the partial sums the
    large call left in the shared array; the unweighted-mean flag; and momentum 0 with a momentum
    buffer present (v is then overwritten by the aggregate)."""
    sizes = [1, 4099, 3 * 8192 + 5, 70_001, 17, 12_288, 250_003, 33][: 3 + K % 6]
    views = _ragged_buckets(K, kind, sizes, 99 + K, shift)
    b = [int(x) for x in np.random.default_rng(7 * K).integers(1, 97, K)]
    bs = B.BucketSet([vw[0] for vw in views], [vw[3] for vw in views], [vw[1] for vw in views], [vw[2] for vw in views])
    ora = [(to_np(vw[0]), to_np(vw[1]), np.zeros(vw[0].numel(), np.uint16), [to_np(g) for g in vw[3]]) for vw in views]
    sq_dev = torch.full((1,), -1.0, device=DEV, dtype=torch.float64)

    def check(flags, mu, wd, tag):
        B.aggregate_bsp_noalloc(bs, b, 0.05, mu, wd, flags=flags, grad_sqnorm_out=sq_dev)
        torch.cuda.synchronize()
        sq_o = 0.0
        for vw, (th_o, v_o, lp_o, g_np) in zip(views, ora):
            sq_o += O.bsp_step_f32(g_np, b, th_o, v_o, 0.05, mu, wd, flags=flags, theta_lp=lp_o)
            assert np.array_equal(to_np(vw[0]), th_o), tag
            assert np.array_equal(to_np(vw[1]), v_o), tag
            assert np.array_equal(to_np(vw[2]), lp_o), tag
        assert abs(float(sq_dev.item()) - sq_o) <= SQNORM_RTOL * sq_o, (tag, float(sq_dev.item()), sq_o)

    check(0, 0.9, 1e-4, "weighted")
    check(B.UNSCALED_MEAN, 0.9, 0.0, "unweighted mean")
    check(0, 0.0, 0.0, "momentum 0 with a buffer")
    # a small call right after the large ones: one bucket of 77 elements
    vw = max(views, key=lambda x: x[0].numel())
    th_s, v_s, g_s = vw[0][:77], vw[1][:77], [g[:77] for g in vw[3]]
    bs_s = B.BucketSet([th_s], [g_s], [v_s])
    th_o, v_o, g_np = to_np(th_s), to_np(v_s), [to_np(g) for g in g_s]
    B.aggregate_bsp_noalloc(bs_s, b, 0.05, 0.9, 0.0, grad_sqnorm_out=sq_dev)
    torch.cuda.synchronize()
    sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.05, 0.9, 0.0)
    assert np.array_equal(to_np(th_s), th_o) and np.array_equal(to_np(v_s), v_o)
    assert abs(float(sq_dev.item()) - sq_o) <= SQNORM_RTOL * sq_o


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
    # flag bits that mean nothing to this call are refused, not ignored
    one = (B.omni_bucket * 1)(bucket(1024))
    assert L.omni_aggregate_bsp_noalloc(K, one, 1, B.F32, b, B.ASP_NO_LR_SCALE, 0.1, 0.0, 0.0, None, None) == B.ERR_BAD_CONFIG
    torch.cuda.synchronize()
    assert np.array_equal(to_np(theta), before)
    # empty buckets do not count against the limit
    ok = (B.omni_bucket * 10)(*([bucket(0)] * 9 + [bucket(1024)]))
    assert call(ok, 10) == B.OK
    torch.cuda.synchronize()
    assert not np.array_equal(to_np(theta), before)
