"""GPU parity of the bulk-copy (TMA + mbarrier ring) variant of the synchronous step, selected
with the OMNI_BULK_COPY flag: same bits as the oracle, hence as the register-staged kernels."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2503_17469_b200 import binding as B
from paper_2503_17469_b200 import workloads as W

from parity_util import SQNORM_RTOL, to_np
from test_gpu_parity import SIZES, _make, _random_batches

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("K", [1, 2, 3, 5, 8, 12, 16, 24, 32])
def test_bulk_copy_flat_parity_over_sizes(K, kind):
    """Sizes below one tile (all ragged), exactly on tile boundaries, and several tiles plus a
    ragged tail; momentum, weight decay and the low-precision copy on."""
    for n in SIZES + [4096, 8192, 5 * 4096 + 4, 300_007]:
        theta, v, grads, plp = _make(K, n, kind, 7000 * K + n % 991, lp=True)
        b = _random_batches(K, 32, K + n)
        o = B.Omni(K, 32 * K, 1, 32 * K, 0.1, flags=B.BULK_COPY)
        bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t], [plp.t])
        th_o, v_o = to_np(theta.t), to_np(v.t)
        lp_o = np.zeros(n, np.uint16)
        g_np = [to_np(g.t) for g in grads]
        for _ in range(2):
            o.aggregate_bsp(bs, b, 0.1, 0.9, 5e-4)
            sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 5e-4, theta_lp=lp_o)
            assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o + 1e-300
        assert np.array_equal(to_np(theta.t), th_o), (K, n)
        assert np.array_equal(to_np(v.t), v_o), (K, n)
        assert np.array_equal(to_np(plp.t), lp_o)
        for buf in (theta, v, plp, *grads):
            assert buf.intact(), "guard band overwritten"


@pytest.mark.parametrize("mu,wd,with_v", [(0.0, 0.0, False), (0.0, 0.0, True), (0.9, 0.0, True), (0.0, 1e-3, False)])
def test_bulk_copy_update_variants(mu, wd, with_v):
    K, n = 4, 50_001
    theta, v, grads, _ = _make(K, n, "bf16", 78, momentum=with_v)
    b = [3, 9, 20, 32]
    o = B.Omni(K, 64, 1, 64, 0.1, flags=B.BULK_COPY)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t] if with_v else None)
    th_o = to_np(theta.t)
    v_o = to_np(v.t) if with_v else None
    g_np = [to_np(g.t) for g in grads]
    for _ in range(2):
        o.aggregate_bsp(bs, b, 0.05, mu, wd)
        O.bsp_step_f32(g_np, b, th_o, v_o, 0.05, mu, wd)
    assert np.array_equal(to_np(theta.t), th_o)
    if with_v:
        assert np.array_equal(to_np(v.t), v_o)


def test_bulk_copy_sixteen_byte_alignment_and_many_buckets():
    """Buffers on 16-byte (not 32-byte) boundaries and 11 buckets of odd sizes (two launches)."""
    K = 5
    sizes = [0, 1, 4097, 20_000, 0, 8192, 33, 12_345, 65_536, 7, 40_001, 4096 * 3]
    o = B.Omni(K, 160, 1, 160, 0.1, flags=B.BULK_COPY)
    b = _random_batches(K, 32, 2)
    params, moms, gl, keep = [], [], [], []
    for i, n in enumerate(sizes):
        theta, v, grads, _ = _make(K, n + 8, "bf16", 900 + i)
        keep.append((theta, v, grads))
        params.append(theta.t[4:4 + n]); moms.append(v.t[4:4 + n]); gl.append([g.t[8:8 + n] for g in grads])
    bs = B.BucketSet(params, gl, moms)
    ref = [(to_np(p), to_np(m), [to_np(g) for g in gs]) for p, m, gs in zip(params, moms, gl)]
    o.aggregate_bsp(bs, b, 0.1, 0.9, 1e-4)
    sq = 0.0
    for (p, m, gs), (th_o, v_o, g_np), n in zip(zip(params, moms, gl), ref, sizes):
        if n:
            sq += O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 1e-4)
        assert np.array_equal(to_np(p), th_o) and np.array_equal(to_np(m), v_o)
    assert abs(o.stats().grad_sqnorm - sq) <= SQNORM_RTOL * sq
    for theta, v, grads in keep:
        assert theta.intact() and v.intact() and all(g.intact() for g in grads)


def test_bulk_copy_headline_config_full_size():
    cfg = W.config("resnet50_bf16")
    buf = W.make_buffers(cfg, DEV)
    o = B.Omni(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, flags=B.BULK_COPY)
    bs = B.BucketSet.from_flat(buf.layout, buf.theta, buf.grads, buf.v)
    gen = torch.Generator().manual_seed(cfg.seed)
    b, _ = o.rebatch(W.draw_throughputs(cfg.K, gen, cfg.ratio))
    th_o, v_o, g_np = to_np(buf.theta), to_np(buf.v), [to_np(g) for g in buf.grads]
    for _ in range(2):
        o.aggregate_bsp(bs, b, cfg.lr, cfg.momentum)
        sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, cfg.lr, cfg.momentum, 0.0)
    st = o.stats()
    assert abs(st.grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o
    assert np.array_equal(to_np(buf.theta), th_o) and np.array_equal(to_np(buf.v), v_o)


def test_bounded_wait_expiry_is_reported_and_the_context_stays_usable():
    """A wait that runs out sets the status word; omni_get_stats reports OMNI_ERR_TIMEOUT once,
    clears it, and the context keeps working (no trap, no hang, no lost context)."""
    K, n = 4, 30_000
    theta, v, grads, _ = _make(K, n, "bf16", 5)
    o = B.Omni(K, 64, 1, 64, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    b = [16] * K
    o.aggregate_bsp(bs, b, 0.1, 0.9)
    assert o.stats().steps == 1
    o.selftest_wait_expiry()
    with pytest.raises(B.OmniError) as e:
        o.stats()
    assert e.value.status == B.ERR_TIMEOUT
    st = o.stats()                       # reported once, then cleared
    assert st.steps == 1
    th_o, v_o, g_np = to_np(theta.t), to_np(v.t), [to_np(g.t) for g in grads]
    o.aggregate_bsp(bs, b, 0.1, 0.9)     # still usable, still correct
    sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 0.0)
    assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o
    assert np.array_equal(to_np(theta.t), th_o)


@pytest.mark.parametrize("kind,K", [("f32", 4), ("bf16", 7), ("bf16", 8)])
def test_short_launches_take_larger_tiles_with_the_same_bits(kind, K):
    """Launches of a few tiles per CTA run the ring in its short-launch shape (two stages of
    4096-element tiles where they fit: float K = 4, bfloat16 K = 7 and 8) when that halves the
    number of rounds.  Sizes inside that window (four regular rounds: a ragged tail, several
    buckets) and outside it (one, two, three and six rounds) give the oracle's bits either way."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for sizes in ([sms * 4096 + 77], [sms * 2048 * 4 - 5], [sms * 2048 + 3], [5 * sms * 2048 + 4099],
                  [300_001, 77, 450_003, 4096], [400_001, 77, 700_003, 4096]):
        bufs = [_make(K, n, kind, 4100 * K + n % 983, lp=True) for n in sizes]
        b = _random_batches(K, 32, K + sizes[0])
        o = B.Omni(K, 32 * K, 1, 32 * K, 0.1, flags=B.BULK_COPY)
        bs = B.BucketSet([x[0].t for x in bufs], [[g.t for g in x[2]] for x in bufs], [x[1].t for x in bufs],
                         [x[3].t for x in bufs])
        ora = [(to_np(x[0].t), to_np(x[1].t), np.zeros(n, np.uint16), [to_np(g.t) for g in x[2]]) for x, n in zip(bufs, sizes)]
        for _ in range(2):
            o.aggregate_bsp(bs, b, 0.1, 0.9, 5e-4)
            sq_o = sum(O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 5e-4, theta_lp=lp_o) for th_o, v_o, lp_o, g_np in ora)
            assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o
        for (theta, v, grads, plp), (th_o, v_o, lp_o, _) in zip(bufs, ora):
            assert np.array_equal(to_np(theta.t), th_o) and np.array_equal(to_np(v.t), v_o), (K, sizes)
            assert np.array_equal(to_np(plp.t), lp_o)
            for buf in (theta, v, plp, *grads):
                assert buf.intact(), "guard band overwritten"
