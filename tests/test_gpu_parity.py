"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle, element by
element on the same seeded inputs."""
import ctypes as C
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2503_17469_b200 import binding as B
from paper_2503_17469_b200 import workloads as W

from parity_util import Guarded, SQNORM_RTOL, assert_close, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(autouse=True, params=["auto", "registers", "bulk"])
def kernel_family(request):
    """Every test of this module runs once per kernel family: the library's own choice, the
    register-staged kernels forced, the bulk-copy ring forced."""
    old = B.DEFAULT_FLAGS
    B.DEFAULT_FLAGS = {"auto": 0, "registers": B.NO_BULK_COPY, "bulk": B.BULK_COPY}[request.param]
    yield
    B.DEFAULT_FLAGS = old


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


def _make(K, n, kind, seed, lp=False, momentum=True, gstd=1e-3):
    gen = _gen(seed)
    gdt = torch.bfloat16 if kind == "bf16" else torch.float32
    theta = Guarded(n, torch.float32, DEV, torch.empty(n, device=DEV).normal_(0, 0.05, generator=gen))
    v = Guarded(n, torch.float32, DEV, torch.zeros(n, device=DEV)) if momentum else None
    grads = [Guarded(n, gdt, DEV, torch.empty(n, device=DEV).normal_(0, gstd, generator=gen).to(gdt)) for _ in range(K)]
    plp = Guarded(n, torch.bfloat16, DEV, torch.zeros(n, device=DEV, dtype=torch.bfloat16)) if lp else None
    return theta, v, grads, plp


def _random_batches(K, per, seed):
    rng = np.random.default_rng(seed)
    if K == 1:
        return [per]
    cuts = np.sort(rng.choice(np.arange(1, K * per), K - 1, replace=False))
    b = np.diff(np.concatenate([[0], cuts, [K * per]]))
    return [int(x) for x in b]


SIZES = [1, 3, 7, 1023, 4095, 4097, 3 * 8192 + 17, 100_003]


@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 8, 11, 16, 17, 32])
def test_bsp_flat_parity_over_sizes(K, kind):
    """Several tiles plus a ragged tail, three steps each, momentum + weight decay + low-precision copy."""
    bit_equal = []
    for n in SIZES:
        theta, v, grads, plp = _make(K, n, kind, 1000 * K + n % 997, lp=True)
        b = _random_batches(K, 32, K + n)
        o = B.Omni(K, 32 * K, 1, 32 * K, 0.1)
        bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t], [plp.t])
        th_o, v_o = to_np(theta.t), to_np(v.t)
        lp_o = np.zeros(n, np.uint16)
        g_np = [to_np(g.t) for g in grads]
        for step in range(3):
            o.aggregate_bsp(bs, b, 0.1, 0.9, 5e-4)
            sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 5e-4, theta_lp=lp_o)
            st = o.stats()
            assert abs(st.grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o + 1e-300
            assert st.steps == step + 1
        bit_equal.append(assert_close(to_np(theta.t), th_o, kind, f"theta K={K} n={n}"))
        bit_equal.append(assert_close(to_np(v.t), v_o, kind, f"v K={K} n={n}"))
        assert np.array_equal(to_np(plp.t), lp_o)
        for buf in (theta, v, plp, *grads):
            assert buf.intact(), "guard band overwritten"
        for g, g0 in zip(grads, g_np):
            assert np.array_equal(to_np(g.t), g0), "gradient buffer modified"
    # both sides are the same ordered chain of correctly rounded FMAs
    assert min(bit_equal) == 1.0


@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("mu,wd,with_v", [(0.0, 0.0, False), (0.0, 0.0, True), (0.9, 0.0, True), (0.0, 1e-3, False)])
def test_bsp_update_variants(kind, mu, wd, with_v):
    K, n = 4, 50_001
    theta, v, grads, _ = _make(K, n, kind, 77, momentum=with_v)
    b = [3, 9, 20, 32]
    o = B.Omni(K, 64, 1, 64, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t] if with_v else None)
    th_o = to_np(theta.t)
    v_o = to_np(v.t) if with_v else None
    g_np = [to_np(g.t) for g in grads]
    for _ in range(2):
        o.aggregate_bsp(bs, b, 0.05, mu, wd)
        O.bsp_step_f32(g_np, b, th_o, v_o, 0.05, mu, wd)
    assert assert_close(to_np(theta.t), th_o, kind) == 1.0
    if with_v:
        assert assert_close(to_np(v.t), v_o, kind) == 1.0


def test_bsp_against_double_definition():
    """Ten steps against the double-precision oracle at the contract tolerance."""
    K, n = 16, 200_003
    theta, v, grads, _ = _make(K, n, "f32", 5)
    b = _random_batches(K, 32, 5)
    o = B.Omni(K, 512, 1, 512, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    th64, v64 = to_np(theta.t).astype(np.float64), np.zeros(n)
    g_np = [to_np(g.t) for g in grads]
    for _ in range(10):
        o.aggregate_bsp(bs, b, 0.1, 0.9, 0.0)
        sq64 = O.bsp_step_f64(g_np, b, th64, v64, 0.1, 0.9, 0.0)
    np.testing.assert_allclose(to_np(theta.t), th64, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(to_np(v.t), v64, rtol=1e-5, atol=1e-8)
    assert abs(o.stats().grad_sqnorm - sq64) <= SQNORM_RTOL * sq64


def test_unscaled_mean_flag_and_equal_batches():
    K, n = 8, 30_000
    theta, v, grads, _ = _make(K, n, "f32", 9)
    g_np = [to_np(g.t) for g in grads]
    th0 = to_np(theta.t)
    o = B.Omni(K, 256, 1, 256, 0.1, flags=B.UNSCALED_MEAN)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    b = _random_batches(K, 32, 9)
    o.aggregate_bsp(bs, b, 1.0, 0.0, 0.0)
    th_o = th0.copy()
    O.bsp_step_f32(g_np, b, th_o, None, 1.0, 0.0, 0.0, flags=O.FLAG_UNSCALED_MEAN)
    assert np.array_equal(to_np(theta.t), th_o)
    # equal batches without the flag give the same bits (lambda = 1/8 exactly)
    theta.t.copy_(torch.from_numpy(th0))
    o2 = B.Omni(K, 256, 1, 256, 0.1)
    o2.aggregate_bsp(bs, [32] * K, 1.0, 0.0, 0.0)
    assert np.array_equal(to_np(theta.t), th_o)
    assert o2.stats().weight_sum == 1.0


@pytest.mark.parametrize("kind", ["f32", "bf16"])
def test_bsp_many_buckets_empty_and_ragged(kind):
    """23 buckets (several launches of at most 8 non-empty ones), some empty, odd sizes, mixed lp."""
    K = 5
    rng = np.random.default_rng(3)
    sizes = [int(x) for x in rng.choice([0, 1, 5, 300, 2048, 6144, 10_007, 40_001], 23)]
    sizes[0], sizes[7], sizes[22] = 0, 0, 12_345
    o = B.Omni(K, 160, 1, 160, 0.1)
    b = _random_batches(K, 32, 1)
    bufs, params, moms, lps, gl = [], [], [], [], []
    for i, n in enumerate(sizes):
        theta, v, grads, plp = _make(K, max(n, 1), kind, 500 + i, lp=(i % 2 == 0))
        bufs.append((theta, v, grads, plp, n))
        params.append(theta.t[:n]); moms.append(v.t[:n]); gl.append([g.t[:n] for g in grads])
        lps.append(plp.t[:n] if plp is not None else None)
    bs = B.BucketSet(params, gl, moms, lps)
    oracle_state = [(to_np(p), to_np(m), [to_np(g) for g in gs]) for p, m, gs in zip(params, moms, gl)]
    before = o.kernel_launches
    o.aggregate_bsp(bs, b, 0.1, 0.9, 1e-4)
    assert o.kernel_launches - before == math.ceil(sum(1 for n in sizes if n) / 8) >= 2
    sq_total = 0.0
    for (theta, v, grads, plp, n), (th_o, v_o, g_np) in zip(bufs, oracle_state):
        lp_o = np.zeros(n, np.uint16)
        if n:
            sq_total += O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 1e-4, theta_lp=lp_o)
        assert np.array_equal(to_np(theta.t[:n]), th_o) and np.array_equal(to_np(v.t[:n]), v_o)
        if plp is not None:
            assert np.array_equal(to_np(plp.t[:n]), lp_o)
        assert theta.intact() and v.intact() and (plp is None or plp.intact())
        if n == 0:   # an empty bucket leaves its storage alone
            assert float(v.t[0]) == 0.0
    assert abs(o.stats().grad_sqnorm - sq_total) <= SQNORM_RTOL * sq_total


@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("K", [1, 4, 16, 32])
def test_buffers_aligned_to_16_bytes_only(K, kind):
    """Buffers that sit on a 16-byte but not a 32-byte boundary take the 128-bit kernels; one
    misaligned buffer among aligned ones is enough.  Same results as the oracle, bit for bit."""
    n = 5 * 8192 + 29
    for which in ("all", "one_grad", "theta"):
        theta, v, grads, plp = _make(K, n + 8, kind, 31 * K, lp=True)
        sh = lambda buf, on: buf.t[(8 if buf.dtype == torch.bfloat16 else 4):][:n] if on else buf.t[:n]
        th_t = sh(theta, which in ("all", "theta"))
        v_t = sh(v, which == "all")
        lp_t = sh(plp, which == "all")
        g_t = [sh(g, which == "all" or (which == "one_grad" and k == K - 1)) for k, g in enumerate(grads)]
        assert th_t.data_ptr() % 32 == (16 if which != "one_grad" else 0)
        b = _random_batches(K, 32, K)
        o = B.Omni(K, 32 * K, 1, 32 * K, 0.1)
        bs = B.BucketSet([th_t], [g_t], [v_t], [lp_t])
        th_o, v_o, g_np = to_np(th_t), to_np(v_t), [to_np(g) for g in g_t]
        lp_o = np.zeros(n, np.uint16)
        for _ in range(2):
            o.aggregate_bsp(bs, b, 0.1, 0.9, 1e-4)
            sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 1e-4, theta_lp=lp_o)
        assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o
        assert np.array_equal(to_np(th_t), th_o) and np.array_equal(to_np(v_t), v_o)
        assert np.array_equal(to_np(lp_t), lp_o)
        a = B.Omni(K, 32 * K, 1, 32 * K, 0.1, 1.0, B.ASP)
        a.apply_asp(bs, K - 1, 17, 2, 0.1, 0.9, 1e-4)
        O.asp_apply_f32(g_np[K - 1], 17, 32 * K, th_o, v_o, 0.1, 0.9, 1e-4, theta_lp=lp_o)
        assert np.array_equal(to_np(th_t), th_o) and np.array_equal(to_np(v_t), v_o)
        assert np.array_equal(to_np(lp_t), lp_o)
        for buf in (theta, v, plp, *grads):
            assert buf.intact()


def test_empty_call_reads_zero_norm():
    o = B.Omni(2, 64, 4, 96, 0.1)
    theta, v, grads, _ = _make(2, 1000, "f32", 1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    o.aggregate_bsp(bs, [32, 32], 0.1, 0.9)
    assert o.stats().grad_sqnorm > 0
    empty = B.BucketSet([], [])
    empty.K, empty.dtype = 2, B.F32
    o.aggregate_bsp(empty, [32, 32], 0.1, 0.9)
    assert o.stats().grad_sqnorm == 0.0


def test_results_are_deterministic():
    K, n = 16, 1_000_003
    outs = []
    for rep in range(2):
        theta, v, grads, _ = _make(K, n, "bf16", 42)
        o = B.Omni(K, 512, 1, 512, 0.1)
        bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
        for _ in range(3):
            o.aggregate_bsp(bs, _random_batches(K, 32, 4), 0.1, 0.9)
        outs.append((to_np(theta.t), o.stats().grad_sqnorm))
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]


@pytest.mark.parametrize("kind", ["f32", "bf16"])
def test_one_call_step_is_aggregate_then_rebatch(kind):
    """omni_step_bsp over twelve iterations with jittered throughputs: each iteration aggregates
    with the batches of the previous re-batch (the ones the gradients were computed with), then
    re-batches; parameters, momentum, norms and batches equal the oracle's and the two-call
    sequence's."""
    K, n = 8, 3 * 8192 + 29
    theta, v, grads, _ = _make(K, n, kind, 1234)
    o = B.Omni(K, 256, 4, 96, 0.1)
    two = B.Omni(K, 256, 4, 96, 0.1)
    ora = O.Controller(K, 256, 4, 96, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    th2, v2 = theta.t.clone(), v.t.clone()
    bs2 = B.BucketSet([th2], [[g.t for g in grads]], [v2])
    th_o, v_o, g_np = to_np(theta.t), to_np(v.t), [to_np(g.t) for g in grads]
    rng = np.random.default_rng(3)
    base = 8.0 ** rng.random(K)
    for it in range(12):
        T = base * (1.0 + 0.2 * (2.0 * rng.random(K) - 1.0))
        used = ora.batches.copy()
        nxt = o.step_bsp(bs, T.tolist(), 0.1, 0.9, 1e-4)
        two.aggregate_bsp(bs2, two.batches, 0.1, 0.9, 1e-4)
        nxt2, _ = two.rebatch(T.tolist())
        sq_o = O.bsp_step_f32(g_np, used, th_o, v_o, 0.1, 0.9, 1e-4)
        want, _ = ora.rebatch(T)
        assert nxt == nxt2 == want.tolist() == o.batches
        st = o.stats()
        assert abs(st.grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o and st.steps == it + 1
    assert np.array_equal(to_np(theta.t), th_o) and np.array_equal(to_np(v.t), v_o)
    assert np.array_equal(to_np(th2), th_o) and np.array_equal(to_np(v2), v_o)


def test_two_contexts_on_two_streams_at_once():
    """Two models stepped concurrently, each through its own context on its own stream (each
    context has its own workspace, so the launches may overlap on the GPU): both end up with the
    oracle's bits and their own squared norms."""
    jobs = []
    for j, (K, n, kind) in enumerate([(4, 700_001, "f32"), (16, 300_007, "bf16")]):
        theta, v, grads, _ = _make(K, n, kind, 900 + j)
        o = B.Omni(K, 32 * K, 1, 32 * K, 0.1)
        bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
        jobs.append(dict(o=o, bs=bs, theta=theta, v=v, b=_random_batches(K, 32, 70 + j), stream=torch.cuda.Stream(),
                         th_o=to_np(theta.t), v_o=to_np(v.t), g_np=[to_np(g.t) for g in grads]))
    torch.cuda.synchronize()
    for step in range(6):
        for jb in jobs:                                   # interleaved enqueues, no synchronisation in between
            jb["o"].aggregate_bsp(jb["bs"], jb["b"], 0.1, 0.9, 1e-4, stream=jb["stream"])
    for jb in jobs:
        jb["stream"].synchronize()
        for step in range(6):
            sq_o = O.bsp_step_f32(jb["g_np"], jb["b"], jb["th_o"], jb["v_o"], 0.1, 0.9, 1e-4)
        assert np.array_equal(to_np(jb["theta"].t), jb["th_o"]) and np.array_equal(to_np(jb["v"].t), jb["v_o"])
        assert abs(jb["o"].stats(stream=jb["stream"]).grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o


def test_steps_replayed_from_a_cuda_graph():
    """Ten steps captured once into a CUDA graph (after one eager call, which binds the context
    to the device and sizes its launches) and replayed twice: the same bits as thirty eager
    steps of the oracle, and the norm of the last step."""
    K, n = 4, 1 << 18
    theta, v, grads, _ = _make(K, n, "f32", 321)
    o = B.Omni(K, 64, 2, 48, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    b = [2, 6, 19, 37]
    th_o, v_o, g_np = to_np(theta.t), to_np(v.t), [to_np(g.t) for g in grads]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(10):                      # eager warm-up on the capture stream
            o.aggregate_bsp(bs, b, 0.1, 0.9)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(10):
            o.aggregate_bsp(bs, b, 0.1, 0.9)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    for _ in range(30):
        sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 0.0)
    assert np.array_equal(to_np(theta.t), th_o) and np.array_equal(to_np(v.t), v_o)
    assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o


def test_ordinary_kernels_between_steps_see_finished_steps():
    """The ring kernels signal early that dependents may launch; a kernel enqueued after a step in
    the ordinary way (here: torch copies, eagerly and inside a captured graph) must still see the
    step's finished theta and v, and a step that follows such a kernel must see its writes (the
    gradient is rewritten between the steps)."""
    K, n = 3, 5 * 8192 + 11
    theta, v, grads, _ = _make(K, n, "f32", 654)
    alt = [g.t.clone().mul_(-0.5) for g in grads]            # a second set of gradients to switch to
    first = [g.t.clone() for g in grads]
    o = B.Omni(K, 48, 1, 48, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    b = [5, 16, 27]
    snaps = [torch.empty(n, device=DEV) for _ in range(4)]

    def sequence():
        for i in range(4):
            src = first if i % 2 == 0 else alt
            for g, s_ in zip(grads, src):
                g.t.copy_(s_)                                    # ordinary kernels before the step ...
            o.aggregate_bsp(bs, b, 0.1, 0.9)
            snaps[i].copy_(theta.t)                              # ... and right after it

    th_o, v_o = to_np(theta.t), to_np(v.t)
    g_sets = [[to_np(x) for x in first], [to_np(x) for x in alt]]
    want = []
    for rep in range(3):                                         # one eager pass, two graph replays
        for i in range(4):
            O.bsp_step_f32(g_sets[i % 2], b, th_o, v_o, 0.1, 0.9, 0.0)
            want.append(th_o.copy())
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        sequence()
    side.synchronize()
    for i in range(4):
        assert np.array_equal(to_np(snaps[i]), want[i]), i
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        sequence()
    for rep in (1, 2):
        graph.replay()
        torch.cuda.synchronize()
        for i in range(4):
            assert np.array_equal(to_np(snaps[i]), want[4 * rep + i]), (rep, i)
    assert np.array_equal(to_np(theta.t), th_o) and np.array_equal(to_np(v.t), v_o)


def test_host_gradient_entry_point():
    K, n = 4, 70_001
    theta, v, grads, _ = _make(K, n, "bf16", 11)
    host = [[g.t.cpu().pin_memory() for g in grads]]
    g_np = [to_np(g.t) for g in grads]
    for g in grads:
        g.t.zero_()                      # staging buffers: the call must fill them
    th_o, v_o = to_np(theta.t), to_np(v.t)
    o = B.Omni(K, 128, 4, 96, 0.1)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t])
    b = [10, 20, 30, 68]
    sq = o.aggregate_bsp_host(bs, host, b, 0.1, 0.9)
    sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, 0.1, 0.9, 0.0)
    assert abs(sq - sq_o) <= SQNORM_RTOL * sq_o
    assert np.array_equal(to_np(theta.t), th_o) and np.array_equal(to_np(v.t), v_o)


# ------------------------------------------------------------------------------------------------
# asynchronous arrivals
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("mu,wd", [(0.0, 0.0), (0.9, 1e-4)])
def test_asp_parity_over_sizes(kind, mu, wd):
    K = 3
    for n in SIZES + [4 * 8192 * 3 + 5]:
        theta, v, grads, plp = _make(K, n, kind, 2000 + n % 991, lp=True, momentum=mu != 0)
        o = B.Omni(K, 96, 4, 96, 0.1, 1.0, B.ASP)
        bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t] if v else None, [plp.t])
        th_o = to_np(theta.t)
        v_o = to_np(v.t) if v else None
        lp_o = np.zeros(n, np.uint16)
        g_np = [to_np(g.t) for g in grads]
        taus = []
        for i, (k, b_used, tau) in enumerate([(0, 32, 0), (2, 7, 3), (1, 96, 40), (2, 33, 1)]):
            o.apply_asp(bs, k, b_used, tau, 0.1, mu, wd)
            O.asp_apply_f32(g_np[k], b_used, 96, th_o, v_o, 0.1, mu, wd, theta_lp=lp_o)
            taus.append(tau)
        assert assert_close(to_np(theta.t), th_o, kind, f"n={n}") == 1.0
        if v:
            assert assert_close(to_np(v.t), v_o, kind) == 1.0
        assert np.array_equal(to_np(plp.t), lp_o)
        assert theta.intact() and plp.intact() and all(g.intact() for g in grads)
        st = o.stats()
        ref = O.TauStats()
        for t in taus:
            ref.record(t)
        assert st.arrivals == 4 and st.tau_hist == ref.hist.tolist() and st.tau_max == ref.tau_max


@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("mu,wd", [(0.0, 0.0), (0.9, 1e-4)])
def test_asp_batched_apply_equals_successive_arrivals(kind, mu, wd):
    """m queued arrivals in one pass give the bits of m single-arrival updates in that order
    (oracle: m successive applications of the per-arrival rule), for several m and ragged sizes."""
    K = 6
    rng = np.random.default_rng(17)
    for m, n in [(1, 4097), (2, 100_003), (3, 7), (5, 3 * 8192 + 17), (16, 60_001)]:
        theta, v, grads, plp = _make(K, n, kind, 3000 + m, lp=True, momentum=mu != 0)
        o = B.Omni(K, 192, 4, 96, 0.1, 1.0, B.ASP)
        bs = B.BucketSet([theta.t], [[g.t for g in grads]], [v.t] if v else None, [plp.t])
        workers = [int(x) for x in rng.integers(0, K, m)]
        b_used = [int(x) for x in rng.integers(4, 97, m)]
        taus = [int(x) for x in rng.integers(0, 50, m)]
        th_o = to_np(theta.t)
        v_o = to_np(v.t) if v else None
        lp_o = np.zeros(n, np.uint16)
        g_np = [to_np(g.t) for g in grads]
        o.apply_asp_batch(bs, workers, b_used, taus, 0.1, mu, wd)
        ref = O.TauStats()
        for k, bu, tau in zip(workers, b_used, taus):
            O.asp_apply_f32(g_np[k], bu, 192, th_o, v_o, 0.1, mu, wd, theta_lp=lp_o)
            ref.record(tau)
        assert np.array_equal(to_np(theta.t), th_o), (m, n)
        if v:
            assert np.array_equal(to_np(v.t), v_o)
        assert np.array_equal(to_np(plp.t), lp_o)
        st = o.stats()
        assert st.arrivals == m and st.tau_hist == ref.hist.tolist() and st.tau_max == ref.tau_max
        assert theta.intact() and plp.intact() and all(g.intact() for g in grads)
    L, h = B.lib(), o._h
    i32 = lambda *a: (C.c_int32 * len(a))(*a)
    assert L.omni_apply_asp_batch(h, bs.array, 1, bs.dtype, 17, i32(*[0] * 17), i32(*[8] * 17), i32(*[0] * 17), 0.1, mu, wd, None) == B.ERR_TOO_LARGE
    assert L.omni_apply_asp_batch(h, bs.array, 1, bs.dtype, 2, i32(0, K), i32(8, 8), i32(0, 0), 0.1, mu, wd, None) == B.ERR_BAD_WORKER
    assert L.omni_apply_asp_batch(h, bs.array, 1, bs.dtype, 2, i32(0, 1), i32(8, 0), i32(0, 0), 0.1, mu, wd, None) == B.ERR_BAD_BATCH
    assert L.omni_apply_asp_batch(h, bs.array, 1, bs.dtype, 2, i32(0, 1), i32(8, 8), i32(0, -1), 0.1, mu, wd, None) == B.ERR_BAD_TAU


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("kind", ["f32", "bf16"])
def test_asp_pull_and_push_with_overwrite(kind, fused):
    """Algorithm 2 literally on a shrunk model: workers pull snapshots at different times and
    push with overwrite; the event stream (with controller feedback) runs on both sides; the
    server copy matches the oracle bit for bit after every event, and differs from what applying
    the same gradients would give.  fused: the push and the worker's next pull in one call."""
    base = W.config("resnet50_asp")
    cfg = W.scaled(W.Config(**{**base.__dict__, "grad_dtype": kind}), 500)
    buf = W.make_buffers(cfg, DEV)
    lay = buf.layout
    K = cfg.K
    o = B.Omni(K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, 1.0, B.ASP)
    ora = O.Controller(K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, 1.0, O.MODE_ASP)
    lp = torch.zeros(lay.total, dtype=torch.bfloat16, device=DEV)
    bs = B.BucketSet.from_flat(lay, buf.theta, buf.grads, None, lp)
    sl = [slice(bk.start, bk.start + bk.n) for bk in lay.buckets]
    snaps = [torch.zeros(lay.total, device=DEV) for _ in range(K)]           # one snapshot set per worker
    th_o = to_np(buf.theta)
    lp_o = np.zeros(lay.total, np.uint16)
    snaps_o = [np.zeros(lay.total, np.float32) for _ in range(K)]
    applied = th_o.copy()
    g_np = [to_np(g) for g in buf.grads]
    for k in range(K):                                                        # everybody pulls theta_0
        o.asp_pull(bs, [snaps[k][s] for s in sl])
        snaps_o[k][:] = th_o
    gen = torch.Generator().manual_seed(cfg.seed)
    T = W.draw_throughputs(K, gen, cfg.ratio)
    u = torch.rand(300, generator=gen, dtype=torch.float64).tolist()
    b = [cfg.global_batch // K] * K
    last = [0] * K
    tally = O.TauStats()
    for i in range(300):
        k = W.pick_worker(u[i], [T[j] / b[j] for j in range(K)])
        tau = i - last[k]
        if fused:
            o.asp_push_pull(bs, k, b[k], tau, [snaps[k][s] for s in sl], cfg.lr, 1e-4)
        else:
            o.asp_push_overwrite(bs, k, b[k], tau, [snaps[k][s] for s in sl], cfg.lr, 1e-4)
            o.asp_pull(bs, [snaps[k][s] for s in sl])                         # next iteration starts with a pull
        for s in sl:                                                          # the oracle walks the same buckets
            O.asp_push_overwrite_f32(g_np[k][s], b[k], cfg.global_batch, th_o[s], snaps_o[k][s], cfg.lr, 1e-4, theta_lp=lp_o[s])
        snaps_o[k][:] = th_o
        O.asp_apply_f32(g_np[k], b[k], cfg.global_batch, applied, None, cfg.lr, 0.0, 1e-4)
        tally.record(tau)
        last[k] = i + 1
        nb = o.asp_report(k, b[k], T[k])
        assert nb == ora.asp_report(k, b[k], T[k])
        b[k] = nb
        if i % 50 == 0 or i == 299:
            assert np.array_equal(to_np(buf.theta), th_o), i
    assert np.array_equal(to_np(lp), lp_o)
    for k in range(K):
        for s_ in sl:
            assert np.array_equal(to_np(snaps[k][s_]), snaps_o[k][s_]), k
    st = o.stats()
    assert st.arrivals == 300 and st.tau_hist == tally.hist.tolist() and st.tau_max == tally.tau_max
    real = np.concatenate([np.arange(a, a + n) for _, a, n in lay.tensor_slices()])
    assert np.abs(th_o[real] - applied[real]).max() > 1e-5      # overwriting loses updates that applying keeps


def test_asp_no_lr_scale_flag():
    n = 10_000
    theta, _, grads, _ = _make(2, n, "f32", 8, momentum=False)
    o = B.Omni(2, 64, 4, 96, 0.1, 1.0, B.ASP, B.ASP_NO_LR_SCALE)
    bs = B.BucketSet([theta.t], [[g.t for g in grads]])
    th_o = to_np(theta.t)
    o.apply_asp(bs, 1, 8, 0, 0.1)
    O.asp_apply_f32(to_np(grads[1].t), 8, 64, th_o, None, 0.1, 0.0, 0.0, flags=O.FLAG_ASP_NO_LR_SCALE)
    assert np.array_equal(to_np(theta.t), th_o)


def _asp_stream(cfg, n_events, apply_fn, report_fn, seed):
    """Throughput-weighted arrival stream with controller feedback (the workload recipe):
    worker drawn with probability proportional to its iteration rate T_k / b_k; staleness =
    server updates since that worker's previous arrival."""
    gen = torch.Generator().manual_seed(seed)
    T = W.draw_throughputs(cfg.K, gen, cfg.ratio)
    u = torch.rand(n_events, generator=gen, dtype=torch.float64).tolist()
    b = [cfg.global_batch // cfg.K] * cfg.K
    last = [0] * cfg.K
    trace = []
    for i in range(n_events):
        k = W.pick_worker(u[i], [T[j] / b[j] for j in range(cfg.K)])
        tau = min(i - last[k], 10**6)
        apply_fn(k, b[k], tau)
        last[k] = i + 1
        b[k] = report_fn(k, b[k], T[k])
        trace.append((k, tau, b[k]))
    return trace


def test_asp_event_stream_with_controller_feedback():
    """The asynchronous configuration on a shrunk model: 1000 arrivals, every arrival applied
    and reported on both sides; batches and staleness tallies bit-exact, parameters at tolerance."""
    cfg = W.scaled(W.config("resnet50_asp"), 600)
    buf = W.make_buffers(cfg, DEV)
    o = B.Omni(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, cfg.ewma_alpha, B.ASP)
    bs = B.BucketSet.from_flat(buf.layout, buf.theta, buf.grads)
    ora = O.Controller(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, cfg.ewma_alpha, O.MODE_ASP)
    th_o = to_np(buf.theta)
    g_np = [to_np(g) for g in buf.grads]
    tally = O.TauStats()

    def ora_apply(k, b_used, tau):
        O.asp_apply_f32(g_np[k], b_used, cfg.global_batch, th_o, None, cfg.lr, 0.0, 0.0)
        tally.record(tau)

    t_lib = _asp_stream(cfg, 1000, lambda k, bu, tau: o.apply_asp(bs, k, bu, tau, cfg.lr), o.asp_report, cfg.seed)
    t_ora = _asp_stream(cfg, 1000, ora_apply, ora.asp_report, cfg.seed)
    assert t_lib == t_ora
    st = o.stats()
    assert st.arrivals == 1000 and st.tau_hist == tally.hist.tolist() and st.tau_max == tally.tau_max
    assert st.tau_sum == sum(tau for _, tau, _ in t_lib) and st.tau_mean == st.tau_sum / 1000
    assert o.batches == ora.batches.tolist()
    assert assert_close(to_np(buf.theta), th_o, "f32") == 1.0


# ------------------------------------------------------------------------------------------------
# the synthetic configurations
# ------------------------------------------------------------------------------------------------

def test_tiny_config_every_step():
    """K=4, 2^20 parameters: one re-batch (expected (2,6,19,37)) then 10 steps, parity at every step."""
    cfg = W.config("tiny")
    buf = W.make_buffers(cfg, DEV)
    o = B.Omni(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband)
    ora = O.Controller(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband)
    b, _ = o.rebatch(cfg.throughputs)
    assert b == ora.rebatch(cfg.throughputs)[0].tolist() == [2, 6, 19, 37]
    bs = B.BucketSet.from_flat(buf.layout, buf.theta, buf.grads, buf.v)
    th_o, v_o, g_np = to_np(buf.theta), to_np(buf.v), [to_np(g) for g in buf.grads]
    for step in range(cfg.steps):
        o.aggregate_bsp(bs, b, cfg.lr, cfg.momentum)
        sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, cfg.lr, cfg.momentum, 0.0)
        assert assert_close(to_np(buf.theta), th_o, "f32", f"step {step}") == 1.0
        assert assert_close(to_np(buf.v), v_o, "f32", f"step {step}") == 1.0
        assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o


def _bsp_config_run(name, steps, numel_cap=None, lp=False):
    cfg = W.config(name)
    if numel_cap:
        cfg = W.scaled(cfg, numel_cap)
    buf = W.make_buffers(cfg, DEV)
    lay = buf.layout
    theta_lp = torch.zeros(lay.total, dtype=torch.bfloat16, device=DEV) if lp else None
    o = B.Omni(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband)
    ora = O.Controller(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband)
    bs = B.BucketSet.from_flat(lay, buf.theta, buf.grads, buf.v, theta_lp)
    gen = torch.Generator().manual_seed(cfg.seed)
    base = W.draw_throughputs(cfg.K, gen, cfg.ratio)
    th_o, v_o, g_np = to_np(buf.theta), to_np(buf.v), [to_np(g) for g in buf.grads]
    lp_o = np.zeros(lay.total, np.uint16) if lp else None
    b = o.batches
    for step in range(steps):
        if step % max(cfg.rebatch_every, 1) == 0 and (cfg.rebatch_every or step == 0):
            T = W.jitter_throughputs(W.interference(base, step) if name == "vgg16" else base, gen)
            b, _ = o.rebatch(T)
            assert b == ora.rebatch(T)[0].tolist() and sum(b) == cfg.global_batch
        o.aggregate_bsp(bs, b, cfg.lr, cfg.momentum, cfg.weight_decay)
        # the oracle walks the same buckets (padding elements are zeros on both sides)
        sq_o = O.bsp_step_f32(g_np, b, th_o, v_o, cfg.lr, cfg.momentum, cfg.weight_decay, theta_lp=lp_o)
        assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o
    kind = cfg.grad_dtype
    assert assert_close(to_np(buf.theta), th_o, kind, name) == 1.0
    assert assert_close(to_np(buf.v), v_o, kind, name) == 1.0
    if lp:
        assert np.array_equal(to_np(theta_lp), lp_o)
    return o


def test_resnet18_config_shrunk_full_schedule():
    """62 tensors, 2 buckets, K=8, 100 steps with a re-batch every 10 (tensors capped at 3000 elements)."""
    _bsp_config_run("resnet18", 100, numel_cap=3000)


def test_resnet18_config_full_size():
    _bsp_config_run("resnet18", 12)


def test_resnet50_bf16_config_full_size():
    """The headline configuration at full size, 3 steps with the low-precision copy."""
    o = _bsp_config_run("resnet50_bf16", 3, lp=True)
    grid, block = o.query_launch(16, B.BF16)
    assert grid % torch.cuda.get_device_properties(0).multi_processor_count == 0 and block in (224, 192, 256)


def test_resnet50_f32_config_full_size():
    _bsp_config_run("resnet50_f32", 2)


def test_vgg16_config_shrunk_with_interference_phase():
    """K=32, 32 tensors, re-batch every step through the interference phase (steps 15-34)."""
    _bsp_config_run("vgg16", 50, numel_cap=5000)


def _chunks(lay, width=1 << 22):
    """Element ranges that tile every bucket of the layout, at most ``width`` elements each."""
    for bk in lay.buckets:
        for s in range(bk.start, bk.start + bk.n, width):
            yield s, min(s + width, bk.start + bk.n)


def _oracle_threads():
    import os

    return max(1, min(16, len(os.sched_getaffinity(0))))


def test_vgg16_config_full_size_every_element():
    """K=32, 138M parameters, 7 buckets: two steps at full size with a re-batch before each (the
    configuration re-batches every step), every element of theta and v against the oracle and the
    squared norm of both steps against the oracle's sums.  The rules are element-wise, so the
    oracle walks the buckets in ranges of 4M elements (bounded host memory), several ranges at a
    time on the host cores."""
    from concurrent.futures import ThreadPoolExecutor

    cfg = W.config("vgg16")
    buf = W.make_buffers(cfg, DEV)
    lay = buf.layout
    o = B.Omni(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband)
    ora = O.Controller(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband)
    gen = torch.Generator().manual_seed(cfg.seed)
    base = W.draw_throughputs(cfg.K, gen, cfg.ratio)
    bs = B.BucketSet.from_flat(lay, buf.theta, buf.grads, buf.v)
    th0, v0 = buf.theta.cpu(), buf.v.cpu()          # the state before the first step
    steps, batches, sq_gpu = 2, [], []
    for step in range(steps):
        T = W.jitter_throughputs(W.interference(base, step), gen)
        b, _ = o.rebatch(T)
        assert b == ora.rebatch(T)[0].tolist() and sum(b) == cfg.global_batch
        batches.append(b)
        o.aggregate_bsp(bs, b, cfg.lr, cfg.momentum)
        sq_gpu.append(o.stats().grad_sqnorm)
    assert batches[0] != batches[1]
    th1, v1 = buf.theta.cpu(), buf.v.cpu()

    def one(rng):
        s, e = rng
        g_np = [to_np(g[s:e]) for g in buf.grads]
        th_o, v_o = th0[s:e].numpy().copy(), v0[s:e].numpy().copy()
        sq = [O.bsp_step_f32(g_np, b, th_o, v_o, cfg.lr, cfg.momentum, 0.0) for b in batches]
        ok = np.array_equal(th1[s:e].numpy(), th_o) and np.array_equal(v1[s:e].numpy(), v_o)
        return ok, sq

    covered = 0
    sq_o = [0.0] * steps
    with ThreadPoolExecutor(max_workers=_oracle_threads()) as ex:
        for (s, e), (ok, sq) in zip(_chunks(lay), ex.map(one, _chunks(lay))):
            assert ok, (s, e)
            covered += e - s
            for i in range(steps):
                sq_o[i] += sq[i]
    assert covered == sum(bk.n for bk in lay.buckets) >= cfg.P
    for got, want in zip(sq_gpu, sq_o):
        assert abs(got - want) <= SQNORM_RTOL * want


def test_resnet50_asp_full_size_every_element():
    """25.6M parameters, 20 arrivals with controller feedback at full size: every element of the
    server parameters against the oracle."""
    from concurrent.futures import ThreadPoolExecutor

    cfg = W.config("resnet50_asp")
    buf = W.make_buffers(cfg, DEV)
    lay = buf.layout
    o = B.Omni(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, 1.0, B.ASP)
    ora = O.Controller(cfg.K, cfg.global_batch, cfg.b_min, cfg.b_max, cfg.deadband, 1.0, O.MODE_ASP)
    bs = B.BucketSet.from_flat(lay, buf.theta, buf.grads)
    th0 = buf.theta.cpu()
    events = []
    t_lib = _asp_stream(cfg, 20, lambda k, bu, tau: (events.append((k, bu, tau)), o.apply_asp(bs, k, bu, tau, cfg.lr)),
                        o.asp_report, cfg.seed)
    t_ora = _asp_stream(cfg, 20, lambda k, bu, tau: None, ora.asp_report, cfg.seed)
    assert t_lib == t_ora
    th1 = buf.theta.cpu()
    g_host = [g.cpu() for g in buf.grads]

    def one(rng):
        s, e = rng
        th_o = th0[s:e].numpy().copy()
        for k, bu, tau in events:
            O.asp_apply_f32(g_host[k][s:e].numpy(), bu, cfg.global_batch, th_o, None, cfg.lr, 0.0, 0.0)
        return np.array_equal(th1[s:e].numpy(), th_o)

    covered = 0
    with ThreadPoolExecutor(max_workers=_oracle_threads()) as ex:
        for (s, e), ok in zip(_chunks(lay), ex.map(one, _chunks(lay))):
            assert ok, (s, e)
            covered += e - s
    assert covered == sum(bk.n for bk in lay.buckets) >= cfg.P
    assert o.stats().arrivals == 20


def test_bucket_longer_than_32_bit_indices():
    """One bucket of 2^32 + 197,637 elements (bf16 gradient, no momentum buffer: 26 GB on the device):
    element offsets do not fit 32 bits.  The oracle checks windows at the start, across 2^31 and
    2^32, and the ragged tail; between the windows the gradient is zero and theta constant, so
    samples there must equal the one value the oracle gives for such an element, and the squared
    norm is the windows' alone."""
    n = (1 << 32) + 3 * 65536 + 1029
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GB of free device memory")
    gen = _gen(2**20 + 3)
    theta = torch.empty(n, device=DEV, dtype=torch.float32)
    grad = torch.zeros(n, device=DEV, dtype=torch.bfloat16)
    theta.fill_(0.25)
    w = 1 << 16
    windows = [0, (1 << 31) - w // 2, (1 << 32) - w // 2, n - w]
    for a in windows:                                   # random values only where the oracle will look
        theta[a:a + w].normal_(0, 0.05, generator=gen)
        grad[a:a + w] = torch.empty(w, device=DEV).normal_(0, 1e-3, generator=gen).to(torch.bfloat16)
    before = [(to_np(theta[a:a + w]), to_np(grad[a:a + w])) for a in windows]
    o = B.Omni(1, 32, 1, 96, 0.1)
    o.aggregate_bsp(B.BucketSet([theta], [[grad]]), [32], 0.1, 0.0, 1e-3)
    sq_want = 0.0
    for a, (th_o, g_o) in zip(windows, before):
        sq_want += O.bsp_step_f32([g_o], [32], th_o, None, 0.1, 0.0, 1e-3)
        assert np.array_equal(to_np(theta[a:a + w]), th_o), a
    # everywhere else the gradient is zero and theta is one value: the oracle says what it becomes
    flat = np.full(8, 0.25, np.float32)
    O.bsp_step_f32([np.zeros(8, np.uint16)], [32], flat, None, 0.1, 0.0, 1e-3)
    want_rest = flat[0]
    for a in (w + 12345, (1 << 31) + (1 << 20), (1 << 32) - (1 << 20), (1 << 32) + w + 7):
        got = to_np(theta[a:a + 4096])
        assert (got == want_rest).all(), a
    assert abs(o.stats().grad_sqnorm - sq_want) <= SQNORM_RTOL * sq_want
