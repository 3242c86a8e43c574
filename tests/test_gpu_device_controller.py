"""GPU parity of the device-resident controller: the one-warp re-batch kernel against the CPU
oracle's controller (bit-exact integers), and the fused step that reads the weights it leaves in
device memory against the oracle's step, eagerly and replayed from a CUDA graph."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2503_17469_b200 import binding as B
from paper_2503_17469_b200 import workloads as W

from parity_util import SQNORM_RTOL, assert_close, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bounds(K, B_):
    per = B_ // K
    return max(1, per // 8), 3 * per


def _case(seed):
    """A seeded controller configuration: (K, B, b_min, b_max, deadband, alpha, mode, flags)."""
    rng = np.random.default_rng(seed)
    K = int(rng.integers(1, 33))
    per = int(rng.choice([4, 8, 32, 100]))
    B_ = K * per + int(rng.integers(0, K))          # K does not always divide B
    b_min, b_max = max(1, per // 8), 3 * per + 1
    deadband = float(rng.choice([0.0, 0.05, 0.10, 0.15]))
    alpha = float(rng.choice([1.0, 0.5, 0.25]))
    mode = int(rng.choice([B.BSP, B.BSP, B.ASP]))
    flags = int(rng.choice([0, 0, B.INPUT_IS_TIME]))
    if rng.random() < 0.3:                           # the multiplicative reading of the global-batch rule
        flags |= B.CONSERVE_MULTIPLICATIVE
    return rng, K, B_, b_min, b_max, deadband, alpha, mode, flags


def _oracle_flags(flags):
    """The oracle numbers its flags independently of the library."""
    return ((O.FLAG_INPUT_IS_TIME if flags & B.INPUT_IS_TIME else 0)
            | (O.FLAG_CONSERVE_MULTIPLICATIVE if flags & B.CONSERVE_MULTIPLICATIVE else 0))


@pytest.mark.parametrize("seed", range(40))
def test_device_rebatch_matches_the_oracle_bit_for_bit(seed):
    """Twelve successive re-batches from jittered heterogeneous throughputs; after each one the
    device copy's batches equal the oracle's, and so do the weights it leaves for the step."""
    rng, K, B_, b_min, b_max, deadband, alpha, mode, flags = _case(1000 + seed)
    o = B.Omni(K, B_, b_min, b_max, deadband, alpha, mode, flags)
    ref = O.Controller(K, B_, b_min, b_max, deadband, alpha, mode, _oracle_flags(flags))
    assert list(ref.batches) == o.batches
    o.ctl_to_device()
    base = 8.0 ** rng.random(K)
    measured = torch.empty(K, dtype=torch.float64, device=DEV)
    new_b = torch.zeros(K, dtype=torch.int32, device=DEV)
    for step in range(12):
        T = base * (1.0 + 0.2 * (2.0 * rng.random(K) - 1.0))
        if step == 6:
            T[: max(1, K // 4)] *= 0.5                       # an interference phase begins
        b_now = ref.batches.astype(np.float64)
        m = b_now / T if flags & B.INPUT_IS_TIME else T
        measured.copy_(torch.from_numpy(m))
        o.rebatch_device(measured, new_b)
        want, _ = ref.rebatch(m)
        got = new_b.cpu().numpy()
        assert np.array_equal(got, want), (seed, step, got, want)
        if mode == B.BSP:
            assert int(got.sum()) == B_
        assert got.min() >= b_min and got.max() <= b_max
    assert o.ctl_from_device() == [int(x) for x in ref.batches]
    _, l32 = O.bsp_weights(ref.batches, 0)
    assert o.stats().weight_sum == sum(float(x) for x in l32)      # ascending sum of the float weights
    # the host controller continues from the downloaded state exactly as the oracle does
    T = base * 1.1
    m = ref.batches.astype(np.float64) / T if flags & B.INPUT_IS_TIME else T
    assert o.rebatch(list(m))[0] == [int(x) for x in ref.rebatch(m)[0]]


@pytest.mark.parametrize("seed", range(12))
def test_device_report_matches_the_oracle_bit_for_bit(seed):
    """evalBsz on the device copy: 150 reports of randomly chosen workers (throughput or time
    input, smoothing, now and then a batch that differs from the server's entry); after every
    report the returned batch equals the oracle's, at the end the whole map does, and the host
    controller continues from the downloaded state exactly as the oracle does."""
    rng = np.random.default_rng(7000 + seed)
    K = int(rng.integers(1, 33))
    alpha = float(rng.choice([1.0, 0.5, 0.25]))
    flags = int(rng.choice([0, B.INPUT_IS_TIME]))
    o = B.Omni(K, 32 * K, 4, 96, 0.10, alpha, B.ASP, flags)
    ref = O.Controller(K, 32 * K, 4, 96, 0.10, alpha, O.MODE_ASP, _oracle_flags(flags))
    o.ctl_to_device()
    T = 8.0 ** rng.random(K)
    cur = [32] * K
    measured = torch.empty(1, dtype=torch.float64, device=DEV)
    out = torch.zeros(1, dtype=torch.int32, device=DEV)
    for ev in range(150):
        k = int(rng.integers(0, K))
        used = cur[k] if rng.random() < 0.8 else int(rng.integers(4, 97))
        thr = float(T[k] * (1.0 + 0.1 * rng.uniform(-1, 1)))
        m = used / thr if flags & B.INPUT_IS_TIME else thr
        measured.fill_(m)
        o.asp_report_device(k, used, measured, out)
        want = ref.asp_report(k, used, m)
        got = int(out.item())
        assert got == want, (seed, ev, k, got, want)
        cur[k] = got
    assert o.ctl_from_device() == [int(x) for x in ref.batches]
    k = int(rng.integers(0, K))
    assert o.asp_report(k, cur[k], float(T[k])) == ref.asp_report(k, cur[k], float(T[k]))


def test_device_report_hand_case_and_refused_measurement():
    """The hand-derived report sequence R1 (a reported batch that differs from the server's entry,
    alpha = 0.25, time input) on the device copy; a measurement that is not positive changes nothing
    and is reported once."""
    o = B.Omni(2, 64, 4, 96, 0.10, 0.25, B.ASP, B.INPUT_IS_TIME)
    o.ctl_to_device()
    m = torch.empty(1, dtype=torch.float64, device=DEV)
    out = torch.zeros(1, dtype=torch.int32, device=DEV)
    for worker, used, t, ret, after in ((0, 32, 8.0, 32, [32, 32]), (1, 32, 4.0, 48, [24, 48]),
                                        (0, 20, 6.0, 15, [15, 69]), (1, 69, 6.0, 92, [12, 92])):
        m.fill_(t)
        o.asp_report_device(worker, used, m, out)
        assert int(out.item()) == ret
        assert o.ctl_from_device() == after
    m.fill_(0.0)
    out.fill_(-7)
    o.asp_report_device(0, 12, m, out)
    with pytest.raises(B.OmniError) as e:
        o.ctl_from_device()
    assert e.value.status == B.ERR_BAD_MEASUREMENT and int(out.item()) == -7
    assert o.ctl_from_device() == [12, 92]


def test_device_rebatch_reproduces_the_hand_case():
    """Throughputs (1,2,4,8), B = 64, bounds (2,48), dead-band 10 %: (2,6,19,37), (6,9,17,32),
    (4,8,16,36), then steady -- the hand-derived trace the host controller is pinned to."""
    o = B.Omni(4, 64, 2, 48, 0.10)
    o.ctl_to_device()
    T = torch.tensor([1.0, 2.0, 4.0, 8.0], dtype=torch.float64, device=DEV)
    out = torch.zeros(4, dtype=torch.int32, device=DEV)
    trace = []
    for _ in range(4):
        o.rebatch_device(T, out)
        trace.append(out.cpu().tolist())
    assert trace == [[2, 6, 19, 37], [6, 9, 17, 32], [4, 8, 16, 36], [4, 8, 16, 36]]


def test_bad_measurement_on_the_device_changes_nothing_and_is_reported_once():
    o = B.Omni(4, 64, 2, 48, 0.10)
    o.ctl_to_device()
    good = torch.tensor([1.0, 2.0, 4.0, 8.0], dtype=torch.float64, device=DEV)
    out = torch.zeros(4, dtype=torch.int32, device=DEV)
    o.rebatch_device(good, out)
    for bad_value in (float("nan"), 0.0, -1.0, float("inf")):
        bad = good.clone()
        bad[2] = bad_value
        out.fill_(-7)
        o.rebatch_device(bad, out)
        with pytest.raises(B.OmniError) as e:
            o.ctl_from_device()
        assert e.value.status == B.ERR_BAD_MEASUREMENT
        assert out.cpu().tolist() == [-7] * 4
        assert o.ctl_from_device() == [2, 6, 19, 37]            # reported once, state untouched
    o.rebatch_device(good, out)
    assert out.cpu().tolist() == [6, 9, 17, 32]


def test_device_calls_need_the_device_copy():
    o = B.Omni(4, 64, 2, 48, 0.10)
    m = torch.ones(4, dtype=torch.float64, device=DEV)
    with pytest.raises(B.OmniError) as e:
        o.rebatch_device(m)
    assert e.value.status == B.ERR_BAD_CONFIG
    with pytest.raises(B.OmniError) as e:
        o.ctl_from_device()
    assert e.value.status == B.ERR_BAD_CONFIG


@pytest.mark.parametrize("kind", ["f32", "bf16"])
@pytest.mark.parametrize("K", [1, 4, 8, 16, 32])
def test_step_with_device_batches_matches_the_oracle(K, kind):
    """Re-batch on the device, then the fused step with the device-resident weights; several
    tiles and a ragged tail; every step against the oracle's controller + f32 step.  K = 4 (float)
    and K = 8 (bfloat16) run a size that falls into the short-launch shape of the ring."""
    n = 3 * 8192 + 17 if K > 8 else 100_003
    if (K, kind) in ((4, "f32"), (8, "bf16")):
        n = torch.cuda.get_device_properties(0).multi_processor_count * 2048 * 3 + 1031
    per = 32
    B_ = K * per
    b_min, b_max = _bounds(K, B_)
    gen = torch.Generator(device=DEV).manual_seed(77 + K)
    gdt = torch.bfloat16 if kind == "bf16" else torch.float32
    theta = torch.empty(n, device=DEV).normal_(0, 0.05, generator=gen)
    v = torch.zeros(n, device=DEV)
    grads = [torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen).to(gdt) for _ in range(K)]
    o = B.Omni(K, B_, b_min, b_max, 0.10)
    ref = O.Controller(K, B_, b_min, b_max, 0.10)
    bs = B.BucketSet([theta], [grads], [v])
    th_o, v_o, g_np = to_np(theta), to_np(v), [to_np(g) for g in grads]
    rng = np.random.default_rng(5 + K)
    base = 8.0 ** rng.random(K)
    measured = torch.empty(K, dtype=torch.float64, device=DEV)
    o.ctl_to_device()
    for step in range(4):
        if step != 1:                                    # step 1 re-uses the weights of step 0
            T = base * (1.0 + 0.2 * (2.0 * rng.random(K) - 1.0))
            measured.copy_(torch.from_numpy(T))
            o.rebatch_device(measured)
            ref.rebatch(T)
        o.aggregate_bsp_device_batches(bs, 0.1, 0.9, 1e-4)
        sq_o = O.bsp_step_f32(g_np, ref.batches, th_o, v_o, 0.1, 0.9, 1e-4)
        frac = assert_close(to_np(theta), th_o, kind, f"theta step {step}")
        assert frac == 1.0
        assert np.array_equal(to_np(v), v_o)
        sq = o.stats().grad_sqnorm
        assert abs(sq - sq_o) <= SQNORM_RTOL * sq_o
    assert o.ctl_from_device() == [int(x) for x in ref.batches]
    _, l32 = O.bsp_weights(ref.batches, 0)
    assert o.stats().weight_sum == sum(float(x) for x in l32)


def test_unscaled_mean_flag_on_the_device():
    K, n = 3, 5000
    gen = torch.Generator(device=DEV).manual_seed(9)
    theta = torch.empty(n, device=DEV).normal_(0, 0.05, generator=gen)
    grads = [torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen) for _ in range(K)]
    o = B.Omni(K, 96, 4, 96, 0.10, flags=B.UNSCALED_MEAN)
    ref = O.Controller(K, 96, 4, 96, 0.10)
    bs = B.BucketSet([theta], [grads])
    th_o, g_np = to_np(theta), [to_np(g) for g in grads]
    T = np.array([1.0, 3.0, 9.0])
    o.ctl_to_device()
    o.rebatch_device(torch.from_numpy(T).to(DEV))
    ref.rebatch(T)
    o.aggregate_bsp_device_batches(bs, 0.1)
    O.bsp_step_f32(g_np, ref.batches, th_o, None, 0.1, 0.0, 0.0, flags=O.FLAG_UNSCALED_MEAN)
    assert np.array_equal(to_np(theta), th_o)


def test_whole_steps_replayed_from_a_cuda_graph():
    """Re-batch + fused step, five times, captured once and replayed three times with fresh
    measurements written into the same device buffer between replays: no host call other than
    the replay, the same bits as the oracle's controller + step."""
    K, n = 4, 1 << 18
    gen = torch.Generator(device=DEV).manual_seed(2024)
    theta = torch.empty(n, device=DEV).normal_(0, 0.05, generator=gen)
    v = torch.zeros(n, device=DEV)
    grads = [torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen) for _ in range(K)]
    o = B.Omni(K, 64, 2, 48, 0.10)
    ref = O.Controller(K, 64, 2, 48, 0.10)
    bs = B.BucketSet([theta], [grads], [v])
    th0, v0 = theta.clone(), v.clone()
    g_np = [to_np(g) for g in grads]
    measured = torch.tensor([1.0, 2.0, 4.0, 8.0], dtype=torch.float64, device=DEV)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        o.ctl_to_device()
        o.rebatch_device(measured)                       # eager call: sizes the launches
        o.aggregate_bsp_device_batches(bs, 0.1, 0.9)
    side.synchronize()
    theta.copy_(th0), v.copy_(v0)                        # start over: the host controller still holds the
    with torch.cuda.stream(side):                        # initial state (device calls never touch it)
        o.ctl_to_device()
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(5):
            o.rebatch_device(measured)
            o.aggregate_bsp_device_batches(bs, 0.1, 0.9)
    th_o, v_o = to_np(th0), to_np(v0)
    rng = np.random.default_rng(3)
    for replay in range(3):
        T = np.array([1.0, 2.0, 4.0, 8.0]) * (1.0 + 0.2 * (2.0 * rng.random(K) - 1.0))
        measured.copy_(torch.from_numpy(T))
        torch.cuda.synchronize()
        graph.replay()
        for _ in range(5):
            ref.rebatch(T)
            sq_o = O.bsp_step_f32(g_np, ref.batches, th_o, v_o, 0.1, 0.9, 0.0)
    torch.cuda.synchronize()
    assert np.array_equal(to_np(theta), th_o) and np.array_equal(to_np(v), v_o)
    assert o.ctl_from_device() == [int(x) for x in ref.batches]
    assert abs(o.stats().grad_sqnorm - sq_o) <= SQNORM_RTOL * sq_o


def test_mixed_call_sequence_on_one_context_and_stream():
    """Two hundred calls of every kind back to back on one stream and one set of buffers --
    synchronous steps with host and with device-resident weights, single and batched
    asynchronous arrivals, push + pull in one pass, the allocation-free step -- with no
    synchronisation in between: the kernels order themselves (dependent launches, alternating
    sweep directions, shared workspace).  State after every twentieth call and at the end equals
    the oracle's, bit for bit."""
    K, n, B_ = 5, 3 * 8192 + 1031, 160
    gen = torch.Generator(device=DEV).manual_seed(4242)
    theta = torch.empty(n, device=DEV).normal_(0, 0.05, generator=gen)
    v = torch.zeros(n, device=DEV)
    snap = theta.clone()
    grads = [torch.empty(n, device=DEV).normal_(0, 1e-3, generator=gen) for _ in range(K)]
    o = B.Omni(K, B_, 4, 96, 0.10)
    ref = O.Controller(K, B_, 4, 96, 0.10)
    bs = B.BucketSet([theta], [grads], [v])
    th_o, v_o, sn_o, g_np = to_np(theta), to_np(v), to_np(snap), [to_np(g) for g in grads]
    rng = np.random.default_rng(17)
    measured = torch.empty(K, dtype=torch.float64, device=DEV)
    o.ctl_to_device()
    lr, mu, wd = 0.05, 0.9, 1e-4
    for i in range(200):
        kind = int(rng.integers(0, 6))
        if kind == 0:
            b = [int(x) for x in ref.batches]
            o.aggregate_bsp(bs, b, lr, mu, wd)
            O.bsp_step_f32(g_np, b, th_o, v_o, lr, mu, wd)
        elif kind == 1:
            T = 8.0 ** rng.random(K)
            measured.copy_(torch.from_numpy(T))
            o.rebatch_device(measured)
            ref.rebatch(T)
            o.aggregate_bsp_device_batches(bs, lr, mu, wd)
            O.bsp_step_f32(g_np, ref.batches, th_o, v_o, lr, mu, wd)
        elif kind == 2:
            k, bu = int(rng.integers(0, K)), int(rng.integers(4, 97))
            o.apply_asp(bs, k, bu, 0, lr, mu, wd)
            O.asp_apply_f32(g_np[k], bu, B_, th_o, v_o, lr, mu, wd)
        elif kind == 3:
            ks = [int(x) for x in rng.integers(0, K, 3)]
            bus = [int(x) for x in rng.integers(4, 97, 3)]
            o.apply_asp_batch(bs, ks, bus, [0, 1, 2], lr, mu, wd)
            for k, bu in zip(ks, bus):
                O.asp_apply_f32(g_np[k], bu, B_, th_o, v_o, lr, mu, wd)
        elif kind == 4:
            k, bu = int(rng.integers(0, K)), int(rng.integers(4, 97))
            o.asp_push_pull(bs, k, bu, 0, [snap], lr, wd)
            O.asp_push_overwrite_f32(g_np[k], bu, B_, th_o, sn_o, lr, wd)
            sn_o[:] = th_o
        else:
            b = [int(x) for x in ref.batches]
            B.aggregate_bsp_noalloc(bs, b, lr, mu, wd)
            O.bsp_step_f32(g_np, b, th_o, v_o, lr, mu, wd)
        if i % 20 == 19:
            assert np.array_equal(to_np(theta), th_o), i
            assert np.array_equal(to_np(v), v_o), i
    assert np.array_equal(to_np(snap), sn_o)
    assert o.ctl_from_device() == [int(x) for x in ref.batches]
    o.stats()                                            # no bounded wait ran out
