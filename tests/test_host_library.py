"""Host-side checks of the C-ABI library that need no GPU: exported symbols, the controller
against the oracle (bit-exact integers), validation and error codes."""
import ctypes as C
import re
from pathlib import Path

import numpy as np
import pytest

from oracle import oracle as O
from paper_2503_17469_b200 import binding as B

ROOT = Path(__file__).resolve().parents[1]


def test_library_exports_every_declared_symbol():
    header = (ROOT / "include" / "omni.h").read_text()
    declared = set(re.findall(r"\b(omni_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    L = B.lib()
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in omni.h but not exported"
    assert declared == set(B.EXPORTS)


def test_strerror_covers_all_codes():
    L = B.lib()
    for code in range(0, -14, -1):
        assert L.omni_strerror(code) and L.omni_strerror(code) != b"unknown status"
    assert L.omni_strerror(-99) == b"unknown status"


def test_create_validation():
    def rc(**kw):
        cfg = dict(K=4, global_batch=64, b_min=2, b_max=48, deadband=0.1, ewma_alpha=1.0, mode=B.BSP, flags=0)
        cfg.update(kw)
        h = C.c_void_p()
        c = B.omni_config(*[cfg[k] for k in ("K", "global_batch", "b_min", "b_max", "deadband", "ewma_alpha", "mode", "flags")])
        r = B.lib().omni_create(C.byref(c), C.byref(h))
        if r == 0:
            B.lib().omni_destroy(h)
        return r

    assert rc() == B.OK
    assert rc(K=0) == B.ERR_BAD_K and rc(K=33) == B.ERR_BAD_K
    assert rc(b_min=17) == B.ERR_INFEASIBLE and rc(b_max=15) == B.ERR_INFEASIBLE
    assert rc(b_min=17, mode=B.ASP) == B.OK          # no global-batch rule in ASP
    assert rc(b_min=0) == B.ERR_BAD_CONFIG and rc(b_max=1) == B.ERR_BAD_CONFIG
    assert rc(deadband=-0.1) == B.ERR_BAD_CONFIG and rc(deadband=float("nan")) == B.ERR_BAD_CONFIG
    assert rc(ewma_alpha=0.0) == B.ERR_BAD_CONFIG and rc(ewma_alpha=1.5) == B.ERR_BAD_CONFIG
    assert rc(mode=7) == B.ERR_BAD_CONFIG
    assert rc(flags=64) == B.ERR_BAD_CONFIG and rc(flags=B.BULK_COPY | B.NO_BULK_COPY) == B.ERR_BAD_CONFIG
    assert rc(flags=B.UNSCALED_MEAN | B.INPUT_IS_TIME | B.CONSERVE_MULTIPLICATIVE | B.BULK_COPY) == B.OK
    assert B.lib().omni_create(None, None) == B.ERR_NULL


def test_controller_matches_oracle_on_hand_case():
    o = B.Omni(4, 64, 2, 48, 0.10)
    assert o.batches == [16, 16, 16, 16]
    assert o.rebatch([1, 2, 4, 8])[0] == [2, 6, 19, 37]


@pytest.mark.parametrize("mode", [B.BSP, B.ASP])
def test_rebatch_bit_exact_against_oracle_random_traces(mode):
    rng = np.random.default_rng(100 + mode)
    for trial in range(300):
        K = int(rng.integers(1, 33))
        per = int(rng.integers(8, 65))
        Bg = K * per + int(rng.integers(0, K))
        b_min, b_max = max(1, per // 8), 3 * per
        db = float(rng.choice([0.0, 0.05, 0.1, 0.15]))
        alpha = float(rng.choice([1.0, 0.5, 0.3]))
        flags = int(rng.choice([0, B.INPUT_IS_TIME]))
        mult = bool(rng.uniform() < 0.4)                 # the multiplicative reading of the global-batch rule
        lib = B.Omni(K, Bg, b_min, b_max, db, alpha, mode, flags | (B.CONSERVE_MULTIPLICATIVE if mult else 0))
        ora = O.Controller(K, Bg, b_min, b_max, db, alpha, mode,
                           (O.FLAG_INPUT_IS_TIME if flags else 0) | (O.FLAG_CONSERVE_MULTIPLICATIVE if mult else 0))
        assert lib.batches == ora.batches.tolist()
        base = 8.0 ** rng.uniform(0, 1, K)
        for step in range(12):
            T = base * (1 + 0.2 * (2 * rng.uniform(0, 1, K) - 1))
            if step in (5, 6):
                T[: max(1, K // 4)] *= 0.5
            meas = (np.array(lib.batches) / T) if flags else T
            nb_l, ch_l = lib.rebatch(meas.tolist())
            nb_o, ch_o = ora.rebatch(meas)
            assert nb_l == nb_o.tolist(), (trial, step)
            assert ch_l == ch_o.tolist()
            if mode == B.BSP:
                assert sum(nb_l) == Bg


def test_asp_report_bit_exact_against_oracle():
    rng = np.random.default_rng(200)
    for trial in range(100):
        K = int(rng.integers(2, 17))
        alpha = float(rng.choice([1.0, 0.5]))
        lib = B.Omni(K, 32 * K, 4, 96, 0.1, alpha, B.ASP)
        ora = O.Controller(K, 32 * K, 4, 96, 0.1, alpha, O.MODE_ASP)
        T = 8.0 ** rng.uniform(0, 1, K)
        cur = [32] * K
        for ev in range(200):
            k = int(rng.integers(0, K))
            meas = float(T[k] * (1 + 0.1 * rng.uniform(-1, 1)))
            # now and then a worker ran another batch than the one the server handed it
            used = cur[k] if rng.uniform() < 0.8 else int(rng.integers(4, 97))
            a = lib.asp_report(k, used, meas)
            b = ora.asp_report(k, used, meas)
            assert a == b
            cur[k] = a
        assert lib.batches == ora.batches.tolist()


def test_multiplicative_conservation_hand_cases():
    import json

    gold = json.loads((ROOT / "tests" / "golden" / "controller_cases.json").read_text())
    for case in gold["multiplicative_cases"]:
        o = B.Omni(case["K"], case["B"], case["b_min"], case["b_max"], case["deadband"], 1.0, B.BSP,
                   B.CONSERVE_MULTIPLICATIVE)
        assert o.batches == case["b0"]
        for want in case["expect"]:
            assert o.rebatch(case["throughput"])[0] == want, case["name"]


def test_asp_report_hand_derived_sequences():
    """The library's evalBsz on the hand-derived report sequences (a reported batch that differs
    from the server's entry, smoothed times): same integers as derived by hand."""
    import json

    gold = json.loads((ROOT / "tests" / "golden" / "controller_cases.json").read_text())
    for case in gold["report_cases"]:
        flags = B.INPUT_IS_TIME if case["input"] == "time" else 0
        o = B.Omni(case["K"], case["B"], case["b_min"], case["b_max"], case["deadband"], case["alpha"], B.ASP, flags)
        for r in case["reports"]:
            assert o.asp_report(r["worker"], r["b_used"], r["measured"]) == r["returns"], case["name"]
            assert o.batches == r["map_after"], case["name"]


def test_library_batches_depend_only_on_throughput_ratios():
    rng = np.random.default_rng(22)
    for _ in range(50):
        K = int(rng.integers(2, 33))
        mult = bool(rng.uniform() < 0.5)
        flags = B.CONSERVE_MULTIPLICATIVE if mult else 0
        a = B.Omni(K, 32 * K, 4, 96, 0.1, 0.5, B.BSP, flags)
        b = B.Omni(K, 32 * K, 4, 96, 0.1, 0.5, B.BSP, flags)
        base = 8.0 ** rng.uniform(0, 1, K)
        for step in range(5):
            T = base * (1 + 0.2 * (2 * rng.uniform(0, 1, K) - 1))
            assert a.rebatch(T.tolist())[0] == b.rebatch((T * 0.25).tolist())[0]


def test_static_rebatch_matches_oracle():
    rng = np.random.default_rng(300)
    for _ in range(200):
        K = int(rng.integers(1, 33))
        mode = int(rng.integers(0, 2))
        lib = B.Omni(K, 32 * K, 4, 96, 0.1, 1.0, mode)
        ora = O.Controller(K, 32 * K, 4, 96, 0.1, 1.0, mode)
        c = rng.integers(1, 33, K).astype(float)
        assert lib.rebatch_static(c.tolist()) == ora.rebatch_static(c).tolist()


def test_rebatch_errors_leave_state():
    o = B.Omni(4, 64, 2, 48, 0.1)
    for bad in ([1, 2, 0, 1], [1, -1, 1, 1], [1, float("nan"), 1, 1], [float("inf"), 1, 1, 1]):
        with pytest.raises(B.OmniError) as e:
            o.rebatch(bad)
        assert e.value.status == B.ERR_BAD_MEASUREMENT
        assert o.batches == [16, 16, 16, 16]
    with pytest.raises(B.OmniError) as e:
        o.set_batches([16, 16, 16, 15])
    assert e.value.status == B.ERR_BAD_BATCH
    with pytest.raises(B.OmniError) as e:
        o.set_batches([0, 32, 16, 16])
    assert e.value.status == B.ERR_BAD_BATCH
    a = B.Omni(4, 64, 2, 48, 0.1, 1.0, B.ASP)
    for args, code in (((4, 16, 1.0), B.ERR_BAD_WORKER), ((-1, 16, 1.0), B.ERR_BAD_WORKER),
                       ((0, 0, 1.0), B.ERR_BAD_BATCH), ((0, 16, 0.0), B.ERR_BAD_MEASUREMENT)):
        with pytest.raises(B.OmniError) as e:
            a.asp_report(*args)
        assert e.value.status == code


def test_argument_validation_happens_before_any_cuda_call():
    """These calls fail on their arguments, so they return the same codes with or without a GPU."""
    L = B.lib()
    o = B.Omni(2, 64, 4, 96, 0.1)
    b = (C.c_int32 * 2)(32, 32)
    grads = (C.c_void_p * 2)(0x1000, 0x2000)
    bk = (B.omni_bucket * 1)(B.omni_bucket(0x1000, 0x1000, None, C.cast(grads, C.POINTER(C.c_void_p)), 64))
    agg = lambda *a: L.omni_aggregate_bsp(o._h, *a)
    assert agg(bk, 1, 0, None, 0.1, 0.9, 0.0, None) == B.ERR_NULL
    assert agg(None, 1, 0, b, 0.1, 0.9, 0.0, None) == B.ERR_NULL
    assert agg(bk, -1, 0, b, 0.1, 0.9, 0.0, None) == B.ERR_BAD_CONFIG
    assert agg(bk, 1, 5, b, 0.1, 0.9, 0.0, None) == B.ERR_BAD_CONFIG
    assert agg(bk, 1, 0, (C.c_int32 * 2)(32, 31), 0.1, 0.9, 0.0, None) == B.ERR_BAD_BATCH
    assert agg(bk, 1, 0, (C.c_int32 * 2)(64, 0), 0.1, 0.9, 0.0, None) == B.ERR_BAD_BATCH
    bk[0].param = 0x1004
    assert agg(bk, 1, 0, b, 0.1, 0.9, 0.0, None) == B.ERR_ALIGN
    bk[0].param = 0x1000
    grads[1] = 0x2008
    assert agg(bk, 1, 0, b, 0.1, 0.9, 0.0, None) == B.ERR_ALIGN
    grads[1] = 0
    assert agg(bk, 1, 0, b, 0.1, 0.9, 0.0, None) == B.ERR_NULL
    grads[1] = 0x2000
    bk[0].momentum = None
    assert agg(bk, 1, 0, b, 0.1, 0.9, 0.0, None) == B.ERR_BAD_CONFIG    # momentum without a buffer
    bk[0].momentum = 0x1000
    asp = lambda *a: L.omni_apply_asp(o._h, bk, 1, 0, *a)
    assert asp(2, 32, 0, 0.1, 0.0, 0.0, None) == B.ERR_BAD_WORKER
    assert asp(0, 0, 0, 0.1, 0.0, 0.0, None) == B.ERR_BAD_BATCH
    assert asp(0, 32, -1, 0.1, 0.0, 0.0, None) == B.ERR_BAD_TAU
    # the one-call step: the measurements are validated before anything is enqueued, and a call that
    # fails afterwards (here: no usable device memory behind the made-up pointers is never reached,
    # the measurement is refused first) leaves the controller as it was
    nb = (C.c_int32 * 2)()
    step = lambda m, *a: L.omni_step_bsp(o._h, bk, 1, 0, m, 0.1, 0.9, 0.0, *a)
    assert step(None, nb, None, None) == B.ERR_NULL
    assert step((C.c_double * 2)(1.0, 2.0), None, None, None) == B.ERR_NULL
    assert step((C.c_double * 2)(1.0, 0.0), nb, None, None) == B.ERR_BAD_MEASUREMENT
    assert step((C.c_double * 2)(float("nan"), 1.0), nb, None, None) == B.ERR_BAD_MEASUREMENT
    assert o.batches == [32, 32]
    # the device-resident controller: nothing works before the device copy exists
    assert L.omni_ctl_to_device(None, None) == B.ERR_NULL
    assert L.omni_ctl_from_device(None, None) == B.ERR_NULL
    assert L.omni_ctl_from_device(o._h, None) == B.ERR_BAD_CONFIG
    assert L.omni_rebatch_device(o._h, None, None, None) == B.ERR_NULL
    assert L.omni_rebatch_device(o._h, 0x1000, None, None) == B.ERR_BAD_CONFIG
    assert L.omni_asp_report_device(o._h, 0, 32, None, None, None) == B.ERR_NULL
    assert L.omni_asp_report_device(o._h, 2, 32, 0x1000, None, None) == B.ERR_BAD_WORKER
    assert L.omni_asp_report_device(o._h, 0, 0, 0x1000, None, None) == B.ERR_BAD_BATCH
    assert L.omni_asp_report_device(o._h, 0, 32, 0x1000, None, None) == B.ERR_BAD_CONFIG   # no device copy yet
    assert L.omni_aggregate_bsp_device_batches(None, bk, 1, 0, 0.1, 0.9, 0.0, None) == B.ERR_NULL
    assert L.omni_aggregate_bsp_device_batches(o._h, bk, 1, 0, 0.1, 0.9, 0.0, None) == B.ERR_BAD_CONFIG
    assert o.kernel_launches == 0
    s = o.stats()
    assert s.steps == 0 and s.arrivals == 0 and sum(s.tau_hist) == 0


def test_the_abi_is_usable_from_plain_c(tmp_path):
    """include/omni.h compiles as C99 with warnings as errors, and a C program linked against the
    library runs the host controller (no GPU involved)."""
    import subprocess

    lib = B._build.build()
    exe = tmp_path / "controller_from_c"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", str(ROOT / "include"),
                    str(ROOT / "tests" / "c_abi" / "controller_from_c.c"), "-o", str(exe),
                    str(lib), f"-Wl,-rpath,{lib.parent}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines()
    assert out[:4] == ["2 6 19 37", "6 9 17 32", "4 8 16 36", "4 8 16 36"]
    assert out[4].startswith(f"{B.ERR_NULL} ")
    assert out[5] == "0+384 384+320 704+296"


def test_controller_state_survives_a_checkpoint():
    """Export after some re-batches with EWMA smoothing, import into a fresh context: both continue
    with identical batches; records for another configuration or damaged records are refused and
    leave the context as it was."""
    mk = lambda K=4, Bt=128: B.Omni(K, Bt, 4, 96, 0.05, ewma_alpha=0.5)
    a = mk()
    rng = np.random.default_rng(3)
    for _ in range(3):
        a.rebatch(list(8.0 ** rng.random(4)))
    rec = a.export_state()
    b = mk()
    b.import_state(rec)
    assert b.batches == a.batches
    for _ in range(5):
        T = list(8.0 ** rng.random(4))
        assert a.rebatch(T) == b.rebatch(T)           # the smoothed times came along
    for bad_ctx in (mk(K=8, Bt=256), mk(Bt=160)):
        with pytest.raises(B.OmniError) as e:
            bad_ctx.import_state(rec)
        assert e.value.status == B.ERR_BAD_CONFIG
    c = mk()
    before = c.batches
    for damaged in (rec[:40], b"\0" * len(rec)):
        with pytest.raises(B.OmniError):
            c.import_state(damaged)
    broken = bytearray(rec)
    broken[16:20] = (0).to_bytes(4, "little", signed=True)      # batch[0] = 0
    with pytest.raises(B.OmniError) as e:
        c.import_state(bytes(broken))
    assert e.value.status == B.ERR_BAD_BATCH and c.batches == before
