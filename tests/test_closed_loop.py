"""The controller in closed loop on the paper's heterogeneity levels (host only): qualitative
statements of the paper that must hold for the implementation."""
import pytest

from paper_2503_17469_b200 import simulate as S


def test_static_hl8_reaches_steady_batches_in_a_few_adjustments():
    """Sec. IV-D: steady state after 2-4 adjustments under static heterogeneity."""
    tr = S.run_bsp(S.stepwise_schedule([8], 12), 128, 4, 96, 0.10)
    changed_epochs = [e for e, a in enumerate(tr.adjustments) if a]
    assert changed_epochs and max(changed_epochs) <= 3
    assert all(sum(b) == 128 for b in tr.batches)
    # in steady state the workers' compute times are within the dead-band of each other
    t = tr.compute_time[-1]
    assert max(t) / min(t) < 1.15
    # and the straggler penalty of uniform batching is gone: 32/4 = 8 time units vs < 3
    assert tr.uniform_time[-1] == 8.0 and tr.iteration_time[-1] < 3.0


def test_uniform_cluster_keeps_uniform_batches():
    """HL1: variable batching equals uniform batching."""
    tr = S.run_bsp(S.stepwise_schedule([1], 5), 128, 4, 96, 0.10)
    assert all(b == [32, 32, 32, 32] for b in tr.batches) and sum(tr.adjustments) == 0
    assert tr.time_reduction() == 0.0


@pytest.mark.parametrize("epochs_per_level", [4, 5, 20, 25])
def test_dynamic_heterogeneity_is_tracked_and_saves_time(epochs_per_level):
    """Sec. IV-E: HL1 -> 2 -> 4 -> 8 -> 4 -> 2 -> 1 in steps, (b_min, b_max) = (4, 96), dead-band 10 %,
    global batch 128 kept fixed.  The paper reports 12.8-29.3 % shorter time-to-accuracy; the
    model cluster (compute time only, no communication) must at least show a clear saving and
    batches that follow each level change within a few epochs."""
    levels = [1, 2, 4, 8, 4, 2, 1]
    sched = S.stepwise_schedule(levels, epochs_per_level)
    tr = S.run_bsp(sched, 128, 4, 96, 0.10)
    assert all(sum(b) == 128 and min(b) >= 4 and max(b) <= 96 for b in tr.batches)
    assert 0.10 < tr.time_reduction() < 0.85
    for i, hl in enumerate(levels):
        last = (i + 1) * epochs_per_level - 1               # last epoch of this level
        t = tr.compute_time[last]
        assert max(t) / min(t) < 1.25, (hl, t)
        if hl == 1:
            assert max(tr.batches[last]) - min(tr.batches[last]) <= 4


def test_static_initialisation_starts_near_the_steady_state():
    """Eq. 4a as the open-loop initialiser: batches proportional to cores need almost no correction."""
    tr = S.run_bsp(S.stepwise_schedule([8], 6), 128, 4, 96, 0.10, static_init=True)
    assert tr.batches[0] == [16, 16, 11, 85]
    assert sum(tr.adjustments) <= 1


def test_static_hl8_without_the_global_batch_rule():
    """Sec. IV-D, static heterogeneity: initial batch 32 everywhere, bounds (12, 96), dead-band 15 %,
    no global-batch rule.  The batches settle within the 2-4 adjustment rounds the paper reports
    (here the first round already lands inside the dead-band), the fastest worker peaks at b_max,
    and without Eq. 8 the global batch grows beyond 4 x 32."""
    tr = S.run_bsp(S.stepwise_schedule([8], 12), 128, conserve=False, **S.CONSTANTS_STATIC)
    rounds = [e for e, a in enumerate(tr.adjustments) if a]
    assert rounds and max(rounds) <= 3
    assert tr.batches[-1] == tr.batches[max(rounds) + 1]
    assert max(tr.batches[-1]) == 96 and min(tr.batches[-1]) >= 12
    assert sum(tr.batches[-1]) > 128
    assert tr.iteration_time[-1] < tr.uniform_time[-1]


def test_gpt2_constants_shrink_the_compute_time_spread():
    """Sec. IV-E, the GPT-2 run: b_min 1, b_max 124, dead-band 5 %, heterogeneity stepped HL1 ->
    HL8 -> HL1 every 5 epochs with the global batch kept at 128.  The paper reports a spread
    between slowest and fastest worker under 12 s with the controller against over 22.7 s
    without at HL8; on the model cluster the spread at the end of the HL8 phase must be well
    under half of uniform batching's, and the HL1 phases at both ends run uniform batches."""
    sched = S.stepwise_schedule(S.UP_AND_DOWN, 5)
    tr = S.run_bsp(sched, 128, **S.CONSTANTS_GPT2)
    assert all(sum(b) == 128 and min(b) >= 1 and max(b) <= 124 for b in tr.batches)
    hl8_last = 5 * 5 - 1                                   # epochs 15-24 run HL8
    uniform_spread = max(32 / T for T in sched[hl8_last]) - min(32 / T for T in sched[hl8_last])
    assert uniform_spread == 7.0
    assert tr.spread(hl8_last) < 0.5 * uniform_spread / 2
    assert tr.spread(hl8_last) < tr.spread(15)             # and it shrank over the phase
    assert tr.batches[0] == tr.batches[4] == [32, 32, 32, 32]
    assert tr.batches[-1] == [32, 32, 32, 32]
    # the worker with the most cores holds the largest batch all through the HL8 phase
    assert all(b[3] == max(b) and b[2] == min(b) for b in tr.batches[16:25])
    assert tr.time_reduction() > 0.10


def test_cluster_of_32_workers():
    """Sec. IV-D, 32 workers (ten each with 2, 4 and 6 cores, one with 16, one with 32): larger
    workers end up with larger batches, the global batch 32 x 32 is kept, and the iteration
    time drops below uniform batching's."""
    cores = list(map(float, S.CLUSTER_32_CORES))
    tr = S.run_bsp([cores] * 10, 32 * 32, **S.CONSTANTS_DYNAMIC)
    b = tr.batches[-1]
    assert all(sum(x) == 1024 and min(x) >= 4 and max(x) <= 96 for x in tr.batches)
    assert max(b[:10]) < min(b[10:20]) and max(b[10:20]) < min(b[20:30]) and max(b[20:30]) < min(b[30:])
    assert sum(tr.adjustments[4:]) == 0                     # steady after a few rounds
    assert tr.iteration_time[-1] < 0.5 * tr.uniform_time[-1]


def test_asynchronous_loop_through_eval_bsz():
    """Algorithm 2 on the ASP core tables, stepped HL1 -> HL8 -> HL1, constants of Sec. IV-E and
    no global-batch rule: batches follow the resources (the 28-core worker runs the largest batch
    in the HL8 phases), every batch respects the bounds, the sum of the batches drifts away from
    4 x 32, and workers with more resources push more updates."""
    sched = S.stepwise_schedule(S.UP_AND_DOWN, 1, S.HL_CORES_ASP)
    tr = S.run_asp(sched, 400.0, 128, **S.CONSTANTS_DYNAMIC)
    assert tr.time == sorted(tr.time) and len(tr.time) > 50
    assert all(4 <= x <= 96 for m in tr.server_map for x in m)
    assert tr.map_at_end_of_phase(0) == [32, 32, 32, 32]                 # HL1: nothing to correct
    for phase in (3, 4):                                                  # HL8: cores (4, 4, 4, 28)
        m = tr.map_at_end_of_phase(phase)
        assert m[3] == max(m) and m[3] >= 2 * max(m[:3])
    assert any(sum(m) != 128 for m in tr.server_map)                      # no conservation in ASP
    assert tr.updates[3] == max(tr.updates)
    # reports carry the batch the worker ran, which need not be the server's current entry for it
    stale = [i for i in range(1, len(tr.time)) if tr.b_used[i] != tr.server_map[i - 1][tr.worker[i]]]
    assert stale, "no report with a batch that differs from the server's entry: the case is not exercised"


def test_asynchronous_loop_equal_resources_changes_nothing():
    tr = S.run_asp([list(map(float, S.HL_CORES_ASP[1]))] * 3, 200.0, 128, **S.CONSTANTS_DYNAMIC)
    assert all(m == [32, 32, 32, 32] for m in tr.server_map)
    assert max(tr.updates) - min(tr.updates) <= 1


def test_traces_serialise_to_json(tmp_path):
    import json

    tr = S.run_bsp(S.stepwise_schedule([1, 8], 3), 128, **S.CONSTANTS_DYNAMIC)
    d = json.loads(tr.to_json(tmp_path / "bsp.json"))
    assert json.loads((tmp_path / "bsp.json").read_text()) == d
    assert d["batches"] == tr.batches and len(d["compute_time"]) == 6
    at = S.run_asp(S.stepwise_schedule([1, 8], 1, S.HL_CORES_ASP), 100.0, 128, **S.CONSTANTS_DYNAMIC)
    d = json.loads(at.to_json(tmp_path / "asp.json"))
    assert d["worker"] == at.worker and d["server_map"] == at.server_map and d["updates"] == at.updates
