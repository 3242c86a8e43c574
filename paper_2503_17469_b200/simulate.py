"""Closed-loop simulation of the batch-size controller on a model cluster.

The controller of the library (host code behind ``omni_rebatch`` / ``omni_asp_report``) is driven
by a simple cluster model: worker k processes ``T_k`` samples per time unit, where ``T_k`` is
proportional to the resources it holds at that moment (for example the CPU-core tables of the
paper's heterogeneity levels), so one iteration with batch ``b_k`` takes ``b_k / T_k``.

* ``run_bsp``: the synchronous loop of Algorithm 1.  Each epoch the workers report their
  throughput, the controller answers with new batches, and the trace records batches, per-worker
  compute times and the synchronous iteration time (the slowest worker).
* ``run_asp``: the asynchronous loop of Algorithm 2.  Every worker iterates at its own pace; after
  each of its epochs it reports its batch and mean compute time through ``omni_asp_report``
  (evalBsz) and continues with the batch the server returns.  The trace records every report in
  time order, the server's batch map after it, and how many updates each worker pushed.

The module only drives the library and keeps books; every batch size comes out of the library's
controller.  Needs no GPU.  Traces serialise to JSON (``Trace.to_json``).
"""
from __future__ import annotations

import heapq
import json
from dataclasses import asdict, dataclass, field
from typing import List, Optional, Sequence

from . import binding as B

# CPU cores per worker at the paper's heterogeneity levels (its Table I)
HL_CORES_BSP = {1: (12, 12, 12, 12), 2: (12, 12, 8, 16), 4: (9, 9, 6, 24), 8: (6, 6, 4, 32)}
HL_CORES_ASP = {1: (10, 10, 10, 10), 2: (8, 8, 8, 16), 4: (10, 10, 4, 16), 8: (4, 4, 4, 28)}
# The 32-worker cluster of Sec. IV-D: ten workers each with 2, 4 and 6 cores, one with 16, one with 32
CLUSTER_32_CORES = (2,) * 10 + (4,) * 10 + (6,) * 10 + (16, 32)
# Heterogeneity is stepped from HL1 up to HL8 and back (Sec. IV-E); the HL8 phase lasts two steps
UP_AND_DOWN = (1, 2, 4, 8, 8, 4, 2, 1)
# Controller constants of the paper's experiments: (b_min, b_max, dead-band)
CONSTANTS_STATIC = dict(b_min=12, b_max=96, deadband=0.15)     # Sec. IV-D, static heterogeneity, no global-batch rule
CONSTANTS_DYNAMIC = dict(b_min=4, b_max=96, deadband=0.10)     # Sec. IV-E, dynamic heterogeneity, B = 128 kept
CONSTANTS_GPT2 = dict(b_min=1, b_max=124, deadband=0.05)       # Sec. IV-E, GPT-2 run


@dataclass
class Trace:
    batches: List[List[int]] = field(default_factory=list)        # per epoch, the batches used in it
    compute_time: List[List[float]] = field(default_factory=list)  # per epoch, b_k / T_k
    iteration_time: List[float] = field(default_factory=list)      # per epoch, max_k compute time (BSP barrier)
    uniform_time: List[float] = field(default_factory=list)        # same epoch with uniform batches B / K
    adjustments: List[int] = field(default_factory=list)           # per epoch, workers whose batch changed

    def time_reduction(self) -> float:
        """Fraction of synchronous training time saved against uniform batching over the run."""
        return 1.0 - sum(self.iteration_time) / sum(self.uniform_time)

    def spread(self, epoch: int) -> float:
        """Slowest minus fastest worker's compute time in an epoch."""
        t = self.compute_time[epoch]
        return max(t) - min(t)

    def to_json(self, path=None) -> str:
        text = json.dumps(asdict(self))
        if path is not None:
            with open(path, "w") as f:
                f.write(text)
        return text


def run_bsp(schedule: Sequence[Sequence[float]], global_batch: int, b_min: int, b_max: int, deadband: float = 0.10,
            ewma_alpha: float = 1.0, static_init: bool = False, conserve: bool = True, flags: int = 0) -> Trace:
    """``schedule[e][k]``: throughput of worker k during epoch e.  Batches for epoch e+1 are
    computed at the end of epoch e from what was measured in it (Algorithm 1).  ``conserve=False``
    drops the global-batch rule of Eq. 8 (the paper's static-heterogeneity experiment runs without
    it): the same getBsz for all workers at once, on a context without that rule."""
    K = len(schedule[0])
    ctl = B.Omni(K, global_batch, b_min, b_max, deadband, ewma_alpha, B.BSP if conserve else B.ASP, flags)
    b = ctl.rebatch_static(list(schedule[0])) if static_init else ctl.batches
    tr = Trace()
    for T in schedule:
        tr.batches.append(list(b))
        t = [bk / Tk for bk, Tk in zip(b, T)]
        tr.compute_time.append(t)
        tr.iteration_time.append(max(t))
        tr.uniform_time.append(max((global_batch / K) / Tk for Tk in T))
        b, changed = ctl.rebatch(list(T))
        tr.adjustments.append(sum(changed))
    return tr


def stepwise_schedule(levels: Sequence[int], epochs_per_level: int, table=HL_CORES_BSP) -> List[List[float]]:
    """The paper's dynamic-heterogeneity pattern: hold each level for a fixed number of epochs."""
    out: List[List[float]] = []
    for hl in levels:
        out += [list(map(float, table[hl]))] * epochs_per_level
    return out


@dataclass
class AspTrace:
    time: List[float] = field(default_factory=list)          # wall time of every report, ascending
    worker: List[int] = field(default_factory=list)          # who reported
    b_used: List[int] = field(default_factory=list)          # the batch it ran during that epoch
    compute_time: List[float] = field(default_factory=list)  # its mean time per iteration in that epoch
    new_b: List[int] = field(default_factory=list)           # what evalBsz returned to it
    server_map: List[List[int]] = field(default_factory=list)  # the server's wrkB after the report
    updates: List[int] = field(default_factory=list)         # per worker: parameter pushes over the whole run
    phase: List[int] = field(default_factory=list)           # index of the schedule entry in force at the report

    def map_at_end_of_phase(self, phase: int) -> List[int]:
        """The server's batch map after the last report made during a schedule phase."""
        idx = [i for i, p in enumerate(self.phase) if p == phase]
        return self.server_map[idx[-1]]

    def to_json(self, path=None) -> str:
        text = json.dumps(asdict(self))
        if path is not None:
            with open(path, "w") as f:
                f.write(text)
        return text


def run_asp(schedule: Sequence[Sequence[float]], phase_time: float, global_batch: int, b_min: int, b_max: int,
            deadband: float = 0.10, ewma_alpha: float = 1.0, iterations_per_epoch: int = 20, flags: int = 0,
            initial_batch: Optional[int] = None) -> AspTrace:
    """The asynchronous loop of Algorithm 2 on the model cluster.  ``schedule[p][k]`` is worker k's
    throughput during phase p; every phase lasts ``phase_time`` time units and the run ends with the
    last phase.  A worker runs ``iterations_per_epoch`` iterations per epoch (each pushes one update
    and takes b_k / T_k at the throughput in force when it starts), then reports the batch it ran
    and its mean time per iteration, and adopts the returned batch.  No global-batch rule."""
    K = len(schedule[0])
    ctl = B.Omni(K, global_batch, b_min, b_max, deadband, ewma_alpha, B.ASP, flags | B.INPUT_IS_TIME)
    b = [initial_batch or global_batch // K] * K
    end = phase_time * len(schedule)
    tr = AspTrace(updates=[0] * K)

    def run_epoch(k: int, start: float):
        """Advance worker k by one epoch; returns (finish time, mean iteration time, iterations done)."""
        now, spent, done = start, 0.0, 0
        for _ in range(iterations_per_epoch):
            if now >= end:
                break
            T = schedule[min(int(now / phase_time), len(schedule) - 1)][k]
            dt = b[k] / T
            now += dt
            spent += dt
            done += 1
        return now, (spent / done if done else 0.0), done

    heap = []
    for k in range(K):
        fin, mean_t, done = run_epoch(k, 0.0)
        if done:
            heapq.heappush(heap, (fin, k, mean_t, done))
    while heap:
        fin, k, mean_t, done = heapq.heappop(heap)
        tr.updates[k] += done
        used = b[k]
        b[k] = ctl.asp_report(k, used, mean_t)
        tr.time.append(fin)
        tr.worker.append(k)
        tr.b_used.append(used)
        tr.compute_time.append(mean_t)
        tr.new_b.append(b[k])
        tr.server_map.append(ctl.batches)
        tr.phase.append(min(int(min(fin, end - 1e-12) / phase_time), len(schedule) - 1))
        if fin < end:
            nfin, nmean, ndone = run_epoch(k, fin)
            if ndone:
                heapq.heappush(heap, (nfin, k, nmean, ndone))
    return tr
