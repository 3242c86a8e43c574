"""Closed-loop simulation of the batch-size controller on a model cluster.

The controller of the library (host code behind ``omni_rebatch`` / ``omni_asp_report``) is driven
by a simple cluster model: worker k processes ``T_k`` samples per time unit, where ``T_k`` is
proportional to the resources it holds during that epoch (for example the CPU-core tables of the
paper's heterogeneity levels), so one iteration with batch ``b_k`` takes ``b_k / T_k``.  Each epoch
the workers report their throughput, the controller answers with new batches, and the trace
records batches, per-worker compute times and the synchronous iteration time (the slowest
worker).  Needs no GPU: only the controller part of the C-ABI library is used.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence

from . import binding as B

# CPU cores per worker at the paper's heterogeneity levels (its Table I, BSP rows)
HL_CORES_BSP = {1: (12, 12, 12, 12), 2: (12, 12, 8, 16), 4: (9, 9, 6, 24), 8: (6, 6, 4, 32)}
HL_CORES_ASP = {1: (10, 10, 10, 10), 2: (8, 8, 8, 16), 4: (10, 10, 4, 16), 8: (4, 4, 4, 28)}


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


def run_bsp(schedule: Sequence[Sequence[float]], global_batch: int, b_min: int, b_max: int, deadband: float = 0.10,
            ewma_alpha: float = 1.0, static_init: bool = False) -> Trace:
    """``schedule[e][k]``: throughput of worker k during epoch e.  Batches for epoch e+1 are
    computed at the end of epoch e from what was measured in it (Algorithm 1)."""
    K = len(schedule[0])
    ctl = B.Omni(K, global_batch, b_min, b_max, deadband, ewma_alpha, B.BSP)
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
