"""The pins are only worth something if a plausible mistake in the oracle fails one of them.
This test plants mistakes (a wrong sign, a dropped term, a transposed operand, a wrong index, a
wrong comparison) one at a time in a COPY of the oracle source, builds the copy, and runs the pin
modules against it in a child process: every mutant must be caught."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parents[1]
SRC = (ROOT / "oracle" / "omni_oracle.c").read_text()

MUTANTS = [
    ("weights divide by the wrong total", "return (double)b[k] / (double)B;", "return (double)b[k] / (double)(B + 1);"),
    ("weights ignore the batches", "return (double)b[k] / (double)B;", "return 1.0 / (double)K;"),
    ("controller correction has the wrong sign", "double bstar = (double)b - T * err;", "double bstar = (double)b + T * err;"),
    ("error measured against the sum, not the mean", "double tbar = tsum / (double)w.K;", "double tbar = tsum;"),
    ("dead-band relative to the old batch", "fabs((bstar - (double)b) / bstar) >= c->deadband", "fabs((bstar - (double)b) / (double)b) >= c->deadband"),
    ("dead-band threshold exclusive", "fabs((bstar - (double)b) / bstar) >= c->deadband", "fabs((bstar - (double)b) / bstar) > c->deadband"),
    ("a batch above the upper bound is sent to the lower bound", "else if (bstar > (double)c->b_max) cand = (double)c->b_max;", "else if (bstar > (double)c->b_max) cand = (double)c->b_min;"),
    ("truncation instead of rounding", "double r = floor(cand + 0.5);", "double r = floor(cand);"),
    ("leftover units go to the smallest batches", "if (best < 0 || n[k] > n[best]) best = k;", "if (best < 0 || n[k] < n[best]) best = k;"),
    ("ties go to the highest index", "if (best < 0 || n[k] > n[best]) best = k;", "if (best < 0 || n[k] >= n[best]) best = k;"),
    ("pinned workers keep moving", "if (dir > 0 ? n[k] < c->b_max : n[k] > c->b_min) movable[m++] = k;", "movable[m++] = k;"),
    ("EWMA weights swapped", "else c->s[k] = c->alpha * x + (1.0 - c->alpha) * c->s[k];", "else c->s[k] = (1.0 - c->alpha) * x + c->alpha * c->s[k];"),
    ("throughput read as time", "return (double)b / measured;", "return measured;"),
    ("momentum multiplies the new term too", "if (v) { vn = mu * v[j] + d; v[j] = vn; }\n        theta[j] = theta[j] - lr * vn;\n        sq += gbar * gbar;",
     "if (v) { vn = mu * (v[j] + d); v[j] = vn; }\n        theta[j] = theta[j] - lr * vn;\n        sq += gbar * gbar;"),
    ("weight decay dropped", "double d = gbar + wd * theta[j];", "double d = gbar;"),
    ("update has the wrong sign", "theta[j] = theta[j] - lr * vn;\n        sq += gbar * gbar;", "theta[j] = theta[j] + lr * vn;\n        sq += gbar * gbar;"),
    ("norm of the decayed gradient", "sq += gbar * gbar;", "sq += d * d;"),
    ("float chain: momentum operands transposed", "if (mu != 0.0f) vn = fmaf(mu, v[j], d);\n        if (v) v[j] = vn;\n        theta[j] = fmaf(-lr, vn, theta[j]);",
     "if (mu != 0.0f) vn = fmaf(mu, d, v[j]);\n        if (v) v[j] = vn;\n        theta[j] = fmaf(-lr, vn, theta[j]);"),
    ("float chain: workers in descending order", "for (int k = 0; k < K; ++k) acc = fmaf(lam[k], (float)grad_at(g, dtype_bf16, k, j), acc);",
     "for (int k = K - 1; k >= 0; --k) acc = fmaf(lam[k], (float)grad_at(g, dtype_bf16, k, j), acc);"),
    ("asynchronous rate scaled the wrong way round", "return lr * (double)b_used / (double)B;", "return lr * (double)B / (double)b_used;"),
    ("bfloat16 rounds half up, not half to even", "u += 0x7fffu + lsb;", "u += 0x8000u;"),
    ("overwrite starts from the server copy", "theta[j] = snapshot[j] - eta_k * d;", "theta[j] = theta[j] - eta_k * d;"),
    ("static split ignores the capacities", "double x = capacity[k] / csum * (double)c->B;", "double x = (double)c->B / (double)c->K;"),
    ("asynchronous report keeps the server's entry instead of the batch the worker ran", "c->b[worker] = b_used;\n    smooth(c, worker,", "smooth(c, worker,"),
    ("asynchronous report skips the smoothing", "smooth(c, worker, measured_time(c, b_used, measured));",
     "c->s[worker] = measured_time(c, b_used, measured); c->seen[worker] = 1;"),
    ("asynchronous report takes the time from the server's entry", "c->b[worker] = b_used;\n    smooth(c, worker, measured_time(c, b_used, measured));",
     "smooth(c, worker, measured_time(c, c->b[worker], measured));\n    c->b[worker] = b_used;"),
    ("multiplicative conservation divides by the global batch, not by the sum of the proposals", "double scaled = cand[k] * (double)w.B / csum;", "double scaled = cand[k] * (double)w.B / (double)w.B;"),
    ("multiplicative conservation scales the wrong way round", "double scaled = cand[k] * (double)w.B / csum;", "double scaled = cand[k] * csum / (double)w.B;"),
    ("multiplicative conservation sums the old batches", "for (int k = 0; k < w.K; ++k) csum += cand[k];", "for (int k = 0; k < w.K; ++k) csum += (double)w.b[k];"),
    ("asynchronous report re-batches before everyone reported", "if (!all) { *new_b = b_used; return ORACLE_OK; }", "if (!all && worker < 0) { *new_b = b_used; return ORACLE_OK; }"),
]


def _caught(args):
    idx, (name, old, new), tmp = args
    assert SRC.count(old) >= 1, f"mutation target not found: {name}"
    src = tmp / f"mutant{idx}.c"
    lib = tmp / f"mutant{idx}.so"
    src.write_text(SRC.replace(old, new, 1))
    subprocess.run(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-o", str(lib), str(src), "-lm"],
                   check=True)
    env = dict(os.environ, OMNI_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        str(ROOT / "tests" / "test_oracle_controller.py"), str(ROOT / "tests" / "test_oracle_update.py")],
                       env=env, capture_output=True, text=True, cwd=str(ROOT))
    return name, r.returncode != 0


def test_every_planted_mistake_fails_a_pin(tmp_path):
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as ex:
        results = list(ex.map(_caught, [(i, m, tmp_path) for i, m in enumerate(MUTANTS)]))
    survivors = [name for name, caught in results if not caught]
    assert not survivors, f"mistakes no pin caught: {survivors}"
