"""The paper's latency / compute model (Section 4) -- part of the oracle, test infrastructure only.

Symbols: d layers, early layer l (paper: d-bar), n generated tokens (paper: l), k candidates,
p = p_correct.  b = min(l, d - l) is the number of layers a branch has finished when it is
verified; the paper's analysis assumes l >= d/2 where b = d - l.  One layer = one time unit.

`*_closed` functions restate the printed formulas; `enumerate_expectation` gets the same
quantities by brute force over all hit patterns, with exact rational arithmetic.
"""
from __future__ import annotations

from fractions import Fraction
from itertools import product


def branch_depth(d: int, l: int) -> int:
    return min(l, d - l)


# ---- approximate analysis, l = d/2, n >> 1 (Section 4.2)

def per_token_latency_approx(d, p):
    """Per-token latency d (1 - p/2)."""
    return d * (1 - Fraction(p) / 2) if isinstance(p, Fraction) else d * (1 - p / 2)


def avg_compute_per_time_unit(k, p):
    """(k + 2 - p) / (2 - p)."""
    return (k + 2 - p) / (2 - p)


def compute_per_token_approx(k, p):
    """(2 + k - p) / 2, per-token latency times average compute, in units of d."""
    return (2 + k - p) / 2


# ---- exact analysis (Theorem 4.1)

def expected_latency_closed(d, l, n, p):
    """d n - b (n - 1) p."""
    return d * n - branch_depth(d, l) * (n - 1) * p


def expected_compute_closed(d, l, n, k, p):
    """d n - b (n - 1) p + k b n."""
    return expected_latency_closed(d, l, n, p) + k * branch_depth(d, l) * n


def run_time(d, l, x):
    """Time to generate a run of x tokens: d + (x - 1)(d - b)  (T_X in the proof)."""
    return d + (x - 1) * (d - branch_depth(d, l))


def realised_units(d, l, k, hits):
    """Latency and compute units of one concrete generation given its per-step hit flags
    (hit[s] = early candidates of step s contained the final token).  A step that follows a
    hit starts at layer b; the hit flag of the last step saves nothing."""
    n = len(hits)
    b = branch_depth(d, l)
    lat = 0
    prev = False
    for s in range(n):
        lat += d - b if prev else d
        prev = bool(hits[s])
    return lat, lat + k * b * n


def runs_from_hits(hits):
    """Split n tokens into runs: a new run starts after every miss among the first n-1 steps."""
    runs, cur = [], 1
    for hflag in hits[:-1]:
        if hflag:
            cur += 1
        else:
            runs.append(cur)
            cur = 1
    runs.append(cur)
    return runs


def enumerate_expectation(d, l, n, k, p: Fraction):
    """Brute force over all 2^(n-1) hit patterns of the first n-1 steps (independent, each a hit
    with probability p).  Returns exact (E[latency], E[compute], E[number of runs])."""
    p = Fraction(p)
    e_lat = e_cmp = e_runs = Fraction(0)
    for pattern in product((0, 1), repeat=n - 1):
        prob = Fraction(1)
        for z in pattern:
            prob *= p if z else 1 - p
        hits = list(pattern) + [0]
        lat, cmp_ = realised_units(d, l, k, hits)
        runs = runs_from_hits(hits)
        assert sum(runs) == n
        assert lat == sum(run_time(d, l, x) for x in runs)
        e_lat += prob * lat
        e_cmp += prob * cmp_
        e_runs += prob * len(runs)
    return e_lat, e_cmp, e_runs
