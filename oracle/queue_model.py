"""Oracle of the paper's analytical model (Sections 4 and 5) -- TEST INFRASTRUCTURE, not the product.

Plain restatements of the printed formulas, pinned in the tests against the paper's own tables
(tests/golden/*.txt).  No code is shared with the library's model.
"""
from __future__ import annotations

import math


def outer_product_throughput(rates, jobs):
    """Section 4, "Little's Law": outer products per cycle = min over pipelines of rate_i / jobs_i.

    Pipelines with no job do not constrain the result."""
    best = math.inf
    for r, l in zip(rates, jobs):
        if l > 0:
            best = min(best, r / l)
    return best


def stalled_throughput(jobs, n_dependent, latency):
    """Section 4, "Estimating throughput": a pipeline whose n dependent instructions of latency k cannot be
    overlapped waits W = L + n*k cycles for its L jobs, so it completes 1/W outer products per cycle."""
    return 1.0 / (jobs + n_dependent * latency)


def flop_per_cycle(lam, mr, nr):
    """Section 6.1: flop/cycle = lambda * mr * nr * 2."""
    return lam * mr * nr * 2.0


def gflops(freq_ghz, fpc):
    """Section 6.1: GFLOP/s = f * flop/cycle."""
    return freq_ghz * fpc


def n_updates(r_total, mr, nr, v, r_a, r_r):
    """Section 5, "Limits imposed by registers": floor((R_total - mr*nr/v - R_A) / R_R)."""
    return math.floor((r_total - (mr * nr) / v - r_a) / r_r)


def sub_block_fits(ms, ns, updates, v):
    """Section 5: the sub-block must satisfy ms*ns <= N_updates * v."""
    return ms * ns <= updates * v
