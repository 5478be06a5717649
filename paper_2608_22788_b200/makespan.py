"""Replica completion times under the paper's all-admit decode model (host-side, scalar).

Consumer of the measured curve tau(b) = time of one decode step with b active requests
(``bench.py``'s concurrency sweep): evaluates how long a replica takes to finish a set of requests
with known lengths, and what top-k tail isolation buys on a length pool.  Section 2.1 gives the
completion time of one replica in two equivalent forms; Appendix D gives the exact per-position sum
and the step makespan as the maximum over replicas; Section 2.2 describes top-k tail isolation.
None of this runs on the GPU.
"""
from __future__ import annotations

from typing import Callable, Sequence

import numpy as np

Tau = Callable[[int], float]


def tau_from_samples(batch_sizes: Sequence[int], step_times: Sequence[float]) -> Tau:
    """Piecewise-linear tau(b) through measured (b, seconds per step) points, tau(0) = 0,
    linear in log b between samples and flat beyond the last one."""
    b = np.asarray(batch_sizes, dtype=np.float64)
    t = np.asarray(step_times, dtype=np.float64)
    order = np.argsort(b)
    lb, t = np.log(b[order]), t[order]

    def tau(n: int) -> float:
        if n <= 0:
            return 0.0
        return float(np.interp(np.log(n), lb, t))

    return tau


def replica_time_by_intervals(lengths: Sequence[int], tau: Tau) -> float:
    """T_total = sum_j tau(j) (L_j - L_{j+1}), lengths sorted descending, L_{n+1} = 0 (Section 2.1):
    while the j longest requests are still active, every step costs tau(j)."""
    L = sorted((int(x) for x in lengths), reverse=True) + [0]
    return float(sum(tau(j) * (L[j - 1] - L[j]) for j in range(1, len(L))))


def replica_time_by_marginals(lengths: Sequence[int], tau: Tau) -> float:
    """T_total = sum_j L_j (tau(j) - tau(j-1)), tau(0) = 0 (Section 2.1, the same sum regrouped):
    the j-th longest request adds its length times the extra per-step time of a batch of j."""
    L = sorted((int(x) for x in lengths), reverse=True)
    return float(sum(L[j - 1] * (tau(j) - tau(j - 1)) for j in range(1, len(L) + 1)))


def replica_time_by_positions(lengths: Sequence[int], tau: Tau) -> float:
    """T_r = sum over decoding positions x of tau(b_r(x)), b_r(x) = number of requests with
    L_i >= x (Appendix D): the definition, one term per position."""
    L = np.asarray(list(lengths), dtype=np.int64)
    if L.size == 0:
        return 0.0
    return float(sum(tau(int((L >= x).sum())) for x in range(1, int(L.max()) + 1)))


def marginal_cost(length: int, longer_requests: int, tau: Tau) -> float:
    """Delta T(L, c) = L (tau(c+1) - tau(c)): cost of adding a request of length L to a replica that
    already holds c longer ones (Section 2.1)."""
    return float(length * (tau(longer_requests + 1) - tau(longer_requests)))


def step_makespan(assignment: Sequence[Sequence[int]], tau: Tau) -> float:
    """max over replicas of their completion time (Appendix D)."""
    return max((replica_time_by_intervals(r, tau) for r in assignment), default=0.0)


def round_robin(lengths: Sequence[int], replicas: int):
    """Requests dealt to replicas in arrival order (the dispatcher inside a pool, Section 3.1)."""
    out = [[] for _ in range(replicas)]
    for i, x in enumerate(lengths):
        out[i % replicas].append(int(x))
    return out


def topk_isolation(lengths: Sequence[int], k: int, tail_replicas: int, bulk_replicas: int):
    """The k longest requests go to the tail pool, the rest to the bulk pool; round robin inside
    each pool (Section 2.2 with known lengths)."""
    order = sorted(range(len(lengths)), key=lambda i: -int(lengths[i]))
    tail = [int(lengths[i]) for i in order[:k]]
    bulk = [int(lengths[i]) for i in sorted(order[k:])]
    return round_robin(tail, tail_replicas) + round_robin(bulk, bulk_replicas)


def best_topk(lengths: Sequence[int], tau: Tau, tail_replicas: int, bulk_replicas: int, ks=None):
    """Sweep k; returns (best k, its makespan, makespan of uniform round robin over all replicas)."""
    n = len(lengths)
    base = step_makespan(round_robin(lengths, tail_replicas + bulk_replicas), tau)
    best = (0, base)
    for k in (ks if ks is not None else range(1, n)):
        t = step_makespan(topk_isolation(lengths, k, tail_replicas, bulk_replicas), tau)
        if t < best[1]:
            best = (k, t)
    return best[0], best[1], base
