"""The replica-time formulas of Section 2.1 and Appendix D agree with each other and with closed forms."""
import math

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from paper_2608_22788_b200 import makespan as mk


@settings(max_examples=60, deadline=None)
@given(lengths=st.lists(st.integers(1, 60), min_size=1, max_size=12), a=st.floats(0.1, 3.0), p=st.floats(0.0, 1.5))
def test_three_forms_of_the_replica_time_agree(lengths, a, p):
    tau = lambda b: a * b ** p if b > 0 else 0.0
    t1 = mk.replica_time_by_intervals(lengths, tau)
    t2 = mk.replica_time_by_marginals(lengths, tau)
    t3 = mk.replica_time_by_positions(lengths, tau)
    assert math.isclose(t1, t2, rel_tol=1e-9) and math.isclose(t1, t3, rel_tol=1e-9)


def test_closed_forms():
    # constant per-step time: the replica finishes with its longest request
    assert mk.replica_time_by_intervals([5, 9, 2], lambda b: 0.5 if b else 0.0) == 4.5
    # tau(b) = b (no batching benefit at all): total = sum of the lengths
    assert mk.replica_time_by_marginals([5, 9, 2], lambda b: float(b)) == 16.0
    # two requests of lengths 10 and 4, tau(1) = 1, tau(2) = 1.5: 4 steps at 1.5 + 6 steps at 1
    tau = lambda b: {0: 0.0, 1: 1.0, 2: 1.5}[b]
    assert mk.replica_time_by_positions([4, 10], tau) == 12.0
    assert mk.marginal_cost(4, 1, tau) == 2.0          # adding the length-4 request to the one holding 10
    assert mk.replica_time_by_intervals([10], tau) + mk.marginal_cost(4, 1, tau) == 12.0


def test_tail_isolation_on_a_long_tailed_pool():
    # 120 requests of 4000 tokens and 8 of 8000; a step costs 1, 1, 2, 4, 5 at b = 1, 2, 8, 32, 64.
    # Uniform round robin over 4 replicas: 30 + 2 each -> 4000 tau(32) + 4000 tau(2) = 20000.
    # 8 longest on one tail replica, the rest on three bulk replicas: max(8000 tau(8), 4000 tau(40)).
    tau = mk.tau_from_samples([1, 2, 8, 32, 64], [1.0, 1.0, 2.0, 4.0, 5.0])
    lengths = [8000 if i % 17 == 0 else 4000 for i in range(128)]      # two long ones per replica under round robin
    uniform = mk.step_makespan(mk.round_robin(lengths, 4), tau)
    assert uniform == pytest.approx(4000 * tau(32) + 4000 * tau(2))
    isolated = mk.step_makespan(mk.topk_isolation(lengths, 8, 1, 3), tau)
    assert isolated == pytest.approx(max(8000 * tau(8), 4000 * tau(40)))
    assert isolated < uniform
    k, t_best, t_uniform = mk.best_topk(lengths, tau, tail_replicas=1, bulk_replicas=3, ks=range(1, 64))
    assert t_uniform == uniform and t_best <= isolated and 1 <= k <= 40
    # too few isolated: the bulk replicas still carry long requests; too many: the tail replica is the slow one
    few = mk.step_makespan(mk.topk_isolation(lengths, 2, 1, 3), tau)
    many = mk.step_makespan(mk.topk_isolation(lengths, 60, 1, 3), tau)
    assert t_best < few and t_best < many


def test_tau_interpolation():
    tau = mk.tau_from_samples([1, 4, 16], [10.0, 12.0, 20.0])
    assert tau(0) == 0.0 and tau(1) == 10.0 and tau(4) == 12.0 and tau(2) == pytest.approx(11.0)
    assert tau(1000) == 20.0
