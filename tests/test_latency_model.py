"""Run-time model of Section III-C: the oracle against hand-worked cases, the closed form of
Appendix D and elementary bounds; then the library's host routine against the oracle."""
import numpy as np
import pytest

from oracle import cr_oracle as O
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import build as cr_build
from paper_1902_01981_b200 import inputs


@pytest.fixture(scope="module", autouse=True)
def built():
    cr_build.build()


def test_hand_worked_single_group():
    # three workers, one straggler tolerated, times 1, 2, 10, a message takes 0.5:
    # worker 1 is received at 1.5, worker 2 at 2.5: done at 2.5 without worker 3
    masks, T = O.latency_trial(3, 1, 1, [1.0, 2.0, 10.0], 0.5)
    assert masks == [0b100] and T == 2.5
    # the port is the bottleneck when messages are ready together: 1, 1, 1 -> received at 1.5 and 2.0
    masks, T = O.latency_trial(3, 1, 1, [1.0, 1.0, 1.0], 0.5)
    assert masks == [0b100] and T == 2.0            # ties: lower index first
    # no communication cost: the (n-s)-th order statistic
    masks, T = O.latency_trial(4, 1, 2, [7.0, 3.0, 9.0, 5.0], 0.0)
    assert masks == [0b0101] and T == 5.0


def test_hand_worked_two_layers():
    # (2,2) tree, s = 1: each parent needs one child.  leaves of (1,1): 4, 1; of (1,2): 2, 8; t_c = 1
    # (1,1): child 2 ready 1 -> received 2; own computation 3 -> message ready 3
    # (1,2): child 1 ready 2 -> received 3; own computation 0.5 -> ready 3
    # master: tie at 3 -> (1,1) first, received 4: done at 4, (1,2) not waited for
    ct = [3.0, 0.5, 4.0, 1.0, 2.0, 8.0]
    masks, T = O.latency_trial(2, 2, 1, ct, 1.0)
    assert masks == [0b10, 0b01, 0b10] and T == 4.0


def test_order_statistic_mean_matches_appendix_d():
    n, s, load, a, mu = 12, 3, 42.0, 5e-3, 2.0
    times = inputs.shifted_exponential_times(n, load, a, mu, seed=0, trials=40000)
    got = np.mean([O.latency_trial(n, 1, s, t, 0.0)[1] for t in times])
    want = O.expected_order_statistic(n, s, load, a, mu)
    assert abs(got - want) <= 0.01 * want
    # sanity of the closed form itself: s = 0 is the expected maximum, H_n scaling
    assert abs(O.expected_order_statistic(1, 0, 1.0, 0.0, 1.0) - 1.0) < 1e-15
    assert np.all(times >= a * load)


@pytest.mark.parametrize("n,L,s", [(3, 2, 1), (4, 3, 1), (5, 2, 2), (12, 2, 3)])
def test_bounds_and_mask_shape(n, L, s):
    N = O.num_nodes(n, L)
    times = inputs.shifted_exponential_times(N, 10.0, 0.01, 1.0, seed=n + L, trials=50)
    t_c = 0.3
    for t in times:
        masks, T = O.latency_trial(n, L, s, t, t_c)
        assert all(bin(m).count("1") == s for m in masks)
        # nothing can finish before the fastest leaf plus one message per layer, nor after every node
        # has computed and every parent has listened to n messages per layer
        assert T >= t[O.layer_offset(n, L):].min() + L * t_c - 1e-12
        assert T <= t.max() + n * L * t_c + 1e-12
        # no communication cost and no stragglers tolerated: everybody waits for the slowest node
        assert O.latency_trial(n, L, 0, t, 0.0)[1] == t.max()


@pytest.mark.parametrize("n,L,s,code", [(3, 2, 1, B.CR_CODE_PAPER_3_1), (4, 3, 1, B.CR_CODE_CYCLIC_RANDOM),
                                        (5, 2, 2, B.CR_CODE_CYCLIC_RANDOM), (4, 2, 1, B.CR_CODE_FRACTIONAL_REPETITION)])
def test_library_matches_oracle(n, L, s, code):
    plan = B.cr_plan_create(n, L, s, O.partition_quantum(n, L, s), 64, code=code, device=-1)
    try:
        N = O.num_nodes(n, L)
        times = inputs.shifted_exponential_times(N, 25.0, 0.002, 1.5, seed=3, trials=200)
        times[7] = np.round(times[7])          # some exact ties
        for t in times:
            masks, T = B.cr_latency_masks(plan, t, 0.05)
            want_masks, want_T = O.latency_trial(n, L, s, t, 0.05)
            assert masks.tolist() == want_masks and T == pytest.approx(want_T, rel=1e-14)
            nodes, _, _ = B.cr_plan_expand(plan, masks)      # every such pattern is decodable
            assert len(nodes) > 0
        with pytest.raises(B.CodedReduceError):
            B.cr_latency_masks(plan, -np.ones(N), 0.1)
    finally:
        B.cr_plan_destroy(plan)


@pytest.mark.parametrize("n,L,s", [(4, 2, 1), (12, 2, 3), (6, 3, 2)])
def test_communication_term_lies_between_the_bounds_of_theorem_2(n, L, s):
    """With instant computations the run time is pure communication: every parent hears n-s messages
    one after the other, layer after layer: T = L (n-s) t_c.  Theorem 2's communication terms bracket
    it: (n(1-alpha) + L - 1) t_c from below (the master's n-s receptions after one message per lower
    layer), n L t_c from above."""
    t_c = 0.25
    N = O.num_nodes(n, L)
    masks, T = O.latency_trial(n, L, s, np.zeros(N), t_c)
    assert T == pytest.approx(L * (n - s) * t_c)
    assert (n - s + L - 1) * t_c <= T <= n * L * t_c
    # the stragglers are then the highest-indexed s children of every group (ties: lower index first)
    assert all(m == sum(1 << j for j in range(n - s, n)) for m in masks)


def test_expected_run_time_against_theorem_2_at_finite_n():
    """E[T_CR] sampled on the (12,2) tree with alpha = 1/4.  Theorem 2's computation term, with the exact
    order-statistic mean (H_n - H_s) of Appendix D in place of its limit log(1/alpha), plus one message
    time bounds it from below (the master waits for the (n-s)-th of its children, whose own
    computations alone take that long, and then receives a message); the expected slowest of all N
    computations plus the theorem's n L t_c bounds it from above."""
    n, L, s, a, mu, t_c = 12, 2, 3, 1e-3, 1.0, 0.05
    P = O.partition_quantum(n, L, s)
    load = O.computation_load(n, L, s) * P            # data units per worker, r_CR * d
    N = O.num_nodes(n, L)
    times = inputs.shifted_exponential_times(N, load, a, mu, seed=5, trials=3000)
    mean_T = float(np.mean([O.latency_trial(n, L, s, t, t_c)[1] for t in times]))
    stat_err = 4.0 * (load / mu) / np.sqrt(3000)      # four standard errors of a sample mean, generously
    assert O.expected_order_statistic(n, s, load, a, mu) + t_c <= mean_T + stat_err
    assert mean_T <= O.expected_order_statistic(N, 0, load, a, mu) + n * L * t_c + stat_err
    # and the communication share is of the order the theorem states: between (n-s) and n L message times
    no_comm = float(np.mean([O.latency_trial(n, L, s, t, 0.0)[1] for t in times]))
    assert t_c <= mean_T - no_comm <= n * L * t_c
