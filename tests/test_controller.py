"""Streaming controller (Section 3.2.3): the oracle's Bellman recursion against what the mathematics fixes, and the
library's host-side table builder against the oracle (no GPU needed: the controller is CPU-side in the paper too)."""
import itertools
import math

import numpy as np
import pytest

from oracle import leanstream_oracle as orc


def random_tables(rng, N, Q, A, S, forbid=0.2):
    t = rng.uniform(0.5, 3.0, size=(N, Q, A))
    t[rng.random((N, Q, A)) < forbid] = np.inf
    t[:, :, 0] = np.where(np.isinf(t[:, :, 0]), 1.7, t[:, :, 0])  # plan 0 is always allowed
    ns = rng.integers(0, Q, size=(N, Q, A, S))
    ns[rng.random((N, Q, A, S)) < 0.1] = -1
    return t, ns


def test_quantizer_bins():
    assert [orc.quantize_state(v, 8.0, 4) for v in (-1.0, 0.0, 0.1, 1.99, 2.0, 5.9, 6.0, 8.0, 100.0)] == [0, 0, 0, 0, 1, 2, 3, 3, 3]
    with pytest.raises(ValueError):
        orc.quantize_state(1.0, 0.0, 4)


def test_horizon_one_is_the_greedy_plan():
    """V^1(q) = min_a t_bar: with a horizon of one layer the table is the cheapest allowed plan of every state."""
    rng = np.random.default_rng(0)
    t, ns = random_tables(rng, 5, 6, 4, 3)
    lut, val = orc.controller_lut(t, ns, 1)
    assert lut.tolist() == np.argmin(t, axis=2).tolist()
    np.testing.assert_array_equal(val, np.min(t, axis=2))


def test_deterministic_transitions_equal_brute_force_over_plan_sequences():
    """One sample per configuration makes the transition deterministic: V_n^H(q) must equal the cheapest total time over all
    plan sequences of length min(H, layers left), enumerated exhaustively."""
    rng = np.random.default_rng(1)
    N, Q, A, H = 4, 3, 3, 3
    t, ns = random_tables(rng, N, Q, A, 1, forbid=0.15)
    ns = np.abs(ns)  # every sample used
    lut, val = orc.controller_lut(t, ns, H)
    for n in range(N):
        for q in range(Q):
            steps = min(H, N - n)
            best, best_first = math.inf, -1
            for seq in itertools.product(range(A), repeat=steps):
                cost, state, ok = 0.0, q, True
                for i, a in enumerate(seq):
                    if math.isinf(t[n + i, state, a]):
                        ok = False
                        break
                    cost += t[n + i, state, a]
                    state = int(ns[n + i, state, a, 0])
                if ok and cost < best - 1e-15:
                    best, best_first = cost, seq[0]
            assert abs(val[n, q] - best) < 1e-12
            assert lut[n, q] == best_first


def test_expectation_is_the_sample_mean_and_ties_take_the_lowest_plan():
    # two layers, one state each way: plan 0 costs 1 and lands in state 0 or 1 (half each); plan 1 costs 1.25 and always lands in 0
    t = np.array([[[1.0, 1.25], [9.0, 9.0]], [[2.0, np.inf], [3.0, np.inf]]])
    ns = np.array([[[[0, 1], [0, 0]], [[0, 0], [0, 0]]], [[[0, 0], [0, 0]], [[0, 0], [0, 0]]]])
    lut, val = orc.controller_lut(t, ns, 2)
    # plan 0: 1 + (2 + 3) / 2 = 3.5 ; plan 1: 1.25 + 2 = 3.25
    assert lut[0, 0] == 1 and abs(val[0, 0] - 3.25) < 1e-15
    t[0, 0, 1] = 1.5  # now both cost 3.5: the lower index wins
    lut, val = orc.controller_lut(t, ns, 2)
    assert lut[0, 0] == 0 and abs(val[0, 0] - 3.5) < 1e-15
    # a state with no allowed plan
    t[1, 1, :] = np.inf
    lut, val = orc.controller_lut(t, ns, 2)
    assert lut[1, 1] == -1 and math.isinf(val[1, 1])


@pytest.mark.parametrize("seed,H", [(3, 1), (4, 2), (5, 4), (6, 9)])
def test_library_table_builder_matches_the_oracle(seed, H):
    from paper_2609_03079_b200 import binding as ls

    rng = np.random.default_rng(seed)
    N, Q, A, S = 7, 5, 4, 6
    t, ns = random_tables(rng, N, Q, A, S)
    lut_ref, val_ref = orc.controller_lut(t, ns, H)
    lut, val = ls.ls_controller_build(t, ns, H)
    assert lut.tolist() == lut_ref.tolist()
    np.testing.assert_allclose(val, val_ref, rtol=1e-13, atol=0)
    for v in (-2.0, 0.0, 0.3, 3.9, 4.0, 7.99, 8.0, 1e9):
        assert ls.ls_controller_quantize(v, 8.0, 16) == orc.quantize_state(v, 8.0, 16)
    with pytest.raises(ls.LeanStreamError):
        ls.ls_controller_build(t, np.full_like(ns, Q), H)  # a sample outside the state range
