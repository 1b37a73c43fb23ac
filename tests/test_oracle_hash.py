"""Pins of the oracle's stacked hashing predictor (Section 3.3.1 - 3.3.3) against what the paper and arithmetic fix."""
import itertools

import numpy as np

from oracle import leanstream_oracle as orc


def test_index_convention_is_the_papers_structured_matrix():
    """Section 3.3.2 prints Z for tau = 3: rows (-1,-1,-1), (-1,-1,+1), (-1,+1,-1), ..., (+1,+1,+1); row i is phi^-1(i)."""
    Z = [(-1, -1, -1), (-1, -1, +1), (-1, +1, -1), (-1, +1, +1), (+1, -1, -1), (+1, -1, +1), (+1, +1, -1), (+1, +1, +1)]
    assert [orc.hash_index(row) for row in Z] == list(range(8))
    # and the alternative formulation of the same section: the bucket is the row of Z that agrees best with the code
    for tau in (1, 2, 5):
        rows = list(itertools.product((-1, 1), repeat=tau))
        for code in rows:
            agree = [sum(a * b for a, b in zip(r, code)) for r in rows]
            assert int(np.argmax(agree)) == orc.hash_index(code)


def test_sign_of_zero_is_plus_one():
    assert orc.sign_pm(np.array([-2.0, -0.0, 0.0, 3.0])).tolist() == [-1, 1, 1, 1]


def hand_predictor():
    # d_model 3, r 2, tau 2, d 4, two layers, three neurons; every number small enough to follow by hand
    return orc.HashPredictor(
        pca=np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]),
        w1=np.array([[1.0, -1.0], [1.0, 1.0]]),
        w=[np.array([[1, 1], [1, -1], [-1, 1], [1, 1]])],
        t=[np.array([[1, 1, 1, 1], [1, -1, 1, -1], [-1, -1, 1, 1], [-1, 1, 1, -1]]),
           np.array([[1, 1, -1, -1], [-1, -1, -1, -1], [1, -1, -1, 1], [1, 1, 1, 1]])],
        codes=np.array([[1, 1, 1, 1], [1, -1, -1, 1], [-1, -1, 1, 1]]),
    )


def test_hand_worked_two_layer_predictor():
    P = hand_predictor()
    # v = (1, -3, 1): z = (1+1, -3+1) = (2, -2); dots = (2-2, -2-2) = (0, -4) -> code (+1, -1) -> bucket 0b10 = 2
    # y1 = T1[2] = (-1,-1,1,1); layer 2: y1.W = (-1-1-1+1, -1+1+1+1) = (-2, 2) -> code (-1,+1) -> bucket 1
    # y2 = T2[1] = (-1,-1,-1,-1); scores = (-4, 0, 0)
    idx, y, dots = orc.hash_predictor_trace(P, np.array([1.0, -3.0, 1.0]))
    assert dots.tolist() == [0.0, -4.0] and idx == [2, 1] and y.tolist() == [-1, -1, -1, -1]
    s = orc.hash_predictor_scores(P, np.array([1.0, -3.0, 1.0]))
    assert s.tolist() == [-4.0, 0.0, 0.0]
    assert orc.topk_order(s, 2).tolist() == [1, 2]  # ties go to the lower index
    # a hyperplane hash does not see a positive scale
    idx2, y2, _ = orc.hash_predictor_trace(P, 7.5 * np.array([1.0, -3.0, 1.0]))
    assert idx2 == idx and y2.tolist() == y.tolist()


def test_binary_layers_are_xnor_and_bitcount():
    """For sign vectors the inner product equals d - 2 * (number of differing positions): the identity behind the XNOR and
    bitcount implementation of Section 3.3.1, checked on the oracle's integer products."""
    rng = np.random.default_rng(0)
    d = 64
    for _ in range(50):
        a, b = rng.choice([-1, 1], size=d), rng.choice([-1, 1], size=d)
        assert int(a @ b) == d - 2 * int(np.sum(a != b))


def test_scores_are_bounded_even_integers_and_every_bucket_is_reachable():
    rng = np.random.default_rng(1)
    tau, d, F, r, dm = 3, 32, 40, 6, 10
    P = orc.HashPredictor(pca=rng.standard_normal((dm, r)), w1=rng.standard_normal((r, tau)),
                          w=[rng.choice([-1, 1], size=(d, tau)) for _ in range(2)],
                          t=[rng.choice([-1, 1], size=(2 ** tau, d)) for _ in range(3)], codes=rng.choice([-1, 1], size=(F, d)))
    seen = set()
    for _ in range(200):
        v = rng.standard_normal(dm)
        idx, y, _ = orc.hash_predictor_trace(P, v)
        seen.add(idx[0])
        s = orc.hash_predictor_scores(P, v)
        assert np.all(np.abs(s) <= d) and np.all(s % 2 == 0) and set(np.unique(y).tolist()) <= {-1, 1}
        assert s.tolist() == [float(np.dot(P.codes[i], P.t[2][idx[2]])) for i in range(F)]
    assert seen == set(range(2 ** tau))
