"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or
index, a transposed operand, an off-by-one in staging) makes it fail.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import leanstream_oracle as orc


def rand_layer(rng, d=16, F=24, r=6, gated=True, bias=-0.3, eps=1e-5):
    return orc.OracleLayer(
        w_gate=rng.standard_normal((F, d)),
        w_up=rng.standard_normal((F, d)) if gated else None,
        w_down_t=rng.standard_normal((F, d)),
        b_gate=np.full(F, bias),
        b_down=None,
        pred_a=rng.standard_normal((d, r)),
        pred_bt=rng.standard_normal((F, r)),
        pred_c=rng.standard_normal(F) * 0.1,
        eps=eps,
    )


# ------------------------------------------------------------------ stored 16-bit operands of Eq. 1
def test_decode16_literal_bit_patterns():
    """Bit patterns written out by hand from the two formats' definitions (sign, exponent bias 127 / 15, 7 / 10
    fraction bits), not produced by any conversion routine."""
    bf = np.array([0x3F80, 0xC040, 0x0000, 0x8000, 0x3F00, 0x4049, 0x0001, 0x7F7F], dtype=np.uint16)
    want_bf = [1.0, -3.0, 0.0, -0.0, 0.5, 3.140625, 2.0 ** -133, (2.0 - 2.0 ** -7) * 2.0 ** 127]
    got = orc.decode16(bf, "bf16")
    assert got.dtype == np.float64 and got.tolist() == want_bf
    assert math.copysign(1.0, got[3]) == -1.0
    fp = np.array([0x3C00, 0xC200, 0x0000, 0x3800, 0x0001, 0x03FF, 0x7BFF, 0x3555], dtype=np.uint16)
    want_fp = [1.0, -3.0, 0.0, 0.5, 2.0 ** -24, 1023 * 2.0 ** -24, 65504.0, (1 + 0x155 / 1024) * 0.25]
    assert orc.decode16(fp, "fp16").tolist() == want_fp
    with pytest.raises(ValueError):
        orc.decode16(bf, "fp8")


def test_silu_branch_of_the_activation():
    """Eq. 1 prints SiLU: g * sigmoid(g).  Closed-form values: SiLU(0) = 0, SiLU(ln 3) = 0.75 ln 3,
    SiLU(-ln 3) = -0.25 ln 3, SiLU(g) - SiLU(-g) = g, and SiLU -> ReLU for large |g|."""
    L = hand_layer()
    L.act = orc.SILU
    ln3 = math.log(3.0)
    g = np.array([0.0, ln3, -ln3, 40.0, -40.0])
    a = orc.activation(L, g)
    np.testing.assert_allclose(a, [0.0, 0.75 * ln3, -0.25 * ln3, 40.0, 0.0], atol=1e-15)
    gg = np.linspace(-5, 5, 41)
    np.testing.assert_allclose(orc.activation(L, gg) - orc.activation(L, -gg), gg, atol=1e-14)
    L.act = orc.RELU
    assert orc.activation(L, g).tolist() == [0.0, ln3, 0.0, 40.0, 0.0]


# ------------------------------------------------------------------ hand-worked layer (Eq. 1)
def hand_layer():
    return orc.OracleLayer(
        w_gate=np.array([[1.0, 0, 0, 0], [0, 1, 0, 0], [1, 1, 1, 0]]),
        w_up=np.array([[0.0, 0, 2, 0], [1, 1, 1, 1], [0, 0, 0, 1]]),
        w_down_t=np.array([[1.0, 2, 3, 4], [5, 5, 5, 5], [2, 0, -2, 4]]),
        b_gate=np.array([0.5, 2.0, -0.5]),
        b_down=None,
        pred_a=np.eye(4),
        pred_bt=np.array([[1.0, 0, 0, 0], [0, 1, 0, 0], [1, 1, 1, 0]]),
        pred_c=np.array([0.5, 2.0, -0.5]),
        eps=0.0,
    )


def test_hand_worked_dense_layer():
    # x has RMS 2, so h = x/2 = (1,-1,1,-1).  Worked by hand:
    # g = (1+.5, -1+2, 1-1+1-.5) = (1.5, 1, .5); u = (2, 0, -1); a = (3, 0, -.5)
    # y = 3*(1,2,3,4) - .5*(2,0,-2,4) = (2, 6, 10, 10)
    L = hand_layer()
    x = np.array([2.0, -2.0, 2.0, -2.0])
    np.testing.assert_allclose(orc.mlp_input(L, x), [1, -1, 1, -1], atol=1e-15)
    np.testing.assert_allclose(orc.dense_ffn(L, x), [2, 6, 10, 10], atol=1e-14)
    # predictor with A = I, B = W_gate, c = b reproduces g; ranking 0 > 1 > 2
    np.testing.assert_allclose(orc.predictor_scores(L, x), [1.5, 1.0, 0.5], atol=1e-15)
    assert orc.topk_order(orc.predictor_scores(L, x), 2).tolist() == [0, 1]
    res = orc.sparse_ffn_step(L, L, x, np.array([0, 1, 2]), K=3, k_next=2)
    # stage outputs: neuron 0 -> (3,6,9,12); neuron 1 -> a = 0, nothing; neuron 2 -> (-1,0,1,-2)
    np.testing.assert_allclose(res["xtilde"][1][0] - x, [3, 6, 9, 12], atol=1e-14)
    np.testing.assert_allclose(res["xtilde"][2][0], res["xtilde"][1][0], atol=0)
    np.testing.assert_allclose(res["xtilde"][3][0] - x, [2, 6, 10, 10], atol=1e-14)
    assert res["survive"].tolist() == [0, 2]  # neuron 1 has g > 0 but u = 0


def test_rmsnorm_eps_and_scale():
    L = hand_layer()
    L.eps = 0.5
    v = np.array([1.0, 2.0, -2.0, 0.0])  # mean square 2.25 -> divide by sqrt(2.75)
    np.testing.assert_allclose(orc.mlp_input(L, v), v / math.sqrt(2.75), rtol=1e-15)


# ------------------------------------------------------------------ dense FFN vs library contraction
@pytest.mark.parametrize("gated", [True, False])
def test_dense_ffn_matches_torch_fp64(gated):
    import torch

    rng = np.random.default_rng(3)
    L = rand_layer(rng, d=32, F=48, gated=gated)
    L.b_down = rng.standard_normal(32) if not gated else None
    x = rng.standard_normal(32)
    tx = torch.from_numpy(x)
    h = tx * torch.rsqrt(tx.pow(2).mean() + L.eps)
    g = torch.nn.functional.linear(h, torch.from_numpy(L.w_gate), torch.from_numpy(L.b_gate))
    a = torch.relu(g)
    if gated:
        a = a * torch.nn.functional.linear(h, torch.from_numpy(L.w_up))
    y = torch.nn.functional.linear(a, torch.from_numpy(L.w_down_t).T.contiguous(),
                                   None if L.b_down is None else torch.from_numpy(L.b_down))
    np.testing.assert_allclose(orc.dense_ffn(L, x), y.numpy(), rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ sparse == dense special cases
@pytest.mark.parametrize("gated", [True, False])
@pytest.mark.parametrize("K", [1, 3, 8])
def test_k_equals_dff_is_dense(gated, K):
    rng = np.random.default_rng(4)
    L = rand_layer(rng, gated=gated)
    x = rng.standard_normal(L.d_model)
    order = orc.topk_order(orc.predictor_scores(L, x), L.d_ff)
    res = orc.sparse_ffn_step(L, None, x, order, K)
    np.testing.assert_allclose(res["y"][0], orc.dense_ffn(L, x), rtol=1e-12, atol=1e-12)


def test_exact_relu_active_set_is_dense():
    rng = np.random.default_rng(5)
    L = rand_layer(rng, d=32, F=64)
    x = rng.standard_normal(32)
    g = L.w_gate @ orc.mlp_input(L, x) + L.b_gate
    active = np.flatnonzero(g > 0)
    assert 0 < len(active) < L.d_ff
    res = orc.sparse_ffn_step(L, None, x, active, K=4)
    np.testing.assert_allclose(res["y"][0], orc.dense_ffn(L, x), rtol=1e-12, atol=1e-12)
    # dropping one active neuron must change the output (the test above is not vacuous)
    res2 = orc.sparse_ffn_step(L, None, x, active[1:], K=4)
    assert np.max(np.abs(res2["y"][0] - res["y"][0])) > 1e-6


def test_full_rank_noise_free_predictor_reproduces_gate():
    """r = d, A orthogonal, B = (W_gate A)^T, c = b  =>  s = g, so top-(#active) is the active set."""
    rng = np.random.default_rng(6)
    d, F = 12, 40
    L = rand_layer(rng, d=d, F=F, r=d)
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    L.pred_a = Q
    L.pred_bt = L.w_gate @ Q
    L.pred_c = L.b_gate.copy()
    x = rng.standard_normal(d)
    g = L.w_gate @ orc.mlp_input(L, x) + L.b_gate
    s = orc.predictor_scores(L, x)
    np.testing.assert_allclose(s, g, rtol=1e-12, atol=1e-12)
    n_act = int(np.sum(g > 0))
    order = orc.topk_order(s, n_act)
    assert set(order.tolist()) == set(np.flatnonzero(g > 0).tolist())
    res = orc.sparse_ffn_step(L, None, x, order, K=2)
    np.testing.assert_allclose(res["y"][0], orc.dense_ffn(L, x), rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ staging invariants (Eq. 2, Sec. 3.2.2)
def test_stage_count_and_permutation_invariance():
    rng = np.random.default_rng(7)
    L = rand_layer(rng)
    x = rng.standard_normal(L.d_model)
    order = orc.topk_order(orc.predictor_scores(L, x), 13)
    ref = orc.sparse_ffn_step(L, None, x, order, K=1)["y"][0]
    for K in (2, 3, 5, 13, 20):
        res = orc.sparse_ffn_step(L, None, x, order, K)
        np.testing.assert_allclose(res["y"][0], ref, rtol=1e-12, atol=1e-12)
        # telescoping: consecutive partial features differ by exactly that stage's neurons
        h = orc.mlp_input(L, x)
        for c, (lo, hi) in enumerate(orc.band_bounds(13, K)):
            a = orc.neuron_activations(L, h, order[lo:hi])
            np.testing.assert_allclose(res["xtilde"][c + 1][0] - res["xtilde"][c][0], a @ L.w_down_t[order[lo:hi]],
                                       rtol=1e-10, atol=1e-10)
    perm = rng.permutation(13)
    np.testing.assert_allclose(orc.sparse_ffn_step(L, None, x, order[perm], 4)["y"][0], ref, rtol=1e-12, atol=1e-12)


def test_band_bounds():
    assert orc.band_bounds(160, 8) == [(20 * c, 20 * c + 20) for c in range(8)]
    assert orc.band_bounds(10, 4) == [(0, 3), (3, 6), (6, 9), (9, 10)]
    assert orc.band_bounds(3, 5) == [(0, 1), (1, 2), (2, 3), (3, 3), (3, 3)]  # K > k: empty stages
    assert orc.band_bounds(0, 2) == [(0, 0), (0, 0)]


def test_stage_zero_is_one_shot_and_last_is_full_context():
    """0/K is the one-shot prediction from x_n; K/K uses the complete (sparse) MLP output."""
    rng = np.random.default_rng(8)
    L, N = rand_layer(rng), rand_layer(rng)
    x = rng.standard_normal(L.d_model)
    order = orc.topk_order(orc.predictor_scores(L, x), 10)
    res = orc.sparse_ffn_step(L, N, x, order, K=4, k_next=7)
    assert len(res["refine_orders"]) == 5
    assert res["refine_orders"][0].tolist() == orc.topk_order(orc.predictor_scores(N, x), 7).tolist()
    x_next = x + res["y"][0]
    assert res["refine_orders"][4].tolist() == orc.topk_order(orc.predictor_scores(N, x_next), 7).tolist()
    # K = 1: C^(1) is the full-context prediction
    r1 = orc.sparse_ffn_step(L, N, x, order, K=1, k_next=7)
    assert r1["refine_orders"][1].tolist() == res["refine_orders"][4].tolist()


def test_zero_down_projection_freezes_refinement():
    rng = np.random.default_rng(9)
    L, N = rand_layer(rng), rand_layer(rng)
    L.w_down_t = np.zeros_like(L.w_down_t)
    x = rng.standard_normal(L.d_model)
    res = orc.sparse_ffn_step(L, N, x, np.arange(12), K=6, k_next=9)
    for j in range(7):
        assert res["refine_orders"][j].tolist() == res["refine_orders"][0].tolist()


def test_predictor_latent_is_linear_in_partial_outputs():
    """Un-normalised latent: A^T xt^(j) = A^T x + sum_k A^T dm^(k)."""
    rng = np.random.default_rng(10)
    L, N = rand_layer(rng), rand_layer(rng)
    N.norm = orc.NORM_NONE
    x = rng.standard_normal(L.d_model)
    res = orc.sparse_ffn_step(L, N, x, np.arange(9), K=3, k_next=5)
    xt = res["xtilde"][:, 0]
    for j in range(4):
        z = xt[j] @ N.pred_a
        z_lin = x @ N.pred_a + sum((xt[k + 1] - xt[k]) @ N.pred_a for k in range(j))
        np.testing.assert_allclose(z, z_lin, rtol=1e-10, atol=1e-10)
        np.testing.assert_allclose(res["refine_prio"][j], N.pred_bt @ z + N.pred_c, rtol=1e-10, atol=1e-10)


def test_xtilde_override_only_feeds_predictor():
    rng = np.random.default_rng(11)
    L, N = rand_layer(rng), rand_layer(rng)
    x = rng.standard_normal(L.d_model)
    base = orc.sparse_ffn_step(L, N, x, np.arange(8), K=2, k_next=5)
    other = rng.standard_normal((3, 1, L.d_model))
    res = orc.sparse_ffn_step(L, N, x, np.arange(8), K=2, k_next=5, xtilde_override=other)
    np.testing.assert_array_equal(res["xtilde"], base["xtilde"])
    for j in range(3):
        assert res["refine_orders"][j].tolist() == orc.topk_order(orc.predictor_scores(N, other[j, 0]), 5).tolist()


# ------------------------------------------------------------------ top-k
def brute_force_topk_sets(s, k):
    """All size-k subsets S with: every selected (score, index) key precedes every unselected one."""
    F = len(s)
    key = lambda i: (-s[i], i)
    out = []
    for S in itertools.combinations(range(F), k):
        rest = [i for i in range(F) if i not in S]
        if all(key(a) < key(b) for a in S for b in rest):
            out.append(set(S))
    return out


def test_topk_brute_force_tiny():
    rng = np.random.default_rng(12)
    for trial in range(30):
        F = int(rng.integers(1, 10))
        s = np.round(rng.standard_normal(F), 1)  # coarse values -> many exact ties
        for k in range(F + 1):
            sets = brute_force_topk_sets(s, k)
            assert len(sets) == 1  # the total order makes the set unique
            got = orc.topk_order(s, k)
            assert set(got.tolist()) == sets[0]
            keys = [(-s[i], i) for i in got]
            assert keys == sorted(keys)  # rank order


def test_topk_ties_zero_sign_nan_and_edges():
    s = np.array([1.0, 2.0, 2.0, -0.0, 0.0, np.nan, 2.0])
    assert orc.topk_order(s, 0).tolist() == []
    assert orc.topk_order(s, 2).tolist() == [1, 2]  # equal scores: lower index wins
    assert orc.topk_order(s, 7).tolist() == [1, 2, 6, 0, 3, 4, 5]  # -0 == +0 by index; NaN last
    with pytest.raises(ValueError):
        orc.topk_order(s, 8)


def test_duplicated_predictor_columns_give_exact_ties():
    rng = np.random.default_rng(13)
    L = rand_layer(rng, d=64, F=96, r=48)
    L.pred_bt[70] = L.pred_bt[5]
    L.pred_c[70] = L.pred_c[5]
    for _ in range(5):
        s = orc.predictor_scores(L, rng.standard_normal(64))
        assert s[70] == s[5]
        order = orc.topk_order(s, 96).tolist()
        assert order.index(5) + 1 == order.index(70)


def test_mask_layout():
    m = orc.mask_of([0, 31, 32, 70], 96)
    assert m.tolist() == [0x80000001, 0x1, 0x40]


# ------------------------------------------------------------------ batch (union of per-token sets)
def test_batch_of_copies_equals_batch_one():
    rng = np.random.default_rng(14)
    L, N = rand_layer(rng), rand_layer(rng)
    x = rng.standard_normal(L.d_model)
    o1, p1 = orc.select_batch(L, x[None], 7)
    o4, p4 = orc.select_batch(L, np.stack([x] * 4), 7)
    assert o1.tolist() == o4.tolist() == orc.topk_order(orc.predictor_scores(L, x), 7).tolist()
    np.testing.assert_array_equal(p1, p4)
    r1 = orc.sparse_ffn_step(L, N, x[None], o1, 3, 5)
    r4 = orc.sparse_ffn_step(L, N, np.stack([x] * 4), o4, 3, 5)
    for b in range(4):
        np.testing.assert_array_equal(r4["y"][b], r1["y"][0])
    assert r4["refine_orders"][3].tolist() == r1["refine_orders"][3].tolist()


def test_batch_union_and_priority():
    rng = np.random.default_rng(15)
    L = rand_layer(rng, F=30)
    X = rng.standard_normal((3, L.d_model))
    order, prio = orc.select_batch(L, X, 6)
    per = [set(orc.topk_order(orc.predictor_scores(L, x), 6).tolist()) for x in X]
    assert set(order.tolist()) == per[0] | per[1] | per[2]
    S = np.stack([orc.predictor_scores(L, x) for x in X])
    np.testing.assert_array_equal(prio, S.max(axis=0))
    keys = [(-prio[i], i) for i in order]
    assert keys == sorted(keys)
    # y_b sums over the whole union for every token
    res = orc.sparse_ffn_step(L, None, X, order, 2)
    for b in range(3):
        a = orc.neuron_activations(L, orc.mlp_input(L, X[b]), order)
        np.testing.assert_allclose(res["y"][b], a @ L.w_down_t[order], rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ stack
def test_decode_token_chains_final_refined_set():
    rng = np.random.default_rng(16)
    layers = [rand_layer(rng) for _ in range(3)]
    x0 = rng.standard_normal(16)
    x_out, results = orc.decode_token(layers, x0, k=8, K=4)
    x = x0.copy()
    order = orc.topk_order(orc.predictor_scores(layers[0], x), 8)
    for n, L in enumerate(layers):
        assert sorted(results[n]["exec_order"].tolist()) == sorted(order.tolist())
        a = orc.neuron_activations(L, orc.mlp_input(L, x), order)
        x = x + a @ L.w_down_t[order]
        nxt = layers[min(n + 1, 2)] if n < 2 else layers[2]
        order = orc.topk_order(orc.predictor_scores(nxt, x), 8)
    np.testing.assert_allclose(x_out[0], x, rtol=1e-11, atol=1e-11)


# ------------------------------------------------------------------ reported statistics
def test_statistics_small_cases():
    act = np.array([0.0, 4.0, 1.0, 0.0, 5.0, 0.0, 0.0, 0.0, 0.0, 0.0])
    assert orc.importance_ratio([1, 2], act) == pytest.approx(0.5)
    assert orc.top_fraction_recall([4, 2], act, 0.10) == 1.0
    assert orc.top_fraction_recall([1, 2], act, 0.20) == 0.5
    assert orc.loading_redundancy([[1, 2], [3]], [1, 3, 9], {9}) == pytest.approx(0.5)
    # LRU, capacity 2: a b a c b  ->  miss miss hit miss miss
    assert orc.lru_miss_ratio([[1, 2], [1, 3], [2]], 2) == pytest.approx(4 / 5)
