"""Pins of the oracle's logical neuron cache and of the cached / tiny-stack step (no GPU)."""
import itertools

import numpy as np
import pytest

from oracle import leanstream_oracle as orc
from paper_2609_03079_b200 import workload as wl


def brute_force_keep(R, M, P, rho, C):
    """Enumerate every candidate resident set and keep those where each kept key precedes each dropped key."""
    universe = sorted(set(R) | set(M))
    pinned = set(M) | set(P)
    key = lambda i: (0 if i in pinned else 1, -rho[i], i)
    size = min(C, len(universe))
    good = []
    for S in itertools.combinations(universe, size):
        rest = [i for i in universe if i not in S]
        if all(key(a) < key(b) for a in S for b in rest):
            good.append(set(S))
    return good


def test_reserve_set_rule_brute_force():
    rng = np.random.default_rng(0)
    n_checked = 0
    for trial in range(300):
        F = int(rng.integers(2, 9))
        C = int(rng.integers(1, F + 1))
        rho = np.round(rng.standard_normal(F), 1)  # coarse: ties happen
        R = set(rng.choice(F, size=int(rng.integers(0, C + 1)), replace=False).tolist())
        M = rng.choice(F, size=int(rng.integers(0, F + 1)), replace=False).tolist()
        P = rng.choice(F, size=int(rng.integers(0, 3)), replace=False).tolist()
        cache = orc.LogicalCache(F, C)
        cache.resident = set(R)
        cache.set_priorities(rho)
        if len(set(M) | set(P)) > C:
            with pytest.raises(OverflowError):
                cache.reserve(M, P)
            assert cache.resident == R  # a refused call changes nothing
            continue
        misses, victims = cache.reserve(M, P)
        good = brute_force_keep(R, M, P, rho, C)
        assert len(good) == 1
        assert cache.resident == good[0]
        assert misses == sorted(set(M) - R)
        assert victims == sorted(R - good[0])
        assert set(M) <= cache.resident and len(cache.resident) <= C
        assert not (set(victims) & (set(M) | set(P)))
        n_checked += 1
    assert n_checked > 100


def test_cache_invariants_over_a_trace():
    rng = np.random.default_rng(1)
    F, C = 64, 24
    cache = orc.LogicalCache(F, C)
    hits = misses = 0
    for t in range(50):
        rho = rng.standard_normal(F)
        cache.set_priorities(rho)
        M = orc.topk_order(rho, 10)
        before = set(cache.resident)
        ms, vs = cache.reserve(M)
        hits += len(set(M.tolist()) & before)
        misses += len(ms)
        assert hits + misses == 10 * (t + 1)
        assert (cache.hits, cache.misses) == (hits, misses)
        assert len(cache.resident) <= C and set(M.tolist()) <= cache.resident
        # identical request again: no misses, nothing evicted
        assert cache.reserve(M) == ([], [])
        cache.hits -= 10
    big = orc.LogicalCache(F, F)
    for t in range(20):
        big.set_priorities(rng.standard_normal(F))
        _, vs = big.reserve(rng.choice(F, 30, replace=False))
        assert vs == []  # capacity >= d_ff: never evicts


def test_evict_lowest_priority_first():
    cache = orc.LogicalCache(8, 6)
    cache.resident = {0, 1, 2, 3, 4, 5}
    cache.set_priorities(np.array([5.0, 1.0, 1.0, 3.0, 0.5, 4.0, 9.0, 9.0]))
    assert cache.evict(0) == []
    assert cache.evict(2, P=[4]) == [1, 2]  # 4 is protected; then the two rho = 1 entries
    cache.resident = {0, 1, 2, 3}
    cache.C = 4
    assert cache.evict(1) == [2]  # tie between 1 and 2: the higher index leaves first
    assert cache.snapshot().tolist() == [0b1011]


def test_execution_order_hits_first():
    cache = orc.LogicalCache(16, 8)
    cache.resident = {3, 9, 11}
    order = np.array([5, 9, 2, 3, 11, 7])
    assert orc.execution_order(order, cache).tolist() == [9, 3, 11, 5, 2, 7]
    assert orc.execution_order(order, None).tolist() == order.tolist()


def test_fetch_prefix_rule():
    # grows linearly and ends at the whole set; F^(j) is that prefix minus the residents
    assert [orc.fetch_prefix(160, j, 8) for j in range(9)] == [18, 36, 54, 72, 89, 107, 125, 143, 160]
    assert orc.fetch_prefix(7, 0, 1) == 4 and orc.fetch_prefix(7, 1, 1) == 7


# ------------------------------------------------------------------ the tiny configuration end to end
@pytest.fixture(scope="module")
def tiny():
    spec = wl.SPECS["tiny"]
    la = wl.make_layer(spec, 0)
    return spec, la, orc.OracleLayer.from_arrays(la), wl.make_tokens(spec)


def test_tiny_workload_recipe(tiny):
    spec, la, L, toks = tiny
    assert spec.k == 160 and (L.d_model, L.d_ff) == (256, 1024) and toks.shape == (16, 256)
    np.testing.assert_allclose(np.sqrt(np.mean(toks.astype(np.float64) ** 2, axis=1)), 1.0, rtol=1e-6)
    act = np.mean([np.mean(L.w_gate @ orc.mlp_input(L, x) + L.b_gate > 0) for x in toks])
    assert 0.10 < act < 0.20  # bias shift gives about 15 % active neurons
    # same seed, same arrays
    la2 = wl.make_layer(spec, 0)
    assert np.array_equal(la.w_gate, la2.w_gate) and np.array_equal(la.pred_b, la2.pred_b)
    # the rank-32 predictor is informative but far from exact on an i.i.d. matrix
    x = toks[0]
    order = orc.topk_order(orc.predictor_scores(L, x), spec.k)
    g = L.w_gate @ orc.mlp_input(L, x) + L.b_gate
    recall = len(set(order.tolist()) & set(np.flatnonzero(g > 0).tolist())) / max(1, int(np.sum(g > 0)))
    assert 0.2 < recall < 0.8


def test_tiny_cached_decode_matches_uncached_values(tiny):
    """The cache changes execution order and residency only, never the layer output."""
    spec, la, L, toks = tiny
    cache = orc.LogicalCache(L.d_ff, 300)
    plain_misses = 0
    for t, x in enumerate(toks[:6]):
        order, prio = orc.select_batch(L, x[None], spec.k)
        cache.set_priorities(prio)
        before = set(cache.resident)
        res_c = orc.sparse_ffn_step(L, None, x, order, 8, cache=cache)
        res_p = orc.sparse_ffn_step(L, None, x, order, 8)
        np.testing.assert_allclose(res_c["y"], res_p["y"], rtol=1e-11, atol=1e-12)
        ex = res_c["exec_order"]
        n_hit = len(set(order.tolist()) & before)
        assert set(ex[:n_hit].tolist()) == set(order.tolist()) & before
        assert set(order.tolist()) <= cache.resident and len(cache.resident) <= 300
        plain_misses += spec.k - n_hit
    assert cache.misses == plain_misses and cache.hits + cache.misses == 6 * spec.k


def test_tiny4_stack_refinement_moves_and_fetch_lists():
    spec = wl.SPECS["tiny4"]
    arrays = wl.make_stack(spec, down_scale=50.0)
    layers = [orc.OracleLayer.from_arrays(a) for a in arrays]
    caches = [orc.LogicalCache(spec.d_ff, 400) for _ in layers]
    x = wl.make_tokens(spec)[0]
    K, k, C = 4, spec.k, 400
    _, results = orc.decode_token(layers, x, k, K, caches)
    moved = 0
    # Independent replay of the residency of every layer's cache (Section 3.3.3: priority-ordered loading, eviction by
    # priority): the set rule is restated here with plain set operations and a sort, not through LogicalCache.
    shadow = [set() for _ in layers]

    def replay_reserve(res_set, wanted, rho):
        universe = res_set | set(wanted)
        keep = sorted(universe, key=lambda i: (0 if i in wanted else 1, -rho[i], i))[:C]
        return set(keep)

    order0 = orc.topk_order(orc.predictor_scores(layers[0], x), k)
    prio_of = [None] * len(layers)
    prio_of[0] = orc._canonical(orc.predictor_scores(layers[0], x))
    sel = [None] * len(layers)
    sel[0] = order0
    for n, res in enumerate(results):
        # the step first reserves its own selection (residents first, then misses)
        shadow[n] = replay_reserve(shadow[n], set(sel[n].tolist()), prio_of[n])
        if n + 1 == len(layers):
            break
        first, last = set(res["refine_orders"][0].tolist()), set(res["refine_orders"][K].tolist())
        moved += len(first ^ last)
        assert len(res["fetch"]) == K
        for j in range(K):
            Cj = res["refine_orders"][j]
            # stage j admits exactly the first ceil(k (j+1)/(K+1)) ranks of C^(j) ...
            n_adm = -(-(len(Cj) * (j + 1)) // (K + 1))
            admitted = Cj[:n_adm].tolist()
            # ... and fetches those of them that hold no slot at that moment, under the priorities of evaluation j
            expect = sorted(set(admitted) - shadow[n + 1])
            assert res["fetch"][j] == expect, (n, j)
            rho = orc._canonical(res["refine_prio"][j])
            shadow[n + 1] = replay_reserve(shadow[n + 1], set(admitted), rho)
        prio_of[n + 1] = orc._canonical(res["refine_prio"][K])
        sel[n + 1] = res["refine_orders"][K]
        assert set(res["refine_orders"][K].tolist()) <= caches[n + 1].resident  # reserved by the next step
    for n in range(len(layers)):
        assert shadow[n] == caches[n].resident, n
    assert moved > 0  # with a 50x down projection the partial features do change the ranking
