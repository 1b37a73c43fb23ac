"""CPU oracle for the speculate-and-refine sparse FFN decode step (fp64, NumPy).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
method computes.  Only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import it; the product (the CUDA library and its Python
binding) never does, and shares no code, table or constant with it.

Notation follows the paper's Section 2.1: ``x_n`` is the residual state before
MLP_n, ``h_n`` the MLP input, stage ``k`` of MLP_n produces ``dm^(k)`` (Eq. 1),
and ``xt^(j) = x_n + sum_{k<=j} dm^(k)`` is the partial residual feature (Eq. 2)
that re-scores the neurons of MLP_{n+1}.

Readings taken where the paper is silent (each is listed in the design notes):
ReLU replaces the SiLU printed in Eq. 1 (the workloads are ReLU-sparse); the MLP
input is the gain-free RMS norm of the residual; the predictor is the rank-r
linear map ``s = B^T (A^T h) + c`` (the PCA projection of Section 3.3.3 followed
by a linear scorer); ties in the ranking go to the lower neuron index; the
amount fetched after stage j is the first ``ceil(k (j+1)/(K+1))`` ranks.

Pins (tests/test_oracle_*.py): hand-worked layer, k = d_ff equals the dense FFN,
exact ReLU-active set equals the dense FFN, stage-count and permutation
invariance (Section 3.2.2 "Permutation-Invariant Execution"), Eq. 2 telescoping,
full-rank noise-free predictor reproduces the gate pre-activations, brute-force
top-k on tiny inputs, brute-force cache set rule on <= 8 neurons, batch of
copies.  No function here is "parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

RELU, SILU = 0, 1
NORM_RMS, NORM_NONE = 0, 1


def decode16(bits: np.ndarray, wdtype: str) -> np.ndarray:
    """Exact value (as fp64) of stored 16-bit weights given as raw ``uint16`` patterns."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if wdtype == "bf16":
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if wdtype == "fp16":
        return bits.view(np.float16).astype(np.float64)
    raise ValueError(wdtype)


@dataclass
class OracleLayer:
    """Operands of Eq. 1 for one layer plus its predictor, all fp64.

    ``w_gate[i]``, ``w_up[i]`` are the gate/up weights of hidden neuron ``i`` (a column of the
    paper's ``W_gate``/``W_up``, stored as a row) and ``w_down_t[i]`` is row ``i`` of ``W_down``.
    """

    w_gate: np.ndarray  # [F, d]
    w_up: Optional[np.ndarray]  # [F, d] or None (non-gated FFN: act(fc1) fc2)
    w_down_t: np.ndarray  # [F, d]
    b_gate: np.ndarray  # [F]
    b_down: Optional[np.ndarray]  # [d]
    pred_a: np.ndarray  # [d, r]
    pred_bt: np.ndarray  # [F, r]  (transposed so that every neuron's score is one row reduction)
    pred_c: np.ndarray  # [F]
    eps: float = 1e-5
    norm: int = NORM_RMS
    act: int = RELU

    @property
    def d_model(self) -> int:
        return self.w_gate.shape[1]

    @property
    def d_ff(self) -> int:
        return self.w_gate.shape[0]

    @staticmethod
    def from_arrays(la) -> "OracleLayer":
        """Build from host arrays holding raw 16-bit patterns (attributes as in the workload module)."""
        dt = la.wdtype
        F = la.d_ff
        return OracleLayer(
            w_gate=decode16(la.w_gate, dt),
            w_up=None if la.w_up is None else decode16(la.w_up, dt),
            w_down_t=decode16(la.w_down_t, dt),
            b_gate=np.zeros(F) if la.b_gate is None else la.b_gate.astype(np.float64),
            b_down=None if la.b_down is None else la.b_down.astype(np.float64),
            pred_a=decode16(la.pred_a, dt),
            pred_bt=np.ascontiguousarray(decode16(la.pred_b, dt).T),
            pred_c=np.zeros(F) if la.pred_c is None else la.pred_c.astype(np.float64),
            eps=float(la.norm_eps),
            act=SILU if getattr(la, "act", "relu") == "silu" else RELU,
        )


# ----------------------------------------------------------------------------------------------
# MLP input and dense FFN (the definition the sparse step is checked against)
# ----------------------------------------------------------------------------------------------
def mlp_input(L: OracleLayer, v: np.ndarray) -> np.ndarray:
    """``h`` from a residual-like vector: gain-free RMS norm, ``v / sqrt(mean(v^2) + eps)``.

    Section 2.1 distinguishes the residual ``x_n`` from the MLP input ``h_n`` without printing
    the normalisation; RMS norm (as in the Llama/Mistral family) is the reading taken.
    """
    v = np.asarray(v, dtype=np.float64)
    if L.norm == NORM_NONE:
        return v.copy()
    return v / math.sqrt(float(np.mean(v * v)) + L.eps)


def activation(L: OracleLayer, g: np.ndarray) -> np.ndarray:
    if L.act == RELU:
        return np.maximum(g, 0.0)
    return g / (1.0 + np.exp(-g))  # SiLU as printed in Eq. 1


def neuron_activations(L: OracleLayer, h: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """``a_i = act(w_gate[i].h + b_i) * (w_up[i].h)`` for the listed neurons (bracket of Eq. 1)."""
    idx = np.asarray(idx, dtype=np.int64)
    g = L.w_gate[idx] @ h + L.b_gate[idx]
    a = activation(L, g)
    if L.w_up is not None:
        a = a * (L.w_up[idx] @ h)
    return a


def dense_ffn(L: OracleLayer, x: np.ndarray) -> np.ndarray:
    """Complete MLP output ``y`` (Eq. 1 with one stage holding every neuron); ``x_{n+1} = x + y``."""
    h = mlp_input(L, x)
    a = neuron_activations(L, h, np.arange(L.d_ff))
    y = a @ L.w_down_t
    if L.b_down is not None:
        y = y + L.b_down
    return y


# ----------------------------------------------------------------------------------------------
# Speculate: predictor scores and total-order top-k
# ----------------------------------------------------------------------------------------------
def predictor_scores(L: OracleLayer, v: np.ndarray) -> np.ndarray:
    """Priority score of every neuron of ``L`` from a (partial) residual feature ``v``.

    Section 3.3.3: the feature first goes through a PCA/SVD projection (``A``), then through
    the predictor, here linear: ``s = B^T (A^T h) + c`` with ``h`` the normalised feature.
    Each score is one row reduction of identical shape, so equal predictor columns give
    bit-equal scores (exact ties).
    """
    h = mlp_input(L, v)
    z = h @ L.pred_a  # [r]
    return np.sum(L.pred_bt * z[None, :], axis=1) + L.pred_c


def _canonical(s: np.ndarray) -> np.ndarray:
    s = np.array(s, dtype=np.float64, copy=True)
    s[np.isnan(s)] = -np.inf  # a NaN score ranks last
    s[s == 0.0] = 0.0  # -0.0 and +0.0 are one value
    return s


def topk_order(s: np.ndarray, k: int) -> np.ndarray:
    """The ``k`` highest-priority neurons in rank order: score descending, lower index first on ties.

    Section 3.3: the predictor estimates the relative ordering of activation magnitudes; the
    order is made total by the index so that every selected set is unique.
    """
    s = _canonical(s)
    F = s.shape[0]
    if not 0 <= k <= F:
        raise ValueError("k out of range")
    order = sorted(range(F), key=lambda i: (-s[i], i))
    return np.asarray(order[:k], dtype=np.int64)


def band_bounds(count: int, K: int) -> List[tuple]:
    """Rank ranges of the ``K`` priority-ordered stages: ``m = ceil(count/K)`` ranks each, the last
    ones shorter or empty (Section 2.1: MLP_n is partitioned into K stages in descending priority)."""
    if K < 1:
        raise ValueError("K >= 1")
    m = -(-count // K) if count > 0 else 0
    return [(min(count, c * m), min(count, (c + 1) * m)) for c in range(K)]


def mask_of(idx: Sequence[int], F: int) -> np.ndarray:
    """Bitmask with neuron ``i`` at bit ``i & 31`` of word ``i >> 5``."""
    m = np.zeros((F + 31) // 32, dtype=np.uint32)
    for i in idx:
        m[int(i) >> 5] |= np.uint32(1) << np.uint32(int(i) & 31)
    return m


def select_batch(L: OracleLayer, V: np.ndarray, k: int):
    """Selection for a batch of features: the union of the per-token top-k sets, ordered by the
    neuron priority ``max_b s_{b,i}`` (descending, lower index first).  Batch 1 is plain top-k.

    Returns ``(order, priority)`` with ``order`` the selected neurons in rank order.
    """
    V = np.atleast_2d(np.asarray(V, dtype=np.float64))
    S = np.stack([_canonical(predictor_scores(L, v)) for v in V])  # [B, F]
    member = np.zeros(L.d_ff, dtype=bool)
    for b in range(S.shape[0]):
        member[topk_order(S[b], k)] = True
    prio = S.max(axis=0)
    members = [i for i in range(L.d_ff) if member[i]]
    members.sort(key=lambda i: (-prio[i], i))
    return np.asarray(members, dtype=np.int64), prio


# ----------------------------------------------------------------------------------------------
# Logical neuron cache (which neurons hold a slot; independent of when their bytes land)
# ----------------------------------------------------------------------------------------------
class LogicalCache:
    """Residency set ``R`` of one layer's HBM neuron cache with capacity ``C`` and retention
    priorities ``rho`` (Section 3.3.3: every cache element has an eviction priority; here the
    priority is the layer's latest refined score vector instead of a learned reuse distance).

    ``reserve(M, P)``: the new resident set is the ``C`` best of ``R | M`` under the key
    (member of ``M | P`` first, then ``rho`` descending, then index ascending).
    """

    def __init__(self, d_ff: int, capacity: int):
        self.F = int(d_ff)
        self.C = int(capacity)
        self.resident: set = set()
        self.rho = np.full(self.F, -np.inf)
        self.hits = 0
        self.misses = 0
        self.evictions = 0

    def set_priorities(self, rho: np.ndarray) -> None:
        self.rho = _canonical(rho)

    def lookup(self, idx: Sequence[int]) -> np.ndarray:
        return np.asarray([int(i) in self.resident for i in idx], dtype=bool)

    def _keep_key(self, i: int, pinned: set):
        return (0 if i in pinned else 1, -self.rho[i], i)

    def reserve(self, M: Sequence[int], P: Sequence[int] = ()):
        """Returns ``(misses, victims)`` as sorted lists; raises if ``|M | P| > C``."""
        Mset = {int(i) for i in M}
        pinned = Mset | {int(i) for i in P}
        if len(pinned) > self.C:
            raise OverflowError("wanted + protected neurons exceed the cache capacity")
        universe = self.resident | Mset
        keep = sorted(universe, key=lambda i: self._keep_key(i, pinned))[: self.C]
        new_res = set(keep)
        misses = sorted(Mset - self.resident)
        victims = sorted(self.resident - new_res)
        self.hits += len(Mset & self.resident)
        self.misses += len(misses)
        self.evictions += len(victims)
        self.resident = new_res
        return misses, victims

    def evict(self, min_free: int, P: Sequence[int] = ()):
        """Evict lowest-priority unprotected residents until ``C - |R| >= min_free``; returns victims
        (fewer than asked when only protected ones remain)."""
        prot = {int(i) for i in P}
        need = min_free - (self.C - len(self.resident))
        if need <= 0:
            return []
        cand = sorted((i for i in self.resident if i not in prot), key=lambda i: (-self.rho[i], i))
        victims = cand[len(cand) - min(need, len(cand)):]
        self.resident -= set(victims)
        self.evictions += len(victims)
        return sorted(victims)

    def snapshot(self) -> np.ndarray:
        return mask_of(sorted(self.resident), self.F)


def execution_order(order: np.ndarray, cache: Optional[LogicalCache]) -> np.ndarray:
    """Order in which the selected neurons run: with a cache, residents first in priority order,
    then the misses in priority order, which is the order their copies are issued and land
    (Section 3.2.2: arrival order is used directly as execution order; Section 1: the GPU runs
    the highest-priority *available* sub-models first)."""
    order = np.asarray(order, dtype=np.int64)
    if cache is None:
        return order
    hit = cache.lookup(order)
    return np.concatenate([order[hit], order[~hit]])


# ----------------------------------------------------------------------------------------------
# The staged sparse step with refinement of the next layer
# ----------------------------------------------------------------------------------------------
def fetch_prefix(k_next: int, j: int, K: int) -> int:
    """Ranks admitted for fetching after stage ``j`` (0..K): a prefix that grows linearly and is the
    whole final set at ``j = K`` (deterministic stand-in for "whatever the link moves before the
    next refinement, in priority order", Section 3.1)."""
    return -(-(k_next * (j + 1)) // (K + 1))


def sparse_ffn_step(
    L: OracleLayer,
    nxt: Optional[OracleLayer],
    X: np.ndarray,
    order: np.ndarray,
    K: int,
    k_next: int = 0,
    cache: Optional[LogicalCache] = None,
    next_cache: Optional[LogicalCache] = None,
    xtilde_override: Optional[np.ndarray] = None,
) -> Dict[str, object]:
    """One layer's speculate-and-refine step for a batch ``X`` [B, d] (B = 1 in the paper).

    ``order`` lists the selected neurons of ``L`` in priority order.  Stages run over equal rank
    slices of the execution order (Eq. 1); after each stage the partial residual feature (Eq. 2)
    re-scores the neurons of ``nxt``.  ``xtilde_override`` [K+1, B, d], when given, replaces the
    features fed to the *predictor* (replay of another implementation's feature bits so that the
    refined sets can be compared exactly); the values returned in ``xtilde`` are always the
    oracle's own.

    Returns ``xtilde`` [K+1, B, d], ``y`` [B, d], ``survive`` (sorted neurons with a nonzero
    activation for some token), ``exec_order``, ``refine_orders`` (list of K+1 rank-ordered index
    arrays for ``nxt``), ``refine_prio``, ``fetch`` (list of K+1 admitted-miss lists).
    """
    X = np.atleast_2d(np.asarray(X, dtype=np.float64))
    B, d = X.shape
    order = np.asarray(order, dtype=np.int64)
    ex = execution_order(order, cache)
    if cache is not None:
        cache.reserve(ex)
    H = np.stack([mlp_input(L, x) for x in X])
    xt = np.empty((K + 1, B, d))
    xt[0] = X if L.b_down is None else X + L.b_down[None, :]
    survive: set = set()
    for c, (lo, hi) in enumerate(band_bounds(len(ex), K)):
        dm = np.zeros((B, d))
        stage = ex[lo:hi]
        for b in range(B):
            a = neuron_activations(L, H[b], stage)
            nz = a != 0.0
            survive.update(int(i) for i in stage[nz])
            dm[b] = a[nz] @ L.w_down_t[stage[nz]]  # only surviving columns are read
        xt[c + 1] = xt[c] + dm
    out: Dict[str, object] = {
        "xtilde": xt, "y": xt[K] - X, "survive": np.asarray(sorted(survive), dtype=np.int64), "exec_order": ex,
    }
    if nxt is not None:
        feats = xt if xtilde_override is None else np.asarray(xtilde_override, dtype=np.float64).reshape(K + 1, B, d)
        orders, prios, fetch = [], [], []
        for j in range(K + 1):
            o, p = select_batch(nxt, feats[j], k_next)
            orders.append(o)
            prios.append(p)
            if next_cache is not None:
                next_cache.set_priorities(p)
                if j < K:  # the final set is reserved when the next layer's own step starts
                    admitted = o[: fetch_prefix(len(o), j, K)]
                    misses, _ = next_cache.reserve(admitted)
                    fetch.append(misses)
        out.update(refine_orders=orders, refine_prio=prios, fetch=fetch)
    return out


def decode_token(layers: Sequence[OracleLayer], x0: np.ndarray, k: int, K: int,
                 caches: Optional[Sequence[Optional[LogicalCache]]] = None):
    """One token through a stack of FFN layers (no attention between them: ``x_{n+1} = xt_n^(K)``).

    The first layer's set comes from the full-context prediction on ``x_0``; every later layer uses
    the final refined set ``C^(K)`` of the step before it.  The last layer refines a weight-tied
    copy of itself so that every step produces the same outputs.  Returns ``(x_out, per-layer results)``.
    """
    X = np.atleast_2d(np.asarray(x0, dtype=np.float64))
    order, prio = select_batch(layers[0], X, k)
    if caches is not None and caches[0] is not None:
        caches[0].set_priorities(prio)
    results = []
    for n, L in enumerate(layers):
        last = n + 1 == len(layers)
        nxt = layers[n] if last else layers[n + 1]
        res = sparse_ffn_step(L, nxt, X, order, K, k,
                              cache=None if caches is None else caches[n],
                              next_cache=None if (caches is None or last) else caches[n + 1])
        results.append(res)
        X = res["xtilde"][K]
        order = res["refine_orders"][K]
    return X, results


# ----------------------------------------------------------------------------------------------
# Reported statistics (Section 4.3 tables; not graded)
# ----------------------------------------------------------------------------------------------
def importance_ratio(pred_idx: Sequence[int], true_abs_act: np.ndarray) -> float:
    """Share of the total activation magnitude captured by the predicted set (Section 4.3.1)."""
    tot = float(np.sum(true_abs_act))
    return float(np.sum(true_abs_act[np.asarray(pred_idx, dtype=np.int64)])) / tot if tot > 0 else 1.0


def top_fraction_recall(pred_idx: Sequence[int], true_abs_act: np.ndarray, frac: float = 0.10) -> float:
    """Recall of the ``frac`` largest-magnitude neurons inside the predicted set (Top-10% recall)."""
    n = max(1, int(round(frac * true_abs_act.shape[0])))
    top = set(topk_order(true_abs_act, n).tolist())
    return len(top & {int(i) for i in pred_idx}) / n


def loading_redundancy(fetch_lists: Sequence[Sequence[int]], final_set: Sequence[int], resident_before: set) -> float:
    """Relative loading redundancy: fetched-but-unused rows over the rows the final set truly missed."""
    fetched = set()
    for f in fetch_lists:
        fetched |= {int(i) for i in f}
    final = {int(i) for i in final_set}
    needed = final - resident_before
    return len(fetched - final) / max(1, len(needed))


def lru_miss_ratio(trace: Sequence[Sequence[int]], capacity: int) -> float:
    """Miss ratio of a textbook LRU cache over a trace of per-token request lists."""
    from collections import OrderedDict

    lru: "OrderedDict[int, None]" = OrderedDict()
    miss = tot = 0
    for req in trace:
        for i in req:
            i = int(i)
            tot += 1
            if i in lru:
                lru.move_to_end(i)
            else:
                miss += 1
                lru[i] = None
                if len(lru) > capacity:
                    lru.popitem(last=False)
    return miss / max(1, tot)


# ----------------------------------------------------------------------------------------------
# Streaming controller (Section 3.2.3): finite-horizon stochastic dynamic programme -> LUT[n, q]
# ----------------------------------------------------------------------------------------------
def quantize_state(remaining: float, vmax: float, n_states: int) -> int:
    """``q = Q(R)``: the remaining-load volume cut into ``n_states`` equal bins over ``[0, vmax]`` (state 0 = nothing
    left to load, the last state collects everything from ``vmax`` on).  The paper says only that Q maps the volume to a
    finite set of controller states (Section 3.2.3, item 1); equal bins are the reading taken."""
    if n_states < 1 or not vmax > 0:
        raise ValueError("n_states >= 1 and vmax > 0")
    if not remaining > 0:
        return 0
    return min(n_states - 1, int(math.floor(remaining / vmax * n_states)))


def controller_lut(t_bar: np.ndarray, next_state: np.ndarray, horizon: int):
    """Bellman backward recursion of Section 3.2.3 (item 3).

    ``t_bar[n, q, a]``: profiled execution time of layer ``n`` from state ``q`` under plan ``a`` (``T^I + T^II``);
    ``inf`` or a negative value marks a plan that is not in ``Phi_n(q)``.  ``next_state[n, q, a, s]``: the profiled
    samples of the next layer's state (the empirical transition distribution; a negative entry is an unused sample).
    ``V_n^0 = 0``; ``V_n^h(q) = min_a [ t_bar[n,q,a] + mean_s V_{n+1}^{h-1}(next_state[n,q,a,s]) ]`` with ``V = 0`` beyond
    the last layer; ``LUT[n, q]`` is the minimising plan at ``h = horizon`` (the lowest plan index among equals, -1 when no
    plan is feasible).  Returns ``(lut, value)`` with ``value[n, q] = V_n^horizon(q)``.
    """
    t_bar = np.asarray(t_bar, dtype=np.float64)
    nxt = np.asarray(next_state, dtype=np.int64)
    N, Q, A = t_bar.shape
    if horizon < 1:
        raise ValueError("horizon >= 1")
    V_prev = np.zeros((N + 1, Q))  # V^{h-1}; row N: beyond the last layer
    lut = np.full((N, Q), -1, dtype=np.int64)
    for h in range(1, horizon + 1):
        V = np.zeros((N + 1, Q))
        for n in range(N):
            for q in range(Q):
                best, best_a = math.inf, -1
                for a in range(A):
                    t = t_bar[n, q, a]
                    if not (t >= 0.0) or math.isinf(t):
                        continue
                    samples = [int(v) for v in nxt[n, q, a] if v >= 0]
                    future = 0.0 if (n + 1 >= N or not samples) else sum(V_prev[n + 1, v] for v in samples) / len(samples)
                    cost = t + future
                    if cost < best:
                        best, best_a = cost, a
                V[n, q] = best if best_a >= 0 else math.inf
                if h == horizon:
                    lut[n, q] = best_a
        V_prev = V
    return lut, V_prev[:N]


# ----------------------------------------------------------------------------------------------
# Stacked learnable hashing predictor, inference only (Section 3.3.1 - 3.3.3)
# ----------------------------------------------------------------------------------------------
def sign_pm(v: np.ndarray) -> np.ndarray:
    """Elementwise sign with values in {-1, +1}; zero counts as +1 (the paper's sign() leaves 0 open)."""
    return np.where(np.asarray(v) >= 0, 1, -1).astype(np.int64)


def hash_index(code: Sequence[int]) -> int:
    """``phi_tau``: a code in {-1,+1}^tau to its bucket number.  The convention is the one the structured matrix Z of
    Section 3.3.2 fixes (for tau = 3 its rows run (-1,-1,-1), (-1,-1,+1), (-1,+1,-1), ..., (+1,+1,+1)): -1 is bit 0,
    +1 is bit 1, and the FIRST component is the most significant bit."""
    idx = 0
    for c in code:
        idx = (idx << 1) | (1 if int(c) > 0 else 0)
    return idx


@dataclass
class HashPredictor:
    """Operands of a stack of learnable hashing layers (Eq. ``y_k = T_k[phi_tau(sign(x_k (*) W_k))]``).

    ``pca`` [d_model, r]: the PCA projection applied to the feature first (Section 3.3.3).  ``w1`` [r, tau]: real
    hyperplanes of the first layer.  ``w[k]`` [d, tau] in {-1,+1}: binary hyperplanes of layer k+2.  ``t[k]`` [2^tau, d]
    in {-1,+1}: the bucket features of layer k+1.  ``codes`` [F, d] in {-1,+1}: one binary code per hidden neuron; a
    neuron's priority is the inner product of the last layer's output with its code (an XNOR-and-bitcount product like the
    inner layers', Section 3.3.1).  The paper does not spell out the output stage for the neuron-activation task; this is
    the reading taken (it reproduces the predictor size the paper reports: d_ff x d bits per block)."""

    pca: np.ndarray
    w1: np.ndarray
    w: List[np.ndarray]
    t: List[np.ndarray]
    codes: np.ndarray

    @property
    def n_layers(self) -> int:
        return len(self.t)


def hash_predictor_trace(P: HashPredictor, v: np.ndarray):
    """Bucket numbers of every layer and the last layer's output for the feature ``v`` (un-normalised: a hyperplane hash
    does not see a positive scale, so the norm of Section 2.1 drops out).  Returns ``(indices, y_last, first_dots)``."""
    z = np.asarray(v, dtype=np.float64) @ P.pca
    dots = z @ P.w1
    idx = [hash_index(sign_pm(dots))]
    y = P.t[0][idx[0]].astype(np.int64)
    for k, W in enumerate(P.w):
        code = sign_pm(y @ W.astype(np.int64))  # XNOR-and-bitcount product: an integer inner product of sign vectors
        idx.append(hash_index(code))
        y = P.t[k + 1][idx[-1]].astype(np.int64)
    return idx, y, dots


def hash_predictor_scores(P: HashPredictor, v: np.ndarray) -> np.ndarray:
    """Priority of every neuron: inner product of the last layer's output with the neuron's code (integers, as fp64)."""
    _, y, _ = hash_predictor_trace(P, v)
    return (P.codes.astype(np.int64) @ y).astype(np.float64)
