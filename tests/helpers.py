"""Comparison helpers shared by the GPU parity tests (oracle on one side, the C-ABI library on the other)."""
from __future__ import annotations

import numpy as np

from oracle import leanstream_oracle as orc

REL_L2_TOL = 1e-3      # spec tolerance: relative L2 error of FFN outputs
MAX_ABS_TOL = 1e-2     # spec tolerance: max-abs error as a fraction of max|y|
TIE_EPS = 1e-12        # scores closer than this (relative to max|s|) to the cut may fall on either side


def mask_to_set(mask: np.ndarray, F: int) -> set:
    bits = np.unpackbits(np.ascontiguousarray(mask).view(np.uint8), bitorder="little")[:F]
    return set(np.flatnonzero(bits).tolist())


def assert_values_close(got: np.ndarray, ref: np.ndarray, scale_ref: np.ndarray = None, what: str = ""):
    """The spec output tolerance: rel-L2 <= 1e-3 and max-abs <= 1e-2 * max|ref| (of the increment when given)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    base = ref if scale_ref is None else np.asarray(scale_ref, dtype=np.float64)
    denom = max(float(np.linalg.norm(base)), 1e-30)
    rel = float(np.linalg.norm(got - ref)) / denom
    mx = float(np.max(np.abs(got - ref))) if got.size else 0.0
    lim = MAX_ABS_TOL * max(float(np.max(np.abs(base))) if base.size else 0.0, 1e-30)
    assert rel <= REL_L2_TOL, f"{what}: rel-L2 {rel:.3e} > {REL_L2_TOL}"
    assert mx <= lim, f"{what}: max-abs {mx:.3e} > {lim:.3e}"
    return rel, mx


def check_selection(gpu_order: np.ndarray, oracle_scores: np.ndarray, k: int, stats: dict = None) -> None:
    """Bit-exact set and rank order against the oracle's total order; a set that differs only inside the tie band
    around the cut (|s - t| <= TIE_EPS * max|s|) is accepted and counted as band-resolved."""
    ref = orc.topk_order(oracle_scores, k)
    gpu_order = np.asarray(gpu_order, dtype=np.int64)
    assert len(gpu_order) == k, f"count {len(gpu_order)} != k {k}"
    if np.array_equal(gpu_order, ref):
        if stats is not None:
            stats["exact"] = stats.get("exact", 0) + 1
        return
    s = orc._canonical(oracle_scores)
    eps = TIE_EPS * float(np.max(np.abs(s[np.isfinite(s)]))) if np.any(np.isfinite(s)) else 0.0
    G = set(gpu_order.tolist())
    assert len(G) == k, "duplicate neurons in the selection"
    if k == 0 or k == len(s):
        assert G == set(ref.tolist())
        return
    t = s[ref[-1]]
    must = set(np.flatnonzero(s > t + eps).tolist())
    may = set(np.flatnonzero(s >= t - eps).tolist())
    assert must <= G <= may, f"selection differs from the oracle outside the tie band: {sorted(G ^ set(ref.tolist()))[:10]}"
    if stats is not None:
        stats["band"] = stats.get("band", 0) + 1


def assert_set_in_tie_band(got: set, oracle_scores: np.ndarray, k: int, stats: dict = None) -> None:
    """A selected SET (no order) against the oracle: equal, or different only among scores inside the tie band."""
    s = orc._canonical(oracle_scores)
    ref = set(orc.topk_order(oracle_scores, k).tolist())
    assert len(got) == k, f"set has {len(got)} members, expected {k}"
    if got == ref:
        if stats is not None:
            stats["exact"] = stats.get("exact", 0) + 1
        return
    eps = TIE_EPS * float(np.max(np.abs(s[np.isfinite(s)]))) if np.any(np.isfinite(s)) else 0.0
    t = min(s[i] for i in ref)
    must = set(np.flatnonzero(s > t + eps).tolist())
    may = set(np.flatnonzero(s >= t - eps).tolist())
    assert must <= got <= may, f"set differs from the oracle outside the tie band: {sorted(got ^ ref)[:10]}"
    if stats is not None:
        stats["band"] = stats.get("band", 0) + 1


def check_survive(gpu_survive: set, L: orc.OracleLayer, x: np.ndarray, order: np.ndarray) -> None:
    """Surviving set: equal to the oracle's except for neurons whose gate pre-activation is within fp32 rounding of 0."""
    h = orc.mlp_input(L, x)
    order = np.asarray(order, dtype=np.int64)
    g = L.w_gate[order] @ h + L.b_gate[order]
    a = orc.neuron_activations(L, h, order)
    ref = set(order[a != 0.0].tolist())
    if L.act == orc.SILU:  # no zeros: every selected neuron survives (an exact zero needs g = 0 or u = 0 exactly)
        assert gpu_survive == ref
        return
    tol = 1e-5 * np.linalg.norm(L.w_gate[order], axis=1) * np.linalg.norm(h)
    fuzzy = set(order[np.abs(g) <= tol].tolist())
    assert (gpu_survive ^ ref) <= fuzzy, f"survive mask differs: {sorted((gpu_survive ^ ref) - fuzzy)[:10]}"
