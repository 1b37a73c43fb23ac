"""Seeded synthetic workloads: FFN stacks, predictors and token streams.

This module only *makes inputs*.  It holds none of the method's arithmetic
(no FFN, no predictor evaluation, no top-k, no cache rule): the CPU oracle and
the CUDA library both receive the arrays produced here and nothing else is
shared between them.

Recipe (stands in for the Mistral-7B / Llama2-7B / Qwen2.5-7B checkpoints and
the Qasper / TruthfulQA / CoQA prompts of the paper's Section 4.1, none of
which is available offline; only the model shapes and sparsity levels are kept):

* RNG: ``numpy.random.Generator(Philox(SeedSequence([cfg_seed, layer, tensor_id])))``.
* gate / up / down^T rows: i.i.d. N(0, 0.02^2), rounded to the 16-bit weight type.
* gate bias: the constant ``-Phi^-1(1-p) * 0.02 * sqrt(d_model)`` so that about a
  fraction ``p`` of the neurons has a positive gate pre-activation when the
  normalised input has squared norm ``d_model``.
* predictor: ``A = V_r`` (top-``r`` right singular vectors of the gate matrix),
  ``B = (W_gate V_r)^T + N(0, 0.01^2)``, both rounded to the weight type, and
  ``c = b_gate``.
* tokens: i.i.d. N(0, I) vectors (optionally scaled to RMS 1), or an AR(1)
  stream ``x_t = rho x_{t-1} + sqrt(1-rho^2) eps_t`` for token-to-token overlap.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from statistics import NormalDist
from typing import Dict, List, Optional

import numpy as np

import threading

_EIGH_LOCK = threading.Lock()

T_GATE, T_UP, T_DOWN, T_PRED_NOISE, T_TOKENS, T_HASH = 0, 1, 2, 3, 4, 5

WEIGHT_STD = 0.02
PRED_NOISE_STD = 0.01


@dataclass(frozen=True)
class StackSpec:
    """Shape of one synthetic FFN stack (one entry per benchmark configuration)."""

    name: str
    seed: int
    n_layers: int
    d_model: int
    d_ff: int
    gated: bool
    wdtype: str  # "bf16" | "fp16"
    rank: int
    activity: float  # fraction of neurons with a positive gate per token
    n_tokens: int
    token_kind: str = "iid"  # "iid" | "iid_rms1" | "ar1"
    ar_rho: float = 0.0
    cache_frac: float = 0.0  # 0: all rows resident; else HBM cache rows / d_ff
    norm_eps: float = 1e-5
    batch: int = 1

    @property
    def k(self) -> int:
        return proposed_k(self.activity, self.d_ff)

    @property
    def cache_rows(self) -> int:
        return int(math.floor(self.cache_frac * self.d_ff)) if self.cache_frac > 0 else 0

    @property
    def row_bytes(self) -> int:
        return 2 * self.d_model

    @property
    def n_in(self) -> int:
        return 2 if self.gated else 1


def proposed_k(p: float, d_ff: int) -> int:
    """Selected neurons per token: 4 % above the expected active count, in units of 32."""
    return 32 * int(math.ceil(1.04 * p * d_ff / 32.0 - 1e-9))


SPECS: Dict[str, StackSpec] = {
    # the small case the oracle finishes in seconds
    "tiny": StackSpec("tiny", 0, 1, 256, 1024, True, "bf16", 32, 0.15, 16, "iid_rms1"),
    # four tied-shape tiny layers with a 50x larger down projection, so that the
    # partial features move the next layer's ranking visibly
    "tiny4": StackSpec("tiny4", 5, 4, 256, 1024, True, "bf16", 32, 0.15, 8, "iid_rms1"),
    "llama2-7b": StackSpec("llama2-7b", 1, 32, 4096, 11008, True, "bf16", 256, 0.15, 128, "iid"),
    "mistral-7b": StackSpec("mistral-7b", 2, 32, 4096, 14336, True, "bf16", 256, 0.12, 256, "ar1",
                            ar_rho=0.817, cache_frac=0.30),
    "opt-13b": StackSpec("opt-13b", 3, 40, 5120, 20480, False, "fp16", 256, 0.08, 128, "ar1",
                         ar_rho=0.851, cache_frac=0.20),
    "llama2-70b": StackSpec("llama2-70b", 4, 80, 8192, 28672, True, "bf16", 512, 0.10, 64, "ar1",
                            ar_rho=0.834, cache_frac=0.50),
}


@dataclass
class LayerArrays:
    """Host arrays of one layer, exactly as handed to the oracle and to ``ls_layer_create``.

    16-bit tensors are raw bit patterns (``uint16``); biases are ``float32``.
    ``w_down_t`` is neuron-major: row ``i`` is column ``i`` of the down projection.
    """

    d_model: int
    d_ff: int
    gated: bool
    wdtype: str
    rank: int
    norm_eps: float
    w_gate: np.ndarray  # [d_ff, d_model] uint16
    w_up: Optional[np.ndarray]  # [d_ff, d_model] uint16 or None when not gated
    w_down_t: np.ndarray  # [d_ff, d_model] uint16
    b_gate: np.ndarray  # [d_ff] float32
    pred_a: np.ndarray  # [d_model, rank] uint16
    pred_b: np.ndarray  # [rank, d_ff] uint16
    pred_c: np.ndarray  # [d_ff] float32
    b_down: Optional[np.ndarray] = None  # [d_model] float32
    meta: dict = field(default_factory=dict)
    act: str = "relu"  # "relu" (the sparsity source of the workloads) or "silu" (as Eq. 1 of the paper prints it)


def _rng(seed: int, layer: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, layer, tensor_id])))


def f32_to_bits16(a: np.ndarray, wdtype: str) -> np.ndarray:
    """Round float32 values to the 16-bit storage type (nearest even) and return the bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if wdtype == "fp16":
        return a.astype(np.float16).view(np.uint16)
    if wdtype != "bf16":
        raise ValueError(f"unknown weight dtype {wdtype!r}")
    import torch  # torch's conversion is a library rounding routine, much faster than numpy bit twiddling

    return torch.from_numpy(a).to(torch.bfloat16).view(torch.uint16).numpy()


def bits16_to_f32(bits: np.ndarray, wdtype: str) -> np.ndarray:
    """Exact widening of stored 16-bit patterns to float32 (used only to build the predictor)."""
    if wdtype == "fp16":
        return bits.view(np.float16).astype(np.float32)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def gate_bias(p: float, d_model: int) -> float:
    return -NormalDist().inv_cdf(1.0 - p) * WEIGHT_STD * math.sqrt(d_model)


def _normal_bits(seed: int, layer: int, tid: int, shape, std: float, wdtype: str) -> np.ndarray:
    out = np.empty(shape, dtype=np.float32)
    _rng(seed, layer, tid).standard_normal(out=out.reshape(-1), dtype=np.float32)
    out *= np.float32(std)
    return f32_to_bits16(out, wdtype)


def _svd_predictor(w_gate_f32: np.ndarray, rank: int, seed: int, layer: int, wdtype: str, svd_device: str):
    """Top-``rank`` right singular vectors of the gate matrix through the Gram matrix."""
    import torch

    F, d = w_gate_f32.shape
    dev = torch.device(svd_device)
    W = torch.from_numpy(w_gate_f32).to(dev)
    if dev.type == "cpu":
        W = W.double()
    else:
        torch.backends.cuda.matmul.allow_tf32 = False
    G = W.T @ W
    with _EIGH_LOCK:  # torch initialises its linear-algebra backend lazily and not thread-safely
        evals, evecs = torch.linalg.eigh(G)
    V = evecs[:, -rank:].flip(1).contiguous()  # [d, r], descending singular value
    Bt = (W @ V).float().cpu().numpy()  # [F, r]
    A = V.float().cpu().numpy()
    noise = np.empty((rank, F), dtype=np.float32)
    _rng(seed, layer, T_PRED_NOISE).standard_normal(out=noise.reshape(-1), dtype=np.float32)
    B = np.ascontiguousarray(Bt.T) + np.float32(PRED_NOISE_STD) * noise
    return f32_to_bits16(A, wdtype), f32_to_bits16(B, wdtype)


def make_layer(spec: StackSpec, layer: int, svd_device: str = "cpu", down_scale: float = 1.0) -> LayerArrays:
    """Arrays of layer ``layer`` of stack ``spec`` (deterministic in ``(spec.seed, layer)``)."""
    F, d = spec.d_ff, spec.d_model
    w_gate = _normal_bits(spec.seed, layer, T_GATE, (F, d), WEIGHT_STD, spec.wdtype)
    w_up = _normal_bits(spec.seed, layer, T_UP, (F, d), WEIGHT_STD, spec.wdtype) if spec.gated else None
    w_down_t = _normal_bits(spec.seed, layer, T_DOWN, (F, d), WEIGHT_STD * down_scale, spec.wdtype)
    b = np.full((F,), gate_bias(spec.activity, d), dtype=np.float32)
    pa, pb = _svd_predictor(bits16_to_f32(w_gate, spec.wdtype), spec.rank, spec.seed, layer, spec.wdtype, svd_device)
    # (eps as the fp32 value the C ABI's `float` field carries, so that the oracle and the library see the same number)
    return LayerArrays(d, F, spec.gated, spec.wdtype, spec.rank, float(np.float32(spec.norm_eps)), w_gate, w_up, w_down_t, b, pa, pb,
                       b.copy(), None, {"spec": spec.name, "layer": layer})


def make_stack(spec: StackSpec, n_layers: Optional[int] = None, svd_device: str = "cpu",
               down_scale: float = 1.0, threads: int = 8) -> List[LayerArrays]:
    n = spec.n_layers if n_layers is None else n_layers
    if n <= 2 or threads <= 1:
        return [make_layer(spec, l, svd_device, down_scale) for l in range(n)]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(lambda l: make_layer(spec, l, svd_device, down_scale), range(n)))


def make_tokens(spec: StackSpec, n_tokens: Optional[int] = None, stream: int = 0) -> np.ndarray:
    """Inputs ``x_{0,t}`` to the first layer, float32 ``[n_tokens, d_model]``."""
    n = spec.n_tokens if n_tokens is None else n_tokens
    d = spec.d_model
    eps = _rng(spec.seed, 1_000_000 + stream, T_TOKENS).standard_normal((n, d)).astype(np.float64)
    if spec.token_kind == "ar1":
        rho = spec.ar_rho
        x = np.empty_like(eps)
        x[0] = eps[0]
        c = math.sqrt(1.0 - rho * rho)
        for t in range(1, n):
            x[t] = rho * x[t - 1] + c * eps[t]
    else:
        x = eps
        if spec.token_kind == "iid_rms1":
            x = x / np.sqrt(np.mean(x * x, axis=1, keepdims=True))
    return np.ascontiguousarray(x.astype(np.float32))


def tied_duplicate_layer(base: LayerArrays, pairs) -> LayerArrays:
    """Copy of ``base`` in which predictor column ``dst`` duplicates column ``src`` for each pair,
    so that the two neurons receive exactly equal scores (tie-break test input)."""
    import copy

    out = copy.copy(base)
    out.pred_b = base.pred_b.copy()
    out.pred_c = base.pred_c.copy()
    for src, dst in pairs:
        out.pred_b[:, dst] = out.pred_b[:, src]
        out.pred_c[dst] = out.pred_c[src]
    return out


@dataclass
class HashPredictorArrays:
    """Host arrays of a stacked hashing predictor with random tables (trained ones do not exist offline), in both forms:
    sign arrays in {-1,+1} for the oracle and the same signs packed one bit per component for the library
    (+1 -> 1, component c at bit c % 32 of word c // 32)."""

    d_model: int
    rank: int
    tau: int
    d_code: int
    n_layers: int
    d_ff: int
    wdtype: str
    pca: np.ndarray        # [d_model, rank] uint16 bit patterns (the layer's PCA projection)
    w1: np.ndarray         # [rank, tau] float32
    w_signs: List[np.ndarray]   # n_layers - 1 arrays [d_code, tau] int8
    t_signs: List[np.ndarray]   # n_layers arrays [2^tau, d_code] int8
    code_signs: np.ndarray      # [d_ff, d_code] int8
    w_bits: np.ndarray     # [n_layers - 1, tau, d_code // 32] uint32
    t_bits: np.ndarray     # [n_layers, 2^tau, d_code // 32] uint32
    code_bits: np.ndarray  # [d_ff, d_code // 32] uint32


def pack_signs(signs: np.ndarray) -> np.ndarray:
    """[..., d] signs in {-1,+1} -> [..., d // 32] uint32, bit (c % 32) of word (c // 32) set where the sign is +1."""
    b = np.ascontiguousarray(np.asarray(signs) > 0, dtype=np.uint8)
    if b.shape[-1] % 32:
        raise ValueError("the number of components must be a multiple of 32")
    return np.ascontiguousarray(np.packbits(b, axis=-1, bitorder="little")).view(np.uint32)


def make_hash_predictor(base: LayerArrays, seed: int, layer: int, tau: int = 8, d_code: int = 256, n_layers: int = 5) -> HashPredictorArrays:
    """Random stacked-hashing tables on top of a layer's PCA projection (the paper's default shape: five layers, tau = 8,
    d = 256).  Random tables serve parity and throughput only: they predict nothing."""
    rng = _rng(seed, layer, T_HASH)
    w1 = rng.standard_normal((base.rank, tau)).astype(np.float32)
    pm = lambda shape: (rng.integers(0, 2, size=shape, dtype=np.int8) * 2 - 1).astype(np.int8)
    w_signs = [pm((d_code, tau)) for _ in range(n_layers - 1)]
    t_signs = [pm((2 ** tau, d_code)) for _ in range(n_layers)]
    code_signs = pm((base.d_ff, d_code))
    w_bits = np.stack([pack_signs(w.T) for w in w_signs]) if w_signs else np.zeros((0, tau, d_code // 32), dtype=np.uint32)
    t_bits = np.stack([pack_signs(t) for t in t_signs])
    return HashPredictorArrays(base.d_model, base.rank, tau, d_code, n_layers, base.d_ff, base.wdtype, base.pred_a, w1, w_signs, t_signs,
                               code_signs, np.ascontiguousarray(w_bits), np.ascontiguousarray(t_bits), np.ascontiguousarray(pack_signs(code_signs)))
