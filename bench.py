#!/usr/bin/env python
"""Benchmark of the speculate-and-refine sparse FFN decode path.

One *step* is one decode token through the whole synthetic FFN stack: for every layer the predictor scores of
the next layer are refined after each of the K stages, the selected gate/up rows are streamed, and the sparse down
projection accumulates the surviving rows.  ``value`` is tokens/s with the token inputs already resident in HBM;
``e2e`` is the same loop with a pinned-host input copied in and the result copied out every step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload llama2-7b] [--chunks 8]

The default workload (``llama2-7b``) is fully resident and runs as one kernel per token.  Workloads with a cache budget
(``mistral-7b``, ``opt-13b``, ``llama2-70b``) keep their weights in pinned host memory behind an HBM neuron cache and
run layer by layer; their line adds the cache statistics and the host-link bound.

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the stack on its own
token stream ("replicas only": the batch-1 path has no exchange step); the line reports the sum over ranks divided
by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "sparse-FFN decode tokens/s and achieved HBM GB/s on active-neuron weight bytes"
REL_L2_TOL, MAX_ABS_TOL = 1e-3, 1e-2  # output tolerance of the parity gate (spec tolerance)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--chunks", type=int, default=8, help="K: stages per layer (Section 4.3.1 of the paper uses 8)")
    ap.add_argument("--k", type=int, default=0, help="selected neurons per layer (default: the workload's)")
    ap.add_argument("--batch", type=int, default=0, help="tokens decoded together (cached workloads; default: the workload's)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (debugging only)")
    ap.add_argument("--distinct-layers", type=int, default=0, help="cached workloads: distinct layers to build (tiled over the stack)")
    ap.add_argument("--no-graph", action="store_true", help="launch every call from the host instead of one CUDA graph per token")
    ap.add_argument("--per-layer", action="store_true", help="one kernel per layer (ls_sparse_ffn_step) instead of one per token")
    ap.add_argument("--phases", action="store_true", help="also print the per-phase timeline of the whole-token kernel (stderr)")
    ap.add_argument("--predictors", action="store_true",
                    help="also time one ranking of a layer's neurons by the linear predictor (ls_predict) and by a stacked hashing "
                         "predictor of the paper's default shape with random tables (ls_hash_predict); stderr")
    ap.add_argument("--miss-path", default="gather", choices=["gather", "lane"],
                    help="cached workloads: misses by a gather kernel reading pinned host memory, or by the host I/O lane (cudaMemcpyAsync)")
    ap.add_argument("--cpu-sample-layers", type=int, default=2)
    return ap.parse_args()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20",
                                          "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except Exception:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info

        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_layer_step_seconds(arrays, spec, K, n_steps, warmup=0, k=None):
    """Times the oracle's sparse step (predict, K stages with refinement, down projection) as it stands."""
    from oracle import leanstream_oracle as orc
    from paper_2609_03079_b200 import workload as wl

    k = spec.k if k is None else k
    layers = [orc.OracleLayer.from_arrays(a) for a in arrays]
    toks = wl.make_tokens(spec, max(1, (n_steps + warmup + len(layers) - 1) // len(layers) + 1))
    times = []
    it = 0
    t_idx = 0
    while it < n_steps + warmup:
        x = toks[t_idx % len(toks)].astype(np.float64)
        t_idx += 1
        order, _ = orc.select_batch(layers[0], x[None], k)
        for n, L in enumerate(layers):
            if it >= n_steps + warmup:
                break
            nxt = layers[(n + 1) % len(layers)]
            t0 = time.perf_counter()
            res = orc.sparse_ffn_step(L, nxt, x, order, K, k)
            dt = time.perf_counter() - t0
            if it >= warmup:
                times.append(dt)
            it += 1
            x = res["xtilde"][K][0]
            order = res["refine_orders"][K]
    return times


def cpu_baseline(arrays, spec, K, n_layers, n_cpu, k=None):
    """The oracle as it stands on this machine's host cores: once with the BLAS library's default threads and once limited to
    one thread.  Most of the oracle's time is single-threaded Python (the ranking is a ``sorted`` over all neurons per
    evaluation), so ``cores`` is what was AVAILABLE to its matrix products, not a parallel efficiency claim."""
    t0 = time.perf_counter()
    times = oracle_layer_step_seconds(arrays, spec, K, n_cpu, warmup=0, k=k)
    wall = time.perf_counter() - t0
    val = 1.0 / (float(np.mean(times)) * n_layers)
    val1 = None
    try:
        from threadpoolctl import threadpool_limits

        with threadpool_limits(limits=1, user_api="blas"):
            t1 = oracle_layer_step_seconds(arrays, spec, K, max(2, n_cpu // 6), warmup=0, k=k)
        val1 = 1.0 / (float(np.mean(t1)) * n_layers)
    except Exception:
        pass
    return {"value": val, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "value_one_thread": val1,
            "threads": "BLAS threads available to the matrix products; the ranking (a Python sort per evaluation) is single-threaded",
            "sample": f"{len(times)} layer-steps on {len(arrays)} distinct layers, scaled to {n_layers} layers; {wall:.1f} s"}


def run_reference(args):
    """Reference arm: the CPU oracle on this machine's host cores, same metric and workload, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch

    from paper_2609_03079_b200 import workload as wl

    spec = wl.SPECS[args.workload]
    n_layers = args.layers or spec.n_layers
    k = args.k or spec.k
    svd_dev = "cuda" if torch.cuda.is_available() else "cpu"
    arrays = [wl.make_layer(spec, l, svd_device=svd_dev) for l in range(min(args.cpu_sample_layers, n_layers))]
    steps = max(1, args.steps)
    t0 = time.perf_counter()
    times = oracle_layer_step_seconds(arrays, spec, args.chunks, steps, args.warmup, k=k)
    wall = time.perf_counter() - t0
    t_layer = float(np.mean(times))
    value = 1.0 / (t_layer * n_layers)
    sample = (f"each of the {len(times)} timed steps is ONE layer-step (K={args.chunks}, k={k}) on one of {len(arrays)} distinct layers of "
              f"the {spec.name} stack, not a whole token; tokens/s = 1 / (mean layer-step time x {n_layers} layers), so ms_per_step "
              f"is an extrapolation that was never spent")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": steps,
        "warmup": args.warmup, "ms_per_step": t_layer * n_layers * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec.name, "n_layers": n_layers, "d_model": spec.d_model, "d_ff": spec.d_ff, "k": k,
                   "chunks": args.chunks, "batch": 1},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": wall,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------------------------
def values_close(got, ref, scale_ref=None):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    base = ref if scale_ref is None else np.asarray(scale_ref, np.float64)
    rel = float(np.linalg.norm(got - ref)) / max(float(np.linalg.norm(base)), 1e-30)
    mx = float(np.max(np.abs(got - ref))) if got.size else 0.0
    return rel <= REL_L2_TOL and mx <= MAX_ABS_TOL * max(float(np.max(np.abs(base))), 1e-30), rel


def mask_to_set(mask, F):
    bits = np.unpackbits(np.ascontiguousarray(mask).view(np.uint8), bitorder="little")[:F]
    return set(np.flatnonzero(bits).tolist())


def parity_gate_stack(ls, wl, spec, host_arrays, stack, layers, x_buf, X0, sels, K, k):
    """One traced token through the benchmarked launch configuration, outside the timed region: for every layer whose host
    arrays are at hand, the selection entering it, its output, its partial features and every refined set are checked
    against the oracle (sets bit-exact from the GPU's own feature bits).  Raises if anything differs."""
    import torch

    from oracle import leanstream_oracle as orc

    trace = ls.StackTrace(stack, k, n_chunks=K)
    x_buf.copy_(X0[1:2])
    ls.ls_predict(layers[0], x_buf, k, sels[0])
    x_out = torch.empty_like(x_buf)
    ls.ls_stack_decode(stack, x_buf, x_out, sels[0], K, k, sels[1], trace)
    torch.cuda.synchronize()
    X, S = trace.x.cpu().numpy(), trace.sel_idx.cpu().numpy()
    XT, M = trace.xtilde.cpu().numpy(), trace.refine_masks.cpu().numpy().view(np.uint32)
    checked = 0
    idxs = sorted(host_arrays)
    OL = {l: orc.OracleLayer.from_arrays(host_arrays[l]) for l in idxs}
    quality = {"stage": [f"{j}/{K}" for j in range(K + 1)], "importance_ratio": [], "top10_recall": []}
    for l in idxs:
        order = S[l, :k].astype(np.int64)
        if order.tolist() != orc.topk_order(orc.predictor_scores(OL[l], X[l]), k).tolist():
            raise RuntimeError(f"parity gate: selection entering layer {l} differs from the oracle")
        res = orc.sparse_ffn_step(OL[l], None, X[l], order, K)
        ok, rel = values_close(X[l + 1] - X[l], res["y"][0])
        if not ok:
            raise RuntimeError(f"parity gate: output of layer {l} off (rel-L2 {rel:.2e})")
        for j in range(1, K + 1):
            ok, rel = values_close(XT[l, j] - XT[l, j - 1], res["xtilde"][j][0] - res["xtilde"][j - 1][0], scale_ref=res["y"][0])
            if not ok:
                raise RuntimeError(f"parity gate: partial feature {j} of layer {l} off (rel-L2 {rel:.2e})")
        if l + 1 in OL:
            # what the next layer truly activates on its real input: the yardstick of the paper's validation across
            # refinement steps (Section 4.3: stages 0/K ... K/K, Importance Ratio and recall of the top 10 %)
            Ln = OL[l + 1]
            true_abs = np.abs(orc.neuron_activations(Ln, orc.mlp_input(Ln, X[l + 1]), np.arange(Ln.d_ff)))
            for j in range(K + 1):
                got = mask_to_set(M[l, j], spec.d_ff)
                want = set(orc.topk_order(orc.predictor_scores(Ln, XT[l, j]), k).tolist())
                if got != want:
                    raise RuntimeError(f"parity gate: refined set {j} of layer {l} differs from the oracle")
                if quality is not None and not quality["importance_ratio"][j:]:
                    quality["importance_ratio"].append(round(orc.importance_ratio(sorted(got), true_abs), 4))
                    quality["top10_recall"].append(round(orc.top_fraction_recall(sorted(got), true_abs, 0.10), 4))
        checked += 1
    out = {"layers_checked": checked, "token": 1, "what": "selections and refined sets bit-exact, outputs within rel-L2 1e-3"}
    if quality is not None and quality["importance_ratio"]:
        out["refine_quality_layer0_to_1"] = quality
    return out


def phase_table(ls, stack, layers, x_buf, X0, sels, K, k):
    """Per-phase timeline of the whole-token kernel from the time stamps it exports (median / slowest CTA, mean over layers)."""
    import torch

    tr = ls.StackTrace(stack, k, phases=True)
    x_buf.copy_(X0[2:3])
    ls.ls_predict(layers[0], x_buf, k, sels[0])
    ls.ls_stack_decode(stack, x_buf, x_buf, sels[0], K, k, sels[1], tr)
    torch.cuda.synchronize()
    P = tr.phase_ns.cpu().numpy().astype(np.float64)
    names = ["layer start", "S: partial output written", "barrier 1 passed", "P1: features, partial latents written", "barrier 2 passed",
             "P2: latents summed", "barrier 3 passed", "P3: scores written", "barrier 4 passed", "P4: own slice of the next selection", "layer end"]
    ref = np.median(P[:, :, 0], axis=1, keepdims=True)
    rows = []
    for i, nm in enumerate(names):
        rel = (P[1:, :, i] - ref[1:]) / 1000.0
        rows.append((nm, float(np.median(rel, axis=1).mean()), float(rel.max(axis=1).mean())))
    return rows


def predictor_times(ls, wl, torch, spec, la, layer, x_buf, k, local, reps=200):
    """One ranking of a layer's neurons (scores of all d_ff neurons + exact top-k) by each predictor, CUDA events around
    `reps` back-to-back calls on the current stream.  The hashing predictor has the paper's default shape (five layers,
    tau = 8, 256-bit codes) and random tables: same arithmetic and memory traffic as a trained one, no predictive value."""
    ha = wl.make_hash_predictor(la, spec.seed, 0)
    hp = ls.ls_hash_predictor_create(ha, local)
    sel = ls.Selection(spec.d_ff, k, local)
    out = {}
    for name, call in (("ls_predict (rank-%d linear, fp64)" % spec.rank, lambda: ls.ls_predict(layer, x_buf, k, sel)),
                       ("ls_hash_predict (5 layers, tau 8, 256-bit codes)", lambda: ls.ls_hash_predict(hp, x_buf.view(-1), k, sel))):
        for _ in range(10):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) / reps * 1e3
        print(f"  {name:52s} {out[name]:8.2f} us per ranking of {spec.d_ff} neurons (k = {k})", file=sys.stderr)
    hp.close()
    return out


def run_resident(args, ls, wl, replicas, torch, dist, world, rank, local, dev, spec):
    n_layers = args.layers or spec.n_layers
    K, k, d = args.chunks, args.k or spec.k, spec.d_model

    # ---- build the stack (seeded, synthetic); host arrays are dropped once uploaded
    t_build = time.perf_counter()
    from concurrent.futures import ThreadPoolExecutor

    keep_host = {}
    layers = [None] * n_layers

    def make(l):
        return l, wl.make_layer(spec, l, svd_device=f"cuda:{local}")

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        for l, la in ex.map(make, range(n_layers)):
            layers[l] = ls.ls_layer_create(la, local)
            if rank == 0 and l < args.cpu_sample_layers:
                keep_host[l] = la
    t_build = time.perf_counter() - t_build

    n_tok = max(spec.n_tokens, 4)
    X0_host = torch.from_numpy(wl.make_tokens(spec, n_tok, stream=replicas.stream_of_rank(rank))).pin_memory()
    X0 = X0_host.to(dev)
    x_buf = torch.zeros(1, d, dtype=torch.float32, device=dev)
    out_host = torch.zeros(1, d, dtype=torch.float32).pin_memory()
    sels = [ls.Selection(spec.d_ff, k, local) for _ in range(2)]

    stack = None if args.per_layer else ls.ls_stack_create(layers)

    def decode_token_layers():
        ls.ls_predict(layers[0], x_buf, k, sels[0])
        for n in range(n_layers):
            nxt = layers[n + 1] if n + 1 < n_layers else layers[n]
            ls.ls_sparse_ffn_step(layers[n], nxt, x_buf, x_buf, sels[n % 2], K, k, sels[(n + 1) % 2], None)

    def decode_token():
        if stack is None:
            return decode_token_layers()
        ls.ls_predict(layers[0], x_buf, k, sels[0])
        ls.ls_stack_decode(stack, x_buf, x_buf, sels[0], K, k, sels[1])

    # ---- warm-up, parity gate, launch count per token, optional CUDA graph of one token
    x_buf.copy_(X0[0:1])
    for _ in range(2):
        decode_token()
    torch.cuda.synchronize()
    gate = None
    if rank == 0 and stack is not None:
        gate = parity_gate_stack(ls, wl, spec, keep_host, stack, layers, x_buf, X0, sels, K, k)
    n0 = ls.ls_kernel_launches()
    decode_token()
    torch.cuda.synchronize()
    launches_per_token = ls.ls_kernel_launches() - n0
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            decode_token()
    run_token = graph.replay if graph is not None else decode_token

    def loop(n_steps, e2e):
        for t in range(n_steps):
            if e2e:
                x_buf.copy_(X0_host[t % n_tok:t % n_tok + 1], non_blocking=True)
            else:
                x_buf.copy_(X0[t % n_tok:t % n_tok + 1])
            run_token()
            if e2e:
                out_host.copy_(x_buf, non_blocking=True)

    def timed(n_steps, e2e):
        """(slowest rank's milliseconds for n_steps, steps of all ranks): barrier + synchronize on both sides."""
        loop(args.warmup, e2e)
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        loop(n_steps, e2e)
        b.record()
        torch.cuda.synchronize()
        replicas.barrier()
        return replicas.aggregate(a.elapsed_time(b), n_steps, dev)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_total, steps_total = timed(args.steps, False)
    clocks = sampler.stop() if rank == 0 else None
    ms_e2e, steps_e2e = timed(args.steps, True)
    status = [ls.ls_layer_status(L) for L in layers]
    assert all(s == 0 for s in status), f"device status {status}"

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        # ---- roofline pass: the dominant kernel timed with CUDA events on its own stream
        ls.ls_timing_enable(True)
        n_prof = min(args.steps, 4)
        for t in range(n_prof):
            x_buf.copy_(X0[t % n_tok:t % n_tok + 1])
            decode_token()
        torch.cuda.synchronize()
        ls.ls_timing_enable(False)
        n_st, ms_st = ls.ls_timing_read(ls.LS_TIMED_STACK)
        n_fz, ms_fz = ls.ls_timing_read(ls.LS_TIMED_FUSED)
        for kind in (ls.LS_TIMED_GATEUP, ls.LS_TIMED_DOWN, ls.LS_TIMED_PREDICT):
            ls.ls_timing_read(kind)
        # surviving rows (up and down bytes) measured on one traced token
        x_buf.copy_(X0[0:1])
        ls.ls_predict(layers[0], x_buf, k, sels[0])
        surv = []
        for n in range(n_layers):
            nxt = layers[n + 1] if n + 1 < n_layers else layers[n]
            tr = ls.StepTrace(layers[n], nxt, K, 1, k)
            ls.ls_sparse_ffn_step(layers[n], nxt, x_buf, x_buf, sels[n % 2], K, k, sels[(n + 1) % 2], tr)
            m = tr.survive_mask.cpu().numpy().view(np.uint32)
            surv.append(int(np.unpackbits(m.view(np.uint8)).sum()))
        k_surv = float(np.mean(surv))
        row = spec.row_bytes
        # Algorithmic bytes of a layer step: the first row of every selected bundle, and the rest of the bundle only for the
        # neurons that survive the ReLU (exact: a zero activation makes the up row irrelevant).
        active_bytes_layer = k * row + k_surv * spec.n_in * row
        all_rows_bytes_layer = k * spec.n_in * row + k_surv * row
        ms_step = ms_total / args.steps
        us_layer = ms_step * 1e3 / n_layers
        active_gbs = active_bytes_layer / (us_layer * 1e-6) / 1e9
        traffic_db = {}
        tp = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(tp):
            with open(tp) as f:
                traffic_db = json.load(f)
        with open(os.path.join(ROOT, "paper_2609_03079_b200", "csrc", "ls_token.cuh"), "rb") as f:
            kernel_sha = hashlib.sha1(f.read()).hexdigest()[:12]
        if n_st:
            kname, bytes_launch, us_launch, n_timed = "ls_token_kernel", active_bytes_layer * n_layers, ms_st / n_st * 1e3, n_st
        else:
            kname, bytes_launch, us_launch, n_timed = "ls_token_kernel (one layer per launch)", active_bytes_layer, ms_fz / max(n_fz, 1) * 1e3, n_fz
        per_layer_traffic = traffic_db.get("dram_bytes_per_layer")
        traffic = per_layer_traffic * (n_layers if n_st else 1) if per_layer_traffic else None
        k_gbs = bytes_launch / (us_launch * 1e-6) / 1e9 if n_timed else None
        phases = phase_table(ls, stack, layers, x_buf, X0, sels, K, k) if (args.phases and stack is not None) else None
        if phases:
            for nm, med, mx in phases:
                print(f"  {nm:42s} median {med:7.2f} us   slowest CTA {mx:7.2f} us", file=sys.stderr)

        if args.predictors and keep_host:
            predictor_times(ls, wl, torch, spec, keep_host[0], layers[0], x_buf, k, local)

        arrays = [keep_host[l] for l in sorted(keep_host)]
        cpu = cpu_baseline(arrays, spec, K, n_layers, 48 * len(arrays), k=k)  # fifteen to twenty seconds of CPU work

        line = {
            "metric": METRIC, "value": steps_total / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights, f32 accumulate, f64 predictor scores", "data": "synthetic",
            "config": {"workload": spec.name, "n_layers": n_layers, "d_model": d, "d_ff": spec.d_ff, "pred_rank": spec.rank, "k": k,
                       "chunks": K, "batch": 1, "cache_rows": 0, "parallelism": "replicas only" if world > 1 else "1 gpu",
                       "l2": "inputs larger than L2 (%.2f GB of weight rows touched per token)" % (active_bytes_layer * n_layers / 1e9),
                       "cuda_graph": graph is not None, "kernel_per": "layer" if stack is None else "token"},
            "us_per_layer": us_layer, "active_bytes_per_layer": active_bytes_layer,
            "active_bytes_per_layer_if_up_rows_of_all_selected": all_rows_bytes_layer, "k_surviving_mean": k_surv,
            "active_gbs": active_gbs, "active_frac_of_hbm_peak": active_gbs / peaks["hbm_gbs"],
            "roofline": {"bound": "hbm", "kernel": kname, "achieved": k_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": (k_gbs / peaks["hbm_gbs"]) if k_gbs else None, "traffic": traffic, "peak_kind": peak_kind,
                         "bytes_per_launch": bytes_launch, "us_per_launch": us_launch, "launches_timed": n_timed,
                         "traffic_source": traffic_db.get("source"), "traffic_kernel_sha": traffic_db.get("kernel_sha"),
                         "kernel_sha": kernel_sha, "traffic_stale": traffic_db.get("kernel_sha") not in (None, kernel_sha)},
            "cpu_baseline": cpu,
            "e2e": {"value": steps_e2e / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": d * 4, "d2h_bytes_per_step": d * 4},
            "gpu_launches": launches_per_token * args.steps, "launches_per_token": launches_per_token,
            "parity_gate": gate, "clocks": clocks, "build_s": t_build,
        }
        if phases:
            line["phases_us"] = [{"phase": nm, "median": med, "slowest_cta": mx} for nm, med, mx in phases]
        print(json.dumps(line))
    if stack is not None:
        stack.close()
    for L in layers:
        L.close()


# ---------------------------------------------------------------------------------------------------------------------
def host_link_gbs(torch, dev):
    """Peak of the host link as this process sees it: one large pinned host-to-device copy, best of five."""
    n = 256 << 20
    h = torch.empty(n, dtype=torch.uint8).pin_memory()
    g = torch.empty(n, dtype=torch.uint8, device=dev)
    best = 0.0
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.copy_(h, non_blocking=True)
        b.record()
        torch.cuda.synchronize()
        best = max(best, n / (a.elapsed_time(b) * 1e-3) / 1e9)
    return best


def mem_available_bytes():
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except Exception:
        pass
    return None


def run_cached(args, ls, wl, replicas, torch, dist, world, rank, local, dev, spec):
    """Workloads whose weights live in pinned host memory behind an HBM neuron cache: layer by layer through
    ls_sparse_ffn_step (refinement between the stages drives the prefetch of the next layer, misses travel on the layer's
    copy stream).  The first eight tokens fill the caches and are reported apart (cold start)."""
    from oracle import leanstream_oracle as orc

    n_layers = args.layers or spec.n_layers
    K, k, d, F = args.chunks, args.k or spec.k, spec.d_model, spec.d_ff
    B = args.batch or spec.batch
    ls.ls_set_option(ls.LS_OPT_MISS_PATH, ls.LS_MISS_PATH_LANE if args.miss_path == "lane" else ls.LS_MISS_PATH_GATHER)
    bundle = spec.row_bytes * (3 if spec.gated else 2)
    cache_rows = spec.cache_rows
    max_sel = min(F, B * k)
    # distinct layers that fit in host memory (pinned) with room to spare; tiled over the stack when fewer than n_layers
    avail = mem_available_bytes()
    per_layer_host = F * bundle * 2.2  # pinned store + generator arrays alive while a layer is built
    n_distinct = args.distinct_layers or n_layers
    if avail is not None:
        n_distinct = max(1, min(n_distinct, int(0.6 * avail / (F * bundle)), max(1, int(0.8 * avail / per_layer_host))))
    n_distinct = min(n_distinct, n_layers)

    t_build = time.perf_counter()
    distinct, keep_host = [], {}
    for l in range(n_distinct):
        la = wl.make_layer(spec, l, svd_device=f"cuda:{local}")
        distinct.append(ls.ls_layer_create(la, local, cache_rows=cache_rows, max_batch=B, max_sel=max_sel))
        if rank == 0 and l < 2:
            keep_host[l] = la
        del la
    t_build = time.perf_counter() - t_build
    layers = [distinct[n % n_distinct] for n in range(n_layers)]

    warm = 8
    n_tok = warm + args.steps
    toks = [wl.make_tokens(spec, n_tok, stream=replicas.stream_of_rank(rank) * 16 + b) for b in range(B)]
    X0 = torch.from_numpy(np.stack(toks, axis=1)).to(dev)  # [n_tok, B, d]
    x_buf = torch.zeros(B, d, dtype=torch.float32, device=dev)
    sels = [ls.Selection(F, max_sel, local) for _ in range(2)]

    nwords = (F + 31) // 32
    snap = [torch.zeros(nwords, dtype=torch.int32, device=dev) for _ in range(2)]

    def bits(m):
        return int(np.unpackbits(m.cpu().numpy().view(np.uint8)).sum())

    def decode_token(t, record=None, redund=None):
        x_buf.copy_(X0[t])
        ls.ls_predict(layers[0], x_buf, k, sels[0])
        for n in range(n_layers):
            nxt = layers[n + 1] if n + 1 < n_layers else layers[n]
            if record is not None:
                record[n].append(sels[n % 2].order().tolist())
            watch = redund is not None and nxt is not layers[n]
            if watch:
                ls.ls_cache_snapshot(nxt, snap[0])  # the next layer's residents before this layer's refinements prefetch
            ls.ls_sparse_ffn_step(layers[n], nxt, x_buf, x_buf, sels[n % 2], K, k, sels[(n + 1) % 2], None)
            if watch:
                # loading redundancy (Section 4.3): rows the refinements brought in that the final set does not use, over the
                # rows the final set truly lacked
                ls.ls_cache_snapshot(nxt, snap[1])
                final = sels[(n + 1) % 2].mask
                fetched = snap[1] & ~snap[0]
                redund[0] += bits(fetched & ~final)
                redund[1] += bits(final & ~snap[0])

    def stats_sum():
        tot = {}
        for L in distinct:
            for key, v in ls.ls_cache_stats(L).items():
                tot[key] = tot.get(key, 0) + v
        return tot

    def timed_tokens(t0, t1):
        torch.cuda.synchronize()
        s0 = stats_sum()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for t in range(t0, t1):
            decode_token(t)
        b.record()
        torch.cuda.synchronize()
        s1 = stats_sum()
        return a.elapsed_time(b), {key: s1[key] - s0[key] for key in s1}

    link = host_link_gbs(torch, dev)
    n0 = ls.ls_kernel_launches()
    ms_warm, st_warm = timed_tokens(0, warm)
    launches_per_token = (ls.ls_kernel_launches() - n0) / warm
    replicas.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_local, st = timed_tokens(warm, n_tok)
    clocks = sampler.stop() if rank == 0 else None
    replicas.barrier()
    ms_total, steps_total = replicas.aggregate(ms_local, args.steps * B, dev)
    status = [ls.ls_layer_status(L) for L in distinct]
    assert all(s == 0 for s in status), f"device status {status}"

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        # ---- untimed window on the same caches: the request trace for the LRU comparison, and the parity sample
        win = min(16, args.steps)
        record = [[] for _ in range(n_layers)]
        s0 = stats_sum()
        redund = [0, 0]
        for t in range(warm, warm + win):
            decode_token(t, record, redund if t < warm + 4 else None)
        torch.cuda.synchronize()
        s1 = stats_sum()
        ours_window = (s1["misses"] - s0["misses"]) / max(1, (s1["hits"] - s0["hits"]) + (s1["misses"] - s0["misses"]))
        lru = float(np.mean([orc.lru_miss_ratio(record[n], cache_rows) for n in range(0, n_layers, max(1, n_layers // 8))]))
        # parity sample: a seeded choice of (token, layer) pairs among the layers whose host arrays are at hand
        parity = None
        if keep_host and B == 1:
            rng = np.random.default_rng(1234)
            OL = {l: orc.OracleLayer.from_arrays(keep_host[l]) for l in keep_host}
            pairs = [(int(rng.integers(warm, n_tok)), l) for l in sorted(keep_host) for _ in range(2)]
            worst = 0.0
            for t, l in pairs:
                if l + 1 not in OL and l != max(OL):
                    continue
                x = X0[t].clone()
                sel, sel_next = ls.Selection(F, k, local), ls.Selection(F, k, local)
                gl = distinct[l]
                gn = distinct[l + 1] if l + 1 in OL else gl
                ls.ls_predict(gl, x, k, sel)
                trace = ls.StepTrace(gl, gn, K, 1, k)
                x_out = torch.empty_like(x)
                ls.ls_sparse_ffn_step(gl, gn, x, x_out, sel, K, k, sel_next, trace)
                torch.cuda.synchronize()
                xn = x.cpu().numpy()[0]
                order = sel.order()
                if order.tolist() != orc.topk_order(orc.predictor_scores(OL[l], xn), k).tolist():
                    raise RuntimeError(f"parity sample: selection of layer {l}, token {t} differs from the oracle")
                res = orc.sparse_ffn_step(OL[l], None, xn, order, K)
                ok, rel = values_close(x_out.cpu().numpy()[0] - xn, res["y"][0])
                worst = max(worst, rel)
                if not ok:
                    raise RuntimeError(f"parity sample: output of layer {l}, token {t} off (rel-L2 {rel:.2e})")
                ON = OL[l + 1] if l + 1 in OL else OL[l]
                xt = trace.xtilde.cpu().numpy()
                M = trace.refine_masks.cpu().numpy().view(np.uint32)
                for j in range(K + 1):
                    if mask_to_set(M[j], F) != set(orc.topk_order(orc.predictor_scores(ON, xt[j, 0]), k).tolist()):
                        raise RuntimeError(f"parity sample: refined set {j} of layer {l}, token {t} differs from the oracle")
            parity = {"pairs": len(pairs), "worst_rel_l2": worst, "what": "selections and refined sets bit-exact, outputs within rel-L2 1e-3"}

        ms_step = ms_total / args.steps
        us_layer = ms_step * 1e3 / n_layers
        reqs = st["hits"] + st["misses"]
        miss_bytes = st["h2d_bytes"]
        # bytes the stage kernels read from HBM (this path reads all input rows of every selected neuron; surviving down
        # rows are not counted: their number is not measured here) and bytes that crossed the host link
        sel_bytes = args.steps * n_layers * min(F, B * k) * spec.n_in * spec.row_bytes
        t_s = ms_local * 1e-3
        arrays = [keep_host[l] for l in sorted(keep_host)]
        cpu = cpu_baseline(arrays, spec, K, n_layers, 12 * len(arrays), k=k) if arrays else None
        line = {
            "metric": METRIC, "value": steps_total / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": f"{spec.wdtype} weights, f32 accumulate, f64 predictor scores", "data": "synthetic",
            "config": {"workload": spec.name, "n_layers": n_layers, "distinct_layers": n_distinct,
                       "tiling": None if n_distinct == n_layers else f"{n_distinct} distinct layers tiled over {n_layers} positions (host memory / build time); positions that share a layer share its cache",
                       "d_model": d, "d_ff": F, "gated": spec.gated, "pred_rank": spec.rank, "k": k, "chunks": K, "batch": B,
                       "cache_rows": cache_rows, "cache_frac": spec.cache_frac, "miss_path": args.miss_path, "token_stream": f"AR(1), rho = {spec.ar_rho}",
                       "parallelism": "replicas only" if world > 1 else "1 gpu", "cuda_graph": False, "kernel_per": "operation",
                       "l2": "inputs larger than L2 (%.2f GB of rows per token)" % (sel_bytes / args.steps / 1e9)},
            "us_per_layer": us_layer,
            "cold_start": {"tokens": warm, "ms_per_token": ms_warm / warm, "miss_ratio": st_warm["misses"] / max(1, st_warm["hits"] + st_warm["misses"])},
            "cache": {"requests": reqs, "hits": st["hits"], "misses": st["misses"], "evictions": st["evictions"],
                      "miss_ratio": st["misses"] / max(1, reqs), "h2d_bytes": miss_bytes, "h2d_copies_per_layer": st["h2d_copies"] / (args.steps * n_layers),
                      "miss_bytes_per_layer": miss_bytes / (args.steps * n_layers),
                      "lru_miss_ratio_same_trace": lru, "miss_ratio_in_that_window": ours_window,
                      "window": f"{win} tokens after the timed region, every {max(1, n_layers // 8)}th layer for the LRU replay",
                      "loading_redundancy": (redund[0] / redund[1]) if redund[1] else None,
                      "loading_redundancy_note": "first 4 tokens of that window, every layer boundary: rows the refinements prefetched that the "
                                                 "final set does not use / rows the final set lacked before them (snapshots of the next "
                                                 "layer's resident set around each step)"},
            "roofline": {"bound": "host link", "achieved": miss_bytes / t_s / 1e9, "peak": link, "unit": "GB/s", "frac": miss_bytes / t_s / 1e9 / link,
                         "peak_kind": "measured here: one 256 MiB pinned host-to-device copy, best of five", "traffic": None,
                         "hbm": {"selected_row_bytes_gbs": sel_bytes / t_s / 1e9, "peak": peaks["hbm_gbs"], "frac": sel_bytes / t_s / 1e9 / peaks["hbm_gbs"], "peak_kind": peak_kind},
                         "time_if_link_bound_ms_per_token": miss_bytes / args.steps / (link * 1e9) * 1e3},
            "cpu_baseline": cpu,
            "e2e": {"value": steps_total / (ms_total * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": int(miss_bytes / args.steps), "d2h_bytes_per_step": 0,
                    "note": "the weights of this workload live in pinned host memory: every miss is a host-to-device copy inside the timed region"},
            "gpu_launches": int(launches_per_token * args.steps), "launches_per_token": launches_per_token,
            "parity_sample": parity, "clocks": clocks, "build_s": t_build,
        }
        print(json.dumps(line))
    for L in distinct:
        L.close()


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2609_03079_b200 import binding as ls
    from paper_2609_03079_b200 import replicas
    from paper_2609_03079_b200 import workload as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    spec = wl.SPECS[args.workload]
    if spec.cache_frac > 0:
        run_cached(args, ls, wl, replicas, torch, dist, world, rank, local, dev, spec)
    else:
        run_resident(args, ls, wl, replicas, torch, dist, world, rank, local, dev, spec)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
