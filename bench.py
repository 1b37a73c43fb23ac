#!/usr/bin/env python
"""Benchmark of the speculate-and-refine sparse FFN decode path.

One *step* is one decode token through the whole synthetic FFN stack: for every layer the predictor scores of
the next layer are refined after each of the K stages, the selected gate/up rows are streamed, and the sparse down
projection accumulates the surviving rows.  ``value`` is tokens/s with the token inputs already resident in HBM;
``e2e`` is the same loop with a pinned-host input copied in and the result copied out every step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload llama2-7b] [--chunks 8]

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the stack on its own
token stream ("replicas only": the batch-1 path has no exchange step); the line reports the sum over ranks divided
by the slowest rank's time.
"""
from __future__ import annotations

import argparse
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--chunks", type=int, default=8, help="K: stages per layer (Section 4.3.1 of the paper uses 8)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (debugging only)")
    ap.add_argument("--no-graph", action="store_true", help="launch every call from the host instead of one CUDA graph per token")
    ap.add_argument("--per-layer", action="store_true", help="one fused kernel per layer (ls_sparse_ffn_step) instead of the whole-token kernel")
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


def oracle_layer_step_seconds(arrays, spec, K, n_steps, warmup=0):
    """Times the oracle's sparse step (predict, K stages with refinement, down projection) as it stands."""
    from oracle import leanstream_oracle as orc
    from paper_2609_03079_b200 import workload as wl

    layers = [orc.OracleLayer.from_arrays(a) for a in arrays]
    toks = wl.make_tokens(spec, max(1, (n_steps + warmup + len(layers) - 1) // len(layers) + 1))
    times = []
    it = 0
    t_idx = 0
    while it < n_steps + warmup:
        x = toks[t_idx % len(toks)].astype(np.float64)
        t_idx += 1
        order, _ = orc.select_batch(layers[0], x[None], spec.k)
        for n, L in enumerate(layers):
            if it >= n_steps + warmup:
                break
            nxt = layers[(n + 1) % len(layers)]
            t0 = time.perf_counter()
            res = orc.sparse_ffn_step(L, nxt, x, order, K, spec.k)
            dt = time.perf_counter() - t0
            if it >= warmup:
                times.append(dt)
            it += 1
            x = res["xtilde"][K][0]
            order = res["refine_orders"][K]
    return times


def run_reference(args):
    """Reference arm: the CPU oracle on this machine's host cores, same metric and workload, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch

    from paper_2609_03079_b200 import workload as wl

    spec = wl.SPECS[args.workload]
    n_layers = args.layers or spec.n_layers
    svd_dev = "cuda" if torch.cuda.is_available() else "cpu"
    arrays = [wl.make_layer(spec, l, svd_device=svd_dev) for l in range(min(args.cpu_sample_layers, n_layers))]
    steps = max(1, args.steps)
    t0 = time.perf_counter()
    times = oracle_layer_step_seconds(arrays, spec, args.chunks, steps, args.warmup)
    wall = time.perf_counter() - t0
    t_layer = float(np.mean(times))
    value = 1.0 / (t_layer * n_layers)
    sample = (f"{len(times)} layer-steps (K={args.chunks}, k={spec.k}) on {len(arrays)} distinct layers of the {spec.name} stack; "
              f"tokens/s = 1 / (mean layer-step time x {n_layers} layers)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": steps,
        "warmup": args.warmup, "ms_per_step": t_layer * n_layers * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec.name, "n_layers": n_layers, "d_model": spec.d_model, "d_ff": spec.d_ff, "k": spec.k,
                   "chunks": args.chunks, "batch": 1},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": wall,
    }
    print(json.dumps(line))


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
    n_layers = args.layers or spec.n_layers
    K, k, d = args.chunks, spec.k, spec.d_model

    # ---- build the stack (seeded, synthetic); host arrays are dropped once uploaded
    t_build = time.perf_counter()
    from concurrent.futures import ThreadPoolExecutor

    keep_host = {}
    layers = [None] * n_layers

    def make(l):
        la = wl.make_layer(spec, l, svd_device=f"cuda:{local}")
        return l, la

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        for l, la in ex.map(make, range(n_layers)):
            layers[l] = ls.ls_layer_create(la, local)
            if rank == 0 and l < args.cpu_sample_layers:
                keep_host[l] = la
    t_build = time.perf_counter() - t_build

    n_tok = max(spec.n_tokens, 1)
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

    # ---- warm-up, launch count per token, optional CUDA graph of one token
    x_buf.copy_(X0[0:1])
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
        n_gu, ms_gu = ls.ls_timing_read(ls.LS_TIMED_GATEUP)
        n_dn, ms_dn = ls.ls_timing_read(ls.LS_TIMED_DOWN)
        n_pr, ms_pr = ls.ls_timing_read(ls.LS_TIMED_PREDICT)
        # surviving rows (down-projection bytes) measured on one traced token
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
        # Algorithmic bytes of a layer step.  The fused kernel reads the first row of every selected bundle and the rest of
        # the bundle only for the neurons that survive the ReLU (exact: a zero activation makes the up row irrelevant), so
        # its figure is k rows + n_in surviving rows + surviving down rows; the staged path reads all n_in rows of every
        # selected neuron.  The smaller figure is the one reported when the fused kernel runs.
        fused_bytes_layer = k * row + k_surv * spec.n_in * row
        staged_bytes_layer = k * spec.n_in * row + k_surv * row
        active_bytes_layer = fused_bytes_layer if (n_st or n_fz) else staged_bytes_layer
        ms_step = ms_total / args.steps
        us_layer = ms_step * 1e3 / n_layers
        active_gbs = active_bytes_layer / (us_layer * 1e-6) / 1e9
        traffic_db = {}
        tp = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(tp):
            with open(tp) as f:
                traffic_db = json.load(f)
        if n_st:
            # one launch = one token = n_layers layer steps: algorithmic bytes are the active-neuron bytes of all layers
            kname, bytes_launch, us_launch, n_timed = "ls_fused_stack_kernel", active_bytes_layer * n_layers, ms_st / n_st * 1e3, n_st
            per_layer_traffic = traffic_db.get("stack_dram_bytes_per_layer")
            traffic = per_layer_traffic * n_layers if per_layer_traffic else None
        elif n_fz:
            # the whole layer step is one kernel: its algorithmic bytes are the active-neuron bytes of the layer
            kname, bytes_launch, us_launch, n_timed = "ls_fused_step_kernel", active_bytes_layer, ms_fz / n_fz * 1e3, n_fz
            traffic = traffic_db.get("fused_dram_bytes_per_launch")
        else:
            kname, bytes_launch, n_timed = "ls_gateup_kernel", (k / K) * spec.n_in * row, n_gu
            us_launch = ms_gu / max(n_gu, 1) * 1e3
            traffic = traffic_db.get("gateup_dram_bytes_per_launch")
        k_gbs = bytes_launch / (us_launch * 1e-6) / 1e9 if n_timed else None

        # ---- CPU baseline: the oracle as it stands on a bounded sample
        t0 = time.perf_counter()
        arrays = [keep_host[l] for l in sorted(keep_host)]
        n_cpu = 48 * len(arrays)  # fifteen to twenty seconds of CPU work at the Llama-2-7B shape
        times = oracle_layer_step_seconds(arrays, spec, K, n_cpu, warmup=0)
        cpu_wall = time.perf_counter() - t0
        cpu_val = 1.0 / (float(np.mean(times)) * n_layers)

        line = {
            "metric": METRIC, "value": steps_total / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights, f32 accumulate, f64 predictor scores", "data": "synthetic",
            "config": {"workload": spec.name, "n_layers": n_layers, "d_model": d, "d_ff": spec.d_ff, "pred_rank": spec.rank, "k": k,
                       "chunks": K, "batch": 1, "parallelism": "replicas only" if world > 1 else "1 gpu",
                       "l2": "inputs larger than L2 (%.2f GB of weight rows touched per token)" % (active_bytes_layer * n_layers / 1e9),
                       "cuda_graph": graph is not None, "kernel_per": "layer" if stack is None else "token"},
            "us_per_layer": us_layer, "active_bytes_per_layer": active_bytes_layer,
            "active_bytes_per_layer_if_up_rows_of_all_selected": staged_bytes_layer, "k_surviving_mean": k_surv,
            "active_gbs": active_gbs, "active_frac_of_hbm_peak": active_gbs / peaks["hbm_gbs"],
            "roofline": {"bound": "hbm", "kernel": kname, "achieved": k_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": (k_gbs / peaks["hbm_gbs"]) if k_gbs else None, "traffic": traffic, "peak_kind": peak_kind,
                         "bytes_per_launch": bytes_launch, "us_per_launch": us_launch, "launches_timed": n_timed,
                         "staged_path": {"gateup_us": ms_gu / max(n_gu, 1) * 1e3, "down_us": ms_dn / max(n_dn, 1) * 1e3,
                                         "predict_us": ms_pr / max(n_pr, 1) * 1e3} if n_gu else None},
            "cpu_baseline": {"value": cpu_val, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                             "sample": f"{len(times)} layer-steps on {len(arrays)} distinct layers, scaled to {n_layers} layers; {cpu_wall:.1f} s"},
            "e2e": {"value": steps_e2e / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": d * 4, "d2h_bytes_per_step": d * 4},
            "gpu_launches": launches_per_token * args.steps, "launches_per_token": launches_per_token,
            "clocks": clocks, "build_s": t_build,
        }
        print(json.dumps(line))
    if stack is not None:
        stack.close()
    for L in layers:
        L.close()
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
