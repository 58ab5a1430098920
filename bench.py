#!/usr/bin/env python
"""Benchmark of the verification hot path: verify-attention + retrieval, microseconds per layer.

One step = one verification pass of a 32-layer Llama-3.1-8B-shaped target over a 16K-token prefix
and a 60-node draft tree (independent K/V per layer, 2.1 GB per step, so every layer comes from
HBM), the last layer also producing chunk scores, followed by SelectChunks and UpdateDraftCache.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-graph]

Prints ONE JSON line on rank 0.  With N > 1 (launched by torch.distributed.run) every rank runs an
independent replica of the step on its own GPU; no collective is on the data path.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verify-attn+retrieval us/layer at 16K prefix, 60-node tree"
UNIT = "us/layer"
WORKLOAD = "c2"
WORKLOAD_DESC = ("c2: Llama-3.1-8B layer shape (32 q heads / 8 kv heads / dim 128, bf16), prefix 16384, "
                 "60-node level tree, 32 layers with independent K/V, scores from layer 31, chunk 32, top-k 32, "
                 "draft KV 8x128 gather of 1024 tokens")
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel (attn_tc2_kernel), from the
# ncu capture summarised in profiles/attn_tc2_kernel_c2_16k.md (67.93 MB read + 2.03 MB written).
NCU_TRAFFIC_BYTES_PER_LAUNCH = 69959424


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "tf_burst": float(p["bf16_tflops"]),
                "tf_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


def tree_depths(parent):
    d = []
    for i, p in enumerate(parent):
        d.append(0 if p < 0 else d[p] + 1)
    return d


def layer_work(w, parent, last_layer):
    L, T, Hq, Hkv, D, C = w.prefix_len, w.n_tree, w.n_q_heads, w.n_kv_heads, w.head_dim, w.chunk_size
    nbytes = 2 * L * Hkv * D * 2 + 2 * T * Hkv * D * 2 + 2 * T * Hq * D * 2 + Hq * T * 4
    if last_layer:
        nbytes += T * (-(-L // C)) * 4
    visible_tree = sum(d + 1 for d in tree_depths(parent))
    flops = 4 * Hq * D * (T * L + visible_tree)
    return nbytes, flops


class ClockSampler:
    """Polls SM clock and throttle reasons of one GPU through NVML while the timed regions run."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.index, self.period = index, period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:                                   # NVML unavailable: no clock record
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake": 0x80, "sync_boost": 0x10,
                 "applications_clocks_setting": 0x2, "display_clocks_setting": 0x100}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def oracle_sample(w, parent, repeats):
    """Times the CPU oracle on one 16K layer (attention with scores) plus select + gather."""
    import numpy as np
    import torch
    from workloads import synth
    from oracle import specext_oracle as orc
    t = synth.make_layer(w, layer=w.n_layers - 1)
    dK, dV = synth.make_draft_kv(w)
    f = lambda x: x.double().numpy()
    args = (f(t["Q"]), f(t["K_prefix"]), f(t["V_prefix"]), f(t["K_tree"]), f(t["V_tree"]))
    dKb, dVb = dK.view(torch.int16).numpy(), dV.view(torch.int16).numpy()
    t_attn, t_retr = [], []
    for _ in range(repeats):
        t0 = time.perf_counter()
        _, _, cs = orc.verify_attn(*args, parent, w.chunk_size)
        t1 = time.perf_counter()
        idx = orc.select_chunks(cs[37], w.prefix_len, w.chunk_size, w.top_k)
        orc.gather_kv(dKb, dVb, idx, w.prefix_len, w.chunk_size)
        t2 = time.perf_counter()
        t_attn.append(t1 - t0)
        t_retr.append(t2 - t1)
    return t_attn, t_retr


def replica_seed(base_seed: int, rank: int) -> int:
    """Every replica (rank) verifies its own sequence."""
    return base_seed + 1000 * rank


def max_over_ranks(ms_total: float, world: int, device) -> float:
    """The slowest rank's device time (all ranks get it); one process = its own time."""
    if world <= 1:
        return ms_total
    import torch
    import torch.distributed as dist
    tt = torch.tensor([ms_total], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def us_per_layer(ms_total: float, steps: int, n_layers: int, world: int) -> float:
    """Whole-job figure: every rank runs `steps` steps of `n_layers` layers in `ms_total`."""
    return ms_total / steps * 1e3 / (n_layers * world)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, rank):
    """The reference arm: the oracle as it stands, on the host cores, bounded sample per step."""
    if rank != 0:
        return
    from workloads import synth
    w = synth.WORKLOADS[WORKLOAD]
    parent = synth.make_tree(w)
    oracle_sample(w, parent, max(0, min(args.warmup, 1)))
    steps = max(1, min(args.steps, 8))
    ta, tr = oracle_sample(w, parent, steps)
    per_layer_us = (sum(ta) / steps + sum(tr) / steps / w.n_layers) * 1e6
    sample = (f"per step: oracle verify_attn on 1 of the 32 layers (16K prefix, all 32 heads x 60 nodes, with "
              f"chunk scores) + select + gather; us/layer = t_attn + t_retrieval/32; {steps} steps timed")
    line = {"impl": "reference", "metric": METRIC, "value": per_layer_us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": per_layer_us * w.n_layers / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD_DESC},
            "cpu_baseline": {"value": per_layer_us, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": per_layer_us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: run only this many layers per step (the JSON line says so; not a bench value)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2505_20776_b200 import api, build
    from workloads import synth
    from paper_2505_20776_b200.hotpath import HotPath

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    build.build()
    api.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = synth.WORKLOADS[WORKLOAD]
    if args.layers > 0:
        import dataclasses
        w = dataclasses.replace(w, n_layers=max(2, args.layers))
    NL, L = w.n_layers, w.prefix_len
    parent_np = synth.make_tree(w)
    parent = torch.from_numpy(parent_np).to(dev)
    seed = replica_seed(w.seed, rank)
    layers = [synth.make_layer(w, layer=i, device=dev, seed=seed) for i in range(NL)]
    dK, dV = synth.make_draft_kv(w, device=dev, seed=seed)
    hp = HotPath(w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_tree, w.chunk_size, w.top_k, L, device=dev)
    row = 37

    def step():
        for i in range(NL):
            hp.verify_attn(layers[i], parent, L, i == NL - 1)
        hp.select_chunks(row, L)
        hp.gather_kv(dK, dV, L)

    stream = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        n0 = api.specext_launch_count()
        step()
        launches_per_step = api.specext_launch_count() - n0
        stream.synchronize()
        graph = None
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step()
        run = graph.replay if graph is not None else step

        for _ in range(args.warmup):
            run()
        stream.synchronize()
        assert hp.read_status() == 0, "device status set during warm-up"

        sampler = ClockSampler(local_rank)
        sampler.start()

        def barrier():
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
                torch.cuda.synchronize()

        # ---- timed region: K steps, device timed ------------------------------------------
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            run()
        e1.record(stream)
        barrier()
        ms_total = e0.elapsed_time(e1)

        # ---- roofline pass: only the score-less verification-attention calls (the dominant
        # launch: attention kernel + merge), 31 distinct layers per replay so K/V comes from HBM
        def attn_only():
            for i in range(NL - 1):
                hp.verify_attn(layers[i], parent, L, False)

        attn_only()
        stream.synchronize()
        run_attn = attn_only
        if not args.no_graph:
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2, stream=stream):
                attn_only()
            run_attn = g2.replay
        rsteps = max(3, min(args.steps, 50))
        run_attn()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(rsteps):
            run_attn()
        b.record(stream)
        barrier()
        attn_us_mean = a.elapsed_time(b) * 1e3 / (rsteps * (NL - 1))

        # ---- the other parts, each timed alone the same way (reported, not part of `value`) --
        def timed_us(fn, calls):
            fn()
            stream.synchronize()
            runner = fn
            if not args.no_graph:
                gg = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gg, stream=stream):
                    fn()
                runner = gg.replay
            runner()
            barrier()
            x, y = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            x.record(stream)
            for _ in range(rsteps):
                runner()
            y.record(stream)
            barrier()
            return x.elapsed_time(y) * 1e3 / (rsteps * calls)

        n_sc = min(NL, 8)                                # 8 distinct layers = 0.5 GB of K/V: from HBM

        def score_layers():
            for i in range(n_sc):
                hp.verify_attn(layers[i], parent, L, True)

        def retrieval():
            hp.select_chunks(row, L)
            hp.gather_kv(dK, dV, L)

        parts = {"scoreless_layer_us": attn_us_mean, "score_layer_us": timed_us(score_layers, n_sc),
                 "select_gather_us": timed_us(retrieval, 1),
                 "note": "each part replayed alone; select+gather re-reads the same 8 MB (L2-resident)"}
        hp.verify_attn(layers[NL - 1], parent, L, True)  # leave the scores of the last layer in place

        # ---- end to end: host buffers, copies inside the timed region ----------------------
        e2e = None
        if args.e2e_steps > 0:
            host_layers = [{k: v.cpu().pin_memory() for k, v in t.items()} for t in layers]
            host_dK, host_dV = dK.cpu().pin_memory(), dV.cpu().pin_memory()
            host_parent = torch.from_numpy(parent_np).pin_memory()
            h_idx = torch.empty(w.top_k, dtype=torch.int32).pin_memory()
            h_K = torch.empty_like(hp.K_compact, device="cpu").pin_memory()
            h_V = torch.empty_like(hp.V_compact, device="cpu").pin_memory()
            h_O = torch.empty_like(hp.O, device="cpu").pin_memory()
            h2d = (sum(v.numel() * v.element_size() for t in host_layers for v in t.values()) +
                   2 * host_dK.numel() * 2 + host_parent.numel() * 4)
            d2h = h_idx.numel() * 4 + 2 * h_K.numel() * 2 + h_O.numel() * 2

            def e2e_step():
                parent.copy_(host_parent, non_blocking=True)
                for i in range(NL):
                    for k in layers[i]:
                        layers[i][k].copy_(host_layers[i][k], non_blocking=True)
                    hp.verify_attn(layers[i], parent, L, i == NL - 1)
                dK.copy_(host_dK, non_blocking=True)
                dV.copy_(host_dV, non_blocking=True)
                hp.select_chunks(row, L)
                hp.gather_kv(dK, dV, L)
                h_O.copy_(hp.O, non_blocking=True)
                h_idx.copy_(hp.idx, non_blocking=True)
                h_K.copy_(hp.K_compact, non_blocking=True)
                h_V.copy_(hp.V_compact, non_blocking=True)

            e2e_step()
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(args.e2e_steps):
                e2e_step()
            b.record(stream)
            barrier()
            e2e_ms = a.elapsed_time(b) / args.e2e_steps
            if world > 1:
                tt = torch.tensor([e2e_ms], device=dev)
                dist.all_reduce(tt, op=dist.ReduceOp.MAX)
                e2e_ms = float(tt.item())
            e2e = {"value": e2e_ms * 1e3 / (NL * world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}
        clocks = sampler.stop()
        assert hp.read_status() == 0, "device status set during the timed region"

    ms_total = max_over_ranks(ms_total, world, dev)
    ms_per_step = ms_total / args.steps
    value = us_per_layer(ms_total, args.steps, NL, world)

    if rank == 0:
        peaks = load_peaks()
        nbytes, flops = layer_work(w, parent_np.tolist(), False)
        t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6
        t_tc = flops / (peaks["tf_sustained"] * 1e12) * 1e6
        t_roof = max(t_hbm, t_tc)
        if t_hbm >= t_tc:
            roof = {"bound": "hbm", "achieved": nbytes / (attn_us_mean * 1e-6) / 1e9, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": flops / (attn_us_mean * 1e-6) / 1e12,
                    "peak": peaks["tf_sustained"], "unit": "TFLOP/s"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["traffic"] = NCU_TRAFFIC_BYTES_PER_LAUNCH
        roof.update({"peak_source": peaks["source"] + (" (sustained bf16: kernel timed inside a long step)"
                                                       if roof["bound"] == "tensor" else ""),
                     "kernel": "verify-attention call of a score-less layer (attention + merge launches)",
                     "launch_us_mean": attn_us_mean,
                     "algorithmic_bytes": nbytes, "algorithmic_flops": flops,
                     "achieved_gbs": nbytes / (attn_us_mean * 1e-6) / 1e9,
                     "achieved_tflops": flops / (attn_us_mean * 1e-6) / 1e12,
                     "t_hbm_us": t_hbm, "t_tensor_us": t_tc,
                     "t_tensor_burst_us": flops / (peaks["tf_burst"] * 1e12) * 1e6,
                     "t_roof_us": t_roof, "frac_of_roofline_time": t_roof / attn_us_mean})
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD_DESC, "l2": "inputs larger than L2 (2.1 GB of K/V read per step)",
                           "cuda_graph": graph is not None, "replicas": world,
                           **({"profiling_layers": NL} if args.layers > 0 else {})},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "roofline": roof, "parts": parts}
        if world == 1 and not args.no_cpu_baseline:
            ta, tr = oracle_sample(w, parent_np, 3)
            cpu_us = (sum(ta) / len(ta) + sum(tr) / len(tr) / NL) * 1e6
            line["cpu_baseline"] = {"value": cpu_us, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                    "sample": "oracle verify_attn on layer 31 of the workload (16K prefix, 32 heads "
                                              "x 60 nodes, with chunk scores) + select + gather, 3 repeats; "
                                              "us/layer = t_attn + t_retrieval/32"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
