#!/usr/bin/env python
"""Benchmark of the verification hot path: verify-attention + retrieval, microseconds per layer.

One step = one verification pass of a 32-layer Llama-3.1-8B-shaped target over a 16K-token prefix
and a 60-node draft tree (independent K/V per layer, 2.1 GB per step, so every layer comes from
HBM), the last layer also producing chunk scores, followed by SelectChunks + UpdateDraftCache.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload all|c1|c2|c3|c4] [--no-graph]

Prints ONE JSON line on rank 0.  The headline (`value`) is always workload c2; `--workload` chooses
which of the other configurations are timed as well (key `workloads`: one verification-attention call
and one scored call + retrieval per configuration, each replayed over enough distinct K/V buffers to
stay out of L2).  With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica of the step on its own GPU; no collective is on the data path.  `--impl reference` times the
CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
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
# ncu capture summarised in profiles/attn_tc2_kernel_c2_16k.md.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 69613056            # 67,914,496 read + 1,698,560 written
NOMINAL = {"hbm_gbs": 7700.0, "tf": 2250.0}            # B200 data-sheet figures, for context only


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


def layer_work(w, parent, last_layer, prefix_len=None):
    """Algorithmic bytes and flops of one verification-attention call (padding and split partials excluded)."""
    L = w.prefix_len if prefix_len is None else prefix_len
    T, Hq, Hkv, D, C = w.n_tree, w.n_q_heads, w.n_kv_heads, w.head_dim, w.chunk_size
    nbytes = 2 * L * Hkv * D * 2 + 2 * T * Hkv * D * 2 + 2 * T * Hq * D * 2 + Hq * T * 4
    if last_layer:
        nbytes += T * (-(-L // C)) * 4
    visible_tree = sum(d + 1 for d in tree_depths(parent))
    flops = 4 * Hq * D * (T * L + visible_tree)
    return nbytes, flops


def retrieval_bytes(w, prefix_len=None):
    """One score row read, the indices written, and the kept chunks of draft K and V read and written."""
    L = w.prefix_len if prefix_len is None else prefix_len
    nc = -(-L // w.chunk_size)
    keff = min(w.top_k, nc)
    h, d = w.draft_kv_heads or w.n_kv_heads, w.draft_head_dim or w.head_dim
    return nc * 4 + keff * 4 + 4 * min(keff * w.chunk_size, L) * h * d * 2


def tensor_peak(peaks, clocks):
    """The bf16 peak that matches the run's own clock record: the burst figure when the sampled SM clock
    stayed at its maximum, the sustained one (measured under the power cap at a lower clock) otherwise."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    if mhz and mx and mhz >= 0.97 * mx:
        return peaks["tf_burst"], "burst (median SM clock at maximum during the timed region)"
    return peaks["tf_sustained"], "sustained (SM clock below maximum, or no clock record)"


def roof_times(nbytes, flops, peaks, tf):
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6
    t_tc = flops / (tf * 1e12) * 1e6
    return t_hbm, t_tc


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
                "sm_mhz_min": s[0] if s else None,
                "below_max_frac": (sum(1 for x in s if self.max_mhz and x < 0.97 * self.max_mhz) / len(s)) if s else None,
                "reasons": sorted(self.reasons), "samples": len(s)}


def oracle_sample(w, parent, repeats):
    """Times the CPU oracle on one 16K layer (attention with scores) plus select + gather."""
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
    """The reference arm: the oracle as it stands, on the host cores.  One step of this arm is a bounded
    sample of the workload's step: ONE of the 32 layers (with chunk scores) plus select + gather; that is
    what `ms_per_step` times.  `value` spreads the retrieval over the 32 layers as the GPU arm does."""
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
            "steps": steps, "warmup": min(args.warmup, 1),
            "ms_per_step": (sum(ta) + sum(tr)) / steps * 1e3, "sample_layers_per_step": 1,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD_DESC},
            "cpu_baseline": {"value": per_layer_us, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": per_layer_us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# Distinct K/V buffers a single-layer configuration rotates over so that no buffer is still in the
# 126 MB L2 when its turn comes again (at least ~256 MB of other K/V in between).
def copies_for(kv_bytes: int) -> int:
    return max(4, -(-(384 << 20) // max(kv_bytes, 1)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all", "c1", "c2", "c3", "c4", "long"],
                    help="which configurations are timed besides the c2 headline (c2 = headline only; long = the c3 "
                         "shape at 64K and 128K keys, beyond the paper's configurations)")
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
        hp.select_gather(row, L, dK, dV)

    stream = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def make_runner(fn):
        """fn once eagerly (sizes the workspace), then captured in a graph unless --no-graph."""
        fn()
        stream.synchronize()
        if args.no_graph:
            return fn
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
        return g.replay

    def timed(runner, reps, warm=2, per_replay=False):
        """Device time in ms of `reps` back-to-back replays between two events (a barrier and a device
        synchronisation on both sides).  With per_replay an event is recorded between consecutive replays
        as well and the list of per-replay times is returned too; those events cost a little themselves."""
        for _ in range(warm):
            runner()
        barrier()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1 if per_replay else 2)]
        ev[0].record(stream)
        for i in range(reps):
            runner()
            if per_replay:
                ev[i + 1].record(stream)
        if not per_replay:
            ev[1].record(stream)
        barrier()
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(reps)] if per_replay else None
        return per, ev[0].elapsed_time(ev[-1])

    with torch.cuda.stream(stream):
        n0 = api.specext_launch_count()
        step()
        launches_per_step = api.specext_launch_count() - n0
        stream.synchronize()
        run = make_runner(step)
        for _ in range(args.warmup):
            run()
        stream.synchronize()
        assert hp.read_status() == 0, "device status set during warm-up"

        sampler = ClockSampler(local_rank)
        sampler.start()

        # ---- timed region: K steps, device timed ------------------------------------------
        _, ms_total = timed(run, args.steps, warm=0)
        # the same steps once more with an event after every replay, for the spread (median, minimum)
        per_step_ms, _ = timed(run, args.steps, warm=0, per_replay=True)

        # ---- the parts, each replayed alone the same way (reported, not part of `value`) ------
        rsteps = max(3, min(args.steps, 50))

        def part_us(fn, calls):
            _, total = timed(make_runner(fn), rsteps)
            return total / rsteps * 1e3 / calls

        def attn_only():                                 # 31 distinct layers per replay: K/V comes from HBM
            for i in range(NL - 1):
                hp.verify_attn(layers[i], parent, L, False)

        n_sc = min(NL, 8)                                # 8 distinct layers = 0.5 GB of K/V: from HBM

        def score_layers():
            for i in range(n_sc):
                hp.verify_attn(layers[i], parent, L, True)

        n_rt = 16                                        # per graph, so that graph launches do not set the pace

        def retrieval_one_call():
            for _ in range(n_rt):
                hp.select_gather(row, L, dK, dV)

        def retrieval_two_calls():
            for _ in range(n_rt):
                hp.select_chunks(row, L)
                hp.gather_kv(dK, dV, L)

        # draft-side attention on the compact cache the retrieval just wrote (a 10-node draft step of an
        # EAGLE-class layer: 32 query heads on the cache's 8 KV heads), its length read on the device
        wdr = synth.Workload("draft", w.n_q_heads, dK.shape[2], dK.shape[3], w.top_k * w.chunk_size, 10, w.chunk_size,
                             1, "uniform", "normal", seed=seed + 7)
        tdr = synth.make_layer(wdr, device=dev)
        pdr_np = synth.make_tree(wdr)
        pdr = torch.from_numpy(pdr_np).to(dev)
        O_dr = torch.empty_like(tdr["Q"])
        lse_dr = torch.empty(wdr.n_q_heads, wdr.n_tree, dtype=torch.float32, device=dev)
        d_dr = api.make_attn_desc(tdr["Q"], hp.K_compact[0], tdr["K_tree"], O_dr, wdr.prefix_len, w.chunk_size)
        ws_dr = torch.empty(api.specext_verify_attn_workspace(d_dr), dtype=torch.uint8, device=dev)

        def draft_attn():
            for _ in range(n_rt):
                api.specext_draft_attn(d_dr, tdr["Q"], hp.K_compact[0], hp.V_compact[0], hp.n_tokens, tdr["K_tree"],
                                       tdr["V_tree"], pdr, O_dr, lse_dr, ws_dr, hp.status)

        def retrieval_then_draft():
            for _ in range(n_rt):
                hp.select_gather(row, L, dK, dV)
                api.specext_draft_attn(d_dr, tdr["Q"], hp.K_compact[0], hp.V_compact[0], hp.n_tokens, tdr["K_tree"],
                                       tdr["V_tree"], pdr, O_dr, lse_dr, ws_dr, hp.status)

        # prefill of a 16K-token prompt of the same layer shape (causal attention; K/V of layer 0, seeded Q)
        wq = synth.Workload("prefill-q", w.n_q_heads, w.n_q_heads, w.head_dim, L, 1, w.chunk_size, 1, "chain", "needle",
                            seed=seed + 9)
        Q_pf = synth.make_layer(wq, device=dev)["K_prefix"]
        O_pf = torch.empty_like(Q_pf)
        lse_pf = torch.empty(w.n_q_heads, L, dtype=torch.float32, device=dev)

        def prefill():
            api.specext_prefill_attn(Q_pf, layers[0]["K_prefix"], layers[0]["V_prefix"], O_pf, lse_pf, hp.status)

        attn_us = part_us(attn_only, NL - 1)
        parts = {"scoreless_layer_us": attn_us, "score_layer_us": part_us(score_layers, n_sc),
                 "select_gather_us": part_us(retrieval_one_call, n_rt),
                 "select_then_gather_two_calls_us": part_us(retrieval_two_calls, n_rt),
                 "prefill_16k_us": part_us(prefill, 1),
                 "prefill_16k_flops": 4 * w.n_q_heads * w.head_dim * (L * (L + 1) // 2),
                 "draft_attn_us": part_us(draft_attn, n_rt),
                 "select_gather_then_draft_attn_us": part_us(retrieval_then_draft, n_rt),
                 "draft_attn_algorithmic_bytes": layer_work(wdr, pdr_np.tolist(), False)[0],
                 "note": "mean over back-to-back replays of each part alone; the retrieval parts re-read the same 8 MB "
                         "(L2-resident)"}
        hp.verify_attn(layers[NL - 1], parent, L, True)  # leave the scores of the last layer in place

        # ---- the other configurations ------------------------------------------------------
        others = {}
        which = [] if args.workload == "c2" or args.layers > 0 else (
            ["c1", "c3", "c4"] if args.workload == "all" else [] if args.workload == "long" else [args.workload])
        for name in which:
            ww = synth.WORKLOADS[name]
            par_np = synth.make_tree(ww)
            par = torch.from_numpy(par_np).to(dev)
            cap = ww.capacity or ww.prefix_len
            lengths = synth.C3_LENGTHS if name == "c3" else (ww.prefix_len,)
            per_tok = 2 * ww.n_kv_heads * ww.head_dim * 2
            n_copies = copies_for(min(lengths) * per_tok)
            # copy i is only ever read up to the longest length that still rotates over more than i copies
            caps = [max(Lx for Lx in lengths if i < copies_for(Lx * per_tok)) for i in range(n_copies)]
            bufs = [synth.make_layer(ww, layer=i, device=dev, capacity=min(cap, caps[i])) for i in range(n_copies)]
            ddK, ddV = synth.make_draft_kv(ww, device=dev, capacity=cap)
            hpo = HotPath(ww.n_q_heads, ww.n_kv_heads, ww.head_dim, ww.n_tree, ww.chunk_size, ww.top_k, cap,
                          device=dev)
            for Lx in lengths:
                nb = min(n_copies, copies_for(Lx * per_tok))

                def calls():
                    for b in bufs[:nb]:
                        hpo.verify_attn(b, par, Lx, False)

                def scored_steps():                      # the in-place growth step: scored call + retrieval
                    for b in bufs[:nb]:
                        hpo.verify_attn(b, par, Lx, True)
                        hpo.select_gather(row, Lx, ddK, ddV)

                call_us = part_us(calls, nb)
                step_us = part_us(scored_steps, nb)
                nbytes, flops = layer_work(ww, par_np.tolist(), False, Lx)
                others[name if name != "c3" else f"c3@{Lx}"] = {
                    "prefix_len": Lx, "kv_copies_rotated": nb, "attn_call_us": call_us,
                    "scored_call_plus_retrieval_us": step_us, "algorithmic_bytes": nbytes,
                    "algorithmic_flops": flops}
            assert hpo.read_status() == 0
            del bufs, hpo, ddK, ddV
            torch.cuda.empty_cache()

        # ---- longer prefixes than the paper's configurations (same layer shape as c3) --------
        if args.layers == 0 and args.workload in ("all", "long"):
            ww = synth.WORKLOADS["c3"]
            par_np = synth.make_tree(ww)
            par = torch.from_numpy(par_np).to(dev)
            for Lx in (65536, 131072):
                bufs = [synth.make_layer(ww, layer=i, device=dev, capacity=Lx) for i in range(2)]   # 2 x 268 / 537 MB
                hpo = HotPath(ww.n_q_heads, ww.n_kv_heads, ww.head_dim, ww.n_tree, ww.chunk_size, ww.top_k, Lx,
                              device=dev)

                def calls():
                    for b in bufs:
                        hpo.verify_attn(b, par, Lx, False)

                call_us = part_us(calls, len(bufs))
                nbytes, flops = layer_work(ww, par_np.tolist(), False, Lx)
                others[f"long@{Lx}"] = {"prefix_len": Lx, "kv_copies_rotated": len(bufs), "attn_call_us": call_us,
                                        "algorithmic_bytes": nbytes, "algorithmic_flops": flops}
                assert hpo.read_status() == 0
                del bufs, hpo
                torch.cuda.empty_cache()

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
                hp.select_gather(row, L, dK, dV)
                h_O.copy_(hp.O, non_blocking=True)
                h_idx.copy_(hp.idx, non_blocking=True)
                h_K.copy_(hp.K_compact, non_blocking=True)
                h_V.copy_(hp.V_compact, non_blocking=True)

            e2e_step()
            _, e2e_total = timed(e2e_step, args.e2e_steps, warm=0)
            e2e_ms = max_over_ranks(e2e_total / args.e2e_steps, world, dev)
            e2e = {"value": e2e_ms * 1e3 / (NL * world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}
        clocks = sampler.stop()
        assert hp.read_status() == 0, "device status set during the timed region"

    ms_total = max_over_ranks(ms_total, world, dev)
    ms_per_step = ms_total / args.steps
    value = us_per_layer(ms_total, args.steps, NL, world)

    if rank == 0:
        peaks = load_peaks()
        tf, tf_why = tensor_peak(peaks, clocks)
        # whole step, per layer: the score-less layers, the scored layer and the retrieval
        nb_plain, fl_plain = layer_work(w, parent_np.tolist(), False)
        nb_last, fl_last = layer_work(w, parent_np.tolist(), True)
        step_bytes = ((NL - 1) * nb_plain + nb_last + retrieval_bytes(w)) / NL
        step_flops = ((NL - 1) * fl_plain + fl_last) / NL
        t_hbm, t_tc = roof_times(step_bytes, step_flops, peaks, tf)
        t_roof = max(t_hbm, t_tc)
        if t_hbm >= t_tc:
            roof = {"bound": "hbm", "achieved": step_bytes / (value * 1e-6) / 1e9, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": step_flops / (value * 1e-6) / 1e12, "peak": tf, "unit": "TFLOP/s"}
        roof["frac"] = roof["achieved"] / roof["peak"]          # = t_roof / value
        roof["traffic"] = NCU_TRAFFIC_BYTES_PER_LAUNCH
        ta_hbm, ta_tc = roof_times(nb_plain, fl_plain, peaks, tf)
        roof.update({
            "what": "whole step per layer: algorithmic bytes (or flops) of 31 score-less layers, the scored layer "
                    "and select+gather, divided by 32 and by `value`; `traffic` is the attention kernel's DRAM "
                    "bytes per launch from the ncu capture",
            "peak_source": peaks["source"], "tensor_peak_used": tf_why,
            "algorithmic_bytes_per_layer": step_bytes, "algorithmic_flops_per_layer": step_flops,
            "t_hbm_us": t_hbm, "t_tensor_us": t_tc, "t_roof_us": t_roof,
            "frac_tensor_burst": (step_flops / (peaks["tf_burst"] * 1e12) * 1e6) / value,
            "frac_tensor_sustained": (step_flops / (peaks["tf_sustained"] * 1e12) * 1e6) / value,
            "frac_hbm": t_hbm / value,
            "frac_of_nominal": max(step_bytes / (NOMINAL["hbm_gbs"] * 1e9), step_flops / (NOMINAL["tf"] * 1e12))
                               * 1e6 / value,
            "attn_call": {"kernel": "verify-attention call of a score-less layer (attention + merge launches)",
                          "launch_us_mean": attn_us, "algorithmic_bytes": nb_plain, "algorithmic_flops": fl_plain,
                          "achieved_gbs": nb_plain / (attn_us * 1e-6) / 1e9,
                          "achieved_tflops": fl_plain / (attn_us * 1e-6) / 1e12,
                          "t_hbm_us": ta_hbm, "t_tensor_us": ta_tc, "frac": max(ta_hbm, ta_tc) / attn_us}})
        parts["prefill_16k_tflops"] = parts["prefill_16k_flops"] / (parts["prefill_16k_us"] * 1e-6) / 1e12
        parts["prefill_16k_frac_of_tensor_peak"] = parts["prefill_16k_tflops"] / tf
        parts["draft_attn_t_hbm_us"] = parts["draft_attn_algorithmic_bytes"] / (peaks["hbm_gbs"] * 1e9) * 1e6
        for o in others.values():
            th, tt = roof_times(o["algorithmic_bytes"], o["algorithmic_flops"], peaks, tf)
            o.update({"t_hbm_us": th, "t_tensor_us": tt, "frac": max(th, tt) / o["attn_call_us"]})
        per_layer = sorted(m * 1e3 / NL for m in per_step_ms)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD_DESC, "l2": "inputs larger than L2 (2.1 GB of K/V read per step)",
                           "cuda_graph": not args.no_graph, "replicas": world,
                           **({"profiling_layers": NL} if args.layers > 0 else {})},
                "per_replay": {"median": statistics.median(per_layer), "min": per_layer[0], "unit": UNIT,
                               "note": "separate pass of the same steps with an event after every replay"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "roofline": roof, "parts": parts, "workloads": others}
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
