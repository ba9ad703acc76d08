#!/usr/bin/env python
"""Benchmark of the Moment-KV decode hot path on B200.

A "step" is one call of mkv_decode_step for one attention layer over the whole batch:
append, GQA attention over prefill U decode pool, momentum score update, lowest-score
eviction, compaction -- all rows of the hot path.  The workload is the Llama-3.1-8B layer
shape at batch 16 (prefill lengths uniform in [512, 4096], decode budget 1024, beta 0.9)
at steady state, i.e. with the decode pool full so that every step evicts.  `--layers`
identical layers are cycled so that every layer-step streams a cache that is cold in L2
(as in a real 32-layer model).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mkv|reference]

prints one JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads.synthetic import CONFIGS, BatchStream  # noqa: E402

ROW_BYTES = 512  # K + V bytes of one cached token of one KV head (d=128 bf16)


# DRAM traffic of the hot kernel from its ncu capture (profiles/), as a ratio to the
# algorithmic bytes of the captured case; valid only for the kernel sources it was taken on.
TRAFFIC_CAPTURE = {"sources_sha1": "88090bc204f461ad5174750b8db4473649be547f", "traffic_over_algorithmic": 1.0260}
KERNEL_SOURCES = ["mkv_mma.cu", "mkv_tail.cuh", "mkv_layer_tail.cuh", "mkv_common.cuh", "mkv_ptx.cuh", "mkv_api.cu"]


def kernel_sources_sha1():
    import hashlib
    h = hashlib.sha1()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2605_29873_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def captured_traffic(alg_bytes):
    """Bytes per launch scaled from the capture (traffic grows with the rows streamed), or
    None once the kernel has changed since the counters were taken."""
    if TRAFFIC_CAPTURE["traffic_over_algorithmic"] and TRAFFIC_CAPTURE["sources_sha1"] == kernel_sources_sha1():
        return alg_bytes * TRAFFIC_CAPTURE["traffic_over_algorithmic"]
    return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def algorithmic_bytes_per_step(w, lens, n_dec, evict):
    """Bytes the method must move per layer-step: K,V of every cached token once per KV
    head, the appended row, score read+write, q in and out, the compaction move."""
    B, Hkv, Hq, d = w.batch, w.kv_heads, w.q_heads, w.head_dim
    es = 2 if w.dtype == "bf16" else 4
    kv = sum(Hkv * (int(lp) + n_dec) * 2 * d * es for lp in lens)
    append = B * Hkv * 2 * d * es
    score = B * Hkv * n_dec * 8
    qo = 2 * B * Hq * d * es
    compact = B * Hkv * evict * 2 * (2 * d * es + 8)
    return kv + append + score + qo + compact


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def time_oracle(w, lens, n_units, steps, warmup, time_cap_s, min_time_s=0.0):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload: the first
    `n_units` (sequence, KV head) units, each with its G query heads, from the start of
    generation (empty decode pool), one host thread per unit up to the core count.  Only the
    oracle calls are timed (input generation is not).  Returns tokens/s of the FULL batch at
    steady state, obtained by scaling the measured KV-row throughput by the rows one full
    steady-state step attends."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import mkv_oracle as O
    from workloads.synthetic import SequenceStream

    G = w.group
    cores = len(os.sched_getaffinity(0))
    threads = max(1, min(cores, n_units))
    seq_ids = sorted({u // w.kv_heads for u in range(n_units)})
    streams = {b: SequenceStream(w, 0, b) for b in seq_ids}
    pre = {b: streams[b].prefill() for b in seq_ids}
    units = []
    for u in range(n_units):
        b, g = divmod(u, w.kv_heads)
        o = O.OracleSequence(G, 1, w.head_dim, w.budget, w.beta, int(lens[b]))
        o.prefill(pre[b][0][g:g + 1], pre[b][1][g:g + 1])
        units.append((b, g, o))
    pool = ThreadPoolExecutor(threads)
    rows = 0
    elapsed = 0.0
    done = {"warm": 0, "timed": 0}
    t_idx = 0
    chunk = 128
    total = warmup + steps
    wall0 = time.perf_counter()
    while t_idx < total or elapsed < min_time_s:
        if t_idx >= total:
            total += chunk          # keep stepping until the sample holds min_time_s of oracle work
        nb = min(chunk, total - t_idx)
        data = {b: streams[b].next(nb) for b in seq_ids}
        for i in range(nb):
            timed = t_idx >= warmup
            t0 = time.perf_counter()
            list(pool.map(lambda it: it[2].step(data[it[0]][0][i, it[1] * G:(it[1] + 1) * G],
                                                data[it[0]][1][i, it[1]:it[1] + 1],
                                                data[it[0]][2][i, it[1]:it[1] + 1]), units))
            dt = time.perf_counter() - t0
            if timed:
                elapsed += dt
                n_i = min(t_idx + 1, w.budget + 1)
                rows += sum(int(lens[b]) + n_i for b, _, _ in units)
                done["timed"] += 1
            else:
                done["warm"] += 1
            t_idx += 1
            if time.perf_counter() - wall0 > time_cap_s and done["timed"] >= 3:
                t_idx = total
                min_time_s = 0.0
                break
            if t_idx >= warmup + steps and elapsed >= min_time_s:
                t_idx = total
                break
    pool.shutdown()
    full_rows = sum(w.kv_heads * (int(lp) + w.budget + 1) for lp in lens)
    tokens_per_s = (rows / elapsed) / full_rows * w.batch
    sample = (f"first {n_units} (sequence, KV head) units of the workload with their {G} query heads, "
              f"{done['timed']} decode steps after {done['warm']} warm-up steps from an empty decode pool; "
              f"{rows} KV rows attended in {elapsed:.2f} s on {threads} threads, scaled by the {full_rows} "
              f"rows a full steady-state step attends")
    return tokens_per_s, threads, sample, done


def run_reference(args, w):
    """The reference arm: the oracle on the host cores, sized to end within a few minutes."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    lens = w.prefill_lens()
    cores = len(os.sched_getaffinity(0))
    # one unit-step costs about (prefill + pool) * G * d * 4 flop at ~1 GFLOP/s
    est_unit_s = (float(np.mean(lens)) + w.budget / 2) * w.group * w.head_dim * 4 / 1.0e9
    per_step_s = 100.0 / max(1, args.steps + args.warmup)
    n_units = int(max(1, min(w.batch * w.kv_heads, cores * per_step_s / est_unit_s)))
    value, threads, sample, done = time_oracle(w, lens, n_units, args.steps, args.warmup, time_cap_s=150.0)
    line = {
        "impl": "reference", "metric": "decode tokens/sec per layer", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": done["timed"], "warmup": done["warm"], "ms_per_step": 1e3 * w.batch / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, lens, args),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, lens, args):
    shape = {"llama_b16": "Llama-3.1-8B attention layer shape", "llama_b1": "Llama-3.1-8B attention layer shape",
             "llama_stack": "Llama-3.1-8B attention layer shape", "qwen_b64": "Qwen2.5-7B-like attention layer shape",
             "tiny": "tiny single-layer shape"}.get(w.name, w.name)
    pre = (f"prefill lengths U[{w.prefill[0]},{w.prefill[1]}]" if not isinstance(w.prefill, int) else f"prefill {w.prefill}")
    return {"workload": f"{w.name}: {shape}, {w.q_heads}/{w.kv_heads} heads, "
                        f"head_dim {w.head_dim}, {w.dtype}, batch {w.batch}, {pre} "
                        f"(sum {int(np.sum(lens))}), decode budget {w.budget}, beta {w.beta}, steady state "
                        f"(decode pool full, one eviction per unit per step)",
            "layers_cycled": args.layers,
            "l2": "inputs larger than L2: each layer-step streams its own ~%d MB cache, %d layers cycled"
                  % (int(sum(w.kv_heads * (int(lp) + w.budget + 1) * 2 * w.head_dim * (2 if w.dtype == "bf16" else 4) for lp in lens) / 1e6), args.layers)}


def rank_workload(w, rank):
    """Weak scaling: every rank holds its own batch of the same shape (units are independent,
    so the data path needs no collective); ranks differ in their seed only."""
    return w.with_(seed=w.seed + rank)


def max_over_ranks(times_ms, world, device):
    """Element-wise maximum of per-rank timings (the job is as slow as its slowest rank)."""
    import torch
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def job_tokens_per_s(batch, steps, world, ms_max):
    """Whole-job throughput: tokens all ranks decoded divided by the slowest rank's time."""
    return world * batch * steps / (ms_max * 1e-3)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="mkv", choices=["mkv", "reference"])
    ap.add_argument("--config", default="llama_b16", choices=sorted(CONFIGS))
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "mma"])
    ap.add_argument("--score-mode", default="group", choices=["group", "layer"],
                    help="group: mean over the query heads of a KV head (headline); layer: Eq. 4 over all heads")
    ap.add_argument("--budget", type=int, default=0, help="override the workload's decode budget (profiling small cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    w = CONFIGS[args.config]
    if args.budget > 0:
        w = w.with_(budget=args.budget)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    import paper_2605_29873_b200 as mkv

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # every rank holds its own batch (weak scaling; units are independent, no collective)
    wr = rank_workload(w, rank)
    lens = wr.prefill_lens()
    Lmax = int(lens.max())
    B, Hq, Hkv, d = w.batch, w.q_heads, w.kv_heads, w.head_dim
    kernel = {"auto": mkv.MKV_KERNEL_AUTO, "simt": mkv.MKV_KERNEL_SIMT, "mma": mkv.MKV_KERNEL_MMA}[args.kernel]
    kv_dtype = mkv.MKV_BF16 if w.dtype == "bf16" else mkv.MKV_F32
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    ctx = mkv.MomentKV(args.layers, Hq, Hkv, d, w.budget, w.beta, B, Lmax, kv_dtype=kv_dtype, out_dtype=kv_dtype,
                       kernel=kernel, device=local,
                       score_mode=mkv.MKV_SCORE_LAYER_MEAN if args.score_mode == "layer" else mkv.MKV_SCORE_GROUP_MEAN)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)
    for layer in range(args.layers):
        K = (torch.randn((B, Hkv, Lmax, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
        V = (torch.randn((B, Hkv, Lmax, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
        ctx.prefill(layer, K, V, lens)
        torch.cuda.synchronize()
        del K, V
    ring = 64
    qs = torch.randn((ring, B, Hq, d), generator=gen, device=dev).to(tdt)
    ks = (torch.randn((ring, B, Hkv, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
    vs = (torch.randn((ring, B, Hkv, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
    out = torch.empty((B, Hq, d), dtype=tdt, device=dev)

    def step(i):
        ctx.decode_step(i % args.layers, qs[i % ring], ks[i % ring], vs[i % ring], out)

    stream = torch.cuda.current_stream(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The ramp: every layer's decode pool from empty to the budget, timed on its own (steps get
    # longer as the pool grows); it also is the set-up of the steady state measured below.
    # Plain attention launches warm the kernel up first: they leave the state alone.
    for i in range(10):
        ctx.attend_only(i % args.layers, qs[i % ring], out)
    torch.cuda.synchronize()
    n_ramp = w.budget * args.layers
    ev0.record(stream)
    for i in range(n_ramp):
        step(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    ms_ramp = ev0.elapsed_time(ev1) / n_ramp
    ctx.status_sync()
    for i in range(args.warmup):
        step(i)
    sampler = ClockSampler(local)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    launches0 = ctx.launch_count()
    sampler.start()
    # five equal segments of the timed region get events of their own (spread of the step time)
    n_seg = 5 if args.steps >= 50 else 1
    seg_ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_seg - 1)]
    seg_at = {args.steps * (j + 1) // n_seg: seg_ev[j] for j in range(n_seg - 1)}
    ev0.record(stream)
    for i in range(args.steps):
        step(i)
        if i + 1 in seg_at:
            seg_at[i + 1].record(stream)
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = ctx.launch_count() - launches0
    ms = ev0.elapsed_time(ev1)
    marks = [ev0] + seg_ev + [ev1]
    bounds = [0] + sorted(seg_at) + [args.steps]
    seg_ms = [marks[j].elapsed_time(marks[j + 1]) / max(bounds[j + 1] - bounds[j], 1) for j in range(n_seg)]
    ctx.status_sync()

    # plain decode attention on the same state (no append/score/evict): overhead reference
    for i in range(10):
        ctx.attend_only(i % args.layers, qs[i % ring], out)
    barrier()
    n_att = max(100, args.steps // 4)
    ev0.record(stream)
    for i in range(n_att):
        ctx.attend_only(i % args.layers, qs[i % ring], out)
    ev1.record(stream)
    barrier()
    ms_att = ev0.elapsed_time(ev1) / n_att

    # the same steps recorded once and replayed as a CUDA graph (what a serving loop would do):
    # launch cost leaves the host, which shows on the small, launch-bound workloads
    ms_graph, n_rec = 0.0, 16 * args.layers
    if not args.no_graph:
        side = torch.cuda.Stream(dev)
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(n_rec):
                step(i)
        reps = max(3, args.steps // n_rec)
        for _ in range(3):
            graph.replay()
        barrier()
        ev0.record(stream)
        for _ in range(reps):
            graph.replay()
        ev1.record(stream)
        barrier()
        ms_graph = ev0.elapsed_time(ev1) / (reps * n_rec)
        ctx.status_sync()

    # end to end through the host-buffer entry point: H2D of q,k,v and D2H of out every step
    e2e = None
    if not args.no_e2e:
        # one pinned buffer per step holding q | k_new | v_new back to back (a single H2D copy)
        nq, nk = qs[0].numel(), ks[0].numel()
        packed = torch.empty((ring, nq + 2 * nk), dtype=tdt).pin_memory()
        packed[:, :nq] = qs.reshape(ring, -1).cpu()
        packed[:, nq:nq + nk] = ks.reshape(ring, -1).cpu()
        packed[:, nq + nk:] = vs.reshape(ring, -1).cpu()
        hq = [packed[i, :nq] for i in range(ring)]
        hk = [packed[i, nq:nq + nk] for i in range(ring)]
        hv = [packed[i, nq + nk:] for i in range(ring)]
        hout = torch.empty((B, Hq, d), dtype=tdt).pin_memory()
        n_e2e = max(100, args.steps // 4)
        for i in range(10):
            ctx.decode_step_host(i % args.layers, hq[i % ring], hk[i % ring], hv[i % ring], hout)
            stream.synchronize()
        barrier()
        ev0.record(stream)
        for i in range(n_e2e):
            ctx.decode_step_host(i % args.layers, hq[i % ring], hk[i % ring], hv[i % ring], hout)
            stream.synchronize()          # the host reads the step's result before the next step
        ev1.record(stream)
        barrier()
        ms_e2e = ev0.elapsed_time(ev1)
        es = qs.element_size()
        e2e = {"ms": ms_e2e, "steps": n_e2e, "h2d": (qs[0].numel() + ks[0].numel() + vs[0].numel()) * es,
               "d2h": hout.numel() * hout.element_size()}

    ms_max, ms_att_max, ms_e2e_max, ms_ramp_max, ms_graph_max = max_over_ranks(
        [ms, ms_att, e2e["ms"] / e2e["steps"] if e2e else 0.0, ms_ramp, ms_graph], world, dev)

    if rank == 0:
        ms_per_step = ms_max / args.steps
        tokens_per_s = job_tokens_per_s(B, args.steps, world, ms_max)
        peak, peak_kind = load_peaks()
        alg = algorithmic_bytes_per_step(w, lens, w.budget + 1, 1)
        achieved = alg / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": "decode tokens/sec per layer", "value": tokens_per_s, "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic (device-generated N(0,1) queries, N(0,1)/sqrt(d) keys and values; shapes, "
                    "lengths and budget of the named workload)",
            "config": workload_config(w, lens, args),
            "steps_per_s": world * args.steps / (ms_max * 1e-3),
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": peak_kind, "frac_of_nominal_8TBs": achieved / 8000.0,
                         "algorithmic_bytes_per_step": alg, "traffic": captured_traffic(alg),
                         "kernel": "mma_kernel" if ctx_uses_mma(args, w) else "simt_kernel"},
            "attend_only": {"ms_per_step": ms_att_max, "overhead_ratio": ms_per_step / ms_att_max},
        }
        # whole run of the workload (its step count per layer): the measured ramp, then steady state
        T = max(int(w.steps), 1)
        fill = min(w.budget, T)
        run_ms = ms_ramp_max * fill + ms_per_step * (T - fill)
        line["ramp"] = {"ms_per_step": ms_ramp_max, "steps_per_layer": w.budget,
                        "what": "decode pool from empty to the budget, mean over the fill"}
        line["whole_run"] = {"steps_per_layer": T, "ms_per_step": run_ms / T,
                             "tokens_per_s": world * B * T / (run_ms * 1e-3),
                             "how": "measured ramp mean x fill steps + measured steady state x the rest"}
        if world == 1:
            srt = sorted(seg_ms)
            line["segments"] = {"n": n_seg, "median_ms_per_step": srt[len(srt) // 2], "min_ms_per_step": srt[0],
                                "max_ms_per_step": srt[-1]}
        if ms_graph_max > 0.0:
            line["graph_replay"] = {"ms_per_step": ms_graph_max, "steps_per_graph": n_rec,
                                    "tokens_per_s": world * B / (ms_graph_max * 1e-3)}
        if e2e:
            line["e2e"] = {"value": world * B / (ms_e2e_max * 1e-3), "unit": "tokens/s",
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": ms_e2e_max, "sync": "stream synchronised after every step",
                           "how": "per step the GPU fetches q|k_new|v_new from the pinned host buffer (a small kernel ahead of the step) and the step's kernel writes out into the pinned host buffer"}
        if not args.no_cpu_baseline and world == 1:
            n_units = min(len(os.sched_getaffinity(0)), B * Hkv)
            v, threads, sample, _ = time_oracle(w, lens, n_units, steps=48, warmup=2, time_cap_s=40.0, min_time_s=12.0)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def ctx_uses_mma(args, w):
    return args.kernel != "simt" and w.dtype == "bf16" and w.head_dim == 128 and w.group <= 8


if __name__ == "__main__":
    main()
