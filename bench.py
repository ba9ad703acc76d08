#!/usr/bin/env python
"""Benchmark of the Moment-KV decode hot path on B200.

A "step" is one call of mkv_decode_step for one attention layer over the whole batch:
append, GQA attention over prefill U decode pool, momentum score update, lowest-score
eviction, compaction -- all rows of the hot path.  The workload is the Llama-3.1-8B layer
shape at batch 16 (prefill lengths uniform in [512, 4096], decode budget 1024, beta 0.9)
at steady state, i.e. with the decode pool full so that every step evicts.  `--layers`
identical layers are cycled so that every layer-step streams a cache that is cold in L2
(as in a real 32-layer model).

Timing.  The steps of a decode loop overlap (a step starts while the previous one ends), so
a timed region must begin with the pipeline full: after the barrier + synchronize, a lead-in
of untimed steps is enqueued, the first event is recorded behind it without any
synchronisation, exactly K steps follow, then the second event and a barrier + synchronize.
Plain attention on the same state (mkv_attend_only: the reference the score/evict overhead is
quoted against) is timed the same way over the same number of steps; the two arms alternate
for a few rounds and the medians are reported.

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
TRAFFIC_CAPTURE = {"sources_sha1": "fd4cb3cf086653becf7a444c0c4f11a47f759db5", "traffic_over_algorithmic": 1.0221}
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
        "config": workload_config(w, lens, args, args.inputs),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, lens, args, inputs="plain", older=None):
    shape = {"llama_b16": "Llama-3.1-8B attention layer shape", "llama_b1": "Llama-3.1-8B attention layer shape",
             "llama_stack": "Llama-3.1-8B attention layer shape", "qwen_b64": "Qwen2.5-7B-like attention layer shape",
             "tiny": "tiny single-layer shape"}.get(w.name, w.name)
    pre = (f"prefill lengths U[{w.prefill[0]},{w.prefill[1]}]" if not isinstance(w.prefill, int) else f"prefill {w.prefill}")
    return {"workload": f"{w.name}: {shape}, {w.q_heads}/{w.kv_heads} heads, "
                        f"head_dim {w.head_dim}, {w.dtype}, batch {w.batch}, {pre} "
                        f"(sum {int(np.sum(lens))}), decode budget {w.budget}, beta {w.beta}, steady state "
                        f"(decode pool full, one eviction per unit per step); " + input_note(inputs, older),
            "layers_cycled": args.layers,
            "l2": "inputs larger than L2: each layer-step streams its own ~%d MB cache, %d layers cycled"
                  % (int(sum(w.kv_heads * (int(lp) + w.budget + 1) * 2 * w.head_dim * (2 if w.dtype == "bf16" else 4) for lp in lens) / 1e6), args.layers)}


def input_note(inputs, older):
    if inputs == "hot":
        note = ("device-generated inputs of the 'hot' kind: queries 2*sqrt(d)*N(0,1), keys N(0,1)/sqrt(d) plus half a "
                "unit vector along the group's mean query, values N(0,1)/sqrt(d), so that evictions hit tokens of all "
                "ages and the fresh row is stored into the evicted slot")
    else:
        note = ("device-generated N(0,1) queries and N(0,1)/sqrt(d) keys and values: attention is near uniform and the "
                "token evicted is almost always the fresh one, whose row is then not stored")
    if older is not None:
        note += f" (in the last timed step {older[0]} of {older[1]} units evicted an older token)"
    return note


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



def make_ring(torch, gen, ring, lead, Hq, Hkv, d, tdt, dev, inputs):
    """A ring of pre-generated step inputs on the device: q [ring, *lead, Hq, d], k_new / v_new
    [ring, *lead, Hkv, d].  They are final before any step is enqueued."""
    G = Hq // Hkv
    z = torch.randn((ring, *lead, Hq, d), generator=gen, device=dev)
    k = torch.randn((ring, *lead, Hkv, d), generator=gen, device=dev) / d ** 0.5
    v = torch.randn((ring, *lead, Hkv, d), generator=gen, device=dev) / d ** 0.5
    if inputs == "hot":
        q = 2.0 * d ** 0.5 * z
        qbar = q.reshape(ring, *lead, Hkv, G, d).mean(dim=-2)
        k = k + 0.5 * qbar / qbar.norm(dim=-1, keepdim=True)
    else:
        q = z
    return q.to(tdt).contiguous(), k.to(tdt).contiguous(), v.to(tdt).contiguous()


class Arm:
    """One configuration set up on the device at steady state: context, input ring, step functions."""

    def __init__(self, torch, mkv, w, lens, layers, dev, seed, inputs, score_mode="group", kernel="auto", stacked=False,
                 out_dtype=None, head_tiles=None, fill=None, early=True, grid_share=None):
        self.torch, self.w, self.layers, self.stacked = torch, w, layers, stacked
        B, Hq, Hkv, d = w.batch, w.q_heads, w.kv_heads, w.head_dim
        kv_dtype = mkv.MKV_BF16 if w.dtype == "bf16" else mkv.MKV_F32
        tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        Lmax = int(lens.max())
        self.ctx = mkv.MomentKV(layers, Hq, Hkv, d, w.budget, w.beta, B, Lmax, kv_dtype=kv_dtype,
                                out_dtype=kv_dtype if out_dtype is None else out_dtype,
                                kernel={"auto": mkv.MKV_KERNEL_AUTO, "simt": mkv.MKV_KERNEL_SIMT, "mma": mkv.MKV_KERNEL_MMA}[kernel],
                                device=dev.index,
                                score_mode=mkv.MKV_SCORE_LAYER_MEAN if score_mode == "layer" else mkv.MKV_SCORE_GROUP_MEAN,
                                flags=mkv.MKV_FLAG_INPUTS_READY if early else 0)
        if head_tiles is not None:
            self.ctx.set_option(mkv.MKV_OPT_HEAD_TILES, head_tiles)
        if grid_share is not None:
            self.ctx.set_option(mkv.MKV_OPT_GRID_SHARE, grid_share)
        gen = torch.Generator(device=dev)
        gen.manual_seed(seed)
        for layer in range(layers):
            K = (torch.randn((B, Hkv, Lmax, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
            V = (torch.randn((B, Hkv, Lmax, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
            self.ctx.prefill(layer, K, V, lens)
            torch.cuda.synchronize()
            del K, V
        self.ring = 8 if stacked else 64
        lead = (layers, B) if stacked else (B,)
        self.qs, self.ks, self.vs = make_ring(torch, gen, self.ring, lead, Hq, Hkv, d, tdt, dev, inputs)
        odt = torch.float32 if (out_dtype is not None and out_dtype == mkv.MKV_F32) else tdt
        # neighbouring steps on different layers may run side by side: they get different outputs
        self.outs = [torch.empty((*lead, Hq, d), dtype=odt, device=dev) for _ in range(2)]
        self.out = self.outs[0]
        torch.cuda.synchronize()
        self.per_call = layers if stacked else 1        # layer-steps one call performs
        self.fill_steps = w.budget if fill is None else fill

    def step(self, i):
        r = i % self.ring
        if self.stacked:
            self.ctx.decode_step_layers(0, self.layers, self.qs[r], self.ks[r], self.vs[r], self.outs[i & 1])
        else:
            self.ctx.decode_step(i % self.layers, self.qs[r], self.ks[r], self.vs[r], self.outs[i & 1])

    def attend(self, i):
        r = i % self.ring
        if self.stacked:
            self.ctx.attend_only_layers(0, self.layers, self.qs[r], self.outs[i & 1])
        else:
            self.ctx.attend_only(i % self.layers, self.qs[r], self.outs[i & 1])

    def fill(self, stream, timed=False):
        """Every layer's decode pool from empty to `fill_steps` tokens; returns ms per layer-step."""
        torch = self.torch
        n = self.fill_steps * (1 if self.stacked else self.layers)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(10):
            self.attend(i)                               # warms the kernel up; leaves the state alone
        torch.cuda.synchronize()
        ev0.record(stream)
        for i in range(n):
            self.step(i)
        ev1.record(stream)
        torch.cuda.synchronize()
        self.ctx.status_sync()
        return ev0.elapsed_time(ev1) / (n * self.per_call)

    def close(self):
        self.ctx.close()


def timed_rounds(torch, stream, barrier, arm, calls, lead_in, rounds, with_attend=True):
    """`rounds` times: [lead-in, event, `calls` decode calls, event] then the same with plain
    attention.  Returns per-round ms per call for both arms and the launches of one timed part."""
    dec, att = [], []
    launches = 0
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    i = 0
    for _ in range(rounds):
        barrier()
        for _ in range(lead_in):
            arm.step(i); i += 1
        l0 = arm.ctx.launch_count()
        ev[0].record(stream)
        for _ in range(calls):
            arm.step(i); i += 1
        ev[1].record(stream)
        launches = arm.ctx.launch_count() - l0
        if with_attend:
            for j in range(lead_in):
                arm.attend(j)
            ev[2].record(stream)
            for j in range(calls):
                arm.attend(j)
            ev[3].record(stream)
        barrier()
        dec.append(ev[0].elapsed_time(ev[1]) / calls)
        if with_attend:
            att.append(ev[2].elapsed_time(ev[3]) / calls)
    return dec, att, launches


def median(xs):
    s = sorted(xs)
    return s[len(s) // 2]


def side_run(torch, mkv, stream, barrier, peak, w, lens, layers, dev, seed, inputs, name, calls=200, rounds=3, **kw):
    """A short steady-state run of another configuration: one entry of `other_configs` / `comparison`."""
    arm = Arm(torch, mkv, w, lens, layers, dev, seed, inputs, **kw)
    ms_fill = arm.fill(stream)
    for i in range(20):
        arm.step(i)
    dec, att, _ = timed_rounds(torch, stream, barrier, arm, calls, 50, rounds)
    arm.ctx.status_sync()
    n_dec = int(arm.ctx.decode_state(0, 0, 0)[0].shape[0])
    arm.close()
    ms = median(dec) / arm.per_call
    ms_att = median(att) / arm.per_call
    alg = algorithmic_bytes_per_step(w, lens, min(n_dec + 1, w.budget + 1), 1 if n_dec >= w.budget else 0)
    gbs = alg / (ms * 1e-3) / 1e9
    return {"name": name, "layers_per_launch": arm.per_call, "decode_pool_tokens": n_dec, "ms_per_layer_step": ms,
            "tokens_per_s": w.batch / (ms * 1e-3), "algorithmic_bytes_per_step": alg, "achieved_gbs": gbs,
            "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0, "attend_only_ms": ms_att,
            "overhead_ratio": median([d / a for d, a in zip(dec, att)]), "ramp_ms_per_layer_step": ms_fill,
            "steps_timed": calls, "rounds": rounds}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="mkv", choices=["mkv", "reference"])
    ap.add_argument("--config", default="llama_b16", choices=sorted(CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="layers cycled (0: 4, or the whole stack for llama_stack)")
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "mma"])
    ap.add_argument("--score-mode", default="group", choices=["group", "layer"],
                    help="group: mean over the query heads of a KV head (headline); layer: Eq. 4 over all heads")
    ap.add_argument("--budget", type=int, default=0, help="override the workload's decode budget (profiling small cases)")
    ap.add_argument("--inputs", default="hot", choices=["hot", "plain"], help="kind of device-generated step inputs")
    ap.add_argument("--head-tiles", type=int, default=-1, help="reserved prompt tiles per CTA (default: the library's)")
    ap.add_argument("--grid-share", type=int, default=-1, help="percent of the resident CTA slots a step uses (default: the library's)")
    ap.add_argument("--no-early", action="store_true", help="do not promise that the inputs are final at enqueue time")
    ap.add_argument("--per-layer", action="store_true", help="llama_stack: one launch per layer instead of one per stack")
    ap.add_argument("--rounds", type=int, default=5)
    ap.add_argument("--lead-in", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    ap.add_argument("--no-others", action="store_true", help="skip the other configurations and the comparison runs")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    w = CONFIGS[args.config]
    if args.budget > 0:
        w = w.with_(budget=args.budget)
    stacked = args.config == "llama_stack" and not args.per_layer
    if args.layers <= 0:
        args.layers = w.layers if args.config == "llama_stack" else 4
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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank holds its own batch (weak scaling; units are independent, no collective)
    wr = rank_workload(w, rank)
    lens = wr.prefill_lens()
    B, Hq, Hkv, d = w.batch, w.q_heads, w.kv_heads, w.head_dim
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    head_tiles = args.head_tiles if args.head_tiles >= 0 else None
    arm = Arm(torch, mkv, w, lens, args.layers, dev, 1234 + rank, args.inputs, score_mode=args.score_mode,
              kernel=args.kernel, stacked=stacked, head_tiles=head_tiles, early=not args.no_early,
              grid_share=args.grid_share if args.grid_share > 0 else None)
    ctx = arm.ctx
    stream = torch.cuda.current_stream(dev)
    # The ramp: every layer's decode pool from empty to the budget, timed on its own (steps get
    # longer as the pool grows); it also is the set-up of the steady state measured below.
    ms_ramp = arm.fill(stream)
    for i in range(args.warmup):
        arm.step(i)
    ctx_grid = ctx.grid(args.layers if stacked else 0)
    sampler = ClockSampler(local)
    calls = max(1, args.steps // arm.per_call) if stacked else args.steps
    sampler.start()
    dec, att, launches = timed_rounds(torch, stream, barrier, arm, calls, args.lead_in, max(1, args.rounds))
    clocks = sampler.stop()
    ctx.status_sync()
    # which tokens the last timed step evicted (the fresh one, or an older one whose slot took the fresh row)
    older = [0, 0]
    for b in range(B):
        for g in range(Hkv):
            ev_pos, _ = ctx.last_evicted(0, b, g)
            if len(ev_pos):
                older[1] += 1
                older[0] += int(int(ev_pos[0]) != ctx.step_count(0) - 1)

    # the same steps recorded once and replayed as a CUDA graph (what a serving loop would do):
    # launch cost leaves the host, which shows on the small, launch-bound workloads
    ms_graph, n_rec = 0.0, (4 if stacked else 16 * args.layers)
    if not args.no_graph:
        side = torch.cuda.Stream(dev)
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(n_rec):
                arm.step(i)
        reps = max(3, calls // n_rec)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        for _ in range(3):
            graph.replay()
        ev0.record(stream)
        for _ in range(reps):
            graph.replay()
        ev1.record(stream)
        barrier()
        ms_graph = ev0.elapsed_time(ev1) / (reps * n_rec * arm.per_call)
        ctx.status_sync()

    # end to end through the host-buffer entry point: H2D of q,k,v and D2H of out every step
    e2e = None
    if not args.no_e2e and not stacked:
        # A caller with host buffers makes no promise about device inputs: a context of its own,
        # without MKV_FLAG_INPUTS_READY (every step synchronised, nothing to run alongside).
        arm.close()
        arm = Arm(torch, mkv, w, lens, args.layers, dev, 1234 + rank, args.inputs, score_mode=args.score_mode,
                  kernel=args.kernel, head_tiles=head_tiles, early=False)
        arm.fill(stream)
        ctx = arm.ctx
        qs, ks, vs = arm.qs, arm.ks, arm.vs
        ring = arm.ring
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
        n_e2e = max(100, min(args.steps, 2000))
        for i in range(10):
            ctx.decode_step_host(i % args.layers, hq[i % ring], hk[i % ring], hv[i % ring], hout)
            stream.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for i in range(n_e2e):
            ctx.decode_step_host(i % args.layers, hq[i % ring], hk[i % ring], hv[i % ring], hout)
            stream.synchronize()          # the host reads the step's result before the next step
        ev1.record(stream)
        barrier()
        es = qs.element_size()
        e2e = {"ms": ev0.elapsed_time(ev1), "steps": n_e2e, "h2d": (qs[0].numel() + ks[0].numel() + vs[0].numel()) * es,
               "d2h": hout.numel() * hout.element_size()}
    arm.close()

    R = len(dec)
    red = max_over_ranks(dec + att + [e2e["ms"] / e2e["steps"] if e2e else 0.0, ms_ramp, ms_graph], world, dev)
    dec_max, att_max = red[:R], red[R:2 * R]
    ms_e2e_max, ms_ramp_max, ms_graph_max = red[2 * R:]

    if rank == 0:
        ms_call = median(dec_max)
        ms_per_step = ms_call / arm.per_call                      # per layer-step
        ms_att = median(att_max) / arm.per_call
        tokens_per_s = world * B / (ms_per_step * 1e-3)
        peak, peak_kind = load_peaks()
        alg = algorithmic_bytes_per_step(w, lens, w.budget + 1, 1)
        achieved = alg / (ms_per_step * 1e-3) / 1e9
        cfg = workload_config(w, lens, args, args.inputs, older)
        cfg["launch"] = (f"one launch per {arm.per_call}-layer stack" if stacked else "one launch per layer-step")
        cfg["early_inputs"] = not args.no_early
        cfg["grid"] = "%d CTAs of %d resident" % ctx_grid
        line = {
            "metric": "decode tokens/sec per layer", "value": tokens_per_s, "unit": "tokens/s",
            "n_gpus": world, "steps": calls * arm.per_call, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic (device-generated; shapes, lengths and budget of the named workload)",
            "config": cfg,
            "steps_per_s": world / (ms_per_step * 1e-3),
            "gpu_launches": int(launches),
            "clocks": clocks,
            "timing": {"how": "barrier + synchronize, an untimed lead-in, event, the timed steps, event, barrier + "
                              "synchronize; decode and plain attention alternate; medians over the rounds",
                       "rounds": R, "lead_in_steps": args.lead_in, "timed_calls_per_round": calls,
                       "layer_steps_per_call": arm.per_call,
                       "ms_per_step_rounds": [x / arm.per_call for x in dec_max],
                       "attend_only_ms_rounds": [x / arm.per_call for x in att_max]},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": peak_kind, "frac_of_nominal_8TBs": achieved / 8000.0,
                         "algorithmic_bytes_per_step": alg, "traffic": captured_traffic(alg),
                         "kernel": "mma_kernel" if ctx_uses_mma(args, w) else "simt_kernel"},
            "attend_only": {"ms_per_step": ms_att,
                            "overhead_ratio": median([a / b for a, b in zip(dec_max, att_max)]),
                            "how": "same state, same number of steps, same lead-in; median over the rounds of decode / plain"},
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
        if ms_graph_max > 0.0:
            line["graph_replay"] = {"ms_per_step": ms_graph_max, "steps_per_graph": n_rec * arm.per_call,
                                    "tokens_per_s": world * B / (ms_graph_max * 1e-3)}
        if e2e:
            line["e2e"] = {"value": world * B / (ms_e2e_max * 1e-3), "unit": "tokens/s",
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": ms_e2e_max, "sync": "stream synchronised after every step",
                           "how": "per step the GPU fetches q|k_new|v_new from the pinned host buffer (a small kernel ahead of the step) and the step's kernel writes out into the pinned host buffer"}
        if world == 1 and not args.no_others and args.config == "llama_b16" and args.budget == 0:
            line["other_configs"], line["comparison"] = other_runs(torch, mkv, stream, barrier, peak, dev, args)
        if not args.no_cpu_baseline and world == 1:
            n_units = min(len(os.sched_getaffinity(0)), B * Hkv)
            v, threads, sample, _ = time_oracle(w, lens, n_units, steps=48, warmup=2, time_cap_s=40.0, min_time_s=12.0)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def other_runs(torch, mkv, stream, barrier, peak, dev, args):
    """Short steady-state runs of the other configurations, and the comparison of the paper's
    throughput figure (Sec. 7.4: full cache against score-tracking methods) inside the library:
    the headline batch with a decode pool that is never evicted from, at the sizes a full cache
    reaches after 4096 and 8192 generated tokens, against the budget of 1024; and the two limits
    of the momentum factor (beta changes no byte that moves)."""
    inputs = args.inputs
    others = []
    ws = CONFIGS["llama_stack"]
    others.append(side_run(torch, mkv, stream, barrier, peak, ws, ws.prefill_lens(), ws.layers, dev, 21, inputs,
                           "llama_stack: 32 layers, batch 4, prefill 2048, budget 2048; one launch per stack",
                           calls=40, rounds=3, stacked=True))
    for budget in (128, 1024):
        wq = CONFIGS["qwen_b64"].with_(budget=budget)
        others.append(side_run(torch, mkv, stream, barrier, peak, wq, wq.prefill_lens(), 4, dev, 22, inputs,
                               f"qwen_b64: 28/4 heads (group 7), batch 64, prefill 512, budget {budget}", calls=400))
    wl = CONFIGS["llama_b16"]
    others.append(side_run(torch, mkv, stream, barrier, peak, wl, wl.prefill_lens(), 4, dev, 23, inputs,
                           "llama_b16 in the score mode LAYER_MEAN (Eq. 4 over all heads of the layer)", calls=400,
                           score_mode="layer"))
    comparison = []
    for pool in (4096, 8192):
        wf = wl.with_(budget=pool + 2048)               # never reached: the pool only grows (full cache)
        comparison.append(side_run(torch, mkv, stream, barrier, peak, wf, wf.prefill_lens(), 2, dev, 24, inputs,
                                   f"full cache (no eviction), decode pool grown to about {pool} tokens", calls=100,
                                   rounds=3, fill=pool - 300))
    for beta in (0.0, 1.0):
        wb = wl.with_(beta=beta)
        comparison.append(side_run(torch, mkv, stream, barrier, peak, wb, wb.prefill_lens(), 2, dev, 25, inputs,
                                   f"budget 1024, beta {beta}", calls=200, rounds=3))
    return others, comparison


def ctx_uses_mma(args, w):
    return args.kernel != "simt" and w.dtype == "bf16" and w.head_dim == 128 and w.group <= 8


if __name__ == "__main__":
    main()
