#!/usr/bin/env python
"""Benchmark of the mixed paged-attention step (ts_mixed_step) on synthetic bursty batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config3] [--impl ours|reference]

One "step" is one pass of the whole path (table sync, KV append, attention over decode rows and
prefill chunks, split combine) over one batch. Prints ONE JSON line on rank 0.
N > 1 runs N independent replicas (the path has no exchange step): weak scaling.

Workloads: config2 decode-only batch, config3 convertible-decoder burst (default, the mixed step
the metric names), config4 chunked-prefill continuation, config5 bursty trace replay on a
70B-shaped layer (there a step is one replay step and K is capped by the replay's 200 steps).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2512_03416_b200 import workloads as wl  # noqa: E402

METRIC = "prefill+decode tokens/s per B200 in mixed paged-attn step"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the workload's dominant kernel, from
# the ncu captures summarised under profiles/ (decode_kernel on config2, mixed_kernel on config3).
# An entry is dropped (null in the output) when its kernel has changed since the capture.
KERNEL_TRAFFIC_BYTES = {"config2": 7.746e8, "config3": 8.415e8, "prefill_8192_70b": 2.873e8}

WORKLOADS = {
    "config2": (wl.config2, "decode-only batch, 8B-shaped layer (64 decode rows, ctx lognormal median 2048)"),
    "config3": (wl.config3, "convertible-decoder burst, 8B-shaped layer (64 decode rows + one fresh 2048-token prefill chunk)"),
    "config4": (wl.config4, "chunked-prefill continuation, 8B-shaped layer (128 decode rows + 4 chunks of 512 tokens)"),
    "prefill_8192_70b": (None, "one fresh 8192-token prefill chunk alone, 70B-shaped layer (the tile path by itself)"),
    "prefill_2048_8b": (None, "one fresh 2048-token prefill chunk alone, 8B-shaped layer (config3's chunk by itself)"),
    "layer_8b": (None, "the whole decoder layer (RMSNorm, QKV + rotary, attention, output projection, gated MLP; hidden 4096, "
                       "intermediate 14336) over config3's batch: 64 decode rows + one fresh 2048-token prefill chunk"),
    "config5": (None, "bursty trace replay, 70B-shaped layer (200 steps, Gamma arrivals CV=4, <=256 decodes, one prefill task at a time)"),
    "config5_chunked": (None, "the same bursty trace under a chunk size of 2304 (2048 prefill tokens + 256 decode rows): "
                              "prompts continue over several steps, up to 4 requests' chunks share a step"),
}
# what the replays change in the trace simulator's defaults
REPLAY_TRACE = {"config5": {}, "config5_chunked": {"chunk_size": 2304, "max_prefill_tasks": 4}}
N_LAYERS_70B = 80          # layers of the model whose attention layer the replay runs (for the TTFT clock)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            p = json.load(open(path))
            if "hbm_gbs" in p and "bf16_tflops" in p:
                return p, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ multi-process plumbing
def dist_env():
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own batch; rank 0 keeps the documented seed."""
    return base_seed + 1000 * rank


def reduce_max(value: float, world: int, device=None) -> float:
    """Max over ranks of a timing (every multi-GPU number is the slowest rank's)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput: units all ranks processed over the slowest rank's time."""
    return world * units_per_rank / seconds_max


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
                 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=1.0)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------- oracle legs
def oracle_sample(batch, stride: int):
    """Every stride-th decode row and every stride-th prefill token of the batch."""
    sel, tok = [], 0
    for ql in batch.q_len.tolist():
        if ql == 1:
            if (tok % stride) == 0:
                sel.append(tok)
            tok += 1
        else:
            sel.extend(range(tok + (stride - 1), tok + ql, stride))
            tok += ql
    if not sel:
        sel = [batch.n_tokens - 1]
    return np.asarray(sel, dtype=np.int32)


def sample_flops(batch, sel):
    s = batch.shape
    starts = np.concatenate([[0], np.cumsum(batch.q_len)])
    rows = np.searchsorted(starts, sel, side="right") - 1
    keys = batch.ctx_len[rows] + (sel - starts[rows]) + 1
    return 4.0 * s.D * s.Hq * float(keys.sum())


class OracleLeg:
    """The CPU oracle on a bounded sample of the workload (imported only here)."""

    def __init__(self, batch):
        import oracle  # test infrastructure; used only for the reported CPU baseline
        self.oracle = oracle
        self.batch = batch
        s = batch.shape
        self.pool = batch.fresh_pool()
        tm = batch.table_matrix()
        if int(batch.ctx_len.sum()) > 0:
            oracle.kv_append(self.pool, s.Hkv, s.D, s.P, tm, np.zeros_like(batch.ctx_len), batch.ctx_len,
                             batch.context_k, batch.context_v)
        oracle.kv_append(self.pool, s.Hkv, s.D, s.P, tm, batch.ctx_len, batch.q_len, batch.k_new, batch.v_new)
        self.tm = tm
        self.cores = oracle.default_threads()

    def run(self, sel, threads=None) -> float:
        b, s = self.batch, self.batch.shape
        t0 = time.perf_counter()
        self.oracle.attention(self.pool, s.Hq, s.Hkv, s.D, s.P, 1.0 / math.sqrt(s.D), self.tm, b.ctx_len,
                              b.q_len, b.q, sel=sel, threads=threads or self.cores)
        return time.perf_counter() - t0

    def stride_for(self, seconds: float) -> int:
        """Sampling stride whose oracle time is about `seconds`, from a quick calibration."""
        b = self.batch
        probe = oracle_sample(b, max(64, b.n_tokens // 16))
        t = self.run(probe)
        rate = sample_flops(b, probe) / max(t, 1e-6)
        total = b.algorithmic_work()[0]
        return int(min(max(1, math.ceil(total / (rate * seconds))), max(1, b.n_tokens)))


def replay_heavy_batch():
    """The replay's heaviest kind of step as a static batch (what the oracle legs sample for config5):
    192 decode rows with the replay's context mix plus one fresh 8192-token prefill chunk."""
    rng = np.random.Generator(np.random.Philox(5))
    ctx = wl._lognormal_lengths(rng, 1024, 1.0, 16, 8192, 192) + wl._lognormal_lengths(rng, 256, 1.0, 1, 2048, 192) // 2
    ctx = np.concatenate([ctx, [0]]).astype(np.int32)
    ql = np.concatenate([np.ones(192, np.int32), [8192]]).astype(np.int32)
    return wl.make_batch("config5_heavy_step", wl.LLAMA70B, ctx, ql, seed=105, chunk_size=8448)


def make_static_batch(workload: str, rank: int):
    if workload in REPLAY_TRACE:
        return replay_heavy_batch()
    if workload == "prefill_8192_70b":
        return wl.make_batch(workload, wl.LLAMA70B, [0], [8192], seed=rank_seed(81, rank), chunk_size=8192)
    if workload == "prefill_2048_8b":
        return wl.make_batch(workload, wl.LLAMA8B, [0], [2048], seed=rank_seed(82, rank), chunk_size=2048)
    make = WORKLOADS[workload][0]
    return make(seed=rank_seed(make.__defaults__[0], rank))


def cpu_baseline_leg(batch, target_s: float = 10.0):
    leg = OracleLeg(batch)
    stride = leg.stride_for(target_s)
    sel = oracle_sample(batch, stride)
    t, reps = 0.0, 0
    while t < target_s * 0.6 and reps < 64:          # repeat small workloads up to a few seconds of CPU work
        t += leg.run(sel)
        reps += 1
    # the same oracle on one thread, on a sample thinned by the core count (a few seconds)
    stride1 = min(max(1, stride * leg.cores * 2), max(1, batch.n_tokens))
    sel1 = oracle_sample(batch, stride1)
    t1 = leg.run(sel1, threads=1)
    return {"value": reps * len(sel) / t, "unit": UNIT, "cores": leg.cores, "kind": "oracle",
            "sample": f"every {stride}th decode row and every {stride}th prefill token of {batch.name} "
                      f"({len(sel)} of {batch.n_tokens} tokens), repeated {reps}x, {t:.1f} s",
            "single_thread": {"value": len(sel1) / t1, "unit": UNIT, "cores": 1,
                              "sample": f"every {stride1}th decode row and prefill token ({len(sel1)} tokens), {t1:.1f} s"}}


def run_reference(args):
    world, rank, _ = dist_env()
    if rank != 0:
        return
    desc = WORKLOADS[args.workload][1]
    if args.workload == "layer_8b":
        vals = [layer_cpu_baseline(wl.LLAMA8B, LAYER_8B["hidden"], LAYER_8B["intermediate"]) for _ in range(args.warmup + args.steps)][args.warmup:]
        value = float(np.mean([v["value"] for v in vals])) if vals else 0.0
        base = dict(vals[-1], value=value) if vals else None
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": 128.0 / max(value, 1e-9) * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": args.workload, "description": desc},
                "cpu_baseline": base, "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line), flush=True)
        return
    batch = make_static_batch(args.workload, 0)
    leg = OracleLeg(batch)
    budget = 150.0 / max(1, args.steps + args.warmup)
    stride = leg.stride_for(budget)
    sel = oracle_sample(batch, stride)
    for _ in range(args.warmup):
        leg.run(sel)
    t = 0.0
    for _ in range(args.steps):
        t += leg.run(sel)
    per_step = t / max(1, args.steps)
    value = len(sel) / per_step
    sample = (f"every {stride}th decode row and every {stride}th prefill token of {batch.name} "
              f"({len(sel)} of {batch.n_tokens} tokens) per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": {"workload": args.workload, "description": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": leg.cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------- our arm
def rooflines(peaks, peak_kind, flops, byts, step_ms, prof, parts, traffic=None, launches_per_step=None):
    """Roofline of the dominant kernel (times from the library's own CUDA events) and of the step.

    `parts` holds algorithmic work per recorded step, averaged over all recorded steps:
    dec_bytes of the steps whose decode rows ran in decode_kernel, pf_flops of the steps whose launch
    held prefill tiles only, and mixed_bytes / mixed_flops of the steps where one launch ran tiles
    and decode rows together (that launch is the whole step: append, attention, split merge).
    The dominant kernel is the one with the largest total time; achieved = its algorithmic work
    over its own time.
    """
    steps = max(1, prof["steps"])
    dec_ms, pf_ms, mixed_ms = prof["decode_ms"] / steps, prof["prefill_ms"] / steps, prof.get("mixed_ms", 0.0) / steps
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    # A step that is a single launch: the kernel's average duration is the step time of the timed
    # region itself (back-to-back launches); the event-per-kernel pass is only needed to split
    # steps of several launches, and its extra events make each kernel a little slower.
    source = "events around each kernel, separate pass"
    if launches_per_step == 1 and mixed_ms > 0:
        mixed_ms, source = step_ms, "timed region (the launch is the whole step)"

    def hbm(kernel, nbytes, ms, tr=None):
        ach = nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": tr, "kernel": kernel, "kernel_ms": ms}

    def tensor(kernel, nflops, ms):
        ach = nflops / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
        return {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops"], "traffic": None, "kernel": kernel, "kernel_ms": ms}

    if mixed_ms >= dec_ms and mixed_ms >= pf_ms and mixed_ms > 0:
        if parts["mixed_bytes"] / (peaks["hbm_gbs"] * 1e9) >= parts["mixed_flops"] / (peaks["bf16_tflops"] * 1e12):
            roof = hbm("mixed_kernel", parts["mixed_bytes"], mixed_ms, traffic)
        else:
            roof = tensor("mixed_kernel", parts["mixed_flops"], mixed_ms)
    elif dec_ms >= pf_ms:
        roof = hbm("decode_kernel", parts["dec_bytes"], dec_ms, traffic)
    else:
        roof = tensor("mixed_kernel (prefill tiles only)", parts["pf_flops"], pf_ms)
    roof.update({"peak_source": f"of {peak_kind}", "kernel_ms_source": source, "decode_ms": dec_ms, "prefill_ms": pf_ms, "mixed_ms": mixed_ms,
                 "mixed_steps": prof.get("mixed_steps", 0), "recorded_steps": prof["steps"],
                 "append_ms": prof["append_ms"] / steps, "combine_ms": prof["combine_ms"] / steps,
                 "decode_GBps": parts["dec_bytes"] / (dec_ms * 1e-3) / 1e9 if dec_ms > 1e-3 else None,
                 "prefill_TFLOPs": parts["pf_flops"] / (pf_ms * 1e-3) / 1e12 if pf_ms > 1e-3 else None,
                 "mixed_GBps": parts["mixed_bytes"] / (mixed_ms * 1e-3) / 1e9 if mixed_ms > 1e-3 else None,
                 "mixed_TFLOPs": parts["mixed_flops"] / (mixed_ms * 1e-3) / 1e12 if mixed_ms > 1e-3 else None})
    roof["frac_nominal"] = roof["achieved"] / (8000.0 if roof["bound"] == "hbm" else 2250.0)
    t_roof = max(t_hbm, t_tc)
    step_roof = {"t_roof_us": t_roof * 1e6, "t_hbm_us": t_hbm * 1e6, "t_tensor_us": t_tc * 1e6,
                 "frac": t_roof / (step_ms * 1e-3), "flops": flops, "bytes": byts,
                 "frac_nominal": max(byts / 8e12, flops / 2.25e15) / (step_ms * 1e-3)}
    return roof, step_roof


MIN_TIMED_S = 0.4          # the timed region lasts at least this long, whatever --steps says
MAX_BLOCKS = 4000


def run_static(args, world, rank, local, barrier, workload=None, light=False):
    """Times blocks of exactly K steps (CUDA events around each block, barrier on both sides of
    the region), repeated until the region has lasted MIN_TIMED_S, and reports the median block:
    a handful of 0.16 ms steps is too short a region for the clocks to be sampled or trusted.
    `light`: no end-to-end leg (the extra workloads of the default line)."""
    import torch
    from paper_2512_03416_b200.harness import LoadedBatch

    workload = workload or args.workload
    batch = make_static_batch(workload, rank)
    lb = LoadedBatch(batch, device=local, nan_fill=False)
    s = batch.shape
    K, W = args.steps, max(args.warmup, 3)
    for _ in range(W):
        lb.step_repeatable()
    barrier()
    v0 = lb.dec.velocity()
    sampler = ClockSampler(local)
    sampler.start()
    events = [torch.cuda.Event(enable_timing=True)]
    barrier()
    t_host = time.perf_counter()
    events[0].record()
    n_blocks = 0
    while True:
        for _ in range(K):
            lb.step_repeatable()
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        events.append(ev)
        n_blocks += 1
        if n_blocks % 8 == 0 or n_blocks < 8:
            ev.synchronize()                          # bounds the queue and gives the region's length so far
            if time.perf_counter() - t_host >= MIN_TIMED_S or n_blocks >= MAX_BLOCKS:
                break
    barrier()
    clocks = sampler.stop()
    block_ms = [events[i].elapsed_time(events[i + 1]) for i in range(n_blocks)]
    ms_step = reduce_max(float(np.median(block_ms)), world, "cuda") / K
    region_s = events[0].elapsed_time(events[-1]) * 1e-3
    launches = int(lb.dec.velocity()["kernel_launches"] - v0["kernel_launches"]) // n_blocks
    tokens = batch.n_tokens
    status = lb.dec.device_status()                   # a bounded wait that ran out would make the timing meaningless
    if status != 0:
        raise SystemExit(f"the device reported status {status} during the timed steps")

    lb.dec.profile_enable(True)                       # separate pass: the extra events cost a little
    for _ in range(300):
        lb.step_repeatable()
    prof = lb.dec.profile_read()
    lb.dec.profile_enable(False)

    flops, byts = batch.algorithmic_work()
    dec = batch.q_len == 1
    dec_bytes = float(((batch.ctx_len[dec] + 1) * s.kv_bytes_per_token).sum() + 2 * dec.sum() * s.Hq * s.D * 2)
    pf_flops = 4.0 * s.D * s.Hq * float(sum(t * c + t * (t + 1) / 2 for c, t in
                                            zip(batch.ctx_len[~dec].tolist(), batch.q_len[~dec].tolist())))
    mixed = prof.get("mixed_steps", 0) > 0          # one launch ran the tiles and the decode rows together
    parts = {"dec_bytes": 0.0 if mixed else dec_bytes, "pf_flops": 0.0 if mixed else pf_flops,
             "mixed_bytes": byts if mixed else 0.0,     # the mixed launch also appends the new K/V
             "mixed_flops": flops if mixed else 0.0}

    kv_tokens = int((batch.ctx_len + batch.q_len).sum())
    cfg = {"decode_rows": batch.decode_tokens, "prefill_tokens": batch.prefill_tokens, "kv_tokens": kv_tokens,
           "l2": ("inputs larger than L2 (KV working set %.2f GB)" if kv_tokens * s.kv_bytes_per_token > 126e6 else
                  "KV working set %.3f GB fits in L2 and is not flushed: a tensor-bound diagnostic, no HBM claim")
                 % (kv_tokens * s.kv_bytes_per_token / 1e9),
           "timing": f"median of {n_blocks} blocks of {K} steps, CUDA events around each block, "
                     f"timed region {region_s:.2f} s"}
    e2e = None
    if not light:
        # end to end: host buffers in, host buffer out, through ts_mixed_step_host; one pipelined
        # region of at least K steps and at least MIN_TIMED_S
        hq = torch.from_numpy(batch.q.view(np.int16)).pin_memory()
        hk = torch.from_numpy(batch.k_new.view(np.int16)).pin_memory()
        hv = torch.from_numpy(batch.v_new.view(np.int16)).pin_memory()
        ho = torch.empty_like(hq).pin_memory()
        ql, cl = batch.q_len.tolist(), batch.ctx_len.tolist()
        t0 = time.perf_counter()
        for _ in range(3):
            lb.dec.mixed_step_host(lb.slots, ql, cl, hq, hk, hv, ho, keep_len=True)
        est = (time.perf_counter() - t0) / 3
        Ke = int(min(max(K, math.ceil(MIN_TIMED_S / max(est, 1e-5))), 5000))
        barrier()
        t0 = time.perf_counter()
        for _ in range(Ke):         # enqueue only: the next step's upload overlaps this step's kernels and download
            lb.dec.mixed_step_host(lb.slots, ql, cl, hq, hk, hv, ho, keep_len=True, wait=False)
        lb.dec.host_fence()
        torch.cuda.synchronize()
        e2e_s = reduce_max(time.perf_counter() - t0, world, "cuda")
        if lb.dec.device_status() != 0:
            raise SystemExit("the device reported a failure during the end-to-end loop")
        e2e = {"value": aggregate_value(tokens, world, e2e_s / Ke), "unit": UNIT,
               "h2d_bytes_per_step": int(hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2),
               "d2h_bytes_per_step": int(ho.numel() * 2), "steps": Ke, "ms_per_step": e2e_s / Ke * 1e3}
    lb.dec.close()
    return dict(batch=batch, ms_step=ms_step, tokens=tokens, prefill_tokens=batch.prefill_tokens,
                decode_tokens=batch.decode_tokens, launches=launches, clocks=clocks, prof=prof, flops=flops,
                byts=byts, parts=parts, e2e=e2e, cfg=cfg, steps=K, warmup=W,
                extra={"timed_blocks": n_blocks, "timed_region_s": region_s})


LAYER_8B = {"hidden": 4096, "intermediate": 14336, "max_position": 16384}


def layer_cpu_baseline(s, hidden, inter, n_tokens=128):
    """The layer oracle (fp64, numpy on all host cores for the projections, the C oracle for the
    attention) on a bounded sample: one fresh chunk of n_tokens tokens through the whole layer."""
    import oracle
    from oracle import layer as OL
    rng = np.random.default_rng(7)
    qd, kvd = s.Hq * s.D, s.Hkv * s.D

    def bits(shape, std):
        return wl.f32_to_bf16_bits((rng.standard_normal(shape, dtype=np.float32) * np.float32(std)))

    wt = dict(w_norm1=bits((hidden,), 1.0), w_qkv=bits((qd + 2 * kvd, hidden), hidden ** -0.5), w_o=bits((hidden, qd), qd ** -0.5),
              w_norm2=bits((hidden,), 1.0), w_gate=bits((inter, hidden), hidden ** -0.5), w_up=bits((inter, hidden), hidden ** -0.5),
              w_down=bits((hidden, inter), inter ** -0.5))
    x = bits((n_tokens, hidden), 1.0)
    b = wl.make_batch("layer_sample", s, [0], [n_tokens], seed=8, identity_tables=True)
    pool, tm = b.fresh_pool(), b.table_matrix()

    def attention(q, k, v):
        return oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, 1.0 / math.sqrt(s.D), tm, b.ctx_len, b.q_len, q, k, v)

    t0 = time.perf_counter()
    OL.layer_step(attention, x, wt, OL.positions(b.ctx_len, b.q_len), s.Hq, s.Hkv, s.D)
    t = time.perf_counter() - t0
    return {"value": n_tokens / t, "unit": UNIT, "cores": oracle.default_threads(), "kind": "oracle",
            "sample": f"one fresh chunk of {n_tokens} tokens through the whole layer oracle (fp64), {t:.1f} s"}


def run_layer(args, world, rank, local, barrier):
    """The decoder layer around the attention step (ts_layer_step) on config3's batch, with seeded
    random weights of the 8B-shaped layer. Timed like run_static; the projection GEMMs are also timed
    by themselves (ts_gemm_bf16 on the same shapes) for the dominant kernel's roofline."""
    import torch
    from paper_2512_03416_b200 import binding as B
    from paper_2512_03416_b200.harness import LoadedBatch
    from paper_2512_03416_b200.layer import DecoderLayer

    batch = wl.config3(seed=rank_seed(2, rank))
    lb = LoadedBatch(batch, device=local, nan_fill=False)
    s = batch.shape
    hidden, inter = LAYER_8B["hidden"], LAYER_8B["intermediate"]
    qd, kvd = s.Hq * s.D, s.Hkv * s.D
    gen = torch.Generator(device="cuda").manual_seed(rank_seed(71, rank))

    def weight(rows, cols, std):
        return (torch.randn(rows, cols, generator=gen, device="cuda") * std).to(torch.bfloat16).view(torch.int16)

    def gain():
        return (1.0 + 0.05 * torch.randn(hidden, generator=gen, device="cuda")).to(torch.bfloat16).view(torch.int16)

    w = dict(w_norm1=gain(), w_qkv=weight(qd + 2 * kvd, hidden, hidden ** -0.5),
             w_o=weight(hidden, qd, qd ** -0.5), w_norm2=gain(),
             w_gate=weight(inter, hidden, hidden ** -0.5), w_up=weight(inter, hidden, hidden ** -0.5),
             w_down=weight(hidden, inter, inter ** -0.5))
    layer = DecoderLayer(lb.dec, w["w_norm1"], w["w_qkv"], w["w_o"], w["w_norm2"], w["w_gate"], w["w_up"], w["w_down"],
                         max_position=LAYER_8B["max_position"])
    del w["w_gate"], w["w_up"]
    N = batch.n_tokens
    x_in = (torch.randn(N, hidden, generator=gen, device="cuda")).to(torch.bfloat16).view(torch.int16)
    x_out = torch.empty_like(x_in)
    st, _keep = layer.make_step(lb.slots, batch.q_len.tolist(), batch.ctx_len.tolist(), keep_len=True)
    K, W = args.steps, max(args.warmup, 3)
    for _ in range(W):
        layer.step_prepared(st, x_in, x_out)
    barrier()
    v0 = lb.dec.velocity()
    sampler = ClockSampler(local)
    sampler.start()
    events = [torch.cuda.Event(enable_timing=True)]
    barrier()
    t_host = time.perf_counter()
    events[0].record()
    n_blocks = 0
    while True:
        for _ in range(K):
            layer.step_prepared(st, x_in, x_out)
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        events.append(ev)
        n_blocks += 1
        ev.synchronize()
        if time.perf_counter() - t_host >= MIN_TIMED_S or n_blocks >= MAX_BLOCKS:
            break
    barrier()
    clocks = sampler.stop()
    block_ms = [events[i].elapsed_time(events[i + 1]) for i in range(n_blocks)]
    ms_step = reduce_max(float(np.median(block_ms)), world, "cuda") / K
    region_s = events[0].elapsed_time(events[-1]) * 1e-3
    attn_launches = int(lb.dec.velocity()["kernel_launches"] - v0["kernel_launches"]) // n_blocks
    launches = attn_launches + 6 * K                     # two RMSNorm and four GEMM launches per step besides attention's
    if lb.dec.device_status() != 0:
        raise SystemExit("the device reported a failure during the timed steps")

    # the four projections by themselves, same shapes, same kernel
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    gemms = {}
    a_buf = torch.randn(N * max(hidden, inter), generator=gen, device="cuda").to(torch.bfloat16).view(torch.int16)
    b_buf = (torch.randn(2 * inter * hidden, generator=gen, device="cuda") * hidden ** -0.5).to(torch.bfloat16).view(torch.int16)
    c_buf = torch.empty(N * 2 * inter, dtype=torch.int16, device="cuda")
    for name, (n_out, k_in) in {"qkv": (qd + 2 * kvd, hidden), "o": (hidden, qd), "gate_up": (2 * inter, hidden),
                                "down": (hidden, inter)}.items():
        tile_m = 128 if name == "qkv" else 0
        call = lambda: B.ts_gemm_bf16(local, N, n_out, k_in, a_buf.data_ptr(), b_buf.data_ptr(), 0, c_buf.data_ptr(), tile_m,
                                      status.data_ptr(), stream)
        for _ in range(3):
            assert call() == B.TS_OK
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 20
        gemms[name] = {"ms": ms, "flops": 2.0 * N * n_out * k_in, "tflops": 2.0 * N * n_out * k_in / ms / 1e9}
    if int(status.item()) != 0:
        raise SystemExit("a projection GEMM reported a failure")

    attn_flops, attn_bytes = batch.algorithmic_work()
    gemm_flops = sum(g["flops"] for g in gemms.values())
    weight_bytes = 2.0 * ((qd + 2 * kvd) * hidden + hidden * qd + 3 * inter * hidden + 2 * hidden)
    act_bytes = 2.0 * N * (2 * hidden + 2 * hidden + 2 * (qd + 2 * kvd) + 2 * qd + 2 * hidden + 2 * inter + 2 * hidden)
    flops, byts = attn_flops + gemm_flops, attn_bytes + weight_bytes + act_bytes

    # end to end: the layer's input starts in pinned host memory and its output returns there
    hx = x_in.cpu().pin_memory()
    ho = torch.empty_like(hx).pin_memory()
    t0 = time.perf_counter()
    for _ in range(3):
        x_in.copy_(hx, non_blocking=True); layer.step_prepared(st, x_in, x_out); ho.copy_(x_out, non_blocking=True)
    torch.cuda.synchronize()
    est = (time.perf_counter() - t0) / 3
    Ke = int(min(max(K, math.ceil(MIN_TIMED_S / max(est, 1e-5))), 2000))
    barrier()
    t0 = time.perf_counter()
    for _ in range(Ke):
        x_in.copy_(hx, non_blocking=True)
        layer.step_prepared(st, x_in, x_out)
        ho.copy_(x_out, non_blocking=True)
    torch.cuda.synchronize()
    e2e_s = reduce_max(time.perf_counter() - t0, world, "cuda")
    e2e = {"value": aggregate_value(N, world, e2e_s / Ke), "unit": UNIT, "h2d_bytes_per_step": int(hx.numel() * 2),
           "d2h_bytes_per_step": int(ho.numel() * 2), "steps": Ke, "ms_per_step": e2e_s / Ke * 1e3}
    layer.close()
    lb.dec.close()
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = layer_cpu_baseline(s, hidden, inter)
    peaks, peak_kind = load_peaks()
    dom = max(gemms.items(), key=lambda kv: kv[1]["ms"])
    roof = {"bound": "tensor", "achieved": dom[1]["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
            "frac": dom[1]["tflops"] / peaks["bf16_tflops"], "frac_nominal": dom[1]["tflops"] / 2250.0, "traffic": None,
            "kernel": f"gemm_kernel ({dom[0]} projection, {N} x {int(dom[1]['flops'] / 2 / N / (hidden if dom[0] != 'down' else inter))} x {hidden if dom[0] != 'down' else inter})",
            "kernel_ms": dom[1]["ms"], "kernel_ms_source": "events around 20 launches of the kernel alone on the same shape",
            "peak_source": f"of {peak_kind}",
            "projections": {k: {"ms": g["ms"], "TFLOPs": g["tflops"], "frac": g["tflops"] / peaks["bf16_tflops"]} for k, g in gemms.items()}}
    t_hbm, t_tc = byts / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    step_roof = {"t_roof_us": max(t_hbm, t_tc) * 1e6, "t_hbm_us": t_hbm * 1e6, "t_tensor_us": t_tc * 1e6,
                 "frac": max(t_hbm, t_tc) / (ms_step * 1e-3), "flops": flops, "bytes": byts,
                 "frac_nominal": max(byts / 8e12, flops / 2.25e15) / (ms_step * 1e-3)}
    cfg = {"decode_rows": batch.decode_tokens, "prefill_tokens": batch.prefill_tokens, "hidden": hidden, "intermediate": inter,
           "l2": "weights (435 MB) and the decode rows' K/V (0.77 GB) are larger than L2",
           "timing": f"median of {n_blocks} blocks of {K} steps, CUDA events around each block, timed region {region_s:.2f} s"}
    return dict(batch=batch, ms_step=ms_step, tokens=N, prefill_tokens=batch.prefill_tokens, decode_tokens=batch.decode_tokens,
                launches=launches, clocks=clocks, e2e=e2e, cfg=cfg, steps=K, warmup=W, roofline=roof, step_roofline=step_roof,
                cpu_baseline=cpu, extra={"timed_blocks": n_blocks, "timed_region_s": region_s})


def run_replay(args, world, rank, local, barrier, workload=None, light=False, n_steps=None):
    """config5: the 200-step bursty replay. Every step is issued once, in order (the state evolves);
    warm-up is a full untimed replay on a fresh instance. `light`: no end-to-end leg."""
    import torch
    from paper_2512_03416_b200.replay import ReplayRunner, ttft_report

    workload = workload or args.workload
    K = n_steps or min(args.steps, 200)
    seed = rank_seed(5, rank)

    def fresh(keep_host=False):
        return ReplayRunner(wl.TraceReplay(seed=seed, n_steps=K, **REPLAY_TRACE[workload]), seed=seed + 45,
                            device=local, keep_host=keep_host)

    warm = fresh()
    warm.run(timed=False)                              # warm-up: every launch shape once
    warm.dec.close()
    del warm
    run = fresh()
    run.start()                                        # requests in flight at step 0: context resident before timing
    s = run.shape
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    step_ms = run.run(timed=True)
    e1.record()
    barrier()
    clocks = sampler.stop()
    total_ms = reduce_max(e0.elapsed_time(e1), world, "cuda")
    status = run.dec.device_status()                  # a bounded wait that ran out would make the timing meaningless
    if status != 0:
        raise SystemExit(f"the device reported status {status} during the replay")
    launches = int(run.dec.velocity()["kernel_launches"])
    tokens = sum(ps.n_tokens for ps in run.steps)
    pf_tok = sum(ps.prefill_tokens for ps in run.steps)
    dec_tok = sum(ps.decode_tokens for ps in run.steps)
    work = [run.step_work(ps) for ps in run.steps]
    flops, byts = sum(w[0] for w in work), sum(w[1] for w in work)
    peaks, _ = load_peaks()
    t_roof = [max(w[1] / (peaks["hbm_gbs"] * 1e9), w[0] / (peaks["bf16_tflops"] * 1e12)) for w in work]
    run.dec.close()

    # per-kernel times: one more replay with the library's events switched on
    prof_run = fresh()
    prof_run.dec.profile_enable(True)
    prof_run.run(timed=False)
    prof = prof_run.dec.profile_read()
    prof_run.dec.close()
    # algorithmic work per kind of launch: a step with prefill tokens and decode rows runs both in one
    # launch (G <= 8 here); a step without prefill tokens runs decode_kernel
    dec_bytes = pf_flops = mixed_bytes = mixed_flops = 0.0
    for ps, w in zip(run.steps, work):
        n_dec = sum(1 for t in ps.q_len if t == 1)
        if ps.prefill_tokens > 0 and n_dec > 0:
            mixed_bytes += w[1]                      # the mixed launch also appends the new K/V
            mixed_flops += w[0]
        elif ps.prefill_tokens > 0:
            pf_flops += w[0]
        else:
            dec_bytes += float(sum((c + 1) * s.kv_bytes_per_token + 2 * s.Hq * s.D * 2 for c in ps.ctx_len))
    n_rec = max(1, prof["steps"])
    parts = {"dec_bytes": dec_bytes / n_rec, "pf_flops": pf_flops / n_rec, "mixed_bytes": mixed_bytes / n_rec,
             "mixed_flops": mixed_flops / n_rec}

    e2e = None
    if not light:
        # end to end: every step's inputs start in pinned host memory and its output returns there
        e2e_run = fresh(keep_host=True)
        pinned = []
        for ps in e2e_run.steps:
            if ps.host is None:
                pinned.append(None)
                continue
            hq, hk, hv = (torch.from_numpy(a.view(np.int16)).pin_memory() for a in ps.host)
            pinned.append((hq, hk, hv, torch.empty_like(hq).pin_memory()))
        e2e_run.start()
        barrier()
        t0 = time.perf_counter()
        h2d = d2h = 0
        for ps, pin in zip(e2e_run.steps, pinned):
            e2e_run.begin_step(ps)
            if pin is not None:
                hq, hk, hv, ho = pin
                e2e_run.dec.mixed_step_host(ps.slots.tolist(), ps.q_len, ps.ctx_len, hq, hk, hv, ho, wait=False)
                h2d += (hq.numel() + hk.numel() + hv.numel()) * 2
                d2h += ho.numel() * 2
            e2e_run.end_step(ps)
        e2e_run.dec.host_fence()
        torch.cuda.synchronize()
        e2e_s = reduce_max(time.perf_counter() - t0, world, "cuda")
        if e2e_run.dec.device_status() != 0:
            raise SystemExit("the device reported a failure during the end-to-end replay")
        e2e_run.dec.close()
        e2e = {"value": aggregate_value(tokens, world, e2e_s), "unit": UNIT, "h2d_bytes_per_step": int(h2d / K),
               "d2h_bytes_per_step": int(d2h / K), "steps": K, "ms_per_step": e2e_s / K * 1e3}
    order = np.argsort(step_ms)
    heavy = [i for i in range(K) if run.steps[i].prefill_tokens >= 4096]
    extra = {"step_ms": {"median": float(np.median(step_ms)), "p90": float(np.percentile(step_ms, 90)),
                         "max": float(np.max(step_ms)), "min": float(step_ms[order[0]])},
             "sum_t_roof_over_sum_t": float(sum(t_roof) / (sum(step_ms) * 1e-3)),
             "steps_with_prefill": int(sum(1 for ps in run.steps if ps.prefill_tokens > 0)),
             # time to first token of the absorbed requests: on the trace's own clock (every step one
             # tick), and with every step lasting its measured attention time x the model's layers
             # (attention alone understates a layer, so this is a lower bound on a real TTFT)
             "ttft": {"tick_s": run.trace.step_s, "trace_clock": ttft_report(run.trace, run.steps),
                      "measured_attention_x_layers": ttft_report(run.trace, run.steps,
                                                                 [m * 1e-3 * N_LAYERS_70B for m in step_ms])},
             "heavy_steps": {"count": len(heavy),
                             "frac": float(sum(t_roof[i] for i in heavy) / (sum(step_ms[i] for i in heavy) * 1e-3)) if heavy else None}}
    cfg = {"decode_rows": "<=%d per step" % max(ps.decode_tokens for ps in run.steps), "prefill_tokens": pf_tok,
           "kv_tokens": None, "l2": "every step reads its own rows' K/V once; KV working set > L2 on all but the first steps"}
    return dict(batch=None, ms_step=total_ms / K, tokens=tokens / K, prefill_tokens=pf_tok / K, decode_tokens=dec_tok / K,
                launches=launches, clocks=clocks, prof=prof, flops=flops / K, byts=byts / K,
                parts=parts, e2e=e2e, cfg=cfg, steps=K, warmup=K, extra=extra)


def run_ours(args):
    import torch
    import torch.distributed as dist

    world, rank, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks, peak_kind = load_peaks()

    def measure(workload, light, n_steps=None):
        if workload == "layer_8b":
            r = run_layer(args, world, rank, local, barrier)
            return r, r["roofline"], r["step_roofline"]
        if workload in REPLAY_TRACE:
            r = run_replay(args, world, rank, local, barrier, workload, light, n_steps)
        else:
            r = run_static(args, world, rank, local, barrier, workload, light)
        lps = r["launches"] / max(1, r["steps"]) if r["batch"] is not None else None
        roof, step_roof = rooflines(peaks, peak_kind, r["flops"], r["byts"], r["ms_step"], r["prof"], r["parts"],
                                    KERNEL_TRAFFIC_BYTES.get(workload), launches_per_step=lps)
        return r, roof, step_roof

    r, roofline, step_roofline = measure(args.workload, light=False)
    # The default line also carries short passes of the other target workloads (no end-to-end and
    # no oracle leg for them): the decode-only batch, the chunked continuation and the 200-step
    # 70B-shaped replay.
    others = {}
    if args.workload == "config3" and not args.headline_only and world == 1:
        for w in ("config2", "config4", "config5"):
            ro, roofo, stepo = measure(w, light=True, n_steps=200 if w in REPLAY_TRACE else None)
            others[w] = {"description": WORKLOADS[w][1], "ms_per_step": ro["ms_step"], "steps": ro["steps"],
                         "tokens_per_s": aggregate_value(ro["tokens"], world, ro["ms_step"] * 1e-3),
                         "step_roofline": {k: stepo[k] for k in ("frac", "frac_nominal", "t_roof_us", "t_hbm_us", "t_tensor_us")},
                         "roofline": {k: roofo[k] for k in ("kernel", "bound", "achieved", "peak", "unit", "frac",
                                                             "frac_nominal", "kernel_ms", "kernel_ms_source", "peak_source")},
                         "clocks": ro["clocks"], "gpu_launches": ro["launches"]}
            for k in ("heavy_steps", "sum_t_roof_over_sum_t", "step_ms", "timed_blocks", "timed_region_s"):
                if k in ro["extra"]:
                    others[w][k] = ro["extra"][k]
    cpu_baseline = None
    if args.workload == "layer_8b":
        cpu_baseline = r.get("cpu_baseline")
    elif rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = cpu_baseline_leg(r["batch"] if r["batch"] is not None else make_static_batch(args.workload, 0))
    if rank == 0:
        shape = wl.LLAMA70B if args.workload in REPLAY_TRACE or args.workload.endswith("70b") else wl.LLAMA8B
        cfg = {"workload": args.workload, "description": WORKLOADS[args.workload][1], "n_q_heads": shape.Hq,
               "n_kv_heads": shape.Hkv, "head_dim": shape.D, "page_size": shape.P,
               "parallelism": f"replicas x{world}"}
        cfg.update(r["cfg"])
        line = {"metric": METRIC, "value": aggregate_value(r["tokens"], world, r["ms_step"] * 1e-3), "unit": UNIT,
                "n_gpus": world, "steps": r["steps"], "warmup": r["warmup"], "ms_per_step": r["ms_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic", "config": cfg, "clocks": r["clocks"], "e2e": r["e2e"],
                "gpu_launches": r["launches"], "roofline": roofline, "step_roofline": step_roofline,
                "cpu_baseline": cpu_baseline,
                "prefill_tokens_per_s": aggregate_value(r["prefill_tokens"], world, r["ms_step"] * 1e-3),
                "decode_tokens_per_s": aggregate_value(r["decode_tokens"], world, r["ms_step"] * 1e-3)}
        line.update(r["extra"])
        if others:
            line["workloads"] = others
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config3", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true",
                    help="default workload only: skip the short passes of config2, config4 and config5")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
