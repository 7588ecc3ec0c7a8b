#!/usr/bin/env python
"""Benchmark of the mixed paged-attention step (ts_mixed_step) on synthetic bursty batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config3] [--impl ours|reference]

One "step" is one pass of the whole path (table sync, KV append, attention over decode rows and
prefill chunks, split combine) over one batch. Prints ONE JSON line on rank 0.
N > 1 runs N independent replicas (the path has no exchange step): weak scaling.
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

WORKLOADS = {
    "config2": (wl.config2, "decode-only batch, 8B-shaped layer (64 decode rows, ctx lognormal median 2048)"),
    "config3": (wl.config3, "convertible-decoder burst, 8B-shaped layer (64 decode rows + one fresh 2048-token prefill chunk)"),
    "config4": (wl.config4, "chunked-prefill continuation, 8B-shaped layer (128 decode rows + 4 chunks of 512 tokens)"),
}


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
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
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

    def run(self, sel) -> float:
        b, s = self.batch, self.batch.shape
        t0 = time.perf_counter()
        self.oracle.attention(self.pool, s.Hq, s.Hkv, s.D, s.P, 1.0 / math.sqrt(s.D), self.tm, b.ctx_len,
                              b.q_len, b.q, sel=sel, threads=self.cores)
        return time.perf_counter() - t0

    def stride_for(self, seconds: float) -> int:
        """Sampling stride whose oracle time is about `seconds`, from a quick calibration."""
        b = self.batch
        probe = oracle_sample(b, max(64, b.n_tokens // 16))
        t = self.run(probe)
        rate = sample_flops(b, probe) / max(t, 1e-6)
        total = b.algorithmic_work()[0]
        return int(min(max(1, math.ceil(total / (rate * seconds))), max(1, b.n_tokens)))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    make, desc = WORKLOADS[args.workload]
    batch = make()
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
    sample = f"every {stride}th decode row and every {stride}th prefill token ({len(sel)} of {batch.n_tokens} tokens) per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": {"workload": args.workload, "description": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": leg.cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2512_03416_b200.harness import LoadedBatch

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    make, desc = WORKLOADS[args.workload]
    batch = make(seed=make.__defaults__[0] + 1000 * rank) if rank else make()
    lb = LoadedBatch(batch, device=local, nan_fill=False)
    flops, byts = batch.algorithmic_work()
    peaks, peak_kind = load_peaks()
    K, W = args.steps, max(args.warmup, 3)

    for _ in range(W):
        lb.step_repeatable()
    barrier()
    v0 = lb.dec.velocity()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(K):
        lb.step_repeatable()
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    v1 = lb.dec.velocity()
    launches = int(v1["kernel_launches"] - v0["kernel_launches"])
    if world > 1:
        t = torch.tensor([ms_total], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / K
    tokens = batch.n_tokens
    value = world * tokens / (ms_step * 1e-3)

    # per-kernel device time (separate pass: the extra events perturb the step a little)
    Kp = min(K, 300)
    lb.dec.profile_enable(True)
    for _ in range(Kp):
        lb.step_repeatable()
    prof = lb.dec.profile_read()
    lb.dec.profile_enable(False)
    attn_ms = prof["attention_ms"] / max(1, prof["steps"])
    s = batch.shape
    kv_tokens = int((batch.ctx_len + batch.q_len).sum())
    attn_bytes = kv_tokens * s.kv_bytes_per_token + 2 * tokens * s.Hq * s.D * 2
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    hbm_bound = t_hbm >= t_tc
    if hbm_bound:
        achieved = attn_bytes / (attn_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": None}
    else:
        achieved = flops / (attn_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops"], "traffic": None}
    roofline.update({"kernel": "attention_kernel", "kernel_ms": attn_ms, "peak_source": f"of {peak_kind}",
                     "append_ms": prof["append_ms"] / max(1, prof["steps"]),
                     "combine_ms": prof["combine_ms"] / max(1, prof["steps"])})
    t_roof = max(t_hbm, t_tc)
    step_roofline = {"t_roof_us": t_roof * 1e6, "t_hbm_us": t_hbm * 1e6, "t_tensor_us": t_tc * 1e6,
                     "frac": t_roof / (ms_step * 1e-3), "flops": flops, "bytes": byts,
                     "frac_nominal_8TBs": max(byts / 8e12, flops / 2.25e15) / (ms_step * 1e-3)}

    # end to end: host buffers in, host buffer out, through ts_mixed_step_host
    Ke = min(K, 300)
    hq = torch.from_numpy(batch.q.view(np.int16)).pin_memory()
    hk = torch.from_numpy(batch.k_new.view(np.int16)).pin_memory()
    hv = torch.from_numpy(batch.v_new.view(np.int16)).pin_memory()
    ho = torch.empty_like(hq).pin_memory()
    ql, cl = batch.q_len.tolist(), batch.ctx_len.tolist()
    for _ in range(3):
        lb.dec.mixed_step_host(lb.slots, ql, cl, hq, hk, hv, ho, keep_len=True)
    barrier()
    t0 = time.perf_counter()
    for _ in range(Ke):
        lb.dec.mixed_step_host(lb.slots, ql, cl, hq, hk, hv, ho, keep_len=True)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([e2e_s], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e = {"value": world * tokens / (e2e_s / Ke), "unit": UNIT,
           "h2d_bytes_per_step": int(hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2),
           "d2h_bytes_per_step": int(ho.numel() * 2), "steps": Ke, "ms_per_step": e2e_s / Ke * 1e3}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        leg = OracleLeg(batch)
        stride = leg.stride_for(15.0)
        sel = oracle_sample(batch, stride)
        t = leg.run(sel)
        cpu_baseline = {"value": len(sel) / t, "unit": UNIT, "cores": leg.cores, "kind": "oracle",
                        "sample": f"every {stride}th decode row and every {stride}th prefill token "
                                  f"({len(sel)} of {tokens} tokens), {t:.1f} s"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": args.workload, "description": desc, "n_q_heads": s.Hq,
                           "n_kv_heads": s.Hkv, "head_dim": s.D, "page_size": s.P,
                           "decode_rows": batch.decode_tokens, "prefill_tokens": batch.prefill_tokens,
                           "kv_tokens": kv_tokens, "parallelism": f"replicas x{world}",
                           "l2": "inputs larger than L2 (KV working set %.2f GB)" % (kv_tokens * s.kv_bytes_per_token / 1e9)},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
                "step_roofline": step_roofline, "cpu_baseline": cpu_baseline,
                "prefill_tokens_per_s": world * batch.prefill_tokens / (ms_step * 1e-3),
                "decode_tokens_per_s": world * batch.decode_tokens / (ms_step * 1e-3)}
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
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
