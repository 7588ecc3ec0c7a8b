"""Chunk-size profiler for a Convertible Decoder (Sec. 4.4, Eq. 5, Eq. 6).

The paper fixes the one parameter of its restricted chunked prefill by measurement: at a given
decode batch the prefill chunk is grown step by step and the iteration time recorded until the
TPOT SLO is violated; the largest chunk size before that is used, Eq. 5 turns it into the
decoder's prefill Token Velocity and Eq. 6 into the memory to hold back for absorbed prefills.
This module takes that measurement on ts_mixed_step itself (CUDA events around the step) and
hands the points to the library's ts_pick_chunk_size / ts_convertible_prefill_velocity /
ts_reserved_pages. With `layer_dims=(hidden, intermediate)` the measured step is the whole
decoder layer (ts_layer_step: projections, rotary embedding, attention, MLP, random weights of that
size) and the iteration time its step time times `n_layers`: a TPOT but for the embedding and the
output head. Without it the step is the attention layer alone (ts_mixed_step), which understates a
full layer and so gives an upper bound on the chunk size.

    python -m paper_2512_03416_b200.profiler --shape 8b --decode-rows 64 --layers 32 --hidden 4096 --intermediate 14336
"""
from __future__ import annotations

import argparse
import json
from typing import Dict, List, Sequence

import numpy as np

from . import binding as B
from . import workloads as wl


def _random_layer(lb, shape: wl.Shape, hidden: int, inter: int, max_position: int, seed: int):
    """A DecoderLayer with seeded random weights of the given size (profiling only needs their shape)."""
    import torch

    from .layer import DecoderLayer

    gen = torch.Generator(device=lb.device).manual_seed(seed)
    qd, kvd = shape.Hq * shape.D, shape.Hkv * shape.D

    def w(rows, cols):
        return (torch.randn(rows, cols, generator=gen, device=lb.device) * cols ** -0.5).to(torch.bfloat16).view(torch.int16)

    def gain():
        return torch.ones(hidden, device=lb.device).to(torch.bfloat16).view(torch.int16)

    return DecoderLayer(lb.dec, gain(), w(qd + 2 * kvd, hidden), w(hidden, qd), gain(), w(inter, hidden), w(inter, hidden),
                        w(hidden, inter), max_position=max_position)


def measure_step_seconds(shape: wl.Shape, decode_ctx: Sequence[int], prefill_tokens: int, steps: int = 20,
                         warmup: int = 3, seed: int = 0, device: int = 0, layer_dims=None) -> float:
    """Seconds of one step over the decode rows plus one fresh prefill chunk: ts_mixed_step, or
    ts_layer_step on a layer of `layer_dims = (hidden, intermediate)`."""
    import torch

    from .harness import LoadedBatch

    ctx = np.concatenate([np.asarray(decode_ctx, np.int32), [0]]).astype(np.int32)
    ql = np.concatenate([np.ones(len(decode_ctx), np.int32), [prefill_tokens]]).astype(np.int32)
    batch = wl.make_batch(f"profile_{prefill_tokens}", shape, ctx, ql, seed + 100,
                          chunk_size=prefill_tokens + len(decode_ctx))
    lb = LoadedBatch(batch, device=device, nan_fill=False)
    layer = None
    try:
        step = lb.step_repeatable
        if layer_dims is not None:
            hidden, inter = layer_dims
            layer = _random_layer(lb, shape, hidden, inter, int(ctx.max()) + prefill_tokens + 16, seed + 7)
            x_in = torch.randn(batch.n_tokens, hidden, device=lb.device).to(torch.bfloat16).view(torch.int16)
            x_out = torch.empty_like(x_in)
            st, _keep = layer.make_step(lb.slots, batch.q_len.tolist(), batch.ctx_len.tolist(), keep_len=True)
            step = lambda: layer.step_prepared(st, x_in, x_out)
        for _ in range(max(warmup, 1)):
            step()
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize(device)
        if lb.dec.device_status() != 0:
            raise RuntimeError("the device reported an error during profiling")
        return e0.elapsed_time(e1) * 1e-3 / steps
    finally:
        if layer is not None:
            layer.close()
        lb.dec.close()


def profile_chunk_size(shape: wl.Shape, decode_ctx: Sequence[int], candidates: Sequence[int], n_layers: int,
                       tpot_slo_s: float, ttft_slo_s: float, steps: int = 20, seed: int = 0,
                       device: int = 0, layer_dims=None) -> Dict:
    """Grows the prefill chunk over `candidates` (ascending) until the iteration time passes the
    TPOT SLO (Sec. 4.4) and derives Eq. 5 and Eq. 6 from the chunk size found."""
    sizes: List[int] = []
    seconds: List[float] = []
    for t in candidates:
        sec = measure_step_seconds(shape, decode_ctx, int(t), steps=steps, seed=seed, device=device,
                                   layer_dims=layer_dims) * n_layers
        sizes.append(int(t))
        seconds.append(sec)
        if sec > tpot_slo_s:               # the paper's sweep ends at the first violation
            break
    batch = len(decode_ctx)
    chunk = B.ts_pick_chunk_size(sizes, seconds, batch, tpot_slo_s)
    if chunk < 0:
        raise ValueError(f"ts_pick_chunk_size: {B.ts_strerror(chunk)}")
    v = B.ts_convertible_prefill_velocity(chunk, float(batch), tpot_slo_s) if chunk > 0 else 0.0
    return {"prefill_tokens": sizes, "iteration_seconds": seconds, "decode_batch_size": batch, "n_layers": n_layers,
            "step": "ts_layer_step" if layer_dims is not None else "ts_mixed_step",
            "tpot_slo_s": tpot_slo_s, "ttft_slo_s": ttft_slo_s, "chunk_size": chunk,
            "prefill_velocity_tokens_per_s": v,
            "reserved_pages": B.ts_reserved_pages(v, ttft_slo_s, shape.P),
            "reserved_bytes": B.ts_reserved_memory(v, float(shape.kv_bytes_per_token), ttft_slo_s)}


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--shape", default="8b", choices=["8b", "70b"])
    ap.add_argument("--decode-rows", type=int, default=64)
    ap.add_argument("--median-ctx", type=int, default=2048)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--tpot-ms", type=float, default=100.0)        # the paper's TPOT SLO
    ap.add_argument("--ttft-ms", type=float, default=250.0)        # its tightest TTFT SLO
    ap.add_argument("--candidates", type=int, nargs="*",
                    default=[256, 512, 1024, 2048, 3072, 4096, 6144, 8192, 12288, 16384])
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--hidden", type=int, default=0, help="with --intermediate: profile the whole layer (ts_layer_step)")
    ap.add_argument("--intermediate", type=int, default=0)
    args = ap.parse_args()
    shape = wl.LLAMA8B if args.shape == "8b" else wl.LLAMA70B
    rng = np.random.Generator(np.random.Philox(9))
    ctx = np.clip(np.round(args.median_ctx * np.exp(rng.standard_normal(args.decode_rows))), 128,
                  4 * args.median_ctx).astype(np.int32)
    out = profile_chunk_size(shape, ctx, args.candidates, args.layers, args.tpot_ms * 1e-3, args.ttft_ms * 1e-3,
                             steps=args.steps,
                             layer_dims=(args.hidden, args.intermediate) if args.hidden and args.intermediate else None)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
