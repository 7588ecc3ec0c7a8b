"""Drives a Decoder through a TraceReplay (bursty arrivals on a Convertible Decoder).

Every replay step becomes one ts_mixed_step: the live decode requests take one token each and at
most one prefill task is absorbed, chunk by chunk (Sec. 3.4, Sec. 4.4). Requests are added, their
pages grown and released through the library's own allocator, so block tables and page
scattering arise the way they do in serving. No oracle code is imported here.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np
import torch

from . import workloads as wl
from . import binding as B
from .decoder import Decoder, TsError
from .harness import to_dev


@dataclass
class PreparedStep:
    index: int
    adds: list
    preload: list
    frees: List[int]
    req_ids: List[int]
    q_len: List[int]
    ctx_len: List[int]
    q: Optional[torch.Tensor] = None       # device tensors of the step (None for an empty step)
    k_new: Optional[torch.Tensor] = None
    v_new: Optional[torch.Tensor] = None
    out: Optional[torch.Tensor] = None
    host: Optional[tuple] = None            # (q, k_new, v_new) bit patterns on the host, when kept
    slots: Optional[np.ndarray] = None      # int32 slots of the rows, known once the requests are admitted
    q_len_np: Optional[np.ndarray] = None
    ctx_len_np: Optional[np.ndarray] = None

    @property
    def n_tokens(self) -> int:
        return int(sum(self.q_len))

    @property
    def prefill_tokens(self) -> int:
        return int(sum(t for t in self.q_len if t > 1))

    @property
    def decode_tokens(self) -> int:
        return int(sum(1 for t in self.q_len if t == 1))


def ttft_report(trace: wl.TraceReplay, steps, step_seconds=None, slos=(0.25, 0.4, 2.0)) -> dict:
    """Time to first token of every request whose prefill the replay absorbed (Sec. 2.2: the time
    from a request's arrival until its first output token), against TTFT SLOs (Sec. 6.1 uses
    250, 400 and 2000 ms by prompt length).

    ``steps``: the replay's steps in order (anything with ``index`` and rows of
    (req_id, q_len, ctx_len), e.g. ReplayStep or PreparedStep with req_ids/q_len/ctx_len).
    A request's first token exists when the step that holds the last chunk of its prompt ends.
    Step i is issued at i * step_s of the trace's virtual clock, or when its predecessor has
    ended if that is later, and lasts ``step_seconds[i]`` (default: step_s, the virtual clock
    alone). TTFT = that end time - arrival: queueing (arrival until the step that takes the
    first chunk is issued) plus the chunk steps. Requests in flight at step 0 are left out;
    requests whose prefill the replay does not finish are counted as ``unfinished``.
    """
    prompt = {r.req_id: r for r in trace.requests}
    first_chunk, last_chunk = {}, {}
    end, ends, starts = 0.0, [], []
    for i, st in enumerate(steps):
        rows = st.rows if hasattr(st, "rows") else zip(st.req_ids, st.q_len, st.ctx_len)
        start = max(i * trace.step_s, end)
        end = start + (trace.step_s if step_seconds is None else float(step_seconds[i]))
        starts.append(start)
        ends.append(end)
        for rid, ql, ctx in rows:
            r = prompt.get(rid)
            if r is None or ctx >= r.prompt_len:
                continue                              # warm request or decode row
            first_chunk.setdefault(rid, i)
            if ctx + ql == r.prompt_len:
                last_chunk[rid] = i
    ttft, queue_s, chunk_steps = [], [], []
    for rid, i in last_chunk.items():
        r = prompt[rid]
        ttft.append(ends[i] - r.arrival_s)
        queue_s.append(starts[first_chunk[rid]] - r.arrival_s)
        chunk_steps.append(i - first_chunk[rid] + 1)
    t = np.asarray(ttft, dtype=np.float64)
    out = {"requests": len(ttft), "unfinished": len(trace.requests) - len(ttft)}
    if len(ttft):
        out.update({"ttft_mean_s": float(t.mean()), "ttft_p50_s": float(np.percentile(t, 50)),
                    "ttft_p99_s": float(np.percentile(t, 99)), "ttft_max_s": float(t.max()),
                    "queue_mean_s": float(np.mean(queue_s)), "chunk_steps_mean": float(np.mean(chunk_steps)),
                    "chunk_steps_max": int(max(chunk_steps)),
                    "attainment": {f"{int(round(x * 1e3))}ms": float((t <= x).mean()) for x in slos}})
    return out


class ReplayRunner:
    def __init__(self, trace: wl.TraceReplay, seed: int = 50, device: int = 0, keep_host: bool = False,
                 pool_pages: Optional[int] = None, nan_fill: bool = False, decode_split_tokens: int = 0):
        self.trace = trace
        self.shape = trace.shape
        self.device = torch.device("cuda", device)
        self.keep_host = keep_host
        s = self.shape
        self.bank = wl.ValueBank(seed, 1.0 / np.sqrt(s.D), log2_size=24)
        self.steps: List[PreparedStep] = []
        live_tokens, peak = {}, 0
        warm_ctx: Dict[int, tuple] = {}
        with torch.cuda.device(self.device):
            for st in trace.steps():
                for r, n in st.preload:                    # context of the requests in flight at step 0
                    k = self.bank.take(n * s.Hkv * s.D).reshape(n, s.Hkv, s.D)
                    v = self.bank.take(n * s.Hkv * s.D).reshape(n, s.Hkv, s.D)
                    warm_ctx[r.req_id] = (k, v)
                    live_tokens[r.req_id] = n
                ps = PreparedStep(st.index, st.adds, st.preload, st.frees, [r[0] for r in st.rows],
                                  [r[1] for r in st.rows], [r[2] for r in st.rows])
                ps.q_len_np = np.asarray(ps.q_len, dtype=np.int32)
                ps.ctx_len_np = np.asarray(ps.ctx_len, dtype=np.int32)
                n = ps.n_tokens
                if n:
                    q, k, v = wl.replay_values(s, seed, n, self.bank)
                    ps.q, ps.k_new, ps.v_new = to_dev(q, self.device), to_dev(k, self.device), to_dev(v, self.device)
                    ps.out = torch.empty((n, s.Hq, s.D), dtype=torch.int16, device=self.device)
                    if keep_host:
                        ps.host = (q, k, v)
                for rid, ql, ctx in st.rows:
                    live_tokens[rid] = ctx + ql
                pages_now = sum((t + s.P - 1) // s.P + 1 for t in live_tokens.values())
                peak = max(peak, pages_now)
                for rid in st.frees:
                    live_tokens.pop(rid, None)
                self.steps.append(ps)
        self.warm_ctx = warm_ctx
        n_pages = pool_pages or int(1.25 * peak) + 64
        width = (trace.max_context + s.P - 1) // s.P + 1
        self.dec = Decoder(s.Hq, s.Hkv, s.D, n_pages, trace.max_decodes + 8, width, chunk_size=trace.chunk_size,
                           device=device, alloc_shuffle_seed=seed, nan_fill=nan_fill,
                           decode_split_tokens=decode_split_tokens)
        self.slot_of: Dict[int, int] = {}
        self._started = False

    def start(self) -> None:
        """Set-up that precedes the first step: admit the requests that are in flight at step 0 and
        put their cached context into the pool (ts_kv_append). Not part of any step."""
        if self._started:
            return
        self._started = True
        ps = self.steps[0]
        for r, cached in ps.preload:
            slot = self.slot_of[r.req_id] = self.dec.request_add(r.req_id, r.prompt_len, r.output_len)
            k, v = self.warm_ctx[r.req_id]
            self.dec.alloc_pages(slot, cached, for_prefill=True)
            with torch.cuda.device(self.device):
                self.dec.kv_append([slot], [cached], [0], to_dev(k, self.device), to_dev(v, self.device))
        torch.cuda.synchronize(self.device)

    # -------------------------------------------------------------------------------- one step
    def begin_step(self, ps: PreparedStep) -> None:
        """Host bookkeeping before the step: admit new requests, grow the rows' tables."""
        self.start()
        for r in ps.adds:
            if r.req_id not in self.slot_of:          # warm requests were admitted by start()
                self.slot_of[r.req_id] = self.dec.request_add(r.req_id, r.prompt_len, r.output_len)
        if ps.req_ids:
            slot_of = self.slot_of
            ps.slots = np.fromiter((slot_of[r] for r in ps.req_ids), dtype=np.int32, count=len(ps.req_ids))
            st, keep = B.make_step_np(ps.slots, ps.q_len_np, ps.ctx_len_np)
            rc = B.ts_alloc_step(self.dec.ctx, st)
            if rc != B.TS_OK:
                raise TsError(rc, "ts_alloc_step")

    def launch(self, ps: PreparedStep) -> None:
        if not ps.req_ids:
            return
        self.dec.step_np(ps.slots, ps.q_len_np, ps.ctx_len_np, ps.q, ps.k_new, ps.v_new, ps.out, alloc=False)

    def end_step(self, ps: PreparedStep) -> None:
        for rid in ps.frees:
            self.dec.request_free(self.slot_of.pop(rid))

    def tables(self, ps: PreparedStep) -> List[np.ndarray]:
        return [self.dec.block_table(self.slot_of[r])[0] for r in ps.req_ids]

    def step_work(self, ps: PreparedStep):
        """(flops, bytes) of the step, same accounting as StepBatch.algorithmic_work."""
        s = self.shape
        keys, kv_tokens = 0.0, 0
        for c, t in zip(ps.ctx_len, ps.q_len):
            keys += t * c + t * (t + 1) / 2
            kv_tokens += c + t
        n = ps.n_tokens
        return (4.0 * s.D * s.Hq * keys,
                float(kv_tokens * s.kv_bytes_per_token + n * s.kv_bytes_per_token + 2 * n * s.Hq * s.D * 2))

    def run(self, timed: bool = True):
        """Runs every step in order; returns per-step milliseconds (CUDA events) when timed."""
        ms = []
        self.start()
        with torch.cuda.device(self.device):
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in self.steps] if timed else None
            for i, ps in enumerate(self.steps):
                self.begin_step(ps)
                if timed:
                    evs[i][0].record()
                self.launch(ps)
                if timed:
                    evs[i][1].record()
                self.end_step(ps)
            torch.cuda.synchronize(self.device)
            if timed:
                ms = [a.elapsed_time(b) for a, b in evs]
        return ms
