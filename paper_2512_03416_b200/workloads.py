"""Seeded synthetic workloads for the mixed paged-attention step.

This module only *draws inputs*: request lengths, page placements and bf16 values. It holds
none of the attention arithmetic and imports neither the CUDA binding nor the CPU oracle, so
that both can be fed the same bits. bf16 tensors are ``numpy.uint16`` bit patterns.

The batches are shaped like the serving workloads of TokenScale (arXiv 2512.03416): decode
batches with long-tailed context lengths, a Convertible Decoder that absorbs a prefill chunk
next to its decode batch (Sec. 3.4, Sec. 4.4), prompts of at most 8192 tokens (Sec. 6 SLO
classes), bursty arrivals (Sec. 2.3). The production traces the paper replays are not
available; every length is drawn from a stated distribution instead.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

BF16_NAN = 0x7FC0  # quiet NaN, used as the "never written" sentinel of pool slots


# --------------------------------------------------------------------------------------
# bf16 helpers (bit-level; round to nearest even)
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------------------
# shapes and batches
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Shape:
    Hq: int
    Hkv: int
    D: int
    P: int = 16

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.Hkv * self.D * 2

    def pool_elems(self, n_pages: int) -> int:
        return n_pages * 2 * self.Hkv * self.P * self.D


TINY = Shape(4, 2, 64)
LLAMA8B = Shape(32, 8, 128)
LLAMA70B = Shape(64, 8, 128)


@dataclass
class StepBatch:
    """One step's inputs. Row r has ctx_len[r] cached tokens (their K/V in context_k/v,
    concatenated over rows in row order) and q_len[r] new tokens."""
    name: str
    shape: Shape
    n_pages: int
    tables: List[np.ndarray]          # per row: int32 page ids covering ctx_len + q_len tokens
    ctx_len: np.ndarray               # int32 [R]
    q_len: np.ndarray                 # int32 [R]
    q: np.ndarray                     # uint16 [N, Hq, D]
    k_new: np.ndarray                 # uint16 [N, Hkv, D]
    v_new: np.ndarray                 # uint16 [N, Hkv, D]
    context_k: np.ndarray             # uint16 [sum ctx, Hkv, D]
    context_v: np.ndarray             # uint16 [sum ctx, Hkv, D]
    chunk_size: int = 0
    profile: str = "paper"

    @property
    def n_rows(self) -> int:
        return len(self.q_len)

    @property
    def n_tokens(self) -> int:
        return int(self.q_len.sum())

    @property
    def prefill_tokens(self) -> int:
        return int(self.q_len[self.q_len > 1].sum())

    @property
    def decode_tokens(self) -> int:
        return int((self.q_len == 1).sum())

    def table_matrix(self, width: Optional[int] = None) -> np.ndarray:
        """Block tables as one int32 matrix [R, width], unused entries -1."""
        w = max([len(t) for t in self.tables] + [1]) if width is None else width
        m = np.full((self.n_rows, w), -1, dtype=np.int32)
        for r, t in enumerate(self.tables):
            m[r, :len(t)] = t
        return m

    def fresh_pool(self) -> np.ndarray:
        """A pool image in which every slot holds the NaN sentinel."""
        return np.full(self.shape.pool_elems(self.n_pages), BF16_NAN, dtype=np.uint16)

    def algorithmic_work(self):
        """(flops, bytes) of the step: causal half only for the chunks; K/V read once,
        append written once, Q read and O written once."""
        s = self.shape
        keys = 0.0
        kv_tokens = 0
        for c, t in zip(self.ctx_len.tolist(), self.q_len.tolist()):
            keys += t * c + t * (t + 1) / 2
            kv_tokens += c + t
        flops = 4.0 * s.D * s.Hq * keys
        n = self.n_tokens
        byts = kv_tokens * s.kv_bytes_per_token + n * s.kv_bytes_per_token + 2 * n * s.Hq * s.D * 2
        return flops, float(byts)


# --------------------------------------------------------------------------------------
# value generators
# --------------------------------------------------------------------------------------
class ValueBank:
    """Gaussian bf16 values served as windows of one seeded bank, so that multi-GB contexts
    cost one pass of the generator. Windows start at seeded offsets and wrap around."""

    def __init__(self, seed: int, std: float, log2_size: int = 24):
        rng = np.random.Generator(np.random.Philox(seed))
        n = 1 << log2_size
        self.bits = f32_to_bf16_bits(rng.standard_normal(n, dtype=np.float32) * np.float32(std))
        self.n = n
        self.rng = np.random.Generator(np.random.Philox(seed ^ 0x9E3779B97F4A7C15))

    def take(self, count: int) -> np.ndarray:
        if count == 0:
            return np.zeros(0, dtype=np.uint16)
        off = int(self.rng.integers(0, self.n))
        out = np.empty(count, dtype=np.uint16)
        at = 0
        while at < count:                      # wrap around the bank in whole slices
            n = min(count - at, self.n - off)
            out[at:at + n] = self.bits[off:off + n]
            at += n
            off = 0
        return out


def _lognormal_lengths(rng, median: float, sigma: float, lo: int, hi: int, n: int) -> np.ndarray:
    z = rng.standard_normal(n)
    return np.clip(np.round(median * np.exp(sigma * z)), lo, hi).astype(np.int32)


def _deal_pages(rng, need_pages: List[int], n_pages: int) -> List[np.ndarray]:
    """One random permutation of all page ids dealt out to the rows in order."""
    perm = rng.permutation(n_pages).astype(np.int32)
    assert sum(need_pages) <= n_pages
    out, at = [], 0
    for n in need_pages:
        out.append(perm[at:at + n].copy())
        at += n
    return out


def make_batch(name: str, shape: Shape, ctx_len, q_len, seed: int, n_pages: Optional[int] = None,
               pool_factor: float = 1.25, profile: str = "paper", chunk_size: int = 0,
               identity_tables: bool = False) -> StepBatch:
    """Build a StepBatch with the given row structure.

    profile "paper":  Q, K, V ~ N(0,1)/sqrt(D)             (the distribution the configs state)
    profile "peaked": Q, K, V ~ N(0,1)                     (logit std ~ 1: a non-flat softmax)
    profile "needle": "paper" values, but per (row, KV head) one key position carries a key
                      aligned with the row's queries and a large value vector, so that every
                      token that may see that position returns (almost exactly) that vector.
    """
    ctx_len = np.asarray(ctx_len, dtype=np.int32)
    q_len = np.asarray(q_len, dtype=np.int32)
    rng = np.random.Generator(np.random.Philox(seed))
    P = shape.P
    need = [int((c + t + P - 1) // P) for c, t in zip(ctx_len, q_len)]
    if n_pages is None:
        n_pages = max(1, int(math.ceil(pool_factor * sum(need))))
    if identity_tables:
        tables, at = [], 0
        for n in need:
            tables.append(np.arange(at, at + n, dtype=np.int32))
            at += n
    else:
        tables = _deal_pages(rng, need, n_pages)
    std = 1.0 if profile == "peaked" else 1.0 / math.sqrt(shape.D)
    N = int(q_len.sum())
    C = int(ctx_len.sum())
    largest = max(N * shape.Hq * shape.D, int(ctx_len.max(initial=0)) * shape.Hkv * shape.D, 1)
    bank = ValueBank(seed + 1, std, log2_size=min(24, max(14, int(math.ceil(math.log2(largest))))))
    q = bank.take(N * shape.Hq * shape.D).reshape(N, shape.Hq, shape.D)
    k_new = bank.take(N * shape.Hkv * shape.D).reshape(N, shape.Hkv, shape.D)
    v_new = bank.take(N * shape.Hkv * shape.D).reshape(N, shape.Hkv, shape.D)
    ck = np.empty((C, shape.Hkv, shape.D), dtype=np.uint16)
    cv = np.empty((C, shape.Hkv, shape.D), dtype=np.uint16)
    at = 0
    for c in ctx_len.tolist():
        ck[at:at + c] = bank.take(c * shape.Hkv * shape.D).reshape(c, shape.Hkv, shape.D)
        cv[at:at + c] = bank.take(c * shape.Hkv * shape.D).reshape(c, shape.Hkv, shape.D)
        at += c
    if profile == "needle":
        _plant_needles(rng, shape, ctx_len, q_len, q, k_new, v_new, ck, cv)
    return StepBatch(name, shape, n_pages, tables, ctx_len, q_len, q, k_new, v_new, ck, cv,
                     chunk_size=chunk_size, profile=profile)


def _plant_needles(rng, shape, ctx_len, q_len, q, k_new, v_new, ck, cv) -> None:
    tok0, c0 = 0, 0
    G = shape.G
    for c, t in zip(ctx_len.tolist(), q_len.tolist()):
        for g in range(shape.Hkv):
            u = rng.standard_normal(shape.D).astype(np.float32)
            ub = f32_to_bf16_bits(1.5 * u)
            val = f32_to_bf16_bits(4.0 * rng.standard_normal(shape.D).astype(np.float32))
            q[tok0:tok0 + t, g * G:(g + 1) * G, :] = ub
            pos = int(rng.integers(0, c + t))
            if pos < c:
                ck[c0 + pos, g] = ub
                cv[c0 + pos, g] = val
            else:
                k_new[tok0 + pos - c, g] = ub
                v_new[tok0 + pos - c, g] = val
        tok0 += t
        c0 += c


# --------------------------------------------------------------------------------------
# the five workload configurations
# --------------------------------------------------------------------------------------
def config1(seed: int = 1, profile: str = "paper") -> StepBatch:
    """Tiny mixed step: 4/2/64 heads, 4 decode rows with context U{16..128}, one fresh
    64-token prefill chunk, tables cut from one permutation of a 64-page pool."""
    rng = np.random.Generator(np.random.Philox(seed))
    ctx = list(rng.integers(16, 129, size=4)) + [0]
    ql = [1, 1, 1, 1, 64]
    return make_batch("config1_tiny_mixed", TINY, ctx, ql, seed + 100, n_pages=64, profile=profile,
                      chunk_size=128)


def config2(seed: int = 2, profile: str = "paper", n_decode: int = 64) -> StepBatch:
    """Decode-only batch, 8B-shaped layer: contexts lognormal (median 2048, sigma 1 in
    log space, clipped to [128, 8192]), pool 1.25x the live pages, pages scattered."""
    rng = np.random.Generator(np.random.Philox(seed))
    ctx = _lognormal_lengths(rng, 2048, 1.0, 128, 8192, n_decode)
    return make_batch("config2_decode_8b", LLAMA8B, ctx, np.ones(n_decode, np.int32), seed + 100,
                      profile=profile, chunk_size=2048 + n_decode)


def config3(seed: int = 2, profile: str = "paper", n_decode: int = 64, chunk: int = 2048) -> StepBatch:
    """Convertible-decoder burst: config 2's decode batch (same seed, same contexts) plus one
    fresh causal prefill chunk of 2048 tokens absorbed in the same step."""
    rng = np.random.Generator(np.random.Philox(seed))
    ctx = _lognormal_lengths(rng, 2048, 1.0, 128, 8192, n_decode)
    ctx = np.concatenate([ctx, [0]]).astype(np.int32)
    ql = np.concatenate([np.ones(n_decode, np.int32), [chunk]]).astype(np.int32)
    return make_batch("config3_burst_8b", LLAMA8B, ctx, ql, seed + 100, profile=profile,
                      chunk_size=chunk + n_decode)


def config4(seed: int = 4, profile: str = "paper", n_decode: int = 128, n_chunks: int = 4,
            chunk: int = 512) -> StepBatch:
    """Chunked-prefill continuation: 128 decode rows (context lognormal, median 4096,
    clipped to [128, 16384]) plus 4 chunks of 512 tokens whose prior context is U{0..6144}."""
    rng = np.random.Generator(np.random.Philox(seed))
    ctx_d = _lognormal_lengths(rng, 4096, 1.0, 128, 16384, n_decode)
    ctx_p = rng.integers(0, 6145, size=n_chunks).astype(np.int32)
    ctx = np.concatenate([ctx_d, ctx_p]).astype(np.int32)
    ql = np.concatenate([np.ones(n_decode, np.int32), np.full(n_chunks, chunk, np.int32)])
    return make_batch("config4_chunked_8b", LLAMA8B, ctx, ql, seed + 100, profile=profile,
                      chunk_size=n_chunks * chunk + n_decode)


# --------------------------------------------------------------------------------------
# config 5: bursty trace replay on a Convertible Decoder
# --------------------------------------------------------------------------------------
@dataclass
class ReplayRequest:
    req_id: int
    prompt_len: int
    output_len: int
    arrival_s: float
    cached: int = 0          # tokens in the KV cache
    decoded: int = 0         # output tokens produced so far
    warm: bool = False       # in flight at step 0 (context preloaded)
    admitted_step: int = -1      # step before which the request entered the instance
    first_token_step: int = -1   # step that held the last chunk of its prompt (-1: not reached)


@dataclass
class ReplayStep:
    index: int
    adds: List[ReplayRequest]                 # requests that enter the instance before the step
    preload: List[tuple]                      # (warm request, tokens cached before step 0): load these first
    rows: List[tuple]                         # (req_id, q_len, ctx_len), decode rows first
    frees: List[int]                          # req_ids that complete with this step


class TraceReplay:
    """Virtual-clock simulator of one Convertible Decoder (Sec. 3.4, Sec. 4.4).

    Arrivals: Gamma inter-arrival times with coefficient of variation ``cv`` and mean rate
    ``rate`` (shape 1/cv^2): long gaps separated by tight clumps, like the bursts of Sec. 2.3.
    Prompts lognormal (median 1024, clip [16, 8192]); outputs lognormal (median 256, clip
    [1, 2048]); sigma 1 in log space. Every step lasts ``step_s`` of virtual time.
    Batch rule: all live decode requests take one token each (decode has priority); at most
    ONE prefill task is in progress at a time and it gets min(remaining prompt,
    chunk_size - decode rows, max_chunk) tokens; a request is admitted only while fewer than
    ``max_decodes`` requests are live. A finished prefill yields the first output token; the
    request then decodes output_len - 1 more tokens and is freed.

    ``max_prefill_tasks`` > 1 generalises the rule: prefill tasks are served in arrival order,
    each with what is left of the step's budget, and while budget is left and fewer than
    ``max_prefill_tasks`` tasks are in progress the next queued request is admitted into the
    same step. A step then carries chunks of several requests, and a prompt longer than the
    budget continues over the following steps.
    """

    def __init__(self, seed: int = 5, shape: Shape = LLAMA70B, n_steps: int = 200, rate: float = 20.0,
                 cv: float = 4.0, step_s: float = 0.030, max_decodes: int = 256, warm: int = 192,
                 max_chunk: int = 8192, chunk_size: int = 8448, max_prefill_tasks: int = 1):
        self.shape = shape
        self.n_steps = n_steps
        self.chunk_size = chunk_size
        self.max_chunk = max_chunk
        self.max_decodes = max_decodes
        self.max_prefill_tasks = max_prefill_tasks
        self.step_s = step_s
        rng = np.random.Generator(np.random.Philox(seed))
        self.rng = rng
        k = 1.0 / (cv * cv)
        theta = (1.0 / rate) / k
        horizon = n_steps * step_s
        t, arrivals = 0.0, []
        while True:
            t += float(rng.gamma(k, theta))
            if t >= horizon:
                break
            arrivals.append(t)
        n = len(arrivals)
        prompts = _lognormal_lengths(rng, 1024, 1.0, 16, 8192, n + warm)
        outputs = _lognormal_lengths(rng, 256, 1.0, 1, 2048, n + warm)
        self.requests: List[ReplayRequest] = []
        rid = 0
        self.warm_requests = []
        for i in range(warm):
            out = int(outputs[i])
            if out < 2:
                continue                      # nothing left to decode: not in flight
            r = ReplayRequest(rid, int(prompts[i]), out, 0.0, warm=True)
            r.decoded = int(rng.integers(1, out))          # 1 .. out-1 tokens already produced
            r.cached = r.prompt_len + r.decoded - 1        # the newest token is not cached yet
            self.warm_requests.append(r)
            rid += 1
        for i, a in enumerate(arrivals):
            self.requests.append(ReplayRequest(rid, int(prompts[warm + i]), int(outputs[warm + i]), a))
            rid += 1
        self.max_context = 8192 + 2048

    def steps(self):
        """Yield ReplayStep objects in order. Deterministic given the seed."""
        live: List[ReplayRequest] = []       # decoding
        queue: List[ReplayRequest] = []      # arrived, waiting for prefill
        tasks: List[ReplayRequest] = []      # prefill tasks in progress, in arrival order
        pending = list(self.requests)
        for s in range(self.n_steps):
            now = s * self.step_s
            adds, preload = [], []
            if s == 0:
                for r in self.warm_requests:
                    live.append(r)
                    adds.append(r)
                    preload.append((r, r.cached))      # the request objects advance as the replay runs
            while pending and pending[0].arrival_s <= now:
                queue.append(pending.pop(0))

            def admit():
                if len(tasks) < self.max_prefill_tasks and queue and len(live) + len(tasks) < self.max_decodes:
                    r = queue.pop(0)
                    r.admitted_step = s
                    tasks.append(r)
                    adds.append(r)
                    return True
                return False

            if not tasks:
                admit()
            rows, frees = [], []
            for r in live:
                rows.append((r.req_id, 1, r.cached))
            budget = self.chunk_size - len(live)
            finished = []
            i = 0
            while budget > 0 and (i < len(tasks) or (i > 0 and admit())):
                task = tasks[i]
                i += 1
                take = min(task.prompt_len - task.cached, budget, self.max_chunk)
                if take > 0:
                    rows.append((task.req_id, take, task.cached))
                    task.cached += take
                    budget -= take
                    if task.cached == task.prompt_len:
                        finished.append(task)
            still = []
            for r in live:
                r.cached += 1
                r.decoded += 1
                if r.decoded >= r.output_len:
                    frees.append(r.req_id)
                else:
                    still.append(r)
            live = still
            for r in finished:
                r.decoded = 1
                r.first_token_step = s
                if r.output_len <= 1:
                    frees.append(r.req_id)
                else:
                    live.append(r)
                tasks.remove(r)
            yield ReplayStep(s, adds, preload, rows, frees)


def replay_values(shape: Shape, seed: int, n_tokens: int, bank: ValueBank):
    """Q, K_new, V_new bit patterns for n_tokens tokens, drawn from the bank."""
    q = bank.take(n_tokens * shape.Hq * shape.D).reshape(n_tokens, shape.Hq, shape.D)
    k = bank.take(n_tokens * shape.Hkv * shape.D).reshape(n_tokens, shape.Hkv, shape.D)
    v = bank.take(n_tokens * shape.Hkv * shape.D).reshape(n_tokens, shape.Hkv, shape.D)
    return q, k, v
