"""Oracle of the Token Velocity bookkeeping. TEST INFRASTRUCTURE ONLY.

Plain restatements of the paper's counting rules, used to check the library's counters:

* Sec. 3.2: Token Velocity is the number of tokens a stage can release per second; an
  instance count follows as (token arrival rate) / (velocity), rounded up (Fig. 7's example:
  10 tokens/s against 8 tokens/s per instance needs 2 instances, at both bursts).
* Eq. 1: Decode Velocity counts the tokens L_r of the requests R that completed, per unit time.
  Reading used here: the numerator is the sum of L_r over requests freed in the window,
  L_r = prompt + generated tokens held in the cache when the request is released.
* Sec. 4.4: chunk size bounds (prefill tokens + decode batch size) of one iteration;
  Eq. 5: V_D^{P'} = (chunk_size - batch_size) / TPOT_SLO.
* Eq. 6: Mem_Reserved = V_D^{P'} * Mem_T * TTFT_SLO.
* Eq. 2: prefillers needed I^P = lambda / min(V_P, V_BW); Eq. 3: decoder demand
  I^D = sum over buckets of lambda'(b) / V_D(b); Eq. 4: regular decoders I^D_r = max(I^D - I^D_c, 0).
  The Scaler allocates the minimum number of instances that provides the velocity (Sec. 4.3), so
  counts are rounded up (Fig. 7: 10 tokens/s against 8 per instance -> 2).
* Algorithm 1: a prefill task goes to the first prefiller whose estimated waiting time
  inflight_tokens / velocity is within the request's SLO, else to the first Convertible Decoder
  that passes the same test with its V_D^{P'}, else it is queued.
* Sec. 4.4, chunk-size selection: the iteration time is profiled while the prefill chunk grows,
  until the TPOT SLO is violated; the chunk size chosen is the largest one before that.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field


def instances_needed(token_rate: float, velocity_per_instance: float) -> int:
    """Sec. 3.2 / Fig. 7: smallest instance count whose combined velocity covers the token rate."""
    return int(math.ceil(token_rate / velocity_per_instance))


def request_policy_fires(request_rate: float, threshold: float) -> bool:
    """Fig. 7's request-count policy: scales only when arrivals exceed the threshold."""
    return request_rate > threshold


def prefill_budget(chunk_size: int, decode_batch_size: int) -> int:
    """Sec. 4.4: prefill tokens one iteration may take next to the decode batch."""
    return max(chunk_size - decode_batch_size, 0)


def convertible_prefill_velocity(chunk_size: int, batch_size: float, tpot_slo_s: float) -> float:
    """Eq. 5."""
    return (chunk_size - batch_size) / tpot_slo_s


def reserved_memory(v_dp: float, mem_per_token: float, ttft_slo_s: float) -> float:
    """Eq. 6."""
    return v_dp * mem_per_token * ttft_slo_s


def prefiller_instances(token_rate: float, v_prefill: float, v_network: float) -> int:
    """Eq. 2, rounded up to whole instances."""
    return int(math.ceil(token_rate / min(v_prefill, v_network)))


def decoder_demand(rates, velocities) -> float:
    """Eq. 3: the (real-valued) number of decoders the per-bucket token rates ask for."""
    total = 0.0
    for lam, v in zip(rates, velocities):
        total += lam / v
    return total


def regular_decoders(demand: float, convertible: int) -> int:
    """Eq. 4 on whole instances."""
    return max(int(math.ceil(demand)) - convertible, 0)


def route_prefill(prefiller_inflight, prefiller_velocity, cd_inflight, cd_velocity, slo_s: float):
    """Algorithm 1. Returns ("prefiller", i), ("convertible", i) or ("queue", -1)."""
    for i, (tok, v) in enumerate(zip(prefiller_inflight, prefiller_velocity)):
        waiting_time = tok / v
        if waiting_time <= slo_s:
            return "prefiller", i
    for i, (tok, v) in enumerate(zip(cd_inflight, cd_velocity)):
        waiting_time = tok / v
        if waiting_time <= slo_s:
            return "convertible", i
    return "queue", -1


def reserved_tokens(v_dp: float, ttft_slo_s: float) -> float:
    """Eq. 6 divided by the per-token footprint Mem_T: the tokens' worth of memory held back."""
    return v_dp * ttft_slo_s


def reserved_pages(v_dp: float, ttft_slo_s: float, page_size: int) -> int:
    """Eq. 6 in whole KV pages."""
    return int(math.ceil(reserved_tokens(v_dp, ttft_slo_s) / page_size))


def pick_chunk_size(prefill_tokens, iteration_seconds, decode_batch_size: int, tpot_slo_s: float) -> int:
    """Sec. 4.4: walk the profile in the order it was taken (growing prefill chunk) and stop at
    the first iteration time above the TPOT SLO; chunk size = the last prefill size before that
    plus the decode batch size (the definition of chunk size), 0 if even the first point is late."""
    best = 0
    for t, sec in zip(prefill_tokens, iteration_seconds):
        if sec > tpot_slo_s:
            break
        best = int(t) + int(decode_batch_size)
    return best


@dataclass
class Counters:
    """Mirror of the library's cumulative counters, advanced by the same events."""
    steps: int = 0
    prefill_tokens: int = 0
    decode_tokens: int = 0
    released_tokens: int = 0
    released_requests: int = 0
    busy_seconds: float = 0.0
    live: dict = field(default_factory=dict)  # slot -> cached tokens

    def step(self, slots, q_len, ctx_len, keep_len: bool = False) -> None:
        if len(q_len) == 0:
            return
        self.steps += 1
        for s, ql, c in zip(slots, q_len, ctx_len):
            if ql == 1:
                self.decode_tokens += 1
            else:
                self.prefill_tokens += int(ql)
            if not keep_len:
                self.live[int(s)] = int(c) + int(ql)

    def free(self, slot: int) -> None:
        self.released_tokens += self.live.pop(int(slot), 0)
        self.released_requests += 1

    def decode_velocity(self, window_s: float) -> float:
        """Eq. 1 over a window: released tokens per second."""
        return self.released_tokens / window_s
