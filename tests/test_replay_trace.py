"""Host-only checks of the bursty-trace simulator and of the TTFT accounting of a replay
(Sec. 3.4 and 4.4: a Convertible Decoder absorbs prefill work chunk by chunk under its chunk-size
budget; Sec. 2.2 and 6.1: TTFT and its SLOs). No GPU, no library call."""
import numpy as np
import pytest

from paper_2512_03416_b200 import workloads as wl
from paper_2512_03416_b200.replay import ttft_report

TRACES = [
    dict(),
    dict(chunk_size=2304, shape=wl.LLAMA8B),
    dict(chunk_size=2304, shape=wl.LLAMA8B, max_prefill_tasks=4),
    dict(seed=11, chunk_size=768, max_prefill_tasks=3, n_steps=150),
    dict(seed=12, chunk_size=300, max_prefill_tasks=8, max_decodes=200, warm=150, n_steps=120),
]


@pytest.mark.parametrize("kw", TRACES)
def test_trace_steps_follow_the_batch_rule(kw):
    t = wl.TraceReplay(**kw)
    by_id = {r.req_id: r for r in t.requests + t.warm_requests}
    cached = {r.req_id: r.cached for r in t.warm_requests}
    produced = {r.req_id: r.decoded for r in t.warm_requests}
    admitted, done_order, live, freed = set(cached), [], set(cached), set()
    multi = 0
    for st in t.steps():
        for r in st.adds:
            assert r.req_id not in freed
            if r.req_id not in admitted:
                assert r.arrival_s <= st.index * t.step_s          # nobody is served before arriving
                admitted.add(r.req_id)
                live.add(r.req_id)
                cached[r.req_id], produced[r.req_id] = 0, 0
        assert len(live) <= t.max_decodes
        q_lens = [ql for _, ql, _ in st.rows]
        assert sum(q_lens) <= t.chunk_size                          # chunk size = prefill tokens + decode rows
        kinds = [ctx >= by_id[rid].prompt_len for rid, _, ctx in st.rows]
        assert kinds == sorted(kinds, reverse=True)                 # decode rows first
        prefill_rows = [(rid, ql, ctx) for (rid, ql, ctx), dec in zip(st.rows, kinds) if not dec]
        assert len(prefill_rows) <= t.max_prefill_tasks
        multi += len(prefill_rows) > 1
        assert len({rid for rid, _, _ in st.rows}) == len(st.rows)   # one row per request
        # every live decoding request gets its token in every step (decode is never starved)
        decoding = {rid for rid in live if cached[rid] >= by_id[rid].prompt_len}
        assert decoding == {rid for (rid, _, _), dec in zip(st.rows, kinds) if dec}
        for (rid, ql, ctx), dec in zip(st.rows, kinds):
            r = by_id[rid]
            assert ctx == cached[rid] and ql >= 1                   # chunks continue where the last one ended
            if dec:
                assert ql == 1
                produced[rid] += 1
            else:
                assert ql <= t.max_chunk and ctx + ql <= r.prompt_len
                if ctx + ql == r.prompt_len:
                    produced[rid] = 1                               # the prefill yields the first output token
                    done_order.append(rid)
            cached[rid] += ql
        # prefill tasks are served in arrival order: an unfinished one blocks no earlier arrival
        pf_ids = [rid for rid, _, _ in prefill_rows]
        assert pf_ids == sorted(pf_ids)
        for rid in st.frees:
            assert produced[rid] >= by_id[rid].output_len and rid in live
            live.discard(rid)
            freed.add(rid)
        for rid in live:
            assert produced[rid] < by_id[rid].output_len or cached[rid] < by_id[rid].prompt_len
    assert done_order == sorted(done_order)                         # first tokens come out in arrival order
    if t.max_prefill_tasks > 1:
        assert multi > 0                                            # some step did carry several requests' chunks
    assert t.max_context >= max(cached.values())


def test_one_task_rule_is_the_default_and_several_tasks_fill_the_budget():
    base = dict(chunk_size=2304, shape=wl.LLAMA8B)
    one = [st.rows for st in wl.TraceReplay(**base).steps()]
    also_one = [st.rows for st in wl.TraceReplay(max_prefill_tasks=1, **base).steps()]
    assert one == also_one
    t = wl.TraceReplay(max_prefill_tasks=4, **base)
    by_id = {r.req_id: r for r in t.requests + t.warm_requests}
    waiting = 0
    for st in t.steps():
        n = sum(ql for _, ql, _ in st.rows)
        pf = [rid for rid, _, ctx in st.rows if ctx < by_id[rid].prompt_len]
        # when the step is neither full nor at a limit, nobody who has arrived is left waiting
        if n < t.chunk_size and len(pf) < t.max_prefill_tasks and len(st.rows) < t.max_decodes:
            arrived = [r for r in t.requests if r.arrival_s <= st.index * t.step_s]
            waiting += sum(1 for r in arrived if r.admitted_step < 0 or r.admitted_step > st.index)
    assert waiting == 0


@pytest.mark.parametrize("kw", TRACES)
def test_ttft_report_against_a_direct_count(kw):
    """TTFT by its definition (Sec. 2.2), counted request by request: walk the steps until the
    request's whole prompt is cached; the first token exists at the end of that step."""
    t = wl.TraceReplay(**kw)
    steps = list(t.steps())
    rng = np.random.default_rng(3)
    durations = rng.uniform(0.2, 1.6, len(steps)) * t.step_s           # some steps overrun the virtual tick
    for secs in (None, durations):
        rep = ttft_report(t, steps, step_seconds=secs)
        ends, end = [], 0.0
        for i in range(len(steps)):
            end = max(i * t.step_s, end) + (t.step_s if secs is None else secs[i])
            ends.append(end)
        ttfts = []
        for r in t.requests:
            got = 0
            for i, st in enumerate(steps):
                got += sum(ql for rid, ql, ctx in st.rows if rid == r.req_id and ctx < r.prompt_len)
                if got == r.prompt_len:
                    ttfts.append(ends[i] - r.arrival_s)
                    assert r.first_token_step == i
                    break
        assert rep["requests"] == len(ttfts) and rep["unfinished"] == len(t.requests) - len(ttfts)
        if ttfts:
            a = np.asarray(ttfts)
            assert abs(rep["ttft_mean_s"] - a.mean()) < 1e-12 and abs(rep["ttft_max_s"] - a.max()) < 1e-12
            for slo, key in ((0.25, "250ms"), (0.4, "400ms"), (2.0, "2000ms")):
                assert abs(rep["attainment"][key] - (a <= slo).mean()) < 1e-12
            assert rep["queue_mean_s"] >= 0 and rep["chunk_steps_max"] >= 1
            assert (a > 0).all()


def test_ttft_hand_example():
    """Two requests, 10 ms steps, budget 8 tokens and no decodes in flight: a 12-token prompt that
    arrives at 5 ms is served in steps 1 and 2 (8 + 4 tokens) -> first token at 30 ms, TTFT 25 ms,
    5 ms of it queueing; a 4-token prompt arriving at 6 ms shares step 2 when two tasks are allowed
    (TTFT 24 ms) and otherwise waits for step 3 (TTFT 34 ms)."""
    for tasks, want_b in ((2, 0.024), (1, 0.034)):
        t = wl.TraceReplay(seed=1, n_steps=6, step_s=0.010, warm=0, chunk_size=8, max_prefill_tasks=tasks)
        t.requests = [wl.ReplayRequest(0, 12, 1, 0.005), wl.ReplayRequest(1, 4, 1, 0.006)]
        steps = list(t.steps())
        rep = ttft_report(t, steps, slos=(0.0245, 0.03))
        assert rep["requests"] == 2 and rep["unfinished"] == 0
        assert abs(rep["ttft_max_s"] - max(0.025, want_b)) < 1e-12
        assert abs(rep["ttft_mean_s"] - (0.025 + want_b) / 2) < 1e-12
        assert abs(rep["queue_mean_s"] - ((0.005 + (0.014 if tasks == 2 else 0.024)) / 2)) < 1e-12
        assert rep["attainment"] == {"24ms": 0.5 if tasks == 2 else 0.0, "30ms": 1.0 if tasks == 2 else 0.5}
