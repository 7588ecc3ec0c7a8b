"""GPU tests of multi-step behaviour through the C ABI: lengths advance, tables grow between
steps, chunked prefill continues across steps, steps can be repeated, host-buffer steps equal
device-buffer steps, counters follow the oracle mirror, and a short bursty replay stays in parity
with the oracle step by step."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import velocity
from paper_2512_03416_b200 import binding as B
from paper_2512_03416_b200 import workloads as wl
from paper_2512_03416_b200.decoder import Decoder, TsError
from paper_2512_03416_b200.harness import LoadedBatch, from_dev, to_dev
from paper_2512_03416_b200.replay import ReplayRunner
from tests.helpers import assert_parity, oracle_step

pytestmark = pytest.mark.gpu


def _oracle_tables(dec, slots, width):
    m = np.zeros((len(slots), width), np.int32)
    for r, s in enumerate(slots):
        pages, _ = dec.block_table(s)
        m[r, :len(pages)] = pages
    return m


def test_chunked_prefill_then_decode_steps():
    """One request prefilled in three uneven chunks, a second decoding alongside, then both
    decode for a few steps; pages are taken step by step from a shuffled free list."""
    s = wl.Shape(32, 8, 128)
    rng = np.random.default_rng(3)
    bank = wl.ValueBank(9, 1.0, 20)
    dec = Decoder(s.Hq, s.Hkv, s.D, 200, 4, 64, chunk_size=400, alloc_shuffle_seed=11, nan_fill=True)
    mirror = velocity.Counters()
    pool = np.full(s.pool_elems(200), wl.BF16_NAN, np.uint16)
    a = dec.request_add(1, 333, 8)
    b = dec.request_add(2, 90, 8)
    # b arrives with its 90-token context already prefilled elsewhere
    ck, cv = bank.take(90 * s.Hkv * s.D).reshape(90, s.Hkv, s.D), bank.take(90 * s.Hkv * s.D).reshape(90, s.Hkv, s.D)
    dec.alloc_pages(b, 90)
    dec.kv_append([b], [90], [0], to_dev(ck), to_dev(cv))
    oracle.kv_append(pool, s.Hkv, s.D, s.P, _oracle_tables(dec, [b], 64), [0], [90], ck, cv)
    len_a, len_b = 0, 90
    plan = [(130, 1), (77, 1), (126, 1), (1, 1), (1, 1), (1, 1)]          # (new tokens of a, of b) per step
    for qa, qb in plan:
        dec.alloc_pages(a, len_a + qa, for_prefill=qa > 1)
        dec.alloc_pages(b, len_b + qb)
        n = qa + qb
        q = bank.take(n * s.Hq * s.D).reshape(n, s.Hq, s.D)
        k = bank.take(n * s.Hkv * s.D).reshape(n, s.Hkv, s.D)
        v = bank.take(n * s.Hkv * s.D).reshape(n, s.Hkv, s.D)
        out = torch.full((n, s.Hq, s.D), 0x7FC0, dtype=torch.int16, device="cuda")
        dec.mixed_step([a, b], [qa, qb], [len_a, len_b], to_dev(q), to_dev(k), to_dev(v), out)
        mirror.step([a, b], [qa, qb], [len_a, len_b])
        want = oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, 1 / math.sqrt(s.D), _oracle_tables(dec, [a, b], 64),
                                 [len_a, len_b], [qa, qb], q, k, v)
        torch.cuda.synchronize()
        assert_parity(wl.bf16_bits_to_f32(from_dev(out)), want, "peaked", f"step {qa},{qb}")
        len_a += qa
        len_b += qb
        assert dec.block_table(a)[1] == len_a and dec.block_table(b)[1] == len_b
    assert dec.device_status() == 0
    assert np.array_equal(from_dev(dec.pool), pool), "pool differs after the step sequence"
    cnt = dec.velocity()
    assert (cnt["steps"], cnt["prefill_tokens"], cnt["decode_tokens"]) == (mirror.steps, mirror.prefill_tokens, mirror.decode_tokens)
    dec.request_free(a)
    mirror.free(a)
    assert dec.velocity()["released_tokens"] == mirror.released_tokens == len_a     # Eq. 1 numerator
    with pytest.raises(TsError):
        dec.mixed_step([a], [1], [len_a], to_dev(q), to_dev(k), to_dev(v), out)    # freed slot
    dec.close()


def test_repeated_step_and_host_buffers_agree():
    b = wl.make_batch("rep", wl.LLAMA8B, [300, 1000, 0], [1, 1, 150], seed=21, profile="peaked", chunk_size=160)
    want, pool_want = oracle_step(b)
    lb = LoadedBatch(b)
    lb.step(keep_len=True)
    first = lb.output()
    lb.out.fill_(0)
    lb.step_repeatable()                                   # same step again, lengths were kept
    assert np.array_equal(lb.output(), first)
    assert_parity(first, want, "peaked", "repeatable step")
    # host-buffer entry point: inputs from (pinned) host memory, result back in host memory
    hq = torch.from_numpy(b.q.view(np.int16)).pin_memory()
    hk = torch.from_numpy(b.k_new.view(np.int16)).pin_memory()
    hv = torch.from_numpy(b.v_new.view(np.int16)).pin_memory()
    ho = torch.zeros_like(hq).pin_memory()
    lb.dec.mixed_step_host(lb.slots, b.q_len.tolist(), b.ctx_len.tolist(), hq, hk, hv, ho, keep_len=False)
    assert np.array_equal(wl.bf16_bits_to_f32(ho.numpy().view(np.uint16)), first)
    assert np.array_equal(lb.pool(), pool_want)
    assert lb.dec.block_table(lb.slots[2])[1] == 150       # this time the lengths advanced
    assert lb.dec.device_status() == 0


def test_pipelined_host_steps_match_device_steps():
    """Seven consecutive steps issued from pinned host buffers without waiting in between (the
    uploads and kernels of later steps overlap a step's download; every staging set is reused) give bit for bit the outputs and the pool of the same steps issued from
    device buffers on a second decoder with the same allocator seed."""
    s = wl.LLAMA8B
    bank = wl.ValueBank(31, 1.0, 20)
    mk = lambda: Decoder(s.Hq, s.Hkv, s.D, 120, 4, 64, chunk_size=400, alloc_shuffle_seed=5, nan_fill=True)
    host, dev = mk(), mk()
    plan = [(130, 1), (77, 1), (126, 1), (1, 1), (1, 1), (1, 1), (1, 1)]      # (new tokens of a, of b) per step
    sa, sb = host.request_add(1, 333, 8), host.request_add(2, 90, 8)
    assert (dev.request_add(1, 333, 8), dev.request_add(2, 90, 8)) == (sa, sb)
    ck, cv = (bank.take(90 * s.Hkv * s.D).reshape(90, s.Hkv, s.D) for _ in range(2))
    for d in (host, dev):
        d.alloc_pages(sb, 90)
        d.kv_append([sb], [90], [0], to_dev(ck), to_dev(cv))
    len_a, len_b = 0, 90
    pinned, dev_out = [], []
    for qa, qb in plan:
        n = qa + qb
        q = bank.take(n * s.Hq * s.D).reshape(n, s.Hq, s.D)
        k = bank.take(n * s.Hkv * s.D).reshape(n, s.Hkv, s.D)
        v = bank.take(n * s.Hkv * s.D).reshape(n, s.Hkv, s.D)
        bufs = [torch.from_numpy(x.view(np.int16).copy()).pin_memory() for x in (q, k, v)]
        bufs.append(torch.full((n, s.Hq, s.D), 0x7FC0, dtype=torch.int16).pin_memory())
        pinned.append(bufs)                                  # inputs and outputs stay alive and untouched
        for d in (host, dev):
            d.alloc_pages(sa, len_a + qa, for_prefill=qa > 1)
            d.alloc_pages(sb, len_b + qb)
        host.mixed_step_host([sa, sb], [qa, qb], [len_a, len_b], *bufs, wait=False)
        out = torch.full((n, s.Hq, s.D), 0x7FC0, dtype=torch.int16, device="cuda")
        dev.mixed_step([sa, sb], [qa, qb], [len_a, len_b], to_dev(q), to_dev(k), to_dev(v), out)
        dev_out.append(out)
        len_a += qa
        len_b += qb
    host.host_fence()
    torch.cuda.synchronize()
    for i, (bufs, out) in enumerate(zip(pinned, dev_out)):
        assert np.array_equal(bufs[3].numpy(), out.cpu().numpy()), f"step {i}"
        assert not np.any(bufs[3].numpy() == 0x7FC0)
    assert np.array_equal(from_dev(host.pool), from_dev(dev.pool))
    assert host.device_status() == 0 and dev.device_status() == 0
    # a waiting call after the pipelined ones still returns with its result in place
    q, k, v, o = pinned[-1]
    o.fill_(0)
    host.alloc_pages(sa, len_a + 1)
    host.alloc_pages(sb, len_b + 1)
    host.mixed_step_host([sa, sb], [1, 1], [len_a, len_b], q, k, v, o)
    assert np.any(o.numpy() != 0)
    host.close()
    dev.close()


def test_step_over_budget_is_refused_on_the_host():
    b = wl.make_batch("bud", wl.TINY, [10], [40], seed=5, chunk_size=32)
    lb = LoadedBatch(b)
    before = lb.dec.velocity()["kernel_launches"]
    with pytest.raises(TsError) as e:
        lb.step()
    assert e.value.code == B.TS_ERR_BUDGET
    assert lb.dec.velocity()["kernel_launches"] == before


def test_short_bursty_replay_matches_the_oracle():
    """A scaled-down replay of the bursty trace (70B-shaped layer): requests come and go, pages
    are recycled, a prefill task is absorbed in chunks next to the decode batch."""
    trace = wl.TraceReplay(seed=8, shape=wl.LLAMA70B, n_steps=30, rate=300.0, cv=4.0, step_s=0.030,
                           max_decodes=40, warm=24, max_chunk=384, chunk_size=424)
    run = ReplayRunner(trace, seed=70, keep_host=True, nan_fill=True)
    s = run.shape
    n_pages = run.dec.cfg.n_pages
    width = run.dec.cfg.max_pages_per_req
    pool = np.full(s.pool_elems(n_pages), wl.BF16_NAN, np.uint16)
    mirror = velocity.Counters()
    rng = np.random.default_rng(0)
    saw_prefill = saw_free = 0
    for ps in run.steps:
        run.begin_step(ps)                                  # the first call also loads the warm contexts
        for r, cached in ps.preload:
            k, v = run.warm_ctx[r.req_id]
            tm = _oracle_tables(run.dec, [run.slot_of[r.req_id]], width)
            oracle.kv_append(pool, s.Hkv, s.D, s.P, tm, [0], [cached], k, v)
            mirror.live[run.slot_of[r.req_id]] = cached
        if ps.req_ids:
            slots = ps.slots.tolist()
            tm = _oracle_tables(run.dec, slots, width)
            run.launch(ps)
            mirror.step(slots, ps.q_len, ps.ctx_len)
            q, k, v = ps.host
            n = ps.n_tokens
            sel = np.arange(n) if n <= 96 else np.unique(np.concatenate([np.arange(0, n, 7), [n - 1], rng.integers(0, n, 24)]))
            want = oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, 1 / math.sqrt(s.D), tm, ps.ctx_len, ps.q_len,
                                     q, k, v, sel=sel.astype(np.int32))
            got = wl.bf16_bits_to_f32(from_dev(ps.out))[sel]
            assert_parity(got, want, "paper", f"replay step {ps.index}")
            saw_prefill += ps.prefill_tokens > 0
        for rid in ps.frees:
            mirror.free(run.slot_of[rid])
        saw_free += len(ps.frees)
        run.end_step(ps)
    assert saw_prefill >= 2 and saw_free >= 2, "the scaled-down trace should absorb prefill work and recycle pages"
    assert run.dec.device_status() == 0
    assert np.array_equal(from_dev(run.dec.pool), pool), "pool differs after the replay"
    v = run.dec.velocity()
    assert (v["steps"], v["prefill_tokens"], v["decode_tokens"], v["released_tokens"], v["released_requests"]) == \
        (mirror.steps, mirror.prefill_tokens, mirror.decode_tokens, mirror.released_tokens, mirror.released_requests)


def _replay_sampled_parity(trace, extra_steps, min_prefill_checked):
    """Runs a replay as the benchmark issues it. The oracle mirrors every append (so the whole pool
    can be compared at the end) and checks the attention output on a sample: steps 0, 1, every 20th
    and the last one, plus `extra_steps(run)`; in a sampled step every decode row and, per prefill
    chunk, 192 seeded tokens plus the first and last token of every 128-token stretch."""
    run = ReplayRunner(trace, keep_host=True, nan_fill=True)
    s = run.shape
    n_pages, width = run.dec.cfg.n_pages, run.dec.cfg.max_pages_per_req
    pool = np.full(s.pool_elems(n_pages), wl.BF16_NAN, np.uint16)
    rng = np.random.default_rng(1)
    last = len(run.steps) - 1
    sampled = {0, 1, last} | set(range(20, last, 20)) | set(extra_steps(run))
    checked = checked_prefill = 0
    for ps in run.steps:
        run.begin_step(ps)
        for r, cached in ps.preload:
            k, v = run.warm_ctx[r.req_id]
            tm = _oracle_tables(run.dec, [run.slot_of[r.req_id]], width)
            oracle.kv_append(pool, s.Hkv, s.D, s.P, tm, [0], [cached], k, v)
        if ps.req_ids:
            slots = ps.slots.tolist()
            tm = _oracle_tables(run.dec, slots, width)
            run.launch(ps)
            q, k, v = ps.host
            if ps.index in sampled:
                sel, t0 = [], 0
                for ql in ps.q_len:
                    if ql == 1:
                        sel.append(t0)
                    else:
                        edges = [t0 + e for b in range(0, ql, 128) for e in (b, min(b + 127, ql - 1))]
                        sel.extend(edges + (t0 + rng.integers(0, ql, 192)).tolist())
                    t0 += ql
                sel = np.unique(np.asarray(sel, np.int32))
                want = oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, 1 / math.sqrt(s.D), tm, ps.ctx_len, ps.q_len,
                                         q, k, v, sel=sel)
                got = wl.bf16_bits_to_f32(from_dev(ps.out))[sel]
                assert_parity(got, want, "paper", f"full replay step {ps.index}")
                checked += 1
                checked_prefill += ps.prefill_tokens > 0
            else:
                oracle.kv_append(pool, s.Hkv, s.D, s.P, tm, ps.ctx_len, ps.q_len, k, v)
        run.end_step(ps)
    assert checked >= 10 and checked_prefill >= min_prefill_checked
    assert run.dec.device_status() == 0
    assert np.array_equal(from_dev(run.dec.pool), pool), "pool differs after the full replay"
    return run


def test_full_size_replay_sampled_parity():
    """The 200-step bursty replay at its full size (70B-shaped layer, up to 256 decode rows with
    contexts up to 32768, prefill chunks up to 8192 tokens); the first two steps that carry at
    least 2048 prefill tokens are among the sampled ones."""
    _replay_sampled_parity(wl.TraceReplay(),
                           lambda run: [ps.index for ps in run.steps if ps.prefill_tokens >= 2048][:2], 2)


def test_chunked_replay_with_several_prefill_tasks_sampled_parity():
    """The same trace under a chunk size of 2304 tokens with up to four prefill tasks in progress
    (Sec. 4.4: chunk size = prefill tokens + decode batch): prompts continue across steps at
    arbitrary, not page-aligned, offsets and one step carries chunks of several requests. Sampled
    as well: the first three steps with more than one prefill row and the first three whose chunk
    continues an earlier one."""
    def extra(run):
        several = [ps.index for ps in run.steps if sum(1 for t in ps.q_len if t > 1) > 1][:3]
        cont = [ps.index for ps in run.steps if any(t > 1 and c > 0 for t, c in zip(ps.q_len, ps.ctx_len))][:3]
        assert len(several) == 3 and len(cont) == 3
        return several + cont

    run = _replay_sampled_parity(wl.TraceReplay(chunk_size=2304, max_prefill_tasks=4), extra, 6)
    assert max(ps.n_tokens for ps in run.steps) <= 2304
