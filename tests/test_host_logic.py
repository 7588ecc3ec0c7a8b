"""CPU-only tests of the library's host side: the shared object loads and exports the header's
symbols, allocator and block-table properties, step validation (nothing launches on a bad step),
the work-list planner's coverage, and the Token Velocity counters against the oracle mirror."""
import os
import re

import numpy as np
import pytest

from oracle import velocity
from paper_2512_03416_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def make_ctx(Hq=32, Hkv=8, D=128, n_pages=1000, max_requests=64, width=512, chunk=2112, reserved=0,
             split=0, seed=0):
    cfg = B.ts_config(Hq, Hkv, D, 16, n_pages, max_requests, width, chunk, reserved, split, 0, 0.0, 0, seed,
                      None, 0, None, 0)
    rc, h = B.ts_create(cfg)
    assert rc == B.TS_OK
    return h


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "tokenscale.h")).read()
    declared = set(re.findall(r"\b(ts_[a-z_0-9]+)\s*\(", hdr))
    declared -= {"ts_ctx"}
    assert declared, "no declarations found"
    lib = B.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in tokenscale.h but not exported"
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)


def test_sizes_and_bad_shapes():
    cfg = B.ts_config(32, 8, 128, 16, 100, 8, 64, 0, 0, 0, 0, 0.0, 0, 0, None, 0, None, 0)
    assert B.ts_pool_bytes(cfg) == 100 * 2 * 8 * 16 * 128 * 2
    assert B.ts_workspace_bytes(cfg) > 0
    for bad in [dict(head_dim=96), dict(page_size=32), dict(n_q_heads=30), dict(n_kv_heads=1, n_q_heads=32)]:
        c = B.ts_config(32, 8, 128, 16, 100, 8, 64, 0, 0, 0, 0, 0.0, 0, 0, None, 0, None, 0)
        for k, v in bad.items():
            setattr(c, k, v)
        assert B.ts_pool_bytes(c) == 0
        rc, _ = B.ts_create(c)
        assert rc == B.TS_ERR_UNSUPPORTED
    assert B.ts_strerror(B.TS_ERR_NO_PAGES) == "not enough free pages"


def test_allocator_properties():
    rng = np.random.default_rng(0)
    h = make_ctx(n_pages=300, max_requests=16, width=40, seed=77)
    live = {}
    for it in range(400):
        op = rng.integers(0, 3)
        if op == 0 and len(live) < 16:
            rc, slot = B.ts_request_add(h, it, 10, 10)
            assert rc == B.TS_OK and slot not in live
            live[slot] = 0
        elif op == 1 and live:
            slot = int(rng.choice(list(live)))
            want = int(rng.integers(0, 700))
            _, before, _ = B.ts_block_table(h, slot)
            rc = B.ts_alloc_pages(h, slot, want, 0)
            _, after, _ = B.ts_block_table(h, slot)
            need = (want + 15) // 16
            if rc == B.TS_OK:
                assert len(after) == max(len(before), need) and after[:len(before)] == before
            else:
                assert rc in (B.TS_ERR_NO_PAGES, B.TS_ERR_TABLE_SHORT) and after == before  # all or nothing
                if rc == B.TS_ERR_TABLE_SHORT:
                    assert need > 40
        elif op == 2 and live:
            slot = int(rng.choice(list(live)))
            assert B.ts_request_free(h, slot) == B.TS_OK
            del live[slot]
            assert B.ts_request_free(h, slot) == B.TS_ERR_INVALID          # double free
        # invariants: no page in two tables; free + in use == n_pages
        seen = set()
        for s in live:
            _, pages, _ = B.ts_block_table(h, s)
            assert not (seen & set(pages)) and all(0 <= p < 300 for p in pages)
            seen |= set(pages)
        _, v = B.ts_velocity(h)
        assert v["pages_in_use"] == len(seen) and v["pages_in_use"] + v["pages_free"] == 300
    B.ts_destroy(h)


def test_free_list_order_and_shuffle():
    h = make_ctx(n_pages=50, max_requests=4, width=50)
    _, s = B.ts_request_add(h, 1, 0, 0)
    B.ts_alloc_pages(h, s, 16 * 5, 0)
    assert B.ts_block_table(h, s)[1] == [0, 1, 2, 3, 4]
    B.ts_destroy(h)
    h = make_ctx(n_pages=50, max_requests=4, width=50, seed=5)
    _, s = B.ts_request_add(h, 1, 0, 0)
    B.ts_alloc_pages(h, s, 16 * 50, 0)
    pages = B.ts_block_table(h, s)[1]
    assert sorted(pages) == list(range(50)) and pages != list(range(50))
    B.ts_destroy(h)


def test_reserved_pages_only_for_prefill():
    h = make_ctx(n_pages=20, max_requests=4, width=20, reserved=8)
    _, a = B.ts_request_add(h, 1, 0, 0)
    _, b = B.ts_request_add(h, 2, 0, 0)
    assert B.ts_alloc_pages(h, a, 16 * 13, 0) == B.TS_ERR_NO_PAGES     # would dip into the reserve
    assert B.ts_alloc_pages(h, a, 16 * 12, 0) == B.TS_OK
    assert B.ts_alloc_pages(h, b, 16 * 1, 0) == B.TS_ERR_NO_PAGES
    assert B.ts_alloc_pages(h, b, 16 * 8, 1) == B.TS_OK                # an absorbed prefill may
    assert B.ts_alloc_pages(h, b, 16 * 9, 1) == B.TS_ERR_NO_PAGES
    B.ts_destroy(h)


def test_block_table_set_rules():
    h = make_ctx(n_pages=32, max_requests=4, width=8)
    _, a = B.ts_request_add(h, 1, 0, 0)
    _, b = B.ts_request_add(h, 2, 0, 0)
    assert B.ts_block_table_set(h, a, [5, 9, 31]) == B.TS_OK
    assert B.ts_block_table(h, a)[1] == [5, 9, 31]
    assert B.ts_block_table_set(h, b, [9]) == B.TS_ERR_INVALID        # owned by a
    assert B.ts_block_table_set(h, b, [4, 4]) == B.TS_ERR_INVALID     # duplicate
    assert B.ts_block_table_set(h, b, [32]) == B.TS_ERR_INVALID       # out of range
    assert B.ts_block_table_set(h, b, list(range(9))) == B.TS_ERR_TABLE_SHORT
    assert B.ts_block_table_set(h, a, [9, 6]) == B.TS_OK              # re-layout keeps own pages
    B.ts_alloc_pages(h, b, 16 * 8, 0)
    pb = B.ts_block_table(h, b)[1]
    assert len(pb) == 8 and not (set(pb) & {9, 6})
    B.ts_destroy(h)


def _step(slots, ql, ctx, ptr=0):
    return B.make_step(slots, ql, ctx, ptr, ptr, ptr, ptr)


def test_step_validation_launches_nothing():
    h = make_ctx(n_pages=100, max_requests=4, width=10, chunk=40)
    _, a = B.ts_request_add(h, 1, 20, 5)
    _, b = B.ts_request_add(h, 2, 10, 5)
    B.ts_alloc_pages(h, a, 32, 0)
    B.ts_alloc_pages(h, b, 16, 0)
    cases = [
        (([a], [1], [3]), B.TS_ERR_INVALID),          # ctx_len disagrees with the cached length
        (([a], [0], [0]), B.TS_ERR_INVALID),          # q_len < 1
        (([a, a], [1, 1], [0, 0]), B.TS_ERR_INVALID),  # slot twice
        (([3], [1], [0]), B.TS_ERR_INVALID),          # dead slot
        (([a], [33], [0]), B.TS_ERR_TABLE_SHORT),     # table covers 32 tokens
        (([a, b], [30, 16], [0, 0]), B.TS_ERR_BUDGET),  # 46 prefill tokens > chunk size 40
    ]
    for (sl, ql, cl), want in cases:
        st, keep = _step(sl, ql, cl, 256)
        assert B.ts_mixed_step(h, st, 0) == want, (sl, ql, cl)
        assert B.ts_plan_step(h, B.make_step(sl, ql, cl)[0])[0] == want
    st, keep = B.make_step([a], [1], [0])                  # null tensors
    assert B.ts_mixed_step(h, st, 0) == B.TS_ERR_INVALID
    st, keep = _step([a], [1], [0], 264)                   # misaligned tensors
    assert B.ts_mixed_step(h, st, 0) == B.TS_ERR_INVALID
    st, keep = _step([a], [1], [0], 256)                   # valid step, but no device buffers
    assert B.ts_mixed_step(h, st, 0) == B.TS_ERR_CUDA
    _, v = B.ts_velocity(h)
    assert v["kernel_launches"] == 0 and v["steps"] == 0
    assert B.ts_block_table(h, a)[2] == 0                  # lengths untouched by failed steps
    B.ts_destroy(h)


def _check_plan(items, G, rows, tile_rows=256):
    """Every (packed query row, key) pair of the step is covered exactly once."""
    by_row = {}
    for it in items:
        by_row.setdefault(it[0], []).append(it)
    partials = []
    for r, (ql, ctx) in enumerate(rows):
        its = by_row.pop(r)
        if ql == 1:
            assert all(i[1] == 0 and i[2] == 0 and i[3] == 1 for i in its)
            spans = sorted((i[4], i[5]) for i in its)
            assert spans[0][0] == 0 and spans[-1][1] == ctx + 1
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            assert all(s[0] % 64 == 0 and s[1] > s[0] for s in spans)
            if len(its) > 1:
                ps = sorted(i[6] for i in its)
                assert ps[0] >= 0 and ps == list(range(ps[0], ps[0] + len(its)))
                partials += ps
            else:
                assert its[0][6] == -1
        else:
            assert all(i[1] == 1 and i[4] == 0 and i[6] == -1 for i in its)
            tiles = sorted((i[2], i[3], i[5]) for i in its)
            at = 0
            for q0, cnt, k_end in tiles:
                assert q0 == at and 1 <= cnt <= tile_rows // G
                at += cnt
                assert k_end == ctx + q0 + cnt
            assert at == ql
    assert not by_row
    assert len(set(partials)) == len(partials)


@pytest.mark.parametrize("split", [0, 64, 200, 4096])
def test_planner_covers_the_step_exactly(split):
    rng = np.random.default_rng(split)
    h = make_ctx(Hq=32, Hkv=8, n_pages=40000, max_requests=64, width=1100, chunk=0, split=split)
    rows, slots = [], []
    for r in range(40):
        ql = int(rng.choice([1, 1, 1, 2, 17, 300]))
        ctx = int(rng.choice([0, 1, 63, 64, 65, 511, 512, 513, 5000, 16000]))
        _, s = B.ts_request_add(h, r, ctx + ql, 0)
        assert B.ts_alloc_pages(h, s, ctx + ql, 0) == B.TS_OK
        assert B.ts_request_set_len(h, s, ctx) == B.TS_OK
        rows.append((ql, ctx))
        slots.append(s)
    st, keep = B.make_step(slots, [r[0] for r in rows], [r[1] for r in rows])
    rc, items = B.ts_plan_step(h, st)
    assert rc == B.TS_OK
    _check_plan(items, 4, rows)
    B.ts_destroy(h)


def test_planner_respects_partial_capacity():
    h = make_ctx(Hq=8, Hkv=8, D=64, n_pages=300000, max_requests=256, width=2048, chunk=0, split=64)
    slots, ctxs = [], []
    for r in range(256):
        _, s = B.ts_request_add(h, r, 16000, 0)
        assert B.ts_alloc_pages(h, s, 16001, 0) == B.TS_OK
        B.ts_request_set_len(h, s, 16000)
        slots.append(s)
        ctxs.append(16000)
    rc, items = B.ts_plan_step(h, B.make_step(slots, [1] * 256, ctxs)[0])
    assert rc == B.TS_OK
    assert max(i[6] for i in items) < 2048 + 2 * 256       # split grew until the partials fit
    _check_plan(items, 1, [(1, 16000)] * 256, 64)
    B.ts_destroy(h)


def test_counters_match_the_oracle_mirror():
    h = make_ctx(Hq=4, Hkv=2, D=64, n_pages=64, max_requests=8, width=16, chunk=128)
    mirror = velocity.Counters()
    slots = []
    for r, L in enumerate([10, 20, 64]):
        _, s = B.ts_request_add(h, r, L, 4)
        slots.append(s)
    # counters of processed tokens move only through steps, which need a device; here the cached
    # lengths are set by hand and the release path (Eq. 1) is checked
    for s, L in zip(slots, [10, 20, 64]):
        B.ts_alloc_pages(h, s, L + 4, 0)
        B.ts_request_set_len(h, s, L + 3)
        mirror.live[s] = L + 3
    for s in slots[:2]:
        assert B.ts_request_free(h, s) == B.TS_OK
        mirror.free(s)
    _, v = B.ts_velocity(h)
    assert v["released_tokens"] == mirror.released_tokens == 13 + 23
    assert v["released_requests"] == mirror.released_requests == 2
    assert B.ts_report_step_time(h, 0.25) == B.TS_OK and B.ts_report_step_time(h, -1.0) == B.TS_ERR_INVALID
    assert B.ts_velocity(h)[1]["busy_seconds"] == 0.25
    assert abs(v["released_tokens"] / 0.25 - mirror.decode_velocity(0.25)) < 1e-9      # Eq. 1
    assert B.ts_prefill_budget(h, 28) == velocity.prefill_budget(128, 28) == 100       # Eq. 5 numerator
    assert B.ts_prefill_budget(h, 500) == 0
    B.ts_destroy(h)


def test_convertible_decoder_configuration_matches_the_oracle():
    """Sec. 4.4 / Eq. 5 / Eq. 6 through the C ABI against oracle/velocity.py on seeded profiles."""
    rng = np.random.Generator(np.random.Philox(44))
    for _ in range(200):
        n = int(rng.integers(1, 12))
        sizes = np.cumsum(rng.integers(1, 2000, size=n)).astype(np.int32)
        secs = np.sort(rng.uniform(0.0, 0.2, size=n))
        if rng.random() < 0.3:                       # a noisy profile: not monotone
            secs = rng.permutation(secs)
        batch, slo = int(rng.integers(0, 300)), float(rng.uniform(0.01, 0.2))
        got = B.ts_pick_chunk_size(sizes.tolist(), secs.tolist(), batch, slo)
        assert got == velocity.pick_chunk_size(sizes.tolist(), secs.tolist(), batch, slo)
        v = B.ts_convertible_prefill_velocity(max(got, 1), float(batch) / 2, slo)
        assert abs(v - max(velocity.convertible_prefill_velocity(max(got, 1), batch / 2, slo), 0.0)) <= 1e-9 * max(v, 1.0)
        ttft = float(rng.uniform(0.05, 2.0))
        assert abs(B.ts_reserved_memory(v, 4096.0, ttft) - (velocity.reserved_memory(v, 4096.0, ttft) if v > 0 else 0.0)) <= 1e-6 * max(v, 1.0)
        assert B.ts_reserved_pages(v, ttft, 16) == (velocity.reserved_pages(v, ttft, 16) if v > 0 else 0)
    # invalid profiles
    assert B.ts_pick_chunk_size([], [], 4, 0.1) == B.TS_ERR_INVALID
    assert B.ts_pick_chunk_size([256, 128], [0.01, 0.02], 4, 0.1) == B.TS_ERR_INVALID      # not ascending
    assert B.ts_pick_chunk_size([128], [0.01], -1, 0.1) == B.TS_ERR_INVALID
    assert B.ts_pick_chunk_size([128], [0.01], 4, 0.0) == B.TS_ERR_INVALID
    assert B.ts_convertible_prefill_velocity(64, 64.0, 0.1) == 0.0
    assert B.ts_reserved_pages(0.0, 0.25, 16) == 0


def test_scaler_and_router_match_the_oracle():
    """Eq. 2-4 and Algorithm 1 through the C ABI against oracle/velocity.py on seeded cases."""
    rng = np.random.Generator(np.random.Philox(45))
    names = {B.TS_ROUTE_PREFILLER: "prefiller", B.TS_ROUTE_CONVERTIBLE: "convertible", B.TS_ROUTE_QUEUE: "queue"}
    for _ in range(300):
        lam, vp, vn = (float(x) for x in rng.uniform(1.0, 5e4, size=3))
        assert B.ts_prefiller_instances(lam, vp, vn) == velocity.prefiller_instances(lam, vp, vn)
        nb = int(rng.integers(1, 10))
        rates, vels = rng.uniform(0.0, 4e4, size=nb), rng.uniform(5e3, 4e4, size=nb)
        d = B.ts_decoder_demand(rates.tolist(), vels.tolist())
        assert abs(d - velocity.decoder_demand(rates.tolist(), vels.tolist())) <= 1e-12 * max(d, 1.0)
        ic = int(rng.integers(0, 4))
        assert B.ts_regular_decoders(d, ic) == velocity.regular_decoders(d, ic)
        n_p, n_c = int(rng.integers(0, 5)), int(rng.integers(0, 3))
        pt, pv = rng.uniform(0, 2e4, size=n_p).tolist(), rng.uniform(5e3, 2e4, size=n_p).tolist()
        ct, cv = rng.uniform(0, 2e4, size=n_c).tolist(), rng.uniform(5e3, 3e4, size=n_c).tolist()
        slo = float(rng.choice([0.25, 0.4, 2.0]))                      # the paper's TTFT SLOs
        idx, kind = B.ts_route_prefill(pt, pv, ct, cv, slo)
        want_kind, want_idx = velocity.route_prefill(pt, pv, ct, cv, slo)
        assert names[kind] == want_kind and idx == max(want_idx, 0)
    assert B.ts_prefiller_instances(10.0, 8.0, 1e9) == 2               # Fig. 7
    assert B.ts_prefiller_instances(0.0, 8.0, 8.0) == 0
    assert B.ts_prefiller_instances(1.0, 0.0, 8.0) == B.TS_ERR_INVALID
    assert B.ts_decoder_demand([1.0], [0.0]) == -1.0
    assert B.ts_regular_decoders(0.0, 1) == 0
    assert B.ts_route_prefill([1.0], [0.0], [], [], 1.0)[0] == B.TS_ERR_INVALID


def test_debug_flag_needs_a_short_wait_limit():
    """The flag that makes a wait run out is refused unless the context's wait limit is short."""
    for limit in (0, 50_000_001):
        cfg = B.ts_config(32, 8, 128, 16, 100, 8, 64, 0, 0, 0, 0, 0.0, 0, 0, None, 0, None, 0, limit,
                          B.TS_DEBUG_LOSE_APPEND_ARRIVAL)
        rc, _ = B.ts_create(cfg)
        assert rc == B.TS_ERR_INVALID
    cfg = B.ts_config(32, 8, 128, 16, 100, 8, 64, 0, 0, 0, 0, 0.0, 0, 0, None, 0, None, 0, 2_000_000,
                      B.TS_DEBUG_LOSE_APPEND_ARRIVAL)
    rc, h = B.ts_create(cfg)
    assert rc == B.TS_OK
    B.ts_destroy(h)
    cfg.debug_flags = 2                      # unknown bit
    assert B.ts_create(cfg)[0] == B.TS_ERR_INVALID
