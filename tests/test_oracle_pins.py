"""Pins of the CPU oracle against things other than itself.

Each pin is a plain function raising AssertionError; `test_planted_mistakes_are_caught` re-runs
the whole set against copies of ts_oracle.c with one mistake planted in each and requires at
least one pin to fail per mutant.
"""
import math
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from oracle import velocity
from paper_2512_03416_b200 import workloads as wl
from tests.helpers import gathered_kv, oracle_pool_with_context, oracle_step

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
bf = wl.f32_to_bf16_bits
f32 = wl.bf16_bits_to_f32


def _manual_batch(shape, ctx, ql, q, k_new, v_new, ck, cv, tables=None, n_pages=None):
    P = shape.P
    need = [int((c + t + P - 1) // P) for c, t in zip(ctx, ql)]
    if tables is None:
        tables, at = [], 0
        for n in need:
            tables.append(np.arange(at, at + n, dtype=np.int32))
            at += n
    n_pages = n_pages or max(1, sum(need))
    return wl.StepBatch("manual", shape, n_pages, tables, np.asarray(ctx, np.int32),
                        np.asarray(ql, np.int32), q, k_new, v_new, ck, cv)


# ---------------------------------------------------------------------------------- closed forms
def pin_single_key_returns_its_value():
    """n = 1 (first token of a fresh chunk): O = V_0 exactly."""
    b = wl.make_batch("t", wl.TINY, [0], [5], seed=11)
    out, _ = oracle_step(b)
    want = f32(b.v_new[0])                              # [Hkv, D]
    for h in range(b.shape.Hq):
        assert np.array_equal(out[0, h], want[h // b.shape.G]), "n=1 must return V_0 bit-exactly"


def pin_two_keys_logistic_weights():
    """Two keys, logits (0, x): weights are 1/(1+e^x) and e^x/(1+e^x); x is set through the
    scale 1/sqrt(D), so a missing or wrong scale fails."""
    s = wl.Shape(1, 1, 64)
    D = s.D
    x = float(f32(bf(np.array([math.log(3.0)], np.float32)))[0])
    q = np.zeros((1, 1, D), np.float32); q[0, 0, 3] = math.sqrt(D)     # scale * q = e_3
    k = np.zeros((2, 1, D), np.float32); k[1, 0, 3] = x
    v = np.zeros((2, 1, D), np.float32); v[0, 0, :] = 1.0; v[1, 0, :] = -2.0; v[1, 0, 7] = 5.0
    b = _manual_batch(s, [1], [1], bf(q), bf(k[1:]), bf(v[1:]), bf(k[:1]), bf(v[:1]))
    out, _ = oracle_step(b)
    w1 = math.exp(x) / (1.0 + math.exp(x))
    want = (1 - w1) * v[0, 0] + w1 * v[1, 0]
    assert np.allclose(out[0, 0], want, atol=2e-6), (out[0, 0][:8], want[:8])
    assert abs(w1 - 0.75) < 2e-3


def pin_equal_keys_give_causal_running_mean():
    """All keys equal => uniform weights => token i returns the mean of V over exactly the
    ctx + i + 1 visible positions. An off-by-one causal mask changes every row."""
    s = wl.TINY
    ctx, T = 21, 19
    b = wl.make_batch("t", s, [ctx], [T], seed=12)
    b.context_k[:] = b.context_k[0, 0]
    b.k_new[:] = b.context_k[0, 0]
    out, _ = oracle_step(b)
    _, v = gathered_kv(b, 0)
    for i in range(T):
        want = v[:ctx + i + 1].mean(axis=0)               # [Hkv, D]
        for h in range(s.Hq):
            assert np.allclose(out[i, h], want[h // s.G], atol=1e-6), f"row {i} head {h}"


def pin_zero_query_gives_uniform_mean():
    s = wl.TINY
    b = wl.make_batch("t", s, [33, 0], [1, 7], seed=13, profile="peaked")
    b.q[:] = 0
    out, _ = oracle_step(b)
    _, v0 = gathered_kv(b, 0)
    assert np.allclose(out[0], np.repeat(v0.mean(axis=0), s.G, axis=0), atol=1e-5)
    _, v1 = gathered_kv(b, 1)
    for i in range(7):
        assert np.allclose(out[1 + i], np.repeat(v1[:i + 1].mean(axis=0), s.G, axis=0), atol=1e-5)


def pin_equal_values_are_returned():
    s = wl.TINY
    b = wl.make_batch("t", s, [40], [9], seed=14, profile="peaked")
    val = b.context_v[0].copy()                            # [Hkv, D]
    b.context_v[:] = val
    b.v_new[:] = val
    out, _ = oracle_step(b)
    want = np.repeat(f32(val), s.G, axis=0)
    assert np.allclose(out, want[None], atol=1e-6)


# ---------------------------------------------------------------------------- library routine
def pin_matches_library_attention_fp64():
    """Special case that reduces to a library routine: gather K/V contiguously and call
    torch's scaled_dot_product_attention in fp64 with the causal-with-offset mask."""
    for shape, ctx, T, seed, prof in [(wl.TINY, 37, 23, 21, "peaked"), (wl.Shape(8, 2, 128), 50, 1, 22, "peaked"),
                                      (wl.Shape(4, 4, 64), 0, 40, 23, "paper"), (wl.Shape(6, 2, 64), 17, 33, 24, "needle")]:
        b = wl.make_batch("t", shape, [5, ctx], [1, T], seed=seed, profile=prof)
        out, _ = oracle_step(b)
        for row, tok0 in [(0, 0), (1, 1)]:
            k, v = gathered_kv(b, row)                                   # [n, Hkv, D]
            c, t = int(b.ctx_len[row]), int(b.q_len[row])
            q = f32(b.q[tok0:tok0 + t]).astype(np.float64)               # [t, Hq, D]
            qt = torch.from_numpy(q).permute(1, 0, 2)[None]              # [1, Hq, t, D]
            kt = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(shape.G, dim=0)[None]
            vt = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(shape.G, dim=0)[None]
            mask = torch.arange(c + t)[None, :] <= (c + torch.arange(t))[:, None]
            ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask)
            ref = ref[0].permute(1, 0, 2).numpy()
            err = np.abs(out[tok0:tok0 + t] - ref).max()
            tol = 1e-5 * max(1.0, np.abs(ref).max())
            assert err <= tol, f"{shape} row {row}: {err}"


def pin_selected_tokens_are_the_named_ones():
    """The `sel` form returns, in the order of `sel` (shuffled, with a repeat), exactly what the
    full call returns for those tokens, and each selected token matches a direct fp64 softmax
    over its own row's gathered keys: the index goes to the right row, position and output slot."""
    s = wl.Shape(6, 2, 64)
    ctx, ql = [9, 40, 0, 21], [1, 1, 35, 18]
    b = wl.make_batch("t", s, ctx, ql, seed=77, profile="peaked")
    full, _ = oracle_step(b)
    rng = np.random.default_rng(3)
    sel = rng.permutation(b.n_tokens)[:23].astype(np.int32)
    sel = np.concatenate([sel, sel[:1], [0, b.n_tokens - 1]]).astype(np.int32)
    got, _ = oracle_step(b, sel=sel)
    assert got.shape == (len(sel), s.Hq, s.D)
    assert np.array_equal(got, full[sel])
    starts = np.concatenate([[0], np.cumsum(ql)])
    for o, tok in enumerate(sel.tolist()):
        r = int(np.searchsorted(starts, tok, side="right") - 1)
        i = tok - int(starts[r])
        k, v = gathered_kv(b, r)                                          # [n, Hkv, D] fp64
        n = ctx[r] + i + 1
        for h in range(s.Hq):
            g = h // s.G
            q = f32(b.q[tok, h]).astype(np.float64)
            sc = (k[:n, g] @ q) / math.sqrt(s.D)
            w = np.exp(sc - sc.max())
            ref = (w[:, None] * v[:n, g]).sum(0) / w.sum()
            assert np.abs(got[o, h] - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max()), (tok, h)



# ----------------------------------------------------------------------------------- invariants
def pin_table_permutation_invariance():
    """Paged == contiguous: any placement of the pages gives bit-identical output."""
    b1 = wl.make_batch("t", wl.TINY, [45, 16, 0], [1, 1, 30], seed=31, profile="peaked",
                       identity_tables=True)
    b2 = wl.make_batch("t", wl.TINY, [45, 16, 0], [1, 1, 30], seed=31, profile="peaked", n_pages=97)
    assert any(not np.array_equal(a, c) for a, c in zip(b1.tables, b2.tables))
    assert np.array_equal(b1.q, b2.q) and np.array_equal(b1.context_k, b2.context_k)
    o1, _ = oracle_step(b1)
    o2, _ = oracle_step(b2)
    assert np.array_equal(o1, o2)


def pin_decode_equals_last_prefill_row():
    """A decode row over n-1 cached tokens equals row n-1 of a full n-token prefill."""
    s = wl.Shape(4, 2, 64)
    n = 53
    full = wl.make_batch("t", s, [0], [n], seed=32, profile="peaked")
    o_full, _ = oracle_step(full)
    dec = _manual_batch(s, [n - 1], [1], full.q[n - 1:], full.k_new[n - 1:], full.v_new[n - 1:],
                        full.k_new[:n - 1], full.v_new[:n - 1])
    o_dec, _ = oracle_step(dec)
    assert np.array_equal(o_dec[0], o_full[n - 1])


def pin_chunked_equals_unchunked():
    """Prefill in one chunk == two chunks over two steps (the second sees the first's K/V
    through the pool, with the causal mask offset by its prior context)."""
    s = wl.Shape(4, 2, 64)
    T, T1 = 70, 27                                     # chunk boundary not page aligned
    full = wl.make_batch("t", s, [0], [T], seed=33, profile="peaked")
    o_full, pool_full = oracle_step(full)
    tables = full.table_matrix()
    pool = full.fresh_pool()
    sc = 1.0 / math.sqrt(s.D)
    o1 = oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, sc, tables, [0], [T1], full.q[:T1],
                           full.k_new[:T1], full.v_new[:T1])
    o2 = oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, sc, tables, [T1], [T - T1], full.q[T1:],
                           full.k_new[T1:], full.v_new[T1:])
    assert np.array_equal(np.concatenate([o1, o2]), o_full)
    assert np.array_equal(pool, pool_full)


def pin_softmax_weights_and_convexity():
    b = wl.make_batch("t", wl.TINY, [100, 3, 0], [1, 1, 20], seed=34, profile="peaked")
    s = b.shape
    pool = oracle_pool_with_context(b)
    oracle.kv_append(pool, s.Hkv, s.D, s.P, b.table_matrix(), b.ctx_len, b.q_len, b.k_new, b.v_new)
    out, ws = oracle.attention(pool, s.Hq, s.Hkv, s.D, s.P, 0.125, b.table_matrix(), b.ctx_len, b.q_len,
                               b.q, return_weight_sum=True)
    assert np.abs(ws - 1.0).max() <= 1e-5
    tok = 0
    for r in range(b.n_rows):
        _, v = gathered_kv(b, r)
        c = int(b.ctx_len[r])
        for i in range(int(b.q_len[r])):
            vis = v[:c + i + 1]
            lo = np.repeat(vis.min(axis=0), s.G, axis=0) - 1e-5
            hi = np.repeat(vis.max(axis=0), s.G, axis=0) + 1e-5
            assert (out[tok] >= lo).all() and (out[tok] <= hi).all()
            tok += 1


def pin_gqa_group_symmetry():
    """Identical queries inside a group give identical outputs; swapping the two KV heads
    together with their query groups swaps the outputs."""
    s = wl.Shape(6, 2, 64)
    b = wl.make_batch("t", s, [29], [6], seed=35, profile="peaked")
    b.q[:, 1] = b.q[:, 0]
    b.q[:, 2] = b.q[:, 0]
    o, _ = oracle_step(b)
    assert np.array_equal(o[:, 0], o[:, 1]) and np.array_equal(o[:, 0], o[:, 2])
    assert not np.array_equal(o[:, 0], o[:, 3])
    b2 = wl.make_batch("t", s, [29], [6], seed=35, profile="peaked")
    b2.q[:, 1] = b2.q[:, 0]
    b2.q[:, 2] = b2.q[:, 0]
    b2.q = np.concatenate([b2.q[:, 3:], b2.q[:, :3]], axis=1).copy()
    for name in ("k_new", "v_new", "context_k", "context_v"):
        a = getattr(b2, name)
        setattr(b2, name, a[:, ::-1].copy())
    o2, _ = oracle_step(b2)
    assert np.array_equal(o2, np.concatenate([o[:, 3:], o[:, :3]], axis=1))


# ------------------------------------------------------------------------- needles: mask, gather
def pin_needle_visibility():
    """Position p carries a key aligned with every query and a signature value. Token i must
    return the signature iff p <= ctx + i; p = ctx + i + 1 must stay invisible."""
    s = wl.Shape(2, 1, 64)
    ctx, T = 19, 24
    for p in (0, 15, 16, 18, 19, 20, 31, 32, ctx + T - 1):
        b = wl.make_batch("t", s, [ctx], [T], seed=40 + p)
        u = np.random.default_rng(p).standard_normal(s.D).astype(np.float32)
        b.q[:] = bf(2.0 * u)
        sig = bf(np.full(s.D, 64.0 + p, np.float32))
        if p < ctx:
            b.context_k[p, 0] = bf(2.0 * u); b.context_v[p, 0] = sig
        else:
            b.k_new[p - ctx, 0] = bf(2.0 * u); b.v_new[p - ctx, 0] = sig
        out, _ = oracle_step(b)
        for i in range(T):
            sees = p <= ctx + i
            hit = abs(float(out[i, 0, 0]) - (64.0 + p)) < 0.5
            assert hit == sees, f"needle at {p}: token {i} (ctx {ctx}) sees={sees} hit={hit}"


def pin_every_position_is_gathered_from_its_slot():
    """Value vector of position j is the constant j: with one dominant key per query the
    output names the position that was read, through scattered pages and both KV heads."""
    s = wl.Shape(4, 2, 64)
    n = 83
    b = wl.make_batch("t", s, [n - 1], [1], seed=50, n_pages=41)
    rng = np.random.default_rng(5)
    dirs = rng.standard_normal((n, s.Hkv, s.D)).astype(np.float32)
    k_all = bf(dirs)                                                   # every key has its own direction
    v_all = np.empty((n, s.Hkv, s.D), np.float32)
    for g in range(s.Hkv):
        v_all[:, g, :] = (np.arange(n)[:, None] + 1000.0 * g)
    b.context_k[:] = k_all[:n - 1]; b.k_new[:] = k_all[n - 1:]
    b.context_v[:] = bf(v_all[:n - 1]); b.v_new[:] = bf(v_all[n - 1:])
    for j in (0, 1, 15, 16, 17, 47, 48, 81, 82):
        for h in range(s.Hq):
            b.q[0, h] = bf(3.0 * f32(k_all[j, h // s.G]))              # aligned with key j of its KV head
        out, _ = oracle_step(b)
        for h in range(s.Hq):
            want = float(f32(bf(np.array([j + 1000.0 * (h // s.G)], np.float32)))[0])
            assert abs(float(out[0, h, 5]) - want) < 0.51, (j, h, out[0, h, 5], want)


# ----------------------------------------------------------------------------------- KV append
def pin_append_writes_exactly_the_live_slots():
    """K/V of position t carries the code (row, t, head) in its bits; after the append the
    pool must hold each code in page table[t/16], slot t%16 and the sentinel elsewhere."""
    s = wl.Shape(4, 2, 64)
    ctx = [5, 16, 0, 31]
    ql = [1, 1, 37, 20]
    b = wl.make_batch("t", s, ctx, ql, seed=60, n_pages=23)
    tok = 0
    for r, (c, t) in enumerate(zip(ctx, ql)):
        for i in range(t):
            for g in range(s.Hkv):
                b.k_new[tok, g, :] = (r << 12) | ((c + i) << 2) | g
                b.v_new[tok, g, :] = 0x8000 | (r << 12) | ((c + i) << 2) | g
            tok += 1
    pool = b.fresh_pool()
    oracle.kv_append(pool, s.Hkv, s.D, s.P, b.table_matrix(), b.ctx_len, b.q_len, b.k_new, b.v_new)
    view = pool.reshape(b.n_pages, 2, s.Hkv, s.P, s.D)
    owner = {}
    for r, t in enumerate(b.tables):
        for idx, page in enumerate(t.tolist()):
            owner[page] = (r, idx)
    written = 0
    for page in range(b.n_pages):
        for slot in range(s.P):
            cell = view[page, :, :, slot, :]
            live = False
            if page in owner:
                r, idx = owner[page]
                t = idx * s.P + slot
                live = ctx[r] <= t < ctx[r] + ql[r]
            if live:
                for g in range(s.Hkv):
                    code = (r << 12) | (t << 2) | g
                    assert (cell[0, g] == code).all() and (cell[1, g] == (0x8000 | code)).all()
                written += 1
            else:
                assert (cell == wl.BF16_NAN).all(), f"page {page} slot {slot} was touched"
    assert written == sum(ql)


# ----------------------------------------------------------------------- Token Velocity counters
def pin_fig7_worked_example():
    path = os.path.join(ROOT, "tests", "golden", "fig7_worked_example.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for name, n_req, tok_per, vel, thr, exp_tok, exp_inst, exp_fire in rows:
        tokens = int(n_req) * int(tok_per)
        assert tokens == int(exp_tok)
        assert velocity.instances_needed(tokens, float(vel)) == int(exp_inst)
        assert velocity.request_policy_fires(int(n_req), float(thr)) == bool(int(exp_fire))


def pin_scaler_and_router():
    """Eq. 2-4 and Algorithm 1 on hand-worked cases."""
    # Fig. 7's numbers through Eq. 2 (network never the bottleneck): 10 tokens/s over 8 -> 2
    assert velocity.prefiller_instances(10.0, 8.0, 1e9) == 2
    assert velocity.prefiller_instances(10.0, 80.0, 4.0) == 3          # the smaller velocity decides
    assert velocity.prefiller_instances(16.0, 8.0, 8.0) == 2           # exact multiples are not rounded up
    # Eq. 3 with two buckets: 6000/4000 + 9000/12000 = 2.25 decoders; Eq. 4 with one convertible: 3 - 1
    d = velocity.decoder_demand([6000.0, 9000.0], [4000.0, 12000.0])
    assert abs(d - 2.25) < 1e-12
    assert velocity.regular_decoders(d, 1) == 2 and velocity.regular_decoders(d, 5) == 0
    # Algorithm 1: waiting times 0.5 s and 0.2 s on the prefillers, 0.1 s on the convertible decoder
    pre_tok, pre_v = [7000.0, 2800.0], [14000.0, 14000.0]
    cd_tok, cd_v = [2048.0], [20480.0]
    assert velocity.route_prefill(pre_tok, pre_v, cd_tok, cd_v, 0.25) == ("prefiller", 1)    # first one within the SLO
    assert velocity.route_prefill(pre_tok, pre_v, cd_tok, cd_v, 0.6) == ("prefiller", 0)
    assert velocity.route_prefill(pre_tok, pre_v, cd_tok, cd_v, 0.15) == ("convertible", 0)  # second round
    assert velocity.route_prefill(pre_tok, pre_v, cd_tok, cd_v, 0.05) == ("queue", -1)
    assert velocity.route_prefill(pre_tok, pre_v, cd_tok, cd_v, 0.2) == ("prefiller", 1)     # the bound is inclusive
    assert velocity.route_prefill([], [], [], [], 1.0) == ("queue", -1)


def pin_chunk_size_selection():
    """Sec. 4.4 against a closed form: with an iteration time that is affine in the prefill
    tokens, a + b*T, the largest admissible T is floor((SLO - a) / b) on a unit grid."""
    a, b, slo, batch = 0.004, 1.0e-5, 0.1, 64
    grid = list(range(0, 20001, 250))
    secs = [a + b * t for t in grid]
    t_max = int(math.floor((slo - a) / b / 250.0 + 1e-9)) * 250
    assert velocity.pick_chunk_size(grid, secs, batch, slo) == t_max + batch == 9500 + 64
    # stops at the FIRST violation: a later point that happens to be fast again does not count
    assert velocity.pick_chunk_size([128, 256, 512, 1024], [0.02, 0.2, 0.03, 0.04], 10, 0.1) == 138
    assert velocity.pick_chunk_size([128, 256], [0.2, 0.01], 10, 0.1) == 0
    assert velocity.pick_chunk_size([], [], 10, 0.1) == 0
    # Eq. 6 in pages: velocity * TTFT_SLO tokens, rounded up to 16-token pages
    v = velocity.convertible_prefill_velocity(9564, 64, 0.1)             # 95,000 tokens/s
    assert abs(v - 95000.0) < 1e-6
    assert abs(velocity.reserved_tokens(v, 0.25) - 23750.0) < 1e-6
    assert velocity.reserved_pages(v, 0.25, 16) == 1485                   # ceil(23750 / 16)
    assert abs(velocity.reserved_memory(v, 4096.0, 0.25) - velocity.reserved_tokens(v, 0.25) * 4096.0) < 1e-3


def pin_eq5_eq6_and_counters():
    assert velocity.prefill_budget(8448, 256) == 8192
    assert velocity.prefill_budget(100, 256) == 0
    v = velocity.convertible_prefill_velocity(2112, 64, 0.1)          # Eq. 5
    assert abs(v - 20480.0) < 1e-9
    assert abs(velocity.reserved_memory(v, 4096 * 32, 0.25) - 20480.0 * 131072 * 0.25) < 1e-3   # Eq. 6
    c = velocity.Counters()
    c.step([0, 1, 2], [1, 1, 64], [10, 20, 0])
    c.step([0, 1, 2], [1, 1, 1], [11, 21, 64])
    assert (c.steps, c.prefill_tokens, c.decode_tokens) == (2, 64, 5)
    c.free(2)
    assert c.released_tokens == 65 and c.released_requests == 1
    assert abs(c.decode_velocity(0.5) - 130.0) < 1e-12                # Eq. 1 over a 0.5 s window


PINS = [pin_single_key_returns_its_value, pin_two_keys_logistic_weights,
        pin_equal_keys_give_causal_running_mean, pin_zero_query_gives_uniform_mean,
        pin_equal_values_are_returned, pin_matches_library_attention_fp64,
        pin_table_permutation_invariance, pin_decode_equals_last_prefill_row,
        pin_chunked_equals_unchunked, pin_softmax_weights_and_convexity, pin_gqa_group_symmetry,
        pin_needle_visibility, pin_every_position_is_gathered_from_its_slot,
        pin_append_writes_exactly_the_live_slots, pin_selected_tokens_are_the_named_ones, pin_fig7_worked_example, pin_eq5_eq6_and_counters, pin_chunk_size_selection, pin_scaler_and_router]


@pytest.mark.parametrize("pin", PINS, ids=[p.__name__ for p in PINS])
def test_pin(pin):
    pin()


# each entry: (name, text in ts_oracle.c, replacement) -- one planted mistake per mutant
MUTANTS = [
    ("mask_one_short", "const int n = ctx + i + 1;", "const int n = ctx + i > 0 ? ctx + i : 1;"),
    ("mask_one_long", "const int n = ctx + i + 1;", "const int n = ctx + i + 2;"),
    ("no_scale", "s[j] = scale * dot;", "s[j] = dot;"),
    ("wrong_sign", "float p = expf(s[j] - m);", "float p = expf(m - s[j]);"),
    ("no_normalise", "for (int d = 0; d < D; ++d) out[d] /= l;", ";"),
    ("head_map_mod", "const int g = h / G;", "const int g = h % Hkv;"),
    ("v_reads_k", "table[j / P], 1, g, j % P", "table[j / P], 0, g, j % P"),
    ("slot_page_swapped_read", "table[j / P], 0, g, j % P", "table[j % P], 0, g, j / P"),
    ("append_ignores_ctx", "int t = ctx_len[r] + i;", "int t = i;"),
    ("append_slot_off", "int slot = t % P;", "int slot = (t + 1) % P;"),
    ("append_v_into_k", "memcpy(pool + pool_index(page, 1, g, slot, Hkv, P, D), vs", "memcpy(pool + pool_index(page, 0, g, slot, Hkv, P, D), vs"),
    ("dropped_d_term", "for (int d = 0; d < D; ++d) dot +=", "for (int d = 1; d < D; ++d) dot +="),
    ("sel_output_slot", "out + ((size_t)o * Hq + h) * D, s);", "out + ((size_t)(sel ? n_out - 1 - o : o) * Hq + h) * D, s);"),
    ("sel_ignored_in_worker", "long tok = sel ? sel[o] : o;\n      int r = tok_row[tok]", "long tok = o;\n      int r = tok_row[tok]"),
    ("pool_kv_stride", "((((size_t)page * 2 + (size_t)kv) * (size_t)Hkv + (size_t)head)", "((((size_t)page * 2 + (size_t)kv) * (size_t)Hkv + (size_t)(Hkv - 1 - head))"),
]


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistakes_are_caught(mutant, tmp_path):
    name, old, new = mutant
    src = open(os.path.join(ROOT, "oracle", "ts_oracle.c")).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique"
    c = tmp_path / "mut.c"
    c.write_text(src.replace(old, new))
    so = tmp_path / "libmut.so"
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-w", "-o", str(so), str(c), "-lm"])
    # A mutant may read outside its buffers, so the pins run in a child process; an assertion
    # failure or a crash both count as "noticed", a clean pass does not.
    code = ("import sys; sys.path.insert(0, %r); import oracle; oracle.use_library(%r); "
            "from tests import test_oracle_pins as t\n"
            "bad = 0\n"
            "for pin in t.PINS:\n"
            "    try:\n"
            "        pin()\n"
            "    except AssertionError:\n"
            "        bad += 1\n"
            "sys.exit(3 if bad else 0)\n") % (ROOT, str(so))
    rc = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True).returncode
    assert rc != 0, f"no pin notices the planted mistake '{name}'"
