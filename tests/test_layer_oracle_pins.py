"""Pins of the decoder-layer oracle (oracle/layer.py): every function against something other
than itself -- loops on tiny inputs, closed forms, invariants of the mathematics -- and a set of
planted mistakes that the pins must notice."""
import importlib.util
import math
import os

import numpy as np
import pytest

from oracle import layer as L

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def bf(x):
    return L.f64_to_bits(np.asarray(x, np.float64))


# ------------------------------------------------------------------------------------- pins
def pin_gemm_matches_three_loops(M=L):
    rng = np.random.default_rng(0)
    a, w = rng.standard_normal((5, 7)), rng.standard_normal((3, 7))
    assert np.abs(M.gemm(a, w) - np.array(M.gemm_loops(a.tolist(), w.tolist()))).max() < 1e-12
    assert M.gemm(a, w).shape == (5, 3)


def pin_gemm_picks_weight_rows(M=L):
    """a = unit vector e_k gives C[0, n] = w[n, k]: catches a transposed or mis-strided operand."""
    w = np.arange(12, dtype=np.float64).reshape(3, 4) + 1.0      # [out 3, in 4]
    for k in range(4):
        a = np.zeros((1, 4)); a[0, k] = 1.0
        assert np.array_equal(M.gemm(a, w)[0], w[:, k])
    assert np.array_equal(M.gemm(np.eye(4), np.eye(4)), np.eye(4))


def pin_bf16_rounding(M=L):
    """Nearest even on known bit patterns (the spacing at 1.0 is 2^-7): 1 + 2^-8 is a tie and goes
    down to 1.0 (even mantissa), 1 + 3*2^-8 is a tie and goes up to 1 + 2^-6 (even mantissa),
    1 + 2^-8 + 2^-20 is above the tie and goes up."""
    assert M.f64_to_bits(np.array([1.0]))[0] == 0x3F80
    assert M.f64_to_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert M.f64_to_bits(np.array([1.0 + 2.0 ** -8 + 2.0 ** -20]))[0] == 0x3F81
    assert M.f64_to_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    assert M.f64_to_bits(np.array([-2.5]))[0] == 0xC020
    x = np.array([0.1, -3.7, 1e-3, 123456.0])
    assert np.abs(M.bits_to_f64(M.f64_to_bits(x)) / x - 1).max() <= 2.0 ** -9


def pin_rope_closed_forms(M=L):
    """D = 2 is a plane rotation by pos radians; D = 4 adds a second pair at frequency theta^-1/2."""
    t = np.array([[[1.0, 0.0]]])
    for p in (0.0, 0.5, 3.0):
        out = M.rope(t, np.array([p]), 10000.0)[0, 0]
        assert np.allclose(out, [math.cos(p), math.sin(p)], atol=1e-12)
    t = np.array([[[1.0, 2.0, 3.0, 4.0]]])                     # pairs (1, 3) and (2, 4)
    p, th = 7.0, 100.0
    a0, a1 = p, p * th ** -0.5
    want = [1 * math.cos(a0) - 3 * math.sin(a0), 2 * math.cos(a1) - 4 * math.sin(a1),
            3 * math.cos(a0) + 1 * math.sin(a0), 4 * math.cos(a1) + 2 * math.sin(a1)]
    assert np.allclose(M.rope(t, np.array([p]), th)[0, 0], want, atol=1e-12)


def pin_rope_invariants(M=L):
    rng = np.random.default_rng(1)
    q, k = rng.standard_normal((3, 2, 16)), rng.standard_normal((3, 2, 16))
    pos = np.array([0, 5, 1000])
    rq = M.rope(q, pos, 500000.0)
    assert np.array_equal(rq[0], q[0])                          # position 0 is the identity
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-12)
    # the score of a query at m and a key at n depends on m - n only
    def score(m, n):
        return float((M.rope(q[:1], np.array([m]), 500000.0)[0, 0] * M.rope(k[:1], np.array([n]), 500000.0)[0, 0]).sum())
    assert abs(score(17, 5) - score(1017, 1005)) < 1e-9
    assert abs(score(17, 5) - score(18, 5)) > 1e-6
    # heads are rotated independently and identically
    assert np.allclose(M.rope(q[:, :1], pos, 500000.0), rq[:, :1])


def pin_rmsnorm(M=L):
    g = np.array([1.0, 2.0, 0.5, 1.0])
    out = M.rmsnorm(np.full((1, 4), 3.0), g, 1e-5)
    assert np.allclose(out[0], 3.0 / math.sqrt(9.0 + 1e-5) * g, rtol=1e-14)
    x = np.array([[3.0, -4.0, 0.0, 0.0]])                       # mean square 25/4
    assert np.allclose(M.rmsnorm(x, np.ones(4), 0.0)[0], x[0] / 2.5, rtol=1e-14)
    assert np.allclose(M.rmsnorm(7.0 * x, np.ones(4), 0.0), M.rmsnorm(x, np.ones(4), 0.0), rtol=1e-14)
    two = M.rmsnorm(np.array([[1.0, 1.0], [2.0, 0.0]]), np.ones(2), 0.0)
    assert np.allclose(two, [[1.0, 1.0], [math.sqrt(2.0), 0.0]], rtol=1e-14)   # rows are independent


def pin_silu(M=L):
    x = np.array([-30.0, -2.0, 0.0, 1.0, 30.0])
    s = M.silu(x)
    assert s[2] == 0.0 and abs(s[3] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert np.allclose(s - M.silu(-x), x, atol=1e-12)           # x s(x) + x s(-x) = x
    assert abs(s[4] - 30.0) < 1e-10 and abs(s[0]) < 1e-10


def pin_positions_and_split(M=L):
    assert M.positions([5, 0, 9], [1, 3, 2]).tolist() == [5, 0, 1, 2, 9, 10]
    # q/k/v are cut from the projection in the order Q heads, K heads, V heads; with a weight matrix
    # whose row r is the unit vector e_(r mod hidden), theta so large that nothing rotates and a
    # unit gain, output feature r is the normalised input feature r mod hidden
    Hq, Hkv, D, hidden = 2, 1, 4, 8
    w = np.zeros(((Hq + 2 * Hkv) * D, hidden))
    for r in range(w.shape[0]):
        w[r, r % hidden] = 1.0
    x = np.arange(1, 9, dtype=np.float64)[None, :]
    xb = bf(x)
    q, k, v = M.qkv_rope(xb, bf(np.ones(hidden)), bf(w), np.array([0]), Hq, Hkv, D, 0.0, 1e30)
    h = M.bits_to_f64(bf(M.rmsnorm(M.bits_to_f64(xb), np.ones(hidden), 0.0)))[0]
    assert np.array_equal(M.bits_to_f64(q).reshape(-1), h[np.arange(8) % hidden])
    assert np.array_equal(M.bits_to_f64(k).reshape(-1), h[(8 + np.arange(4)) % hidden])
    assert np.array_equal(M.bits_to_f64(v).reshape(-1), h[(12 + np.arange(4)) % hidden])


def pin_layer_residuals_and_mlp(M=L):
    """Zero output and down projections leave the input untouched (two residual connections);
    with W_o = 0 only, out = x + W_down . (silu(g) * u) of the normalised x, checked by hand."""
    rng = np.random.default_rng(2)
    Hq, Hkv, D, hidden, inter, N = 2, 1, 4, 8, 6, 3
    x = bf(rng.standard_normal((N, hidden)))
    wt = dict(w_norm1=bf(np.ones(hidden)), w_qkv=bf(rng.standard_normal(((Hq + 2 * Hkv) * D, hidden))),
              w_o=bf(np.zeros((hidden, Hq * D))), w_norm2=bf(1.0 + 0.1 * rng.standard_normal(hidden)),
              w_gate=bf(rng.standard_normal((inter, hidden))), w_up=bf(rng.standard_normal((inter, hidden))),
              w_down=bf(np.zeros((hidden, inter))))
    attn = lambda q, k, v: rng.standard_normal((N, Hq, D))
    out, _ = M.layer_step(attn, x, wt, np.arange(N), Hq, Hkv, D)
    assert np.array_equal(out, x)
    wt["w_down"] = bf(rng.standard_normal((hidden, inter)))
    out, mid = M.layer_step(attn, x, wt, np.arange(N), Hq, Hkv, D, eps=1e-5)
    xf = M.bits_to_f64(x)
    assert np.array_equal(mid["y"], x)                           # W_o = 0
    h2 = M.bits_to_f64(bf(xf / np.sqrt((xf * xf).mean(-1, keepdims=True) + 1e-5) * M.bits_to_f64(wt["w_norm2"])))
    g = M.bits_to_f64(bf(h2 @ M.bits_to_f64(wt["w_gate"]).T))
    u = M.bits_to_f64(bf(h2 @ M.bits_to_f64(wt["w_up"]).T))
    z = M.bits_to_f64(bf(g / (1.0 + np.exp(-g)) * u))
    want = bf(xf + z @ M.bits_to_f64(wt["w_down"]).T)
    assert np.array_equal(out, want)
    # the attention output enters through W_o: a one-hot W_o copies one attention feature
    wt["w_down"] = bf(np.zeros((hidden, inter)))
    wo = np.zeros((hidden, Hq * D)); wo[2, 5] = 1.0
    wt["w_o"] = bf(wo)
    a_fixed = rng.standard_normal((N, Hq, D))
    out, mid = M.layer_step(lambda q, k, v: a_fixed, x, wt, np.arange(N), Hq, Hkv, D)
    want = xf.copy(); want[:, 2] += M.bits_to_f64(bf(a_fixed.reshape(N, -1)))[:, 5]
    assert np.array_equal(out, bf(want))


PINS = [pin_gemm_matches_three_loops, pin_gemm_picks_weight_rows, pin_bf16_rounding, pin_rope_closed_forms,
        pin_rope_invariants, pin_rmsnorm, pin_silu, pin_positions_and_split, pin_layer_residuals_and_mlp]


@pytest.mark.parametrize("pin", PINS, ids=[p.__name__ for p in PINS])
def test_pin(pin):
    pin()


# each entry: (name, text in oracle/layer.py, replacement) -- one planted mistake per mutant
MUTANTS = [
    ("gemm_operand_reversed", "np.asarray(a, np.float64) @ np.asarray(w, np.float64).T", "np.asarray(a, np.float64)[:, ::-1] @ np.asarray(w, np.float64).T"),
    ("rope_sign", "lo * c - hi * s", "lo * c + hi * s"),
    ("rope_adjacent_frequency", "theta ** (-2.0 * np.arange(half, dtype=np.float64) / D)", "theta ** (-1.0 * np.arange(half, dtype=np.float64) / D)"),
    ("rope_second_half_unrotated", "hi * c + lo * s", "hi"),
    ("rmsnorm_sum_not_mean", "(x * x).mean(axis=-1, keepdims=True)", "(x * x).sum(axis=-1, keepdims=True)"),
    ("rmsnorm_no_gain", "x / np.sqrt(ms + eps) * np.asarray(gain, np.float64)", "x / np.sqrt(ms + eps)"),
    ("silu_sign", "x / (1.0 + np.exp(-x))", "x / (1.0 + np.exp(x))"),
    ("kv_swapped", "k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(N, Hkv, D)\n    v = qkv[:, (Hq + Hkv) * D:].reshape(N, Hkv, D)", "v = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(N, Hkv, D)\n    k = qkv[:, (Hq + Hkv) * D:].reshape(N, Hkv, D)"),
    ("no_first_residual", "bits_to_f64(x_bits) + gemm(bits_to_f64(attn_bits), bits_to_f64(w_o))", "gemm(bits_to_f64(attn_bits), bits_to_f64(w_o))"),
    ("gate_up_swapped", "silu(bits_to_f64(g)) * bits_to_f64(u)", "silu(bits_to_f64(u)) * bits_to_f64(g)"),
    ("positions_ignore_ctx", "np.arange(c, c + t)", "np.arange(0, t)"),
    ("rounding_truncates", "rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))", "rounded = u"),
]


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistakes_are_caught(mutant, tmp_path):
    name, old, new = mutant
    src = open(os.path.join(ROOT, "oracle", "layer.py")).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique"
    path = tmp_path / "layer_mut.py"
    path.write_text(src.replace(old, new))
    spec = importlib.util.spec_from_file_location("layer_mut", str(path))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    noticed = 0
    for pin in PINS:
        try:
            pin(mod)
        except AssertionError:
            noticed += 1
        except Exception:
            noticed += 1
    assert noticed, f"no pin notices the planted mistake '{name}'"
