"""Oracle of the decoder layer around the attention step. TEST INFRASTRUCTURE ONLY.

The paper's prefill velocity (Sec. 3.2) and its chunk-size profiling (Sec. 4.4) are about whole
iterations of the model, i.e. for every layer: the projections in front of attention, attention
over the paged KV cache (Sec. 2.1), the output projection and the MLP. The paper runs Llama-3.1-8B
and Qwen-2.5-32B (Sec. 6.1) and describes none of this; the layer below is the standard
pre-norm Llama-style block those models share, written out as its definition in fp64:

    h   = rmsnorm(x; w_norm1)                      x: [N, hidden]
    qkv = h . W_qkv^T                              W_qkv: [(Hq + 2 Hkv) D, hidden], rows: Q heads, K heads, V heads
    q, k = rope(q, pos), rope(k, pos)              rotate-half convention, angle = pos * theta^(-2i/D)
    a   = attention(q, k, v)                       the mixed paged-attention step (oracle/ts_oracle.c)
    y   = x + a . W_o^T                            W_o: [hidden, Hq D]
    h2  = rmsnorm(y; w_norm2)
    g, u = h2 . W_gate^T, h2 . W_up^T              W_gate, W_up: [intermediate, hidden]
    out = y + (silu(g) * u) . W_down^T             W_down: [hidden, intermediate]

Readings where the paper is silent (it names the models, not their layer): RMSNorm with eps inside
the root and a learned gain; the rotate-half pairing (i, i + D/2) of rotary embeddings; SiLU-gated
MLP; weights stored [out features, in features]. Precision: the serving precision is bf16
(Sec. 6.1), so every tensor that crosses a kernel boundary is a bf16 tensor; `layer_step` rounds to
bf16 (nearest even) exactly at those boundaries -- h, q, k, v, a, y, h2, g, u, silu(g)*u, out -- and
computes everything between them in fp64. bf16 tensors are numpy.uint16 bit patterns.

A matmul in fp64 (numpy) is the library primitive of the GEMM step; `gemm_loops` is the same
definition as three nested loops for tiny inputs.
"""
from __future__ import annotations

import numpy as np


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bits(x: np.ndarray) -> np.ndarray:
    """Round to bf16, nearest even (through fp32, whose extra rounding only matters on exact ties
    of 2^-9 relative spacing that fp32 cannot represent either way)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def gemm(a: np.ndarray, w: np.ndarray) -> np.ndarray:
    """C[m, n] = sum_k a[m, k] * w[n, k]  (weights stored [out features, in features]); fp64."""
    return np.asarray(a, np.float64) @ np.asarray(w, np.float64).T


def gemm_loops(a, w):
    """The same definition as three loops (tiny inputs only)."""
    M, K = len(a), len(a[0])
    N = len(w)
    c = [[0.0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(a[m][k]) * float(w[n][k])
            c[m][n] = acc
    return c


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row by row; fp64."""
    x = np.asarray(x, np.float64)
    ms = (x * x).mean(axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gain, np.float64)


def rope(t: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position embedding of t [N, H, D] at positions pos [N] (rotate-half pairing):
    for i < D/2 and angle = pos * theta^(-2 i / D),
        out[i]       = t[i] cos - t[i + D/2] sin
        out[i + D/2] = t[i + D/2] cos + t[i] sin."""
    t = np.asarray(t, np.float64)
    N, H, D = t.shape
    half = D // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / D)
    ang = np.asarray(pos, np.float64)[:, None] * inv_freq[None, :]          # [N, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = t[..., :half], t[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, np.float64)
    return x / (1.0 + np.exp(-x))


def positions(ctx_len, q_len) -> np.ndarray:
    """Position of every new token of a step: row r's token i sits at ctx_len[r] + i."""
    return np.concatenate([np.arange(c, c + t) for c, t in zip(ctx_len, q_len)]).astype(np.int64) \
        if len(q_len) else np.zeros(0, np.int64)


def qkv_rope(x_bits, w_norm1, w_qkv, pos, Hq, Hkv, D, eps, theta):
    """Steps 1-3 up to the attention inputs: bf16 bit patterns q [N, Hq, D], k, v [N, Hkv, D]."""
    h = f64_to_bits(rmsnorm(bits_to_f64(x_bits), bits_to_f64(w_norm1), eps))
    qkv = gemm(bits_to_f64(h), bits_to_f64(w_qkv))                            # [N, (Hq + 2 Hkv) D]
    N = qkv.shape[0]
    q = qkv[:, :Hq * D].reshape(N, Hq, D)
    k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(N, Hkv, D)
    v = qkv[:, (Hq + Hkv) * D:].reshape(N, Hkv, D)
    return f64_to_bits(rope(q, pos, theta)), f64_to_bits(rope(k, pos, theta)), f64_to_bits(v)


def post_attention(x_bits, attn_bits, w_o, w_norm2, w_gate, w_up, w_down, eps):
    """Steps 5-8: from the attention output (bf16 [N, Hq*D]) to the layer output (bf16 [N, hidden])."""
    y = f64_to_bits(bits_to_f64(x_bits) + gemm(bits_to_f64(attn_bits), bits_to_f64(w_o)))
    h2 = f64_to_bits(rmsnorm(bits_to_f64(y), bits_to_f64(w_norm2), eps))
    g = f64_to_bits(gemm(bits_to_f64(h2), bits_to_f64(w_gate)))
    u = f64_to_bits(gemm(bits_to_f64(h2), bits_to_f64(w_up)))
    z = f64_to_bits(silu(bits_to_f64(g)) * bits_to_f64(u))
    out = f64_to_bits(bits_to_f64(y) + gemm(bits_to_f64(z), bits_to_f64(w_down)))
    return out, dict(y=y, h2=h2, g=g, u=u, z=z)


def layer_step(attention_fn, x_bits, weights, pos, Hq, Hkv, D, eps=1e-5, theta=500000.0):
    """The whole layer. `attention_fn(q_bits, k_bits, v_bits) -> fp32/fp64 [N, Hq, D]` is the
    attention step (the caller binds the paged pool, block tables and row lengths to it).
    `weights`: dict with w_norm1, w_qkv, w_o, w_norm2, w_gate, w_up, w_down as bf16 bit patterns.
    Returns (out bits [N, hidden], dict of the intermediate bf16 tensors)."""
    q, k, v = qkv_rope(x_bits, weights["w_norm1"], weights["w_qkv"], pos, Hq, Hkv, D, eps, theta)
    a = f64_to_bits(np.asarray(attention_fn(q, k, v), np.float64).reshape(len(pos), Hq * D))
    out, mid = post_attention(x_bits, a, weights["w_o"], weights["w_norm2"], weights["w_gate"],
                              weights["w_up"], weights["w_down"], eps)
    mid.update(q=q, k=k, v=v, a=a)
    return out, mid
