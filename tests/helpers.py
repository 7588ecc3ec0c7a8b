"""Shared test plumbing: runs a StepBatch through the CPU oracle."""
import math

import numpy as np

import oracle
from paper_2512_03416_b200 import workloads as wl


def oracle_pool_with_context(batch):
    """Pool image (NaN sentinel everywhere) with every row's cached context appended."""
    s = batch.shape
    pool = batch.fresh_pool()
    if int(batch.ctx_len.sum()) > 0:
        oracle.kv_append(pool, s.Hkv, s.D, s.P, batch.table_matrix(), np.zeros_like(batch.ctx_len),
                         batch.ctx_len, batch.context_k, batch.context_v)
    return pool


def oracle_step(batch, sel=None, scale=None, threads=0):
    """Returns (out fp32 [n, Hq, D], pool after the step)."""
    s = batch.shape
    pool = oracle_pool_with_context(batch)
    scale = 1.0 / math.sqrt(s.D) if scale is None else scale
    out = oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, scale, batch.table_matrix(), batch.ctx_len,
                            batch.q_len, batch.q, batch.k_new, batch.v_new, sel=sel, threads=threads)
    return out, pool


def gathered_kv(batch, row):
    """Contiguous fp64 K, V [n, Hkv, D] of one row (context followed by the new tokens)."""
    c0 = int(batch.ctx_len[:row].sum())
    t0 = int(batch.q_len[:row].sum())
    c, t = int(batch.ctx_len[row]), int(batch.q_len[row])
    k = np.concatenate([batch.context_k[c0:c0 + c], batch.k_new[t0:t0 + t]])
    v = np.concatenate([batch.context_v[c0:c0 + c], batch.v_new[t0:t0 + t]])
    return wl.bf16_bits_to_f32(k).astype(np.float64), wl.bf16_bits_to_f32(v).astype(np.float64)


def parity_metrics(got_f32, want_f32):
    d = np.abs(got_f32.astype(np.float64) - want_f32.astype(np.float64))
    return float(d.max()) if d.size else 0.0, float(d.mean()) if d.size else 0.0


# ------------------------------------------------------------------------------------ GPU side
class GpuRun:
    """LoadedBatch plus the checks every parity test wants after a step."""

    def __init__(self, batch, **kw):
        from paper_2512_03416_b200.harness import LoadedBatch
        self.lb = LoadedBatch(batch, **kw)
        self.dec = self.lb.dec
        self.slots = self.lb.slots

    def step(self, keep_len=False):
        self.lb.step(keep_len=keep_len)
        out = self.lb.output()
        assert self.dec.device_status() == 0
        return out

    def pool(self):
        return self.lb.pool()


def assert_parity(got, want, profile="paper", what=""):
    """Absolute gates on the stated value distribution, relative gates on every profile."""
    max_abs, mean_abs = parity_metrics(got, want)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    if profile in ("paper", "peaked"):
        assert max_abs <= 2e-2, f"{what}: max-abs {max_abs}"
        assert mean_abs <= 2e-3, f"{what}: mean-abs {mean_abs}"
    peak = float(np.abs(want).max()) if want.size else 0.0
    assert max_abs <= 2.0 ** -7 * peak + 1e-6, f"{what}: max-abs {max_abs} vs peak {peak}"
    g = got.reshape(-1, got.shape[-1]).astype(np.float64)
    w = want.reshape(-1, want.shape[-1]).astype(np.float64)
    rel = np.linalg.norm(g - w, axis=1) / np.maximum(np.linalg.norm(w, axis=1), 1e-30)
    assert rel.max() <= 1e-2, f"{what}: worst relative row error {rel.max()}"
    return max_abs, mean_abs
