"""ts_decode_attention_static against ts_mixed_step and against the CPU oracle.

The static entry point is for callers that cannot hand the library a workspace because they
cannot allocate device memory where they run (all of HBM already claimed by their framework,
no permission to own memory, or no tolerance for an allocation's synchronisation). It keeps its
split partials in an array built into the library. These tests feed both entry points the same
decode batch through the C ABI and require the same answers, on two calls in a row: the second
call uses other queries and another split count, so stale contents of the shared array would
show. Both calls are also held to the oracle's result for the same inputs.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2512_03416_b200 import binding as B
from paper_2512_03416_b200 import workloads as wl
from paper_2512_03416_b200.harness import LoadedBatch, from_dev, to_dev
from tests.helpers import assert_parity, oracle_step

pytestmark = pytest.mark.gpu


def _close(a, b, what):
    d = np.abs(a.astype(np.float64) - b.astype(np.float64))
    assert np.isfinite(a).all(), f"{what}: non-finite output"
    assert d.max() <= 2e-2 and d.mean() <= 2e-3, f"{what}: max {d.max()} mean {d.mean()}"
    peak = np.abs(b).max()
    assert d.max() <= 2.0 ** -7 * peak + 1e-6, f"{what}: max {d.max()} vs peak {peak}"


class _Static:
    """A loaded decode batch plus what the static call needs (tables and lengths on the device)."""

    def __init__(self, shape, ctx, seed):
        self.s, self.ctx = shape, ctx
        self.b = wl.make_batch("static", shape, ctx, [1] * len(ctx), seed=seed, profile="peaked")
        self.lb = LoadedBatch(self.b)
        self.width = max(len(t) for t in self.b.tables)
        self.tables = torch.from_numpy(np.maximum(self.b.table_matrix(self.width), 0)).cuda()
        self.kv_len = torch.tensor([c + 1 for c in ctx], dtype=torch.int32, device="cuda")
        self.stream = torch.cuda.current_stream().cuda_stream

    def call(self, q_dev, n_splits, kv_len=None, n_rows=None, shape=None):
        s = shape or self.s
        out = torch.full((len(self.ctx), self.s.Hq, self.s.D), 0x7FC0, dtype=torch.int16, device="cuda")
        rc = B.ts_decode_attention_static(0, s.Hq, s.Hkv, s.D, self.b.n_pages, self.lb.dec.pool.data_ptr(),
                                          self.tables.data_ptr(), self.width,
                                          (self.kv_len if kv_len is None else kv_len).data_ptr(),
                                          len(self.ctx) if n_rows is None else n_rows, n_splits, 0.0,
                                          q_dev.data_ptr(), out.data_ptr(), self.stream)
        torch.cuda.synchronize()
        return rc, wl.bf16_bits_to_f32(from_dev(out))


def test_static_scratch_decode_matches_mixed_step():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    s = wl.LLAMA8B
    st = _Static(s, [1, 63, 64, 700, 2049, 5000, 130, 16], seed=77)
    b, lb = st.b, st.lb

    # call 1: the batch's own queries (the step also appends the new K/V the static call reads)
    want1, _ = oracle_step(b)
    lb.step(keep_len=True)
    ref1 = lb.output()
    rc, got1 = st.call(lb.q, 8)
    assert rc == B.TS_OK, B.ts_strerror(rc)
    _close(got1, ref1, "first call")
    assert_parity(got1, want1, "peaked", "first call against the oracle")

    # call 2, straight after: other queries, other split count, same pool
    q2_bits = wl.ValueBank(5, 1.0, 20).take(b.q.size).reshape(b.q.shape)
    q2 = to_dev(q2_bits)
    lb.q.copy_(q2)
    b.q[:] = q2_bits
    want2, _ = oracle_step(b)
    lb.step(keep_len=True)
    ref2 = lb.output()
    rc, got2 = st.call(q2, 3)
    assert rc == B.TS_OK, B.ts_strerror(rc)
    _close(got2, ref2, "second call")
    assert_parity(got2, want2, "peaked", "second call against the oracle")
    assert not np.array_equal(ref1, ref2)

    # a row whose length is outside 1 .. 16 * table_width is not processed: its output is NaN and
    # the other rows are as before
    bad_len = st.kv_len.clone()
    bad_len[2] = 0
    bad_len[5] = 16 * st.width + 1
    rc, got3 = st.call(q2, 4, kv_len=bad_len)
    assert rc == B.TS_OK
    assert np.isnan(got3[2]).all() and np.isnan(got3[5]).all()
    keep = [0, 1, 3, 4, 6, 7]
    assert_parity(got3[keep], want2[keep], "peaked", "rows next to rejected ones")

    # sizes beyond the built-in scratch are refused before anything is launched
    rc, _ = st.call(q2, 8, n_rows=257)
    assert rc == B.TS_ERR_WORKSPACE
    rc, _ = st.call(q2, 16, n_rows=256, shape=wl.LLAMA70B)
    assert rc == B.TS_ERR_WORKSPACE


@pytest.mark.parametrize("shape,ctx", [(wl.Shape(8, 2, 64), [0, 15, 16, 300, 1025]),
                                       (wl.LLAMA70B, [5, 127, 128, 3000]),
                                       (wl.Shape(16, 1, 128), [40, 700])],
                         ids=["8-2-64", "64-8-128", "16-1-128"])
def test_static_scratch_decode_other_shapes(shape, ctx):
    """head_dim 64, eight and sixteen query heads per KV head: two calls in a row with different
    split counts, each against ts_mixed_step's output and against the oracle."""
    st = _Static(shape, ctx, seed=78)
    want, _ = oracle_step(st.b)
    st.lb.step(keep_len=True)
    ref = st.lb.output()
    for n_splits in (5, 1):
        rc, got = st.call(st.lb.q, n_splits)
        assert rc == B.TS_OK, B.ts_strerror(rc)
        _close(got, ref, f"{n_splits} splits")
        assert_parity(got, want, "peaked", f"{n_splits} splits against the oracle")
