"""ts_decode_attention_static against ts_mixed_step.

The static entry point is for callers that cannot hand the library a workspace because they
cannot allocate device memory where they run (all of HBM already claimed by their framework,
no permission to own memory, or no tolerance for an allocation's synchronisation). It keeps its
split partials in an array built into the library. This test feeds both entry points the same
decode batch through the C ABI and requires the same answers, on two calls in a row: the second
call uses other queries and another split count, so stale contents of the shared array would show.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2512_03416_b200 import binding as B
from paper_2512_03416_b200 import workloads as wl
from paper_2512_03416_b200.harness import LoadedBatch, from_dev, to_dev

pytestmark = pytest.mark.gpu


def _close(a, b, what):
    d = np.abs(a.astype(np.float64) - b.astype(np.float64))
    assert np.isfinite(a).all(), f"{what}: non-finite output"
    assert d.max() <= 2e-2 and d.mean() <= 2e-3, f"{what}: max {d.max()} mean {d.mean()}"
    peak = np.abs(b).max()
    assert d.max() <= 2.0 ** -7 * peak + 1e-6, f"{what}: max {d.max()} vs peak {peak}"


def test_static_scratch_decode_matches_mixed_step():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    s = wl.LLAMA8B
    ctx = [1, 63, 64, 700, 2049, 5000, 130, 16]
    b = wl.make_batch("static", s, ctx, [1] * len(ctx), seed=77, profile="peaked")
    lb = LoadedBatch(b)
    width = max(len(t) for t in b.tables)
    tables = torch.from_numpy(np.maximum(b.table_matrix(width), 0)).cuda()
    kv_len = torch.tensor([c + 1 for c in ctx], dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def static_call(q_dev, n_splits):
        out = torch.full((len(ctx), s.Hq, s.D), 0x7FC0, dtype=torch.int16, device="cuda")
        rc = B.ts_decode_attention_static(0, s.Hq, s.Hkv, s.D, b.n_pages, lb.dec.pool.data_ptr(),
                                          tables.data_ptr(), width, kv_len.data_ptr(), len(ctx), n_splits,
                                          0.0, q_dev.data_ptr(), out.data_ptr(), stream)
        assert rc == B.TS_OK, B.ts_strerror(rc)
        torch.cuda.synchronize()
        return wl.bf16_bits_to_f32(from_dev(out))

    # call 1: the batch's own queries (the step also appends the new K/V the static call reads)
    lb.step(keep_len=True)
    ref1 = lb.output()
    got1 = static_call(lb.q, 8)
    _close(got1, ref1, "first call")

    # call 2, straight after: other queries, other split count, same pool
    q2 = to_dev(wl.ValueBank(5, 1.0, 20).take(b.q.size).reshape(b.q.shape))
    lb.q.copy_(q2)
    lb.step(keep_len=True)
    ref2 = lb.output()
    got2 = static_call(q2, 3)
    _close(got2, ref2, "second call")
    assert not np.array_equal(ref1, ref2)

    # sizes beyond the built-in scratch are refused before anything is launched
    rc = B.ts_decode_attention_static(0, s.Hq, s.Hkv, s.D, b.n_pages, lb.dec.pool.data_ptr(),
                                      tables.data_ptr(), width, kv_len.data_ptr(), 257, 8, 0.0,
                                      q2.data_ptr(), q2.data_ptr(), stream)
    assert rc == B.TS_ERR_WORKSPACE
    rc = B.ts_decode_attention_static(0, 64, 8, 128, b.n_pages, lb.dec.pool.data_ptr(), tables.data_ptr(),
                                      width, kv_len.data_ptr(), 256, 16, 0.0, q2.data_ptr(), q2.data_ptr(), stream)
    assert rc == B.TS_ERR_WORKSPACE
