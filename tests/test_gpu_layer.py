"""GPU parity of the decoder layer around attention: the projection GEMM by itself and the whole
ts_layer_step, through the C ABI, against the fp64 layer oracle (oracle/layer.py)."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import layer as OL
from paper_2512_03416_b200 import binding as B
from paper_2512_03416_b200 import workloads as wl
from paper_2512_03416_b200.harness import LoadedBatch, from_dev, to_dev
from paper_2512_03416_b200.layer import DecoderLayer

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")


def bits(rng, shape, std):
    return wl.f32_to_bf16_bits((rng.standard_normal(shape) * std).astype(np.float32))


def assert_close_bf16(got_bits, want_f64, what, ulps=1.0):
    """A bf16 result of an fp32-accumulated sum against the fp64 value of the same sum: within `ulps`
    bf16 spacings (2^-8 relative each, for a value just above a power of two) of the exact value,
    plus the accumulation error, which is far below that."""
    got = OL.bits_to_f64(got_bits)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    scale = float(np.abs(want_f64).max())
    err = np.abs(got - want_f64)
    tol = ulps * 2.0 ** -8 * np.abs(want_f64) + 1e-4 * scale
    bad = err > tol
    assert not bad.any(), f"{what}: {int(bad.sum())} of {bad.size} outside tolerance, worst {float((err / (np.abs(want_f64) + 1e-4 * scale)).max())}"


GEMM_CASES = [
    # M, N, K, residual
    (1, 256, 64, False),
    (130, 512, 192, True),
    (300, 264, 72, False),        # N and K only multiples of 8: ragged last tile column and K block
    (257, 768, 1024, True),
    (2112, 1024, 4096, False),    # the 8B-shaped projections' row count and depth
]


@pytest.mark.parametrize("tile_m", [128, 256])
@pytest.mark.parametrize("case", GEMM_CASES, ids=[f"{c[0]}x{c[1]}x{c[2]}" for c in GEMM_CASES])
def test_gemm_matches_the_oracle(case, tile_m):
    M, N, K, with_r = case
    rng = np.random.default_rng(M * 7 + N + K)
    a, w = bits(rng, (M, K), 1.0), bits(rng, (N, K), 1.0 / math.sqrt(K))
    r = bits(rng, (M, N), 1.0) if with_r else None
    want = OL.gemm(OL.bits_to_f64(a), OL.bits_to_f64(w))
    if with_r:
        want = want + OL.bits_to_f64(r)
    da, dw = to_dev(a), to_dev(w)
    dr = to_dev(r) if with_r else None
    dc = torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = B.ts_gemm_bf16(0, M, N, K, da.data_ptr(), dw.data_ptr(), dr.data_ptr() if with_r else 0, dc.data_ptr(), tile_m,
                        status.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == B.TS_OK, B.ts_strerror(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_close_bf16(from_dev(dc), want, f"gemm {case} tile_m {tile_m}")


def test_gemm_rejects_bad_arguments():
    t = torch.zeros(64, dtype=torch.int16, device="cuda")
    s = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert B.ts_gemm_bf16(0, 8, 12, 64, t.data_ptr(), t.data_ptr(), 0, t.data_ptr(), 0, s.data_ptr(), st) == B.TS_ERR_INVALID
    assert B.ts_gemm_bf16(0, 8, 16, 60, t.data_ptr(), t.data_ptr(), 0, t.data_ptr(), 0, s.data_ptr(), st) == B.TS_ERR_INVALID
    assert B.ts_gemm_bf16(0, 8, 16, 64, t.data_ptr(), t.data_ptr(), 0, t.data_ptr(), 64, s.data_ptr(), st) == B.TS_ERR_INVALID
    assert B.ts_gemm_bf16(0, 0, 16, 64, t.data_ptr(), t.data_ptr(), 0, t.data_ptr(), 0, s.data_ptr(), st) == B.TS_OK


def make_weights(rng, s, hidden, inter):
    qd, kvd = s.Hq * s.D, s.Hkv * s.D
    return dict(w_norm1=bits(rng, (hidden,), 0.1) + np.uint16(0), w_qkv=bits(rng, (qd + 2 * kvd, hidden), 1.0 / math.sqrt(hidden)),
                w_o=bits(rng, (hidden, qd), 1.0 / math.sqrt(qd)), w_norm2=bits(rng, (hidden,), 0.1),
                w_gate=bits(rng, (inter, hidden), 1.0 / math.sqrt(hidden)), w_up=bits(rng, (inter, hidden), 1.0 / math.sqrt(hidden)),
                w_down=bits(rng, (hidden, inter), 1.0 / math.sqrt(inter)))


@pytest.mark.parametrize("shape,hidden,inter,ctx,ql", [
    (wl.Shape(4, 2, 128), 256, 384, [40, 0, 7], [1, 150, 1]),
    (wl.Shape(8, 2, 128), 512, 1024, [300, 17, 33], [1, 1, 200]),
], ids=["4-2-128", "8-2-128"])
def test_layer_step_matches_the_oracle(shape, hidden, inter, ctx, ql):
    """One layer iteration over decode rows and a prefill chunk: output and KV pages against the fp64
    layer oracle, whose attention is the paged-attention oracle on the oracle's own pool."""
    s = shape
    rng = np.random.default_rng(hidden + inter)
    b = wl.make_batch("layer", s, ctx, ql, seed=91, profile="peaked", chunk_size=sum(ql))
    wt = make_weights(rng, s, hidden, inter)
    for k in ("w_norm1", "w_norm2"):                      # gains around 1
        wt[k] = wl.f32_to_bf16_bits((1.0 + wl.bf16_bits_to_f32(wt[k])).astype(np.float32))
    N = b.n_tokens
    x = bits(rng, (N, hidden), 1.0)
    pos = OL.positions(b.ctx_len, b.q_len)
    # oracle: its own pool with the cached context, attention through the C oracle
    pool = b.fresh_pool()
    tm = b.table_matrix()
    if int(b.ctx_len.sum()) > 0:
        oracle.kv_append(pool, s.Hkv, s.D, s.P, tm, np.zeros_like(b.ctx_len), b.ctx_len, b.context_k, b.context_v)

    def attention(q, k, v):
        return oracle.mixed_step(pool, s.Hq, s.Hkv, s.D, s.P, 1.0 / math.sqrt(s.D), tm, b.ctx_len, b.q_len, q, k, v)

    want_bits, mid = OL.layer_step(attention, x, wt, pos, s.Hq, s.Hkv, s.D, eps=1e-5, theta=500000.0)
    want = OL.bits_to_f64(want_bits)
    # the library
    lb = LoadedBatch(b)
    dev = {k: to_dev(v) for k, v in wt.items()}
    layer = DecoderLayer(lb.dec, dev["w_norm1"], dev["w_qkv"], dev["w_o"], dev["w_norm2"], dev["w_gate"], dev["w_up"],
                         dev["w_down"], max_position=4096, rms_eps=1e-5, rope_theta=500000.0)
    x_in = to_dev(x)
    x_out = torch.full((N, hidden), 0x7FC0, dtype=torch.int16, device="cuda")
    layer.step(lb.slots, b.q_len.tolist(), b.ctx_len.tolist(), x_in, x_out)
    torch.cuda.synchronize()
    assert lb.dec.device_status() == 0
    got = OL.bits_to_f64(from_dev(x_out))
    assert np.isfinite(got).all()
    # Tolerance: the output is a sum of the input and two projections, each a chain of bf16 tensors
    # (q/k/v -> attention -> y -> g, u -> z): a one-spacing difference early in the chain shows
    # up as a few spacings at the end. Bound: 2^-6 of the largest output, and 2 % per token in L2.
    err = np.abs(got - want)
    assert err.max() <= 2.0 ** -6 * np.abs(want).max(), (err.max(), np.abs(want).max())
    rel = np.linalg.norm(got - want, axis=1) / np.linalg.norm(want, axis=1)
    assert rel.max() <= 2e-2, rel.max()
    # pages: the new K (rotated) and V sit where the oracle put them, to one bf16 spacing; every
    # other slot is untouched
    got_pool, want_pool = lb.pool(), pool
    same = got_pool == want_pool
    gp, wp = OL.bits_to_f64(got_pool[~same]), OL.bits_to_f64(want_pool[~same])
    assert np.isfinite(wp).all() and np.isfinite(gp).all(), "a dead slot was written, or a live one was not"
    assert (np.abs(gp - wp) <= 2.0 ** -7 * np.abs(wp) + 1e-3).all()
    assert (~same).mean() < 0.2                            # most values round the same way
    layer.close()


def test_layer_step_validation_launches_nothing():
    s = wl.Shape(4, 2, 128)
    b = wl.make_batch("v", s, [5], [1], seed=3, chunk_size=8)
    lb = LoadedBatch(b)
    rng = np.random.default_rng(1)
    dev = {k: to_dev(v) for k, v in make_weights(rng, s, 256, 384).items()}
    layer = DecoderLayer(lb.dec, dev["w_norm1"], dev["w_qkv"], dev["w_o"], dev["w_norm2"], dev["w_gate"], dev["w_up"],
                         dev["w_down"], max_position=5)        # the row reaches position 5: one past the table
    x = torch.zeros((1, 256), dtype=torch.int16, device="cuda")
    out = torch.zeros_like(x)
    before = lb.dec.velocity()
    st, _keep = layer.make_step(lb.slots, [1], [5])
    stream = torch.cuda.current_stream().cuda_stream
    assert B.ts_layer_step(layer.handle, st, x.data_ptr(), out.data_ptr(), stream) == B.TS_ERR_INVALID
    st2, _keep2 = layer.make_step(lb.slots, [1], [4])            # wrong cached length
    assert B.ts_layer_step(layer.handle, st2, x.data_ptr(), out.data_ptr(), stream) == B.TS_ERR_INVALID
    after = lb.dec.velocity()
    assert after["kernel_launches"] == before["kernel_launches"] and after["steps"] == before["steps"]
    layer.close()
