"""GPU test of the chunk-size profiler (Sec. 4.4): the measured profile goes through the C ABI's
selection and Eq. 5 / Eq. 6, and must agree with the oracle's restatement on the same points."""
import pytest
import torch

from oracle import velocity
from paper_2512_03416_b200 import profiler
from paper_2512_03416_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")


def test_profile_matches_oracle_selection():
    ctx = [300, 500, 1000, 64]
    r = profiler.profile_chunk_size(wl.LLAMA8B, ctx, [64, 128, 256], n_layers=32, tpot_slo_s=0.1, ttft_slo_s=0.25,
                                    steps=5)
    assert r["prefill_tokens"] == [64, 128, 256]
    assert all(0.0 < s < 0.1 for s in r["iteration_seconds"])        # tiny steps: far inside the SLO
    want = velocity.pick_chunk_size(r["prefill_tokens"], r["iteration_seconds"], len(ctx), 0.1)
    assert r["chunk_size"] == want == 256 + len(ctx)
    v = velocity.convertible_prefill_velocity(want, len(ctx), 0.1)
    assert abs(r["prefill_velocity_tokens_per_s"] - v) <= 1e-9 * v
    assert r["reserved_pages"] == velocity.reserved_pages(v, 0.25, 16)
    assert abs(r["reserved_bytes"] - velocity.reserved_memory(v, wl.LLAMA8B.kv_bytes_per_token, 0.25)) <= 1e-6 * v


def test_profile_stops_at_the_first_violation():
    r = profiler.profile_chunk_size(wl.LLAMA8B, [100, 200], [64, 128, 256], n_layers=32, tpot_slo_s=1e-9,
                                    ttft_slo_s=0.25, steps=3)
    assert r["prefill_tokens"] == [64]                                # the sweep ended at the first point
    assert r["chunk_size"] == 0 and r["prefill_velocity_tokens_per_s"] == 0.0 and r["reserved_pages"] == 0


def test_profile_on_the_whole_layer():
    """The same sweep with ts_layer_step as the measured step: a layer costs more than its attention."""
    ctx = [300, 500, 64]
    attn = profiler.profile_chunk_size(wl.LLAMA8B, ctx, [256], n_layers=32, tpot_slo_s=0.1, ttft_slo_s=0.25, steps=5)
    full = profiler.profile_chunk_size(wl.LLAMA8B, ctx, [256], n_layers=32, tpot_slo_s=0.1, ttft_slo_s=0.25, steps=5,
                                       layer_dims=(1024, 2048))
    assert full["step"] == "ts_layer_step" and attn["step"] == "ts_mixed_step"
    assert full["iteration_seconds"][0] > attn["iteration_seconds"][0] > 0.0
    assert full["chunk_size"] == velocity.pick_chunk_size(full["prefill_tokens"], full["iteration_seconds"], len(ctx), 0.1)
