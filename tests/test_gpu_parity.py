"""GPU parity: ts_mixed_step / ts_kv_append through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2512_03416_b200 import workloads as wl
from tests.helpers import GpuRun, assert_parity, oracle_step

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")


@pytest.mark.parametrize("profile", ["paper", "peaked", "needle"])
def test_config1_tiny_mixed(profile):
    b = wl.config1(profile=profile)
    want, pool_want = oracle_step(b)
    run = GpuRun(b)
    got = run.step()
    assert_parity(got, want, profile, f"config1/{profile}")
    assert np.array_equal(run.pool(), pool_want), "pool differs after append"


@pytest.mark.parametrize("profile", ["paper", "peaked", "needle"])
def test_config2_decode_8b(profile):
    b = wl.config2(profile=profile)
    want, pool_want = oracle_step(b)
    run = GpuRun(b)
    got = run.step()
    assert_parity(got, want, profile, f"config2/{profile}")
    assert np.array_equal(run.pool(), pool_want)


CASES = [
    # (Hq, Hkv, D, ctx list, q_len list)
    (4, 2, 64, [1, 15, 16, 17], [1, 1, 1, 1]),
    (8, 1, 128, [255, 256, 257, 0], [1, 1, 1, 1]),
    (8, 8, 64, [0, 3], [2, 17]),
    (16, 2, 128, [0, 31, 100], [64, 130, 1]),
    (6, 2, 64, [5, 77], [33, 1]),
    (32, 8, 128, [700, 0, 1300], [1, 200, 1]),
    (64, 8, 128, [513, 64], [1, 96]),
    (2, 2, 128, [0], [1]),
    (12, 4, 64, [19], [300]),
    (16, 1, 64, [40, 41], [1, 5]),
    # head_dim 128 with group sizes that do not divide 128 (query tiles of 126, 125, 126, 120 packed rows)
    (24, 8, 128, [300, 0, 77], [1, 200, 1]),
    (40, 8, 128, [33, 5], [1, 150]),
    (48, 8, 128, [129, 600, 18], [140, 1, 1]),
    (7, 1, 128, [0, 260], [90, 1]),
    (12, 1, 128, [70, 15, 0], [1, 1, 75]),
    # sixteen query heads per KV head at head_dim 128: 8-token query tiles, the decode rows in a
    # launch of their own (two head groups per unit) followed by the split merge
    (16, 1, 128, [900, 0, 4500, 31], [1, 70, 1, 1]),
    (32, 2, 128, [257, 5000, 12], [1, 1, 100]),
    (32, 2, 128, [255, 256, 4700, 0], [1, 1, 1, 1]),
    (16, 1, 128, [4200, 63], [1, 1]),
]


@pytest.mark.parametrize("case", CASES, ids=[f"{c[0]}-{c[1]}-{c[2]}-{i}" for i, c in enumerate(CASES)])
@pytest.mark.parametrize("profile", ["peaked", "needle"])
def test_shape_sweep(case, profile):
    Hq, Hkv, D, ctx, ql = case
    b = wl.make_batch("sweep", wl.Shape(Hq, Hkv, D), ctx, ql, seed=hash(case[:3]) % 1000 + len(ctx), profile=profile)
    want, pool_want = oracle_step(b)
    run = GpuRun(b, chunk_size=0)
    got = run.step()
    assert_parity(got, want, profile, f"sweep {case}")
    assert np.array_equal(run.pool(), pool_want)


def test_empty_step_launches_nothing():
    b = wl.make_batch("e", wl.TINY, [3], [1], seed=3)
    run = GpuRun(b)
    before = run.dec.velocity()
    run.dec.mixed_step([], [], [], None, None, None, None)
    after = run.dec.velocity()
    assert after["kernel_launches"] == before["kernel_launches"] and after["steps"] == before["steps"]


@pytest.mark.parametrize("split", [64, 128, 192, 1024, 1 << 20])
def test_split_count_invariance(split):
    b = wl.make_batch("s", wl.LLAMA8B, [1000, 63, 64, 4095], [1, 1, 1, 1], seed=9, profile="peaked")
    want, _ = oracle_step(b)
    got = GpuRun(b, decode_split_tokens=split).step()
    assert_parity(got, want, "peaked", f"split {split}")


@pytest.mark.parametrize("profile", ["paper", "peaked", "needle"])
def test_config3_burst_8b(profile):
    b = wl.config3(profile=profile)
    want, pool_want = oracle_step(b)
    run = GpuRun(b)
    got = run.step()
    assert_parity(got, want, profile, f"config3/{profile}")
    assert np.array_equal(run.pool(), pool_want)


@pytest.mark.parametrize("profile", ["paper", "peaked", "needle"])
def test_config4_chunked_8b(profile):
    b = wl.config4(profile=profile)
    want, pool_want = oracle_step(b)
    run = GpuRun(b)
    got = run.step()
    assert_parity(got, want, profile, f"config4/{profile}")
    assert np.array_equal(run.pool(), pool_want)


@pytest.mark.parametrize("prefill_ctas", [-1, 0, 1, 3, 100, 1000])
def test_mixed_launch_split_invariance(prefill_ctas):
    """The result does not depend on how the attention launch divides its CTAs between prefill
    tiles and decode rows: two launches (-1), the cost model (0), one or three prefill CTAs (the
    decode CTAs then take most tiles from the queue, many work units per CTA), or more prefill
    CTAs than there are SMs (clamped)."""
    b = wl.make_batch("mix", wl.LLAMA8B, [700, 50, 1300, 3000, 9, 0, 200], [1, 1, 1, 1, 1, 600, 130], seed=21,
                      profile="peaked")
    want, pool_want = oracle_step(b)
    run = GpuRun(b, chunk_size=0, mixed_prefill_ctas=prefill_ctas)
    got = run.step()
    assert_parity(got, want, "peaked", f"mixed launch, prefill_ctas={prefill_ctas}")
    assert np.array_equal(run.pool(), pool_want)


def test_prefill_only_many_units_per_cta():
    """A prefill-only step with more work units (tile pairs x KV heads) than SMs: every CTA of the
    persistent kernel walks through several units, and the units differ in length."""
    b = wl.make_batch("pf", wl.LLAMA8B, [37, 0], [1300, 75], seed=22, profile="needle")
    want, pool_want = oracle_step(b)
    run = GpuRun(b, chunk_size=0)
    got = run.step()
    assert_parity(got, want, "needle", "prefill-only, many units")
    assert np.array_equal(run.pool(), pool_want)


def test_mixed_70b_shape_group8():
    """Eight query heads per KV head (the 70B-shaped layer): 16-token query tiles, decode rows in the same launch."""
    b = wl.make_batch("m70", wl.LLAMA70B, [900, 17, 2500, 0], [1, 1, 1, 200], seed=23, profile="peaked")
    want, pool_want = oracle_step(b)
    run = GpuRun(b, chunk_size=0)
    got = run.step()
    assert_parity(got, want, "peaked", "70B-shaped mixed step")
    assert np.array_equal(run.pool(), pool_want)


def test_maximum_sizes_sampled():
    """The largest shapes the workloads allow (70B-shaped layer): a decode row whose context fills
    a 2048-page block table (32768 tokens with its new one) and an 8192-token prefill chunk that
    continues 24576 cached tokens, so its last token also sees 32768 keys. The oracle checks every
    decode row and a sample of the chunk (its first and last tokens, the edges of every 128-token
    stretch and 200 seeded tokens); the pool is compared in full."""
    b = wl.make_batch("max", wl.LLAMA70B, [32767, 24576, 15], [1, 8192, 1], seed=31, profile="peaked",
                      chunk_size=8194)
    rng = np.random.default_rng(2)
    chunk = 1 + np.unique(np.concatenate([[0, 8191], np.arange(0, 8192, 128), np.arange(127, 8192, 128),
                                          rng.integers(0, 8192, 200)]))
    sel = np.concatenate([[0], chunk, [8193]]).astype(np.int32)
    want, pool_want = oracle_step(b, sel=sel)
    run = GpuRun(b)
    got = run.step()[sel]
    assert_parity(got, want, "peaked", "maximum sizes")
    assert np.array_equal(run.pool(), pool_want)


def test_a_wait_that_runs_out_is_reported_and_the_next_step_is_clean():
    """Failure path without a fault: with TS_DEBUG_LOSE_APPEND_ARRIVAL the barrier after the KV
    append of a mixed step waits for one thread block more than the launch has, under a limit of
    2 million clock cycles (about a millisecond; never the library's default second). Every block
    then gives that wait up, raises TS_DEV_TIMEOUT and carries on. The step must return, the status
    call must report TS_ERR_DEVICE_TIMEOUT once and then be clean, and a normal context's next
    step on the same device must match the oracle, pool included."""
    from paper_2512_03416_b200 import binding as B
    b = wl.make_batch("tmo", wl.LLAMA8B, [300, 40, 0], [1, 1, 300], seed=41, profile="peaked")
    want, pool_want = oracle_step(b)
    run = GpuRun(b, chunk_size=0, wait_limit_cycles=2_000_000, debug_flags=B.TS_DEBUG_LOSE_APPEND_ARRIVAL)
    run.lb.step(keep_len=True)
    rc, bits = B.ts_last_device_status(run.dec.ctx, torch.cuda.current_stream().cuda_stream)
    assert rc == B.TS_ERR_DEVICE_TIMEOUT and bits & B.TS_DEV_TIMEOUT
    # all blocks had in fact arrived, so even this step's result is complete
    assert_parity(run.lb.output(), want, "peaked", "step whose append barrier gave up")
    rc, bits = B.ts_last_device_status(run.dec.ctx, torch.cuda.current_stream().cuda_stream)
    assert rc == B.TS_OK and bits == 0, "the status word was not cleared"
    # the launch's counters are back at zero: the same context runs the step again, still flagged
    run.lb.step(keep_len=True)
    assert run.dec.device_status() == B.TS_DEV_TIMEOUT
    run.dec.close()
    # and a context without the flag is clean
    ok = GpuRun(b, chunk_size=0)
    got = ok.step()
    assert_parity(got, want, "peaked", "step after a timed-out one")
    assert np.array_equal(ok.pool(), pool_want)

