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


@pytest.mark.parametrize("profile", ["paper", "needle"])
def test_config4_chunked_8b(profile):
    b = wl.config4(profile=profile)
    want, pool_want = oracle_step(b)
    run = GpuRun(b)
    got = run.step()
    assert_parity(got, want, profile, f"config4/{profile}")
    assert np.array_equal(run.pool(), pool_want)
