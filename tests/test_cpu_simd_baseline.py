"""The vectorised CPU codec (benchmark baseline) against the oracle: same stream byte for byte, bit-exact decode."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.join(ROOT, "baseline", "cpu_simd"))
import enec_cpu  # noqa: E402

pytestmark = pytest.mark.skipif(not enec_cpu.available(), reason="needs AVX2 and BMI2")

TORCH = {0: torch.bfloat16, 1: torch.float16}


def words16(count, seed, dt, sigma=0.02, mean=0.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(count, generator=g) * sigma + mean).to(TORCH[dt]).view(torch.int16).numpy().view(np.uint16)


def both_ways(oracle, w, dt, threads):
    want = oracle.compress(w, dt)
    got = enec_cpu.compress(w, dt, threads)
    assert got.size == want.size and np.array_equal(got, want)
    assert np.array_equal(enec_cpu.decompress(want, dt, w.size, threads), w)


@pytest.mark.parametrize("dt", [0, 1])
@pytest.mark.parametrize("count", [0, 1, 15, 16, 17, 100, 2048, 16383, 16384, 16385, 16384 * 5 + 4097, 16384 * 33 + 7])
def test_streams_match_the_oracle(oracle, dt, count):
    both_ways(oracle, words16(count, 7 + count, dt), dt, threads=3)


@pytest.mark.parametrize("threads", [1, 2, 8])
def test_thread_count_does_not_change_the_stream(oracle, threads):
    both_ways(oracle, words16(16384 * 21 + 5, 3, 0, sigma=1.0 / 64), 0, threads)


def test_all_bit_patterns(oracle):
    for dt in (0, 1):
        w = np.random.default_rng(dt).permutation(1 << 16).astype(np.uint16)
        both_ways(oracle, w, dt, threads=4)


def test_fp32(oracle):
    g = torch.Generator().manual_seed(5)
    w = (torch.randn(16384 * 6 + 99, generator=g) * 0.02).view(torch.int32).numpy().view(np.uint32)
    both_ways(oracle, w, 2, threads=4)


def test_heavy_tails_and_constant_tensors(oracle):
    rng = np.random.default_rng(9)
    t = torch.from_numpy(rng.standard_t(3, 16384 * 4 + 11).astype(np.float32) * 0.05)
    t[::97] = 0.0
    both_ways(oracle, t.to(torch.float16).view(torch.int16).numpy().view(np.uint16), 1, threads=4)
    both_ways(oracle, np.full(16384 * 2 + 3, 0x3F80, np.uint16), 0, threads=2)


def test_damaged_header_is_refused(oracle):
    w = words16(4096, 1, 0)
    s = oracle.compress(w, 0).copy()
    s[21] = 9
    with pytest.raises(ValueError):
        enec_cpu.decompress(s, 0, w.size)
