"""GPU parity: enec_decompress (through the C-ABI) on streams written by the CPU oracle must reproduce the
original tensor bit for bit (tolerance 0)."""
import numpy as np
import pytest
import torch

from gpu_util import status_tensor, tensor_of, to_dev_bytes, words_of

pytestmark = pytest.mark.gpu

DT = {0: torch.bfloat16, 1: torch.float16}


def gpu_decompress(stream_np, dt, count):
    import paper_2604_03298_b200 as enec
    d_in = to_dev_bytes(stream_np)
    out = torch.empty(count, dtype=DT[dt], device="cuda")
    # canary padding behind the output to catch out-of-range stores
    guard = torch.full((count + 64,), 0x5A5A, dtype=torch.int16, device="cuda")
    out = guard[:count].view(DT[dt])
    status = status_tensor()
    st = enec.enec_decompress(d_in, d_in.numel(), dt, count, out, status)
    torch.cuda.synchronize()
    assert (guard[count:] == 0x5A5A).all()
    return st, int(status.item()), out


def check_roundtrip(oracle, words, dt, params=None):
    stream = oracle.compress(words, dt, params)
    st, dev, out = gpu_decompress(stream, dt, words.size)
    assert (st, dev) == (0, 0)
    got = words_of(out)
    if not np.array_equal(got, words):
        bad = np.flatnonzero(got != words)
        raise AssertionError(f"{bad.size} mismatches, first at {bad[:8]}, got {got[bad[:4]]}, want {words[bad[:4]]}")


@pytest.mark.parametrize("dt", [0, 1])
@pytest.mark.parametrize("count", [0, 1, 7, 16, 17, 40, 64, 100, 128, 1000, 2048, 4096, 16383, 16384, 16385,
                                   16384 * 3 + 16, 16384 * 5 + 8191, 16384 * 37 + 129])
def test_sizes_and_tails(oracle, dt, count):
    g = torch.Generator().manual_seed(count + dt)
    w = (torch.randn(count, generator=g) * 0.02).to(DT[dt]).view(torch.int16).numpy().view(np.uint16)
    check_roundtrip(oracle, w, dt)


@pytest.mark.parametrize("n,m", [(n, m) for n in range(1, 9) for m in range(1, n + 1)])
def test_every_width_pair_bf16(oracle, n, m):
    rng = np.random.default_rng(100 * n + m)
    count = 16384 * 4 + 2048 + 40
    half = 1 << (n - 1)
    if n < 8:
        x = rng.integers(max(0, 120 - (half - 1)), min(255, 120 + half) + 1, count)
        x = np.where(rng.random(count) < 0.8, 120 - rng.integers(0, min(1 << max(m - 1, 0), half), count), x)
    else:
        x = rng.integers(0, 256, count)
        x = np.where(rng.random(count) < 0.8, 120 - rng.integers(0, 1 << (m - 1), count), x)
    words = ((x.astype(np.uint16) << 7) | rng.integers(0, 128, count).astype(np.uint16)
             | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)
    check_roundtrip(oracle, words, 0, (120, n, m))


@pytest.mark.parametrize("n,m", [(n, m) for n in range(1, 6) for m in range(1, n + 1)])
def test_every_width_pair_fp16(oracle, n, m):
    rng = np.random.default_rng(200 * n + m)
    count = 16384 * 3 + 512 + 24
    half = 1 << (n - 1)
    if n < 5:
        x = rng.integers(max(0, 12 - (half - 1)), min(31, 12 + half) + 1, count)
    else:
        x = rng.integers(0, 32, count)
    x = np.where(rng.random(count) < 0.7, 12 - rng.integers(0, min(1 << (m - 1), half), count), x)
    words = ((x.astype(np.uint16) << 10) | rng.integers(0, 1024, count).astype(np.uint16)
             | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)
    check_roundtrip(oracle, words, 1, (12, n, m))


@pytest.mark.parametrize("dt", [0, 1])
def test_all_bit_patterns(oracle, dt):
    allw = np.arange(1 << 16, dtype=np.uint16)
    rng = np.random.default_rng(5)
    check_roundtrip(oracle, allw, dt)
    check_roundtrip(oracle, rng.permutation(allw), dt)
    check_roundtrip(oracle, np.repeat(allw, 16)[:20 * 16384 + 77], dt)


def test_mask_extremes(oracle):
    # no group wide, every group wide, only first / only last group of a block wide
    count = 16384 * 3
    base = np.full(count, 123 << 7, np.uint16)
    check_roundtrip(oracle, base, 0, (123, 6, 3))
    allwide = base.copy()
    allwide[::16] = 125 << 7
    check_roundtrip(oracle, allwide, 0, (123, 6, 3))
    first = base.copy(); first[16384] = 100 << 7
    check_roundtrip(oracle, first, 0, (123, 6, 3))
    last = base.copy(); last[2 * 16384 - 1] = 126 << 7
    check_roundtrip(oracle, last, 0, (123, 6, 3))


def test_config1_gaussian(oracle):
    from paper_2604_03298_b200 import synth
    spec = synth.config_specs(1)[0]
    t = synth.make_tensor(spec, "cuda")
    check_roundtrip(oracle, words_of(t), 0)


def test_damaged_stream_reports_status(oracle):
    rng = np.random.default_rng(9)
    words = rng.integers(0x3A00, 0x3FFF, 50000).astype(np.uint16)
    s = oracle.compress(words, 0)
    for off, val in ((0, 0x58), (6, 1), (8, 1), (21, 0), (22, 9), (24, 77), (40, 3)):
        bad = s.copy(); bad[off] = val
        st, dev, _ = gpu_decompress(bad, 0, words.size)
        assert st == 0 and dev == -4, (off, st, dev)
    # table entry beyond the record count
    bad = s.copy(); bad[64 + 4:64 + 8] = 0xFF
    st, dev, _ = gpu_decompress(bad, 0, words.size)
    assert dev == -4
    st, dev, _ = gpu_decompress(s, 1, words.size)
    assert dev == -4
    st, dev, _ = gpu_decompress(s[:-16], 0, words.size)
    assert dev == -4


def test_host_argument_checks():
    import paper_2604_03298_b200 as enec
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    out = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    assert enec.enec_decompress(buf, 4096, 7, 64, out) == -2
    assert enec.enec_decompress(buf[1:], 4000, 0, 64, out) == -1
    assert enec.enec_decompress(buf, 10, 0, 64, out) == -4
    assert enec.enec_decompress(None, 4096, 0, 64, out) == -1


@pytest.mark.parametrize("b,n,m", [(250, 6, 3), (240, 5, 2), (3, 3, 1), (255, 8, 4), (200, 7, 7)])
def test_exponents_near_the_ends_of_the_field(oracle, b, n, m):
    # b + 2^(n-1) beyond 255 and b near 0: the byte arithmetic of the inverse transform must not leak between bytes
    rng = np.random.default_rng(b)
    count = 16384 * 6 + 100
    half = 1 << (n - 1)
    lo, hi = max(0, b - (half - 1)), min(255, b + half)
    x = rng.integers(lo, hi + 1, count) if n < 8 else rng.integers(0, 256, count)
    x = np.where(rng.random(count) < 0.7, np.clip(b - rng.integers(0, 1 << max(m - 1, 0), count), 0, 255), x)
    words = ((x.astype(np.uint16) << 7) | rng.integers(0, 128, count).astype(np.uint16)
             | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)
    check_roundtrip(oracle, words, 0, (b, n, m))


def test_fp16_full_width_field(oracle):
    # n = E = 5: b - y wraps modulo 32
    rng = np.random.default_rng(77)
    count = 16384 * 5 + 9
    for b in (0, 7, 31):
        x = rng.integers(0, 32, count)
        words = ((x.astype(np.uint16) << 10) | rng.integers(0, 1024, count).astype(np.uint16)
                 | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)
        for m in (1, 3, 5):
            check_roundtrip(oracle, words, 1, (b, 5, m))


@pytest.mark.parametrize("n,m", [(5, 3), (5, 1), (4, 2), (5, 4), (3, 1)])
def test_fp16_blocks_with_many_wide_groups(oracle, n, m):
    """fp16 blocks whose number of wide groups runs from below what a stage holds as sixteen-byte records, through the
    range of the eight-byte form, up to every group: one block per count, with exact per-block counts."""
    rng = np.random.default_rng(10 * n + m)
    b = 12
    wide_counts = [0, 1, 300, 392, 393, 394, 500, 610, 640, 655, 656, 657, 700, 900, 1023, 1024]
    blocks = []
    for wide in wide_counts:
        # narrow values keep y = b - x below 2^m; one element of each chosen group gets a y with a high bit set
        y = rng.integers(0, 1 << m, 16384)
        groups = rng.choice(1024, size=wide, replace=False)
        spots = groups * 16 + rng.integers(0, 16, wide)
        y[spots] = rng.integers(1 << m, 1 << (n - 1), wide) if n - 1 > m else (1 << m)
        x = (b - y) & 31
        blocks.append(((x.astype(np.uint16) << 10) | rng.integers(0, 1024, 16384).astype(np.uint16)
                       | (rng.integers(0, 2, 16384).astype(np.uint16) << 15)).astype(np.uint16))
    words = np.concatenate(blocks + [blocks[3][:5000]])
    stream = oracle.compress(words, 1, (b, n, m))
    table = np.frombuffer(stream[64:64 + 4 * (len(wide_counts) + 2)].tobytes(), dtype=np.uint32)
    assert np.diff(table)[:len(wide_counts)].tolist() == wide_counts
    check_roundtrip(oracle, words, 1, (b, n, m))
