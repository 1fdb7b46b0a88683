"""GPU parity for fp32 tensors (Sec. 6.2 "Float32 support": the exponent goes through the bf16 pipeline, the
sign and the 23 mantissa bits are kept as they are). The stream written on the GPU must equal the CPU oracle's
byte for byte; decompression must give back every 32-bit pattern (tolerance 0)."""
import numpy as np
import pytest
import torch

from gpu_util import status_tensor, to_dev_bytes

pytestmark = pytest.mark.gpu

FP32 = 2
CANARY = 0xA5


def dev_words(words):
    return torch.from_numpy(words.view(np.int32).copy()).cuda().view(torch.float32)


def host_words(t):
    return t.detach().reshape(-1).view(torch.int32).cpu().numpy().view(np.uint32)


def gpu_compress(words, params=None, entry="enec_compress"):
    import paper_2604_03298_b200 as enec
    count = int(words.size)
    d_in = dev_words(words) if count else torch.empty(0, dtype=torch.float32, device="cuda")
    cap = enec.enec_max_compressed_size(FP32, count)
    buf = torch.full((cap + 256,), CANARY, dtype=torch.uint8, device="cuda")
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = status_tensor()
    if params is None:
        st = getattr(enec, entry)(d_in, FP32, count, buf, cap, size, status)
    else:
        st = enec.enec_compress_with_params(d_in, FP32, count, *params, buf, cap, size, status)
    torch.cuda.synchronize()
    assert (buf[cap:] == CANARY).all(), "write behind the output capacity"
    return st, int(status.item()), buf[:int(size.item())].cpu().numpy()


def gpu_decompress(stream_np, count):
    import paper_2604_03298_b200 as enec
    d_in = to_dev_bytes(stream_np)
    guard = torch.full((count + 64,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    out = guard[:count].view(torch.float32)
    status = status_tensor()
    st = enec.enec_decompress(d_in, d_in.numel(), FP32, count, out, status)
    torch.cuda.synchronize()
    assert (guard[count:] == 0x5A5A5A5A).all(), "store behind the output"
    return st, int(status.item()), host_words(out)


def check(oracle, words, params=None):
    want = oracle.compress(words, FP32, params)
    # the GPU decoder on the oracle's stream
    st, dev, back = gpu_decompress(want, words.size)
    assert (st, dev) == (0, 0)
    if not np.array_equal(back, words):
        bad = np.flatnonzero(back != words)
        raise AssertionError(f"decode: {bad.size} mismatches, first at {bad[:8]}: got {back[bad[:4]]} want {words[bad[:4]]}")
    # the GPU encoder against the oracle's stream
    st, dev, got = gpu_compress(words, params)
    assert (st, dev) == (0, 0)
    if got.size != want.size or not np.array_equal(got, want):
        if got.size != want.size:
            raise AssertionError(f"encode: size {got.size} != {want.size}; header {got[:48].tolist()} / {want[:48].tolist()}")
        bad = np.flatnonzero(got != want)
        raise AssertionError(f"encode: {bad.size} bytes differ, first at {bad[:8].tolist()}")


def gaussian_words(count, seed, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(count, generator=g) * sigma).view(torch.int32).numpy().view(np.uint32)


@pytest.mark.parametrize("count", [0, 1, 7, 16, 17, 40, 64, 100, 128, 129, 1000, 2048, 4096, 5000, 16383, 16384, 16385,
                                   16384 * 3 + 16, 16384 * 5 + 8191, 16384 * 37 + 129, 16384 * 600 + 3])
def test_sizes_and_tails(oracle, count):
    check(oracle, gaussian_words(count, 1000 + count))


def field_words(rng, count, center, n, m):
    half = 1 << (n - 1)
    if n < 8:
        x = rng.integers(max(0, center - (half - 1)), min(255, center + half) + 1, count)
    else:
        x = rng.integers(0, 256, count)
    narrow = center - rng.integers(0, min(1 << (m - 1), half), count)
    x = np.where(rng.random(count) < 0.8, narrow, x)
    return ((x.astype(np.uint32) << 23) | rng.integers(0, 1 << 23, count).astype(np.uint32)
            | (rng.integers(0, 2, count).astype(np.uint32) << 31)).astype(np.uint32)


@pytest.mark.parametrize("n,m", [(n, m) for n in range(1, 9) for m in range(1, n + 1)])
def test_every_width_pair(oracle, n, m):
    rng = np.random.default_rng(100 * n + m)
    check(oracle, field_words(rng, 16384 * 3 + 777, 124, n, m), (124, n, m))


@pytest.mark.parametrize("count", [16, 24, 33, 64, 100, 16384 + 50])
@pytest.mark.parametrize("n,m", [(3, 1), (6, 3), (8, 8)])
def test_short_tail_blocks_with_params(oracle, n, m, count):
    rng = np.random.default_rng(count * 10 + n)
    check(oracle, field_words(rng, count, 126, n, m), (126, n, m))


def test_every_high_half_pattern(oracle):
    """Every sign/exponent/mantissa-top pattern once, with random low halves: infinities, NaNs, zeros, subnormals."""
    rng = np.random.default_rng(5)
    hi = rng.permutation(1 << 16).astype(np.uint32)
    check(oracle, (hi << 16) | rng.integers(0, 1 << 16, hi.size).astype(np.uint32))


def test_low_halves_survive_bit_for_bit(oracle):
    """Low halves 0x0000 .. 0xFFFF under a constant high half (one exponent: n = m = 1)."""
    lo = np.arange(1 << 16, dtype=np.uint32)
    check(oracle, np.uint32(0x3F800000) | lo)


def test_device_parameter_search(oracle):
    """The parameters the device picks are the oracle's (header bytes 20..22) on a wide, skewed histogram."""
    w = np.concatenate([gaussian_words(200_000, 7, 0.02), gaussian_words(3_000, 8, 30.0), gaussian_words(500, 9, 1e-12)])
    want = oracle.compress(w, FP32)
    st, dev, got = gpu_compress(w)
    assert (st, dev) == (0, 0)
    assert got[20:23].tolist() == want[20:23].tolist()
    assert np.array_equal(got, want)


def test_noalloc_entry_point(oracle):
    w = gaussian_words(16384 * 9 + 5, 11)
    st, dev, got = gpu_compress(w, entry="enec_compress_noalloc")
    assert (st, dev) == (0, 0)
    assert np.array_equal(got, oracle.compress(w, FP32))


def test_batched_decompress(oracle):
    import paper_2604_03298_b200 as enec
    counts = [16384 * 4, 100, 16384 * 2 + 9, 16]
    ws = [gaussian_words(c, 20 + i) for i, c in enumerate(counts)]
    streams = [to_dev_bytes(oracle.compress(w, FP32)) for w in ws]
    outs = [torch.zeros(c, dtype=torch.float32, device="cuda") for c in counts]
    status = status_tensor()
    items = [(s, s.numel(), o, c) for s, o, c in zip(streams, outs, counts)]
    assert enec.enec_decompress_batched(items, FP32, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for w, o in zip(ws, outs):
        assert np.array_equal(host_words(o), w)


def test_stream_of_another_dtype_is_refused(oracle):
    """An fp32 stream handed over as bf16 (and the reverse) ends with a bad-stream status, not with output."""
    import paper_2604_03298_b200 as enec
    w = gaussian_words(16384, 3)
    s = to_dev_bytes(oracle.compress(w, FP32))
    out = torch.zeros(16384, dtype=torch.bfloat16, device="cuda")
    status = status_tensor()
    assert enec.enec_decompress(s, s.numel(), 0, 16384, out, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == -4


def test_ratio_of_gaussian_weights(oracle):
    """Table 4 reports about 1.15 for fp32 models: exponent bits saved over 32 bits per value."""
    import paper_2604_03298_b200 as enec
    t = torch.randn(4096 * 1024, generator=torch.Generator().manual_seed(1)) * 0.02
    stream = enec.compress_tensor(t.cuda())
    ratio = t.numel() * 4 / stream.numel()
    assert 1.12 < ratio < 1.20
    back = enec.decompress_tensor(stream, torch.float32, t.shape)
    assert torch.equal(back.view(torch.int32).cpu(), t.view(torch.int32))


def test_buffers_on_odd_sixteen_byte_boundaries(oracle):
    """Input and output that start 16 bytes behind a 32-byte boundary take the paths with 16-byte accesses."""
    import paper_2604_03298_b200 as enec
    count = 16384 * 5 + 300
    w = gaussian_words(count, 31)
    want = oracle.compress(w, FP32)
    holder = torch.zeros(count + 4, dtype=torch.float32, device="cuda")
    assert holder.data_ptr() % 32 == 0
    d_in = holder[4:]
    d_in.copy_(dev_words(w))
    cap = enec.enec_max_compressed_size(FP32, count)
    buf = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = status_tensor()
    assert enec.enec_compress(d_in, FP32, count, buf, cap, size, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = buf[:int(size.item())].cpu().numpy()
    assert np.array_equal(got, want)
    out_holder = torch.full((count + 8,), 7.0, dtype=torch.float32, device="cuda")
    out = out_holder[4:4 + count]
    assert enec.enec_decompress(buf, cap, FP32, count, out, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(host_words(out), w)
    assert (out_holder[:4] == 7.0).all() and (out_holder[4 + count:] == 7.0).all()
