"""GPU parity for the block-wise variant (the search of Sec. 5.5 on every block's own histogram):
enec_compress_blockwise must write the oracle's stream byte for byte, and enec_decompress_blockwise must decode such
streams bit for bit and refuse damaged block tables."""
import numpy as np
import pytest
import torch

from gpu_util import status_tensor, to_dev_bytes

pytestmark = pytest.mark.gpu

TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}


def to_dev(w, dt):
    if not w.size:
        return torch.empty(0, dtype=TD[dt], device="cuda")
    return torch.from_numpy(w.view(np.int32 if dt == 2 else np.int16).copy()).cuda().view(TD[dt])


def from_dev(t, dt, like):
    return t.view(torch.int32 if dt == 2 else torch.int16).cpu().numpy().view(like.dtype)


def decode(enec, stream, dt, count):
    out = torch.full((count + 16,), 1.0, dtype=TD[dt], device="cuda")
    status = status_tensor()
    d = to_dev_bytes(stream)
    assert enec.enec_decompress_blockwise(d, d.numel(), dt, count, out, status) == 0
    torch.cuda.synchronize()
    return out, int(status.item())


def check(oracle, w, dt):
    import paper_2604_03298_b200 as enec
    count = int(w.size)
    want = oracle.compress_blockwise(w, dt)
    # decoder on the oracle's stream
    out, st = decode(enec, want, dt, count)
    assert st == 0
    assert np.array_equal(from_dev(out[:count], dt, w), w)
    assert (out[count:] == 1.0).all()
    # encoder against the oracle's stream
    cap = enec.enec_max_compressed_size_blockwise(dt, count)
    assert cap == oracle.max_compressed_size_blockwise(dt, count)
    buf = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = status_tensor()
    for _ in range(2):  # the second call finds the scratch as the first one left it
        size.zero_()
        assert enec.enec_compress_blockwise(to_dev(w, dt), dt, count, buf, cap, size, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = buf[:int(size.item())].cpu().numpy()
        assert (buf[cap:] == 0xA5).all()
        if got.size != want.size or not np.array_equal(got, want):
            k = min(got.size, want.size)
            bad = np.flatnonzero(got[:k] != want[:k])
            raise AssertionError(f"sizes {got.size}/{want.size}, first differences at {bad[:8].tolist()}, "
                                 f"header {got[:48].tolist()} / {want[:48].tolist()}")


def gaussian(count, seed, dt, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(count, generator=g) * sigma
    if dt == 2:
        return t.view(torch.int32).numpy().view(np.uint32)
    return t.to(TD[dt]).view(torch.int16).numpy().view(np.uint16)


def drifting(count, seed, dt):
    """Blocks whose exponent ranges differ (scale changes by block), so that the per-block searches disagree."""
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(count, generator=g)
    scale = torch.tensor([2.0 ** ((i * 7) % 23 - 14) for i in range((count + 16383) // 16384)])
    t = t * scale.repeat_interleave(16384)[:count]
    if dt == 2:
        return t.view(torch.int32).numpy().view(np.uint32)
    return t.to(TD[dt]).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dt", [0, 1, 2])
@pytest.mark.parametrize("count", [0, 1, 16, 17, 64, 100, 128, 2048, 5000, 8193, 16383, 16384, 16385, 16384 * 5 + 8191,
                                   16384 * 37 + 129, 16384 * 300 + 16380, 16384 * 2100 + 3])
def test_sizes_and_tails(oracle, dt, count):
    check(oracle, gaussian(count, 900 + count + dt, dt), dt)


@pytest.mark.parametrize("dt", [0, 1, 2])
def test_blocks_with_different_parameters(oracle, dt):
    w = drifting(16384 * 70 + 4097, 17 + dt, dt)
    stream = oracle.compress_blockwise(w, dt)
    entries = stream[64:64 + 16 * 71].reshape(71, 16)
    assert len({tuple(e[:3]) for e in entries}) > 3   # the searches really disagree
    check(oracle, w, dt)


@pytest.mark.parametrize("dt", [0, 1])
def test_all_bit_patterns(oracle, dt):
    w = np.random.default_rng(dt).permutation(1 << 16).astype(np.uint16)
    check(oracle, np.concatenate([w, w, w[:777]]), dt)


def test_constant_and_sparse_blocks(oracle):
    rng = np.random.default_rng(5)
    w = np.zeros(16384 * 6 + 40, dtype=np.uint16)
    w[16384:2 * 16384] = 0x3C00                              # one exponent, n = m = 1
    w[2 * 16384:3 * 16384] = rng.integers(0, 1 << 16, 16384)  # everything occupied
    w[3 * 16384 + 5] = 0x7F80                                 # a single outlier in a block of zeros
    w[4 * 16384:5 * 16384:16] = rng.integers(0x3000, 0x4000, 1024)  # one value per group
    check(oracle, w, 0)


def test_decoder_refuses_other_variants_and_damaged_tables(oracle):
    import paper_2604_03298_b200 as enec
    w = drifting(16384 * 9 + 100, 3, 0)
    count = int(w.size)
    good = oracle.compress_blockwise(w, 0)
    for other in (oracle.compress(w, 0), oracle.compress_ranked(w, 0)):
        assert decode(enec, other, 0, count)[1] == -4
    status = status_tensor()
    d = to_dev_bytes(good)
    out = torch.empty(count, dtype=torch.bfloat16, device="cuda")
    assert enec.enec_decompress(d, d.numel(), 0, count, out, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == -4
    rng = np.random.default_rng(11)
    for trial in range(40):
        bad = good.copy()
        entry = int(rng.integers(0, 11))
        byte = 64 + 16 * entry + int(rng.integers(0, 16))
        bad[byte] ^= 1 << int(rng.integers(0, 8))
        out, st = decode(enec, bad, 0, count)
        try:
            want = oracle.decompress(bad, 0, count)
        except oracle.OracleError:
            assert st == -4, (trial, entry, byte)
        else:  # the damage left a well-formed stream (of another tensor)
            assert st == 0, (trial, entry, byte)
            assert np.array_equal(from_dev(out[:count], 0, want), want)
        assert (out[count:] == 1.0).all()
