"""GPU parity for the frequency-rank variant (Sec. 4.2, Algorithm 1; the ablation's V1): enec_compress_ranked must
write the oracle's stream byte for byte, and enec_decompress_ranked must decode such streams bit for bit."""
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


def check(oracle, w, dt):
    import paper_2604_03298_b200 as enec
    count = int(w.size)
    want = oracle.compress_ranked(w, dt)
    # decoder on the oracle's stream
    out = torch.full((count + 16,), 1.0, dtype=TD[dt], device="cuda")
    status = status_tensor()
    d_want = to_dev_bytes(want)
    assert enec.enec_decompress_ranked(d_want, d_want.numel(), dt, count, out, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(from_dev(out[:count], dt, w), w)
    assert (out[count:] == 1.0).all()
    # encoder against the oracle's stream
    cap = enec.enec_max_compressed_size_ranked(dt, count)
    assert cap == enec.enec_max_compressed_size(dt, count) + 256
    buf = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    assert enec.enec_compress_ranked(to_dev(w, dt), dt, count, buf, cap, size, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = buf[:int(size.item())].cpu().numpy()
    assert (buf[cap:] == 0xA5).all()
    if got.size != want.size or not np.array_equal(got, want):
        bad = np.flatnonzero(got[:min(got.size, want.size)] != want[:min(got.size, want.size)])
        raise AssertionError(f"sizes {got.size}/{want.size}, first differences at {bad[:8].tolist()}, header {got[:48].tolist()} / {want[:48].tolist()}")


def gaussian(count, seed, dt, sigma=0.02):
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(count, generator=g) * sigma
    if dt == 2:
        return t.view(torch.int32).numpy().view(np.uint32)
    return t.to(TD[dt]).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dt", [0, 1, 2])
@pytest.mark.parametrize("count", [0, 1, 16, 17, 64, 100, 128, 2048, 5000, 16383, 16384, 16385, 16384 * 5 + 8191,
                                   16384 * 37 + 129, 16384 * 300 + 3])
def test_sizes_and_tails(oracle, dt, count):
    check(oracle, gaussian(count, 500 + count + dt, dt), dt)


@pytest.mark.parametrize("dt", [0, 1])
def test_all_bit_patterns(oracle, dt):
    """Every exponent occupied: n = E, the table is a full permutation."""
    w = np.random.default_rng(dt).permutation(1 << 16).astype(np.uint16)
    check(oracle, np.concatenate([w, w[:777]]), dt)


def test_skewed_histograms_and_ties(oracle):
    rng = np.random.default_rng(3)
    for k in (1, 2, 3, 5, 9, 17, 33, 70, 130):           # number of occupied exponents -> n = 1 .. 8
        expo = rng.choice(np.arange(20, 230), size=k, replace=False)
        p = rng.random(k) ** 3 + 1e-3
        x = rng.choice(expo, size=16384 * 6 + 555, p=p / p.sum()).astype(np.uint16)
        w = (x << 7) | rng.integers(0, 128, x.size).astype(np.uint16) | (rng.integers(0, 2, x.size).astype(np.uint16) << 15)
        check(oracle, w.astype(np.uint16), 0)
    flat = np.repeat(np.arange(100, 116, dtype=np.uint16), 4096)   # sixteen exponents with equal counts: all ties
    check(oracle, (flat << 7).astype(np.uint16), 0)


def test_heavy_tails_with_zeros_fp16(oracle):
    rng = np.random.default_rng(6)
    t = torch.from_numpy(rng.standard_t(3, 16384 * 9 + 40).astype(np.float32) * 0.05)
    t[::53] = 0.0
    check(oracle, t.to(torch.float16).view(torch.int16).numpy().view(np.uint16), 1)


def test_each_decoder_refuses_the_other_kind_of_stream(oracle):
    import paper_2604_03298_b200 as enec
    w = gaussian(16384 * 2 + 77, 70, 0)
    ranked, linear = to_dev_bytes(oracle.compress_ranked(w, 0)), to_dev_bytes(oracle.compress(w, 0))
    out = torch.zeros(w.size, dtype=torch.bfloat16, device="cuda")
    for fn, stream in ((enec.enec_decompress, ranked), (enec.enec_decompress_ranked, linear)):
        status = status_tensor()
        assert fn(stream, stream.numel(), 0, w.size, out, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == -4
    status = status_tensor()
    assert enec.enec_decompress_batched([(ranked, ranked.numel(), out, w.size)], 0, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == -4


def test_ranked_and_linear_calls_alternate_on_one_stream(oracle):
    """Both variants share the compressor's scratch area and its call numbering."""
    import paper_2604_03298_b200 as enec
    status = status_tensor()
    jobs = []
    for i, count in enumerate([16384 * 4 + 9, 300, 16384 * 12, 16384 * 2 + 1, 70000, 16]):
        w = gaussian(count, 90 + i, 0, sigma=0.02 * (1 + i))
        ranked = i % 2 == 0
        cap = enec.enec_max_compressed_size_ranked(0, count)
        buf = torch.empty(cap, dtype=torch.uint8, device="cuda")
        size = torch.zeros(1, dtype=torch.int64, device="cuda")
        fn = enec.enec_compress_ranked if ranked else enec.enec_compress
        d_in = to_dev(w, 0)
        assert fn(d_in, 0, count, buf, cap, size, status) == 0
        jobs.append((w, ranked, buf, size, d_in))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for w, ranked, buf, size, _ in jobs:
        want = oracle.compress_ranked(w, 0) if ranked else oracle.compress(w, 0)
        assert np.array_equal(buf[:int(size.item())].cpu().numpy(), want)
