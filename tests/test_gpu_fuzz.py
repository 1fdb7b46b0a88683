"""Seeded random cases, GPU against the oracle: random dtype, size (0 .. 600 K values, around block boundaries),
value distribution (Gaussian at random scales, Student-t, shifted, with zeros, constant, random bit patterns) and
entry point (single, allocation-free, batched, frequency-rank, block-wise). Streams byte for byte, decoded tensors bit for bit."""
import numpy as np
import pytest
import torch

from gpu_util import status_tensor

pytestmark = pytest.mark.gpu

TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}


def draw(rng, dt, count):
    kind = rng.integers(0, 6)
    if kind == 0:
        f = rng.standard_normal(count).astype(np.float32) * float(10.0 ** rng.uniform(-4, 1))
    elif kind == 1:
        f = rng.standard_t(3, count).astype(np.float32) * float(10.0 ** rng.uniform(-3, 0))
    elif kind == 2:
        f = rng.standard_normal(count).astype(np.float32) * 0.02 + float(rng.uniform(-2, 2))
    elif kind == 3:
        f = np.where(rng.random(count) < 0.3, 0.0, rng.standard_normal(count) * 0.05).astype(np.float32)
    elif kind == 4:
        f = np.full(count, float(rng.uniform(-3, 3)), np.float32)
    else:
        bits = rng.integers(0, 1 << 32, count, dtype=np.uint64).astype(np.uint32)
        return bits if dt == 2 else (bits >> 16).astype(np.uint16)
    t = torch.from_numpy(f).to(TD[dt])
    if dt == 2:
        return t.view(torch.int32).numpy().view(np.uint32).copy()
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def to_dev(w, dt):
    if not w.size:
        return torch.empty(0, dtype=TD[dt], device="cuda")
    return torch.from_numpy(w.view(np.int32 if dt == 2 else np.int16)).cuda().view(TD[dt])


def from_dev(t, dt, like):
    return t.view(torch.int32 if dt == 2 else torch.int16).cpu().numpy().view(like.dtype)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_single_calls(oracle, seed):
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(seed)
    for case in range(120):
        dt = int(rng.integers(0, 3))
        count = max(0, int(rng.choice([rng.integers(0, 200), rng.integers(0, 40000), rng.integers(0, 600000),
                                       16384 * int(rng.integers(1, 30)) + int(rng.integers(-2, 3))])))
        w = draw(rng, dt, count)
        want = oracle.compress(w, dt)
        cap = enec.enec_max_compressed_size(dt, count)
        buf = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        size = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = status_tensor()
        entry = enec.enec_compress if rng.random() < 0.8 else enec.enec_compress_noalloc
        assert entry(to_dev(w, dt), dt, count, buf, cap, size, status) == 0
        out = torch.empty(count + 16, dtype=TD[dt], device="cuda")
        d_want = torch.from_numpy(want).cuda()
        assert enec.enec_decompress(d_want, d_want.numel(), dt, count, out, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (seed, case, dt, count)
        got = buf[:int(size.item())].cpu().numpy()
        assert got.size == want.size and np.array_equal(got, want), (seed, case, dt, count)
        assert (buf[cap:] == 0xA5).all()
        assert np.array_equal(from_dev(out[:count], dt, w), w), (seed, case, dt, count)


@pytest.mark.parametrize("seed", [21, 22])
def test_batched_calls(oracle, seed):
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(seed)
    for case in range(25):
        dt = int(rng.integers(0, 3))
        n = int(rng.integers(1, 40))
        counts = [max(0, int(rng.choice([rng.integers(0, 100), rng.integers(0, 5000), rng.integers(0, 120000)]))) for _ in range(n)]
        ws = [draw(rng, dt, c) for c in counts]
        srcs = [to_dev(w, dt) for w in ws]
        caps = [enec.enec_max_compressed_size(dt, c) for c in counts]
        bufs = [torch.empty(c, dtype=torch.uint8, device="cuda") for c in caps]
        sizes = torch.zeros(n, dtype=torch.int64, device="cuda")
        status = status_tensor()
        assert enec.enec_compress_batched([(s, b, c, cap) for s, b, c, cap in zip(srcs, bufs, counts, caps)], dt, sizes, status) == 0
        outs = [torch.empty(c, dtype=TD[dt], device="cuda") for c in counts]
        assert enec.enec_decompress_batched([(b, cap, o, c) for b, cap, o, c in zip(bufs, caps, outs, counts)], dt, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (seed, case)
        nbytes = sizes.tolist()
        for i, w in enumerate(ws):
            want = oracle.compress(w, dt)
            got = bufs[i][:nbytes[i]].cpu().numpy()
            assert got.size == want.size and np.array_equal(got, want), (seed, case, i, counts[i])
            assert np.array_equal(from_dev(outs[i], dt, w), w), (seed, case, i, counts[i])


@pytest.mark.parametrize("seed", [31, 32])
def test_ranked_calls(oracle, seed):
    """The frequency-rank variant over the same random inputs."""
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(seed)
    for case in range(80):
        dt = int(rng.integers(0, 3))
        count = max(0, int(rng.choice([rng.integers(0, 200), rng.integers(0, 40000), rng.integers(0, 400000),
                                       16384 * int(rng.integers(1, 20)) + int(rng.integers(-2, 3))])))
        w = draw(rng, dt, count)
        want = oracle.compress_ranked(w, dt)
        cap = enec.enec_max_compressed_size_ranked(dt, count)
        buf = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        size = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = status_tensor()
        assert enec.enec_compress_ranked(to_dev(w, dt), dt, count, buf, cap, size, status) == 0
        out = torch.empty(count + 16, dtype=TD[dt], device="cuda")
        d_want = torch.from_numpy(want).cuda()
        assert enec.enec_decompress_ranked(d_want, d_want.numel(), dt, count, out, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (seed, case, dt, count)
        got = buf[:int(size.item())].cpu().numpy()
        assert got.size == want.size and np.array_equal(got, want), (seed, case, dt, count)
        assert (buf[cap:] == 0xA5).all()
        assert np.array_equal(from_dev(out[:count], dt, w), w), (seed, case, dt, count)


@pytest.mark.parametrize("seed", [41, 42])
def test_blockwise_calls(oracle, seed):
    """The variant with parameters per block over the same random inputs; every second tensor is cut into stretches
    of different scale, so that the blocks' searches disagree."""
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(seed)
    for case in range(80):
        dt = int(rng.integers(0, 3))
        count = max(0, int(rng.choice([rng.integers(0, 200), rng.integers(0, 40000), rng.integers(0, 400000),
                                       16384 * int(rng.integers(1, 20)) + int(rng.integers(-2, 3))])))
        w = draw(rng, dt, count)
        if case % 2 and count > 40000:
            other = draw(rng, dt, count)
            cut = int(rng.integers(1, count))
            w = np.concatenate([w[:cut], other[cut:]])
        want = oracle.compress_blockwise(w, dt)
        cap = enec.enec_max_compressed_size_blockwise(dt, count)
        buf = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        size = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = status_tensor()
        assert enec.enec_compress_blockwise(to_dev(w, dt), dt, count, buf, cap, size, status) == 0
        out = torch.empty(count + 16, dtype=TD[dt], device="cuda")
        d_want = torch.from_numpy(want).cuda()
        assert enec.enec_decompress_blockwise(d_want, d_want.numel(), dt, count, out, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (seed, case, dt, count)
        got = buf[:int(size.item())].cpu().numpy()
        assert got.size == want.size and np.array_equal(got, want), (seed, case, dt, count)
        assert (buf[cap:] == 0xA5).all()
        assert np.array_equal(from_dev(out[:count], dt, w), w), (seed, case, dt, count)
