"""GPU parity: enec_compress / enec_compress_with_params (through the C-ABI) must write the CPU oracle's stream
byte for byte, and enec_decompress of that stream must give back the tensor bit for bit (tolerance 0)."""
import numpy as np
import pytest
import torch

from gpu_util import status_tensor, tensor_of, words_of

pytestmark = pytest.mark.gpu

DT = {0: torch.bfloat16, 1: torch.float16}
CANARY = 0xA5


def gpu_compress(words, dt, params=None):
    """Returns (host status, device status, stream bytes as numpy) for a numpy uint16 array."""
    import paper_2604_03298_b200 as enec
    count = int(words.size)
    d_in = tensor_of(words, DT[dt]) if count else torch.empty(0, dtype=DT[dt], device="cuda")
    cap = enec.enec_max_compressed_size(dt, count)
    buf = torch.full((cap + 256,), CANARY, dtype=torch.uint8, device="cuda")   # canary behind the capacity
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = status_tensor()
    if params is None:
        st = enec.enec_compress(d_in, dt, count, buf, cap, size, status)
    else:
        st = enec.enec_compress_with_params(d_in, dt, count, *params, buf, cap, size, status)
    torch.cuda.synchronize()
    assert (buf[cap:] == CANARY).all(), "write behind the output capacity"
    n = int(size.item())
    return st, int(status.item()), buf[:n].cpu().numpy()


def describe_mismatch(got, want):
    if got.size != want.size:
        return f"size {got.size} != {want.size}; header got {got[:48].tolist()} want {want[:48].tolist()}"
    bad = np.flatnonzero(got != want)
    return f"{bad.size} bytes differ, first at {bad[:8].tolist()}: got {got[bad[:8]].tolist()} want {want[bad[:8]].tolist()}"


def check_stream(oracle, words, dt, params=None):
    import paper_2604_03298_b200 as enec
    want = oracle.compress(words, dt, params)
    st, dev, got = gpu_compress(words, dt, params)
    assert (st, dev) == (0, 0)
    assert got.size == want.size and np.array_equal(got, want), describe_mismatch(got, want)
    # and back through the GPU decoder
    d_stream = torch.from_numpy(got).cuda()
    out = torch.empty(words.size, dtype=DT[dt], device="cuda")
    status = status_tensor()
    assert enec.enec_decompress(d_stream, d_stream.numel(), dt, words.size, out, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(words_of(out), words)


@pytest.mark.parametrize("dt", [0, 1])
@pytest.mark.parametrize("count", [0, 1, 7, 16, 17, 40, 64, 100, 128, 129, 1000, 2048, 4096, 5000, 16383, 16384, 16385,
                                   16384 * 3 + 16, 16384 * 5 + 8191, 16384 * 37 + 129, 16384 * 600 + 3])
def test_sizes_and_tails(oracle, dt, count):
    g = torch.Generator().manual_seed(count + dt)
    w = (torch.randn(count, generator=g) * 0.02).to(DT[dt]).view(torch.int16).numpy().view(np.uint16)
    check_stream(oracle, w, dt)


def _field_words(rng, count, dt, center, n, m):
    E, mant = (8, 7) if dt == 0 else (5, 10)
    top = (1 << E) - 1
    half = 1 << (n - 1)
    if n < E:
        x = rng.integers(max(0, center - (half - 1)), min(top, center + half) + 1, count)
    else:
        x = rng.integers(0, top + 1, count)
    narrow = center - rng.integers(0, min(1 << (m - 1), half), count)
    x = np.where(rng.random(count) < 0.8, narrow, x)
    return ((x.astype(np.uint16) << mant) | rng.integers(0, 1 << mant, count).astype(np.uint16)
            | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)


@pytest.mark.parametrize("n,m", [(n, m) for n in range(1, 9) for m in range(1, n + 1)])
def test_every_width_pair_bf16(oracle, n, m):
    rng = np.random.default_rng(100 * n + m)
    check_stream(oracle, _field_words(rng, 16384 * 4 + 2048 + 40, 0, 120, n, m), 0, (120, n, m))


@pytest.mark.parametrize("n,m", [(n, m) for n in range(1, 6) for m in range(1, n + 1)])
def test_every_width_pair_fp16(oracle, n, m):
    rng = np.random.default_rng(200 * n + m)
    check_stream(oracle, _field_words(rng, 16384 * 3 + 512 + 24, 1, 12, n, m), 1, (12, n, m))


@pytest.mark.parametrize("n,m", [(6, 3), (8, 1), (5, 5), (3, 2)])
@pytest.mark.parametrize("count", [16, 24, 48, 64, 100, 200, 700])
def test_short_tail_blocks_with_params(oracle, n, m, count):
    rng = np.random.default_rng(count * 10 + n)
    check_stream(oracle, _field_words(rng, count, 0, 120, n, m), 0, (120, n, m))
    if n <= 5:
        check_stream(oracle, _field_words(rng, count, 1, 12, n, m), 1, (12, n, m))


@pytest.mark.parametrize("dt", [0, 1])
def test_all_bit_patterns(oracle, dt):
    allw = np.arange(1 << 16, dtype=np.uint16)
    rng = np.random.default_rng(5)
    check_stream(oracle, allw, dt)
    check_stream(oracle, rng.permutation(allw), dt)
    check_stream(oracle, np.repeat(allw, 16)[:20 * 16384 + 77], dt)


def test_mask_extremes(oracle):
    count = 16384 * 3
    base = np.full(count, 123 << 7, np.uint16)
    check_stream(oracle, base, 0, (123, 6, 3))
    check_stream(oracle, base, 0)                         # constant tensor: n = 1, m = 1
    allwide = base.copy()
    allwide[::16] = 125 << 7
    check_stream(oracle, allwide, 0, (123, 6, 3))
    first = base.copy(); first[16384] = 100 << 7
    check_stream(oracle, first, 0, (123, 6, 3))
    last = base.copy(); last[2 * 16384 - 1] = 126 << 7
    check_stream(oracle, last, 0, (123, 6, 3))


def test_parameter_search_matches_oracle_on_odd_histograms(oracle):
    rng = np.random.default_rng(21)
    for trial in range(12):
        count = int(rng.integers(1000, 90000))
        center = int(rng.integers(5, 250))
        spread = float(rng.choice([0.3, 1.0, 2.5, 8.0, 40.0]))
        x = np.clip(np.round(rng.normal(center, spread, count)), 0, 255).astype(np.uint16)
        words = ((x << 7) | rng.integers(0, 128, count).astype(np.uint16)).astype(np.uint16)
        check_stream(oracle, words, 0)
    for trial in range(6):
        count = int(rng.integers(1000, 60000))
        x = np.clip(np.round(rng.normal(rng.integers(2, 30), rng.choice([0.5, 2.0, 9.0]), count)), 0, 31).astype(np.uint16)
        words = ((x << 10) | rng.integers(0, 1024, count).astype(np.uint16)).astype(np.uint16)
        check_stream(oracle, words, 1)


def test_config1_gaussian(oracle):
    from paper_2604_03298_b200 import synth
    spec = synth.config_specs(1)[0]
    t = synth.make_tensor(spec, "cuda")
    check_stream(oracle, words_of(t), 0)


def test_heavy_tailed_tensors(oracle):
    from paper_2604_03298_b200 import synth
    specs = synth.config_specs(4, scale=8)                # 512 x 512 versions of the stress set
    for spec in (specs[0], specs[31], specs[40], specs[63], specs[64], specs[100], specs[127]):
        t = synth.make_tensor(spec, "cuda")
        check_stream(oracle, words_of(t), 0 if spec.dtype == torch.bfloat16 else 1)


def test_params_that_lose_exponents_are_reported(oracle):
    words = (np.array([100, 130] * 8000, np.uint16) << 7).astype(np.uint16)
    st, dev, got = gpu_compress(words, 0, (120, 3, 2))
    assert st == 0 and dev == -5 and got.size == 0
    with pytest.raises(oracle.OracleError):
        oracle.compress(words, 0, (120, 3, 2))


def test_host_argument_checks():
    import paper_2604_03298_b200 as enec
    src = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    cap = enec.enec_max_compressed_size(0, 4096)
    dst = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    assert enec.enec_compress(src, 7, 4096, dst, cap) == -2
    assert enec.enec_compress(src, 0, 4096, dst, cap - 1) == -3
    assert enec.enec_compress(src[1:], 0, 4000, dst, cap) == -1
    assert enec.enec_compress(src, 0, 4096, None, cap) == -1
    assert enec.enec_compress_with_params(src, 0, 4096, 120, 9, 3, dst, cap) == -1
    assert enec.enec_compress_with_params(src, 0, 4096, 120, 3, 4, dst, cap) == -1
    assert enec.enec_compress_with_params(src, 0, 4096, 256, 6, 3, dst, cap) == -1
    assert enec.enec_compress_with_params(src, 1, 4096, 12, 6, 3, dst, cap) == -1
    assert enec.enec_max_compressed_size(5, 10) == 0
    assert enec.enec_max_compressed_size(0, 1 << 36) == 0
    torch.cuda.synchronize()


def test_max_size_agrees_with_oracle(oracle):
    import paper_2604_03298_b200 as enec
    for dt in (0, 1):
        for count in (0, 1, 16, 17, 4096, 16384, 16385, 1 << 20, (1 << 20) + 5, 128256 * 4096):
            assert enec.enec_max_compressed_size(dt, count) == oracle.max_compressed_size(dt, count)


def test_back_to_back_calls_on_one_stream(oracle):
    # the library's scratch is reused by consecutive calls on a stream; results must not leak between them
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(33)
    tensors = [(_field_words(rng, c, 0, 121, 6, 3), 0) for c in (16384 * 9 + 5, 300, 16384 * 2, 16384 * 40 + 17)]
    outs = []
    for words, dt in tensors:
        d_in = tensor_of(words, DT[dt])
        cap = enec.enec_max_compressed_size(dt, words.size)
        buf = torch.empty(cap, dtype=torch.uint8, device="cuda")
        size = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = status_tensor()
        assert enec.enec_compress(d_in, dt, words.size, buf, cap, size, status) == 0
        outs.append((d_in, buf, size, status))
    torch.cuda.synchronize()
    for (words, dt), (_, buf, size, status) in zip(tensors, outs):
        assert int(status.item()) == 0
        want = oracle.compress(words, dt)
        got = buf[:int(size.item())].cpu().numpy()
        assert np.array_equal(got, want), describe_mismatch(got, want)


def test_scratch_state_survives_mixed_call_sequences(oracle):
    """The compressor's scratch area is not cleared between calls: shrinking and growing tensors, both dtypes,
    calls with and without the parameter search and a call that reports lost exponents, all queued on one stream
    without a host synchronisation in between, must each give the oracle's stream."""
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(77)
    plan = []   # (words, dt, params or None, expect_error)
    for rep in range(3):
        for count in (16384 * 20 + 7, 40, 16384 * 3, 16384 * 64, 5000):
            plan.append((_field_words(rng, count, 0, 121, 6, 3), 0, None, False))
            plan.append((_field_words(rng, count, 1, 12, 4, 2), 1, (12, 4, 2), False))
        lossy = (np.array([100, 130] * 9000, np.uint16) << 7).astype(np.uint16)
        plan.append((lossy, 0, (120, 3, 2), True))
        plan.append((_field_words(rng, 16384 * 5 + 1, 0, 124, 5, 2), 0, (124, 5, 2), False))
    queued = []
    for words, dt, params, _ in plan:
        d_in = tensor_of(words, DT[dt])
        cap = enec.enec_max_compressed_size(dt, words.size)
        buf = torch.empty(cap, dtype=torch.uint8, device="cuda")
        size = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = status_tensor()
        if params is None:
            assert enec.enec_compress(d_in, dt, words.size, buf, cap, size, status) == 0
        else:
            assert enec.enec_compress_with_params(d_in, dt, words.size, *params, buf, cap, size, status) == 0
        queued.append((d_in, buf, size, status))
    torch.cuda.synchronize()
    for (words, dt, params, expect_error), (_, buf, size, status) in zip(plan, queued):
        if expect_error:
            assert int(status.item()) == -5 and int(size.item()) == 0
            continue
        assert int(status.item()) == 0
        want = oracle.compress(words, dt, params)
        got = buf[:int(size.item())].cpu().numpy()
        assert np.array_equal(got, want), describe_mismatch(got, want)


def test_compress_refuses_a_stream_that_is_being_captured():
    """Compress calls keep state between calls, so they cannot be part of a CUDA graph; decompress can."""
    import paper_2604_03298_b200 as enec
    src = (torch.randn(16384 * 4, device="cuda") * 0.02).to(torch.bfloat16)
    cap = enec.enec_max_compressed_size(0, src.numel())
    dst = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = status_tensor()
    out = torch.zeros_like(src)
    assert enec.enec_compress(src, 0, src.numel(), dst, cap, size, status) == 0
    assert enec.enec_decompress(dst, cap, 0, src.numel(), out, status) == 0     # first use outside a capture
    torch.cuda.synchronize()
    codes = {}
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        codes["compress"] = enec.enec_compress(src, 0, src.numel(), dst, cap, size, status)
        codes["decompress"] = enec.enec_decompress(dst, cap, 0, src.numel(), out, status)
    assert codes == {"compress": -1, "decompress": 0}
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out.view(torch.int16), src.view(torch.int16))
