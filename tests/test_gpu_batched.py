"""GPU parity of enec_decompress_batched: many streams, one launch, every tensor bit-exact (tolerance 0)."""
import numpy as np
import pytest
import torch

from gpu_util import status_tensor, tensor_of, to_dev_bytes, words_of

pytestmark = pytest.mark.gpu

DT = {0: torch.bfloat16, 1: torch.float16}


def _words(rng, count, dt, spread):
    E, mant = (8, 7) if dt == 0 else (5, 10)
    center = 120 if dt == 0 else 12
    x = np.clip(np.round(rng.normal(center, spread, count)), 0, (1 << E) - 1).astype(np.uint16)
    return ((x << mant) | rng.integers(0, 1 << mant, count).astype(np.uint16)
            | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)


@pytest.mark.parametrize("dt", [0, 1])
def test_mixed_batch_against_oracle_streams(oracle, dt):
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(40 + dt)
    counts = [16384 * 7 + 5, 0, 1, 16, 2048, 16384, 100, 16384 * 30, 17, 16384 * 3 + 8000, 0, 40, 16384 * 2 + 1] + [2048] * 40
    spreads = [0.4, 1.0, 2.0, 4.0, 30.0]
    items, wants = [], []
    for i, c in enumerate(counts):
        w = _words(rng, c, dt, spreads[i % len(spreads)])       # different (b, n, m) per tensor
        s = oracle.compress(w, dt)
        d_in = to_dev_bytes(s)
        guard = torch.full((c + 64,), 0x5A5A, dtype=torch.int16, device="cuda")
        items.append((d_in, d_in.numel(), guard, c))
        wants.append(w)
    status = status_tensor()
    call = [(src, nbytes, g[:c].view(DT[dt]) if c else g[:0].view(DT[dt]), c) for src, nbytes, g, c in items]
    before = enec.enec_launch_count()
    assert enec.enec_decompress_batched(call, dt, status) == 0
    torch.cuda.synchronize()
    assert enec.enec_launch_count() - before == 1
    assert int(status.item()) == 0
    for (src, nbytes, g, c), w in zip(items, wants):
        assert (g[c:] == 0x5A5A).all()
        got = g[:c].cpu().numpy().view(np.uint16)
        assert np.array_equal(got, w)


def test_moe_shaped_set_full_size():
    """Workload 5 at full size (768 expert matrices + 4096 vectors of 2048, bf16): streams written by enec_compress
    (checked byte for byte against the oracle elsewhere), all decompressed by one batched launch."""
    import paper_2604_03298_b200 as enec
    from paper_2604_03298_b200 import runner, synth
    specs = synth.config_specs(5)
    assert len(specs) == 768 + 4096
    # the expert matrices share three shapes and one distribution: draw 24 distinct ones and reuse them
    distinct = {}
    raw = []
    for i, s in enumerate(specs):
        key = (s.shape, i % 24) if len(s.shape) == 2 else ("v", i)
        if key not in distinct:
            distinct[key] = synth.make_tensor(s, "cuda")
        raw.append(distinct[key])
    cs = runner.CodecSet.allocate(raw)
    cs.compress_all()
    torch.cuda.synchronize()
    cs.check_status()
    sizes = cs.sizes.cpu().tolist()
    items = [(cs.streams[i], sizes[i], cs.outs[i], raw[i].numel()) for i in range(len(raw))]
    before = enec.enec_launch_count()
    assert enec.enec_decompress_batched(items, 0, cs.status) == 0
    torch.cuda.synchronize()
    assert enec.enec_launch_count() - before == 1
    cs.check_status()
    cs.verify_roundtrip()


def test_damaged_member_is_reported(oracle):
    import paper_2604_03298_b200 as enec
    rng = np.random.default_rng(50)
    streams = [oracle.compress(_words(rng, 16384 * 4 + 9, 0, 2.0), 0) for _ in range(6)]
    streams[3] = streams[3].copy()
    streams[3][22] = 9                                   # m beyond n
    call = []
    for s in streams:
        d = to_dev_bytes(s)
        call.append((d, d.numel(), torch.empty(16384 * 4 + 9, dtype=torch.bfloat16, device="cuda"), 16384 * 4 + 9))
    status = status_tensor()
    assert enec.enec_decompress_batched(call, 0, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == -4


def test_host_argument_checks():
    import paper_2604_03298_b200 as enec
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    out = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    assert enec.enec_decompress_batched([], 0) == 0
    assert enec.enec_decompress_batched([(buf, 4096, out, 64)], 9) == -2
    assert enec.enec_decompress_batched([(buf[1:], 4000, out, 64)], 0) == -1
    assert enec.enec_decompress_batched([(buf, 10, out, 64)], 0) == -4
    torch.cuda.synchronize()


# ---- enec_compress_batched ---------------------------------------------------------------------------
def _compress_batched(words_list, dt):
    import paper_2604_03298_b200 as enec
    from gpu_util import status_tensor
    dtype = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}[dt]
    view = np.int32 if dt == 2 else np.int16
    srcs = [torch.from_numpy(w.view(view).copy()).cuda().view(dtype) if w.size else torch.empty(0, dtype=dtype, device="cuda")
            for w in words_list]
    caps = [enec.enec_max_compressed_size(dt, int(w.size)) for w in words_list]
    bufs = [torch.full((c + 64,), 0xA5, dtype=torch.uint8, device="cuda") for c in caps]
    sizes = torch.zeros(len(words_list), dtype=torch.int64, device="cuda")
    status = status_tensor()
    items = [(s, b, int(w.size), c) for s, b, w, c in zip(srcs, bufs, words_list, caps)]
    st = enec.enec_compress_batched(items, dt, sizes, status)
    torch.cuda.synchronize()
    for b, c in zip(bufs, caps):
        assert (b[c:] == 0xA5).all(), "write behind an output buffer"
    return st, int(status.item()), [b[:n].cpu().numpy() for b, n in zip(bufs, sizes.tolist())]


def _gaussian16(count, seed, dtype=torch.bfloat16, sigma=0.02, mean=0.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(count, generator=g) * sigma + mean).to(dtype).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dt", [0, 1])
def test_compress_batched_matches_the_oracle_per_tensor(oracle, dt):
    dtype = torch.bfloat16 if dt == 0 else torch.float16
    counts = [16384 * 30 + 11, 2048, 16, 0, 16384, 5, 16384 * 7, 2048, 100, 16384 * 64 + 1, 4096, 33]
    ws = [_gaussian16(c, 900 + i, dtype, sigma=0.02 if i % 3 else 0.5, mean=1.0 if i % 4 == 1 else 0.0) for i, c in enumerate(counts)]
    st, dev, got = _compress_batched(ws, dt)
    assert (st, dev) == (0, 0)
    for i, (w, g) in enumerate(zip(ws, got)):
        want = oracle.compress(w, dt)
        assert g.size == want.size and np.array_equal(g, want), f"tensor {i} (count {w.size}): stream differs"


def test_compress_batched_fp32(oracle):
    rng = np.random.default_rng(12)
    ws = []
    for i, c in enumerate([16384 * 9 + 3, 64, 16384 * 2, 7, 2048]):
        g = torch.Generator().manual_seed(40 + i)
        ws.append((torch.randn(c, generator=g) * 0.02).view(torch.int32).numpy().view(np.uint32))
    st, dev, got = _compress_batched(ws, 2)
    assert (st, dev) == (0, 0)
    for i, (w, g) in enumerate(zip(ws, got)):
        assert np.array_equal(g, oracle.compress(w, 2)), f"tensor {i}"


def test_compress_batched_many_small_tensors_round_trip(oracle):
    """The shape of the MoE set at reduced size: expert matrices plus hundreds of one-block vectors, compressed by
    one call and decompressed by one call; a sample is compared with the oracle."""
    import paper_2604_03298_b200 as enec
    from gpu_util import status_tensor
    counts = [176 * 16384 // 8] * 24 + [2048] * 700
    srcs = [(torch.randn(c, device="cuda", generator=torch.Generator(device="cuda").manual_seed(i)) * 0.02).to(torch.bfloat16)
            for i, c in enumerate(counts)]
    caps = [enec.enec_max_compressed_size(0, c) for c in counts]
    bufs = [torch.empty(c, dtype=torch.uint8, device="cuda") for c in caps]
    sizes = torch.zeros(len(counts), dtype=torch.int64, device="cuda")
    status = status_tensor()
    for _ in range(2):   # twice: the call's scratch area is reused
        assert enec.enec_compress_batched([(s, b, c, cap) for s, b, c, cap in zip(srcs, bufs, counts, caps)], 0, sizes, status) == 0
    outs = [torch.zeros_like(s) for s in srcs]
    nbytes = sizes.tolist()
    assert enec.enec_decompress_batched([(b, n, o, c) for b, n, o, c in zip(bufs, nbytes, outs, counts)], 0, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for s, o in zip(srcs, outs):
        assert torch.equal(s.view(torch.int16), o.view(torch.int16))
    for i in (0, 23, 24, 300, 723):
        want = oracle.compress(s_words(srcs[i]), 0)
        assert np.array_equal(bufs[i][:nbytes[i]].cpu().numpy(), want)


def s_words(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def test_compress_batched_argument_checks():
    import paper_2604_03298_b200 as enec
    src = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    cap = enec.enec_max_compressed_size(0, 4096)
    dst = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    assert enec.enec_compress_batched([], 0) == 0
    assert enec.enec_compress_batched([(src, dst, 4096, cap)], 9) == -2
    assert enec.enec_compress_batched([(src, dst, 4096, cap - 1)], 0) == -3
    assert enec.enec_compress_batched([(src[1:], dst, 4000, cap)], 0) == -1
    torch.cuda.synchronize()


def test_batched_decompress_checks_members_without_elements():
    """A member with count 0 has an 80-byte stream and no block: its header must still be looked at, alone or among
    tensors that do have blocks, as enec_decompress does for an empty tensor."""
    import paper_2604_03298_b200 as enec
    empty = torch.empty(0, dtype=torch.bfloat16, device="cuda")
    full = (torch.randn(40000, device="cuda") * 0.02).to(torch.bfloat16)
    s_empty, s_full = enec.compress_tensor(empty), enec.compress_tensor(full)
    assert s_empty.numel() == 80
    out = torch.empty_like(full)
    none = torch.empty(16, dtype=torch.bfloat16, device="cuda")
    for streams in ([s_empty.clone()], [s_full, s_empty.clone()]):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        items = [(s, s.numel(), out if s.numel() > 80 else none, full.numel() if s.numel() > 80 else 0) for s in streams]
        assert enec.enec_decompress_batched(items, 0, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        streams[-1][0] = 0x58           # damage the empty member's magic
        assert enec.enec_decompress_batched(items, 0, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == -4
    assert torch.equal(out.view(torch.int16), full.view(torch.int16))


def test_batched_calls_under_stream_capture():
    """A batch of more than 16 tensors recorded into a CUDA graph: the decompress call records launches whose
    tensor lists travel in their parameters (nothing of the call's host memory or the library's scratch is in the
    graph), and replays bit for bit after the outputs were wiped; the compress call is refused."""
    import paper_2604_03298_b200 as enec
    g = torch.Generator(device="cuda").manual_seed(77)
    raw = [(torch.randn(16384 * 2 + 100 * i + 5, generator=g, device="cuda") * 0.02).to(torch.bfloat16) for i in range(17)]
    streams = [enec.compress_tensor(t) for t in raw]
    outs = [torch.zeros_like(t) for t in raw]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    items = enec.make_batch([(s, o, t.numel(), s.numel()) for s, o, t in zip(streams, outs, raw)])
    comp_items = enec.make_batch([(t, torch.empty(enec.enec_max_compressed_size(0, t.numel()), dtype=torch.uint8, device="cuda"),
                                   t.numel(), enec.enec_max_compressed_size(0, t.numel())) for t in raw])
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    before = enec.enec_launch_count()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            assert enec.enec_compress_batched(comp_items, 0, None, status) == -1
            assert enec.enec_decompress_batched(items, 0, status) == 0
    assert enec.enec_launch_count() - before == 2      # 16 + 1 tensors
    for _ in range(2):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for o, t in zip(outs, raw):
            assert torch.equal(o.view(torch.int16), t.view(torch.int16))
