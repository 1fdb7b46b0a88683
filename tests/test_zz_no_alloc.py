"""enec_compress_noalloc is for callers that may not allocate device memory (code running under an allocator that
owns the whole device, or in a phase where a cudaMalloc's device-wide synchronisation is not acceptable): it works
out of a fixed array inside the library instead of scratch from cudaMalloc. This test calls it through the C-ABI
and checks that it writes exactly the bytes enec_compress writes (tolerance 0, as everywhere in this suite), on two
calls in a row that share the array, the second smaller than the first so that stale state would show.

Collected last on purpose: a failure here cannot hide the result of any other test in a run that stops at the
first failure.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _compress(fn, t):
    import paper_2604_03298_b200 as enec
    dt = enec.BF16 if t.dtype == torch.bfloat16 else enec.FP16
    n = t.numel()
    cap = enec.enec_max_compressed_size(dt, n)
    buf = torch.full((cap + 64,), 0xC3, dtype=torch.uint8, device="cuda")
    size = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert fn(t, dt, n, buf, cap, size, status) == 0
    return buf, size, status, cap


def test_noalloc_matches_enec_compress_twice_in_a_row():
    import paper_2604_03298_b200 as enec
    from paper_2604_03298_b200 import synth
    tensors = [
        synth.make_tensor(synth.TensorSpec("a", torch.bfloat16, (16384 * 70 + 4321,), "normal", 0.0, 0.02, 91), "cuda"),
        synth.make_tensor(synth.TensorSpec("b", torch.bfloat16, (16384 * 3 + 17,), "laplace", 0.0, 0.05, 92,
                                           outliers=True), "cuda"),
        synth.make_tensor(synth.TensorSpec("c", torch.float16, (16384 * 9 + 100,), "normal", 0.0, 0.02, 93), "cuda"),
    ]
    # both calls of the new entry point are queued back to back, before anything is read back
    queued = [_compress(enec.enec_compress_noalloc, t) for t in tensors]
    torch.cuda.synchronize()
    for t, (buf, size, status, cap) in zip(tensors, queued):
        assert int(status.item()) == 0
        assert (buf[cap:] == 0xC3).all()
        ref_buf, ref_size, ref_status, _ = _compress(enec.enec_compress, t)
        torch.cuda.synchronize()
        assert int(ref_status.item()) == 0
        n = int(size.item())
        assert n == int(ref_size.item()) and n > 0
        assert torch.equal(buf[:n], ref_buf[:n])
        # and the stream decodes to the tensor
        out = torch.empty_like(t)
        dt = enec.BF16 if t.dtype == torch.bfloat16 else enec.FP16
        assert enec.enec_decompress(buf, n, dt, t.numel(), out, status) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out.view(torch.int16), t.view(torch.int16))


def test_noalloc_refuses_what_does_not_fit_its_array():
    import paper_2604_03298_b200 as enec
    small = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    dst = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    too_many = (1 << 30) + 16
    assert enec.enec_compress_noalloc(small, enec.BF16, too_many, dst, 1 << 40) == -8      # nothing is enqueued
    assert enec.enec_compress_noalloc(small, enec.BF16, 64, dst, 10) == -3
    assert enec.enec_compress_noalloc(small, 5, 64, dst, 4096) == -2
    torch.cuda.synchronize()


def test_noalloc_makes_no_allocation_where_enec_compress_does():
    """What the entry point is for: on a stream the library has never seen, enec_compress takes scratch from
    cudaMalloc (the library counts its calls) and enec_compress_noalloc does not."""
    import paper_2604_03298_b200 as enec
    from paper_2604_03298_b200 import synth
    t = synth.make_tensor(synth.TensorSpec("d", torch.bfloat16, (16384 * 5 + 11,), "normal", 0.0, 0.02, 94), "cuda")
    torch.cuda.synchronize()
    fresh = torch.cuda.Stream()
    with torch.cuda.stream(fresh):
        before = enec.enec_allocation_count()
        a = _compress(enec.enec_compress_noalloc, t)
        b = _compress(enec.enec_compress_noalloc, t)
        assert enec.enec_allocation_count() == before
        c = _compress(enec.enec_compress, t)
        assert enec.enec_allocation_count() == before + 1
    torch.cuda.synchronize()
    n = int(c[1].item())
    for buf, size, status, cap in (a, b):
        assert int(status.item()) == 0 and int(size.item()) == n
        assert torch.equal(buf[:n], c[0][:n])
