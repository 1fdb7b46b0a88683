"""GPU parity for two forms the library takes only for large tensors: the two-kernel form of enec_compress (pack kernel
+ the kernel that moves every block's records to their offsets, Sec. 5.1 / 5.4) and the decoder that hands a tensor's
blocks out by a ticket. Here a child process lowers their bounds through the environment so that small tensors, tails
and all dtypes go through them too, and compares every stream with the oracle's byte for byte and every decoded
tensor bit for bit. (The bounds are read once per process, hence the child.)"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
import numpy as np
import torch
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "oracle"))
import enec_oracle as oracle
import paper_2604_03298_b200 as enec

TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}
launches_per_call = []

def check(w, dt):
    count = int(w.size)
    want = oracle.compress(w, dt)
    d_in = torch.from_numpy(w.view(np.int32 if dt == 2 else np.int16).copy()).cuda().view(TD[dt])
    cap = enec.enec_max_compressed_size(dt, count)
    buf = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    size_word = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(2):   # the second call finds the scratch as the first one left it
        size_word.zero_()
        before = enec.enec_launch_count()
        assert enec.enec_compress(d_in, dt, count, buf, cap, size_word, status) == 0
        launches_per_call.append(enec.enec_launch_count() - before)
        torch.cuda.synchronize()
        size, st = int(size_word.item()), int(status.item())
        assert st == 0, st
        got = buf[:size].cpu().numpy()
        assert bool((buf[cap:] == 0xA5).all()), "wrote behind the capacity"
        assert got.size == want.size and np.array_equal(got, want), (dt, count, got.size, want.size)
    out = torch.empty(count, dtype=TD[dt], device="cuda")
    status.zero_()
    assert enec.enec_decompress(buf, cap, dt, count, out, status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    back = out.view(torch.int32 if dt == 2 else torch.int16).cpu().numpy().view(w.dtype)
    assert np.array_equal(back, w)

def gaussian(count, seed, dt, sigma):
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(count, generator=g) * sigma
    if dt == 2:
        return t.view(torch.int32).numpy().view(np.uint32)
    return t.to(TD[dt]).view(torch.int16).numpy().view(np.uint16)

for dt in (0, 1, 2):
    for count in (1, 16, 100, 5000, 16384, 16385, 16384 * 5 + 8191, 16384 * 37 + 129, 16384 * 300 + 16380,
                  16384 * 1300 + 3):
        check(gaussian(count, 77 + count + dt, dt, 0.02), dt)
# every group wide (the records stay where the pack kernel put them), no group wide, and a mix with empty blocks
rng = np.random.default_rng(4)
check(rng.integers(0, 1 << 16, 16384 * 40 + 77).astype(np.uint16), 0)
check(np.full(16384 * 9 + 5, 0x3C00, dtype=np.uint16), 0)
w = gaussian(16384 * 64, 5, 0, 0.02)
w[16384 * 3:16384 * 20] = 0x3F80
w[16384 * 30:16384 * 31] = rng.integers(0, 1 << 16, 16384)
check(w, 0)
assert min(launches_per_call) == 3 and max(launches_per_call) == 3, launches_per_call   # histogram, pack, place
print("split form ok", len(launches_per_call))
"""


def test_split_form_writes_the_oracles_streams():
    env = dict(os.environ, ENEC_SPLIT_MIN_BLOCKS="1", ENEC_SPLIT_MAX_BLOCKS="100000000", ENEC_DECODE_TICKET_MIN_BLOCKS="1")
    res = subprocess.run([sys.executable, "-c", "ROOT = %r\n" % ROOT + CHILD], env=env, capture_output=True, text=True,
                         timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "split form ok" in res.stdout
