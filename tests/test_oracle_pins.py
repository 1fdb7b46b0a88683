"""Pins for the CPU oracle: values the paper prints, hand traces, closed forms, library special cases,
brute force and invariants. No GPU, no CUDA library."""
from fractions import Fraction
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_fixture(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            k, v = line.split(":", 1)
            out.setdefault(k.strip(), []).append(v.strip())
    return out


def hexbytes(s):
    return np.array([int(t, 16) for t in s.split()], dtype=np.uint8)


# ---------------------------------------------------------------- split / join
def test_split_fields_bf16_fp16(oracle):
    # bf16 1.0 = 0x3F80: exponent 127, mantissa 0; -1.5 = 0xBFC0: sign 1, exponent 127, mantissa 0x40
    assert oracle.split(0x3F80, 0) == (127, 0x00)
    assert oracle.split(0xBFC0, 0) == (127, 0x80 | 0x40)
    # fp16 1.0 = 0x3C00: exponent 15; -2.5 = 0xC100: sign 1, exponent 16, mantissa 0x100
    assert oracle.split(0x3C00, 1) == (15, 0)
    assert oracle.split(0xC100, 1) == (16, 0x400 | 0x100)
    for dt in (0, 1):
        for w in range(0, 1 << 16, 7):
            x, sm = oracle.split(w, dt)
            assert oracle.join(x, sm, dt) == w


def test_split_matches_float_decomposition(oracle):
    # exponent field = floor(log2 |v|) + bias for normal numbers (numpy frexp as the library routine)
    rng = np.random.default_rng(1)
    vals = rng.normal(0, 0.02, 200).astype(np.float16)
    for v, w in zip(vals, vals.view(np.uint16)):
        if v == 0 or abs(float(v)) < 6.2e-5:
            continue
        _, e = np.frexp(np.float64(v))
        assert oracle.split(int(w), 1)[0] == e - 1 + 15


# ---------------------------------------------------------------- Sec. 5.3 / Eq. 2
def test_transform_worked_example(oracle):
    fx = read_fixture("transform_example.txt")
    b, n = int(fx["b"][0]), int(fx["n"][0])
    assert oracle.transform(125, b, n) == int(fx["x125"][0])
    assert oracle.transform(122, b, n) == int(fx["x122"][0])
    assert oracle.inverse_transform(62, b, n, 8) == 125
    assert oracle.inverse_transform(1, b, n, 8) == 122


def test_transform_is_twos_complement_of_b_minus_x(oracle):
    for n in range(1, 9):
        for b in (0, 5, 122, 123, 255):
            for x in range(256):
                assert oracle.transform(x, b, n) == (b - x) % (1 << n)


# ---------------------------------------------------------------- Eq. 1
def test_eq1_hand_values(oracle):
    assert oracle.width_eq1(122, 99, 123, 8) == 6      # max(bw(23) = 5, cl2(1) = 0) + 1
    assert oracle.width_eq1(123, 99, 125, 8) == 6      # max(bw(24) = 5, cl2(2) = 1) + 1
    assert oracle.width_eq1(121, 121, 121, 8) == 1     # single occupied bin
    assert oracle.width_eq1(121, 121, 122, 8) == 1     # h - b = 1 -> y in {0, 1 (= -1 mod 2)}
    assert oracle.width_eq1(121, 121, 123, 8) == 2     # -2..0 needs two bits
    assert oracle.width_eq1(120, 0, 130, 8) == 8       # clamped to the field width
    assert oracle.width_eq1(7, 0, 15, 5) == 4          # bw(7) = 3, cl2(8) = 3


def test_eq1_is_minimal_twos_complement_width(oracle):
    # independent definition: smallest n with -2^(n-1) <= b - x <= 2^(n-1) - 1 for all x in [l, h]
    E = 8
    for l in range(100, 132, 3):
        for h in range(l, 140, 2):
            for b in range(l, h + 1):
                n = 1
                while not (-(1 << (n - 1)) <= b - h and b - l <= (1 << (n - 1)) - 1):
                    n += 1
                assert oracle.width_eq1(b, l, h, E) == min(n, E)


def test_transform_roundtrip_over_occupied_range(oracle):
    for E in (5, 8):
        top = (1 << E) - 1
        for l in range(0, top + 1, 5):
            for h in range(l, top + 1, 3):
                for b in range(l, h + 1, 2):
                    n = oracle.width_eq1(b, l, h, E)
                    for x in range(l, h + 1):
                        assert oracle.inverse_transform(oracle.transform(x, b, n), b, n, E) == x
    for b in (0, 17, 255):  # n = E: every field value
        for x in range(256):
            assert oracle.inverse_transform(oracle.transform(x, b, 8), b, 8, 8) == x


# ---------------------------------------------------------------- Algorithm 2
def test_alg2_hand_traces(oracle):
    fx = read_fixture("alg2_hand.txt")
    for c in "ABCDE":
        N, a = int(fx[f"{c}_N"][0]), int(fx[f"{c}_a"][0])
        data = np.array(fx[f"{c}_data"][0].split(), dtype=np.uint16)
        assert data.size == N
        got = oracle.alg2_pack(data, a)
        assert got.tolist() == hexbytes(fx[f"{c}_bytes"][0]).tolist(), c
        assert oracle.alg2_unpack(got, N, a).tolist() == data.tolist()


def test_alg2_length_rule(oracle):
    for N in (2, 4, 8, 16, 64, 1024, 16384):
        for a in range(1, 9):
            n_out = oracle.alg2_pack(np.zeros(N, np.uint16), a).size
            if N >= 16:
                assert n_out == N * a // 8          # exact, already even
            assert n_out % 2 == 0
            assert n_out >= (N * a + 7) // 8


def test_alg2_a8_is_half_interleave(oracle):
    # a = 8: no fold; bytes are the values; final fold interleaves first and second half
    rng = np.random.default_rng(2)
    for N in (16, 256):
        v = rng.integers(0, 256, N).astype(np.uint16)
        expect = np.stack([v[:N // 2], v[N // 2:]], axis=1).reshape(-1).astype(np.uint8)
        assert oracle.alg2_pack(v, 8).tolist() == expect.tolist()


def test_alg2_a4_is_nibble_pairs(oracle):
    rng = np.random.default_rng(3)
    N = 64
    v = rng.integers(0, 16, N).astype(np.uint16)
    nb = (v[:N // 2] | (v[N // 2:] << 4)).astype(np.uint8)            # one fold
    expect = np.stack([nb[:N // 4], nb[N // 4:]], axis=1).reshape(-1)
    assert oracle.alg2_pack(v, 4).tolist() == expect.tolist()


def test_alg2_a1_is_packbits_of_a_strided_view(oracle):
    # a = 1: byte j bit p holds element j + (p&1) N/2 + (p>>1 & 1) N/4 + (p>>2) N/8  -> numpy packbits
    rng = np.random.default_rng(4)
    N = 128
    v = rng.integers(0, 2, N).astype(np.uint16)
    j = np.arange(N // 8)[:, None]
    p = np.arange(8)[None, :]
    idx = j + (p & 1) * (N // 2) + ((p >> 1) & 1) * (N // 4) + (p >> 2) * (N // 8)
    nb = np.packbits(v[idx].astype(np.uint8), axis=1, bitorder="little").reshape(-1)
    expect = np.stack([nb[:N // 16], nb[N // 16:]], axis=1).reshape(-1)
    assert oracle.alg2_pack(v, 1).tolist() == expect.tolist()


def test_alg2_a3_closed_form_block(oracle):
    # N = 16384, a = 3 derived from the pseudocode by hand: lane j < 4096 holds
    # e[j] | e[j+8192]<<3 | e[j+4096]<<6 | e[j+12288]<<9 ; first 4096 bytes = low bytes ; residue nibbles
    # r[j] | r[j+2048]<<4 form the next 2048 bytes ; output byte 2i = nb[i], 2i+1 = nb[i+3072].
    rng = np.random.default_rng(5)
    N = 16384
    e = rng.integers(0, 8, N).astype(np.uint32)
    lane = e[:4096] | (e[8192:12288] << 3) | (e[4096:8192] << 6) | (e[12288:] << 9)
    r = lane >> 8
    nb = np.concatenate([lane & 0xFF, r[:2048] | (r[2048:] << 4)]).astype(np.uint8)
    expect = np.stack([nb[:3072], nb[3072:]], axis=1).reshape(-1)
    assert oracle.alg2_pack(e.astype(np.uint16), 3).tolist() == expect.tolist()


@pytest.mark.parametrize("N", [2, 4, 16, 64])
def test_alg2_is_a_bit_permutation(oracle, N):
    # every input bit lands on exactly one output bit, all distinct; OR-linearity; all-ones fills the stream
    for a in range(1, 9):
        seen = set()
        for i in range(N):
            for bit in range(a):
                v = np.zeros(N, np.uint16)
                v[i] = 1 << bit
                out = oracle.alg2_pack(v, a)
                pos = np.flatnonzero(np.unpackbits(out, bitorder="little"))
                assert pos.size == 1
                assert int(pos[0]) not in seen
                seen.add(int(pos[0]))
        assert len(seen) == N * a
        ones = oracle.alg2_pack(np.full(N, (1 << a) - 1, np.uint16), a)
        assert int(np.unpackbits(ones).sum()) == N * a
        rng = np.random.default_rng(N * 10 + a)
        u = rng.integers(0, 1 << a, N).astype(np.uint16)
        w = rng.integers(0, 1 << a, N).astype(np.uint16)
        assert (oracle.alg2_pack(u, a) | oracle.alg2_pack(w, a)).tolist() == oracle.alg2_pack(u | w, a).tolist()
        assert oracle.alg2_unpack(oracle.alg2_pack(u, a), N, a).tolist() == u.tolist()


def test_alg2_roundtrip_large(oracle):
    rng = np.random.default_rng(6)
    for N in (128, 2048, 16384):
        for a in range(1, 9):
            u = rng.integers(0, 1 << a, N).astype(np.uint16)
            assert np.array_equal(oracle.alg2_unpack(oracle.alg2_pack(u, a), N, a), u)


# ---------------------------------------------------------------- Sec. 5.5 parameter search
def test_phase2_cost_matches_elementwise_sum(oracle):
    rng = np.random.default_rng(7)
    x = np.clip(np.round(rng.normal(121, 2.0, 5000)), 100, 130).astype(np.int64)
    hist = np.bincount(x, minlength=256).astype(np.uint64)
    b, n, m, cost, bexp = oracle.param_search(hist, 8)
    l, h = int(x.min()), int(x.max())
    best = None
    for cand in range(l, h + 1):
        width = 1
        while not (-(1 << (width - 1)) <= cand - h and cand - l <= (1 << (width - 1)) - 1):
            width += 1
        width = min(width, 8)
        d = int(((cand - x) % (1 << width)).sum())      # Eq. 3 times N, element by element
        assert int(cost[cand]) == d
        key = (d, width, cand)
        if best is None or key < best:
            best = key
    assert (b, n) == (best[2], best[1])
    assert all(int(cost[c]) == np.iinfo(np.uint64).max for c in list(range(0, l)) + list(range(h + 1, 256)))


def test_phase3_eq4_exact_rational(oracle):
    # histogram chosen so that Phase 2 gives b = 122: counts of y = 0, 1, 2, 3, 20 -> widths 0, 1, 2, 2, 5
    hist = np.zeros(256, np.uint64)
    hist[122], hist[121], hist[120], hist[119], hist[102] = 4000, 2500, 900, 500, 100
    b, n, m, cost, bexp = oracle.param_search(hist, 8)
    assert (b, n) == (122, 6)           # bw(122 - 102 = 20) = 5, +1 sign bit
    total = int(hist.sum())
    y_of = {122: 0, 121: 1, 120: 2, 119: 3, 102: 20}
    best = None
    for mm in range(1, n + 1):
        cnt = sum(int(hist[x]) for x, y in y_of.items() if y.bit_length() <= mm)
        exact = Fraction(1, 16) + n + (mm - n) * Fraction(cnt, total) ** 16     # Eq. 4, L = 16
        assert abs(bexp[mm] - float(exact)) < 1e-12
        if best is None or exact < best[0]:
            best = (exact, mm)
    assert m == best[1]


def test_param_search_degenerate(oracle):
    hist = np.zeros(256, np.uint64)
    assert oracle.param_search(hist, 8)[:3] == (0, 1, 1)
    hist[77] = 10
    assert oracle.param_search(hist, 8)[:3] == (77, 1, 1)      # constant tensor
    hist[:] = 1
    b, n, m, _, _ = oracle.param_search(hist, 8)
    assert n == 8


def test_gaussian_weights_land_on_table5(oracle):
    # Table 5: bf16 models use b in 121..123, n = 6, m = 3 (L = 16); iid Gaussian weights at LLM scales agree
    fx = read_fixture("table5_params.txt")
    bf16_rows = [tuple(map(int, fx[k][0].split())) for k in ("Falcon", "Qwen3-8B", "DeepSeek", "Qwen3-32B", "Llama")]
    assert {r[1:] for r in bf16_rows} == {(6, 3, 16)}
    import torch
    for std, seed in ((0.02, 0), (1.0 / 64.0, 1), (1.0 / np.sqrt(14336.0), 2)):
        g = torch.Generator().manual_seed(seed)
        w = (torch.randn(1 << 20, generator=g) * std).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        hist = np.bincount((w >> 7) & 0xFF, minlength=256).astype(np.uint64)
        b, n, m, _, _ = oracle.param_search(hist, 8)
        assert 119 <= b <= 123 and n == 6 and m == 3, (std, b, n, m)


# ---------------------------------------------------------------- whole streams
def _check_stream(oracle, fx):
    dt, count = int(fx["dtype"][0]), int(fx["count"][0])
    words = np.array([int(t, 16) for t in fx["words"][0].split()], dtype=np.uint16)
    assert words.size == count
    params = tuple(map(int, fx["params"][0].split())) if "params" in fx else None
    keys = ("header", "table", "mask", "low", "smhi", "sm", "high") if dt == 1 else ("header", "table", "mask", "low", "sm", "high")
    expect = np.concatenate([hexbytes(fx[k][0]) for k in keys])
    assert hexbytes(fx["header"][0]).size == 64
    got = oracle.compress(words, dt, params)
    assert got.tolist() == expect.tolist()
    assert oracle.decompress(got, dt, count).tolist() == words.tolist()


def test_stream_hand_16(oracle):
    _check_stream(oracle, read_fixture("stream_hand_16.txt"))


def test_stream_hand_32(oracle):
    _check_stream(oracle, read_fixture("stream_hand_32.txt"))


def test_stream_hand_fp16(oracle):
    # fixes, byte by byte, the 3-bit sign/mantissa-high plane: its width, its bit order (sign above mantissa bits
    # 9..8), its Algorithm 2 packing and its place between the low plane and the byte plane
    fx = read_fixture("stream_hand_fp16.txt")
    assert int(fx["dtype"][0]) == 1
    _check_stream(oracle, fx)


def test_fp16_plane_position_and_content_on_a_large_tensor(oracle):
    # independent of the hand trace: the section after the low plane, undone with the a = 3 closed form of
    # Algorithm 2 for a full block (numpy, not the oracle's unpacker), is sign<<2 | mantissa[9:8] of every element
    rng = np.random.default_rng(41)
    count = 2 * 16384
    words = rng.integers(0, 1 << 16, count).astype(np.uint16)
    s = oracle.compress(words, 1, (15, 5, 2))
    a16 = lambda v: (v + 15) // 16 * 16
    off = 64 + a16(4 * 3) + a16(2048 // 8) + a16(count * 2 // 8)
    want = (((words >> 15) << 2) | ((words >> 8) & 3)).astype(np.uint32)
    for k in range(2):
        sec = s[off + k * 6144: off + (k + 1) * 6144]
        nb = np.concatenate([sec[0::2], sec[1::2]]).astype(np.uint32)        # undo the final fold
        r = np.concatenate([nb[4096:] & 15, nb[4096:] >> 4])                 # residue nibbles of lanes 0..4095
        lane = nb[:4096] | (r << 8)
        e = np.concatenate([lane & 7, (lane >> 6) & 7, (lane >> 3) & 7, (lane >> 9) & 7])
        assert e.tolist() == want[k * 16384:(k + 1) * 16384].tolist()
    byte_plane = s[off + 2 * 6144: off + 2 * 6144 + count]
    assert byte_plane.tolist() == (words & 0xFF).tolist()


def test_fp16_gaussian_lands_on_table5_and_table4(oracle):
    # Table 5: the fp16 models use (7, 4, 3, 16) and (11, 5, 3, 16); Table 4: ratios 1.12 and 1.09. Gaussian fp16
    # weights at checkpoint scales must land in the same regime: n <= E = 5, m = 3, b a little above the mode.
    fx = read_fixture("table5_params.txt")
    rows = [tuple(map(int, fx[k][0].split())) for k in ("Mistral-fp16", "Diffusion-fp16")]
    assert {r[2:] for r in rows} == {(3, 16)} and {r[1] for r in rows} == {4, 5}
    t4 = read_fixture("table4_ratios.txt")
    ratios = [float(t4[k][0]) for k in ("Mistral-fp16", "Diffusion-fp16")]
    lo, hi = min(ratios) - 0.02, max(ratios) + 0.02
    import torch
    for std, seed in ((0.02, 0), (0.01, 1), (0.05, 2)):
        g = torch.Generator().manual_seed(seed)
        w = (torch.randn(1 << 21, generator=g) * std).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
        s = oracle.compress(w, 1)
        b, n, m = int(s[20]), int(s[21]), int(s[22])
        assert n in (4, 5) and m == 3 and min(r[0] for r in rows) <= b <= max(r[0] for r in rows) + 1, (std, b, n, m)
        assert lo < w.nbytes / s.size < hi, (std, w.nbytes / s.size)
        # the sign/mantissa bits cost exactly 11 per element (8 + 3): what is left is Eq. 4's exponent cost
        A = int(s[32:36].view(np.uint32)[0])
        exp_bits = (w.size / 16 + w.size * m + 16 * (n - m) * A) / w.size
        assert abs(8 * s.size / w.size - (11 + exp_bits)) < 0.01


def _sizes_case(oracle, row, dt):
    count, n, m, A, nblocks, padded, groups, total = map(int, row.split())
    b, wide_x, shift = (123, 125, 7) if dt == 0 else (10, 11, 10)
    x = np.full(count, b, np.uint16)
    flagged = np.arange(A) * 16               # one wide value in each of the first A groups
    flagged = flagged[flagged < count]
    assert flagged.size == A
    x[flagged] = wide_x
    words = (x << shift).astype(np.uint16)
    s = oracle.compress(words, dt, (b, n, m))
    assert s.size == total
    hdr = s[:64]
    assert int(hdr[24:28].view(np.uint32)[0]) == nblocks
    assert int(hdr[28:32].view(np.uint32)[0]) == groups
    assert int(hdr[32:36].view(np.uint32)[0]) == A
    assert int(hdr[40:48].view(np.uint64)[0]) == total
    assert oracle.max_compressed_size(dt, count) >= total
    assert np.array_equal(oracle.decompress(s, dt, count), words)


def test_sizes_closed_form_fp16(oracle):
    fx = read_fixture("sizes_hand.txt")
    assert len(fx["case_fp16"]) == 5
    for row in fx["case_fp16"]:
        _sizes_case(oracle, row, 1)


def test_sizes_closed_form(oracle):
    fx = read_fixture("sizes_hand.txt")
    for row in fx["case"]:
        count, n, m, A, nblocks, padded, groups, total = map(int, row.split())
        x = np.full(count, 123, np.uint16)
        flagged = np.arange(A) * 16               # one y = 62 in each of the first A groups
        flagged = flagged[flagged < count]
        assert flagged.size == A
        x[flagged] = 125
        words = (x << 7).astype(np.uint16)
        s = oracle.compress(words, 0, (123, n, m))
        assert s.size == total
        hdr = s[:64]
        assert int(hdr[24:28].view(np.uint32)[0]) == nblocks
        assert int(hdr[28:32].view(np.uint32)[0]) == groups
        assert int(hdr[32:36].view(np.uint32)[0]) == A
        assert int(hdr[40:48].view(np.uint64)[0]) == total
        assert oracle.max_compressed_size(0, count) >= total
        assert np.array_equal(oracle.decompress(s, 0, count), words)


def test_table_is_prefix_sum_of_mask_popcounts(oracle):
    import torch
    g = torch.Generator().manual_seed(11)
    count = 5 * 16384 + 777
    w = (torch.randn(count, generator=g) * 0.02).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    s = oracle.compress(w, 0)
    nblocks = int(s[24:28].view(np.uint32)[0])
    assert nblocks == 6
    table = s[64:64 + 4 * (nblocks + 1)].view(np.uint32)
    mask_off = 64 + ((4 * (nblocks + 1) + 15) // 16) * 16
    groups = int(s[28:32].view(np.uint32)[0])
    bits = np.unpackbits(s[mask_off:mask_off + (groups + 7) // 8], bitorder="little")[:groups]
    per_block = [int(bits[k * 1024:(k + 1) * 1024].sum()) for k in range(nblocks)]
    assert table.tolist() == np.concatenate([[0], np.cumsum(per_block)]).tolist()   # textbook exclusive scan
    assert int(s[32:36].view(np.uint32)[0]) == int(bits.sum())


def test_eq4_predicts_measured_exponent_bits(oracle):
    # For iid data the expected-bits model of Eq. 4 must match the stream actually written (mask + low + high)
    import torch
    g = torch.Generator().manual_seed(12)
    count = 64 * 16384
    w = (torch.randn(count, generator=g) * 0.02).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    hist = np.bincount((w >> 7) & 0xFF, minlength=256).astype(np.uint64)
    b, n, m, _, bexp = oracle.param_search(hist, 8)
    s = oracle.compress(w, 0)
    assert (int(s[20]), int(s[21]), int(s[22])) == (b, n, m)
    A = int(s[32:36].view(np.uint32)[0])
    measured = (count / 16 + count * m + 16 * (n - m) * A) / count
    assert abs(measured - bexp[m]) < 0.01
    # and the artifact's Qwen3-32B figure (8 + 3.8465 bits) is in the same regime as Gaussian weights
    fx = read_fixture("artifact_bits.txt")
    assert abs(float(fx["bits_per_element"][0]) - 8 - float(fx["exponent_bits_per_element"][0])) < 1e-9
    assert 3.3 < measured < float(fx["exponent_bits_per_element"][0]) + 0.2
    ratio = 2.0 * count / s.size
    assert 1.33 < ratio < 1.42


@pytest.mark.parametrize("dt", [0, 1])
def test_all_bit_patterns_roundtrip(oracle, dt):
    allw = np.arange(1 << 16, dtype=np.uint16)
    rng = np.random.default_rng(13)
    for words in (allw, rng.permutation(allw), np.repeat(allw, 16)[: 40 * 16384 + 5]):
        s = oracle.compress(words, dt)
        assert s.size <= oracle.max_compressed_size(dt, words.size)
        assert np.array_equal(oracle.decompress(s, dt, words.size), words)


@pytest.mark.parametrize("dt", [0, 1])
def test_tiny_and_ragged_roundtrip(oracle, dt):
    rng = np.random.default_rng(14)
    for count in (0, 1, 2, 15, 16, 17, 31, 33, 127, 1000, 16383, 16384, 16385, 16384 + 16, 3 * 16384 + 4097):
        words = rng.integers(0x3000, 0x3FFF, count).astype(np.uint16)
        s = oracle.compress(words, dt)
        assert s.size % 16 == 0 and s.size <= oracle.max_compressed_size(dt, count)
        assert np.array_equal(oracle.decompress(s, dt, count), words)
    const = np.full(100, 0x3C00, np.uint16)
    s = oracle.compress(const, dt)
    assert (int(s[21]), int(s[22])) == (1, 1)       # constant tensor: n = 1, m = 1


def test_every_param_combination_roundtrips(oracle):
    rng = np.random.default_rng(15)
    count = 16384 + 300
    for n in range(1, 9):
        for m in range(1, n + 1):
            half = 1 << (n - 1)
            lo, hi = max(0, 120 - (half - 1)), min(255, 120 + half)
            x = rng.integers(lo, hi + 1, count).astype(np.uint16) if n < 8 else rng.integers(0, 256, count).astype(np.uint16)
            words = ((x << 7) | rng.integers(0, 128, count).astype(np.uint16) | (rng.integers(0, 2, count).astype(np.uint16) << 15)).astype(np.uint16)
            s = oracle.compress(words, 0, (120, n, m))
            assert np.array_equal(oracle.decompress(s, 0, count), words), (n, m)


def test_forced_params_must_be_lossless(oracle):
    words = (np.array([100, 130] * 8, np.uint16) << 7).astype(np.uint16)
    with pytest.raises(oracle.OracleError) as e:
        oracle.compress(words, 0, (120, 3, 2))
    assert e.value.status == -5


def test_decoder_rejects_damaged_streams(oracle):
    rng = np.random.default_rng(16)
    words = rng.integers(0x3A00, 0x3FFF, 40000).astype(np.uint16)
    s = oracle.compress(words, 0)
    for off, val in ((0, 0x58), (4, 9), (6, 1), (8, 1), (21, 0), (22, 9), (24, 77), (40, 3)):
        bad = s.copy()
        bad[off] = val
        with pytest.raises(oracle.OracleError):
            oracle.decompress(bad, 0, words.size)
    with pytest.raises(oracle.OracleError):
        oracle.decompress(s[:-16], 0, words.size)
    with pytest.raises(oracle.OracleError):
        oracle.decompress(s, 1, words.size)


# ---------------------------------------------------------------- fp32 (Sec. 6.2: the mantissa is not compressed)
def test_fp32_split_fields(oracle):
    # 1.0f = 0x3F800000: exponent 127; -2.5f = 0xC0200000: sign 1, exponent 128, mantissa 0x200000
    assert oracle.split(0x3F800000, 2) == (127, 0)
    assert oracle.split(0xC0200000, 2) == (128, 0x800000 | 0x200000)
    rng = np.random.default_rng(31)
    for w in rng.integers(0, 1 << 32, 4000, dtype=np.uint64):
        x, sm = oracle.split(int(w), 2)
        assert oracle.join(x, sm, 2) == int(w)
    vals = rng.normal(0, 0.02, 300).astype(np.float32)
    for v, w in zip(vals, vals.view(np.uint32)):
        _, e = np.frexp(np.float64(v))
        assert oracle.split(int(w), 2)[0] == e - 1 + 127          # exponent field = floor(log2 |v|) + bias


def test_fp32_stream_hand(oracle):
    fx = read_fixture("stream_hand_fp32.txt")
    words = np.array([int(t, 16) for t in fx["words"][0].split()], dtype=np.uint32)
    expect = np.concatenate([hexbytes(fx[k][0]) for k in ("header", "table", "mask", "low", "sm", "smlo")])
    got = oracle.compress(words, 2)
    assert got.tolist() == expect.tolist()
    assert oracle.decompress(got, 2, 16).tolist() == words.tolist()


def test_fp32_is_the_bf16_stream_of_the_high_halves_plus_raw_low_halves(oracle):
    # an fp32 word's high half has bf16's layout, so the fp32 stream must be the bf16 stream of the high halves
    # (same parameters, table, mask, planes, records) with the low halves stored as they are in between
    rng = np.random.default_rng(32)
    count = 3 * 16384 + 777
    w = rng.normal(0, 0.02, count).astype(np.float32).view(np.uint32)
    s32 = oracle.compress(w, 2)
    s16 = oracle.compress((w >> 16).astype(np.uint16), 0)
    a16 = lambda v: (v + 15) // 16 * 16
    high_bytes = int(s16[32:36].view(np.uint32)[0]) * 2 * (int(s16[21]) - int(s16[22]))
    cut = s16.size - a16(high_bytes)                          # where the bf16 stream's records start
    assert s32[20:24].tolist() == s16[20:24].tolist()          # b, n, m, L
    assert s32[64:cut].tolist() == s16[64:cut].tolist()        # table, mask, low plane, byte plane
    lo = s32[cut:cut + 2 * count].view(np.uint16)
    assert lo.tolist() == (w & 0xFFFF).astype(np.uint16).tolist()
    assert s32[cut + a16(2 * count):].tolist() == s16[cut:].tolist()   # records
    assert s32.size == s16.size + a16(2 * count)
    assert int(s32[40:48].view(np.uint64)[0]) == s32.size and s32[6] == 2


def test_fp32_special_values_and_tails_roundtrip(oracle):
    rng = np.random.default_rng(33)
    special = np.array([0x00000000, 0x80000000, 0x7F800000, 0xFF800000, 0x7FC00001, 0x00000001, 0x007FFFFF,
                        0x7F7FFFFF, 0xFFFFFFFF, 0x3F800000], dtype=np.uint32)
    for count in (0, 1, 15, 16, 17, 1000, 16384, 16385, 2 * 16384 + 4097):
        w = rng.integers(0, 1 << 32, count, dtype=np.uint64).astype(np.uint32)
        w[: min(count, special.size)] = special[: min(count, special.size)]
        s = oracle.compress(w, 2)
        assert s.size % 16 == 0 and s.size <= oracle.max_compressed_size(2, count)
        assert np.array_equal(oracle.decompress(s, 2, count), w)
    with pytest.raises(oracle.OracleError):
        oracle.decompress(oracle.compress(special, 2), 0, special.size)


def test_fp32_gaussian_lands_on_table5_and_table4(oracle):
    # Table 5: fp32 models use (121..125, 6, 3, 16); Table 4: ratio 1.15 for the fp32 models
    fx = read_fixture("table5_params.txt")
    rows = [tuple(map(int, fx[k][0].split())) for k in ("OLMo", "BERT", "Wav2Vec")]
    assert {r[1:] for r in rows} == {(6, 3, 16)}
    rng = np.random.default_rng(34)
    w = rng.normal(0, 0.02, 1 << 21).astype(np.float32).view(np.uint32)
    s = oracle.compress(w, 2)
    assert 119 <= int(s[20]) <= 125 and (int(s[21]), int(s[22])) == (6, 3)
    assert 1.13 < w.nbytes / s.size < 1.18


# ---------------------------------------------------------------- frequency-rank variant (Sec. 4.2, Algorithm 1)
def test_ranked_stream_hand(oracle):
    fx = read_fixture("stream_hand_ranked.txt")
    words = np.array([int(t, 16) for t in fx["words"][0].split()], dtype=np.uint16)
    unmap = np.zeros(256, np.uint8)
    head = hexbytes(fx["unmap_head"][0])
    unmap[:head.size] = head
    expect = np.concatenate([hexbytes(fx["header"][0]), unmap] + [hexbytes(fx[k][0]) for k in ("table", "mask", "low", "sm", "high")])
    got = oracle.compress_ranked(words, 0)
    assert got.tolist() == expect.tolist()
    assert oracle.decompress(got, 0, words.size).tolist() == words.tolist()


def test_ranked_table_sorts_exponents_by_falling_count(oracle):
    rng = np.random.default_rng(4)
    x = rng.choice(np.arange(100, 140), size=50000, p=np.r_[np.full(20, 0.04), np.full(20, 0.01)]).astype(np.uint16)
    x[:7] = 3                       # a rare exponent far away, and ties among the plentiful ones are likely
    words = (x << 7) | rng.integers(0, 128, x.size).astype(np.uint16)
    s = oracle.compress_ranked(words, 0)
    counts = np.bincount(x, minlength=256)
    occupied = int((counts > 0).sum())
    table = s[64:64 + 256]
    order = sorted(np.flatnonzero(counts), key=lambda e: (-counts[e], e))     # textbook: count down, exponent up
    assert table[:occupied].tolist() == order and not table[occupied:].any()
    n, m = int(s[21]), int(s[22])
    assert n == max(1, int(occupied - 1).bit_length()) and 1 <= m <= n and s[7] == 1 and s[20] == 0
    assert np.array_equal(oracle.decompress(s, 0, words.size), words)


def test_ranked_cost_never_exceeds_the_linear_transform(oracle):
    """Sorting by frequency minimises sum count * code over all one-to-one codes (rearrangement inequality), so
    the rank code's Eq. 3 cost is at most the best linear transform's, for any histogram."""
    rng = np.random.default_rng(8)
    for trial in range(40):
        hist = np.zeros(256, np.uint64)
        lo = int(rng.integers(0, 200)); width = int(rng.integers(1, 50))
        hist[lo:lo + width] = rng.integers(0, 10000, width).astype(np.uint64)
        if not hist.any():
            continue
        ranked_cost = int(sum(int(c) * r for r, c in enumerate(sorted((int(v) for v in hist if v), reverse=True))))
        b, n, m, cost, _ = oracle.param_search(hist, 8)
        assert ranked_cost <= int(cost[b]), trial


def test_ranked_roundtrip_patterns_tails_and_dtypes(oracle):
    import torch
    rng = np.random.default_rng(15)
    for dt in (0, 1):
        w = rng.permutation(1 << 16).astype(np.uint16)               # every bit pattern: all exponents occupied
        s = oracle.compress_ranked(w, dt)
        assert int(s[21]) == (8 if dt == 0 else 5)
        assert np.array_equal(oracle.decompress(s, dt, w.size), w)
    for count in (0, 1, 15, 16, 17, 100, 16384, 16385, 16384 * 3 + 5000):
        g = torch.Generator().manual_seed(count)
        w = (torch.randn(count, generator=g) * 0.02).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        s = oracle.compress_ranked(w, 0)
        assert np.array_equal(oracle.decompress(s, 0, count), w)
    f = (torch.randn(40000, generator=torch.Generator().manual_seed(2)) * 0.02).view(torch.int32).numpy().view(np.uint32)
    assert np.array_equal(oracle.decompress(oracle.compress_ranked(f, 2), 2, f.size), f)
    one = np.full(16384 + 3, 0x3F80, np.uint16)                      # one exponent: n = m = 1, every y = 0
    s = oracle.compress_ranked(one, 0)
    assert (int(s[21]), int(s[22]), int(s[32])) == (1, 1, 0) and s[64] == 127


def test_ranked_is_a_little_smaller_on_gaussian_weights(oracle):
    """Sec. 6.6 (ablation): the linear transform approximates the frequency order and gives up a little ratio."""
    import torch
    w = (torch.randn(1 << 20, generator=torch.Generator().manual_seed(5)) * 0.02).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    linear, ranked = oracle.compress(w, 0).size, oracle.compress_ranked(w, 0).size
    assert ranked < linear < ranked * 1.03


# ---------------------------------------------------------------- block-wise variant (Sec. 5.5 per block)
def _blockwise_table(s, nblocks):
    """(b, n, m, sum of m before, record bytes before) of every entry of a block-wise stream's block table."""
    t = s[64:64 + 16 * (nblocks + 1)]
    return [(int(t[16 * k]), int(t[16 * k + 1]), int(t[16 * k + 2]), int(t[16 * k + 4:16 * k + 8].view(np.uint32)[0]),
             int(t[16 * k + 8:16 * k + 16].view(np.uint64)[0])) for k in range(nblocks + 1)]


def test_blockwise_stream_hand(oracle):
    fx = read_fixture("stream_hand_blockwise.txt")
    base = int(fx["block0_word_base"][0], 16)
    words = np.concatenate([(base + (np.arange(16384) & 127)).astype(np.uint16),
                            np.array([int(t, 16) for t in fx["block1_words"][0].split()], dtype=np.uint16)])
    assert words.size == int(fx["count"][0])
    expect = np.concatenate([hexbytes(fx["header"][0]), hexbytes(fx["table"][0]),
                             np.zeros(int(fx["mask_zero_bytes"][0]), np.uint8),
                             np.zeros(int(fx["low_zero_bytes"][0]), np.uint8), hexbytes(fx["low_tail"][0]),
                             (np.arange(16384) % 128).astype(np.uint8), hexbytes(fx["sm_block1"][0])])
    got = oracle.compress_blockwise(words, 0)
    assert got.size == 18720 and got.tolist() == expect.tolist()
    assert oracle.decompress(got, 0, words.size).tolist() == words.tolist()


def test_blockwise_equals_the_per_tensor_stream_when_all_blocks_agree(oracle):
    # every block holds the same multiset of exponents, so every block's search gives the tensor's (b, n, m):
    # mask, low plane, sign/mantissa bytes and records must then be the per-tensor stream's, byte for byte
    rng = np.random.default_rng(51)
    nblocks = 3
    one = np.clip(np.round(rng.normal(121, 2.0, 16384)), 100, 130).astype(np.uint16)
    x = np.concatenate([rng.permutation(one) for _ in range(nblocks)])
    words = ((x << 7) | rng.integers(0, 128, x.size).astype(np.uint16)).astype(np.uint16)
    a = oracle.compress(words, 0)
    b = oracle.compress_blockwise(words, 0)
    params = (int(a[20]), int(a[21]), int(a[22]))
    table = _blockwise_table(b, nblocks)
    assert [e[:3] for e in table[:nblocks]] == [params] * nblocks
    assert [e[3] for e in table] == [k * params[2] for k in range(nblocks + 1)]
    per_tensor_table = a[64:64 + 4 * (nblocks + 1)].view(np.uint32)
    assert [e[4] for e in table] == [int(v) * 2 * (params[1] - params[2]) for v in per_tensor_table]
    a16 = lambda v: (v + 15) // 16 * 16
    assert a[64 + a16(4 * (nblocks + 1)):].tolist() == b[64 + a16(16 * (nblocks + 1)):].tolist()
    assert b[7] == 2 and not b[20:23].any() and b[32:36].tolist() == a[32:36].tolist()
    assert int(b[40:48].view(np.uint64)[0]) == b.size == a.size + a16(16 * (nblocks + 1)) - a16(4 * (nblocks + 1))


def test_blockwise_parameters_are_each_blocks_own_search(oracle):
    # blocks drawn at different scales choose different parameters; each must be what the search of Sec. 5.5 gives
    # on that block's histogram alone, the offsets must chain, and the size must follow the closed form
    import torch
    g = torch.Generator().manual_seed(52)
    parts = [torch.randn(16384, generator=g) * 0.02, torch.randn(16384, generator=g) * 3.0, torch.zeros(16384),
             torch.randn(5000, generator=g) * 1e-3]
    parts[2][::7] = 1.0                      # exact zeros next to ones: exponents 0 and 127, n = 8
    words = torch.cat(parts).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    s = oracle.compress_blockwise(words, 0)
    nblocks = 4
    table = _blockwise_table(s, nblocks)
    m_sum = high = wide_total = 0
    low_bytes = 0
    for k in range(nblocks):
        blk = words[k * 16384:(k + 1) * 16384]
        hist = np.bincount((blk >> 7) & 0xFF, minlength=256).astype(np.uint64)
        b, n, m, _, _ = oracle.param_search(hist, 8)
        assert table[k][:3] == (b, n, m), k
        assert table[k][3] == m_sum and table[k][4] == high
        y = (b - ((blk.astype(np.int64) >> 7) & 0xFF)) % (1 << n)
        padded = 16384 if k < 3 else 8192
        y = np.concatenate([y, np.zeros(padded - y.size, np.int64)]).reshape(-1, 16)
        wide = int((np.bitwise_or.reduce(y, axis=1) >> m != 0).sum())
        wide_total += wide
        high += wide * 2 * (n - m)
        low_bytes += padded * m // 8
        m_sum += m
    assert table[nblocks] == (0, 0, 0, m_sum, high)
    assert len({e[:3] for e in table[:nblocks]}) >= 3
    assert int(s[32:36].view(np.uint32)[0]) == wide_total
    a16 = lambda v: (v + 15) // 16 * 16
    groups = (3 * 16384 + 8192) // 16
    assert s.size == 64 + a16(16 * 5) + a16((groups + 7) // 8) + a16(low_bytes) + a16(words.size) + a16(high)
    assert s.size <= oracle.max_compressed_size_blockwise(0, words.size)
    assert np.array_equal(oracle.decompress(s, 0, words.size), words)
    # where one stray zero forces n = 8 on the whole tensor, the blocks without it keep their narrow codes
    assert s.size < oracle.compress(words, 0).size


@pytest.mark.parametrize("dt", [0, 1, 2])
def test_blockwise_roundtrip_patterns_and_tails(oracle, dt):
    rng = np.random.default_rng(53 + dt)
    if dt == 2:
        full = rng.integers(0, 1 << 32, 70000, dtype=np.uint64).astype(np.uint32)
    else:
        full = rng.permutation(1 << 16).astype(np.uint16)
    s = oracle.compress_blockwise(full, dt)
    assert s.size <= oracle.max_compressed_size_blockwise(dt, full.size)
    assert np.array_equal(oracle.decompress(s, dt, full.size), full)
    for count in (0, 1, 15, 16, 17, 1000, 16384, 16385, 2 * 16384 + 4097):
        w = full[:count]
        s = oracle.compress_blockwise(w, dt)
        assert s.size % 16 == 0 and s.size <= oracle.max_compressed_size_blockwise(dt, count)
        assert np.array_equal(oracle.decompress(s, dt, count), w)
    worst = np.tile(np.array([0x0000, 0x7F80] * 8, np.uint16), 2048 * 2 + 3) if dt == 0 else None
    if worst is not None:    # every group wide with n = 8 in every block: the size bound must hold
        s = oracle.compress_blockwise(worst, 0)
        assert s.size <= oracle.max_compressed_size_blockwise(0, worst.size)


def test_blockwise_decoder_rejects_damaged_tables(oracle):
    rng = np.random.default_rng(54)
    words = rng.integers(0x3A00, 0x3FFF, 40000).astype(np.uint16)
    s = oracle.compress_blockwise(words, 0)
    assert np.array_equal(oracle.decompress(s, 0, words.size), words)
    for off, val in ((7, 3), (20, 1), (64 + 1, 9), (64 + 2, 0), (64 + 16 + 4, 7), (64 + 16 + 8, 1), (64 + 48 + 4, 0)):
        bad = s.copy()
        bad[off] = val
        with pytest.raises(oracle.OracleError):
            oracle.decompress(bad, 0, words.size)
