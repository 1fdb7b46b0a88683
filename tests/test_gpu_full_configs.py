"""The five workload families at their full sizes, through the calls and launch configuration the benchmark times
(runner.CodecSet: one enec_compress and one enec_decompress per tensor on one stream).

Every tensor must come back bit for bit (tolerance 0). Every stream must be self-consistent (header length = the
length the device reported, within the bound of enec_max_compressed_size). A sample of tensors that the CPU oracle
can encode in seconds must match the oracle's stream byte for byte."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _run_set(specs, oracle, sample, reuse=None):
    import paper_2604_03298_b200 as enec
    from paper_2604_03298_b200 import runner, synth
    cache = {}
    raw = []
    for i, s in enumerate(specs):
        key = reuse(i, s) if reuse else i
        if key not in cache:
            cache[key] = synth.make_tensor(s, "cuda")
        raw.append(cache[key])
    cs = runner.CodecSet.allocate(raw)
    cs.compress_all()
    cs.decompress_all()
    torch.cuda.synchronize()
    cs.check_status()
    cs.verify_roundtrip()
    sizes = cs.sizes.cpu().tolist()
    for i, t in enumerate(raw):
        dt = 0 if t.dtype == torch.bfloat16 else 1
        assert 80 <= sizes[i] <= enec.enec_max_compressed_size(dt, t.numel())
        assert sizes[i] % 16 == 0
    heads = torch.stack([st[:64] for st in cs.streams]).cpu().numpy()
    for i, t in enumerate(raw):
        assert heads[i, :4].tobytes() == b"ENEC"
        assert int(heads[i, 8:16].view(np.uint64)[0]) == t.numel()
        assert int(heads[i, 40:48].view(np.uint64)[0]) == sizes[i]
    for i in sample:
        t = raw[i]
        dt = 0 if t.dtype == torch.bfloat16 else 1
        words = t.reshape(-1).view(torch.int16).cpu().numpy().view(np.uint16)
        want = oracle.compress(words, dt)
        got = cs.streams[i][:sizes[i]].cpu().numpy()
        assert got.size == want.size and np.array_equal(got, want), f"tensor {i} ({specs[i].name}): stream differs"
    return sum(t.numel() * 2 for t in raw) / sum(sizes)


def test_config2_llama_layer_full(oracle):
    from paper_2604_03298_b200 import synth
    specs = synth.config_specs(2)
    ratio = _run_set(specs, oracle, sample=range(len(specs)))          # every tensor against the oracle
    assert 1.36 < ratio < 1.40


def test_config3_llama8b_full(oracle):
    from paper_2604_03298_b200 import synth
    specs = synth.config_specs(3)
    assert len(specs) == 291
    names = [s.name for s in specs]
    sample = [names.index(n) for n in ("l0.input_norm", "l5.k", "l17.q", "l31.down", "final_norm", "lm_head")]
    ratio = _run_set(specs, oracle, sample)
    assert 1.36 < ratio < 1.40                                          # Table 4 reports 1.36 for Llama-3.1-8B


def test_config4_heavy_tailed_full(oracle):
    from paper_2604_03298_b200 import synth
    specs = synth.config_specs(4)
    assert len(specs) == 128 and specs[0].shape == (4096, 4096)
    ratio = _run_set(specs, oracle, sample=(0, 31, 45, 63, 64, 95, 100, 127))
    assert 1.0 < ratio < 1.35                                           # zeros force the full exponent width


def test_config5_moe_full(oracle):
    from paper_2604_03298_b200 import synth
    specs = synth.config_specs(5)
    assert len(specs) == 768 + 4096
    # expert matrices share three shapes and one distribution: 24 distinct draws stand for the 768
    reuse = lambda i, s: (s.shape, i % 24) if len(s.shape) == 2 else ("v", i)
    ratio = _run_set(specs, oracle, sample=(0, 1, 2, 767, 768, 769, 2000, 4863), reuse=reuse)
    assert 1.36 < ratio < 1.40
