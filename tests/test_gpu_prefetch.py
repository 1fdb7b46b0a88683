"""Layer-wise prefetch: every layer's weights, decompressed on the side stream while the previous layer is in
use, must be bit-identical to the original tensors, with and without overlap."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _compressed_layers(n_layers, scale):
    from paper_2604_03298_b200 import runner, synth
    raw_layers, layers = [], []
    for li in range(n_layers):
        specs = [s for s in synth.config_specs(2, scale=scale)]
        specs = [type(s)(s.name, s.dtype, s.shape, s.dist, s.mean, s.std, s.seed + 100 * li) for s in specs]
        raw = [synth.make_tensor(s, "cuda") for s in specs]
        cs = runner.CodecSet.allocate(raw)
        cs.compress_all()
        torch.cuda.synchronize()
        cs.check_status()
        sizes = cs.sizes.cpu().tolist()
        raw_layers.append(raw)
        layers.append([(cs.streams[i][:sizes[i]].clone(), sizes[i], tuple(raw[i].shape)) for i in range(len(raw))])
    return raw_layers, layers


@pytest.mark.parametrize("overlap", [True, False])
def test_prefetched_layers_are_bit_exact(overlap):
    from paper_2604_03298_b200.prefetch import LayerPrefetcher
    raw_layers, layers = _compressed_layers(n_layers=6, scale=8)
    pf = LayerPrefetcher(layers, torch.bfloat16)
    seen = []
    sink = torch.zeros(len(layers), dtype=torch.int64, device="cuda")

    def forward(i, weights):
        # stays on the stream (no host synchronisation): counts differing 16-bit words against the original
        diff = sum((w.view(torch.int16) != r.view(torch.int16)).sum() for w, r in zip(weights, raw_layers[i]))
        sink[i] = diff
        # some extra work on the weights so that the side stream really runs ahead of the main stream
        x = torch.ones(64, weights[0].shape[1], dtype=torch.bfloat16, device="cuda")
        for _ in range(4):
            x = (x @ weights[0].t())[:, :weights[0].shape[1]].contiguous()
        seen.append(i)

    for _ in range(3):
        pf.run(forward, overlap=overlap)
    torch.cuda.synchronize()
    pf.check_status()
    assert seen == list(range(len(layers))) * 3
    assert int(sink.sum().item()) == 0


def test_a_captured_pass_replays_bit_exact():
    """The whole prefetched pass recorded into a CUDA graph: every replay decompresses every layer again."""
    from paper_2604_03298_b200.prefetch import LayerPrefetcher
    raw_layers, layers = _compressed_layers(n_layers=5, scale=8)
    pf = LayerPrefetcher(layers, torch.bfloat16)
    sink = torch.zeros(len(layers), dtype=torch.int64, device="cuda")
    scratch = [torch.zeros_like(w, dtype=torch.bool) for w in raw_layers[0]]

    def forward(i, weights):
        total = sink[i] * 0
        for w, r, tmp in zip(weights, raw_layers[i], scratch):
            torch.ne(w.view(torch.int16), r.view(torch.int16), out=tmp)
            total = total + tmp.sum()
        sink[i] += total + 1       # one per visit, plus the number of differing words

    graph = pf.capture(forward)
    torch.cuda.synchronize()
    sink.zero_()
    for rep in range(3):
        for buf in pf.buffers:     # a replay must not pass on what an earlier pass left in the buffers
            for t in buf:
                t.zero_()
        graph.replay()
    torch.cuda.synchronize()
    pf.check_status()
    assert sink.tolist() == [3] * len(layers)
