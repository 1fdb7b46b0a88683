"""Measures what layer-wise decompression costs a forward pass on one GPU: Llama-3-8B-shaped layers, GEMMs of
`tokens` rows against every weight matrix, (a) weights resident uncompressed, (b) each layer decompressed on the
same stream right before use, (c) the next layer decompressed on a side stream meanwhile, (d) pass (c) recorded
into a CUDA graph and replayed. Prints one JSON line.

    python -m paper_2604_03298_b200.prefetch_demo [--layers 8] [--tokens 2048] [--steps 10]
"""
import argparse
import json

import torch

from . import runner, synth
from .prefetch import LayerPrefetcher


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--tokens", type=int, default=2048)
    ap.add_argument("--steps", type=int, default=10)
    args = ap.parse_args()
    import dataclasses
    raw_layers, layers = [], []
    for li in range(args.layers):
        specs = [dataclasses.replace(s, seed=s.seed + 100 * li) for s in synth.config_specs(2) if len(s.shape) == 2]
        raw = [synth.make_tensor(s, "cuda") for s in specs]
        cs = runner.CodecSet.allocate(raw)
        cs.compress_all()
        torch.cuda.synchronize()
        cs.check_status()
        sizes = cs.sizes.cpu().tolist()
        raw_layers.append(raw)
        layers.append([(cs.streams[i][:sizes[i]].clone(), sizes[i], tuple(raw[i].shape)) for i in range(len(raw))])
        del cs
    acts = {w.shape[1]: torch.randn(args.tokens, w.shape[1], device="cuda").to(torch.bfloat16) for w in raw_layers[0]}
    outs = {w.shape: torch.empty(args.tokens, w.shape[0], dtype=torch.bfloat16, device="cuda") for w in raw_layers[0]}

    def forward(i, weights):
        for w in weights:
            torch.matmul(acts[w.shape[1]], w.t(), out=outs[w.shape])

    pf = LayerPrefetcher(layers, torch.bfloat16)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.steps

    ms_resident = timed(lambda: [forward(i, raw_layers[i]) for i in range(args.layers)])
    ms_serial = timed(lambda: pf.run(forward, overlap=False))
    ms_overlap = timed(lambda: pf.run(forward, overlap=True))
    ms_decode_only = timed(lambda: pf.run(lambda i, w: None, overlap=False))
    graph = pf.capture(forward, overlap=True)
    ms_graph = timed(graph.replay)
    pf.check_status()
    flops = 2.0 * args.tokens * sum(w.numel() for w in raw_layers[0]) * args.layers
    raw_bytes = sum(w.numel() * 2 for layer in raw_layers for w in layer)
    comp_bytes = sum(n for layer in layers for _, n, _ in layer)
    print(json.dumps({
        "layers": args.layers, "tokens": args.tokens, "steps": args.steps,
        "weights_raw_bytes": raw_bytes, "weights_compressed_bytes": comp_bytes,
        "ms_forward_resident": ms_resident, "ms_forward_decompress_same_stream": ms_serial,
        "ms_forward_prefetch_side_stream": ms_overlap, "ms_forward_prefetch_cuda_graph": ms_graph,
        "ms_decompress_only": ms_decode_only,
        "gemm_tflops_resident": flops / (ms_resident * 1e-3) / 1e12,
        "overlap_cost_ms": ms_overlap - ms_resident, "serial_cost_ms": ms_serial - ms_resident,
        "hidden_fraction_of_decompress": 1.0 - (ms_overlap - ms_resident) / ms_decode_only,
    }))


if __name__ == "__main__":
    main()
