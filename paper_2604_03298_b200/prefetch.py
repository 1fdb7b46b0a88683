"""Layer-wise weight prefetch: decompress layer i + 1 on a side stream while layer i computes (Sec. 6.3
"End-to-End Inference Speedup": the paper overlaps layer-wise decompression with the forward pass).

The weights of all layers stay compressed in device memory; two layer-sized buffers hold the layer being used
and the layer being decompressed. Each layer is one `enec_decompress_batched` launch on the side stream; CUDA
events order the two streams (the side stream must not overwrite a buffer the main stream still reads, the main
stream must not read a buffer before its decompression has finished). Only allocation, streams and events are
torch's; every codec step runs in the CUDA library.
"""
from typing import Callable, List, Sequence

import torch

from . import binding as enec

_DT = {torch.bfloat16: enec.BF16, torch.float16: enec.FP16, torch.float32: enec.FP32}


class LayerPrefetcher:
    """`layers[i]` is a list of (stream_tensor, stream_bytes, shape) of one dtype; all layers have the same shapes."""

    def __init__(self, layers: Sequence[Sequence[tuple]], dtype: torch.dtype, device="cuda"):
        self.layers = layers
        self.dtype = dtype
        self.dt = _DT[dtype]
        shapes = [tuple(shape) for _, _, shape in layers[0]]
        for layer in layers:
            assert [tuple(shape) for _, _, shape in layer] == shapes, "layers must share their tensor shapes"
        self.buffers = [[torch.empty(shape, dtype=dtype, device=device) for shape in shapes] for _ in range(2)]
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.side = torch.cuda.Stream(device=device)
        self.ready = [torch.cuda.Event() for _ in range(2)]   # buffer b holds a decompressed layer
        self.freed = [torch.cuda.Event() for _ in range(2)]   # the main stream is done reading buffer b

    def _decompress_into(self, layer_index: int, b: int) -> None:
        items = [(src, nbytes, dst, dst.numel()) for (src, nbytes, _), dst in zip(self.layers[layer_index], self.buffers[b])]
        st = enec.enec_decompress_batched(items, self.dt, self.status)
        if st != 0:
            raise enec.EnecError(st, f"enec_decompress_batched layer {layer_index}")

    def run(self, forward: Callable[[int, List[torch.Tensor]], None], overlap: bool = True) -> None:
        """Calls forward(i, weights_of_layer_i) for every layer on the current stream. With overlap the next
        layer is decompressed on the side stream meanwhile; without it every layer is decompressed on the
        current stream right before its use."""
        main = torch.cuda.current_stream()
        n = len(self.layers)
        if not overlap:
            for i in range(n):
                self._decompress_into(i, 0)
                forward(i, self.buffers[0])
            return
        self.side.wait_stream(main)
        with torch.cuda.stream(self.side):
            self._decompress_into(0, 0)
            self.ready[0].record(self.side)
        for i in range(n):
            b = i & 1
            if i + 1 < n:
                with torch.cuda.stream(self.side):
                    if i >= 1:
                        self.side.wait_event(self.freed[b ^ 1])   # layer i - 1 has finished with that buffer
                    self._decompress_into(i + 1, b ^ 1)
                    self.ready[b ^ 1].record(self.side)
            main.wait_event(self.ready[b])
            forward(i, self.buffers[b])
            self.freed[b].record(main)
        main.wait_stream(self.side)

    def capture(self, forward: Callable[[int, List[torch.Tensor]], None], overlap: bool = True) -> "torch.cuda.CUDAGraph":
        """Records one run() (all layers: decompress launches, the events between the two streams and whatever
        `forward` enqueues) into a CUDA graph and returns it; `graph.replay()` then repeats the whole pass with
        one submission. A layer's batched launch carries its tensor list in the kernel parameters, so the
        recorded launches need no descriptor copy. `forward` must not synchronise with the host."""
        self.run(forward, overlap)          # first use outside the capture: module attributes, allocator warm-up
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run(forward, overlap)
        return graph

    def check_status(self) -> None:
        code = int(self.status.item())
        if code != 0:
            raise enec.EnecError(code, "device status")
