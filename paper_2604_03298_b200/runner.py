"""Host-side driver of the codec over a set of tensors: allocation, one compress pass, one decompress pass,
sharding of a tensor list over ranks and max-over-ranks timing. Used by the benchmark and the tests.

Every codec step runs in the CUDA library; this module only allocates with torch, marshals through the
binding and reads status words.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import torch

from . import binding as enec

_DT = {torch.bfloat16: enec.BF16, torch.float16: enec.FP16, torch.float32: enec.FP32}


def shard(items: list, rank: int, world: int) -> list:
    """Round-robin split of a tensor list over ranks: tensors are independent streams, so a rank needs no
    data from any other rank (no collective on the data path)."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    return items[rank::world]


def max_over_ranks(value: float, group=None) -> float:
    """Largest value over all ranks of the process group (the rank's own value without a group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def sum_over_ranks(value: float, group=None) -> float:
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t.item())


@dataclass
class CodecSet:
    """Device buffers of a tensor set: raw tensors, one stream buffer each (at capacity) and outputs."""
    raw: List[torch.Tensor]
    streams: List[torch.Tensor] = field(default_factory=list)
    outs: List[torch.Tensor] = field(default_factory=list)
    sizes: Optional[torch.Tensor] = None      # int64 [n]: stream lengths, written by the device
    status: Optional[torch.Tensor] = None     # int32 [1]: first device error of any call
    shared_outs: bool = False
    batches: Optional[list] = None   # cached item arrays of the batched calls
    side: List[torch.cuda.Stream] = field(default_factory=list)   # side streams of the multi-stream passes

    @classmethod
    def allocate(cls, raw: List[torch.Tensor], share_output: bool = False) -> "CodecSet":
        dev = raw[0].device
        cs = cls(raw=[t.contiguous() for t in raw])
        # room for every variant of the stream (the frequency-rank variant is 256 bytes longer, the block-wise one
        # has the larger table)
        cs.streams = [torch.empty(max(enec.enec_max_compressed_size_ranked(_DT[t.dtype], t.numel()),
                                      enec.enec_max_compressed_size_blockwise(_DT[t.dtype], t.numel())),
                                  dtype=torch.uint8, device=dev)
                      for t in cs.raw]
        cs.shared_outs = share_output
        if share_output:
            biggest = max(t.numel() for t in cs.raw)
            pool = {dt: torch.empty(biggest, dtype=dt, device=dev) for dt in {t.dtype for t in cs.raw}}
            cs.outs = [pool[t.dtype][:t.numel()] for t in cs.raw]
        else:
            cs.outs = [torch.empty(t.numel(), dtype=t.dtype, device=dev) for t in cs.raw]
        cs.sizes = torch.zeros(len(cs.raw), dtype=torch.int64, device=dev)
        cs.status = torch.zeros(1, dtype=torch.int32, device=dev)
        return cs

    @property
    def raw_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.raw)

    def spread(self, n_streams: int, call, count: Optional[int] = None) -> None:
        """Runs call(i) for i < count (default: for every tensor). With n_streams > 1 tensor i is enqueued on side stream i % n_streams:
        the tensors are independent, so the start of one launch may overlap the end of another. The side
        streams start after everything enqueued so far on the current stream, and the current stream
        continues after all of them (events; no host synchronisation)."""
        if n_streams > 1 and self.shared_outs:
            raise ValueError("outputs that share one buffer cannot be written from several streams")
        count = len(self.raw) if count is None else count
        if n_streams <= 1:
            for i in range(count):
                call(i)
            return
        main = torch.cuda.current_stream()
        while len(self.side) < n_streams:
            self.side.append(torch.cuda.Stream(device=self.raw[0].device))
        side = self.side[:n_streams]
        start = torch.cuda.Event()
        start.record(main)
        for s in side:
            s.wait_event(start)
        for i in range(count):
            with torch.cuda.stream(side[i % n_streams]):
                call(i)
        for s in side:
            done = torch.cuda.Event()
            done.record(s)
            main.wait_event(done)

    def compress_all(self, params=None, n_streams: int = 1, ranked: bool = False, blockwise: bool = False) -> None:
        """One enec_compress per tensor (no host synchronisation), on the current stream or spread over
        n_streams side streams. ranked: the frequency-rank variant (enec_compress_ranked) instead; blockwise: the
        variant with parameters per block (enec_compress_blockwise)."""
        self.spread(n_streams, lambda i: self._compress_one(i, params, ranked, blockwise))

    def _compress_one(self, i: int, params, ranked: bool = False, blockwise: bool = False) -> None:
        t = self.raw[i]
        dt = _DT[t.dtype]
        if blockwise:
            st = enec.enec_compress_blockwise(t, dt, t.numel(), self.streams[i], self.streams[i].numel(),
                                              self.sizes[i:i + 1], self.status)
        elif ranked:
            st = enec.enec_compress_ranked(t, dt, t.numel(), self.streams[i], self.streams[i].numel(),
                                           self.sizes[i:i + 1], self.status)
        elif params is None:
            st = enec.enec_compress(t, dt, t.numel(), self.streams[i], self.streams[i].numel(),
                                    self.sizes[i:i + 1], self.status)
        else:
            st = enec.enec_compress_with_params(t, dt, t.numel(), *params, self.streams[i],
                                                self.streams[i].numel(), self.sizes[i:i + 1], self.status)
        if st != 0:
            raise enec.EnecError(st, f"enec_compress tensor {i}")

    def decompress_all(self, n_streams: int = 1, ranked: bool = False, blockwise: bool = False) -> None:
        """One enec_decompress per tensor, on the current stream or spread over n_streams side streams. The
        stream length passed is the buffer's capacity; the true length is in the stream header and is checked
        against it on the device."""
        self.spread(n_streams, lambda i: self._decompress_one(i, ranked, blockwise))

    def _decompress_one(self, i: int, ranked: bool = False, blockwise: bool = False) -> None:
        t = self.raw[i]
        fn = enec.enec_decompress_blockwise if blockwise else enec.enec_decompress_ranked if ranked else enec.enec_decompress
        st = fn(self.streams[i], self.streams[i].numel(), _DT[t.dtype], t.numel(),
                                  self.outs[i], self.status)
        if st != 0:
            raise enec.EnecError(st, f"enec_decompress tensor {i}")

    def _dtype_groups(self):
        groups = {}
        for i, t in enumerate(self.raw):
            groups.setdefault(t.dtype, []).append(i)
        return groups

    def _batches(self):
        """Per dtype of the set: the item arrays of the two batched calls, built once (the buffers do not move)."""
        if self.batches is None:
            self.batches = []
            for dtype, idx in self._dtype_groups().items():
                whole = len(idx) == len(self.raw)
                comp = enec.make_batch([(self.raw[i], self.streams[i], self.raw[i].numel(), self.streams[i].numel()) for i in idx])
                dec = enec.make_batch([(self.streams[i], self.outs[i], self.raw[i].numel(), self.streams[i].numel()) for i in idx])
                sizes = self.sizes if whole else torch.zeros(len(idx), dtype=torch.int64, device=self.sizes.device)
                where = None if whole else torch.tensor(idx, device=self.sizes.device)
                self.batches.append((_DT[dtype], comp, dec, sizes, where))
        return self.batches

    def compress_batched(self) -> None:
        """One enec_compress_batched call per dtype of the set (two launches each) on the current stream."""
        for dt, comp, _, sizes, where in self._batches():
            st = enec.enec_compress_batched(comp, dt, sizes, self.status)
            if st != 0:
                raise enec.EnecError(st, "enec_compress_batched")
            if where is not None:
                self.sizes[where] = sizes

    def decompress_batched(self) -> None:
        """One enec_decompress_batched call (one launch) per dtype of the set on the current stream. The stream
        length passed is the buffer's capacity, as in decompress_all."""
        for dt, _, dec, _, _ in self._batches():
            st = enec.enec_decompress_batched(dec, dt, self.status)
            if st != 0:
                raise enec.EnecError(st, "enec_decompress_batched")

    def check_status(self) -> None:
        code = int(self.status.item())
        if code != 0:
            raise enec.EnecError(code, "device status")

    def compressed_bytes(self) -> int:
        return int(self.sizes.sum().item())

    def verify_roundtrip(self) -> None:
        """Outputs must equal the raw tensors bit for bit (needs unshared outputs)."""
        for i, t in enumerate(self.raw):
            bits = torch.int32 if t.element_size() == 4 else torch.int16
            if not torch.equal(self.outs[i].view(bits), t.reshape(-1).view(bits)):
                raise AssertionError(f"tensor {i}: decompressed bits differ from the input")
