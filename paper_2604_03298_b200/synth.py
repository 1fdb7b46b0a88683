"""Seeded synthetic weight tensors shaped like the paper's LLM workloads (Table 3 models stand-ins).

This module only draws random tensors; it holds none of the codec's arithmetic, so the CUDA path's
tests/benchmarks and the CPU oracle can both take their inputs from it.

Five workload families (``config_specs(cfg)``):
  1  one bf16 1024x4096 tensor, N(0, 0.02^2)
  2  one Llama-3-8B-shaped decoder layer in bf16 (q/o/k/v/gate/up/down + two RMSNorm vectors)
  3  32 such layers + embedding + LM head + final norm (about 16 GB)
  4  heavy-tailed stress set: 64 fp16 + 64 bf16 4096x4096 tensors (Laplace / Student-t, outliers, zeros)
  5  many-small-tensor MoE set: 768 expert matrices + 4096 vectors of 2048
  6  OLMo-1B-shaped fp32 set (Table 3's fp32 family): 16 layers of hidden 2048 / MLP 8192, embedding and
     LM head of 50304 rows, about 5.1 GB
  7  one decoder layer of family 6 (seven fp32 matrices, 268 MB)
``scale`` divides the large matrix dimensions so CPU tests can use the same recipes at small sizes.
"""
from dataclasses import dataclass
import math

import torch


@dataclass(frozen=True)
class TensorSpec:
    name: str
    dtype: torch.dtype
    shape: tuple
    dist: str          # "normal" | "laplace" | "student3"
    mean: float
    std: float
    seed: int
    outliers: bool = False   # 1 % of positions at +-50 std and 0.5 % exact +0.0

    @property
    def numel(self) -> int:
        return math.prod(self.shape)


def _d(v: int, scale: int) -> int:
    return max(16, v // scale)


def _llama_layer(layer: int, seed0: int, scale: int):
    H, KV, F = _d(4096, scale), _d(1024, scale), _d(14336, scale)
    shapes = [("q", (H, H)), ("k", (KV, H)), ("v", (KV, H)), ("o", (H, H)),
              ("gate", (F, H)), ("up", (F, H)), ("down", (H, F))]
    specs = []
    for i, (nm, shp) in enumerate(shapes):
        specs.append(TensorSpec(f"l{layer}.{nm}", torch.bfloat16, shp, "normal", 0.0,
                                1.0 / math.sqrt(shp[1]), seed0 + i))
    for j, nm in enumerate(("input_norm", "post_norm")):
        specs.append(TensorSpec(f"l{layer}.{nm}", torch.bfloat16, (H,), "normal", 1.0, 0.05, seed0 + 7 + j))
    return specs


def config_specs(cfg: int, scale: int = 1):
    """List of TensorSpec for workload family ``cfg`` (1..7)."""
    if cfg == 1:
        return [TensorSpec("w", torch.bfloat16, (_d(1024, scale), _d(4096, scale)), "normal", 0.0, 0.02, 0)]
    if cfg == 2:
        return _llama_layer(0, 2000, scale)
    if cfg == 3:
        specs = [TensorSpec("embed", torch.bfloat16, (_d(128256, scale), _d(4096, scale)), "normal", 0.0, 0.02, 3000)]
        for layer in range(32):
            specs += _llama_layer(layer, 3010 + 10 * layer, scale)
        specs.append(TensorSpec("final_norm", torch.bfloat16, (_d(4096, scale),), "normal", 1.0, 0.05, 3400))
        specs.append(TensorSpec("lm_head", torch.bfloat16, (_d(128256, scale), _d(4096, scale)), "normal", 0.0, 0.02, 3401))
        return specs
    if cfg == 4:
        specs = []
        side = _d(4096, scale)
        for di, dt in enumerate((torch.float16, torch.bfloat16)):
            for i in range(64):
                std = 0.01 * 10.0 ** ((i % 32) / 31.0)
                dist = "laplace" if i < 32 else "student3"
                specs.append(TensorSpec(f"{'fp16' if di == 0 else 'bf16'}.{i}", dt, (side, side), dist, 0.0, std,
                                        4000 + 64 * di + i, outliers=True))
        return specs
    if cfg == 5:
        specs = []
        I, H = _d(1408, scale), _d(2048, scale)
        idx = 0
        for layer in range(32):
            for e in range(8):
                for nm, shp in (("gate", (I, H)), ("up", (I, H)), ("down", (H, I))):
                    specs.append(TensorSpec(f"l{layer}.e{e}.{nm}", torch.bfloat16, shp, "normal", 0.0, 0.02, 5000 + idx))
                    idx += 1
        for v in range(4096):
            specs.append(TensorSpec(f"vec{v}", torch.bfloat16, (H,), "normal", 0.0, 0.02, 5000 + idx))
            idx += 1
        return specs
    if cfg in (6, 7):
        H, F, V = _d(2048, scale), _d(8192, scale), _d(50304, scale)
        specs = [TensorSpec("embed", torch.float32, (V, H), "normal", 0.0, 0.02, 6000)] if cfg == 6 else []
        for layer in range(16 if cfg == 6 else 1):
            shapes = [("q", (H, H)), ("k", (H, H)), ("v", (H, H)), ("o", (H, H)),
                      ("gate", (F, H)), ("up", (F, H)), ("down", (H, F))]
            for i, (nm, shp) in enumerate(shapes):
                specs.append(TensorSpec(f"l{layer}.{nm}", torch.float32, shp, "normal", 0.0, 1.0 / math.sqrt(shp[1]),
                                        6010 + 10 * layer + i))
        if cfg == 6:
            specs.append(TensorSpec("final_norm", torch.float32, (H,), "normal", 1.0, 0.05, 6400))
            specs.append(TensorSpec("lm_head", torch.float32, (V, H), "normal", 0.0, 0.02, 6401))
        return specs
    raise ValueError(f"unknown config {cfg}")


def make_tensor(spec: TensorSpec, device="cpu", keep_zeros: bool = False) -> torch.Tensor:
    """Draws the tensor in fp32 on ``device`` and rounds it to the spec's dtype (nearest even; fp32 stays as drawn).
    keep_zeros: leave the normal generator's rare exact zeros in (see below)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(spec.seed)
    n = spec.numel
    if spec.dist == "normal":
        t = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
        # A float32 normal generator emits exact 0.0 about once per 2^24 draws; a Gaussian has no atom at
        # zero, and one such value would set the lowest occupied exponent to 0 for the whole tensor.
        if not keep_zeros:
            t = torch.where(t == 0, torch.full_like(t, 2.0 ** -10), t)
        t = t * spec.std + spec.mean
    elif spec.dist == "laplace":
        u = torch.rand(n, generator=gen, device=device, dtype=torch.float32) - 0.5
        scale = spec.std / math.sqrt(2.0)
        t = -scale * torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.5 - 1e-7))
    elif spec.dist == "student3":
        z = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
        chi = torch.randn(3, n, generator=gen, device=device, dtype=torch.float32).pow(2).sum(0)
        t = z / torch.sqrt(chi / 3.0) * (spec.std / math.sqrt(3.0))
        del z, chi
    else:
        raise ValueError(spec.dist)
    if spec.outliers:
        r = torch.rand(n, generator=gen, device=device, dtype=torch.float32)
        sign = torch.where(torch.rand(n, generator=gen, device=device) < 0.5, -1.0, 1.0)
        t = torch.where(r < 0.01, sign * (50.0 * spec.std), t)
        t = torch.where((r >= 0.01) & (r < 0.015), torch.zeros_like(t), t)
        del r, sign
    return t.to(spec.dtype).reshape(spec.shape)


def as_words(t: torch.Tensor) -> torch.Tensor:
    """Raw 16-bit patterns of a bf16/fp16 tensor as a flat int16 view (same storage)."""
    return t.reshape(-1).view(torch.int16)
