"""Seeded synthetic KV caches shaped like the long-context workloads LagKV is run on.

This module holds input generation only -- none of the method's arithmetic -- so that
the CUDA library's tests, the benchmark and the CPU oracle's tests can all draw the
same bytes from it.  Everything is bf16; ``to_bits`` gives the uint16 view the oracle
takes.

Recipe (one call = one layer's cache ``[B, H, S, D]``):
  K: standard normal, times a per-(head, channel) scale exp(N(0, sigma_k)) shared by
     all tokens and sequences (channel outliers), then rotary position embedding at
     positions 0..S-1 with base ``rope_theta`` pairing channel c with c + D/2;
  V: standard normal times a per-(sequence, head, token) scale exp(N(0, sigma_v)).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    """Shape and LagKV parameters of one benchmark configuration."""
    name: str
    layers: int
    B: int
    H: int
    D: int
    S: int          # sequence length Ls
    sink: int
    lag: int
    ratio: float
    sigma_k: float = 1.0
    sigma_v: float = 0.5
    seed_base: int = 0

    def seed(self, layer: int) -> int:
        return self.seed_base + layer


# The single-pass (prefill) configurations; the append and sweep configurations are
# built from these fields by the tests and the benchmark.
WORKLOADS = {
    "tiny": Workload("tiny", 1, 1, 8, 128, 4096, 16, 128, 0.25, seed_base=0),
    "llama8b_32k": Workload("llama8b_32k", 32, 1, 8, 128, 32768, 16, 1024, 0.25, seed_base=1000),
    "llama8b_128k": Workload("llama8b_128k", 32, 1, 8, 128, 131072, 16, 2048, 0.125,
                             sigma_k=1.5, seed_base=2000),
    "decode_append": Workload("decode_append", 28, 16, 4, 128, 16384, 16, 512, 0.25, seed_base=3000),
    "sweep": Workload("sweep", 1, 1, 8, 128, 65536, 4, 128, 0.25, seed_base=4000),
}


def make_kv(B: int, H: int, S: int, D: int, seed: int, sigma_k: float = 1.0, sigma_v: float = 0.5,
            rope_theta: float = 500000.0, device="cpu", pos_offset: int = 0, dtype=torch.bfloat16):
    """Return ``(K, V)`` tensors ``[B, H, S, D]`` of ``dtype`` (bf16, or fp16 for an fp16 cache) on
    ``device`` (see module docstring); the same fp32 draws are rounded to either format."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    half = D // 2
    k = torch.randn((B, H, S, D), generator=g, device=dev, dtype=torch.float32)
    k *= torch.exp(sigma_k * torch.randn((1, H, 1, D), generator=g, device=dev, dtype=torch.float32))
    if half > 0 and 2 * half == D:
        pos = torch.arange(pos_offset, pos_offset + S, device=dev, dtype=torch.float64)
        inv = rope_theta ** (-torch.arange(0, half, device=dev, dtype=torch.float64) * 2.0 / D)
        ang = pos[:, None] * inv[None, :]
        cos, sin = ang.cos().float(), ang.sin().float()
        a, b = k[..., :half].clone(), k[..., half:].clone()
        k[..., :half] = a * cos - b * sin
        k[..., half:] = b * cos + a * sin
        del a, b, cos, sin, ang
    K = _store(k, dtype)
    del k
    v = torch.randn((B, H, S, D), generator=g, device=dev, dtype=torch.float32)
    v *= torch.exp(sigma_v * torch.randn((B, H, S, 1), generator=g, device=dev, dtype=torch.float32))
    V = _store(v, dtype)
    return K, V


def _store(x: torch.Tensor, dtype) -> torch.Tensor:
    """Round fp32 draws to the cache's storage format.  fp8 (e4m3) holds at most 448: the draws are
    first divided by a per-tensor scale (largest magnitude -> 400), which is what a quantising
    engine does and what the compress pass never needs to know (it cancels in Eq. 9)."""
    if dtype == torch.float8_e4m3fn:
        return (x * (400.0 / float(x.abs().max()))).to(dtype)
    return x.to(dtype)


def make_workload_layer(w: Workload, layer: int, device="cpu", S: int | None = None):
    """K, V of one layer of a named workload."""
    return make_kv(w.B, w.H, w.S if S is None else S, w.D, w.seed(layer), w.sigma_k, w.sigma_v,
                   device=device)


def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 / fp16 tensor -> numpy uint16 array of the same shape, fp8 tensor -> uint8 array (bit
    patterns, on the host)."""
    if t.dtype == torch.float8_e4m3fn:
        return t.detach().contiguous().view(torch.uint8).cpu().numpy()
    assert t.dtype in (torch.bfloat16, torch.float16)
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def bits_to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bits(x) -> np.ndarray:
    """Round float values to bf16 (nearest even, via torch) and return the bit patterns."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return to_bits(t)
