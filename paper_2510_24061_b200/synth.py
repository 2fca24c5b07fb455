"""Seeded synthetic inputs for the melded FP8-LoRA layer.

This module holds no arithmetic of the method itself: it only draws the
tensors a layer is fed (activations X, backbone W, adapter A and B, output
gradient dY) with the shapes and value distributions of LLaMA-shaped linear
layers.  Both the CPU oracle's tests and the CUDA path's tests/bench call it,
so the two sides see identical arrays by construction.

The generator is counter based and uses only integer arithmetic plus exactly
rounded IEEE operations, so it gives the same bits on the CPU and on a GPU:

  key      = mix64(seed * 0x9E3779B97F4A7C15 + tensor_id)
  word(i,d)= mix64(key + (3*i + d + 1) * 0x9E3779B97F4A7C15)       d = 0,1,2
  uniform  = top 24 bits of word(i,0) * 2**-24                      in [0,1)
  normal   = (sum of the twelve 16-bit fields of word(i,0..2) - 393210) * 2**-16
             (Irwin-Hall, unit variance, clipped at +-6 sigma)

mix64 is the SplitMix64 finaliser.  Every value is scaled in fp32 and rounded
to bf16 (round to nearest even), the storage type of activations and weights.
"""
from __future__ import annotations

import torch

_GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK = (1 << 64) - 1

# tensor ids (add 16*matrix index and 256*step index)
TID_X, TID_W, TID_A, TID_B, TID_DY = 0, 1, 2, 3, 4


def _s64(v: int) -> int:
    """Python int (mod 2**64) -> the signed value torch.int64 stores."""
    v &= _MASK
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor holding uint64 bit patterns."""
    if s == 0:
        return x
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def _mix64_i(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * _M1) & _MASK
    z = ((z ^ (z >> 27)) * _M2) & _MASK
    return z ^ (z >> 31)


def tensor_key(seed: int, tensor_id: int) -> int:
    return _mix64_i(seed * _GOLD + tensor_id)


def _words(key: int, idx: torch.Tensor, draw: int) -> torch.Tensor:
    return _mix64_t((idx * 3 + (draw + 1)) * _s64(_GOLD) + _s64(key))


def _normal_chunk(key: int, idx: torch.Tensor) -> torch.Tensor:
    total = torch.zeros_like(idx)
    for d in range(3):
        w = _words(key, idx, d)
        for f in range(4):
            total += _lsr(w, 16 * f) & 0xFFFF
    return (total - 393210).to(torch.float32) * (2.0 ** -16)


def _uniform_chunk(key: int, idx: torch.Tensor) -> torch.Tensor:
    return _lsr(_words(key, idx, 0), 40).to(torch.float32) * (2.0 ** -24)


def _draw(kind: str, seed: int, tensor_id: int, numel: int, device, chunk: int = 1 << 24) -> torch.Tensor:
    key = tensor_key(seed, tensor_id)
    out = torch.empty(numel, dtype=torch.float32, device=device)
    for lo in range(0, numel, chunk):
        hi = min(numel, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        out[lo:hi] = _normal_chunk(key, idx) if kind == "normal" else _uniform_chunk(key, idx)
    return out


def normal_bf16(seed: int, tensor_id: int, shape, std: float, device="cpu") -> torch.Tensor:
    """bf16(N(0, std)) of the given shape (std is the standard deviation)."""
    numel = 1
    for s in shape:
        numel *= int(s)
    z = _draw("normal", seed, tensor_id, numel, device)
    return (z * torch.tensor(std, dtype=torch.float32, device=device)).to(torch.bfloat16).reshape(*shape)


def uniform_bf16(seed: int, tensor_id: int, shape, bound: float, device="cpu") -> torch.Tensor:
    """bf16(U(-bound, bound))."""
    numel = 1
    for s in shape:
        numel *= int(s)
    u = _draw("uniform", seed, tensor_id, numel, device)
    v = (u * 2.0 - 1.0) * torch.tensor(bound, dtype=torch.float32, device=device)
    return v.to(torch.bfloat16).reshape(*shape)


def student_t3_bf16(seed: int, tensor_id: int, shape, scale: float, device="cpu") -> torch.Tensor:
    """bf16(scale * t_3), t_3 = z0 / sqrt((z1^2+z2^2+z3^2)/3) from four normals."""
    numel = 1
    for s in shape:
        numel *= int(s)
    z = [_draw("normal", seed, tensor_id + 1024 * j, numel, device) for j in range(4)]
    den = torch.sqrt((z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0)
    den = torch.clamp(den, min=2.0 ** -16)
    v = (z[0] / den) * torch.tensor(scale, dtype=torch.float32, device=device)
    return v.to(torch.bfloat16).reshape(*shape)


def outlier_columns(n: int, count: int) -> list[int]:
    """Evenly spaced input channels that carry outliers: floor(j*n/count)."""
    return [(j * n) // count for j in range(count)]


def activations(seed: int, matrix: int, T: int, n: int, n_outliers: int, device="cpu") -> torch.Tensor:
    """X[T, n] = bf16(N(0,1)); `n_outliers` evenly spaced channels scaled x16 (exact in bf16)."""
    x = normal_bf16(seed, TID_X + 16 * matrix, (T, n), 1.0, device)
    if n_outliers > 0:
        cols = torch.tensor(outlier_columns(n, n_outliers), dtype=torch.int64, device=device)
        x[:, cols] = x[:, cols] * 16
    return x


def backbone(seed: int, matrix: int, m: int, n: int, device="cpu", heavy_tailed: bool = False) -> torch.Tensor:
    """W[m, n] = bf16(N(0, 0.02)), or bf16(0.02 * t_3) for the heavy-tailed variant."""
    if heavy_tailed:
        return student_t3_bf16(seed, TID_W + 16 * matrix, (m, n), 0.02, device)
    return normal_bf16(seed, TID_W + 16 * matrix, (m, n), 0.02, device)


def adapter_a(seed: int, matrix: int, r: int, n: int, device="cpu") -> torch.Tensor:
    """A[r, n] = bf16(U(-1/32, 1/32))."""
    return uniform_bf16(seed, TID_A + 16 * matrix, (r, n), 1.0 / 32.0, device)


def adapter_b(seed: int, matrix: int, m: int, r: int, device="cpu") -> torch.Tensor:
    """B[m, r] = bf16(N(0, 1e-3))."""
    return normal_bf16(seed, TID_B + 16 * matrix, (m, r), 1e-3, device)


def out_grad(seed: int, matrix: int, step: int, T: int, m: int, device="cpu") -> torch.Tensor:
    """dY[T, m] = bf16(N(0, 1e-2)), a fresh draw per step."""
    return normal_bf16(seed, TID_DY + 16 * matrix + 256 * step, (T, m), 1e-2, device)


# The workloads (one entry per linear layer: name, n = in features, m = out features).
LLAMA_7B_LINEARS = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                    ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096)]
LLAMA_13B_LINEARS = [("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
                     ("gate", 5120, 13824), ("up", 5120, 13824), ("down", 13824, 5120)]


def config0():
    """Single layer: in=out=1024, tokens 512, rank 16, alpha 32, 8 outlier channels, top-32 rows."""
    return dict(seed=0, m=1024, n=1024, T=512, r=16, alpha=32.0, n_outliers=8, k=32, steps=3, lr=2e-4)


def config1():
    """LLaMA-7B projection set of one decoder layer: tokens 4096, rank 64, 1% outlier channels, top-256."""
    return dict(seed=0, linears=LLAMA_7B_LINEARS, T=4096, r=64, alpha=64.0, k=256, steps=10, lr=2e-4,
                outlier_frac=0.01)


def config3():
    """LLaMA-13B projection set: hidden 5120, MLP 13824, tokens 8192, rank 64, top-512; heavy-tailed backbone rows
    (0.02 * Student-t with 3 degrees of freedom) with one scale per row."""
    return dict(seed=0, linears=LLAMA_13B_LINEARS, T=8192, r=64, alpha=64.0, k=512, steps=10, lr=2e-4,
                outlier_frac=0.01, per_row=True, heavy_tailed=True)

