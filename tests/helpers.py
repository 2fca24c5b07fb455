"""Shared helpers of the parity tests: seeded layer inputs and comparison metrics."""
from __future__ import annotations

import numpy as np
import torch

from paper_2510_24061_b200 import synth


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def u8(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").numpy()


def bits32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def rel_fro(got, want) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.linalg.norm(want)
    return float(np.linalg.norm(got - want) / den) if den > 0 else float(np.linalg.norm(got))


def layer_inputs(seed: int, matrix: int, m: int, n: int, r: int, T: int, n_outliers: int, device="cpu",
                 with_b: bool = True):
    """W, A, B, X for one linear layer (bf16 tensors on `device`)."""
    W = synth.backbone(seed, matrix, m, n, device)
    A = synth.adapter_a(seed, matrix, r, n, device)
    B = synth.adapter_b(seed, matrix, m, r, device) if with_b else None
    X = synth.activations(seed, matrix, T, n, n_outliers, device)
    return W, A, B, X


def max_abs_err_rel(got, want) -> float:
    """Largest element-wise error, relative to the largest magnitude of the expected tensor."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.max(np.abs(want)) if want.size else 0.0
    err = np.max(np.abs(got - want)) if want.size else 0.0
    return float(err / den) if den > 0 else float(err)


def product_close(got, want, tol: float = 2e-5) -> bool:
    """The tolerance of the tensor-core stages: relative Frobenius error <= tol, AND no single element further than
    tol x max|want| from its expected value -- a norm over millions of elements would hide one wrong entry; an fp32
    accumulation error is about 1e-7 of the row's magnitude, a wrong entry is of the order of the magnitude itself."""
    return rel_fro(got, want) <= tol and max_abs_err_rel(got, want) <= tol
