"""Pins of the oracle's "update A" variant (the paper's appendix ablation with a trainable A: dL/dA = B^T dL/dO x^T).

What fixes it, other than itself: exact rational arithmetic for the fma step; the library matmul on library-decoded
codes for the code product; exactly representable cases in which every cast is exact, so that the FP8 pipeline must
reproduce the textbook gradient B^T G X and the textbook SGD step in integers; the full-precision gradient within the
FP8 error bound on random data; and the invariants of the step (A~ = Q(gamma A; s_W), nothing else in the backbone
touched, lr = 0 re-creates the A~ rows from the master copy).
"""
from fractions import Fraction

import numpy as np
import torch

from oracle import falqon_oracle as orc


def _round_f32(v: Fraction) -> np.float32:
    """Round-to-nearest-even of an exact rational to fp32 (normal range), without going through a double."""
    if v == 0:
        return np.float32(0.0)
    sign = -1 if v < 0 else 1
    a = abs(v)
    e = 0
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    assert -126 <= e <= 127
    scaled = a * (1 << 23)                      # in [2^23, 2^24)
    q = scaled.numerator // scaled.denominator
    rem = scaled - q
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and q % 2 == 1):
        q += 1
    return np.float32(sign * float(q) * 2.0 ** (e - 23))


def test_sgd_step_is_one_correctly_rounded_fma():
    rng = np.random.default_rng(5)
    p = (rng.standard_normal(400) * 10.0 ** rng.integers(-3, 3, 400)).astype(np.float32)
    g = (rng.standard_normal(400) * 10.0 ** rng.integers(-3, 3, 400)).astype(np.float32)
    # cases where a separately rounded product would differ from the fused one
    p[:3] = [1.0, 2.0 ** 24, -1.0]
    g[:3] = [1.0 + 2.0 ** -23, 3.0, 1.0 - 2.0 ** -24]
    lr = np.float32(0.3)
    got = p.copy()
    orc.sgd_step(got, g, lr)
    for i in range(p.size):
        exact = Fraction(p[i].item()) - Fraction(lr.item()) * Fraction(g[i].item())
        assert got[i] == _round_f32(exact), i
    unfused = (p - lr * g).astype(np.float32)
    assert np.any(unfused != got)               # the pin can tell a two-rounding step from the fma


def test_codes_gemm_against_library_matmul_and_integers():
    rng = np.random.default_rng(6)
    a = rng.integers(0, 256, size=(13, 40), dtype=np.uint8)
    b = rng.integers(0, 256, size=(7, 40), dtype=np.uint8)
    a[(a & 0x7F) == 0x7F] = 0x10                 # no E4M3 NaN codes
    b[(b & 0x7C) == 0x7C] = 0x20                 # no E5M2 inf / NaN codes
    sa, sb = np.float32(3.0), np.float32(0.5)
    got = orc.codes_gemm(a, orc.E4M3, sa, b, orc.E5M2, sb)
    da = torch.from_numpy(a).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    db = torch.from_numpy(b).view(torch.float8_e5m2).to(torch.float64).numpy()
    want = da @ db.T / 1.5
    assert np.allclose(got, want, rtol=1e-13, atol=0)
    # small integers are exact codes: the product is an integer matrix, transposition mistakes show at once
    ia = rng.integers(-8, 9, size=(5, 6))
    ib = rng.integers(-8, 9, size=(4, 6))
    ca = orc.encode_array(ia.astype(np.float32), orc.E4M3).reshape(ia.shape)
    cb = orc.encode_array(ib.astype(np.float32), orc.E4M3).reshape(ib.shape)
    assert np.array_equal(orc.codes_gemm(ca, orc.E4M3, 1.0, cb, orc.E4M3, 1.0), (ia @ ib.T).astype(np.float64))


def _exact_case():
    """Operands for which every cast of the step is exact: every tensor's absmax is 7 x 2^e or 3.5 x 2^e (so every scale is
    a power of two) and every value has at most three (E5M2) or four (E4M3) significant bits -- also the values of the
    intermediate P = G B, by construction: only rows 0, 1, 2 of B are non-zero."""
    m, n, r, T = 6, 8, 2, 5
    G = np.array([[2, 1, 0, 0, 0, 0], [1, -1, 2, 0, 1, 0], [-1, 2, -2, 1, 0, 0], [0, 0, 1, -1, 0, 7], [1, 1, 1, 0, -2, 0]], dtype=np.float64)
    X = np.array([[((3 * t + 5 * c) % 9) - 4 for c in range(n)] for t in range(T)], dtype=np.float64)
    X[0, 0] = 7.0
    B = np.zeros((m, r))
    B[0, 0], B[2, 0], B[1, 1] = 1.75, 0.5, 1.0
    return m, n, r, T, G, X, B


def test_exact_case_reproduces_textbook_gradient_and_step():
    m, n, r, T, G, X, B = _exact_case()
    gq, s_g, _ = orc.quantize(G.astype(np.float32), orc.E5M2)
    xq, s_x, _ = orc.quantize(X.astype(np.float32), orc.E4M3)
    assert s_g == 8192.0 and s_x == 64.0
    assert np.array_equal(orc.decode_array(gq, orc.E5M2).reshape(T, m) / s_g, G)          # the casts are exact here
    assert np.array_equal(orc.decode_array(xq, orc.E4M3).reshape(T, n) / s_x, X)
    P_true = G @ B                                # [T, r]; column 0 = 3.5, 2.75, -2.75, 0.5, 2.25
    assert np.abs(P_true).max() == 3.5
    A = (np.arange(r * n).reshape(r, n) % 5 - 2).astype(np.float32)
    wq = np.zeros((m + r, n), np.uint8)
    s_w = np.float32(4.0)
    A_master = A.copy()
    lr = np.float32(2.0 ** -6)
    out = orc.update_a(gq, s_g, xq, s_x, B.astype(np.float32), A_master, wq, s_w, 1.0, lr, m, r)
    dA_true = B.T @ G.T @ X                       # the paper's formula, [r, n]
    assert out["s_B"] == 256.0 and out["s_P"] == 128.0
    assert np.array_equal(out["P"].astype(np.float64), P_true)
    assert np.array_equal(orc.decode_array(out["Pq"], orc.E4M3).reshape(T, r) / 128.0, P_true)
    assert np.array_equal(out["dA"].astype(np.float64), dA_true)
    assert np.array_equal(A_master.astype(np.float64), A - float(lr) * dA_true)          # exact: small dyadic numbers
    want_rows, _, _ = orc.quantize(A_master, orc.E4M3, scale_in=s_w)
    assert np.array_equal(wq[m:], want_rows) and not wq[:m].any()
    assert np.count_nonzero(dA_true) > r * n // 2           # not a degenerate case


def test_random_case_within_fp8_bound_and_invariants():
    rng = np.random.default_rng(8)
    m, n, r, T = 48, 64, 8, 40
    G = (rng.standard_normal((T, m)) * 1e-2).astype(np.float32)
    X = rng.standard_normal((T, n)).astype(np.float32)
    B = (rng.standard_normal((m, r)) * 1e-1).astype(np.float32)
    A = (rng.uniform(-1, 1, (r, n)) / 32).astype(np.float32)
    gq, s_g, _ = orc.quantize(G, orc.E5M2)
    xq, s_x, _ = orc.quantize(X, orc.E4M3)
    s_w = np.float32(4000.0)
    wq = rng.integers(0, 0x70, size=(m + r, n), dtype=np.uint8)
    before = wq.copy()
    A_master = A.copy()
    out = orc.update_a(gq, s_g, xq, s_x, B, A_master, wq, s_w, 2.0, np.float32(0.05), m, r)
    dA_true = B.astype(np.float64).T @ G.astype(np.float64).T @ X.astype(np.float64)
    rel = np.linalg.norm(out["dA"] - dA_true) / np.linalg.norm(dA_true)
    assert rel < 0.08, rel                        # three FP8 casts (E5M2 2^-3, E4M3 2^-4 per element) averaged over the sums
    assert np.array_equal(wq[:m], before[:m])     # only the A~ rows change
    rows, _, _ = orc.quantize(A_master, orc.E4M3, scale_in=s_w, premul=2.0)
    assert np.array_equal(wq[m:], rows)
    # a transposed or sign-flipped gradient would not pass: the step moves A against the true gradient
    assert np.sum((A_master - A).astype(np.float64) * dA_true) < 0
    # lr = 0: the master copy is unchanged and the rows are re-created from it
    A2 = A_master.copy()
    wq2 = wq.copy()
    wq2[m:] = 0
    orc.update_a(gq, s_g, xq, s_x, B, A2, wq2, s_w, 2.0, np.float32(0.0), m, r)
    assert np.array_equal(A2, A_master) and np.array_equal(wq2, wq)
