"""Pins of the oracle's SVD initialisation (Alg. 1 lines 3-5) against facts that do not depend on it: the
Eckart-Young residual computed from an eigenvalue routine, a backbone whose quantization error is a planted
low-rank matrix, and the defining identities of the factors."""
import numpy as np

from oracle import falqon_oracle as orc


def planted_backbone(rng, m, n, rank, gap=8.0):
    """W whose E4M3 codes are known and whose quantization error is (almost exactly) a planted rank-`rank` matrix
    L with singular values gap^0, gap^-1, ...: W = dec(C) / s0 + L with every |L_ij| s0 < 0.45 of the smallest code
    spacing in use, so quantizing W gives back C; one anchor element pins the absmax (and hence the scale)."""
    s0 = np.float32(64.0)
    mags = rng.integers(0x58, 0x70, size=(m, n)).astype(np.uint8)          # |values| in [16, 224): spacing >= 2
    codes = mags | (rng.integers(0, 2, size=(m, n)).astype(np.uint8) << 7)
    codes[0, 0] = 0x7E                                                       # 448: the absmax anchor
    base = orc.decode_array(codes, orc.E4M3).reshape(m, n) / np.float64(s0)
    U, _ = np.linalg.qr(rng.standard_normal((m, rank)))
    V, _ = np.linalg.qr(rng.standard_normal((n, rank)))
    sv = gap ** -np.arange(rank, dtype=np.float64)
    L = (U * sv) @ V.T
    L *= 0.45 / (np.abs(L).max() * float(s0))                               # max |L| s0 = 0.45 < half the spacing (1.0)
    L[0, 0] = 0.0
    W = (base + L).astype(np.float32)
    return W, codes, s0, L


def test_planted_low_rank_error_is_recovered():
    rng = np.random.default_rng(0)
    m, n, rank = 96, 80, 4
    W, codes, s0, L = planted_backbone(rng, m, n, rank)
    wq, s_w, A_hat, B_hat, sigma = orc.svd_init(W, rank)
    assert np.array_equal(wq, codes) and s_w == s0
    # Delta W = L up to the fp32 rounding of W (1e-7 per element against entries of 7e-3) and the anchor element:
    # the rank-4 factors reproduce it
    assert np.linalg.norm(B_hat @ A_hat - L) <= 2e-3 * np.linalg.norm(L)
    # the row space of A^ is the row space of L
    Vt_L = np.linalg.svd(L)[2][:rank]
    q = np.linalg.qr(A_hat.T)[0]
    assert np.allclose(np.linalg.svd(Vt_L[:3] @ q)[1], 1.0, atol=1e-4)     # the three directions well above the rounding noise


def test_factors_are_the_truncated_svd_and_its_residual_is_eckart_young():
    rng = np.random.default_rng(1)
    m, n, r = 64, 48, 6
    W = (rng.standard_normal((m, n)) * 0.02).astype(np.float32)
    wq, s_w, A_hat, B_hat, sigma = orc.svd_init(W, r)
    E = W.astype(np.float64) - orc.decode_array(wq, orc.E4M3).reshape(m, n) / np.float64(s_w)
    # residual of the best rank-r approximation from the eigenvalues of E^T E (a different routine)
    ev = np.sort(np.linalg.eigvalsh(E.T @ E))[::-1]
    assert np.isclose(np.linalg.norm(E - B_hat @ A_hat) ** 2, ev[r:].sum(), rtol=1e-9)
    assert np.allclose(sigma[:r] ** 2, ev[:r], rtol=1e-9)
    # even split: A^ A^T = B^T B^ = diag(sigma_r); B^ = E A^T diag(1/sigma)
    assert np.allclose(A_hat @ A_hat.T, np.diag(sigma[:r]), atol=1e-12)
    assert np.allclose(B_hat.T @ B_hat, np.diag(sigma[:r]), atol=1e-12)
    assert np.allclose(E @ A_hat.T / sigma[:r], B_hat, atol=1e-12)
    # Eq. q_error: dec(W~)/s + Delta W = W exactly in fp64
    assert np.array_equal(orc.decode_array(wq, orc.E4M3).reshape(m, n) / np.float64(s_w) + E, W.astype(np.float64))
