"""GPU check of the SVD initialisation (Alg. 1 lines 4-5) against the oracle's LAPACK SVD of the same quantization
error.  The GPU runs a randomized subspace iteration in fp32, so the comparison is in the quantities that are
unique: singular values, the subspace spanned by the rows of A^ (principal angles), and the energy that subspace
captures; individual rows are compared up to sign only where the singular values are well separated."""
import numpy as np
import pytest
import torch

from helpers import f32, u8
from paper_2510_24061_b200 import synth
from test_oracle_svd_init import planted_backbone

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def fq():
    from paper_2510_24061_b200 import binding
    return binding


@pytest.fixture(scope="module")
def orc():
    from oracle import falqon_oracle
    return falqon_oracle


def _omega(seed, n, l):
    return synth.normal_bf16(seed, 4242, (n, l), 1.0).float().contiguous()


def test_planted_low_rank_error(fq, orc):
    """The quantization error is a planted rank-6 matrix with singular values 1, 1/4, 1/16, ...: every factor that
    stands above the fp32 rounding noise of W must come out as the oracle's, row by row up to sign."""
    rng = np.random.default_rng(5)
    m, n, rank, r = 384, 512, 6, 6
    W, codes, s0, L = planted_backbone(rng, m, n, rank, gap=4.0)
    wq_o, s_w_o, A_o, _, sigma_o = orc.svd_init(W, r)
    Wd = torch.from_numpy(W).to(DEV)
    wq, s_w, _ = fq.quantize(Wd, fq.E4M3)
    assert np.array_equal(u8(wq), wq_o)
    A_g, sigma_g = fq.svd_init(Wd, wq, s_w, r, _omega(5, n, r + 16).to(DEV), power_iters=2)
    A_g, sigma_g = f32(A_g).astype(np.float64), f32(sigma_g).astype(np.float64)
    assert np.allclose(sigma_g[:4], sigma_o[:4], rtol=2e-3)
    for i in range(4):                                            # rows up to sign
        a, b = A_g[i], A_o[i]
        sign = 1.0 if a @ b > 0 else -1.0
        assert np.linalg.norm(sign * a - b) <= 2e-2 * np.linalg.norm(b), i
    q_g = np.linalg.qr(A_g[:4].T)[0]
    q_o = np.linalg.qr(A_o[:4].T)[0]
    assert np.linalg.svd(q_o.T @ q_g)[1].min() > 1 - 1e-4       # cosines of the principal angles


@pytest.mark.parametrize("m,n,r", [(1024, 768, 16), (4096, 4096, 64)])
def test_random_backbone_captures_the_optimal_energy(fq, orc, m, n, r):
    """A random-init backbone: the quantization error has a flat spectrum, no individual direction is defined, but
    the r-dimensional row space of A^ must capture nearly as much of it as the optimal one, A^ A^T must be
    diag(sigma) and the leading singular values must be close to LAPACK's."""
    W = synth.backbone(9, 0, m, n)
    Wf = f32(W)
    wq_o, s_w_o, A_o, _, sigma_o = orc.svd_init(Wf, r)
    E = Wf.astype(np.float64) - orc.decode_array(wq_o, orc.E4M3).reshape(m, n) / np.float64(s_w_o)
    Wd = W.to(DEV)
    wq, s_w, _ = fq.quantize(Wd, fq.E4M3)
    A_g, sigma_g = fq.svd_init(Wd, wq, s_w, r, _omega(9, n, r + 16).to(DEV), power_iters=3)
    A_g, sigma_g = f32(A_g).astype(np.float64), f32(sigma_g).astype(np.float64)
    q_g = np.linalg.qr(A_g.T)[0]                                  # orthonormal basis of the row space
    captured = np.linalg.norm(E @ q_g) ** 2
    optimal = float((sigma_o[:r] ** 2).sum())
    assert captured >= 0.85 * optimal, captured / optimal
    gram = A_g @ A_g.T
    assert np.allclose(np.diag(gram), sigma_g, rtol=1e-3)
    assert np.abs(gram - np.diag(np.diag(gram))).max() <= 2e-3 * sigma_g.max()
    assert np.all(sigma_g <= sigma_o[:r] * (1 + 1e-3)) and sigma_g[0] >= 0.9 * sigma_o[0]
    # and the layer that results runs
    layer = fq.setup_layer_svd(Wd, r, _omega(9, n, r + 16).to(DEV), power_iters=3)
    X = synth.activations(9, 0, 64, n, 4).to(DEV)
    Y, OA, _, _ = fq.melded_forward(layer, X, y_dtype=torch.float32)
    assert bool(torch.isfinite(Y).all()) and float(OA.abs().max()) > 0
    assert fq.last_device_status() == 0
