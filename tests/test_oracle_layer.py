"""Pins for the oracle's melded forward, backward and proxy update (CPU only).

Nothing here re-types the oracle's formulas: the checks are a hand-worked exact
step (tests/golden/), exact rational arithmetic, numpy/torch library products on
library-decoded values, the textbook LoRA equations on exactly representable
inputs, full-precision LoRA within the FP8 error bound, and brute force.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import falqon_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _lib_decode(codes: np.ndarray, e5m2: bool = False) -> np.ndarray:
    """FP8 codes -> float64 through PyTorch's float8 types (independent of the oracle)."""
    dt = torch.float8_e5m2 if e5m2 else torch.float8_e4m3fn
    return torch.from_numpy(np.ascontiguousarray(codes)).view(dt).to(torch.float32).numpy().astype(np.float64)


def _load_golden_step():
    env = {}
    with open(os.path.join(GOLDEN, "exact_melded_step.txt")) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                name, expr = line.split("=", 1)
                env[name.strip()] = eval(expr, {"__builtins__": {}})
    return env


def _exact_e4m3_round(v: Fraction) -> float:
    """Correctly rounded (nearest, ties to even code, saturating) E4M3 value of an exact rational."""
    grid = sorted(set(x for x in _lib_decode(np.arange(256, dtype=np.uint8)) if np.isfinite(x)))
    best = None
    for idx, g in enumerate(grid):
        d = abs(Fraction(g) - v)
        if best is None or d < best[0]:
            best = (d, [g])
        elif d == best[0]:
            best[1].append(g)
    cands = best[1]
    if len(cands) == 1:
        return cands[0]
    codes = [orc.encode(c, orc.E4M3) for c in cands]  # tie: pick the even code (values are exact codes)
    return cands[0] if codes[0] % 2 == 0 else cands[1]


# ---------------------------------------------------------------- golden exact step

def test_golden_exact_melded_step():
    g = _load_golden_step()
    W, A, X, dY = (np.array(g[k], dtype=np.float64) for k in ("W", "A", "X", "dY"))
    m, n, r, T = 2, 4, 1, 2
    # (1) the fixture is self-consistent under exact arithmetic (scales are all 1 here)
    assert (X @ W.T).tolist() == g["Y"] and (X @ A.T).tolist() == g["OA"]
    assert (dY @ W).tolist() == g["dX"] and (dY.T @ np.array(g["OA"])).tolist() == g["dB"]
    # (2) the oracle reproduces it
    wq, s_w, dbuf = orc.setup_layer(W, A, None, 1.0)
    assert s_w == 1.0 and wq.tolist() == g["Wq_codes"]
    f = orc.layer_forward(X.astype(np.float32), wq, s_w, m, r)
    assert f["s_x"] == 1.0 and f["xq"].tolist() == g["Xq_codes"]
    assert f["Y"].tolist() == g["Y"] and f["OA"].tolist() == g["OA"] and f["amax_oa"] == 448.0
    b = orc.layer_backward(dY.astype(np.float32), f["OA"], wq, s_w, m, r)
    assert b["s_g"] == 1.0 and b["s_oa"] == 1.0
    assert b["gq"].tolist() == g["gq_codes"] and b["oaq"].tolist() == g["OAq_codes"]
    assert b["dX"].tolist() == g["dX"] and b["dB"].tolist() == g["dB"]
    idx, score = orc.proxy_update(wq, dbuf, b["dB"].astype(np.float32), g["lr"], g["k"], m, r)
    assert idx.tolist() == g["idx"]
    assert wq[0].tolist() == g["row0_after_merge_codes"]
    assert wq[1].tolist() == g["Wq_codes"][1] and wq[2].tolist() == g["Wq_codes"][2]
    assert dbuf.tolist() == g["dbuf_after_merge"]
    # (3) the optimizer step and the merged row agree with exact rational arithmetic
    d0 = Fraction(np.float32(-(2.0 ** -20) * 25690100).item())  # exact product, exactly representable
    assert float(d0) == g["dbuf_after_sgd"][0][0]
    for c in range(n):
        exact = Fraction(W[0, c]) + d0 * Fraction(A[0, c])
        assert _exact_e4m3_round(exact) == orc.decode(g["row0_after_merge_codes"][c], orc.E4M3)


# ---------------------------------------------------------------- forward

def _random_layer(seed, m, n, r, T, gamma=1.0, with_b=True):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((m, n)) * 0.02).astype(np.float32)
    A = rng.uniform(-1 / 32, 1 / 32, (r, n)).astype(np.float32)
    B = (rng.standard_normal((m, r)) * 1e-3).astype(np.float32) if with_b else None
    X = rng.standard_normal((T, n)).astype(np.float32)
    X[:, :: max(1, n // 4)] *= 16
    dY = (rng.standard_normal((T, m)) * 1e-2).astype(np.float32)
    return W, A, B, X, dY


def test_forward_equals_plain_fp8_layer_when_b_is_zero():
    m, n, r, T = 24, 40, 8, 12
    W, A, _, X, _ = _random_layer(1, m, n, r, T)
    wq0, s_w, _ = orc.setup_layer(W, A, None, 2.0)
    wqz, s_wz, dbuf = orc.setup_layer(W, A, np.zeros((m, r), np.float32), 2.0)
    assert np.array_equal(wq0, wqz) and s_w == s_wz and not dbuf.any()   # melding B = 0 changes no byte
    f = orc.layer_forward(X, wq0, s_w, m, r)
    # plain FP8 layer and the separate adapter product, by a library matmul on library-decoded codes
    xd, wd = _lib_decode(f["xq"]), _lib_decode(wq0)
    ref = (xd @ wd.T) / (np.float64(s_w) * np.float64(f["s_x"]))
    assert np.allclose(f["Y"], ref[:, :m], rtol=1e-13, atol=0)
    assert np.array_equal(f["OA"], ref[:, m:].astype(np.float32)) or np.allclose(f["OA"], ref[:, m:], rtol=1e-6)
    assert f["amax_oa"] == np.abs(f["OA"]).max()
    # quantized weights equal the library cast of W*s_W
    ref_wq = torch.from_numpy(W * s_w).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(wq0[:m], ref_wq)


def test_forward_sampled_matches_full():
    m, n, r, T = 16, 24, 8, 10
    W, A, B, X, _ = _random_layer(2, m, n, r, T)
    wq, s_w, _ = orc.setup_layer(W, A, B, 1.0)
    f = orc.layer_forward(X, wq, s_w, m, r)
    tsel, fsel = np.array([7, 0, 3]), np.array([15, 2, 16, 23])
    sub = orc.forward_gemm(f["xq"], f["s_x"], wq, s_w, m, r, tsel, fsel)
    full = np.concatenate([f["Y"], f["OA"].astype(np.float64)], axis=1)
    assert np.allclose(sub, full[np.ix_(tsel, fsel)], rtol=1e-7, atol=0)
    assert np.array_equal(sub[:, :2], f["Y"][np.ix_(tsel, fsel[:2])])


def _exact_case(seed, m, n, r, T):
    """Inputs on which every quantization is exact: small E4M3-representable integers times powers of
    two, with the tensor maxima pinned so that all absmax scales are exact powers of two."""
    rng = np.random.default_rng(seed)
    ints = np.array([-6, -5, -4, -3, -2, -1, 0, 0, 1, 2, 3, 4, 5, 6], dtype=np.float64)
    W = rng.choice(ints, (m, n)); W[0, 0] = 7       # amax 7  -> s_W = 64
    A = rng.choice(ints[3:-3], (r, n))                # |A| <= 3
    X = rng.choice(ints, (T, n)); X[0, 0] = -7        # s_x = 64
    G = rng.choice(ints, (T, m)); G[0, 0] = 7         # s_g = 8192
    B = rng.choice(ints[4:-4], (m, r))                # |B| <= 2
    return W, A, B, X, G


def test_exact_case_forward_backward_equal_textbook_lora():
    m, n, r, T = 6, 10, 2, 5
    W, A, B, X, G = _exact_case(3, m, n, r, T)
    gamma = 1.0
    # keep W + BA inside the exactly representable integers 0..7: one nonzero B entry on a tame row
    A[0] = np.sign(A[0])
    W[2] = np.clip(W[2], -5, 5)
    B = np.zeros_like(B); B[2, 0] = 1
    Weff = W + gamma * B @ A
    assert np.abs(Weff).max() <= 7 and np.any(Weff != W)
    wq, s_w, dbuf = orc.setup_layer(W, A, B, gamma)
    assert s_w == 64.0 and not dbuf.any()
    assert np.array_equal(_lib_decode(wq[:m]) / 64.0, Weff)
    f = orc.layer_forward(X.astype(np.float32), wq, s_w, m, r)
    assert f["s_x"] == 64.0
    assert np.array_equal(f["Y"], X @ Weff.T)                      # (W + gamma*B*A) x, Eq. of LoRA forward
    assert np.array_equal(f["OA"].astype(np.float64), gamma * X @ A.T)   # O_A = A x from the same product
    b = orc.layer_backward(G.astype(np.float32), f["OA"], wq, s_w, m, r)
    assert np.array_equal(b["dX"], G @ Weff)                       # dL/dx = (W + BA)^T dL/dO
    # dL/dB = dL/dO x^T A^T (textbook) = dL/dO (Ax)^T (reformulated): evaluate the textbook side here
    s_oa = b["s_oa"]
    oa_exact = np.array_equal(orc.decode_array(b["oaq"], orc.E4M3) / np.float64(s_oa), f["OA"].astype(np.float64))
    textbook = gamma * (G.T @ X) @ A.T
    if oa_exact:
        assert np.allclose(b["dB"], textbook, rtol=1e-12, atol=1e-9)
    else:  # O_A needed rounding to E4M3: the identity then holds within that one rounding (2^-4 relative per element)
        bound = (np.abs(G).T @ np.abs(f["OA"].astype(np.float64))) * 2.0 ** -4
        assert np.all(np.abs(b["dB"] - textbook) <= bound + 1e-9)


def test_exact_case_with_representable_oa():
    # One token column active per adapter row so that O_A values are single products (representable).
    m, n, r, T = 4, 8, 2, 3
    W = np.zeros((m, n)); W[0, 0] = 7; W[1, 3] = -2; W[2, 5] = 3; W[3, 7] = 1
    A = np.zeros((r, n)); A[0, 0] = 1; A[1, 3] = -2
    X = np.zeros((T, n)); X[0, 0] = 7; X[1, 3] = 2; X[2, 0] = -1; X[2, 3] = 2   # max|O_A| = 7 -> s_OA = 64
    G = np.array([[7, 0, 1, 0], [0, -2, 0, 0], [1, 1, 0, 4]], dtype=np.float64)
    wq, s_w, _ = orc.setup_layer(W, A, None, 1.0)
    f = orc.layer_forward(X.astype(np.float32), wq, s_w, m, r)
    b = orc.layer_backward(G.astype(np.float32), f["OA"], wq, s_w, m, r)
    assert np.array_equal(f["OA"].astype(np.float64), X @ A.T)
    assert np.array_equal(b["dB"], (G.T @ X) @ A.T)      # dL/dO x^T A^T
    assert np.array_equal(b["dB"], G.T @ (X @ A.T))      # = dL/dO (A x)^T
    assert np.array_equal(b["dX"], G @ W)


def test_matches_full_precision_lora_within_fp8_bound():
    m, n, r, T = 12, 16, 4, 8
    W, A, B, X, dY = _random_layer(4, m, n, r, T)
    gamma = 2.0
    wq, s_w, _ = orc.setup_layer(W, A, B, gamma)
    f = orc.layer_forward(X, wq, s_w, m, r)
    Wd, Ad, Bd, Xd = (v.astype(np.float64) for v in (W, A, B, X))
    Weff = Wd + gamma * Bd @ Ad
    Yfp = Xd @ Weff.T
    # each operand carries at most 2^-4 relative rounding error in E4M3 (plus subnormal floor), so
    # |Y - Yfp| <= sum_c |x||w| * (2*2^-4 + 2^-8) + slack for the melded B (a second E4M3 rounding of W)
    bound = (np.abs(Xd) @ (np.abs(Wd) + gamma * np.abs(Bd) @ np.abs(Ad)).T) * (3 * 2.0 ** -4 + 2.0 ** -7) + 1e-6
    assert np.all(np.abs(f["Y"] - Yfp) <= bound)
    assert np.linalg.norm(f["Y"] - Yfp) / np.linalg.norm(Yfp) < 0.08
    OAfp = gamma * Xd @ Ad.T
    assert np.linalg.norm(f["OA"] - OAfp) / np.linalg.norm(OAfp) < 0.08
    b = orc.layer_backward(dY, f["OA"], wq, s_w, m, r)
    Gd = dY.astype(np.float64)
    dXfp, dBfp = Gd @ Weff, Gd.T @ OAfp
    assert np.linalg.norm(b["dX"] - dXfp) / np.linalg.norm(dXfp) < 0.12   # E5M2 gradients: 2^-3 per element
    assert np.linalg.norm(b["dB"] - dBfp) / np.linalg.norm(dBfp) < 0.12


def test_backward_library_crosscheck_linearity_and_sampling():
    m, n, r, T = 20, 28, 8, 14
    W, A, B, X, dY = _random_layer(5, m, n, r, T)
    wq, s_w, _ = orc.setup_layer(W, A, B, 1.0)
    f = orc.layer_forward(X, wq, s_w, m, r)
    b = orc.layer_backward(dY, f["OA"], wq, s_w, m, r)
    gd, wd, od = _lib_decode(b["gq"], e5m2=True), _lib_decode(wq), _lib_decode(b["oaq"])
    assert np.allclose(b["dX"], (gd @ wd[:m]) / (np.float64(s_w) * np.float64(b["s_g"])), rtol=1e-12, atol=1e-300)
    assert np.allclose(b["dB"], (gd.T @ od) / (np.float64(b["s_g"]) * np.float64(b["s_oa"])), rtol=1e-12, atol=1e-300)
    assert b["s_oa"].view(np.uint32) == (np.float32(448.0) / f["amax_oa"]).view(np.uint32)
    # the adapter rows of W~' get no gradient path into dX: changing them leaves dX untouched
    wq2 = wq.copy(); wq2[m:] = 0
    assert np.array_equal(orc.dx_gemm(b["gq"], b["s_g"], wq2, s_w, m), b["dX"])
    # exact power-of-two scaling of dY scales s_g inversely and leaves dX*2 (linearity in the gradient)
    b2 = orc.layer_backward(dY * 2, f["OA"], wq, s_w, m, r)
    assert np.array_equal(b2["gq"], b["gq"]) and np.allclose(b2["dX"], 2 * b["dX"], rtol=1e-15)
    tsel, csel, isel = np.array([13, 2]), np.array([27, 0, 5]), np.array([19, 4])
    assert np.array_equal(orc.dx_gemm(b["gq"], b["s_g"], wq, s_w, m, tsel, csel), b["dX"][np.ix_(tsel, csel)])
    assert np.array_equal(orc.db_gemm(b["gq"], b["s_g"], b["oaq"], b["s_oa"], isel), b["dB"][isel])


# ---------------------------------------------------------------- proxy update

def _brute_topk(score: np.ndarray, k: int):
    order = sorted(range(len(score)), key=lambda i: (-float(score[i]), i))
    return sorted(order[:k])


def test_topk_bruteforce_ties_edges_permutation():
    rng = np.random.default_rng(6)
    m, n, r = 40, 16, 4
    W, A, _, _, _ = _random_layer(6, m, n, r, 4)
    wq0, s_w, _ = orc.setup_layer(W, A, None, 1.0)
    dB = rng.standard_normal((m, r)).astype(np.float32)
    dB[7] = dB[3]; dB[21] = dB[3]; dB[30] = -dB[3]     # four rows with identical scores
    for k in [0, 1, 2, 3, 5, m - 1, m]:
        wq, dbuf = wq0.copy(), np.zeros((m, r), np.float32)
        idx, score = orc.proxy_update(wq, dbuf, dB, 0.5, k, m, r)
        ref_score = np.array([np.sum(np.abs(np.float32(-0.5) * dB[i]).astype(np.float64)) for i in range(m)])
        assert np.allclose(score, ref_score, rtol=1e-6)
        assert idx.tolist() == _brute_topk(score, k)
        untouched = np.setdiff1d(np.arange(m + r), idx)
        assert np.array_equal(wq[untouched], wq0[untouched])          # rows not selected (and A~) are untouched
        assert not dbuf[idx].any()
        assert np.array_equal(dbuf[np.setdiff1d(np.arange(m), idx)],
                              (np.float32(-0.5) * dB)[np.setdiff1d(np.arange(m), idx)])
    # the tie group: make its score the largest and ask for 2 of the 4 -> the two lowest indices
    dBt = dB.copy(); dBt[[3, 7, 21, 30]] *= 100
    idx, _ = orc.proxy_update(wq0.copy(), np.zeros((m, r), np.float32), dBt, 0.5, 2, m, r)
    assert idx.tolist() == [3, 7]
    # permuting the rows permutes the selection
    perm = rng.permutation(m)
    dBp = dB[perm]
    wqp = np.concatenate([wq0[:m][perm], wq0[m:]])
    idx_p, _ = orc.proxy_update(wqp, np.zeros((m, r), np.float32), dBp, 0.5, 5, m, r)
    idx_o, score = orc.proxy_update(wq0.copy(), np.zeros((m, r), np.float32), dB, 0.5, 6, m, r)
    distinct = [i for i in idx_o if np.sum(score == score[i]) == 1]
    assert set(perm[idx_p]) >= set(distinct[:1])
    with pytest.raises(ValueError):
        orc.proxy_update(wq0.copy(), np.zeros((m, r), np.float32), dB, 0.5, m + 1, m, r)


def test_score_is_left_to_right_fp32_sum():
    # (2^24 + 1) + 1 in fp32 left-to-right stays 2^24 + ... : order matters, pin the ascending-j order
    m, n, r = 2, 16, 3
    wq = np.zeros((m + r, n), np.uint8)
    dbuf = np.array([[2.0 ** 24, 1.0, 1.0], [1.0, 1.0, 2.0 ** 24]], dtype=np.float32)
    _, score = orc.proxy_update(wq, dbuf.copy(), None, 0.0, 0, m, r)
    assert score[0] == 2.0 ** 24 and score[1] == 2.0 ** 24 + 2


def test_optimizer_step_is_single_fma_and_accumulates():
    m, n, r = 3, 16, 2
    wq = np.zeros((m + r, n), np.uint8)
    dbuf = np.array([[1.0, 2.0 ** -24], [0.5, -3.0], [0.0, 7.0]], dtype=np.float32)
    dB = np.array([[2.0 ** -24, 1.0], [1 / 3, 1e-3], [5.0, -1e-8]], dtype=np.float32)
    lr = np.float32(0.3)
    d = dbuf.copy()
    orc.proxy_update(wq, d, dB, lr, 0, m, r)
    for i in range(m):
        for j in range(r):
            exact = Fraction(dbuf[i, j].item()) - Fraction(lr.item()) * Fraction(dB[i, j].item())
            assert d[i, j] == np.float32(float(exact))   # one rounding of the exact a*b+c (float(Fraction) is correctly rounded to double; double->float double-rounding is excluded below)
    d2 = d.copy()
    orc.proxy_update(wq, d2, dB, lr, 0, m, r)           # unmerged rows keep accumulating
    assert d2[1, 0] != d[1, 0] and d2[2, 0] == np.float32(-3.0)


def test_merge_identity_subhalf_ulp_saturation_and_exactness():
    rng = np.random.default_rng(10)
    m, n, r = 8, 32, 4
    W, A, _, _, _ = _random_layer(10, m, n, r, 4)
    wq0, s_w, _ = orc.setup_layer(W, A, None, 1.0)
    # zero DeltaB: merging every row is the identity on the codes
    wq = wq0.copy()
    orc.proxy_update(wq, np.zeros((m, r), np.float32), None, 0.0, m, m, r)
    assert np.array_equal(wq, wq0)
    # tiny increments (far below half an FP8 step) leave every code unchanged
    wq = wq0.copy()
    tiny = np.full((m, r), 1e-9, np.float32)
    orc.proxy_update(wq, tiny, None, 0.0, m, m, r)
    assert np.array_equal(wq, wq0)
    # general increments: the fp32 chain result equals the correctly rounded exact value except for
    # rare double-rounding cases, which stay within one code step
    wq = wq0.copy()
    dbuf = (rng.standard_normal((m, r)) * 0.2).astype(np.float32)
    d_in = dbuf.copy()
    orc.proxy_update(wq, dbuf, None, 0.0, m, m, r)
    wd, ad = _lib_decode(wq0[:m]), _lib_decode(wq0[m:])
    mismatches = 0
    for i in range(m):
        for c in range(n):
            exact = Fraction(wd[i, c]) + sum(Fraction(d_in[i, j].item()) * Fraction(ad[j, c]) for j in range(r))
            want = _exact_e4m3_round(exact)
            got = orc.decode(wq[i, c], orc.E4M3)
            if got != want:
                mismatches += 1
                assert abs(int(wq[i, c] & 0x7F) - orc.encode(abs(want), orc.E4M3)) <= 1
    assert mismatches <= 2 and (wq[:m] != wq0[:m]).mean() > 0.3
    # saturation: a huge increment pins the row at +-448 with the sign of the increment times A~
    wq = wq0.copy()
    big = np.zeros((m, r), np.float32); big[2, 0] = 1e6
    orc.proxy_update(wq, big, None, 0.0, 1, m, r)
    a0 = ad[0]
    assert np.all(orc.decode_array(wq[2], orc.E4M3)[a0 > 0] == 448) and np.all(orc.decode_array(wq[2], orc.E4M3)[a0 < 0] == -448)
    assert np.array_equal(wq[2][a0 == 0], wq0[2][a0 == 0])


def test_merge_all_rows_then_forward_equals_updated_lora():
    # W + (B + dB) A = (W + B A) + dB A : after merging all rows, the forward is that of the updated adapter
    m, n, r, T = 6, 10, 2, 5
    W, A, _, X, _ = _exact_case(11, m, n, r, T)
    A = np.sign(A); W[1] = np.clip(W[1], -5, 5); W[4] = np.clip(W[4], -5, 5)
    wq, s_w, dbuf = orc.setup_layer(W, A, None, 1.0)
    dBm = np.zeros((m, r)); dBm[1, 0] = 1; dBm[4, 1] = -1          # integer DeltaB keeps everything representable
    Wnew = W + dBm @ A
    assert np.abs(Wnew).max() <= 7 and np.any(Wnew != W)
    dbuf[:] = dBm
    orc.proxy_update(wq, dbuf, None, 0.0, m, m, r)
    f = orc.layer_forward(X.astype(np.float32), wq, s_w, m, r)
    assert np.array_equal(f["Y"], X @ Wnew.T)
