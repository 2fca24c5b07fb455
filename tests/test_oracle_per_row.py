"""Pins for the oracle's per-row-scaled backbone mode (an extension beyond the paper's per-tensor scheme:
every row of W has its own absmax scale, the A~ block one scale of its own).

Pins: (1) when all scales coincide and are powers of two the mode must reproduce the per-tensor path bit
for bit; (2) exactly representable inputs with different row scales must give the textbook LoRA results
exactly; (3) library products on library-decoded codes; (4) the mode's purpose: smaller error on
heavy-tailed rows.
"""
import numpy as np
import torch

from oracle import falqon_oracle as orc


def _lib_decode(codes, e5m2=False):
    dt = torch.float8_e5m2 if e5m2 else torch.float8_e4m3fn
    return torch.from_numpy(np.ascontiguousarray(codes)).view(dt).to(torch.float32).numpy().astype(np.float64)


def test_equal_power_of_two_scales_reduce_to_per_tensor_path():
    rng = np.random.default_rng(0)
    m, n, r, T, k = 12, 24, 4, 9, 5
    top = np.float32(7.0 / 256.0)                       # every row's absmax -> scale 448/top = 16384
    W = np.clip((rng.standard_normal((m, n)) * 0.01).astype(np.float32), -top, top)
    W[:, 0] = top * np.where(rng.random(m) < 0.5, -1, 1)
    A = np.clip(rng.uniform(-0.02, 0.02, (r, n)).astype(np.float32), -top, top)
    A[0, 1] = top
    B = (rng.standard_normal((m, r)) * 1e-2).astype(np.float32)
    X = rng.standard_normal((T, n)).astype(np.float32)
    dY = (rng.standard_normal((T, m)) * 1e-2).astype(np.float32)
    wq_t, s_t, _ = orc.setup_layer(W, A, B, 1.0)
    wq_r, s_r, _ = orc.setup_layer(W, A, B, 1.0, per_row=True)
    assert s_t == 16384.0 and np.all(s_r == 16384.0) and s_r.size == m + 1
    assert np.array_equal(wq_t, wq_r)
    ft, fr = orc.layer_forward(X, wq_t, s_t, m, r), orc.layer_forward(X, wq_r, s_r, m, r)
    assert np.array_equal(ft["Y"], fr["Y"]) and np.array_equal(ft["OA"], fr["OA"])
    bt, br = orc.layer_backward(dY, ft["OA"], wq_t, s_t, m, r), orc.layer_backward(dY, fr["OA"], wq_r, s_r, m, r)
    assert np.array_equal(bt["gq"], br["gq"]) and br["s_g"] == bt["s_g"] * 16384.0
    assert np.array_equal(bt["dX"], br["dX"]) and np.array_equal(bt["dB"], br["dB"])
    db_t, db_r = np.zeros((m, r), np.float32), np.zeros((m, r), np.float32)
    it, _ = orc.proxy_update(wq_t, db_t, bt["dB"].astype(np.float32), 0.5, k, m, r)
    ir, _ = orc.proxy_update(wq_r, db_r, br["dB"].astype(np.float32), 0.5, k, m, r, row_scales=s_r)
    assert np.array_equal(it, ir) and np.array_equal(wq_t, wq_r) and np.array_equal(db_t, db_r)


def test_exact_case_with_different_row_scales():
    m, n, r, T = 4, 8, 2, 3
    Wint = np.zeros((m, n)); Wint[0, 0] = 7; Wint[0, 2] = -3; Wint[1, 3] = -7; Wint[1, 1] = 2
    Wint[2, 5] = 7; Wint[2, 6] = 1; Wint[3, 7] = -7; Wint[3, 4] = 5
    row_pow = np.array([0, 3, -2, 1])                   # row i holds integers times 2^row_pow[i]
    W = Wint * np.exp2(row_pow)[:, None]
    A = np.zeros((r, n)); A[0, 0] = 7; A[1, 3] = -2     # one active input per adapter row: O_A stays representable
    X = np.zeros((T, n)); X[0, 0] = 1; X[1, 3] = 2; X[2, 0] = -1; X[2, 3] = 2; X[0, 5] = 7
    # column 1 has the smallest row scale (8): its entry 7 makes max|dY / s_w| = 7/8, so s_g = 65536 exactly
    G = np.array([[3, 0, 1, 0], [0, -7, 0, 0], [1, 1, 0, 4]], dtype=np.float64)
    wq, s_w, dbuf = orc.setup_layer(W, A, None, 1.0, per_row=True)
    assert np.array_equal(s_w, np.concatenate([64.0 * np.exp2(-row_pow), [64.0]]).astype(np.float32))
    assert np.array_equal(_lib_decode(wq[:m]) / s_w[:m, None], W)
    f = orc.layer_forward(X.astype(np.float32), wq, s_w, m, r)
    assert np.array_equal(f["Y"], X @ W.T) and np.array_equal(f["OA"].astype(np.float64), X @ A.T)
    b = orc.layer_backward(G.astype(np.float32), f["OA"], wq, s_w, m, r)
    assert np.array_equal(b["dX"], G @ W)                # (W)^T dL/dO with the row scales divided out and back
    assert np.array_equal(b["dB"], G.T @ (X @ A.T))      # dL/dO (A x)^T
    # merge all rows with an integer DeltaB (scaled like its row so everything stays representable)
    dBm = np.zeros((m, r)); dBm[0, 1] = 1; dBm[1, 0] = -8 / 7; dBm[1, 0] = 0; dBm[2, 1] = 0.25
    Wnew = W + dBm @ A
    dbuf[:] = dBm
    orc.proxy_update(wq, dbuf, None, 0.0, m, m, r, row_scales=s_w)
    assert not dbuf.any()
    assert np.array_equal(_lib_decode(wq[:m]) / s_w[:m, None], Wnew) and np.any(Wnew != W)
    f2 = orc.layer_forward(X.astype(np.float32), wq, s_w, m, r)
    assert np.array_equal(f2["Y"], X @ Wnew.T)


def test_library_crosscheck_random_per_row():
    rng = np.random.default_rng(3)
    m, n, r, T = 20, 32, 8, 11
    W = (rng.standard_t(3, (m, n)) * 0.02).astype(np.float32)
    A = rng.uniform(-1 / 32, 1 / 32, (r, n)).astype(np.float32)
    B = (rng.standard_normal((m, r)) * 1e-3).astype(np.float32)
    X = rng.standard_normal((T, n)).astype(np.float32)
    dY = (rng.standard_normal((T, m)) * 1e-2).astype(np.float32)
    wq, s_w, _ = orc.setup_layer(W, A, B, 2.0, per_row=True)
    for i in range(m):                                   # row scales are the per-row absmax scales, to the bit
        assert s_w[i].view(np.uint32) == (np.float32(448.0) / np.abs(W[i]).max()).view(np.uint32)
    assert s_w[m].view(np.uint32) == (np.float32(448.0) / np.abs(np.float32(2.0) * A).max()).view(np.uint32)
    f = orc.layer_forward(X, wq, s_w, m, r)
    xd, wd = _lib_decode(f["xq"]), _lib_decode(wq)
    col = np.concatenate([s_w[:m], np.full(r, s_w[m])]).astype(np.float64)
    ref = (xd @ wd.T) / (col[None, :] * np.float64(f["s_x"]))
    assert np.allclose(f["Y"], ref[:, :m], rtol=1e-13, atol=0) and np.allclose(f["OA"], ref[:, m:], rtol=1e-6)
    b = orc.layer_backward(dY, f["OA"], wq, s_w, m, r)
    inv = (np.float32(1.0) / s_w[:m]).astype(np.float32)
    scaled = dY * inv[None, :]
    s_g = np.float32(57344.0) / np.abs(scaled).max()
    assert b["s_g"].view(np.uint32) == s_g.view(np.uint32)
    ref_gq = torch.from_numpy(scaled * s_g).clamp(-57344, 57344).to(torch.float8_e5m2).view(torch.uint8).numpy()
    assert np.array_equal(b["gq"], ref_gq)
    gd, od = _lib_decode(b["gq"], e5m2=True), _lib_decode(b["oaq"])
    assert np.allclose(b["dX"], (gd @ wd[:m]) / np.float64(b["s_g"]), rtol=1e-12, atol=1e-300)
    ref_db = (gd.T @ od) / (np.float64(b["s_g"]) * np.float64(b["s_oa"])) * s_w[:m, None].astype(np.float64)
    assert np.allclose(b["dB"], ref_db, rtol=1e-12, atol=1e-300)
    # against full-precision LoRA: FP8-sized error only
    Weff = W.astype(np.float64) + 2.0 * B.astype(np.float64) @ A.astype(np.float64)
    assert np.linalg.norm(f["Y"] - X @ Weff.T) / np.linalg.norm(X @ Weff.T) < 0.08
    assert np.linalg.norm(b["dX"] - dY.astype(np.float64) @ Weff) / np.linalg.norm(dY.astype(np.float64) @ Weff) < 0.12


def test_per_row_scaling_helps_heavy_tailed_rows():
    rng = np.random.default_rng(5)
    m, n = 64, 256
    W = (rng.standard_t(3, (m, n)) * 0.02).astype(np.float32)
    W[7, 3] = 3.0e4                                      # one huge outlier pushes every other row into E4M3 subnormals
    qt, st, _ = orc.quantize(W, orc.E4M3)
    qr, sr, _ = orc.quantize(W, orc.E4M3, gran=orc.PER_ROW)
    err_t = np.linalg.norm(orc.decode_array(qt, orc.E4M3) / st - W)
    err_r = np.linalg.norm(orc.decode_array(qr, orc.E4M3) / sr[:, None] - W)
    assert err_r < 0.5 * err_t
