"""ctypes/numpy front end of the CPU oracle (oracle/falqon_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the
benchmark's CPU-baseline leg; the product path never touches it.  Argument
marshalling only -- every arithmetic step is in the C++ file.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

E4M3, E5M2 = 0, 1
BF16, F32 = 0, 1
PER_TENSOR, PER_ROW = 0, 1
FP8_MAX = {E4M3: 448.0, E5M2: 57344.0}

_lib = C.CDLL(_build.build())

_i64, _f32, _i32 = C.c_int64, C.c_float, C.c_int
_p = C.c_void_p

_lib.orc_fp8_decode.restype = C.c_double
_lib.orc_fp8_decode.argtypes = [C.c_uint8, _i32]
_lib.orc_fp8_encode.restype = C.c_uint8
_lib.orc_fp8_encode.argtypes = [_f32, _i32]
_lib.orc_fp8_encode_array.restype = None
_lib.orc_fp8_encode_array.argtypes = [_p, _i64, _i32, _p]
_lib.orc_fp8_decode_array.restype = None
_lib.orc_fp8_decode_array.argtypes = [_p, _i64, _i32, _p]
_lib.orc_f32_to_bf16.restype = C.c_uint16
_lib.orc_f32_to_bf16.argtypes = [_f32]
_lib.orc_quantize.restype = _i32
_lib.orc_quantize.argtypes = [_p, _i32, _i64, _i64, _i32, _i32, _p, _f32, _p, _p, _p]
_lib.orc_forward_gemm.restype = _i32
_lib.orc_forward_gemm.argtypes = [_p, _f32, _p, _p, _i32, _i64, _i64, _i64, _i64, _p, _i64, _p, _i64, _p]
_lib.orc_forward.restype = _i32
_lib.orc_forward.argtypes = [_p, _f32, _p, _p, _i32, _i64, _i64, _i64, _i64, _p, _p, _p]
_lib.orc_dx_gemm.restype = _i32
_lib.orc_dx_gemm.argtypes = [_p, _f32, _p, _p, _i32, _i64, _i64, _i64, _p, _i64, _p, _i64, _p]
_lib.orc_db_gemm.restype = _i32
_lib.orc_db_gemm.argtypes = [_p, _f32, _p, _f32, _p, _i64, _i64, _i64, _p, _i64, _p]
_lib.orc_proxy_update.restype = _i32
_lib.orc_proxy_update.argtypes = [_p, _p, _p, _f32, _p, _i64, _i64, _i64, _i64, _p, _p]
_lib.orc_proxy_update_exact.restype = _i32
_lib.orc_proxy_update_exact.argtypes = [_p, _p, _p, _f32, _p, _i64, _i64, _i64, _i64, _p, _p]
_lib.orc_exact_merge_element.restype = C.c_uint8
_lib.orc_exact_merge_element.argtypes = [C.c_uint8, _p, _p, _i64]
_lib.orc_quantize_colscaled.restype = _i32
_lib.orc_quantize_colscaled.argtypes = [_p, _i32, _i64, _i64, _i32, _p, _p, _p, _p]
_lib.orc_adamw_step.restype = _i32
_lib.orc_adamw_step.argtypes = [_p, _p, _p, _p, _i64, _f32, _f32, _f32, _f32, _f32, _i64]
_lib.orc_codes_gemm.restype = _i32
_lib.orc_codes_gemm.argtypes = [_p, _i32, _f32, _p, _i32, _f32, _i64, _i64, _i64, _p]
_lib.orc_sgd_step.restype = _i32
_lib.orc_sgd_step.argtypes = [_p, _p, _f32, _i64]
_lib.orc_num_threads.restype = _i32


def _ptr(a):
    return None if a is None else a.ctypes.data_as(_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _sw(s_w):
    """Scale argument -> (float32 array, granularity): a scalar is per tensor, an array of m+1 is per row."""
    a = _c(np.atleast_1d(s_w), np.float32)
    return a, (PER_ROW if a.size > 1 else PER_TENSOR)


def _sel(s):
    if s is None:
        return None, 0
    s = _c(s, np.int64)
    return s, s.size


def num_threads() -> int:
    return int(_lib.orc_num_threads())


def decode(code: int, fmt: int) -> float:
    return float(_lib.orc_fp8_decode(int(code), fmt))


def encode(value: float, fmt: int) -> int:
    return int(_lib.orc_fp8_encode(float(np.float32(value)), fmt))


def encode_array(values, fmt: int) -> np.ndarray:
    v = _c(values, np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    _lib.orc_fp8_encode_array(_ptr(v), v.size, fmt, _ptr(out))
    return out


def decode_array(codes, fmt: int) -> np.ndarray:
    c = _c(codes, np.uint8)
    out = np.empty(c.shape, dtype=np.float64)
    _lib.orc_fp8_decode_array(_ptr(c), c.size, fmt, _ptr(out))
    return out


def f32_to_bf16_bits(value: float) -> int:
    return int(_lib.orc_f32_to_bf16(float(np.float32(value))))


def bf16_bits(x) -> np.ndarray:
    """fp32 array whose values are bf16-representable -> uint16 bf16 bit patterns (exact)."""
    x = _c(x, np.float32)
    bits = x.view(np.uint32)
    assert not np.any(bits & 0xFFFF), "values are not bf16-representable"
    return (bits >> 16).astype(np.uint16)


def quantize(src, fmt: int, gran: int = PER_TENSOR, scale_in=None, premul: float = 1.0, src_is_bf16_bits=False):
    """Q_fp8.  src: 2-D fp32 array, or uint16 bf16 bit patterns.  Returns (codes, scale, amax)."""
    if src_is_bf16_bits:
        a, dt = _c(src, np.uint16), BF16
    else:
        a, dt = _c(src, np.float32), F32
    rows, cols = a.shape
    groups = rows if gran == PER_ROW else 1
    dst = np.empty((rows, cols), dtype=np.uint8)
    scale_out = np.empty(groups, dtype=np.float32)
    amax_out = np.empty(groups, dtype=np.float32)
    s_in = None if scale_in is None else _c(np.atleast_1d(scale_in), np.float32)
    rc = _lib.orc_quantize(_ptr(a), dt, rows, cols, fmt, gran, _ptr(s_in), float(np.float32(premul)),
                           _ptr(dst), _ptr(scale_out), _ptr(amax_out))
    assert rc == 0
    if gran == PER_TENSOR:
        return dst, np.float32(scale_out[0]), np.float32(amax_out[0])
    return dst, scale_out, amax_out


def quantize_colscaled(src, fmt: int, col_div):
    """Q_fp8 of a tensor whose column c is first multiplied by 1/col_div[c] (dY in the per-row mode)."""
    a = _c(src, np.float32)
    rows, cols = a.shape
    div = _c(col_div, np.float32)
    assert div.size >= cols
    dst = np.empty((rows, cols), dtype=np.uint8)
    scale_out = np.empty(1, dtype=np.float32)
    amax_out = np.empty(1, dtype=np.float32)
    rc = _lib.orc_quantize_colscaled(_ptr(a), F32, rows, cols, fmt, _ptr(div), _ptr(dst), _ptr(scale_out), _ptr(amax_out))
    assert rc == 0
    return dst, np.float32(scale_out[0]), np.float32(amax_out[0])


def forward_gemm(xq, s_x, wq, s_w, m: int, r: int, tsel=None, fsel=None) -> np.ndarray:
    """Sampled O_merged: tokens tsel x merged features fsel (None = all), float64."""
    xq, wq = _c(xq, np.uint8), _c(wq, np.uint8)
    T, n = xq.shape
    assert wq.shape == (m + r, n)
    ts, nt = _sel(tsel)
    fs, nf = _sel(fsel)
    out = np.empty((nt if ts is not None else T, nf if fs is not None else m + r), dtype=np.float64)
    sw, gran = _sw(s_w)
    assert gran == PER_TENSOR or sw.size == m + 1
    rc = _lib.orc_forward_gemm(_ptr(xq), float(s_x), _ptr(wq), _ptr(sw), gran, T, m, n, r,
                               _ptr(ts), nt, _ptr(fs), nf, _ptr(out))
    assert rc == 0
    return out


def forward(xq, s_x, wq, s_w, m: int, r: int):
    """Returns (Y float64 [T,m], OA float32 [T,r], amax_oa float32)."""
    xq, wq = _c(xq, np.uint8), _c(wq, np.uint8)
    T, n = xq.shape
    assert wq.shape == (m + r, n)
    Y = np.empty((T, m), dtype=np.float64)
    OA = np.empty((T, r), dtype=np.float32)
    amax = np.zeros(1, dtype=np.float32)
    sw, gran = _sw(s_w)
    assert gran == PER_TENSOR or sw.size == m + 1
    rc = _lib.orc_forward(_ptr(xq), float(s_x), _ptr(wq), _ptr(sw), gran, T, m, n, r, _ptr(Y), _ptr(OA), _ptr(amax))
    assert rc == 0
    return Y, OA, np.float32(amax[0])


def dx_gemm(gq, s_g, wq, s_w, m: int, tsel=None, csel=None) -> np.ndarray:
    gq, wq = _c(gq, np.uint8), _c(wq, np.uint8)
    T = gq.shape[0]
    n = wq.shape[1]
    assert gq.shape == (T, m) and wq.shape[0] >= m
    ts, nt = _sel(tsel)
    cs, nc = _sel(csel)
    out = np.empty((nt if ts is not None else T, nc if cs is not None else n), dtype=np.float64)
    sw, gran = _sw(s_w)
    rc = _lib.orc_dx_gemm(_ptr(gq), float(s_g), _ptr(wq), _ptr(sw), gran, T, m, n, _ptr(ts), nt, _ptr(cs), nc, _ptr(out))
    assert rc == 0
    return out


def db_gemm(gq, s_g, oaq, s_oa, isel=None, row_scale=None) -> np.ndarray:
    gq, oaq = _c(gq, np.uint8), _c(oaq, np.uint8)
    T, m = gq.shape
    r = oaq.shape[1]
    assert oaq.shape[0] == T
    is_, ni = _sel(isel)
    out = np.empty((ni if is_ is not None else m, r), dtype=np.float64)
    rs = None if row_scale is None else _c(row_scale, np.float32)
    rc = _lib.orc_db_gemm(_ptr(gq), float(s_g), _ptr(oaq), float(s_oa), _ptr(rs), T, m, r, _ptr(is_), ni, _ptr(out))
    assert rc == 0
    return out


def proxy_update(wq, dbuf, dB, lr: float, k: int, m: int, r: int, row_scales=None):
    """In place on wq (uint8 [(m+r), n]) and dbuf (float32 [m, r]).  Returns (idx int32 [k], score float32 [m])."""
    assert wq.dtype == np.uint8 and wq.flags.c_contiguous and wq.shape[0] == m + r
    assert dbuf.dtype == np.float32 and dbuf.flags.c_contiguous and dbuf.shape == (m, r)
    n = wq.shape[1]
    g = None if dB is None else _c(dB, np.float32)
    idx = np.empty(max(k, 0), dtype=np.int32)
    score = np.empty(m, dtype=np.float32)
    rs = None if row_scales is None else _c(row_scales, np.float32)
    assert rs is None or rs.size == m + 1
    rc = _lib.orc_proxy_update(_ptr(wq), _ptr(dbuf), _ptr(g), float(np.float32(lr)), _ptr(rs), m, n, r, k, _ptr(idx),
                               _ptr(score))
    if rc != 0:
        raise ValueError("orc_proxy_update rejected its arguments")
    return idx, score


def proxy_update_exact(wq, dbuf, dB, lr: float, k: int, m: int, r: int, row_scales=None):
    """proxy_update with the correctly rounded merge (exact sum, one rounding to E4M3)."""
    assert wq.dtype == np.uint8 and wq.flags.c_contiguous and wq.shape[0] == m + r
    assert dbuf.dtype == np.float32 and dbuf.flags.c_contiguous and dbuf.shape == (m, r)
    n = wq.shape[1]
    g = None if dB is None else _c(dB, np.float32)
    idx = np.empty(max(k, 0), dtype=np.int32)
    score = np.empty(m, dtype=np.float32)
    rs = None if row_scales is None else _c(row_scales, np.float32)
    assert rs is None or rs.size == m + 1
    rc = _lib.orc_proxy_update_exact(_ptr(wq), _ptr(dbuf), _ptr(g), float(np.float32(lr)), _ptr(rs), m, n, r, k, _ptr(idx),
                                     _ptr(score))
    if rc != 0:
        raise ValueError("orc_proxy_update_exact rejected its arguments")
    return idx, score


def exact_merge_element(w: int, d, a) -> int:
    """Code of sat_rne_e4m3(dec(w) + sum_j d[j] * dec(a[j])) with the sum exact (d float32, a uint8 codes)."""
    d = _c(d, np.float32)
    a = _c(a, np.uint8)
    assert d.size == a.size
    return int(_lib.orc_exact_merge_element(int(w), _ptr(d), _ptr(a), d.size))


def adamw_step(p, g, exp_avg, exp_avg_sq, lr, beta1, beta2, eps, weight_decay, step: int):
    """AdamW on the DeltaBuffer, in place on p, exp_avg, exp_avg_sq (float32, contiguous)."""
    for a in (p, exp_avg, exp_avg_sq):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    g = _c(g, np.float32)
    rc = _lib.orc_adamw_step(_ptr(p), _ptr(g), _ptr(exp_avg), _ptr(exp_avg_sq), p.size, float(np.float32(lr)),
                             float(np.float32(beta1)), float(np.float32(beta2)), float(np.float32(eps)),
                             float(np.float32(weight_decay)), int(step))
    if rc != 0:
        raise ValueError("orc_adamw_step rejected its arguments")


# ---- whole-layer compositions in the paper's order (each step is one oracle call) ----

def setup_layer(W, A, B, gamma: float, per_row: bool = False):
    """Alg. 1 without the SVD (A and B are given): W~, s_W = Q(W); A~ = Q(gamma*A; s_W);
    W~' = [W~; A~]; the initial B is melded by the merge operator itself over all rows
    (W + BA = W~ + B A~ in the scaled domain), leaving DeltaBuffer = 0.
    per_row: every row of W gets its own absmax scale and the A~ block one absmax scale of its own;
    s_w is then an array of m + 1 scales."""
    W = _c(W, np.float32)
    A = _c(A, np.float32)
    m, n = W.shape
    r = A.shape[0]
    if per_row:
        wq_w, s_rows, _ = quantize(W, E4M3, gran=PER_ROW)
        aq, s_a, _ = quantize(A, E4M3, premul=gamma)
        s_w = np.concatenate([s_rows, [s_a]]).astype(np.float32)
    else:
        wq_w, s_w, _ = quantize(W, E4M3)
        aq, _, _ = quantize(A, E4M3, scale_in=s_w, premul=gamma)
    wq = np.ascontiguousarray(np.concatenate([wq_w, aq], axis=0))
    dbuf = np.zeros((m, r), dtype=np.float32)
    if B is not None:
        dbuf[:] = _c(B, np.float32)
        proxy_update(wq, dbuf, None, 0.0, m, m, r, row_scales=s_w if per_row else None)
    return wq, s_w, dbuf


def svd_init(W, r: int):
    """Alg. 1 lines 3-5 (Eq. q_error, Eq. reform): W~, s_W = Q(W); Delta W = W - W~ / s_W; (B^, A^) = the rank-r
    truncated SVD of Delta W, the singular values split evenly: B^ = U_r sqrt(S_r), A^ = sqrt(S_r) V_r^T (the paper
    does not say how they are split; only A^ enters the melded layer, and only up to the sign of each row).
    fp64 throughout, numpy's LAPACK SVD as the library step.  Returns (wq [m, n] codes, s_W, A^ [r, n], B^ [m, r],
    sigma [min(m, n)] all singular values)."""
    W = _c(W, np.float32)
    wq, s_w, _ = quantize(W, E4M3)
    E = W.astype(np.float64) - decode_array(wq, E4M3).reshape(W.shape) / np.float64(s_w)
    U, S, Vt = np.linalg.svd(E, full_matrices=False)
    root = np.sqrt(S[:r])
    return wq, s_w, root[:, None] * Vt[:r], U[:, :r] * root[None, :], S


def layer_forward(X, wq, s_w, m: int, r: int):
    """Alg. 2 lines 5-9 for one layer.  Returns dict(xq, s_x, Y, OA, amax_oa)."""
    xq, s_x, _ = quantize(X, E4M3)
    Y, OA, amax_oa = forward(xq, s_x, wq, s_w, m, r)
    return dict(xq=xq, s_x=s_x, Y=Y, OA=OA, amax_oa=amax_oa)


def layer_backward(dY, OA, wq, s_w, m: int, r: int):
    """Alg. 3 line 3 plus the implied input gradient.  Returns dict(gq, s_g, oaq, s_oa, dX, dB)."""
    per_row = np.atleast_1d(s_w).size > 1
    if per_row:
        gq, s_g, _ = quantize_colscaled(dY, E5M2, np.asarray(s_w)[:m])
    else:
        gq, s_g, _ = quantize(dY, E5M2)
    oaq, s_oa, _ = quantize(OA, E4M3)
    dX = dx_gemm(gq, s_g, wq, s_w, m)
    dB = db_gemm(gq, s_g, oaq, s_oa, row_scale=np.asarray(s_w)[:m] if per_row else None)
    return dict(gq=gq, s_g=s_g, oaq=oaq, s_oa=s_oa, dX=dX, dB=dB)


# ---- the "update A" variant (the paper's ablation with a trainable A) ----

def codes_gemm(a, fmt_a: int, s_a, b, fmt_b: int, s_b) -> np.ndarray:
    """out[i, j] = sum_k dec(a[i, k]) dec(b[j, k]) / (s_a s_b) in float64; a uint8 [M, K], b uint8 [N, K]."""
    a, b = _c(a, np.uint8), _c(b, np.uint8)
    M, K = a.shape
    N = b.shape[0]
    assert b.shape[1] == K
    out = np.empty((M, N), dtype=np.float64)
    rc = _lib.orc_codes_gemm(_ptr(a), fmt_a, float(np.float32(s_a)), _ptr(b), fmt_b, float(np.float32(s_b)), M, N, K, _ptr(out))
    assert rc == 0
    return out


def sgd_step(p, g, lr: float):
    """In place: p = fma(-lr, g, p) element by element (float32)."""
    assert p.dtype == np.float32 and p.flags.c_contiguous
    g = _c(g, np.float32)
    assert g.size == p.size
    assert _lib.orc_sgd_step(_ptr(p), _ptr(g), float(np.float32(lr)), p.size) == 0


def update_a(gq, s_g, xq, s_x, B, A_master, wq, s_w, gamma: float, lr: float, m: int, r: int):
    """One step of a trainable A (the paper's appendix ablation: dL/dA = B^T dL/dO x^T), in the same FP8 scheme as the
    rest of the layer.  gq [T, m] E5M2 codes of dY with scale s_g and xq [T, n] E4M3 codes of X with scale s_x are the
    operands the backward and the forward already cast.  Steps, in this order:
      B~, s_B = Q_e4m3(B)                       (per tensor; B fp32 [m, r] is the caller's record of the adapter's B)
      P = g~ B~ / (s_g s_B)                     ([T, r]: dY B, contraction over the m outputs), rounded to fp32
      P~, s_P = Q_e4m3(P)                       (per tensor)
      dA = P~^T x~ / (s_P s_x)                  ([r, n], contraction over the tokens), rounded to fp32
      A_master = fma(-lr, dA, A_master)         (fp32 master copy of A, [r, n], in place)
      A~ = Q_e4m3(gamma * A_master; s_W)        (written over rows m.. of wq; Eq. A_integ)
    Rows of W~ merged earlier keep the products with the A~ of their time.  Returns a dict of the intermediates."""
    B = _c(B, np.float32)
    Bq, s_B, _ = quantize(B, E4M3)
    P = codes_gemm(gq, E5M2, s_g, np.ascontiguousarray(Bq.T), E4M3, s_B).astype(np.float32)
    Pq, s_P, amax_P = quantize(P, E4M3)
    dA = codes_gemm(np.ascontiguousarray(Pq.T), E4M3, s_P, np.ascontiguousarray(_c(xq, np.uint8).T), E4M3, s_x).astype(np.float32)
    sgd_step(A_master, dA, lr)
    Aq, _, _ = quantize(A_master, E4M3, scale_in=s_w, premul=gamma)
    wq[m:m + r] = Aq
    return dict(Bq=Bq, s_B=s_B, P=P, Pq=Pq, s_P=s_P, amax_P=amax_P, dA=dA)
