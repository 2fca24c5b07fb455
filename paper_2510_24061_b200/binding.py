"""ctypes binding of libfalqon.so: the same names as the C ABI in include/falqon.h.

Argument marshalling only.  PyTorch supplies device memory (torch.empty) and the
current CUDA stream; every step of the path runs in the library's kernels.  There
is no fallback: importing this module raises if the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfalqon.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
E4M3, E5M2 = 0, 1
BF16, F32 = 0, 1
PER_TENSOR, PER_ROW = 0, 1
LAYER_FUSED_CAST, LAYER_EMIT_XQ, LAYER_DB_OWN_KERNEL = 1, 2, 4
WS_XQ, WS_GQ, WS_OAQ_T, WS_SCALES, WS_SCORE = range(5)

EXPORTS = ["falqon_absmax", "falqon_selftest_wait_timeout", "falqon_workspace_bytes", "falqon_workspace_region", "falqon_quantize", "falqon_melded_forward",
           "falqon_melded_forward_codes", "falqon_melded_forward_amax", "falqon_melded_backward_amax",
           "falqon_melded_forward_dump", "falqon_melded_backward_dump", "falqon_melded_backward_dx", "falqon_melded_backward_codes",
           "falqon_exact_merge_prepare", "falqon_proxy_update_batched_exact",
           "falqon_update_a", "falqon_update_a_scratch_bytes", "falqon_update_a_region",
           "falqon_melded_backward_update", "falqon_proxy_update_scored", "falqon_proxy_update_scored_batched", "falqon_exact_merge_scratch_bytes", "falqon_proxy_update_exact",
           "falqon_svd_init_scratch_bytes", "falqon_svd_init", "falqon_tensor_ceiling", "falqon_tensor_ceiling_ctas",
           "falqon_melded_backward", "falqon_proxy_update", "falqon_proxy_update_batched", "falqon_proxy_update_batched_adamw", "falqon_last_device_status", "falqon_launch_count",
           "falqon_profile_start", "falqon_profile_stop", "falqon_proxy_update_static", "falqon_workspace_init", "falqon_proxy_update_adamw"]
STATIC_MAX_ROWS = 16384
STAGES = ["quant_x", "gemm_fwd", "quant_dy", "quant_oa", "gemm_dx", "gemm_db", "reduce_db", "sgd_score", "topk", "merge"]

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_24061_b200.build` "
                      "(there is no non-CUDA fallback)")
lib = C.CDLL(LIB_PATH)


class falqon_layer(C.Structure):
    _fields_ = [("m", C.c_int64), ("n", C.c_int64), ("r", C.c_int64),
                ("wq", C.c_void_p), ("s_w", C.c_void_p), ("dbuf", C.c_void_p),
                ("gran", C.c_int32), ("flags", C.c_int32)]


_i64, _sz, _p, _f, _i = C.c_int64, C.c_size_t, C.c_void_p, C.c_float, C.c_int
lib.falqon_workspace_bytes.restype = _sz
lib.falqon_workspace_bytes.argtypes = [_i64, _i64, _i64, _i64]
lib.falqon_workspace_region.restype = _i
lib.falqon_workspace_region.argtypes = [_i64, _i64, _i64, _i64, _i, C.POINTER(_sz), C.POINTER(_sz)]
lib.falqon_workspace_init.restype = _i
lib.falqon_workspace_init.argtypes = [_p, _sz, _p]
lib.falqon_quantize.restype = _i
lib.falqon_quantize.argtypes = [_p, _i, _i64, _i64, _i, _i, _p, _f, _p, _p, _p, _p, _sz, _p]
lib.falqon_melded_forward.restype = _i
lib.falqon_melded_forward.argtypes = [C.POINTER(falqon_layer), _p, _i, _i64, _p, _i, _p, _p, _p, _p, _sz, _p]
lib.falqon_melded_forward_amax.restype = _i
lib.falqon_melded_forward_amax.argtypes = [C.POINTER(falqon_layer), _p, _i, _p, _i64, _p, _i, _p, _p, _p, _p, _sz, _p]
lib.falqon_melded_backward_amax.restype = _i
lib.falqon_melded_backward_amax.argtypes = [C.POINTER(falqon_layer), _p, _i, _p, _i64, _p, _p, _p, _i, _p, _p, _p, _sz, _p]
lib.falqon_melded_forward_dump.restype = _i
lib.falqon_melded_forward_dump.argtypes = [C.POINTER(falqon_layer), _p, _i, _p, _i64, _p, _i, _p, _p, _p, C.c_int32, _p, _sz, _p]
lib.falqon_melded_backward_dump.restype = _i
lib.falqon_melded_backward_dump.argtypes = [C.POINTER(falqon_layer), _p, _i, _p, _i64, _p, _p, _p, _i, _p, _p, C.c_int32, _p, _sz, _p]
lib.falqon_exact_merge_prepare.restype = _i
lib.falqon_exact_merge_prepare.argtypes = [C.POINTER(falqon_layer), _p, _sz, _p]
lib.falqon_proxy_update_batched_exact.restype = _i
lib.falqon_proxy_update_batched_exact.argtypes = [C.POINTER(falqon_layer), C.c_int32, C.POINTER(_p), _f, C.POINTER(_i64), C.POINTER(_p),
                                                  C.POINTER(_p), C.POINTER(_sz), C.POINTER(_p), C.POINTER(_sz), C.c_int32, _p]
lib.falqon_update_a_scratch_bytes.restype = _sz
lib.falqon_update_a_scratch_bytes.argtypes = [_i64, _i64, _i64, _i64]
lib.falqon_update_a_region.restype = _i
lib.falqon_update_a_region.argtypes = [_i64, _i64, _i64, _i64, _i, C.POINTER(_sz), C.POINTER(_sz)]
lib.falqon_update_a.restype = _i
lib.falqon_update_a.argtypes = [C.POINTER(falqon_layer), _p, _p, _p, _p, _f, _f, _i64, _p, _sz, _p, _sz, _p]
lib.falqon_melded_backward_update.restype = _i
lib.falqon_melded_backward_update.argtypes = [C.POINTER(falqon_layer), _p, _i, _p, _i64, _p, _p, _p, _i, _p, _f, _p, _p, _sz, _p]
lib.falqon_proxy_update_scored.restype = _i
lib.falqon_proxy_update_scored.argtypes = [C.POINTER(falqon_layer), _i64, _p, _p, _sz, _p]
lib.falqon_proxy_update_scored_batched.restype = _i
lib.falqon_proxy_update_scored_batched.argtypes = [C.POINTER(falqon_layer), C.c_int32, C.POINTER(_i64), C.POINTER(_p), C.POINTER(_p),
                                                   C.POINTER(_sz), _p]
lib.falqon_melded_backward_codes.restype = _i
lib.falqon_melded_backward_codes.argtypes = [C.POINTER(falqon_layer), _p, _p, _i64, _p, _p, _p, _i, _p, _p, _sz, _p]
lib.falqon_melded_backward_dx.restype = _i
lib.falqon_melded_backward_dx.argtypes = [C.POINTER(falqon_layer), _i64, _p, _i, _p, _sz, _p]
lib.falqon_melded_forward_codes.restype = _i
lib.falqon_melded_forward_codes.argtypes = [C.POINTER(falqon_layer), _p, _p, _i64, _p, _i, _p, _p, _p, _sz, _p]
lib.falqon_melded_backward.restype = _i
lib.falqon_melded_backward.argtypes = [C.POINTER(falqon_layer), _p, _i, _i64, _p, _p, _p, _i, _p, _p, _p, _sz, _p]
lib.falqon_proxy_update.restype = _i
lib.falqon_proxy_update.argtypes = [C.POINTER(falqon_layer), _p, _f, _i64, _p, _p, _sz, _p]
lib.falqon_proxy_update_batched.restype = _i
lib.falqon_proxy_update_batched.argtypes = [C.POINTER(falqon_layer), C.c_int32, C.POINTER(_p), _f, C.POINTER(_i64), C.POINTER(_p),
                                            C.POINTER(_p), C.POINTER(_sz), _p]
lib.falqon_proxy_update_batched_adamw.restype = _i
lib.falqon_proxy_update_batched_adamw.argtypes = [C.POINTER(falqon_layer), C.c_int32, C.POINTER(_p), C.POINTER(_p), C.POINTER(_p),
                                                  C.c_void_p, C.POINTER(_i64), C.POINTER(_p), C.POINTER(_p), C.POINTER(_sz), _p]
lib.falqon_selftest_wait_timeout.restype = _i
lib.falqon_selftest_wait_timeout.argtypes = [C.c_uint32, _p]
lib.falqon_absmax.restype = _i
lib.falqon_absmax.argtypes = [_p, _i, _i64, _p, _p, _sz, _p]
lib.falqon_tensor_ceiling.restype = _i
lib.falqon_tensor_ceiling.argtypes = [_i64, C.c_uint32, C.c_int32, _p, C.POINTER(C.c_double), _p, _sz, C.c_int32, _p]
lib.falqon_tensor_ceiling_ctas.restype = _i
lib.falqon_tensor_ceiling_ctas.argtypes = []
class falqon_adamw(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("step", C.c_int64)]


lib.falqon_proxy_update_adamw.restype = _i
lib.falqon_proxy_update_adamw.argtypes = [C.POINTER(falqon_layer), _p, _p, _p, C.POINTER(falqon_adamw), _i64, _p, _p, _sz, _p]
lib.falqon_exact_merge_scratch_bytes.restype = _sz
lib.falqon_exact_merge_scratch_bytes.argtypes = [_i64, _i64, _i64]
lib.falqon_proxy_update_exact.restype = _i
lib.falqon_proxy_update_exact.argtypes = [C.POINTER(falqon_layer), _p, _f, _i64, _p, _p, _sz, _p, _sz, _p, _p, _p]
lib.falqon_svd_init_scratch_bytes.restype = _sz
lib.falqon_svd_init_scratch_bytes.argtypes = [_i64, _i64, _i64]
lib.falqon_svd_init.restype = _i
lib.falqon_svd_init.argtypes = [_p, _i, _i64, _i64, _p, _p, _i64, _p, _i64, C.c_int32, _p, _p, _p, _sz, _p]
lib.falqon_proxy_update_static.restype = _i
lib.falqon_proxy_update_static.argtypes = [C.POINTER(falqon_layer), _p, _f, _i64, _p, _p]
lib.falqon_last_device_status.restype = _i
lib.falqon_last_device_status.argtypes = [_p]
lib.falqon_profile_start.restype = _i
lib.falqon_profile_start.argtypes = [_i, C.c_uint]
lib.falqon_profile_stop.restype = _i
lib.falqon_profile_stop.argtypes = [C.POINTER(_f), C.POINTER(_i), _i]
lib.falqon_launch_count.restype = _i
lib.falqon_launch_count.argtypes = [C.c_char_p, _i64, _i64, _i64, _i64, _i64]


class FalqonError(RuntimeError):
    def __init__(self, call: str, status: int):
        super().__init__(f"{call} returned status {status}")
        self.status = status


def _check(call: str, status: int):
    if status != OK:
        raise FalqonError(call, status)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream():
    return torch.cuda.current_stream().cuda_stream


class Layer:
    """Owns the device tensors of one melded layer and the host struct that points at them."""

    def __init__(self, wq: torch.Tensor, s_w: torch.Tensor, dbuf: torch.Tensor, r: int, flags: int = 0):
        assert wq.dtype == torch.uint8 and wq.is_contiguous() and dbuf.dtype == torch.float32 and dbuf.is_contiguous()
        self.wq, self.s_w, self.dbuf = wq, s_w, dbuf
        self.m, self.n, self.r = wq.shape[0] - r, wq.shape[1], r
        assert s_w.numel() in (1, self.m + 1) and s_w.dtype == torch.float32 and s_w.is_contiguous()
        self.gran = PER_ROW if s_w.numel() == self.m + 1 else PER_TENSOR
        self.c = falqon_layer(self.m, self.n, self.r, wq.data_ptr(), s_w.data_ptr(), dbuf.data_ptr(), self.gran, flags)
        self._ws = None

    @property
    def flags(self) -> int:
        return int(self.c.flags)

    @flags.setter
    def flags(self, value: int):
        """falqon_layer.flags: LAYER_FUSED_CAST moves the casts of X and dY into the products' producers; LAYER_DB_OWN_KERNEL
        keeps the adapter gradient out of the input-gradient product's launch."""
        self.c.flags = int(value)

    def workspace(self, T: int) -> torch.Tensor:
        need = workspace_bytes(self.m, self.n, self.r, T)
        if need == 0:
            raise FalqonError("falqon_workspace_bytes", ERR_INVALID_ARG)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.wq.device)
            workspace_init(self._ws)
        return self._ws


def workspace_init(ws: torch.Tensor):
    """falqon_workspace_init: clears the control words of a freshly allocated workspace."""
    _check("falqon_workspace_init", lib.falqon_workspace_init(_ptr(ws), ws.numel(), _stream()))


def workspace_bytes(m: int, n: int, r: int, T: int) -> int:
    return int(lib.falqon_workspace_bytes(m, n, r, T))


def workspace_region(m: int, n: int, r: int, T: int, which: int):
    off, size = _sz(), _sz()
    _check("falqon_workspace_region", lib.falqon_workspace_region(m, n, r, T, which, C.byref(off), C.byref(size)))
    return off.value, size.value


def ws_view(layer: Layer, ws: torch.Tensor, T: int, which: int) -> torch.Tensor:
    off, size = workspace_region(layer.m, layer.n, layer.r, T, which)
    return ws[off:off + size]


def launch_count(entry_point: str, m=0, n=0, r=0, T=0, k=0) -> int:
    return int(lib.falqon_launch_count(entry_point.encode(), m, n, r, T, k))


def last_device_status() -> int:
    return int(lib.falqon_last_device_status(_stream()))


def profile_start(max_records: int, stages=None):
    mask = 0
    for s in (STAGES if stages is None else stages):
        mask |= 1 << STAGES.index(s)
    _check("falqon_profile_start", lib.falqon_profile_start(max_records, mask))


def profile_stop(capacity: int):
    """Returns a list of (stage name, milliseconds) in call order."""
    ms = (_f * capacity)()
    kinds = (_i * capacity)()
    n = lib.falqon_profile_stop(ms, kinds, capacity)
    if n < 0:
        raise FalqonError("falqon_profile_stop", n)
    return [(STAGES[kinds[i]], float(ms[i])) for i in range(n)]


def quantize(src: torch.Tensor, fmt: int, gran: int = PER_TENSOR, scale_in: torch.Tensor | None = None,
             premul: float = 1.0, want_amax: bool = True, dst: torch.Tensor | None = None):
    """falqon_quantize.  Returns (codes uint8 [rows, cols], scale fp32 [1] or [rows], amax or None)."""
    assert src.dim() == 2 and src.is_contiguous()
    rows, cols = src.shape
    groups = rows if gran == PER_ROW else 1
    dev = src.device
    if dst is None:
        dst = torch.empty((rows, cols), dtype=torch.uint8, device=dev)
    scale_out = torch.empty(groups, dtype=torch.float32, device=dev)
    amax_out = torch.empty(groups, dtype=torch.float32, device=dev) if want_amax else None
    ws = torch.empty(8192, dtype=torch.uint8, device=dev)
    _check("falqon_quantize", lib.falqon_quantize(_ptr(src), _dt(src), rows, cols, fmt, gran, _ptr(scale_in), premul,
                                                  _ptr(dst), _ptr(scale_out), _ptr(amax_out), _ptr(ws), ws.numel(),
                                                  _stream()))
    return dst, scale_out, amax_out


def melded_forward(layer: Layer, X: torch.Tensor, y_dtype=torch.bfloat16, ws: torch.Tensor | None = None, out=None,
                   amax_x: torch.Tensor | None = None):
    """falqon_melded_forward (falqon_melded_forward_amax when amax_x, fp32 [1] = max |X|, is given).
    Returns (Y [T, m], OA fp32 [T, r], amax_oa fp32 [1], s_x fp32 [1])."""
    assert X.dim() == 2 and X.is_contiguous() and X.shape[1] == layer.n
    T = X.shape[0]
    dev = X.device
    ws = layer.workspace(T) if ws is None else ws
    if out is None:
        Y = torch.empty((T, layer.m), dtype=y_dtype, device=dev)
        OA = torch.empty((T, layer.r), dtype=torch.float32, device=dev)
        amax_oa = torch.empty(1, dtype=torch.float32, device=dev)
        s_x = torch.empty(1, dtype=torch.float32, device=dev)
    else:
        Y, OA, amax_oa, s_x = out
    if amax_x is not None:
        assert amax_x.dtype == torch.float32 and amax_x.numel() == 1
        _check("falqon_melded_forward_amax",
               lib.falqon_melded_forward_amax(C.byref(layer.c), _ptr(X), _dt(X), _ptr(amax_x), T, _ptr(Y), _dt(Y), _ptr(OA),
                                              _ptr(amax_oa), _ptr(s_x), _ptr(ws), ws.numel(), _stream()))
        return Y, OA, amax_oa, s_x
    _check("falqon_melded_forward", lib.falqon_melded_forward(C.byref(layer.c), _ptr(X), _dt(X), T, _ptr(Y), _dt(Y),
                                                              _ptr(OA), _ptr(amax_oa), _ptr(s_x), _ptr(ws), ws.numel(),
                                                              _stream()))
    return Y, OA, amax_oa, s_x


def melded_forward_dump(layer: Layer, X: torch.Tensor, n_block: int, y_dtype=torch.float32, ws: torch.Tensor | None = None,
                        amax_x: torch.Tensor | None = None):
    """falqon_melded_forward_dump: the fused forward whose column block n_block also writes its staged codes to WS_XQ.
    Returns (Y, OA, amax_oa, s_x) like melded_forward."""
    T = X.shape[0]
    dev = X.device
    ws = layer.workspace(T) if ws is None else ws
    Y = torch.empty((T, layer.m), dtype=y_dtype, device=dev)
    OA = torch.empty((T, layer.r), dtype=torch.float32, device=dev)
    amax_oa = torch.empty(1, dtype=torch.float32, device=dev)
    s_x = torch.empty(1, dtype=torch.float32, device=dev)
    _check("falqon_melded_forward_dump",
           lib.falqon_melded_forward_dump(C.byref(layer.c), _ptr(X), _dt(X), _ptr(amax_x), T, _ptr(Y), _dt(Y), _ptr(OA),
                                          _ptr(amax_oa), _ptr(s_x), n_block, _ptr(ws), ws.numel(), _stream()))
    return Y, OA, amax_oa, s_x


def melded_backward_dump(layer: Layer, dY: torch.Tensor, OA: torch.Tensor, amax_oa: torch.Tensor, n_block: int,
                         dx_dtype=torch.float32, ws: torch.Tensor | None = None, amax_dy: torch.Tensor | None = None):
    """falqon_melded_backward_dump: the fused backward whose dX column block n_block writes the codes of dY to WS_GQ.
    Returns (dX, dB, s_g) like melded_backward."""
    T = dY.shape[0]
    dev = dY.device
    ws = layer.workspace(T) if ws is None else ws
    dX = torch.empty((T, layer.n), dtype=dx_dtype, device=dev)
    dB = torch.empty((layer.m, layer.r), dtype=torch.float32, device=dev)
    s_g = torch.empty(1, dtype=torch.float32, device=dev)
    _check("falqon_melded_backward_dump",
           lib.falqon_melded_backward_dump(C.byref(layer.c), _ptr(dY), _dt(dY), _ptr(amax_dy), T, _ptr(OA), _ptr(amax_oa),
                                           _ptr(dX), _dt(dX), _ptr(dB), _ptr(s_g), n_block, _ptr(ws), ws.numel(), _stream()))
    return dX, dB, s_g


def melded_forward_codes(layer: Layer, xq: torch.Tensor, s_x: torch.Tensor, y_dtype=torch.bfloat16,
                         ws: torch.Tensor | None = None, out=None):
    """falqon_melded_forward_codes: the forward product on activations another layer already quantized
    (xq uint8 [T, n], s_x fp32 [1]).  Returns (Y [T, m], OA fp32 [T, r], amax_oa fp32 [1])."""
    assert xq.dim() == 2 and xq.is_contiguous() and xq.shape[1] == layer.n and xq.dtype == torch.uint8
    assert s_x.dtype == torch.float32 and s_x.numel() == 1
    T = xq.shape[0]
    dev = xq.device
    ws = layer.workspace(T) if ws is None else ws
    if out is None:
        Y = torch.empty((T, layer.m), dtype=y_dtype, device=dev)
        OA = torch.empty((T, layer.r), dtype=torch.float32, device=dev)
        amax_oa = torch.empty(1, dtype=torch.float32, device=dev)
    else:
        Y, OA, amax_oa = out
    _check("falqon_melded_forward_codes", lib.falqon_melded_forward_codes(C.byref(layer.c), _ptr(xq), _ptr(s_x), T, _ptr(Y),
                                                                          _dt(Y), _ptr(OA), _ptr(amax_oa), _ptr(ws),
                                                                          ws.numel(), _stream()))
    return Y, OA, amax_oa


def melded_backward(layer: Layer, dY: torch.Tensor, OA: torch.Tensor, amax_oa: torch.Tensor, need_dx: bool = True,
                    dx_dtype=torch.bfloat16, ws: torch.Tensor | None = None, out=None, amax_dy: torch.Tensor | None = None):
    """falqon_melded_backward (falqon_melded_backward_amax when amax_dy, fp32 [1] = max |dY|, is given).
    Returns (dX [T, n] or None, dB fp32 [m, r], s_g fp32 [1])."""
    assert dY.dim() == 2 and dY.is_contiguous() and dY.shape[1] == layer.m
    T = dY.shape[0]
    dev = dY.device
    ws = layer.workspace(T) if ws is None else ws
    if out is None:
        dX = torch.empty((T, layer.n), dtype=dx_dtype, device=dev) if need_dx else None
        dB = torch.empty((layer.m, layer.r), dtype=torch.float32, device=dev)
        s_g = torch.empty(1, dtype=torch.float32, device=dev)
    else:
        dX, dB, s_g = out
    dx_dt = _dt(dX) if dX is not None else BF16
    if amax_dy is not None:
        assert amax_dy.dtype == torch.float32 and amax_dy.numel() == 1
        _check("falqon_melded_backward_amax",
               lib.falqon_melded_backward_amax(C.byref(layer.c), _ptr(dY), _dt(dY), _ptr(amax_dy), T, _ptr(OA), _ptr(amax_oa),
                                               _ptr(dX), dx_dt, _ptr(dB), _ptr(s_g), _ptr(ws), ws.numel(), _stream()))
        return dX, dB, s_g
    _check("falqon_melded_backward", lib.falqon_melded_backward(C.byref(layer.c), _ptr(dY), _dt(dY), T, _ptr(OA),
                                                                _ptr(amax_oa), _ptr(dX), dx_dt, _ptr(dB), _ptr(s_g),
                                                                _ptr(ws), ws.numel(), _stream()))
    return dX, dB, s_g


UA_SCALARS, UA_BQ_T, UA_P, UA_PQ_T, UA_DA_T = range(5)


def update_a(layer: Layer, xq: torch.Tensor, s_x: torch.Tensor, B: torch.Tensor, A_master: torch.Tensor, gamma: float, lr: float,
             T: int, ws: torch.Tensor | None = None, scratch: torch.Tensor | None = None) -> torch.Tensor:
    """falqon_update_a: one SGD step of a trainable A after the backward of the same step (in place on A_master fp32 [r, n]
    and on the A~ rows of layer.wq).  xq uint8 [T, n], s_x fp32 [1]: the forward's codes of X, kept by the caller; B fp32
    [m, r].  Returns the scratch tensor; ua_view gives its regions."""
    assert xq.dtype == torch.uint8 and xq.is_contiguous() and B.dtype == torch.float32 and B.is_contiguous()
    assert A_master.dtype == torch.float32 and A_master.is_contiguous() and A_master.shape == (layer.r, layer.n)
    ws = layer.workspace(T) if ws is None else ws
    if scratch is None:
        scratch = torch.empty(int(lib.falqon_update_a_scratch_bytes(layer.m, layer.n, layer.r, T)), dtype=torch.uint8,
                              device=layer.wq.device)
    _check("falqon_update_a", lib.falqon_update_a(C.byref(layer.c), _ptr(xq), _ptr(s_x), _ptr(B), _ptr(A_master), gamma, lr, T,
                                                  _ptr(ws), ws.numel(), _ptr(scratch), scratch.numel(), _stream()))
    return scratch


def ua_view(layer: Layer, scratch: torch.Tensor, T: int, which: int) -> torch.Tensor:
    off, size = _sz(), _sz()
    _check("falqon_update_a_region", lib.falqon_update_a_region(layer.m, layer.n, layer.r, T, which, C.byref(off), C.byref(size)))
    return scratch[off.value:off.value + size.value]


def melded_backward_update(layer: Layer, dY: torch.Tensor, OA: torch.Tensor, amax_oa: torch.Tensor, lr: float, need_dx: bool = True,
                           dx_dtype=torch.bfloat16, ws: torch.Tensor | None = None, out=None, amax_dy: torch.Tensor | None = None):
    """falqon_melded_backward_update: the backward with the plain-SGD step on the DeltaBuffer and the row scores fused into
    the adapter-gradient kernel (the scores stay in the workspace for proxy_update_scored).  Returns (dX or None, dB, s_g)."""
    T = dY.shape[0]
    dev = dY.device
    ws = layer.workspace(T) if ws is None else ws
    if out is None:
        dX = torch.empty((T, layer.n), dtype=dx_dtype, device=dev) if need_dx else None
        dB = torch.empty((layer.m, layer.r), dtype=torch.float32, device=dev)
        s_g = torch.empty(1, dtype=torch.float32, device=dev)
    else:
        dX, dB, s_g = out
    _check("falqon_melded_backward_update",
           lib.falqon_melded_backward_update(C.byref(layer.c), _ptr(dY), _dt(dY), _ptr(amax_dy), T, _ptr(OA), _ptr(amax_oa), _ptr(dX),
                                             _dt(dX) if dX is not None else BF16, _ptr(dB), lr, _ptr(s_g), _ptr(ws), ws.numel(),
                                             _stream()))
    return dX, dB, s_g


def proxy_update_scored(layer: Layer, k: int, ws: torch.Tensor | None = None, idx_out: torch.Tensor | None = None):
    """falqon_proxy_update_scored: selection and merge from the scores melded_backward_update left in the workspace."""
    ws = layer.workspace(1) if ws is None else ws
    if idx_out is None and 0 < k <= layer.m:
        idx_out = torch.empty(k, dtype=torch.int32, device=layer.wq.device)
    _check("falqon_proxy_update_scored", lib.falqon_proxy_update_scored(C.byref(layer.c), k, _ptr(idx_out), _ptr(ws), ws.numel(),
                                                                        _stream()))
    return idx_out


def melded_backward_codes(layer: Layer, gq: torch.Tensor, s_g: torch.Tensor, OA: torch.Tensor, amax_oa: torch.Tensor,
                          need_dx: bool = True, dx_dtype=torch.bfloat16, ws: torch.Tensor | None = None, out=None):
    """falqon_melded_backward_codes: the backward on gradient codes another layer already cast (gq uint8 [T, m], s_g fp32 [1]).
    Returns (dX or None, dB)."""
    assert gq.dim() == 2 and gq.is_contiguous() and gq.shape[1] == layer.m and gq.dtype == torch.uint8
    T = gq.shape[0]
    dev = gq.device
    ws = layer.workspace(T) if ws is None else ws
    if out is None:
        dX = torch.empty((T, layer.n), dtype=dx_dtype, device=dev) if need_dx else None
        dB = torch.empty((layer.m, layer.r), dtype=torch.float32, device=dev)
    else:
        dX, dB = out
    _check("falqon_melded_backward_codes",
           lib.falqon_melded_backward_codes(C.byref(layer.c), _ptr(gq), _ptr(s_g), T, _ptr(OA), _ptr(amax_oa), _ptr(dX),
                                            _dt(dX) if dX is not None else BF16, _ptr(dB), _ptr(ws), ws.numel(), _stream()))
    return dX, dB


def melded_backward_dx(layer: Layer, T: int, dx_dtype=torch.bfloat16, ws: torch.Tensor | None = None, out: torch.Tensor | None = None):
    """falqon_melded_backward_dx: dX [T, n] from the gradient codes the preceding melded_backward(need_dx=False) on the same
    workspace left behind."""
    ws = layer.workspace(T) if ws is None else ws
    dX = torch.empty((T, layer.n), dtype=dx_dtype, device=layer.wq.device) if out is None else out
    _check("falqon_melded_backward_dx", lib.falqon_melded_backward_dx(C.byref(layer.c), T, _ptr(dX), _dt(dX), _ptr(ws), ws.numel(),
                                                                      _stream()))
    return dX


def proxy_update(layer: Layer, dB: torch.Tensor | None, lr: float, k: int, ws: torch.Tensor | None = None,
                 idx_out: torch.Tensor | None = None):
    """falqon_proxy_update (in place on layer.wq / layer.dbuf).  Returns idx int32 [k] ascending."""
    ws = layer.workspace(1) if ws is None else ws
    if idx_out is None and 0 < k <= layer.m:
        idx_out = torch.empty(k, dtype=torch.int32, device=layer.wq.device)
    _check("falqon_proxy_update", lib.falqon_proxy_update(C.byref(layer.c), _ptr(dB), lr, k, _ptr(idx_out), _ptr(ws),
                                                          ws.numel(), _stream()))
    return idx_out


def absmax(x: torch.Tensor, out: torch.Tensor | None = None, ws: torch.Tensor | None = None) -> torch.Tensor:
    """falqon_absmax: max |x| of a contiguous bf16 / fp32 tensor as an fp32 device tensor [1]."""
    assert x.is_contiguous()
    dev = x.device
    out = torch.empty(1, dtype=torch.float32, device=dev) if out is None else out
    ws = torch.empty(8192, dtype=torch.uint8, device=dev) if ws is None else ws
    _check("falqon_absmax", lib.falqon_absmax(_ptr(x), _dt(x), x.numel(), _ptr(out), _ptr(ws), ws.numel(), _stream()))
    return out


def tensor_ceiling(kblocks: int, seed: int = 1, random_fill: int = 1, sink: torch.Tensor | None = None,
                   load_src: torch.Tensor | None = None, bytes_per_kblock: int = 0) -> float:
    """falqon_tensor_ceiling: one launch of the MMA-issue-only measurement kernel on the current stream.  Returns the
    floating-point operations of the launch (time a sequence of launches with events to get a rate).  load_src: an
    optional uint8 device buffer whose 16 KB chunks are streamed into the operand slots as a product's operands are."""
    flops = C.c_double()
    _check("falqon_tensor_ceiling", lib.falqon_tensor_ceiling(kblocks, seed, int(random_fill), _ptr(sink), C.byref(flops),
                                                             _ptr(load_src), 0 if load_src is None else load_src.numel(),
                                                             bytes_per_kblock, _stream()))
    return flops.value


def tensor_ceiling_ctas() -> int:
    return int(lib.falqon_tensor_ceiling_ctas())


class ProxyBatch:
    """The host arrays of one falqon_proxy_update_batched call, marshalled once and reusable while the tensors live:
    layers, their adapter gradients (entries may be None), k per layer, workspaces and index outputs."""

    def __init__(self, layers, dBs, ks, wss=None, idx_outs=None):
        n = len(layers)
        assert len(dBs) == n and len(ks) == n
        self.layers, self.dBs, self.ks = list(layers), list(dBs), [int(k) for k in ks]
        self.wss = [L.workspace(1) for L in layers] if wss is None else list(wss)
        if idx_outs is None:
            idx_outs = [torch.empty(k, dtype=torch.int32, device=L.wq.device) if 0 < k <= L.m else None
                        for L, k in zip(self.layers, self.ks)]
        self.idx_outs = list(idx_outs)
        self.c_layers = (falqon_layer * max(n, 1))(*[L.c for L in self.layers])
        self.c_dB = (_p * max(n, 1))(*[_ptr(t) for t in self.dBs])
        self.c_k = (_i64 * max(n, 1))(*self.ks)
        self.c_idx = (_p * max(n, 1))(*[_ptr(t) for t in self.idx_outs])
        self.c_ws = (_p * max(n, 1))(*[_ptr(t) for t in self.wss])
        self.c_ws_bytes = (_sz * max(n, 1))(*[t.numel() for t in self.wss])
        self.count = n

    def run_adamw(self, exp_avgs, exp_avg_sqs, lr: float, beta1: float, beta2: float, eps: float, weight_decay: float, step: int):
        """falqon_proxy_update_batched_adamw with the per-layer state tensors exp_avgs / exp_avg_sqs (fp32 [m, r] each)."""
        n = max(self.count, 1)
        hp = falqon_adamw(lr, beta1, beta2, eps, weight_decay, step)
        c_ea = (_p * n)(*[_ptr(t) for t in exp_avgs])
        c_es = (_p * n)(*[_ptr(t) for t in exp_avg_sqs])
        _check("falqon_proxy_update_batched_adamw",
               lib.falqon_proxy_update_batched_adamw(self.c_layers, self.count, self.c_dB, c_ea, c_es, C.byref(hp), self.c_k,
                                                     self.c_idx, self.c_ws, self.c_ws_bytes, _stream()))
        return self.idx_outs

    def prepare_exact(self):
        """Scratch for the correctly rounded merge of every layer, with the bf16 copy of its A~ rows prepared once
        (falqon_exact_merge_prepare).  Call again after anything changed the A~ rows."""
        self.scratch = [torch.empty(int(lib.falqon_exact_merge_scratch_bytes(L.m, L.n, L.r)), dtype=torch.uint8, device=L.wq.device)
                        for L in self.layers]
        n = max(self.count, 1)
        self.c_scratch = (_p * n)(*[_ptr(t) for t in self.scratch])
        self.c_scratch_bytes = (_sz * n)(*[t.numel() for t in self.scratch])
        for L, sc in zip(self.layers, self.scratch):
            _check("falqon_exact_merge_prepare", lib.falqon_exact_merge_prepare(C.byref(L.c), _ptr(sc), sc.numel(), _stream()))

    def run_exact(self, lr: float, prepared: bool = True):
        """falqon_proxy_update_batched_exact (prepare_exact must have been called once)."""
        _check("falqon_proxy_update_batched_exact",
               lib.falqon_proxy_update_batched_exact(self.c_layers, self.count, self.c_dB, lr, self.c_k, self.c_idx, self.c_ws,
                                                     self.c_ws_bytes, self.c_scratch, self.c_scratch_bytes, 1 if prepared else 0,
                                                     _stream()))
        return self.idx_outs

    def run_scored(self):
        """falqon_proxy_update_scored_batched: selection and merge only, after melded_backward_update on every layer."""
        _check("falqon_proxy_update_scored_batched",
               lib.falqon_proxy_update_scored_batched(self.c_layers, self.count, self.c_k, self.c_idx, self.c_ws, self.c_ws_bytes,
                                                      _stream()))
        return self.idx_outs

    def run(self, lr: float):
        _check("falqon_proxy_update_batched",
               lib.falqon_proxy_update_batched(self.c_layers, self.count, self.c_dB, lr, self.c_k, self.c_idx, self.c_ws,
                                               self.c_ws_bytes, _stream()))
        return self.idx_outs


def proxy_update_batched(layers, dBs, lr: float, ks, wss=None, idx_outs=None):
    """falqon_proxy_update_batched: the proxy update of several layers in two launches.  Returns the list of idx tensors."""
    return ProxyBatch(layers, dBs, ks, wss, idx_outs).run(lr)


def proxy_update_exact(layer: Layer, dB: torch.Tensor | None, lr: float, k: int, ws: torch.Tensor | None = None,
                       idx_out: torch.Tensor | None = None, scratch: torch.Tensor | None = None, want_sums: bool = False,
                       want_count: bool = True):
    """falqon_proxy_update_exact: the proxy update with the correctly rounded merge.  Returns (idx int32 [k] ascending,
    number of elements that took the exact path as a device int32 [1] or None, the tensor-core sums fp32 [k, n] or None)."""
    ws = layer.workspace(1) if ws is None else ws
    dev = layer.wq.device
    if idx_out is None and 0 < k <= layer.m:
        idx_out = torch.empty(k, dtype=torch.int32, device=dev)
    if scratch is None:
        scratch = torch.empty(int(lib.falqon_exact_merge_scratch_bytes(layer.m, layer.n, layer.r)), dtype=torch.uint8, device=dev)
    fixed = torch.zeros(1, dtype=torch.int32, device=dev) if want_count else None
    sums = torch.empty((k, layer.n), dtype=torch.float32, device=dev) if want_sums and k > 0 else None
    _check("falqon_proxy_update_exact",
           lib.falqon_proxy_update_exact(C.byref(layer.c), _ptr(dB), lr, k, _ptr(idx_out), _ptr(ws), ws.numel(), _ptr(scratch),
                                         scratch.numel(), _ptr(sums), _ptr(fixed), _stream()))
    return idx_out, fixed, sums


def svd_init(W: torch.Tensor, wq: torch.Tensor, s_w: torch.Tensor, r: int, omega: torch.Tensor, power_iters: int = 2):
    """falqon_svd_init: A^ [r, n] fp32 and the r leading singular values of Delta W = W - dec(wq) / s_w.
    wq: uint8 [m, n] codes of W (per-tensor scale s_w); omega: fp32 [n, l] standard normal, l even, r <= l <= 160."""
    m, n = W.shape
    l = omega.shape[1]
    assert wq.shape == (m, n) and wq.dtype == torch.uint8 and wq.is_contiguous() and W.is_contiguous()
    assert omega.shape[0] == n and omega.dtype == torch.float32 and omega.is_contiguous()
    dev = W.device
    A_hat = torch.empty((r, n), dtype=torch.float32, device=dev)
    sigma = torch.empty(r, dtype=torch.float32, device=dev)
    scratch = torch.empty(int(lib.falqon_svd_init_scratch_bytes(m, n, l)), dtype=torch.uint8, device=dev)
    _check("falqon_svd_init", lib.falqon_svd_init(_ptr(W), _dt(W), m, n, _ptr(wq), _ptr(s_w), r, _ptr(omega), l, power_iters,
                                                  _ptr(A_hat), _ptr(sigma), _ptr(scratch), scratch.numel(), _stream()))
    return A_hat, sigma


def setup_layer_svd(W: torch.Tensor, r: int, omega: torch.Tensor, power_iters: int = 2) -> Layer:
    """Alg. 1 in full for one layer: W~, s_W = Q(W); A^ from the SVD of the quantization error; A~ = Q(A^; s_W);
    W~' = [W~; A~]; DeltaBuffer = 0.  omega: fp32 [n, l] standard normal drawn by the caller."""
    m, n = W.shape
    wq = torch.empty((m + r, n), dtype=torch.uint8, device=W.device)
    _, s_w, _ = quantize(W.contiguous(), E4M3, dst=wq[:m])
    A_hat, _ = svd_init(W.contiguous(), wq[:m], s_w, r, omega, power_iters)
    quantize(A_hat, E4M3, scale_in=s_w, want_amax=False, dst=wq[m:])
    return Layer(wq, s_w, torch.zeros((m, r), dtype=torch.float32, device=W.device), r)


def setup_layer(W: torch.Tensor, A: torch.Tensor, B: torch.Tensor | None, gamma: float, per_row: bool = False) -> Layer:
    """Builds a melded layer from W [m, n], A [r, n] and an optional initial B [m, r] (all on the device):
    W~, s_W = Q(W); A~ = Q(gamma*A; s_W); W~' = [W~; A~]; then melds B by the merge operator over all rows
    (dbuf := B, falqon_proxy_update with dB = NULL, k = m), which leaves DeltaBuffer = 0.
    per_row: each row of W gets its own absmax scale and the A~ block one absmax scale of its own."""
    m, n = W.shape
    r = A.shape[0]
    dev = W.device
    wq = torch.empty((m + r, n), dtype=torch.uint8, device=dev)
    if per_row:
        _, s_rows, _ = quantize(W.contiguous(), E4M3, gran=PER_ROW, dst=wq[:m])
        _, s_a, _ = quantize(A.contiguous(), E4M3, premul=gamma, dst=wq[m:])
        s_w = torch.cat([s_rows, s_a]).contiguous()
    else:
        _, s_w, _ = quantize(W.contiguous(), E4M3, dst=wq[:m])
        quantize(A.contiguous(), E4M3, scale_in=s_w, premul=gamma, want_amax=False, dst=wq[m:])
    dbuf = torch.zeros((m, r), dtype=torch.float32, device=dev)
    layer = Layer(wq, s_w, dbuf, r)
    if B is not None:
        dbuf.copy_(B.to(torch.float32))
        proxy_update(layer, None, 0.0, m)
    return layer


def proxy_update_static(layer: Layer, dB: torch.Tensor | None, lr: float, k: int, idx_out: torch.Tensor | None = None):
    """falqon_proxy_update_static: the proxy update for callers that cannot supply a workspace (guests
    of a runtime whose allocator owns the device's memory).  Scratch is a fixed array inside the
    library, so layer.m may not exceed STATIC_MAX_ROWS, calls must not overlap on the GPU, and the
    first call on a device should be made outside any stream capture.  The caller still passes every
    input and output; here idx_out is created with torch only when the caller gave none."""
    if idx_out is None and 0 < k <= layer.m:
        idx_out = torch.empty(k, dtype=torch.int32, device=layer.wq.device)
    _check("falqon_proxy_update_static",
           lib.falqon_proxy_update_static(C.byref(layer.c), _ptr(dB), lr, k, _ptr(idx_out), _stream()))
    return idx_out


def proxy_update_adamw(layer: Layer, dB: torch.Tensor, exp_avg: torch.Tensor, exp_avg_sq: torch.Tensor, step: int, k: int,
                       lr: float = 2e-4, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                       weight_decay: float = 0.0, ws: torch.Tensor | None = None, idx_out: torch.Tensor | None = None):
    """falqon_proxy_update_adamw: AdamW step on the DeltaBuffer (state in exp_avg / exp_avg_sq, fp32 [m, r], zero before
    step 1), then scores, top-k, merge and clearing as in proxy_update.  Returns idx int32 [k] ascending."""
    ws = layer.workspace(1) if ws is None else ws
    if idx_out is None and 0 < k <= layer.m:
        idx_out = torch.empty(k, dtype=torch.int32, device=layer.wq.device)
    hp = falqon_adamw(lr, beta1, beta2, eps, weight_decay, step)
    _check("falqon_proxy_update_adamw",
           lib.falqon_proxy_update_adamw(C.byref(layer.c), _ptr(dB), _ptr(exp_avg), _ptr(exp_avg_sq), C.byref(hp), k,
                                         _ptr(idx_out), _ptr(ws), ws.numel(), _stream()))
    return idx_out
