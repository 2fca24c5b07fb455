"""A chain of decoder-shaped blocks built from melded FP8-LoRA linear layers: the workload of the "32-layer stack"
configuration.  It exists to run the layer in the launch pattern of a training step -- seven projections per block,
q/k/v and gate/up sharing one quantized input, each block's backward followed by its seven proxy updates -- not to
model attention: the token mixing is a stand-in.

Per block (T tokens, hidden H, MLP width F; every linear is a melded layer, everything between them is a bf16
kernel of falqon_chain.h):
    x1 = rmsnorm(h);   q, k, v = L_q(x1), L_k(x1), L_v(x1)      one shared x~
    a  = (q + k + v) / sqrt(3)                                    stand-in for the attention mixing
    h' = h + L_o(a)
    x2 = rmsnorm(h');  g, u = L_gate(x2), L_up(x2)               one shared x~
    z  = silu(g) * u
    h_next = (h' + L_down(z)) / sqrt(2)
Loss = <h_last, G>.  The backward mirrors this; kept for it per block are h, h' (for the norms), g, u (for the
gate) and each projection's O_A -- the melded layer needs neither its input nor A for its gradients.  (Without the
norms the gated MLP squares the scale of the residual stream in every block and bf16 overflows within a few.)

Only argument marshalling and buffer bookkeeping happen here; every arithmetic step runs in the library's kernels.
"""
import ctypes as C
import math

import torch

from . import binding as fq
from . import synth

lib = fq.lib
_p, _f, _i64 = C.c_void_p, C.c_float, C.c_int64
lib.falqon_chain_combine.restype = C.c_int
lib.falqon_chain_combine.argtypes = [_p, _p, _f, _p, _f, _p, _f, _p, _f, _i64, _p, _p]
lib.falqon_chain_silu_mul.restype = C.c_int
lib.falqon_chain_silu_mul.argtypes = [_p, _p, _p, _i64, _p, _p]
lib.falqon_chain_silu_mul_grad.restype = C.c_int
lib.falqon_chain_silu_mul_grad.argtypes = [_p, _p, _p, _p, _p, _i64, _p, _p, _p]
lib.falqon_chain_rmsnorm.restype = C.c_int
lib.falqon_chain_rmsnorm.argtypes = [_p, _p, _p, _i64, _i64, _f, _p, _p]
lib.falqon_chain_rmsnorm_grad.restype = C.c_int
lib.falqon_chain_rmsnorm_grad.argtypes = [_p, _p, _p, _p, _i64, _i64, _p]
lib.falqon_chain_combine_rmsnorm.restype = C.c_int
lib.falqon_chain_combine_rmsnorm.argtypes = [_p, _p, _p, _p, _f, _p, _f, _i64, _i64, _f, _p, _p]
lib.falqon_chain_rmsnorm_grad_combine.restype = C.c_int
lib.falqon_chain_rmsnorm_grad_combine.argtypes = [_p, _p, _p, _p, _p, _p, _p, _f, _i64, _i64, _p, _p]
_fp, _int = C.c_void_p, C.c_int
lib.falqon_chain_combine_quantize.restype = C.c_int
lib.falqon_chain_combine_quantize.argtypes = [_p, _fp, _int, _p, _int, _p, _f, _p, _f, _p, _f, _p, _f, _i64, _p, _p]
lib.falqon_chain_silu_mul_quantize.restype = C.c_int
lib.falqon_chain_silu_mul_quantize.argtypes = [_p, _fp, _int, _p, _int, _p, _p, _i64, _p, _p]
lib.falqon_chain_silu_mul_grad_quantize.restype = C.c_int
lib.falqon_chain_silu_mul_grad_quantize.argtypes = [_p, _p, _fp, _fp, _int, _p, _p, _int, _p, _p, _p, _i64, _p, _p]
lib.falqon_chain_rmsnorm_quantize.restype = C.c_int
lib.falqon_chain_rmsnorm_quantize.argtypes = [_p, _fp, _int, _p, _int, _p, _p, _p, _f, _p, _f, _i64, _i64, _f, _p, _p]
lib.falqon_chain_rmsnorm_grad_combine_quantize.restype = C.c_int
lib.falqon_chain_rmsnorm_grad_combine_quantize.argtypes = [_p, _fp, _int, _p, _p, _p, _p, _p, _p, _p, _f, _i64, _i64, _p, _p]
CHAIN_EXPORTS = ["falqon_chain_combine", "falqon_chain_silu_mul", "falqon_chain_silu_mul_grad", "falqon_chain_rmsnorm",
                 "falqon_chain_rmsnorm_grad", "falqon_chain_combine_rmsnorm", "falqon_chain_rmsnorm_grad_combine",
                 "falqon_chain_combine_quantize", "falqon_chain_silu_mul_quantize", "falqon_chain_silu_mul_grad_quantize",
                 "falqon_chain_rmsnorm_quantize", "falqon_chain_rmsnorm_grad_combine_quantize"]
CHAIN_SCRATCH_BYTES = 4096
NORM_EPS = 1e-6

PROJ = ["q", "k", "v", "o", "gate", "up", "down"]
INV_SQRT3 = 1.0 / math.sqrt(3.0)
INV_SQRT2 = 1.0 / math.sqrt(2.0)


def _ptr(t):
    return None if t is None else t.data_ptr()


def combine(out, a, sa=1.0, b=None, sb=1.0, c=None, sc=1.0, d=None, sd=1.0, amax=None):
    """out = bf16(sa*a + sb*b + sc*c + sd*d); b, c, d optional.  amax (fp32 [1], zero beforehand): raised to max |out|."""
    for t in (out, a, b, c, d):
        assert t is None or (t.dtype == torch.bfloat16 and t.is_contiguous() and t.numel() == out.numel())
    fq._check("falqon_chain_combine", lib.falqon_chain_combine(_ptr(out), _ptr(a), sa, _ptr(b), sb, _ptr(c), sc, _ptr(d), sd,
                                                                out.numel(), _ptr(amax), fq._stream()))
    return out


def silu_mul(z, g, u, amax=None):
    for t in (z, g, u):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.numel() == z.numel()
    fq._check("falqon_chain_silu_mul", lib.falqon_chain_silu_mul(_ptr(z), _ptr(g), _ptr(u), z.numel(), _ptr(amax), fq._stream()))
    return z


def silu_mul_grad(dg, du, g, u, dz, amax_dg=None, amax_du=None):
    for t in (dg, du, g, u, dz):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.numel() == g.numel()
    fq._check("falqon_chain_silu_mul_grad", lib.falqon_chain_silu_mul_grad(_ptr(dg), _ptr(du), _ptr(g), _ptr(u), _ptr(dz),
                                                                            g.numel(), _ptr(amax_dg), _ptr(amax_du),
                                                                            fq._stream()))
    return dg, du


def rmsnorm(y, inv_rms, x, amax=None):
    assert x.dtype == torch.bfloat16 and x.dim() == 2 and x.is_contiguous() and y.shape == x.shape and y.is_contiguous()
    assert inv_rms.dtype == torch.float32 and inv_rms.numel() == x.shape[0]
    fq._check("falqon_chain_rmsnorm", lib.falqon_chain_rmsnorm(_ptr(y), _ptr(inv_rms), _ptr(x), x.shape[0], x.shape[1],
                                                                NORM_EPS, _ptr(amax), fq._stream()))
    return y


def rmsnorm_grad(dx, dy, x, inv_rms):
    for t in (dx, dy, x):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape == x.shape
    fq._check("falqon_chain_rmsnorm_grad", lib.falqon_chain_rmsnorm_grad(_ptr(dx), _ptr(dy), _ptr(x), _ptr(inv_rms), x.shape[0],
                                                                          x.shape[1], fq._stream()))
    return dx


def combine_rmsnorm(sum_out, y, inv_rms, a, sa, b, sb, amax=None):
    """sum_out = bf16(sa*a + sb*b) and y = rmsnorm(sum_out) in one pass (bit for bit combine followed by rmsnorm)."""
    for t in (sum_out, y, a, b):
        assert t.dtype == torch.bfloat16 and t.dim() == 2 and t.is_contiguous() and t.shape == a.shape
    assert inv_rms.dtype == torch.float32 and inv_rms.numel() == a.shape[0]
    fq._check("falqon_chain_combine_rmsnorm",
              lib.falqon_chain_combine_rmsnorm(_ptr(sum_out), _ptr(y), _ptr(inv_rms), _ptr(a), sa, _ptr(b), sb, a.shape[0], a.shape[1],
                                               NORM_EPS, _ptr(amax), fq._stream()))
    return y


def rmsnorm_grad_combine(out, dys, x, inv_rms, res, s_res, amax=None):
    """out = bf16(s_res*res + rmsnorm_grad(bf16(sum of the two or three dys), x, inv_rms)) in one pass (bit for bit the three
    separate kernels)."""
    assert len(dys) in (2, 3)
    for t in (out, x, res, *dys):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape == x.shape
    fq._check("falqon_chain_rmsnorm_grad_combine",
              lib.falqon_chain_rmsnorm_grad_combine(_ptr(out), _ptr(dys[0]), _ptr(dys[1]), _ptr(dys[2]) if len(dys) == 3 else None,
                                                    _ptr(x), _ptr(inv_rms), _ptr(res), s_res, x.shape[0], x.shape[1], _ptr(amax),
                                                    fq._stream()))
    return out


def chain_scratch(device):
    """The zeroed scratch of the quantizing chain calls (one per stream that runs them)."""
    return torch.zeros(CHAIN_SCRATCH_BYTES, dtype=torch.uint8, device=device)


def _q_args(codes, scale, out16, count):
    assert codes.dtype == torch.uint8 and codes.is_contiguous() and codes.numel() >= count
    assert scale.dtype == torch.float32 and scale.numel() == 1
    assert out16.dtype == torch.bfloat16 and out16.is_contiguous() and out16.numel() == count


def combine_quantize(codes, scale, fmt, out16, keep16, scratch, a, sa=1.0, b=None, sb=1.0, c=None, sc=1.0, d=None, sd=1.0):
    """combine(...) and the per-tensor cast of its result in one launch: codes (uint8) and scale (fp32 [1]) as quantize gives
    them for the bf16 result; out16 receives that result only if keep16 (otherwise it is working space)."""
    _q_args(codes, scale, out16, a.numel())
    for t in (a, b, c, d):
        assert t is None or (t.dtype == torch.bfloat16 and t.is_contiguous() and t.numel() == a.numel())
    fq._check("falqon_chain_combine_quantize",
              lib.falqon_chain_combine_quantize(_ptr(codes), _ptr(scale), fmt, _ptr(out16), int(keep16), _ptr(a), sa, _ptr(b), sb,
                                                _ptr(c), sc, _ptr(d), sd, a.numel(), _ptr(scratch), fq._stream()))


def silu_mul_quantize(codes, scale, fmt, out16, keep16, scratch, g, u):
    _q_args(codes, scale, out16, g.numel())
    for t in (g, u):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.numel() == g.numel()
    fq._check("falqon_chain_silu_mul_quantize",
              lib.falqon_chain_silu_mul_quantize(_ptr(codes), _ptr(scale), fmt, _ptr(out16), int(keep16), _ptr(g), _ptr(u), g.numel(),
                                                 _ptr(scratch), fq._stream()))


def silu_mul_grad_quantize(codes_dg, codes_du, scale_dg, scale_du, fmt, dg16, du16, keep16, scratch, g, u, dz):
    _q_args(codes_dg, scale_dg, dg16, g.numel())
    _q_args(codes_du, scale_du, du16, g.numel())
    for t in (g, u, dz):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.numel() == g.numel()
    fq._check("falqon_chain_silu_mul_grad_quantize",
              lib.falqon_chain_silu_mul_grad_quantize(_ptr(codes_dg), _ptr(codes_du), _ptr(scale_dg), _ptr(scale_du), fmt, _ptr(dg16),
                                                      _ptr(du16), int(keep16), _ptr(g), _ptr(u), _ptr(dz), g.numel(), _ptr(scratch),
                                                      fq._stream()))


def rmsnorm_quantize(codes, scale, fmt, y16, keep16, scratch, inv_rms, a, sum_out=None, sa=1.0, b=None, sb=1.0):
    """rmsnorm(a), or combine_rmsnorm(sum_out, ., a, sa, b, sb) when b and sum_out are given, with the cast of the result."""
    _q_args(codes, scale, y16, a.numel())
    assert a.dtype == torch.bfloat16 and a.dim() == 2 and a.is_contiguous()
    assert inv_rms.dtype == torch.float32 and inv_rms.numel() == a.shape[0]
    for t in (b, sum_out):
        assert t is None or (t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape == a.shape)
    fq._check("falqon_chain_rmsnorm_quantize",
              lib.falqon_chain_rmsnorm_quantize(_ptr(codes), _ptr(scale), fmt, _ptr(y16), int(keep16), _ptr(inv_rms), _ptr(sum_out),
                                                _ptr(a), sa, _ptr(b), sb, a.shape[0], a.shape[1], NORM_EPS, _ptr(scratch),
                                                fq._stream()))


def rmsnorm_grad_combine_quantize(codes, scale, fmt, out, scratch, dys, x, inv_rms, res, s_res):
    """rmsnorm_grad_combine(out, ...) with the cast of out in the same launch."""
    assert len(dys) in (2, 3)
    _q_args(codes, scale, out, x.numel())
    for t in (x, res, *dys):
        assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape == x.shape
    fq._check("falqon_chain_rmsnorm_grad_combine_quantize",
              lib.falqon_chain_rmsnorm_grad_combine_quantize(_ptr(codes), _ptr(scale), fmt, _ptr(out), _ptr(dys[0]), _ptr(dys[1]),
                                                             _ptr(dys[2]) if len(dys) == 3 else None, _ptr(x), _ptr(inv_rms),
                                                             _ptr(res), s_res, x.shape[0], x.shape[1], _ptr(scratch), fq._stream()))


class Stack:
    """n_layers blocks with hidden size H and MLP width F, T tokens per step, LoRA rank r, top-k rows per update."""

    def __init__(self, n_layers: int, H: int, F: int, T: int, r: int, k: int, seed: int, device, lr: float = 2e-4,
                 producer_amax: bool = True, batched_proxy: bool = True, adamw: dict | None = None, fuse_chain: bool = True,
                 fuse_cast: bool | None = None, layer_flags: int = 0):
        """producer_amax: the chain kernels hand the absmax of their outputs to the layers that consume them, whose
        input casts are then single-pass (False: every layer takes the absmax of its input itself).
        batched_proxy: the seven proxy updates of a block run as one falqon_proxy_update_batched call at the end of
        the block's backward (False: one falqon_proxy_update after every projection's backward; same results, since
        nothing later in the backward reads an updated backbone).
        fuse_cast: every tensor a layer consumes (x1, a, x2, z and the output gradients) leaves the chain kernel that
        produces it as FP8 codes (the *_quantize calls above): no separate cast kernel runs, the layers take codes
        (falqon_melded_forward_codes / falqon_melded_backward_codes).  Same codes, so the same results bit for bit.
        layer_flags: falqon_layer.flags of every layer (binding.LAYER_*).
        adamw: None for the plain SGD step with lr, or the hyper-parameters (beta1, beta2, eps, weight_decay; lr is the
        argument above) of AdamW on every DeltaBuffer -- the optimizer the paper trains with; needs batched_proxy."""
        self.n_layers, self.H, self.F, self.T, self.r, self.k, self.lr = n_layers, H, F, T, r, k, lr
        self.adamw, self.steps_done = adamw, 0
        assert adamw is None or batched_proxy
        self.producer_amax = producer_amax
        self.fuse_chain = fuse_chain        # residual sums fused with the normalisation (or its gradient) that follows them
        if fuse_cast is None:               # the default wherever it applies
            fuse_cast = fuse_chain and producer_amax
        self.fuse_cast = fuse_cast
        self.own_db = (layer_flags & fq.LAYER_DB_OWN_KERNEL) != 0
        assert not fuse_cast or (fuse_chain and producer_amax)
        self.device = torch.device(device)
        self.seed = seed
        self.shapes = {"q": (H, H), "k": (H, H), "v": (H, H), "o": (H, H), "gate": (H, F), "up": (H, F), "down": (F, H)}  # n -> m
        self.layers = []
        for l in range(n_layers):
            block = {}
            for pi, name in enumerate(PROJ):
                n, m = self.shapes[name]
                mat = l * len(PROJ) + pi
                W = synth.backbone(seed, mat, m, n, self.device)
                A = synth.adapter_a(seed, mat, r, n, self.device)
                B = synth.adapter_b(seed, mat, m, r, self.device)
                block[name] = fq.setup_layer(W, A, B, 1.0)
                block[name].flags = layer_flags
                del W, A, B
            self.layers.append(block)
        dev, bf = self.device, torch.bfloat16
        # one workspace per projection kind, shared by all blocks (the stream serialises their use)
        self.ws = {}
        for name in PROJ:
            n, m = self.shapes[name]
            self.ws[name] = torch.empty(fq.workspace_bytes(m, n, r, T), dtype=torch.uint8, device=dev)
            fq.workspace_init(self.ws[name])
        # saved for the backward, per block: h, h' and their row norms, g, u, and every projection's O_A (+ its amax)
        self.saved = [dict(g=torch.empty((T, F), dtype=bf, device=dev), u=torch.empty((T, F), dtype=bf, device=dev),
                           h=torch.empty((T, H), dtype=bf, device=dev), hp=torch.empty((T, H), dtype=bf, device=dev),
                           inv1=torch.empty(T, dtype=torch.float32, device=dev),
                           inv2=torch.empty(T, dtype=torch.float32, device=dev),
                           oa={p: torch.empty((T, r), dtype=torch.float32, device=dev) for p in PROJ},
                           amax={p: torch.empty(1, dtype=torch.float32, device=dev) for p in PROJ})
                      for _ in range(n_layers)]
        # transients, reused by every block
        e = lambda cols: torch.empty((T, cols), dtype=bf, device=dev)
        self.x1, self.x2 = e(H), e(H)
        self.q, self.kk, self.v, self.a, self.o, self.dn = e(H), e(H), e(H), e(H), e(H), e(H)
        self.h_out = e(H)
        self.z = e(F)
        self.dh, self.dhp, self.da, self.dqkv = e(H), e(H), e(H), e(H)
        self.dx = [e(H), e(H), e(H)]
        self.dz, self.dg, self.du, self.ddn = e(F), e(F), e(F), e(H)
        self.s_x = torch.empty(1, dtype=torch.float32, device=dev)
        self.s_g = torch.empty(1, dtype=torch.float32, device=dev)
        self.dB = {p: torch.empty((self.shapes[p][1], r), dtype=torch.float32, device=dev) for p in PROJ}
        self.idx = torch.empty(max(k, 1), dtype=torch.int32, device=dev)
        # one batched proxy update per block (its seven projections), or None: one call after every backward
        self.batches = None
        if batched_proxy:
            self.batches = [fq.ProxyBatch([self.layers[l][p] for p in PROJ], [self.dB[p] for p in PROJ], [k] * len(PROJ),
                                          wss=[self.ws[p] for p in PROJ], idx_outs=[None] * len(PROJ))
                            for l in range(n_layers)]
        if adamw is not None:   # first and second moments of every DeltaBuffer, zero before the first step
            z = lambda p: torch.zeros((self.shapes[p][1], r), dtype=torch.float32, device=dev)
            self.exp_avg = [[z(p) for p in PROJ] for _ in range(n_layers)]
            self.exp_avg_sq = [[z(p) for p in PROJ] for _ in range(n_layers)]
        # absmax words of the chain's outputs, one row per block: x1, a, x2, z | ddn, dg, du, dhp, dqkv (cleared every step)
        self.amax = torch.zeros((n_layers, 16), dtype=torch.float32, device=dev)
        self.capture = None   # optional: {(block, proj): dict} filled with references / copies for parity checks
        if fuse_cast:         # codes and scales of the chain's outputs (reused by every block) and the kernels' scratch
            u8e = lambda cols: torch.empty((T, cols), dtype=torch.uint8, device=dev)
            self.cq_H, self.cq_F, self.gq_H = u8e(H), u8e(F), u8e(H)
            self.cscale = torch.zeros(16, dtype=torch.float32, device=dev)
            self.cscratch = chain_scratch(dev)

    # ---- one linear: forward on X (quantizing it) or on another projection's codes
    def _am(self, l, slot):
        return self.amax[l, slot:slot + 1] if self.producer_amax else None

    def _fwd(self, l, name, X, Y, amax_x=None):
        sv = self.saved[l]
        fq.melded_forward(self.layers[l][name], X, ws=self.ws[name], out=(Y, sv["oa"][name], sv["amax"][name], self.s_x),
                          amax_x=amax_x)
        self._cap(l, name, X=X, Y=Y)

    def _fwd_shared(self, l, name, owner, X, Y):
        n, _ = self.shapes[name]
        lo = self.layers[l][owner]
        xq = fq.ws_view(lo, self.ws[owner], self.T, fq.WS_XQ)[: self.T * n].view(self.T, n)
        s_x = fq.ws_view(lo, self.ws[owner], self.T, fq.WS_SCALES).view(torch.float32)[1:2]
        sv = self.saved[l]
        fq.melded_forward_codes(self.layers[l][name], xq, s_x, ws=self.ws[name], out=(Y, sv["oa"][name], sv["amax"][name]))
        self._cap(l, name, X=X, Y=Y)

    def _bwd(self, l, name, dY, dX, amax_dy=None):
        sv = self.saved[l]
        fq.melded_backward(self.layers[l][name], dY, sv["oa"][name], sv["amax"][name], ws=self.ws[name],
                           out=(dX, self.dB[name], self.s_g), amax_dy=amax_dy)
        self._cap(l, name, dY=dY, dX=dX, dB=self.dB[name], OA=sv["oa"][name])
        if self.batches is None:
            fq.proxy_update(self.layers[l][name], self.dB[name], self.lr, self.k, ws=self.ws[name],
                            idx_out=self.idx if self.k > 0 else None)

    def _bwd_shared(self, l, name, owner, dY, dX):
        """The backward of a projection whose output gradient is the one `owner` has just cast (q, k and v all receive
        da / sqrt(3)): it multiplies the owner's codes instead of casting dY again."""
        m = self.shapes[name][1]
        lo = self.layers[l][owner]
        gq = fq.ws_view(lo, self.ws[owner], self.T, fq.WS_GQ)[: self.T * m].view(self.T, m)
        s_g = fq.ws_view(lo, self.ws[owner], self.T, fq.WS_SCALES).view(torch.float32)[3:4]
        sv = self.saved[l]
        fq.melded_backward_codes(self.layers[l][name], gq, s_g, sv["oa"][name], sv["amax"][name], ws=self.ws[name],
                                 out=(dX, self.dB[name]))
        self._cap(l, name, dY=dY, dX=dX, dB=self.dB[name], OA=sv["oa"][name])
        if self.batches is None:
            fq.proxy_update(self.layers[l][name], self.dB[name], self.lr, self.k, ws=self.ws[name],
                            idx_out=self.idx if self.k > 0 else None)

    def _sc(self, slot):
        return self.cscale[slot:slot + 1]

    def _fwd_codes(self, l, name, X16, xq, slot, Y):
        sv = self.saved[l]
        fq.melded_forward_codes(self.layers[l][name], xq, self._sc(slot), ws=self.ws[name], out=(Y, sv["oa"][name], sv["amax"][name]))
        self._cap(l, name, X=X16, Y=Y)

    def _bwd_codes(self, l, name, dY16, gq, slot, dX):
        sv = self.saved[l]
        fq.melded_backward_codes(self.layers[l][name], gq, self._sc(slot), sv["oa"][name], sv["amax"][name], ws=self.ws[name],
                                 out=(dX, self.dB[name]))
        self._cap(l, name, dY=dY16, dX=dX, dB=self.dB[name], OA=sv["oa"][name])
        if self.batches is None:
            fq.proxy_update(self.layers[l][name], self.dB[name], self.lr, self.k, ws=self.ws[name],
                            idx_out=self.idx if self.k > 0 else None)

    def _forward_fused_cast(self, h0):
        keep = self.capture is not None      # the bf16 tensors are only needed by the parity checks
        E4 = fq.E4M3
        for l in range(self.n_layers):
            sv = self.saved[l]
            if l == 0:
                sv["h"].copy_(h0)
                rmsnorm_quantize(self.cq_H, self._sc(0), E4, self.x1, keep, self.cscratch, sv["inv1"], sv["h"])
            h, hp = sv["h"], sv["hp"]
            self._fwd_codes(l, "q", self.x1, self.cq_H, 0, self.q)
            self._fwd_codes(l, "k", self.x1, self.cq_H, 0, self.kk)
            self._fwd_codes(l, "v", self.x1, self.cq_H, 0, self.v)
            combine_quantize(self.cq_H, self._sc(1), E4, self.a, keep, self.cscratch, self.q, INV_SQRT3, self.kk, INV_SQRT3,
                             self.v, INV_SQRT3)
            self._fwd_codes(l, "o", self.a, self.cq_H, 1, self.o)
            rmsnorm_quantize(self.cq_H, self._sc(2), E4, self.x2, keep, self.cscratch, sv["inv2"], h, sum_out=hp, sa=1.0, b=self.o,
                             sb=1.0)
            self._fwd_codes(l, "gate", self.x2, self.cq_H, 2, sv["g"])
            self._fwd_codes(l, "up", self.x2, self.cq_H, 2, sv["u"])
            silu_mul_quantize(self.cq_F, self._sc(3), E4, self.z, keep, self.cscratch, sv["g"], sv["u"])
            self._fwd_codes(l, "down", self.z, self.cq_F, 3, self.dn)
            if l + 1 < self.n_layers:
                nx = self.saved[l + 1]
                rmsnorm_quantize(self.cq_H, self._sc(0), E4, self.x1, keep, self.cscratch, nx["inv1"], hp, sum_out=nx["h"],
                                 sa=INV_SQRT2, b=self.dn, sb=INV_SQRT2)
            else:
                combine(self.h_out, hp, INV_SQRT2, self.dn, INV_SQRT2)
        return self.h_out

    def _backward_fused_cast(self, G):
        self.amax.zero_()
        keep = self.capture is not None
        E5 = fq.E5M2
        dh = G
        for l in reversed(range(self.n_layers)):
            sv = self.saved[l]
            combine_quantize(self.gq_H, self._sc(4), E5, self.ddn, keep, self.cscratch, dh, INV_SQRT2)
            self._bwd_codes(l, "down", self.ddn, self.gq_H, 4, self.dz)
            # dg and du (two [T][F] tensors at once) would mostly pass through memory between the two phases of a
            # quantizing kernel, which then loses to the plain kernel and two single-pass casts: these two stay separate
            silu_mul_grad(self.dg, self.du, sv["g"], sv["u"], self.dz, self.amax[l, 5:6], self.amax[l, 6:7])
            self._bwd(l, "gate", self.dg, self.dx[0], self.amax[l, 5:6])
            self._bwd(l, "up", self.du, self.dx[1], self.amax[l, 6:7])
            rmsnorm_grad_combine_quantize(self.gq_H, self._sc(7), E5, self.dhp, self.cscratch, [self.dx[0], self.dx[1]], sv["hp"],
                                          sv["inv2"], dh, INV_SQRT2)
            self._bwd_codes(l, "o", self.dhp, self.gq_H, 7, self.da)
            combine_quantize(self.gq_H, self._sc(8), E5, self.dqkv, keep, self.cscratch, self.da, INV_SQRT3)
            self._bwd_codes(l, "q", self.dqkv, self.gq_H, 8, self.dx[0])
            self._bwd_codes(l, "k", self.dqkv, self.gq_H, 8, self.dx[1])
            self._bwd_codes(l, "v", self.dqkv, self.gq_H, 8, self.dx[2])
            rmsnorm_grad_combine(self.dh, [self.dx[0], self.dx[1], self.dx[2]], sv["h"], sv["inv1"], self.dhp, 1.0)
            dh = self.dh
            self._run_batch(l)
        return dh

    def _run_batch(self, l):
        if self.batches is not None:
            if self.adamw is None:
                self.batches[l].run(self.lr)
            else:
                self.batches[l].run_adamw(self.exp_avg[l], self.exp_avg_sq[l], lr=self.lr, step=self.steps_done + 1, **self.adamw)

    def _cap(self, l, name, **tensors):
        if self.capture is not None and (l, name) in self.capture:
            self.capture[(l, name)].update({k2: v.clone() for k2, v in tensors.items()})

    def forward(self, h0: torch.Tensor) -> torch.Tensor:
        if self.fuse_cast:
            return self._forward_fused_cast(h0)
        if self.producer_amax:
            self.amax.zero_()
        for l in range(self.n_layers):
            sv = self.saved[l]
            if l == 0:
                sv["h"].copy_(h0)
            h, hp = sv["h"], sv["hp"]
            if l == 0 or not self.fuse_chain:      # (fused: the block before has already normalised its output into x1)
                rmsnorm(self.x1, sv["inv1"], h, amax=self._am(l, 0))
            self._fwd(l, "q", self.x1, self.q, self._am(l, 0))
            self._fwd_shared(l, "k", "q", self.x1, self.kk)
            self._fwd_shared(l, "v", "q", self.x1, self.v)
            combine(self.a, self.q, INV_SQRT3, self.kk, INV_SQRT3, self.v, INV_SQRT3, amax=self._am(l, 1))
            self._fwd(l, "o", self.a, self.o, self._am(l, 1))
            if self.fuse_chain:
                combine_rmsnorm(hp, self.x2, sv["inv2"], h, 1.0, self.o, 1.0, amax=self._am(l, 2))
            else:
                combine(hp, h, 1.0, self.o, 1.0)
                rmsnorm(self.x2, sv["inv2"], hp, amax=self._am(l, 2))
            self._fwd(l, "gate", self.x2, sv["g"], self._am(l, 2))
            self._fwd_shared(l, "up", "gate", self.x2, sv["u"])
            silu_mul(self.z, sv["g"], sv["u"], amax=self._am(l, 3))
            self._fwd(l, "down", self.z, self.dn, self._am(l, 3))
            out = self.saved[l + 1]["h"] if l + 1 < self.n_layers else self.h_out   # the next block's saved input
            if self.fuse_chain and l + 1 < self.n_layers:   # ... and, in the same pass, its first normalisation
                combine_rmsnorm(out, self.x1, self.saved[l + 1]["inv1"], hp, INV_SQRT2, self.dn, INV_SQRT2, amax=self._am(l + 1, 0))
            else:
                combine(out, hp, INV_SQRT2, self.dn, INV_SQRT2)
        return self.h_out

    def backward(self, G: torch.Tensor):
        """G = d loss / d h_last.  Each block's backward is followed at once by the proxy updates of its layers
        (one batched call, or inside _bwd), as in the paper's layer-wise training loop."""
        if self.fuse_cast:
            return self._backward_fused_cast(G)
        dh = G
        for l in reversed(range(self.n_layers)):
            sv = self.saved[l]
            combine(self.ddn, dh, INV_SQRT2, amax=self._am(l, 4))               # d(down output) = dh / sqrt(2)
            self._bwd(l, "down", self.ddn, self.dz, self._am(l, 4))
            silu_mul_grad(self.dg, self.du, sv["g"], sv["u"], self.dz, self._am(l, 5), self._am(l, 6))
            self._bwd(l, "gate", self.dg, self.dx[0], self._am(l, 5))
            self._bwd(l, "up", self.du, self.dx[1], self._am(l, 6))
            if self.fuse_chain:                                                 # dh' = dh/sqrt(2) + norm'(d x2), d x2 = the two dX
                rmsnorm_grad_combine(self.dhp, [self.dx[0], self.dx[1]], sv["hp"], sv["inv2"], dh, INV_SQRT2, amax=self._am(l, 7))
            else:
                combine(self.dx[0], self.dx[0], 1.0, self.dx[1], 1.0)               # d x2
                rmsnorm_grad(self.dx[1], self.dx[0], sv["hp"], sv["inv2"])
                combine(self.dhp, dh, INV_SQRT2, self.dx[1], 1.0, amax=self._am(l, 7))   # dh' = dh/sqrt(2) + norm'(d x2)
            self._bwd(l, "o", self.dhp, self.da, self._am(l, 7))
            combine(self.dqkv, self.da, INV_SQRT3, amax=self._am(l, 8))         # dq = dk = dv = da / sqrt(3)
            self._bwd(l, "q", self.dqkv, self.dx[0], self._am(l, 8))
            self._bwd_shared(l, "k", "q", self.dqkv, self.dx[1])       # the same gradient: q's codes serve all three
            self._bwd_shared(l, "v", "q", self.dqkv, self.dx[2])
            if self.fuse_chain:                                                 # dh = dh' + norm'(d x1), d x1 = the three dX
                rmsnorm_grad_combine(self.dh, [self.dx[0], self.dx[1], self.dx[2]], sv["h"], sv["inv1"], self.dhp, 1.0)
            else:
                combine(self.dx[0], self.dx[0], 1.0, self.dx[1], 1.0, self.dx[2], 1.0)   # d x1
                rmsnorm_grad(self.dx[1], self.dx[0], sv["h"], sv["inv1"])
                combine(self.dh, self.dhp, 1.0, self.dx[1], 1.0)
            dh = self.dh
            self._run_batch(l)
        return dh

    def step(self, h0: torch.Tensor, G: torch.Tensor):
        h = self.forward(h0)
        self.backward(G)
        self.steps_done += 1
        return h

    # ---- bookkeeping for the benchmark line
    def flops_per_step(self) -> float:
        T, r = self.T, self.r
        return float(self.n_layers * sum(2 * T * (n * (m + r) + m * n + m * r) for n, m in self.shapes.values()))

    def launches_per_step(self) -> int:
        if self.fuse_cast:
            # per block: 7 forward products; 7 dX products with the O_A cast and dB riding on them (each a kernel of its own
            # with own_db: + 2 per layer) + the two single-pass casts of dg and du; 4 + 5 chain kernels; the proxy update(s);
            # plus the first block's normalisation (the last block's plain residual sum stands in for a quantizing one)
            per_block = 7 + 7 * (3 if self.own_db else 1) + 2 + 4 + 5
            if self.batches is None:
                per_block += 7 * fq.launch_count("falqon_proxy_update", k=self.k)
            else:
                per_block += fq.launch_count("falqon_proxy_update_batched", k=self.k)
            return per_block * self.n_layers + 1
        per_block = 0
        for name in PROJ:
            shared = name in ("k", "v", "up")
            per_block += (1 if shared else fq.launch_count("falqon_melded_forward"))   # codes: the product alone
            if name in ("k", "v"):
                per_block += 3 if self.own_db else 1            # on q's gradient codes: dX, with the O_A cast and dB riding on it
            else:                                               # cast, dX (with own_db: + dB, + the O_A cast after a single-pass cast)
                per_block += fq.launch_count("falqon_melded_backward" + (":own_db" if self.own_db else "")) + (1 if self.producer_amax and self.own_db else 0)
            if self.batches is None:
                per_block += fq.launch_count("falqon_proxy_update", k=self.k)
        if self.batches is not None:
            per_block += fq.launch_count("falqon_proxy_update_batched", k=self.k)
        per_block += 6 + 9   # chain kernels: forward 6 (2 norms, mix, 2 residuals, gate), backward 9
        total = per_block * self.n_layers
        if self.fuse_chain:  # per block 2 residual + norm pairs in one launch each (the last block keeps its plain residual, the
            total -= self.n_layers * (2 + 4) - 1   # first its plain norm) and 2 x (sum, norm gradient, residual) in one each
        return total

    def bytes_resident(self) -> int:
        tot = 0
        for block in self.layers:
            for L in block.values():
                tot += L.wq.numel() + 4 * L.s_w.numel() + 4 * L.dbuf.numel()
        return tot
