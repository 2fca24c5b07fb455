"""GPU parity of the fused casts (FALQON_LAYER_FUSED_CAST): the products whose producers cast X / dY themselves.

Two things are established, through the C ABI:
  * identical FP8 operands -- the codes every column block of the fused products stages in shared memory, written out
    by the debug hook, equal the oracle's cast of the same tensor byte for byte (and the scales bit for bit);
  * identical results -- Y, O_A, amax(O_A), dX and dB of the fused calls equal those of the un-fused calls bit for
    bit (same codes, same tile schedule, same MMA order), so every oracle comparison of the un-fused path carries over.
"""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, layer_inputs, u8
from paper_2510_24061_b200 import synth

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


def _twin(fq, layer, flags):
    """A second host struct over the same device tensors with other flags."""
    return fq.Layer(layer.wq, layer.s_w, layer.dbuf, layer.r, flags=flags)


SHAPES = [
    # (m, n, r, T, outliers, all_blocks)
    (1024, 1024, 16, 512, 8, True),          # configs[0]
    (400, 272, 16, 333, 3, True),            # ragged in T, K and N; two row tiles, one partial
    (272, 1040, 32, 700, 5, True),           # K tail of 16, N = 304: a narrow last column block
    (4096, 4096, 64, 4096, 41, False),       # configs[1]: q
    (11008, 4096, 64, 4096, 41, False),      # configs[1]: gate / up
    (4096, 11008, 64, 4096, 110, False),     # configs[1]: down
]


@pytest.mark.parametrize("m,n,r,T,outl,all_blocks", SHAPES)
def test_fused_forward_and_backward_match_unfused_and_oracle_codes(fq, orc, m, n, r, T, outl, all_blocks):
    W, A, B, X = layer_inputs(11, 2, m, n, r, T, outl, DEV)
    dY = synth.out_grad(11, 2, 0, T, m, DEV)
    plain = fq.setup_layer(W, A, B, 1.0)
    plain.flags = fq.LAYER_DB_OWN_KERNEL    # the fused backward runs dB as a kernel of its own: the reference does the same
    fused = _twin(fq, plain, fq.LAYER_FUSED_CAST)
    ws = plain.workspace(T)

    # ---- forward: un-fused reference run, then the fused one
    Y0, OA0, amax0, sx0 = fq.melded_forward(plain, X, y_dtype=torch.float32, ws=ws)
    xq0 = fq.ws_view(plain, ws, T, fq.WS_XQ).clone()
    Y1, OA1, amax1, sx1 = fq.melded_forward(fused, X, y_dtype=torch.float32, ws=ws)
    assert torch.equal(sx0, sx1) and torch.equal(amax0, amax1)
    assert torch.equal(Y0.view(torch.int32), Y1.view(torch.int32)), "fused Y differs from un-fused Y"
    assert torch.equal(OA0.view(torch.int32), OA1.view(torch.int32)), "fused O_A differs"
    # known absmax: no reduction pass at all
    amax_x = X.float().abs().max().reshape(1)
    Y2, OA2, amax2, sx2 = fq.melded_forward(fused, X, y_dtype=torch.float32, ws=ws, amax_x=amax_x)
    assert torch.equal(sx0, sx2) and torch.equal(Y0.view(torch.int32), Y2.view(torch.int32))
    assert torch.equal(OA0.view(torch.int32), OA2.view(torch.int32)) and torch.equal(amax0, amax2)
    # bf16 output: the rounding of the same fp32 values
    Yb0, _, _, _ = fq.melded_forward(plain, X, y_dtype=torch.bfloat16, ws=ws)
    Yb1, _, _, _ = fq.melded_forward(fused, X, y_dtype=torch.bfloat16, ws=ws)
    assert torch.equal(Yb0.view(torch.int16), Yb1.view(torch.int16))

    # ---- identical operands: the oracle's cast of X against what each column block staged
    xq_o, sx_o, _ = orc.quantize(f32(X), orc.E4M3)
    assert bits32(f32(sx1))[0] == bits32(sx_o)
    xq_o_dev = torch.from_numpy(xq_o).to(DEV).reshape(-1)
    assert torch.equal(xq0, xq_o_dev)
    n_blocks = (m + r + 255) // 256
    blocks = range(n_blocks) if all_blocks else sorted({0, 1, n_blocks // 2, n_blocks - 1})
    for nb in blocks:
        region = fq.ws_view(plain, ws, T, fq.WS_XQ)
        region.fill_(0xAA)
        Yd, OAd, _, _ = fq.melded_forward_dump(fused, X, nb, ws=ws)
        assert torch.equal(region, xq_o_dev), f"staged codes of column block {nb} differ from the oracle's cast"
        assert torch.equal(Yd.view(torch.int32), Y0.view(torch.int32))

    # ---- backward
    dX0, dB0, sg0 = fq.melded_backward(plain, dY, OA0, amax0, dx_dtype=torch.float32, ws=ws)
    gq0 = fq.ws_view(plain, ws, T, fq.WS_GQ).clone()
    fq.ws_view(plain, ws, T, fq.WS_GQ).fill_(0x55)
    dX1, dB1, sg1 = fq.melded_backward(fused, dY, OA0, amax0, dx_dtype=torch.float32, ws=ws)
    assert torch.equal(sg0, sg1)
    assert torch.equal(dX0.view(torch.int32), dX1.view(torch.int32)), "fused dX differs from un-fused dX"
    assert torch.equal(dB0.view(torch.int32), dB1.view(torch.int32)), "dB after the fused dX differs"
    gq_o, sg_o, _ = orc.quantize(f32(dY), orc.E5M2)
    assert bits32(f32(sg1))[0] == bits32(sg_o)
    gq_o_dev = torch.from_numpy(gq_o).to(DEV).reshape(-1)
    assert torch.equal(gq0, gq_o_dev)
    assert torch.equal(fq.ws_view(plain, ws, T, fq.WS_GQ), gq_o_dev), "g~ written by the fused dX differs from the oracle's cast"
    amax_dy = dY.float().abs().max().reshape(1)
    dX2, dB2, sg2 = fq.melded_backward(fused, dY, OA0, amax0, dx_dtype=torch.float32, ws=ws, amax_dy=amax_dy)
    assert torch.equal(sg0, sg2) and torch.equal(dX0.view(torch.int32), dX2.view(torch.int32))
    assert torch.equal(dB0.view(torch.int32), dB2.view(torch.int32))
    n_blocks = (n + 255) // 256
    blocks = range(n_blocks) if all_blocks else sorted({0, 1, n_blocks // 2, n_blocks - 1})
    for nb in blocks:
        region = fq.ws_view(plain, ws, T, fq.WS_GQ)
        region.fill_(0xAA)
        dXd, dBd, _ = fq.melded_backward_dump(fused, dY, OA0, amax0, nb, ws=ws)
        assert torch.equal(region, gq_o_dev), f"staged gradient codes of column block {nb} differ from the oracle's cast"
        assert torch.equal(dXd.view(torch.int32), dX0.view(torch.int32)) and torch.equal(dBd.view(torch.int32), dB0.view(torch.int32))
    assert fq.last_device_status() == 0


def test_fused_flag_falls_back_where_the_kernel_does_not_apply(fq, orc):
    """fp32 inputs, (m + r) not a multiple of 16, per-row scales, dX not requested: the flag is accepted and the
    un-fused path runs (same results, codes in the workspace); the dump hook reports FALQON_ERR_UNSUPPORTED."""
    m, n, r, T = 272, 256, 16, 100     # the product shape is fine, but the input is fp32
    W, A, B, X = layer_inputs(12, 0, m, n, r, T, 2, DEV)
    plain = fq.setup_layer(W, A, B, 1.0)
    fused = _twin(fq, plain, fq.LAYER_FUSED_CAST)
    ws = plain.workspace(T)
    Xf = X.float()
    Y0, OA0, amax0, _ = fq.melded_forward(plain, Xf, y_dtype=torch.float32, ws=ws)
    Y1, OA1, _, _ = fq.melded_forward(fused, Xf, y_dtype=torch.float32, ws=ws)
    assert torch.equal(Y0, Y1) and torch.equal(OA0, OA1)
    with pytest.raises(fq.FalqonError) as e:
        fq.melded_forward_dump(fused, Xf, 0, ws=ws)
    assert e.value.status == fq.ERR_UNSUPPORTED
    # rank 8 on m = 256: m + r = 264 is not a multiple of 16
    W, A, B, X = layer_inputs(12, 1, 256, 256, 8, T, 2, DEV)
    plain = fq.setup_layer(W, A, B, 1.0)
    fused = _twin(fq, plain, fq.LAYER_FUSED_CAST)
    ws = plain.workspace(T)
    Y0, OA0, amax0, _ = fq.melded_forward(plain, X, y_dtype=torch.float32, ws=ws)
    Y1, OA1, _, _ = fq.melded_forward(fused, X, y_dtype=torch.float32, ws=ws)
    assert torch.equal(Y0, Y1) and torch.equal(OA0, OA1)
    # backward without dX: nothing to fuse the cast into
    dY = synth.out_grad(12, 1, 0, T, 256, DEV)
    _, dB0, _ = fq.melded_backward(plain, dY, OA0, amax0, need_dx=False, ws=ws)
    _, dB1, _ = fq.melded_backward(fused, dY, OA0, amax0, need_dx=False, ws=ws)
    assert torch.equal(dB0, dB1)
    # a dump block beyond the product is an argument error; unknown flag bits are rejected
    W, A, B, X = layer_inputs(12, 2, 256, 256, 16, T, 2, DEV)
    plain = fq.setup_layer(W, A, B, 1.0)
    fused = _twin(fq, plain, fq.LAYER_FUSED_CAST)
    with pytest.raises(fq.FalqonError) as e:
        fq.melded_forward_dump(fused, X, 2, ws=plain.workspace(T))
    assert e.value.status == fq.ERR_INVALID_ARG
    bad = _twin(fq, plain, 64)
    with pytest.raises(fq.FalqonError) as e:
        fq.melded_forward(bad, X, ws=plain.workspace(T))
    assert e.value.status == fq.ERR_INVALID_ARG
    assert fq.last_device_status() == 0


def test_fused_forward_emits_shared_codes(fq, orc):
    """FALQON_LAYER_EMIT_XQ: the fused forward leaves x~ in the workspace for the layers that share it."""
    m, n, r, T = 512, 768, 32, 600
    W, A, B, X = layer_inputs(13, 0, m, n, r, T, 6, DEV)
    plain = fq.setup_layer(W, A, B, 1.0)
    fused = _twin(fq, plain, fq.LAYER_FUSED_CAST | fq.LAYER_EMIT_XQ)
    ws = plain.workspace(T)
    fq.ws_view(plain, ws, T, fq.WS_XQ).fill_(0xAA)
    Y1, OA1, amax1, sx1 = fq.melded_forward(fused, X, y_dtype=torch.float32, ws=ws)
    xq = fq.ws_view(plain, ws, T, fq.WS_XQ).clone().reshape(T, n)
    xq_o, _, _ = orc.quantize(f32(X), orc.E4M3)
    assert np.array_equal(u8(xq), xq_o)
    Y2, OA2, amax2 = fq.melded_forward_codes(plain, xq, sx1, y_dtype=torch.float32, ws=ws)
    assert torch.equal(Y1, Y2) and torch.equal(OA1, OA2) and torch.equal(amax1, amax2)
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("amax", [448.0, 448.0 / 3.7, 57344.0, 1.0e-3])
def test_fused_converters_on_every_bf16_value(fq, orc, amax):
    """The converters' cast (packed multiply, cvt.rn.satfinite, in-place swizzled store) on ALL finite bf16 inputs: a
    [512][128] activation tensor that holds every bit pattern once, cast with a given absmax (scale 1, an odd scale, a tiny
    one that underflows most values, a huge one that saturates many), dumped and compared with the oracle's cast; the same
    values as an output gradient through the input-gradient product's E5M2 converters."""
    bits = torch.arange(1 << 16, dtype=torch.int32).to(torch.int16).view(torch.bfloat16).reshape(512, 128)
    X = torch.where(torch.isfinite(bits.float()), bits, torch.zeros_like(bits)).to(DEV)
    T, n, m, r = 512, 128, 240, 16
    W, A, B, _ = layer_inputs(14, 0, m, n, r, 16, 0, DEV)
    layer = fq.setup_layer(W, A, B, 1.0)
    layer.flags = fq.LAYER_FUSED_CAST
    ws = layer.workspace(T)
    am = torch.tensor([amax], dtype=torch.float32, device=DEV)
    s = np.float32(448.0) / np.float32(amax)
    fq.ws_view(layer, ws, T, fq.WS_XQ).fill_(0xAA)
    _, _, _, s_x = fq.melded_forward_dump(layer, X, 0, ws=ws, amax_x=am)
    assert bits32(f32(s_x))[0] == bits32(s)
    want, _, _ = orc.quantize(f32(X), orc.E4M3, scale_in=s)
    assert np.array_equal(u8(fq.ws_view(layer, ws, T, fq.WS_XQ)).reshape(T, n), want)
    # E5M2: the same patterns as dY of a layer with m = 128 outputs
    m2, n2 = 128, 256
    W2, A2, B2, X2 = layer_inputs(14, 1, m2, n2, r, T, 2, DEV)
    back = fq.setup_layer(W2, A2, B2, 1.0)
    back.flags = fq.LAYER_FUSED_CAST
    ws2 = back.workspace(T)
    _, OA, amax_oa, _ = fq.melded_forward(back, X2, ws=ws2)
    s5 = np.float32(57344.0) / np.float32(amax)
    fq.ws_view(back, ws2, T, fq.WS_GQ).fill_(0xAA)
    fq.melded_backward_dump(back, X, OA, amax_oa, 0, ws=ws2, amax_dy=am)
    want5, _, _ = orc.quantize(f32(X), orc.E5M2, scale_in=s5)
    assert np.array_equal(u8(fq.ws_view(back, ws2, T, fq.WS_GQ)).reshape(T, m2), want5)
    assert fq.last_device_status() == 0
