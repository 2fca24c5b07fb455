"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, stage by stage.

Each stage is teacher-forced: the oracle is fed the GPU's actual inputs of that stage, so the
comparison isolates the stage.  Casts, scales, scores, top-k indices and merged rows must match bit
for bit; tensor-core products must be within 2e-5 relative Frobenius error of the oracle's
fp64-accumulated product of the identical FP8 operand bytes, taken on fp32 outputs.
"""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, layer_inputs, product_close, rel_fro, u8
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu

GEMM_TOL = 2e-5  # relative Frobenius error bound on tensor-core outputs


@pytest.fixture(scope="module")
def fq():
    from paper_2510_24061_b200 import binding
    return binding


@pytest.fixture(scope="module")
def orc():
    from oracle import falqon_oracle
    return falqon_oracle


DEV = "cuda:0"


# ------------------------------------------------------------------ quantizer (S1 / S3 / S0)

@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("shape,dtype", [((512, 1024), torch.bfloat16), ((37, 48), torch.float32),
                                         ((1, 16), torch.float32), ((1500, 4112), torch.bfloat16)])
def test_quantize_per_tensor_bit_exact(fq, orc, fmt, shape, dtype):
    x = synth.activations(5, 1, shape[0], shape[1], 4).to(dtype)
    codes, scale, amax = fq.quantize(x.to(DEV), fmt)
    q, s, a = orc.quantize(f32(x), fmt)
    assert bits32(f32(amax))[0] == bits32(a) and bits32(f32(scale))[0] == bits32(s)
    assert np.array_equal(u8(codes), q)
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("fmt", [0, 1])
def test_cast_exhaustive_bf16_and_fp32_sample(fq, orc, fmt):
    one = torch.ones(1, dtype=torch.float32, device=DEV)
    bits = torch.arange(1 << 16, dtype=torch.int32).to(torch.int16).view(torch.bfloat16).reshape(4096, 16)
    finite = torch.isfinite(bits.float())
    x = torch.where(finite, bits, torch.zeros_like(bits))
    codes, _, _ = fq.quantize(x.to(DEV), fmt, scale_in=one, want_amax=False)
    assert np.array_equal(u8(codes), orc.encode_array(f32(x), fmt))
    # every 64th fp32 bit pattern (2^26 values), NaN/inf replaced by 0
    raw = (torch.arange(1 << 26, dtype=torch.int64) * 64 + 17).to(torch.int32).view(torch.float32)
    raw = torch.where(torch.isfinite(raw), raw, torch.zeros_like(raw)).reshape(1 << 14, 1 << 12)
    codes, _, _ = fq.quantize(raw.to(DEV), fmt, scale_in=one, want_amax=False)
    assert np.array_equal(u8(codes), orc.encode_array(raw.numpy(), fmt))


def test_quantize_given_scale_premul_and_per_row(fq, orc):
    a = synth.adapter_a(3, 0, 16, 1024)
    s_w = torch.tensor([4611.5], dtype=torch.float32)
    codes, _, _ = fq.quantize(a.to(DEV), 0, scale_in=s_w.to(DEV), premul=2.0, want_amax=False)
    q, _, _ = orc.quantize(f32(a), 0, scale_in=s_w.numpy(), premul=2.0)
    assert np.array_equal(u8(codes), q)
    w = synth.student_t3_bf16(3, 1, (96, 272), 0.02)
    codes, scale, amax = fq.quantize(w.to(DEV), 0, gran=fq.PER_ROW)
    q, s, am = orc.quantize(f32(w), 0, gran=orc.PER_ROW)
    assert np.array_equal(bits32(f32(scale)), bits32(s)) and np.array_equal(bits32(f32(amax)), bits32(am))
    assert np.array_equal(u8(codes), q)


# ------------------------------------------------------------------ one layer, all stages

def _run_layer_stages(fq, orc, seed, m, n, r, T, k, gamma, n_outliers, steps, lr, y_dtype=torch.float32,
                      per_row=False, heavy_tailed=False):
    W, A, B, X = layer_inputs(seed, 0, m, n, r, T, n_outliers)
    if heavy_tailed:
        W = synth.backbone(seed, 0, m, n, heavy_tailed=True)
    # S0: set-up (quantize W, A; meld B over all rows)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), gamma, per_row=per_row)
    wq_o, s_w_o, dbuf_o = orc.setup_layer(f32(W), f32(A), f32(B), gamma, per_row=per_row)
    assert np.array_equal(bits32(f32(layer.s_w)), bits32(np.atleast_1d(s_w_o)))
    s_w_g = f32(layer.s_w) if per_row else np.float32(f32(layer.s_w)[0])
    row_scales = s_w_g if per_row else None
    assert np.array_equal(u8(layer.wq), wq_o), "melded backbone codes differ after set-up"
    assert not f32(layer.dbuf).any()
    ws = layer.workspace(T)
    Xd = X.to(DEV)
    for step in range(steps):
        # ---- forward
        Y, OA, amax_oa, s_x = fq.melded_forward(layer, Xd, y_dtype=y_dtype, ws=ws)
        xq_g = u8(fq.ws_view(layer, ws, T, fq.WS_XQ)).reshape(T, n)
        xq_o, s_x_o, _ = orc.quantize(f32(X), orc.E4M3)
        assert bits32(f32(s_x))[0] == bits32(s_x_o) and np.array_equal(xq_g, xq_o)
        wq_now = u8(layer.wq)
        Y_o, OA_o, _ = orc.forward(xq_g, np.float32(f32(s_x)[0]), wq_now, s_w_g, m, r)
        OA_g = f32(OA)
        assert product_close(f32(Y), Y_o, GEMM_TOL), f"Y step {step}"
        assert product_close(OA_g, OA_o, GEMM_TOL), f"OA step {step}"
        assert bits32(f32(amax_oa))[0] == bits32(np.abs(OA_g).max())
        # ---- backward
        dY = synth.out_grad(seed, 0, step, T, m)
        dX, dB, s_g = fq.melded_backward(layer, dY.to(DEV), OA, amax_oa, dx_dtype=torch.float32, ws=ws)
        gq_g = u8(fq.ws_view(layer, ws, T, fq.WS_GQ)).reshape(T, m)
        if per_row:
            gq_o, s_g_o, _ = orc.quantize_colscaled(f32(dY), orc.E5M2, s_w_g[:m])
        else:
            gq_o, s_g_o, _ = orc.quantize(f32(dY), orc.E5M2)
        assert bits32(f32(s_g))[0] == bits32(s_g_o) and np.array_equal(gq_g, gq_o)
        oaq_o, s_oa_o, _ = orc.quantize(OA_g, orc.E4M3)
        scales = f32(fq.ws_view(layer, ws, T, fq.WS_SCALES).view(torch.float32))
        assert bits32(scales[5]) == bits32(s_oa_o)
        r16, t16 = (r + 15) // 16 * 16, (T + 15) // 16 * 16
        oaq_t = u8(fq.ws_view(layer, ws, T, fq.WS_OAQ_T)).reshape(r16, t16)
        assert np.array_equal(oaq_t[:r, :T].T, oaq_o)
        dX_o = orc.dx_gemm(gq_g, s_g_o, wq_now, s_w_g, m)
        dB_o = orc.db_gemm(gq_g, s_g_o, oaq_o, s_oa_o, row_scale=s_w_g[:m] if per_row else None)
        assert product_close(f32(dX), dX_o, GEMM_TOL), f"dX step {step}"
        assert product_close(f32(dB), dB_o, GEMM_TOL), f"dB step {step}"
        # ---- proxy update, fed the GPU's own dB
        dbuf_o = f32(layer.dbuf).copy()
        wq_o2 = wq_now.copy()
        idx = fq.proxy_update(layer, dB, lr, k, ws=ws)
        idx_o, score_o = orc.proxy_update(wq_o2, dbuf_o, f32(dB), lr, k, m, r, row_scales=row_scales)
        score_g = f32(fq.ws_view(layer, ws, T, fq.WS_SCORE).view(torch.float32))
        assert np.array_equal(bits32(score_g), bits32(score_o)), f"scores step {step}"
        if k > 0:
            assert np.array_equal(u8(idx), idx_o), f"top-k step {step}"
        assert np.array_equal(u8(layer.wq), wq_o2), f"merged rows step {step}"
        assert np.array_equal(bits32(f32(layer.dbuf)), bits32(dbuf_o)), f"DeltaBuffer step {step}"
    assert fq.last_device_status() == 0
    return layer


@pytest.mark.parametrize("lr", [2e-4, 2e-2, 2e-1])
def test_config0_three_steps_all_stages(fq, orc, lr):
    c = synth.config0()
    _run_layer_stages(fq, orc, c["seed"], c["m"], c["n"], c["r"], c["T"], c["k"], c["alpha"] / c["r"],
                      c["n_outliers"], c["steps"], lr)


@pytest.mark.parametrize("m,n,r,T,k", [(272, 208, 8, 200, 5), (128, 128, 16, 128, 0), (144, 400, 24, 77, 144),
                                       (1040, 528, 72, 333, 1), (256, 1024, 128, 640, 31), (512, 256, 256, 130, 512)])
def test_ragged_and_edge_shapes(fq, orc, m, n, r, T, k):
    _run_layer_stages(fq, orc, 11, m, n, r, T, k, 1.0, 3, 2, 2e-2)


@pytest.mark.parametrize("m,n,r,T,k", [(1024, 768, 16, 512, 32), (272, 208, 8, 200, 272), (640, 1280, 64, 300, 17)])
def test_per_row_scaled_backbone_all_stages(fq, orc, m, n, r, T, k):
    """Heavy-tailed backbone rows (Student-t, 3 degrees of freedom) with one scale per row."""
    _run_layer_stages(fq, orc, 13, m, n, r, T, k, 1.0, 4, 2, 2e-2, per_row=True, heavy_tailed=True)


@pytest.mark.parametrize("m,n,r,T,k", [(3840, 1024, 64, 1280, 64), (1024, 3872, 64, 1200, 16)])
def test_more_tiles_than_cta_pairs_all_stages(fq, orc, m, n, r, T, k):
    """80 output tiles for 74 CTA pairs, element by element: the forward product (first shape) and the
    input-gradient product (second shape, with a ragged last tile row and column) give some pairs two tiles."""
    _run_layer_stages(fq, orc, 29, m, n, r, T, k, 1.0, 3, 2, 2e-2)


@pytest.mark.parametrize("T", [1, 5, 17])
def test_a_handful_of_tokens(fq, orc, T):
    """Fewer tokens than one tile row, than one 16-byte vector of codes, than one k-block of the adapter gradient."""
    _run_layer_stages(fq, orc, 37, 272, 208, 24, T, 9, 1.0, 2, 2, 2e-2)


@pytest.mark.parametrize("per_row", [False, True])
def test_fp32_inputs_larger_than_the_staging_ring(fq, orc, per_row):
    """fp32 activations and output gradients of 49 MB each: more than the fused quantizer keeps on chip, so part
    of the tensor is fetched a second time for the cast; the last 16 KB chunk is partial.  Codes and scales
    must match bit for bit (per-row mode: the gradient is divided by the row scales before its cast)."""
    T, big, small, r = 3001, 4112, 128, 16
    # forward: X is [T][big]
    W, A, B, _ = layer_inputs(31, 0, small, big, r, 16, 0)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0, per_row=per_row)
    X = synth.normal_bf16(31, 7, (T, big), 1.0).float() * 1.0009765625 + 3.0e-4   # not bf16-representable
    ws = layer.workspace(T)
    _, _, _, s_x = fq.melded_forward(layer, X.to(DEV), y_dtype=torch.float32, ws=ws)
    xq_o, s_x_o, _ = orc.quantize(f32(X), orc.E4M3)
    assert bits32(f32(s_x))[0] == bits32(s_x_o)
    assert np.array_equal(u8(fq.ws_view(layer, ws, T, fq.WS_XQ)).reshape(T, big), xq_o)
    # backward: dY is [T][big]
    W, A, B, X2 = layer_inputs(32, 0, big, small, r, T, 0)
    if per_row:
        W = synth.backbone(32, 0, big, small, heavy_tailed=True)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0, per_row=per_row)
    ws = layer.workspace(T)
    _, OA, amax_oa, _ = fq.melded_forward(layer, X2.to(DEV), y_dtype=torch.float32, ws=ws)
    dY = synth.normal_bf16(32, 9, (T, big), 1.0e-3).float() * 0.99951171875 - 1.0e-7
    _, _, s_g = fq.melded_backward(layer, dY.to(DEV), OA, amax_oa, dx_dtype=torch.float32, ws=ws)
    if per_row:
        gq_o, s_g_o, _ = orc.quantize_colscaled(f32(dY), orc.E5M2, f32(layer.s_w)[:big])
    else:
        gq_o, s_g_o, _ = orc.quantize(f32(dY), orc.E5M2)
    assert bits32(f32(s_g))[0] == bits32(s_g_o)
    assert np.array_equal(u8(fq.ws_view(layer, ws, T, fq.WS_GQ)).reshape(T, big), gq_o)
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("per_row", [False, True])
def test_many_steps_keep_every_stage_fresh(fq, orc, per_row):
    """Twenty-five steps with a new output gradient each: every kernel overlaps the launch of the next one, so a
    stage that read anything stale (a scale, a slab, a score from the step before) would show up here."""
    _run_layer_stages(fq, orc, 23, 640, 1280, 64, 300, 17, 1.0, 4, 25, 2e-2, per_row=per_row, heavy_tailed=per_row)


def test_bf16_outputs_are_rounded_fp32_outputs(fq):
    c = synth.config0()
    W, A, B, X = layer_inputs(0, 0, c["m"], c["n"], c["r"], c["T"], c["n_outliers"])
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 2.0)
    Y32, OA, amax_oa, _ = fq.melded_forward(layer, X.to(DEV), y_dtype=torch.float32)
    Y16, OA2, _, _ = fq.melded_forward(layer, X.to(DEV), y_dtype=torch.bfloat16)
    assert torch.equal(Y32.to(torch.bfloat16), Y16) and torch.equal(OA, OA2)
    dY = synth.out_grad(0, 0, 0, c["T"], c["m"]).to(DEV)
    dX32, dB, _ = fq.melded_backward(layer, dY, OA, amax_oa, dx_dtype=torch.float32)
    dX16, dB2, _ = fq.melded_backward(layer, dY, OA, amax_oa, dx_dtype=torch.bfloat16)
    assert torch.equal(dX32.to(torch.bfloat16), dX16) and torch.equal(dB, dB2)   # run-to-run deterministic
    # without dX there is no product for dB to ride on: it runs as a kernel of its own, which sums four token slabs instead
    # of accumulating over all tokens in one go -- the same numbers up to the order of the fp32 sums; with
    # LAYER_DB_OWN_KERNEL the call with dX uses that kernel too, and then the two agree bit for bit
    _, dB3, _ = fq.melded_backward(layer, dY, OA, amax_oa, need_dx=False)
    assert float((dB - dB3).abs().max()) <= 2e-6 * float(dB.abs().max())
    layer.flags = fq.LAYER_DB_OWN_KERNEL
    dX32b, dB4, _ = fq.melded_backward(layer, dY, OA, amax_oa, dx_dtype=torch.float32)
    assert torch.equal(dB4, dB3) and torch.equal(dX32b, dX32)


@pytest.mark.parametrize("per_row", [False, True])
def test_forward_on_shared_codes_equals_forward(fq, per_row):
    """Two layers that read the same activations (q and k of a block): the second one takes the first one's x~ and
    s_x from its workspace and must produce what a forward of its own on X produces, bit for bit."""
    m, n, r, T = 640, 1280, 64, 300
    W1, A1, B1, X = layer_inputs(41, 0, m, n, r, T, 4)
    W2, A2, B2, _ = layer_inputs(41, 1, m, n, r, T, 4)
    first = fq.setup_layer(W1.to(DEV), A1.to(DEV), B1.to(DEV), 1.0, per_row=per_row)
    second = fq.setup_layer(W2.to(DEV), A2.to(DEV), B2.to(DEV), 1.0, per_row=per_row)
    ws1, ws2 = first.workspace(T), second.workspace(T)
    fq.melded_forward(first, X.to(DEV), y_dtype=torch.float32, ws=ws1)
    xq = fq.ws_view(first, ws1, T, fq.WS_XQ)[:T * n].reshape(T, n)
    s_x = fq.ws_view(first, ws1, T, fq.WS_SCALES).view(torch.float32)[1:2]
    Y_c, OA_c, amax_c = fq.melded_forward_codes(second, xq, s_x, y_dtype=torch.float32, ws=ws2)
    Y, OA, amax, _ = fq.melded_forward(second, X.to(DEV), y_dtype=torch.float32, ws=ws2)
    assert torch.equal(Y_c, Y) and torch.equal(OA_c, OA) and torch.equal(amax_c, amax)
    assert fq.last_device_status() == 0


def test_known_absmax_variants_equal_the_plain_calls(fq):
    """A caller that knows max |X| and max |dY| gets single-pass casts; every output must equal the plain calls' bit for
    bit (same scale, same codes, same products).  Per-row layers reject the backward variant."""
    m, n, r, T = 640, 1280, 64, 300
    W, A, B, X = layer_inputs(43, 0, m, n, r, T, 4)
    dY = synth.out_grad(43, 0, 0, T, m).to(DEV)
    Xd = X.to(DEV)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0)
    ws = layer.workspace(T)
    Y, OA, amax_oa, s_x = [t.clone() for t in fq.melded_forward(layer, Xd, y_dtype=torch.float32, ws=ws)]
    xq = fq.ws_view(layer, ws, T, fq.WS_XQ).clone()
    dX, dB, s_g = [t.clone() for t in fq.melded_backward(layer, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)]
    gq = fq.ws_view(layer, ws, T, fq.WS_GQ).clone()
    oaq = fq.ws_view(layer, ws, T, fq.WS_OAQ_T).clone()
    ws2 = torch.empty_like(ws)
    fq.workspace_init(ws2)
    Y2, OA2, amax2, s_x2 = fq.melded_forward(layer, Xd, y_dtype=torch.float32, ws=ws2, amax_x=Xd.float().abs().max().reshape(1))
    assert torch.equal(fq.ws_view(layer, ws2, T, fq.WS_XQ), xq) and torch.equal(s_x2, s_x)
    assert torch.equal(Y2, Y) and torch.equal(OA2, OA) and torch.equal(amax2, amax_oa)
    dX2, dB2, s_g2 = fq.melded_backward(layer, dY, OA2, amax2, dx_dtype=torch.float32, ws=ws2,
                                        amax_dy=dY.float().abs().max().reshape(1))
    assert torch.equal(fq.ws_view(layer, ws2, T, fq.WS_GQ), gq) and torch.equal(s_g2, s_g)
    assert torch.equal(fq.ws_view(layer, ws2, T, fq.WS_OAQ_T)[: r * ((T + 15) // 16 * 16)], oaq[: r * ((T + 15) // 16 * 16)])
    assert torch.equal(dX2, dX) and torch.equal(dB2, dB)
    per_row = fq.setup_layer(W.to(DEV), A.to(DEV), None, 1.0, per_row=True)
    with pytest.raises(fq.FalqonError):
        fq.melded_backward(per_row, dY, OA, amax_oa, amax_dy=dY.float().abs().max().reshape(1))
    assert fq.last_device_status() == 0


def test_b_zero_leaves_plain_fp8_layer(fq):
    c = synth.config0()
    W, A, _, X = layer_inputs(0, 0, c["m"], c["n"], c["r"], c["T"], c["n_outliers"])
    Wd, Ad = W.to(DEV), A.to(DEV)
    plain = fq.setup_layer(Wd, Ad, None, 2.0)
    melded = fq.setup_layer(Wd, Ad, torch.zeros(c["m"], c["r"], device=DEV), 2.0)
    assert torch.equal(plain.wq, melded.wq)
    Y0, _, _, _ = fq.melded_forward(plain, X.to(DEV), y_dtype=torch.float32)
    Y1, _, _, _ = fq.melded_forward(melded, X.to(DEV), y_dtype=torch.float32)
    assert torch.equal(Y0, Y1)


def test_topk_ties_go_to_lowest_index(fq, orc):
    m, n, r = 256, 128, 16
    W, A, _, _ = layer_inputs(2, 0, m, n, r, 16, 0)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), None, 1.0)
    dB = synth.normal_bf16(2, 99, (m, r), 1.0).float()
    dB[40] = dB[7]; dB[200] = dB[7]; dB[100] = -dB[7]
    dB[[7, 40, 100, 200]] *= 50           # the four tied rows carry the largest score
    for k in (1, 2, 3, 4, 5):
        layer.dbuf.zero_()
        wq_o, dbuf_o = u8(layer.wq).copy(), np.zeros((m, r), np.float32)
        idx = fq.proxy_update(layer, dB.to(DEV), 0.01, k)
        idx_o, _ = orc.proxy_update(wq_o, dbuf_o, dB.numpy(), 0.01, k, m, r)
        assert u8(idx).tolist() == idx_o.tolist()
        assert set([7, 40, 100, 200][:min(k, 4)]) <= set(u8(idx).tolist())
        assert np.array_equal(u8(layer.wq), wq_o)


# ------------------------------------------------------------------ full-size projections, sampled

def _sampled_projection(fq, orc, matrix, n, m, T, r, k, lr, outlier_frac, per_row=False, heavy_tailed=False):
    """One full-size projection: bit-exact stages on every element, tensor-core outputs on sampled rows / columns."""
    n_out = round(outlier_frac * n)
    W = synth.backbone(0, matrix, m, n, DEV, heavy_tailed=heavy_tailed)
    A = synth.adapter_a(0, matrix, r, n, DEV)
    B = synth.adapter_b(0, matrix, m, r, DEV)
    X = synth.activations(0, matrix, T, n, n_out, DEV)
    dY = synth.out_grad(0, matrix, 0, T, m, DEV)
    layer = fq.setup_layer(W, A, B, 1.0, per_row=per_row)
    ws = layer.workspace(T)
    Y, OA, amax_oa, s_x = fq.melded_forward(layer, X, y_dtype=torch.float32, ws=ws)
    xq_g = u8(fq.ws_view(layer, ws, T, fq.WS_XQ)).reshape(T, n)
    xq_o, s_x_o, _ = orc.quantize(f32(X), orc.E4M3)
    assert bits32(f32(s_x))[0] == bits32(s_x_o) and np.array_equal(xq_g, xq_o)
    wq = u8(layer.wq)
    s_w = f32(layer.s_w) if per_row else np.float32(f32(layer.s_w)[0])
    rng = np.random.default_rng(1)
    tsel = np.sort(rng.choice(T, 48, replace=False))
    fsel = np.sort(rng.choice(m, 48, replace=False))
    merged = torch.cat([Y, OA], dim=1)
    rows_o = orc.forward_gemm(xq_g, s_x_o, wq, s_w, m, r, tsel=tsel)                 # 48 token rows x all features
    assert product_close(f32(merged[torch.from_numpy(tsel).to(DEV)]), rows_o, GEMM_TOL)
    cols_o = orc.forward_gemm(xq_g, s_x_o, wq, s_w, m, r, fsel=fsel)                 # all tokens x 48 features
    assert product_close(f32(Y[:, torch.from_numpy(fsel).to(DEV)]), cols_o, GEMM_TOL)
    assert bits32(f32(amax_oa))[0] == bits32(f32(OA.abs().max()))
    dX, dB, s_g = fq.melded_backward(layer, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
    gq_g = u8(fq.ws_view(layer, ws, T, fq.WS_GQ)).reshape(T, m)
    if per_row:
        gq_o, s_g_o, _ = orc.quantize_colscaled(f32(dY), orc.E5M2, s_w[:m])
    else:
        gq_o, s_g_o, _ = orc.quantize(f32(dY), orc.E5M2)
    assert bits32(f32(s_g))[0] == bits32(s_g_o) and np.array_equal(gq_g, gq_o)
    csel = np.sort(rng.choice(n, 48, replace=False))
    assert product_close(f32(dX[torch.from_numpy(tsel).to(DEV)]), orc.dx_gemm(gq_g, s_g_o, wq, s_w, m, tsel=tsel), GEMM_TOL)
    assert product_close(f32(dX[:, torch.from_numpy(csel).to(DEV)]), orc.dx_gemm(gq_g, s_g_o, wq, s_w, m, csel=csel), GEMM_TOL)
    oaq_o, s_oa_o, _ = orc.quantize(f32(OA), orc.E4M3)
    isel = np.sort(rng.choice(m, 96, replace=False))
    dB_o = orc.db_gemm(gq_g, s_g_o, oaq_o, s_oa_o, isel=isel, row_scale=s_w[:m] if per_row else None)
    assert product_close(f32(dB[torch.from_numpy(isel).to(DEV)]), dB_o, GEMM_TOL)
    dbuf_o, wq_o = f32(layer.dbuf).copy(), wq.copy()
    idx = fq.proxy_update(layer, dB, lr, k, ws=ws)
    idx_o, score_o = orc.proxy_update(wq_o, dbuf_o, f32(dB), lr, k, m, r, row_scales=s_w if per_row else None)
    assert np.array_equal(u8(idx), idx_o)
    assert np.array_equal(u8(layer.wq), wq_o) and np.array_equal(bits32(f32(layer.dbuf)), bits32(dbuf_o))
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("name,n,m", [("q", 4096, 4096), ("gate", 4096, 11008), ("down", 11008, 4096)])
def test_config1_projection_sampled(fq, orc, name, n, m):
    c = synth.config1()
    _sampled_projection(fq, orc, {"q": 0, "gate": 4, "down": 6}[name], n, m, c["T"], c["r"], c["k"], c["lr"],
                        c["outlier_frac"])


@pytest.mark.parametrize("name,n,m", [("q", 5120, 5120), ("down", 13824, 5120)])
def test_config3_projection_sampled_per_row(fq, orc, name, n, m):
    """LLaMA-13B shapes, 8192 tokens, heavy-tailed rows (0.02 * t_3) with per-row scales, top-512."""
    _sampled_projection(fq, orc, {"q": 0, "down": 6}[name], n, m, 8192, 64, 512, 2e-4, 0.01, per_row=True,
                        heavy_tailed=True)


@pytest.mark.parametrize("r,T,k", [(8, 512, 4096), (128, 2048, 64), (32, 512, 0), (128, 32768, 4096)])
def test_config4_sweep_corner_shapes(fq, orc, r, T, k):
    """Corners of the rank x tokens x top-k sweep on the 4096 -> 11008 projection (the last one is its largest point:
    268 MB of activations, 721 MB of output gradients, 2.1 G fma in the merge)."""
    if k == 0:
        _run_layer_stages(fq, orc, 0, 11008, 4096, r, T, 0, 1.0, 41, 1, 2e-4)
    else:
        _sampled_projection(fq, orc, 4, 4096, 11008, T, r, k, 2e-4, 0.01)


def test_adamw_proxy_update_bit_exact(fq, orc):
    """AdamW on the DeltaBuffer (the optimizer the paper trains with), three steps with merges in between."""
    m, n, r, k = 1024, 512, 32, 48
    W, A, B, _ = layer_inputs(17, 0, m, n, r, 16, 0)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0)
    wq_o, dbuf_o = u8(layer.wq).copy(), f32(layer.dbuf).copy()
    m_g = torch.zeros((m, r), dtype=torch.float32, device=DEV)
    v_g = torch.zeros((m, r), dtype=torch.float32, device=DEV)
    m_o, v_o = np.zeros((m, r), np.float32), np.zeros((m, r), np.float32)
    hp = dict(lr=2e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    for step in range(1, 4):
        dB = synth.normal_bf16(17, 40 + step, (m, r), 1e-2).float()
        idx = fq.proxy_update_adamw(layer, dB.to(DEV), m_g, v_g, step, k, **hp)
        orc.adamw_step(dbuf_o, dB.numpy(), m_o, v_o, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], step)
        idx_o, _ = orc.proxy_update(wq_o, dbuf_o, None, 0.0, k, m, r)
        assert np.array_equal(u8(idx), idx_o), step
        assert np.array_equal(bits32(f32(m_g)), bits32(m_o)) and np.array_equal(bits32(f32(v_g)), bits32(v_o)), step
        assert np.array_equal(bits32(f32(layer.dbuf)), bits32(dbuf_o)), step
        assert np.array_equal(u8(layer.wq), wq_o), step
    assert fq.last_device_status() == 0


def test_backward_on_shared_gradient_codes(fq, orc):
    """falqon_melded_backward_codes: a second layer of the same output width multiplies the gradient codes the first one
    cast -- bit for bit what its own falqon_melded_backward gives; per-row layers are refused."""
    m, n1, n2, r, T = 768, 512, 1024, 32, 700
    W1, A1, B1, X1 = layer_inputs(81, 0, m, n1, r, T, 3, DEV)
    W2, A2, B2, X2 = layer_inputs(81, 1, m, n2, r, T, 3, DEV)
    dY = synth.out_grad(81, 0, 0, T, m, DEV)
    L1, L2 = fq.setup_layer(W1, A1, B1, 1.0), fq.setup_layer(W2, A2, B2, 1.0)
    ws1, ws2 = L1.workspace(T), L2.workspace(T)
    _, OA1, am1, _ = fq.melded_forward(L1, X1, ws=ws1)
    _, OA2, am2, _ = fq.melded_forward(L2, X2, ws=ws2)
    dX_ref, dB_ref, _ = fq.melded_backward(L2, dY, OA2, am2, dx_dtype=torch.float32, ws=ws2)
    dX_ref, dB_ref = dX_ref.clone(), dB_ref.clone()
    fq.ws_view(L2, ws2, T, fq.WS_GQ).fill_(0)          # L2's own codes are gone: the shared call must not need them
    fq.melded_backward(L1, dY, OA1, am1, ws=ws1)
    gq = fq.ws_view(L1, ws1, T, fq.WS_GQ)[: T * m].view(T, m)
    s_g = fq.ws_view(L1, ws1, T, fq.WS_SCALES).view(torch.float32)[3:4]
    dX, dB = fq.melded_backward_codes(L2, gq, s_g, OA2, am2, dx_dtype=torch.float32, ws=ws2)
    assert torch.equal(dX.view(torch.int32), dX_ref.view(torch.int32)) and torch.equal(dB.view(torch.int32), dB_ref.view(torch.int32))
    # (here the O_A cast ran inside the product's launch, synchronised through two control words of the workspace: they
    # are back at zero, and O~_A^T is what the output-gradient quantizer's rider wrote in the reference call)
    assert int(ws2[256:264].view(torch.int32).abs().sum()) == 0
    # (without dX, dB is a kernel of its own that sums token slabs: the same numbers in another order of the fp32 sums)
    _, dB_only = fq.melded_backward_codes(L2, gq, s_g, OA2, am2, need_dx=False, ws=ws2)
    assert float((dB_only - dB_ref).abs().max()) <= 2e-6 * float(dB_ref.abs().max())
    gq_o, s_g_o, _ = orc.quantize(f32(dY), orc.E5M2)
    assert np.array_equal(u8(gq), gq_o) and bits32(f32(s_g))[0] == bits32(s_g_o)
    Lr = fq.setup_layer(W2, A2, B2, 1.0, per_row=True)
    with pytest.raises(fq.FalqonError) as e:
        fq.melded_backward_codes(Lr, gq, s_g, OA2, am2, ws=Lr.workspace(T))
    assert e.value.status == fq.ERR_UNSUPPORTED
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("m,T", [(16, 40), (1040, 333), (1040, 20011), (14336, 131), (16384, 37), (28688, 19)])
def test_column_scaled_cast_of_bf16_gradients_in_every_chunk_geometry(fq, orc, m, T):
    """The output-gradient cast of a per-row-scaled layer (dY[:, i] / s_w[i], then Eq. quantize in E5M2) on bf16 input:
    rows that fit a staging chunk many times, exactly twice, once (the row-aligned mode: chunks are whole rows, the absmax
    pass takes column maxima first and multiplies once), and rows longer than a chunk (linear chunks, a multiply per
    element); a ragged last chunk; a tensor larger than the chip's shared memory (chunks fetched twice).  Codes and scale
    bit for bit against the oracle."""
    n, r = 64, 16
    W = synth.backbone(41, 0, m, n, DEV, heavy_tailed=True)
    A = synth.adapter_a(41, 0, r, n, DEV)
    B = synth.adapter_b(41, 0, m, r, DEV)
    X = synth.activations(41, 0, T, n, 2, DEV)
    layer = fq.setup_layer(W, A, B, 1.0, per_row=True)
    ws = layer.workspace(T)
    _, OA, amax_oa, _ = fq.melded_forward(layer, X, y_dtype=torch.float32, ws=ws)
    dY = synth.out_grad(41, 0, 0, T, m, DEV)
    dY[T // 2, m - 3] = 0.75          # the absmax sits where only the column factor decides
    assert dY.dtype == torch.bfloat16
    fq.ws_view(layer, ws, T, fq.WS_GQ).fill_(0x55)
    _, _, s_g = fq.melded_backward(layer, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
    gq_o, s_g_o, _ = orc.quantize_colscaled(f32(dY), orc.E5M2, f32(layer.s_w)[:m])
    assert bits32(f32(s_g))[0] == bits32(s_g_o)
    assert np.array_equal(u8(fq.ws_view(layer, ws, T, fq.WS_GQ))[: T * m].reshape(T, m), gq_o)
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("m,n,r,T", [
    (16, 16, 8, 16),            # the smallest layer: one pair, one tile of dB with 16 valid rows, 8 of 16 instruction columns
    (400, 272, 24, 333),        # two dB tiles, the second partial; r16 = 32 > r; fewer product tiles than SM pairs
    (4112, 64, 256, 130),       # 17 dB tiles of the widest rank behind ONE product tile: every pair takes some
    (28688, 128, 8, 1000),      # 113 dB tiles, more than there are pairs: round robin over all of them
    (1024, 4096, 64, 2049),     # tokens one past a k-block; the product has a partial last wave (8 x 16 tiles)
])
@pytest.mark.parametrize("per_row", [False, True])
def test_adapter_gradient_riding_on_the_input_gradient_product(fq, orc, m, n, r, T, per_row):
    """dB computed inside the launch of the input-gradient product (the default) against the oracle on the GPU's own
    codes, against dB from the kernel of its own (same numbers in another summation order), and dX unchanged by the rider;
    once after the fused quantizer (which carries the O_A cast) and once with a known absmax (the O_A cast rides in the
    product's launch too).  Shapes at the corners of the rider's tiling."""
    W = synth.backbone(51, 0, m, n, DEV, heavy_tailed=per_row)
    A, B = synth.adapter_a(51, 0, r, n, DEV), synth.adapter_b(51, 0, m, r, DEV)
    X = synth.activations(51, 0, T, n, 1, DEV)
    dY = synth.out_grad(51, 0, 0, T, m, DEV)
    ride = fq.setup_layer(W, A, B, 1.0, per_row=per_row)
    own = fq.Layer(ride.wq, ride.s_w, ride.dbuf, r, flags=fq.LAYER_DB_OWN_KERNEL)
    ws = ride.workspace(T)
    _, OA, amax_oa, _ = fq.melded_forward(ride, X, ws=ws)
    dX0, dB0, s_g0 = fq.melded_backward(own, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
    dX0, dB0 = dX0.clone(), dB0.clone()
    oaq0 = fq.ws_view(ride, ws, T, fq.WS_OAQ_T).clone()
    fq.ws_view(ride, ws, T, fq.WS_OAQ_T).fill_(0x7F)           # NaN codes: whoever multiplies stale O~_A shows it
    dX1, dB1, s_g1 = fq.melded_backward(ride, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
    assert torch.equal(dX0.view(torch.int32), dX1.view(torch.int32)) and torch.equal(s_g0, s_g1)
    scale = float(dB0.abs().max())
    assert float((dB1 - dB0).abs().max()) <= 4e-6 * scale
    s_w = f32(ride.s_w)
    gq = u8(fq.ws_view(ride, ws, T, fq.WS_GQ))[: T * m].reshape(T, m)
    oaq_o, s_oa_o, _ = orc.quantize(f32(OA), orc.E4M3)
    dB_o = orc.db_gemm(gq, np.float32(f32(s_g1)[0]), oaq_o, s_oa_o, row_scale=s_w[:m] if per_row else None)
    assert product_close(f32(dB1), dB_o, GEMM_TOL)
    if not per_row:     # known absmax of dY: a single-pass cast, and the O_A cast inside the product's launch
        amax_dy = dY.float().abs().max().reshape(1)
        fq.ws_view(ride, ws, T, fq.WS_OAQ_T).fill_(0x7F)
        dX2, dB2, s_g2 = fq.melded_backward(ride, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws, amax_dy=amax_dy)
        assert torch.equal(dX2.view(torch.int32), dX0.view(torch.int32)) and torch.equal(dB2.view(torch.int32), dB1.view(torch.int32))
        got = fq.ws_view(ride, ws, T, fq.WS_OAQ_T)
        t16 = got.numel() // ((r + 15) // 16 * 16)
        assert torch.equal(got.view(-1, t16)[:r, :T], oaq0.view(-1, t16)[:r, :T])      # the codes the quantizer's rider wrote
        assert int(ws[256:264].view(torch.int32).abs().sum()) == 0
    assert fq.last_device_status() == 0
