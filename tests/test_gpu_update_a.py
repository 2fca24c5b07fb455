"""GPU parity of falqon_update_a (the paper's appendix ablation with a trainable A) against the CPU oracle, stage by stage
and teacher-forced: the codes of B and of P and the scales bit for bit, the two tensor-core products within 2e-5 of the
oracle's fp64 products of the identical codes, the fma step on the master copy and the re-created A~ rows bit for bit from
the GPU's own gradient; untouched backbone rows unchanged; and the whole step against the oracle's composition."""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, layer_inputs, product_close, u8
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("m,n,r,T,gamma", [(1024, 1024, 16, 512, 2.0), (400, 272, 24, 333, 1.0), (512, 768, 64, 1000, 1.0),
                                           (272, 528, 256, 200, 1.0)])
def test_update_a_stage_by_stage(m, n, r, T, gamma):
    from paper_2510_24061_b200 import binding as fq
    from oracle import falqon_oracle as orc
    lr = 0.05
    W, A, B, X = layer_inputs(51, 0, m, n, r, T, 3, DEV)
    dY = synth.out_grad(51, 0, 0, T, m, DEV)
    layer = fq.setup_layer(W, A, B, gamma)
    ws = layer.workspace(T)
    _, OA, amax_oa, s_x = fq.melded_forward(layer, X, ws=ws)
    xq = fq.ws_view(layer, ws, T, fq.WS_XQ).clone().reshape(T, n)          # the caller keeps x~ (the backward reuses the region)
    fq.melded_backward(layer, dY, OA, amax_oa, ws=ws)
    gq = u8(fq.ws_view(layer, ws, T, fq.WS_GQ)).reshape(T, m)
    s_g = np.float32(f32(fq.ws_view(layer, ws, T, fq.WS_SCALES).view(torch.float32))[3])
    B32 = B.float().contiguous()
    A_master = A.float().contiguous()
    A_before = f32(A_master).copy()
    wq_before = u8(layer.wq).copy()
    scratch = fq.update_a(layer, xq, s_x, B32, A_master, gamma, lr, T, ws=ws)
    assert fq.last_device_status() == 0
    r16, t16 = (r + 15) // 16 * 16, (T + 15) // 16 * 16
    scal = f32(fq.ua_view(layer, scratch, T, fq.UA_SCALARS).view(torch.float32))
    bq_t = u8(fq.ua_view(layer, scratch, T, fq.UA_BQ_T)).reshape(r16, m)[:r]
    P = f32(fq.ua_view(layer, scratch, T, fq.UA_P).view(torch.float32)).reshape(T, r)
    pq_t = u8(fq.ua_view(layer, scratch, T, fq.UA_PQ_T)).reshape(r16, t16)[:r, :T]
    da_t = f32(fq.ua_view(layer, scratch, T, fq.UA_DA_T).view(torch.float32)).reshape(n, r)
    # casts of B and of the GPU's own P: bit for bit
    Bq_o, s_B_o, amax_B_o = orc.quantize(f32(B32), orc.E4M3)
    assert bits32(scal[0]) == bits32(amax_B_o) and bits32(scal[1]) == bits32(s_B_o)
    assert np.array_equal(bq_t, Bq_o.T)
    Pq_o, s_P_o, amax_P_o = orc.quantize(P, orc.E4M3)
    assert bits32(scal[2]) == bits32(amax_P_o) and bits32(scal[3]) == bits32(s_P_o)
    assert np.array_equal(pq_t, Pq_o.T)
    # the two products on identical codes
    P_o = orc.codes_gemm(gq, orc.E5M2, s_g, np.ascontiguousarray(bq_t), orc.E4M3, scal[1])
    assert product_close(P, P_o, 2e-5), "P = dY B"
    s_x_o = np.float32(f32(s_x)[0])
    dA_o = orc.codes_gemm(np.ascontiguousarray(pq_t), orc.E4M3, scal[3], np.ascontiguousarray(u8(xq).T), orc.E4M3, s_x_o)
    assert product_close(da_t.T, dA_o, 2e-5), "dA = P~^T x~"
    # the step on the master copy and the A~ rows, from the GPU's own gradient
    A_o = A_before.copy()
    orc.sgd_step(A_o, np.ascontiguousarray(da_t.T), lr)
    assert np.array_equal(bits32(f32(A_master)), bits32(A_o))
    s_w = np.float32(f32(layer.s_w)[0])
    rows_o, _, _ = orc.quantize(A_o, orc.E4M3, scale_in=s_w, premul=gamma)
    wq_after = u8(layer.wq)
    assert np.array_equal(wq_after[m:], rows_o) and np.array_equal(wq_after[:m], wq_before[:m])
    assert not np.array_equal(wq_after[m:], wq_before[m:])          # the step did move A~
    # the whole step against the oracle's own composition, fed the same operand codes: same A~ rows up to the few codes
    # that the last bits of the two products can flip
    wq_c, A_c = wq_before.copy(), A_before.copy()
    out = orc.update_a(gq, s_g, u8(xq), s_x_o, f32(B32), A_c, wq_c, s_w, gamma, lr, m, r)
    assert np.array_equal(out["Bq"], Bq_o) and abs(float(out["s_P"]) / float(scal[3]) - 1.0) < 1e-6   # max |P| may differ in its last bit
    assert float(np.mean(wq_c[m:] != wq_after[m:])) < 2e-3
    assert np.linalg.norm(A_c.astype(np.float64) - f32(A_master)) / np.linalg.norm(A_c) < 1e-6


def test_update_a_rejects_bad_arguments():
    from paper_2510_24061_b200 import binding as fq
    m, n, r, T = 256, 256, 16, 64
    W, A, B, X = layer_inputs(52, 0, m, n, r, T, 2, DEV)
    per_row = fq.setup_layer(W, A, B, 1.0, per_row=True)
    xq = torch.zeros((T, n), dtype=torch.uint8, device=DEV)
    s_x = torch.ones(1, dtype=torch.float32, device=DEV)
    with pytest.raises(fq.FalqonError) as e:
        fq.update_a(per_row, xq, s_x, B.float().contiguous(), A.float().contiguous(), 1.0, 0.1, T)
    assert e.value.status == fq.ERR_UNSUPPORTED
    layer = fq.setup_layer(W, A, B, 1.0)
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(fq.FalqonError) as e:
        fq.update_a(layer, xq, s_x, B.float().contiguous(), A.float().contiguous(), 1.0, 0.1, T, scratch=small)
    assert e.value.status == fq.ERR_WORKSPACE
