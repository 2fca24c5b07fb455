"""GPU parity of the fused optimizer step: falqon_melded_backward_update runs Alg. 3 line 4 (plain SGD on the DeltaBuffer)
and the row scores inside the adapter-gradient kernel, falqon_proxy_update_scored[_batched] then selects and merges from
those scores.  Teacher-forced against the CPU oracle (fed the GPU's own dB): DeltaBuffer, scores, selected rows and merged
rows bit for bit; and bit for bit against the un-fused sequence backward + proxy update on a twin layer."""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, layer_inputs, u8
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _twin(fq, layer):
    return fq.Layer(layer.wq.clone(), layer.s_w.clone(), layer.dbuf.clone(), layer.r, flags=layer.flags)


@pytest.mark.parametrize("m,n,r,T,k,per_row,lr", [
    (1024, 1024, 16, 512, 32, False, 2e-2),      # configs[0]
    (400, 272, 24, 333, 17, False, 2e-1),        # ragged everywhere, one partial row tile
    (4096, 4096, 64, 4096, 256, False, 2e-4),    # configs[1]: q
    (528, 384, 256, 130, 40, False, 2e-2),       # rank 256 with two token blocks: no room in shared memory, separate pass
    (384, 512, 32, 700, 25, True, 2e-2),         # per-row-scaled backbone: dB rows are multiplied back by s_w[i] first
])
@pytest.mark.parametrize("own_kernel", [False, True])
def test_backward_update_and_scored_proxy_update(m, n, r, T, k, per_row, lr, own_kernel):
    from paper_2510_24061_b200 import binding as fq
    from oracle import falqon_oracle as orc
    W, A, B, X = layer_inputs(41, 1, m, n, r, T, 3, DEV)
    if per_row:
        W = synth.backbone(41, 1, m, n, DEV, heavy_tailed=True)
    dY = synth.out_grad(41, 1, 0, T, m, DEV)
    ref = fq.setup_layer(W, A, B, 1.0, per_row=per_row)
    # the step and the scores ride with dB inside the dX launch, or (own_kernel, and always at ranks above 128) live in the
    # adapter-gradient kernel: the reference computes dB the same way, so that the two sequences see the same bits
    if own_kernel or r > 128:
        ref.flags = fq.LAYER_DB_OWN_KERNEL
    ref.dbuf.copy_(synth.normal_bf16(41, 90, (m, r), 1e-3, DEV).float())      # something for the step to accumulate onto
    new = _twin(fq, ref)
    ws_r, ws_n = ref.workspace(T), new.workspace(T)
    rs = f32(ref.s_w) if per_row else None
    for step in range(2):
        dYs = synth.out_grad(41, 1, step, T, m, DEV)
        _, OA, amax_oa, _ = fq.melded_forward(ref, X, ws=ws_r)
        dX0, dB0, _ = fq.melded_backward(ref, dYs, OA, amax_oa, dx_dtype=torch.float32, ws=ws_r)
        wq_o, dbuf_o = u8(ref.wq).copy(), f32(ref.dbuf).copy()
        idx0 = fq.proxy_update(ref, dB0, lr, k, ws=ws_r)
        _, OA1, amax_oa1, _ = fq.melded_forward(new, X, ws=ws_n)
        dX1, dB1, _ = fq.melded_backward_update(new, dYs, OA1, amax_oa1, lr, dx_dtype=torch.float32, ws=ws_n)
        # after the fused step and before the selection: DeltaBuffer and scores against the oracle's update of the same dB
        idx_o, score_o = orc.proxy_update(wq_o, dbuf_o.copy(), f32(dB1), lr, 0, m, r, row_scales=rs)    # k = 0: step and scores only
        dbuf_step = dbuf_o.copy()
        orc.proxy_update(wq_o.copy(), dbuf_step, f32(dB1), lr, 0, m, r, row_scales=rs)
        assert np.array_equal(bits32(f32(new.dbuf)), bits32(dbuf_step)), f"DeltaBuffer after the fused step, step {step}"
        assert np.array_equal(bits32(f32(fq.ws_view(new, ws_n, T, fq.WS_SCORE).view(torch.float32))), bits32(score_o)), "row scores"
        idx1 = fq.proxy_update_scored(new, k, ws=ws_n)
        idx_o, _ = orc.proxy_update(wq_o, dbuf_o, f32(dB1), lr, k, m, r, row_scales=rs)
        assert np.array_equal(u8(idx1), idx_o) and np.array_equal(u8(new.wq), wq_o), f"selection / merge vs the oracle, step {step}"
        assert np.array_equal(bits32(f32(new.dbuf)), bits32(dbuf_o))
        # and the un-fused sequence on the twin
        assert torch.equal(dX0, dX1) and torch.equal(dB0.view(torch.int32), dB1.view(torch.int32))
        assert torch.equal(idx0, idx1) and torch.equal(ref.wq, new.wq)
        assert torch.equal(ref.dbuf.view(torch.int32), new.dbuf.view(torch.int32))
    assert fq.last_device_status() == 0


def test_scored_batched_equals_per_layer_calls():
    from paper_2510_24061_b200 import binding as fq
    shapes = [(512, 256, 16, 300, 20), (272, 400, 8, 300, 0), (1024, 512, 64, 300, 64)]
    lr = 5e-2
    per, bat = [], []
    for i, (m, n, r, T, k) in enumerate(shapes):
        W, A, B, X = layer_inputs(42, i, m, n, r, T, 3, DEV)
        a = fq.setup_layer(W, A, B, 1.0)
        b = _twin(fq, a)
        dY = synth.out_grad(42, i, 0, T, m, DEV)
        for L, dst in ((a, per), (b, bat)):
            ws = L.workspace(T)
            _, OA, amax_oa, _ = fq.melded_forward(L, X, ws=ws)
            fq.melded_backward_update(L, dY, OA, amax_oa, lr, ws=ws)
            dst.append((L, ws, k))
    idx_per = [fq.proxy_update_scored(L, k, ws=ws) for L, ws, k in per]
    batch = fq.ProxyBatch([L for L, _, _ in bat], [None] * len(bat), [k for _, _, k in bat], wss=[ws for _, ws, _ in bat])
    idx_bat = batch.run_scored()
    for (La, _, k), (Lb, _, _), ia, ib in zip(per, bat, idx_per, idx_bat):
        assert (ia is None and ib is None) or torch.equal(ia, ib)
        assert torch.equal(La.wq, Lb.wq) and torch.equal(La.dbuf.view(torch.int32), Lb.dbuf.view(torch.int32))
    assert fq.last_device_status() == 0
