"""Token-sharded data parallelism on the CUDA path, on ONE device: three replicas of a layer -- two that each take a
shard of the tokens and run the phases of TokenShardedLayer one after another (the test combines the maxima and sums
the partial gradients itself, as the collectives of `step()` would between ranks), and one that takes all tokens in a
single call.  Every shard's codes, Y and dX must be bit for bit the rows of the unsharded call, the summed dB must agree
with the unsharded dB to fp32 summation order, and the two sharded replicas must be identical after the update."""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, layer_inputs, product_close, rel_fro, u8
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("m,n,r,T,split,k", [(1024, 768, 16, 640, 384, 48), (512, 1280, 64, 1000, 300, 32)])
def test_two_token_shards_against_the_unsharded_call(m, n, r, T, split, k):
    from paper_2510_24061_b200 import binding as fq
    from paper_2510_24061_b200.token_parallel import TokenShardedLayer
    from oracle import falqon_oracle as orc
    lr = 2e-2
    W, A, B, X = layer_inputs(31, 0, m, n, r, T, 4)
    dY = synth.out_grad(31, 0, 0, T, m)
    full = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0)
    reps = [fq.Layer(full.wq.clone(), full.s_w.clone(), full.dbuf.clone(), r) for _ in range(2)]
    Xd, dYd = X.to(DEV), dY.to(DEV)
    shards = [(0, split), (split, T)]
    ts = [TokenShardedLayer(rep) for rep in reps]
    # absmax of X: per shard, then the maximum (the collective of step())
    assert float(fq.absmax(Xd).item()) == float(Xd.float().abs().max().item())
    ax = torch.maximum(*[t.input_absmax(Xd[lo:hi].contiguous()) for t, (lo, hi) in zip(ts, shards)])
    outs = [t.forward(Xd[lo:hi].contiguous(), ax, y_dtype=torch.float32) for t, (lo, hi) in zip(ts, shards)]
    amax_oa = torch.maximum(ts[0].amax_oa, ts[1].amax_oa)
    for t in ts:
        t.amax_oa.copy_(amax_oa)
    ag = torch.maximum(*[t.output_grad_absmax(dYd[lo:hi].contiguous()) for t, (lo, hi) in zip(ts, shards)])
    grads = [t.backward(dYd[lo:hi].contiguous(), ag, dx_dtype=torch.float32) for t, (lo, hi) in zip(ts, shards)]
    dB_total = grads[0][1] + grads[1][1]                                 # the exchange step
    # the unsharded call on the third replica
    ws = full.workspace(T)
    Y_f, OA_f, amax_oa_f, s_x_f = fq.melded_forward(full, Xd, y_dtype=torch.float32, ws=ws)
    dX_f, dB_f, s_g_f = fq.melded_backward(full, dYd, OA_f, amax_oa_f, dx_dtype=torch.float32, ws=ws)
    assert float(amax_oa.item()) == float(amax_oa_f.item())
    for (Y, OA), (dX, _), (lo, hi) in zip(outs, grads, shards):
        assert torch.equal(Y, Y_f[lo:hi]) and torch.equal(OA, OA_f[lo:hi]), "a shard's outputs are rows of the unsharded call"
        assert torch.equal(dX, dX_f[lo:hi])
    assert rel_fro(f32(dB_total), f32(dB_f).astype(np.float64)) < 1e-6
    # and against the oracle: dB of the whole batch from the unsharded call's operand codes
    gq = u8(fq.ws_view(full, ws, T, fq.WS_GQ)).reshape(T, m)
    oaq_o, s_oa_o, _ = orc.quantize(f32(OA_f), orc.E4M3)
    dB_o = orc.db_gemm(gq, np.float32(s_g_f.item()), oaq_o, s_oa_o)
    assert product_close(f32(dB_total), dB_o, 2e-5)
    # the update: identical on both sharded replicas, and the oracle's update of the same summed gradient
    wq_o, dbuf_o = u8(reps[0].wq).copy(), f32(reps[0].dbuf).copy()
    idx = [t.update(dB_total, lr, k) for t in ts]
    idx_o, _ = orc.proxy_update(wq_o, dbuf_o, f32(dB_total), lr, k, m, r)
    assert torch.equal(idx[0], idx[1]) and np.array_equal(u8(idx[0]), idx_o)
    assert torch.equal(reps[0].wq, reps[1].wq) and np.array_equal(u8(reps[0].wq), wq_o)
    assert torch.equal(reps[0].dbuf.view(torch.int32), reps[1].dbuf.view(torch.int32))
    assert np.array_equal(bits32(f32(reps[0].dbuf)), bits32(dbuf_o))
    assert fq.last_device_status() == 0


def test_split_backward_and_overlapped_step_equal_the_single_call():
    """falqon_melded_backward_dx after a backward without dX gives the dX of the single call bit for bit, and a step whose
    dB exchange runs on a side stream between the two halves (one rank: the reductions are identities) leaves the same
    results and the same layer as the step that runs them in order."""
    from paper_2510_24061_b200 import binding as fq
    from paper_2510_24061_b200.token_parallel import TokenShardedLayer
    m, n, r, T, k, lr = 768, 1024, 32, 900, 40, 2e-2
    W, A, B, X = layer_inputs(32, 0, m, n, r, T, 5, DEV)
    dY = synth.out_grad(32, 0, 0, T, m, DEV)
    base = fq.setup_layer(W, A, B, 1.0)
    base.flags = fq.LAYER_DB_OWN_KERNEL     # the split backward computes dB by itself: the single call shall use the same kernel
    ws = base.workspace(T)
    Y, OA, amax_oa, _ = fq.melded_forward(base, X, y_dtype=torch.float32, ws=ws)
    dX0, dB0, _ = fq.melded_backward(base, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
    _, dB1, _ = fq.melded_backward(base, dY, OA, amax_oa, need_dx=False, ws=ws)
    dX1 = fq.melded_backward_dx(base, T, dx_dtype=torch.float32, ws=ws)
    assert torch.equal(dX0.view(torch.int32), dX1.view(torch.int32)) and torch.equal(dB0.view(torch.int32), dB1.view(torch.int32))

    class OneRank:
        def all_reduce_max(self, t):
            pass

        def all_reduce_sum(self, t):
            t.mul_(1.0)        # some work on whatever stream is current, in place like a collective

    results = []
    for overlap in (False, True):
        rep = fq.Layer(base.wq.clone(), base.s_w.clone(), base.dbuf.clone(), r, flags=fq.LAYER_DB_OWN_KERNEL)
        ts = TokenShardedLayer(rep, comm=OneRank())
        out = ts.step(X, dY, lr, k, y_dtype=torch.float32, dx_dtype=torch.float32, overlap=overlap)
        torch.cuda.synchronize()
        results.append((out, rep))
    (a, ra), (b, rb) = results
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert torch.equal(ra.wq, rb.wq) and torch.equal(ra.dbuf.view(torch.int32), rb.dbuf.view(torch.int32))
    assert fq.last_device_status() == 0
