"""Token-sharded data parallelism (paper_2510_24061_b200/token_parallel.py) on two gloo ranks on the CPU.  The layer
calls are served by the CPU oracle through a small adapter (the package itself has no CPU implementation), so what is
checked here is the host logic: which values are exchanged, in which order, and that the result is what the unsharded
step computes -- each rank's Y and dX are bit for bit the corresponding rows of the unsharded run, the summed dB agrees
with the unsharded dB to the fp32 rounding of the two partial sums, and the replicas are identical after the update."""
import os
import sys
import types

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
M, N, R, T, K, LR = 96, 128, 8, 64, 12, 5e-2


class OracleOps:
    """The calls TokenShardedLayer makes, on CPU tensors, computed by the oracle."""

    def __init__(self, orc):
        self.orc = orc

    @staticmethod
    def _scale(amax, fp8max):      # one IEEE fp32 division, amax == 0 -> 1 (Eq. quantize)
        a = np.float32(amax)
        return np.float32(1.0) if not a > 0 else np.float32(fp8max) / a

    def absmax(self, x):
        return x.float().abs().max().reshape(1)

    def melded_forward(self, layer, X, y_dtype=torch.float32, amax_x=None):
        o = self.orc
        s_x = self._scale(amax_x.item(), 448.0)
        xq, _, _ = o.quantize(X.float().numpy(), o.E4M3, scale_in=s_x)
        Y, OA, amax_oa = o.forward(xq, s_x, layer.wq, layer.s_w, layer.m, layer.r)
        return (torch.from_numpy(Y.astype(np.float32)), torch.from_numpy(OA), torch.tensor([amax_oa], dtype=torch.float32),
                torch.tensor([s_x]))

    def melded_backward(self, layer, dY, OA, amax_oa, need_dx=True, dx_dtype=torch.float32, amax_dy=None):
        o = self.orc
        s_g = self._scale(amax_dy.item(), 57344.0)
        s_oa = self._scale(amax_oa.item(), 448.0)
        gq, _, _ = o.quantize(dY.float().numpy(), o.E5M2, scale_in=s_g)
        oaq, _, _ = o.quantize(OA.numpy(), o.E4M3, scale_in=s_oa)
        self._gq, self._s_g = gq, s_g
        dX = torch.from_numpy(o.dx_gemm(gq, s_g, layer.wq, layer.s_w, layer.m).astype(np.float32)) if need_dx else None
        dB = o.db_gemm(gq, s_g, oaq, s_oa)
        return dX, torch.from_numpy(dB.astype(np.float32)), torch.tensor([s_g])

        # (need_dx=False: the first half of the split backward; the codes stay behind for melded_backward_dx)

    def melded_backward_dx(self, layer, T, dx_dtype=torch.float32):
        dX = self.orc.dx_gemm(self._gq, self._s_g, layer.wq, layer.s_w, layer.m)
        assert dX.shape[0] == T
        return torch.from_numpy(dX.astype(np.float32))

    def proxy_update(self, layer, dB, lr, k):
        idx, _ = self.orc.proxy_update(layer.wq, layer.dbuf, dB.numpy(), lr, k, layer.m, layer.r)
        return torch.from_numpy(idx.copy())


def _inputs():
    sys.path.insert(0, ROOT)
    from paper_2510_24061_b200 import synth
    from oracle import falqon_oracle as orc
    W = synth.backbone(21, 0, M, N).float().numpy()
    A = synth.adapter_a(21, 0, R, N).float().numpy()
    B = synth.adapter_b(21, 0, M, R).float().numpy()
    X = synth.activations(21, 0, T, N, 2).float()
    dY = synth.out_grad(21, 0, 0, T, M).float()
    wq, s_w, dbuf = orc.setup_layer(W, A, B, 1.0)
    return orc, wq, np.float32(s_w), dbuf, X, dY


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    orc, wq, s_w, dbuf, X, dY = _inputs()
    from paper_2510_24061_b200.token_parallel import TokenShardedLayer
    layer = types.SimpleNamespace(wq=wq.copy(), s_w=s_w, dbuf=dbuf.copy(), m=M, n=N, r=R)
    lo, hi = (0, 40) if rank == 0 else (40, T)            # uneven shards
    ts = TokenShardedLayer(layer, ops=OracleOps(orc))
    Y, dX, dB, idx = ts.step(X[lo:hi].contiguous(), dY[lo:hi].contiguous(), LR, K, y_dtype=torch.float32,
                             dx_dtype=torch.float32)
    out[rank] = dict(Y=Y.numpy(), dX=dX.numpy(), dB=dB.numpy(), idx=idx.numpy(), wq=layer.wq.copy(), dbuf=layer.dbuf.copy(),
                     rows=(lo, hi))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_step():
    world = 2
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29641, out), nprocs=world, join=True)
    orc, wq, s_w, dbuf, X, dY = _inputs()
    f = orc.layer_forward(X.numpy(), wq, s_w, M, R)                       # the unsharded step
    b = orc.layer_backward(dY.numpy(), f["OA"], wq, s_w, M, R)
    dB_full = b["dB"].astype(np.float32)
    wq_full, dbuf_full = wq.copy(), dbuf.copy()
    idx_full, _ = orc.proxy_update(wq_full, dbuf_full, dB_full, LR, K, M, R)
    for rank in range(world):
        o = out[rank]
        lo, hi = o["rows"]
        assert np.array_equal(o["Y"], f["Y"][lo:hi].astype(np.float32)), "a shard's Y is the unsharded Y's rows"
        assert np.array_equal(o["dX"], b["dX"][lo:hi].astype(np.float32))
        err = np.linalg.norm(o["dB"].astype(np.float64) - b["dB"]) / np.linalg.norm(b["dB"])
        assert err < 1e-6, err                                           # fp32 sum of two fp32 partials
    a, c = out[0], out[1]
    assert np.array_equal(a["dB"], c["dB"]) and np.array_equal(a["idx"], c["idx"])
    assert np.array_equal(a["wq"], c["wq"]) and np.array_equal(a["dbuf"].view(np.uint32), c["dbuf"].view(np.uint32))
    # against the unsharded update: the same rows unless two scores are within the last bit of each other
    assert len(set(a["idx"].tolist()) & set(idx_full.tolist())) >= K - 1
    assert float((a["wq"] != wq_full).mean()) < 2e-2


def test_exchange_of_db_is_issued_between_the_two_halves_of_backward():
    """The order in which TokenShardedLayer.step issues its work when the exchange overlaps the input-gradient product:
    dB is computed first, its sum is started on the side stream right after a fork, dX is enqueued while it runs, and the
    update comes only after the join.  A recording communicator and a recording side stream stand in for the real ones;
    the result equals the un-overlapped order's."""
    sys.path.insert(0, ROOT)
    from paper_2510_24061_b200.token_parallel import TokenShardedLayer
    orc, wq, s_w, dbuf, X, dY = _inputs()
    log = []

    class Ops(OracleOps):
        def melded_forward(self, *a, **k):
            log.append("forward")
            return super().melded_forward(*a, **k)

        def melded_backward(self, layer, dY, OA, amax_oa, need_dx=True, **k):
            log.append("backward" if need_dx else "backward_db")
            return super().melded_backward(layer, dY, OA, amax_oa, need_dx=need_dx, **k)

        def melded_backward_dx(self, *a, **k):
            log.append("backward_dx")
            return super().melded_backward_dx(*a, **k)

        def proxy_update(self, *a, **k):
            log.append("update")
            return super().proxy_update(*a, **k)

    class Comm:     # a single rank: the reductions are identities
        def all_reduce_max(self, t):
            log.append("max")

        def all_reduce_sum(self, t):
            log.append("sum")

    class Side:
        def fork(self):
            log.append("fork")

        def run(self, fn):
            log.append("side:")
            fn()

        def join(self):
            log.append("join")

    results = {}
    for overlap in (True, False):
        del log[:]
        layer = types.SimpleNamespace(wq=wq.copy(), s_w=s_w, dbuf=dbuf.copy(), m=M, n=N, r=R)
        ts = TokenShardedLayer(layer, ops=Ops(orc), comm=Comm())
        ts.side = Side()
        Y, dX, dB, idx = ts.step(X, dY, LR, K, y_dtype=torch.float32, dx_dtype=torch.float32, overlap=overlap)
        results[overlap] = (Y.numpy(), dX.numpy(), dB.numpy(), idx.numpy(), layer.wq.copy(), list(log))
    assert results[True][5] == ["max", "forward", "max", "max", "backward_db", "fork", "side:", "sum", "backward_dx", "join", "update"]
    assert results[False][5] == ["max", "forward", "max", "max", "backward", "sum", "update"]
    for a, b in zip(results[True][:5], results[False][:5]):
        assert np.array_equal(a, b)
