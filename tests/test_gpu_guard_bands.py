"""Out-of-range WRITES: every buffer a call may write (outputs, workspace, the layer's own tensors, scratch) sits inside
a larger allocation whose margins are filled with a pattern; after the calls -- on shapes whose last tiles, row groups,
chunks and slabs are all partial -- the margins must be untouched.  (The memory checker of the CUDA toolkit is not
available on the test machines; this and the comparison with the CPU oracle stand in for it.)"""
import pytest
import torch

from helpers import layer_inputs
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 8192
PATTERN = 0xA5


class Guarded:
    """A tensor of the given shape and dtype with GUARD bytes of pattern before and after it."""
    all = []

    def __init__(self, shape, dtype, fill=None):
        nbytes = int(torch.tensor([], dtype=dtype).element_size()) * int(torch.Size(shape).numel())
        padded = (nbytes + 255) // 256 * 256
        self.raw = torch.full((GUARD + padded + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        self.nbytes = nbytes
        self.t = self.raw[GUARD:GUARD + nbytes].view(dtype).view(shape)
        if fill is not None:
            self.t.copy_(fill)
        Guarded.all.append(self)

    def intact(self):
        head = self.raw[:GUARD]
        tail = self.raw[GUARD + self.nbytes:]
        return bool((head == PATTERN).all()) and bool((tail == PATTERN).all())


def _guarded_layer(fq, seed, m, n, r, per_row):
    W, A, B, _ = layer_inputs(seed, 0, m, n, r, 16, 0)
    if per_row:
        W = synth.backbone(seed, 0, m, n, heavy_tailed=True)
    plain = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0, per_row=per_row)
    wq = Guarded(plain.wq.shape, torch.uint8, plain.wq)
    s_w = Guarded(plain.s_w.shape, torch.float32, plain.s_w)
    dbuf = Guarded(plain.dbuf.shape, torch.float32, plain.dbuf)
    return fq.Layer(wq.t, s_w.t, dbuf.t, r)


@pytest.mark.parametrize("m,n,r,T,k,per_row", [(272, 208, 24, 77, 19, False), (1040, 528, 72, 130, 1040, False),
                                               (144, 400, 8, 1, 5, False), (640, 1296, 64, 333, 133, True)])
def test_no_call_writes_outside_its_buffers(m, n, r, T, k, per_row):
    from paper_2510_24061_b200 import binding as fq
    Guarded.all = []
    layer = _guarded_layer(fq, 41, m, n, r, per_row)
    X = synth.activations(41, 0, T, n, 2).to(DEV)
    dY = synth.out_grad(41, 0, 0, T, m).to(DEV)
    ws = Guarded((fq.workspace_bytes(m, n, r, T),), torch.uint8)
    ws.t.zero_()
    fq.workspace_init(ws.t)
    Y, OA = Guarded((T, m), torch.bfloat16), Guarded((T, r), torch.float32)
    amax_oa, s_x = Guarded((1,), torch.float32), Guarded((1,), torch.float32)
    fq.melded_forward(layer, X, ws=ws.t, out=(Y.t, OA.t, amax_oa.t, s_x.t))
    dX, dB, s_g = Guarded((T, n), torch.bfloat16), Guarded((m, r), torch.float32), Guarded((1,), torch.float32)
    fq.melded_backward(layer, dY, OA.t, amax_oa.t, ws=ws.t, out=(dX.t, dB.t, s_g.t))
    idx = Guarded((max(k, 1),), torch.int32)
    fq.proxy_update(layer, dB.t, 2e-2, k, ws=ws.t, idx_out=idx.t[:k])
    # a second layer and a batched call; then the exact merge with its scratch; the absmax call
    layer2 = _guarded_layer(fq, 42, m, n, r, per_row)
    ws2 = Guarded((fq.workspace_bytes(m, n, r, 1),), torch.uint8)
    ws2.t.zero_()
    fq.workspace_init(ws2.t)
    k2 = min(k, 7)
    idx_a, idx_b = Guarded((max(k, 1),), torch.int32), Guarded((k2,), torch.int32)
    fq.proxy_update_batched([layer, layer2], [dB.t, dB.t], 2e-2, [k, k2], wss=[ws.t, ws2.t], idx_outs=[idx_a.t[:k], idx_b.t])
    scratch = Guarded((int(fq.lib.falqon_exact_merge_scratch_bytes(m, n, r)),), torch.uint8)
    idx_x = Guarded((k2,), torch.int32)
    fq.proxy_update_exact(layer2, dB.t, 2e-2, k2, ws=ws2.t, idx_out=idx_x.t, scratch=scratch.t, want_count=False)
    am, ws3 = Guarded((1,), torch.float32), Guarded((8192,), torch.uint8)
    fq.absmax(X, out=am.t, ws=ws3.t)
    torch.cuda.synchronize()
    assert fq.last_device_status() == 0
    bad = [i for i, g in enumerate(Guarded.all) if not g.intact()]
    assert not bad, f"margins written for buffers {bad} (in order of creation)"
    assert float(am.t.item()) == float(X.float().abs().max().item())
