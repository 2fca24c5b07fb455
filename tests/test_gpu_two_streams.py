"""Two layers driven from two streams at once.  The cast inside falqon_melded_forward / _backward is one kernel whose CTAs
wait for one another at a grid-wide barrier; it is launched cooperatively, so the driver starts each such kernel only when
its whole grid can be resident, whatever the other stream has running.  The results must be those of the same calls made
one after another, and no bounded wait may run out."""
import pytest
import torch

from helpers import layer_inputs
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_forward_and_backward_of_two_layers_on_two_streams():
    from paper_2510_24061_b200 import binding as fq
    shapes = [(1024, 2048, 32, 2048), (2048, 1024, 64, 1536)]
    layers, inputs, ref = [], [], []
    for i, (m, n, r, T) in enumerate(shapes):
        W, A, B, X = layer_inputs(71, i, m, n, r, T, 4, DEV)
        dY = synth.out_grad(71, i, 0, T, m, DEV)
        L = fq.setup_layer(W, A, B, 1.0)
        ws = L.workspace(T)
        layers.append((L, ws))
        inputs.append((X, dY))
        Y, OA, amax_oa, _ = fq.melded_forward(L, X, y_dtype=torch.float32, ws=ws)
        dX, dB, _ = fq.melded_backward(L, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
        ref.append((Y.clone(), OA.clone(), dX.clone(), dB.clone()))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [None, None]
    for rep in range(8):                       # interleave the enqueues so that the two streams really overlap
        for i, ((L, ws), (X, dY)) in enumerate(zip(layers, inputs)):
            with torch.cuda.stream(streams[i]):
                Y, OA, amax_oa, _ = fq.melded_forward(L, X, y_dtype=torch.float32, ws=ws)
                dX, dB, _ = fq.melded_backward(L, dY, OA, amax_oa, dx_dtype=torch.float32, ws=ws)
                outs[i] = (Y, OA, dX, dB)
    torch.cuda.synchronize()
    for got, want in zip(outs, ref):
        for a, b in zip(got, want):
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    assert fq.last_device_status() == 0


def test_quantizing_chain_kernels_on_two_streams():
    """The same for the chain kernels that cast their own result (one CTA per SM, a grid barrier in the middle): two
    streams, each with its own scratch, enqueue them alternately; codes and scales must equal those of the calls made alone."""
    from paper_2510_24061_b200 import binding as fq
    from paper_2510_24061_b200 import stack as st
    rows, cols = 2048, 4096
    xs = [synth.normal_bf16(72, 9100 + i, (rows, cols), 1.0 + i, DEV) for i in range(2)]
    res = [synth.normal_bf16(72, 9110 + i, (rows, cols), 0.5, DEV) for i in range(2)]
    def run(i, scratch):
        codes = torch.empty(rows * cols, dtype=torch.uint8, device=DEV)
        scale = torch.zeros(2, dtype=torch.float32, device=DEV)
        y16, s16 = torch.empty_like(xs[i]), torch.empty_like(xs[i])
        inv = torch.empty(rows, dtype=torch.float32, device=DEV)
        st.rmsnorm_quantize(codes, scale[0:1], fq.E4M3, y16, False, scratch, inv, xs[i], sum_out=s16, sa=1.0, b=res[i], sb=0.5)
        codes2 = torch.empty(rows * cols, dtype=torch.uint8, device=DEV)
        st.combine_quantize(codes2, scale[1:2], fq.E5M2, y16, False, scratch, s16, 0.25)
        return codes, codes2, scale, inv
    scratches = [st.chain_scratch(DEV) for _ in range(2)]
    ref = [run(i, scratches[i]) for i in range(2)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [None, None]
    for rep in range(8):
        for i in range(2):
            with torch.cuda.stream(streams[i]):
                outs[i] = run(i, scratches[i])
    torch.cuda.synchronize()
    for got, want in zip(outs, ref):
        assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
        assert torch.equal(got[2].view(torch.int32), want[2].view(torch.int32))
        assert torch.equal(got[3].view(torch.int32), want[3].view(torch.int32))
    assert all(int(s.view(torch.int32)[:2].abs().sum()) == 0 for s in scratches)
    assert fq.last_device_status() == 0
