"""The library's calls only enqueue kernels on the caller's stream (no allocation, no synchronisation, tensor maps passed
by value), so a whole step can be captured into a CUDA graph and replayed: forward, backward and the batched proxy
update of two layers, captured once and replayed three times, against the same three steps run call by call on twin
layers -- bit for bit."""
import pytest
import torch

from helpers import layer_inputs
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _make(fq, seed, i, m, n, r, T):
    W, A, B, X = layer_inputs(seed, i, m, n, r, T, 2)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), B.to(DEV), 1.0)
    dY = synth.out_grad(seed, i, 0, T, m).to(DEV)
    ws = layer.workspace(T)
    out_f = (torch.empty((T, m), dtype=torch.bfloat16, device=DEV), torch.empty((T, r), dtype=torch.float32, device=DEV),
             torch.empty(1, dtype=torch.float32, device=DEV), torch.empty(1, dtype=torch.float32, device=DEV))
    out_b = (torch.empty((T, n), dtype=torch.bfloat16, device=DEV), torch.empty((m, r), dtype=torch.float32, device=DEV),
             torch.empty(1, dtype=torch.float32, device=DEV))
    return dict(layer=layer, X=X.to(DEV), dY=dY, ws=ws, out_f=out_f, out_b=out_b)


def _step(fq, Ls, batch, lr):
    for L in Ls:
        _, OA, amax_oa, _ = fq.melded_forward(L["layer"], L["X"], ws=L["ws"], out=L["out_f"])
        fq.melded_backward(L["layer"], L["dY"], OA, amax_oa, ws=L["ws"], out=L["out_b"])
    batch.run(lr)


def test_a_captured_step_replays_bit_for_bit():
    from paper_2510_24061_b200 import binding as fq
    shapes = [(512, 384, 16, 200), (400, 640, 32, 200)]
    k, lr = 24, 2e-2
    sets = []
    for _ in range(2):     # two identical sets of layers: one replayed from a graph, one run call by call
        Ls = [_make(fq, 51, i, m, n, r, T) for i, (m, n, r, T) in enumerate(shapes)]
        batch = fq.ProxyBatch([L["layer"] for L in Ls], [L["out_b"][1] for L in Ls], [k] * len(Ls), wss=[L["ws"] for L in Ls])
        sets.append((Ls, batch))
    (Lg, bg), (Le, be) = sets
    # warm-up on a side stream (kernel attributes are set on first use), then undo its effect on the layer state
    saved = [(L["layer"].wq.clone(), L["layer"].dbuf.clone()) for L in Lg]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        _step(fq, Lg, bg, lr)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for L, (wq, dbuf) in zip(Lg, saved):
        L["layer"].wq.copy_(wq)
        L["layer"].dbuf.copy_(dbuf)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        _step(fq, Lg, bg, lr)
    # the capture itself runs nothing: restore is not needed; now three replays against three eager steps
    for step in range(3):
        graph.replay()
        _step(fq, Le, be, lr)
        torch.cuda.synchronize()
        for a, b in zip(Lg, Le):
            assert torch.equal(a["layer"].wq, b["layer"].wq), f"step {step}: backbone"
            assert torch.equal(a["layer"].dbuf.view(torch.int32), b["layer"].dbuf.view(torch.int32)), f"step {step}: DeltaBuffer"
            assert torch.equal(a["out_f"][0], b["out_f"][0]) and torch.equal(a["out_b"][0], b["out_b"][0])
            assert torch.equal(a["out_b"][1].view(torch.int32), b["out_b"][1].view(torch.int32))
    assert fq.last_device_status() == 0


def test_the_benchmarks_graph_replay_equals_call_by_call_at_full_size():
    """configs[1] exactly as bench.py runs it (the seven 7B projections, 4096 tokens, rank 64, top-256, batched proxy
    update): two replays of the captured step against two steps run call by call on a twin workload, bit for bit."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    from paper_2510_24061_b200 import binding as fq
    c = synth.config1()
    T, r, k, lr = c["T"], c["r"], c["k"], c["lr"]
    sets = []
    for _ in range(2):
        layers = bench.build_workload(fq, torch.device(DEV), c["seed"], T, r, k, c["linears"], c["outlier_frac"])
        sets.append((layers, bench.make_proxy_batch(fq, layers, k)))
    (Lg, bg), (Le, be) = sets
    bench.run_step(fq, Lg, lr, k, bg)          # first use of every kernel happens outside the capture
    bench.run_step(fq, Le, lr, k, be)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        bench.run_step(fq, Lg, lr, k, bg)
    for step in range(2):
        graph.replay()
        bench.run_step(fq, Le, lr, k, be)
        torch.cuda.synchronize()
        for a, b in zip(Lg, Le):
            assert torch.equal(a["layer"].wq, b["layer"].wq), f"{a['name']} step {step}: backbone"
            assert torch.equal(a["layer"].dbuf.view(torch.int32), b["layer"].dbuf.view(torch.int32)), f"{a['name']}: DeltaBuffer"
            assert torch.equal(a["out_f"][0], b["out_f"][0]) and torch.equal(a["out_b"][0], b["out_b"][0]), f"{a['name']}: Y / dX"
            assert torch.equal(a["idx"], b["idx"]), f"{a['name']}: selected rows"
    assert fq.last_device_status() == 0


def test_a_captured_stack_step_replays_bit_for_bit():
    """The same for the chained stack in its default form: chain kernels that cast their own results (cooperative launches
    with a grid barrier), products that carry the adapter gradient and the O_A cast, one batched proxy update per block --
    two steps as replays of one captured graph against two steps run call by call on a twin stack."""
    from paper_2510_24061_b200 import binding as fq
    from paper_2510_24061_b200 import stack as st
    H, F, T, r, k = 256, 512, 300, 16, 24
    h0 = synth.normal_bf16(5, 9001, (T, H), 1.0, DEV)
    G = synth.normal_bf16(5, 9002, (T, H), 1.0e-2, DEV)
    eager = st.Stack(2, H, F, T, r, k, seed=5, device=DEV, lr=2e-2)
    graphed = st.Stack(2, H, F, T, r, k, seed=5, device=DEV, lr=2e-2)
    assert eager.fuse_cast and graphed.fuse_cast
    state = [(L.wq.clone(), L.dbuf.clone()) for blk in graphed.layers for L in blk.values()]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):          # warm-up (kernel attributes are set on first use) ...
        graphed.step(h0, G)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for L, (wq, dbuf) in zip([L for blk in graphed.layers for L in blk.values()], state):   # ... and its effect undone
        L.wq.copy_(wq)
        L.dbuf.copy_(dbuf)
    graphed.steps_done = 0
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        graphed.step(h0, G)
    for _ in range(2):
        g.replay()
        eager.step(h0, G)
    torch.cuda.synchronize()
    assert torch.equal(graphed.h_out.view(torch.int16), eager.h_out.view(torch.int16))
    assert torch.equal(graphed.dh.view(torch.int16), eager.dh.view(torch.int16))
    for bg, be in zip(graphed.layers, eager.layers):
        for name in bg:
            assert torch.equal(bg[name].wq, be[name].wq), name
            assert torch.equal(bg[name].dbuf.view(torch.int32), be[name].dbuf.view(torch.int32)), name
    assert fq.last_device_status() == 0
