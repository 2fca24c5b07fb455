"""GPU parity of falqon_proxy_update_batched (the proxy update of several layers in two launches) against the
oracle's proxy update run layer by layer: indices, every byte of every backbone and every DeltaBuffer bit."""
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


def _make(fq, seed, i, m, n, r, per_row):
    W, A, _, _ = layer_inputs(seed, i, m, n, r, 16, 0)
    if per_row:
        W = synth.backbone(seed, i, m, n, heavy_tailed=True)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), None, 1.0, per_row=per_row)
    layer.dbuf.copy_(synth.normal_bf16(seed, 50 + 16 * i, (m, r), 0.05).float().to(DEV))
    dB = (synth.normal_bf16(seed, 51 + 16 * i, (m, r), 1.0).float() * 0.337).to(DEV)
    return layer, dB


def _check_against_oracle(fq, orc, specs, lr, seed, steps=1):
    """specs: (m, n, r, k, per_row, with_dB) per layer."""
    made = [_make(fq, seed, i, m, n, r, per_row) for i, (m, n, r, k, per_row, _) in enumerate(specs)]
    layers = [l for l, _ in made]
    dBs = [dB if spec[5] else None for (_, dB), spec in zip(made, specs)]
    ks = [spec[3] for spec in specs]
    batch = fq.ProxyBatch(layers, dBs, ks)
    for step in range(steps):
        before = [(u8(l.wq).copy(), f32(l.dbuf).copy()) for l in layers]
        idxs = batch.run(lr)
        for i, (layer, spec) in enumerate(zip(layers, specs)):
            m, n, r, k, per_row, with_dB = spec
            wq_o, dbuf_o = before[i]
            idx_o, _ = orc.proxy_update(wq_o, dbuf_o, f32(dBs[i]) if with_dB else None, lr, k, m, r,
                                        row_scales=f32(layer.s_w) if per_row else None)
            if k > 0:
                assert np.array_equal(u8(idxs[i]), idx_o), f"layer {i} step {step}: indices"
            assert np.array_equal(u8(layer.wq), wq_o), f"layer {i} step {step}: backbone"
            assert np.array_equal(bits32(f32(layer.dbuf)), bits32(dbuf_o)), f"layer {i} step {step}: DeltaBuffer"
    assert fq.last_device_status() == 0


def test_mixed_layers_match_the_oracle(fq, orc):
    """Different shapes, ranks and k in one call; a per-row layer; a layer without an optimizer step; k = 0 and k = m;
    a ragged last column tile and a ragged last row group; two steps, so the control words must be back at zero."""
    specs = [(256, 128, 16, 40, False, True), (272, 208, 8, 272, False, True), (144, 400, 24, 0, False, True),
             (640, 1280, 64, 133, True, True), (512, 256, 32, 17, False, False), (1040, 528, 72, 1, False, True)]
    _check_against_oracle(fq, orc, specs, 2e-2, 71, steps=2)


def test_more_layers_than_one_launch_takes(fq, orc):
    specs = [(128 + 16 * i, 128 + 32 * (i % 3), 8 * (1 + i % 4), 5 + 3 * i, i % 5 == 4, True) for i in range(11)]
    _check_against_oracle(fq, orc, specs, 5e-2, 72)


def test_all_layers_with_k_zero_and_an_empty_call(fq, orc):
    specs = [(256, 128, 16, 0, False, True), (128, 256, 8, 0, False, True)]
    _check_against_oracle(fq, orc, specs, 1e-2, 73)
    assert fq.proxy_update_batched([], [], 0.1, []) == []


def test_batched_equals_per_layer_calls_on_the_7b_projection_set(fq):
    """The seven projections of configs[1] (r = 64, k = 256): one batched call against seven single calls, bit for bit."""
    c = synth.config1()
    shapes = [(m, n) for _, n, m in c["linears"]]
    r, k, lr = c["r"], c["k"], c["lr"]
    a, b = [], []
    for i, (m, n) in enumerate(shapes):
        layer, dB = _make(fq, 74, i, m, n, r, False)
        a.append((layer, dB))
        twin = fq.Layer(layer.wq.clone(), layer.s_w.clone(), layer.dbuf.clone(), r)
        b.append((twin, dB))
    idx_a = fq.proxy_update_batched([l for l, _ in a], [d for _, d in a], lr, [k] * len(a))
    for i, (twin, dB) in enumerate(b):
        idx_b = fq.proxy_update(twin, dB, lr, k)
        assert torch.equal(idx_a[i], idx_b)
        assert torch.equal(a[i][0].wq, twin.wq)
        assert torch.equal(a[i][0].dbuf.view(torch.int32), twin.dbuf.view(torch.int32))
    assert fq.last_device_status() == 0


def test_invalid_entries_reject_the_whole_call(fq):
    l0, dB0 = _make(fq, 75, 0, 128, 128, 8, False)
    l1, dB1 = _make(fq, 75, 1, 128, 128, 8, False)
    wq_before = l0.wq.clone()
    with pytest.raises(fq.FalqonError) as e:
        fq.proxy_update_batched([l0, l1], [dB0, dB1], 0.1, [4, 129])          # k > m in the second layer
    assert e.value.status == fq.ERR_INVALID_ARG
    with pytest.raises(fq.FalqonError):
        fq.proxy_update_batched([l0, l0], [dB0, dB0], 0.1, [4, 4])            # the same layer twice
    ws = l0.workspace(1)
    with pytest.raises(fq.FalqonError):
        fq.proxy_update_batched([l0, l1], [dB0, dB1], 0.1, [4, 4], wss=[ws, ws])   # a shared workspace
    torch.cuda.synchronize()
    assert torch.equal(l0.wq, wq_before)


def test_batched_adamw_equals_per_layer_calls_and_the_oracle(fq, orc):
    """Three AdamW steps on four layers of different shapes: one batched call per step against one call per layer, bit
    for bit (backbone, DeltaBuffer, both moments, indices); the first layer is also checked against the oracle."""
    specs = [(256, 128, 16, 40), (640, 1280, 64, 133), (144, 400, 24, 0), (512, 256, 32, 512)]
    hp = dict(lr=3e-3, beta1=0.9, beta2=0.99, eps=1e-8, weight_decay=0.01)
    a, b = [], []
    for i, (m, n, r, k) in enumerate(specs):
        layer, _ = _make(fq, 76, i, m, n, r, False)
        twin = fq.Layer(layer.wq.clone(), layer.s_w.clone(), layer.dbuf.clone(), r)
        z = lambda: torch.zeros((m, r), dtype=torch.float32, device=DEV)
        a.append(dict(layer=layer, ea=z(), es=z()))
        b.append(dict(layer=twin, ea=z(), es=z()))
    dBs = [torch.empty((m, r), dtype=torch.float32, device=DEV) for m, _, r, _ in specs]
    batch = fq.ProxyBatch([x["layer"] for x in a], dBs, [s[3] for s in specs])
    m0, n0, r0, k0 = specs[0]
    wq_o, dbuf_o = u8(a[0]["layer"].wq).copy(), f32(a[0]["layer"].dbuf).copy()
    ea_o, es_o = np.zeros((m0, r0), np.float32), np.zeros((m0, r0), np.float32)
    for step in (1, 2, 3):
        for i, (m, n, r, k) in enumerate(specs):
            dBs[i].copy_((synth.normal_bf16(76, 300 + 16 * i + step, (m, r), 1.0).float() * 0.3).to(DEV))
        idx_a = batch.run_adamw([x["ea"] for x in a], [x["es"] for x in a], step=step, **hp)
        for i, (m, n, r, k) in enumerate(specs):
            idx_b = fq.proxy_update_adamw(b[i]["layer"], dBs[i], b[i]["ea"], b[i]["es"], step, k, **hp)
            if k > 0:
                assert torch.equal(idx_a[i], idx_b), f"layer {i} step {step}: indices"
            assert torch.equal(a[i]["layer"].wq, b[i]["layer"].wq), f"layer {i} step {step}: backbone"
            for what, x, y in (("DeltaBuffer", a[i]["layer"].dbuf, b[i]["layer"].dbuf), ("exp_avg", a[i]["ea"], b[i]["ea"]),
                               ("exp_avg_sq", a[i]["es"], b[i]["es"])):
                assert torch.equal(x.view(torch.int32), y.view(torch.int32)), f"layer {i} step {step}: {what}"
        orc.adamw_step(dbuf_o, f32(dBs[0]), ea_o, es_o, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], step)
        idx_o, _ = orc.proxy_update(wq_o, dbuf_o, None, 0.0, k0, m0, r0)
        assert np.array_equal(u8(idx_a[0]), idx_o) and np.array_equal(u8(a[0]["layer"].wq), wq_o)
        assert np.array_equal(bits32(f32(a[0]["layer"].dbuf)), bits32(dbuf_o))
        assert np.array_equal(bits32(f32(a[0]["ea"])), bits32(ea_o)) and np.array_equal(bits32(f32(a[0]["es"])), bits32(es_o))
    assert fq.last_device_status() == 0


def test_ctas_that_walk_several_row_groups(fq, orc):
    """Eight layers of ten column tiles each and many selected rows: the launch has more (column tile, row group) pairs
    than resident CTAs, so every CTA walks two or three row groups (prefetch of the next group, ring of row indices,
    late clearing of the DeltaBuffer rows), with a ragged last group and a ragged last column tile, per-tensor and
    per-row layers mixed."""
    specs = [(656 + 16 * i, 1264, 16, 600 + 7 * i, i % 3 == 2, True) for i in range(8)]
    _check_against_oracle(fq, orc, specs, 2e-2, 77, steps=2)


def test_single_layer_call_whose_ctas_walk_several_row_groups(fq, orc):
    """falqon_proxy_update on one wide layer with every row selected (the set-up meld): 32 column tiles x 64 row groups
    exceed the resident CTAs, so each CTA of the single-layer merge kernel walks three or four row groups."""
    m, n, r = 2048, 4096, 16
    layer, dB = _make(fq, 78, 0, m, n, r, False)
    wq_o, dbuf_o = u8(layer.wq).copy(), f32(layer.dbuf).copy()
    idx = fq.proxy_update(layer, dB, 5e-2, m)
    idx_o, _ = orc.proxy_update(wq_o, dbuf_o, f32(dB), 5e-2, m, m, r)
    assert np.array_equal(u8(idx), idx_o)
    assert np.array_equal(u8(layer.wq), wq_o)
    assert not f32(layer.dbuf).any() and not dbuf_o.any()
    assert fq.last_device_status() == 0
