"""falqon_proxy_update_static: the proxy update whose scratch is a fixed array inside the library,
for callers that cannot allocate a workspace (guests of a runtime whose allocator owns the device).

Collected last on purpose.  The GPU test drives the new entry point through the C ABI next to the
workspace-taking falqon_proxy_update on identical inputs, twice in a row (the second call finds the
first call's leftovers in the shared array), and wants identical bytes: merged backbone rows,
DeltaBuffer and selected indices are all bit-exact stages.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2510_24061_b200 import synth


def _fq():
    from paper_2510_24061_b200 import build
    build.build()
    from paper_2510_24061_b200 import binding
    return binding


def test_static_variant_rejects_oversized_and_bad_arguments():
    fq = _fq()
    fake = 0x10000
    too_big = fq.falqon_layer(fq.STATIC_MAX_ROWS + 16, 256, 16, fake, fake, fake, 0, 0)
    assert fq.lib.falqon_proxy_update_static(C.byref(too_big), None, 0.1, 1, None, None) == fq.ERR_UNSUPPORTED
    ok_shape = fq.falqon_layer(256, 256, 16, fake, fake, fake, 0, 0)
    assert fq.lib.falqon_proxy_update_static(C.byref(ok_shape), None, 0.1, 257, None, None) == fq.ERR_INVALID_ARG
    assert fq.lib.falqon_proxy_update_static(None, None, 0.1, 1, None, None) == fq.ERR_INVALID_ARG


@pytest.mark.gpu
def test_static_variant_matches_workspace_variant_on_two_calls():
    fq = _fq()
    dev = "cuda:0"
    m, n, r, k = 1024, 512, 32, 48
    W = synth.backbone(21, 0, m, n, dev)
    A = synth.adapter_a(21, 0, r, n, dev)
    B = synth.adapter_b(21, 0, m, r, dev)
    ref = fq.setup_layer(W, A, B, 1.0)
    new = fq.Layer(ref.wq.clone(), ref.s_w.clone(), ref.dbuf.clone(), r)
    for call, lr in enumerate((0.05, 0.5)):
        dB = synth.normal_bf16(21, 50 + call, (m, r), 1.0, dev).float()
        idx_ref = fq.proxy_update(ref, dB, lr, k)
        idx_new = fq.proxy_update_static(new, dB, lr, k)
        torch.cuda.synchronize()
        assert torch.equal(idx_ref, idx_new), f"selected rows differ on call {call}"
        assert torch.equal(ref.wq, new.wq), f"merged backbone differs on call {call}"
        assert torch.equal(ref.dbuf.view(torch.int32), new.dbuf.view(torch.int32)), f"DeltaBuffer differs on call {call}"
        assert (ref.dbuf[idx_ref.long()] == 0).all()
    # optimizer-only call (k = 0) and a caller-provided index buffer
    dB = synth.normal_bf16(21, 60, (m, r), 1.0, dev).float()
    fq.proxy_update(ref, dB, 0.1, 0)
    fq.proxy_update_static(new, dB, 0.1, 0)
    out = torch.empty(m, dtype=torch.int32, device=dev)
    fq.proxy_update_static(new, None, 0.0, m, idx_out=out)
    fq.proxy_update(ref, None, 0.0, m)
    torch.cuda.synchronize()
    assert torch.equal(out.cpu(), torch.arange(m, dtype=torch.int32))
    assert torch.equal(ref.wq, new.wq) and not new.dbuf.any()
    assert fq.last_device_status() == 0


@pytest.mark.gpu
@pytest.mark.parametrize("k", [1, 300, 16384])
def test_static_variant_at_its_row_limit_against_the_oracle(k):
    """m = FALQON_STATIC_MAX_ROWS: the selection kernel of this path then needs its opted-in 64 KB of shared memory and
    16 rows per thread.  Narrow rows keep the oracle quick.  Duplicated DeltaBuffer rows give tied scores, which must
    go to the lower index.  Checked against the CPU oracle and against the workspace entry point, bit for bit."""
    fq = _fq()
    from oracle import falqon_oracle as orc
    dev = "cuda:0"
    m, n, r, lr = fq.STATIC_MAX_ROWS, 128, 8, 0.25
    W = synth.backbone(22, 0, m, n, dev)
    A = synth.adapter_a(22, 0, r, n, dev)
    ref = fq.setup_layer(W, A, None, 1.0)
    dB = synth.normal_bf16(22, 70, (m, r), 1.0, dev).float()
    dB[1::2] = dB[0::2]                       # every odd row repeats the row before it: 8192 pairs of tied scores
    new = fq.Layer(ref.wq.clone(), ref.s_w.clone(), ref.dbuf.clone(), r)
    wq_o, dbuf_o = ref.wq.cpu().numpy().copy(), ref.dbuf.cpu().numpy().copy()
    idx_ref = fq.proxy_update(ref, dB, lr, k)
    idx_new = fq.proxy_update_static(new, dB, lr, k)
    idx_o, _ = orc.proxy_update(wq_o, dbuf_o, dB.cpu().numpy(), lr, k, m, r)
    torch.cuda.synchronize()
    assert np.array_equal(idx_new.cpu().numpy(), idx_o), "selected rows differ from the oracle"
    assert np.array_equal(new.wq.cpu().numpy(), wq_o), "merged rows differ from the oracle"
    assert np.array_equal(new.dbuf.cpu().numpy().view(np.uint32), dbuf_o.view(np.uint32)), "DeltaBuffer differs from the oracle"
    assert torch.equal(idx_ref, idx_new) and torch.equal(ref.wq, new.wq)
    assert torch.equal(ref.dbuf.view(torch.int32), new.dbuf.view(torch.int32))
    if k == 300:   # ties went to the lower index: an odd row is selected only together with its even twin
        chosen = set(idx_o.tolist())
        assert all((i - 1) in chosen for i in chosen if i % 2 == 1)
    assert fq.last_device_status() == 0
