"""GPU parity of the correctly rounded merge (falqon_proxy_update_exact) against the oracle's exact merge: selected
indices, every byte of the backbone and every DeltaBuffer bit must agree, whatever the tensor cores' summation order.
The accumulated sums are also checked against their error bound (the guard band must hold with room to spare) and
the share of elements that needs the exact fallback must stay small."""
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


def _kappa(r):
    r_pad = (r + 63) // 64 * 64
    return np.float32(1.02) * np.float32(3 * r_pad + 8) * np.float32(2.0 ** -23)


def _check_sums(orc, sums, idx, wq_before, dprime, m, r):
    """|tensor-core sum - exact sum| against the guard band eps = kappa (|w| + sum|d'| max_j|a_jc|)."""
    dec = np.array([orc.decode(c, orc.E4M3) if (c & 0x7F) != 0x7F else 0.0 for c in range(256)])
    a = dec[wq_before[m:]]                                   # [r][n] float64
    w = dec[wq_before[idx]]                                  # [k][n]
    exact = w + dprime.astype(np.float64) @ a               # products exact in fp64, 256 terms: error ~1e-16 relative
    eps = float(_kappa(r)) * (np.abs(w) + np.abs(dprime.astype(np.float64)).sum(axis=1, keepdims=True) * np.abs(a).max(axis=0))
    ratio = np.abs(sums.astype(np.float64) - exact) / np.maximum(eps, 1e-300)
    return float(ratio.max())


def _run(fq, orc, seed, m, n, r, k, lr, per_row=False, dbuf_scale=0.05, want_sums=True):
    W, A, _, _ = layer_inputs(seed, 0, m, n, r, 16, 0)
    if per_row:
        W = synth.backbone(seed, 0, m, n, heavy_tailed=True)
    layer = fq.setup_layer(W.to(DEV), A.to(DEV), None, 1.0, per_row=per_row)
    layer.dbuf.copy_(synth.normal_bf16(seed, 50, (m, r), dbuf_scale).float().to(DEV) * 1.0009765625)
    dB = (synth.normal_bf16(seed, 51, (m, r), 1.0).float() * 0.337).to(DEV)
    wq_before, dbuf_before = u8(layer.wq).copy(), f32(layer.dbuf).copy()
    row_scales = f32(layer.s_w) if per_row else None
    idx, fixed, sums = fq.proxy_update_exact(layer, dB, lr, k, want_sums=want_sums)
    wq_o, dbuf_o = wq_before.copy(), dbuf_before.copy()
    idx_o, _ = orc.proxy_update_exact(wq_o, dbuf_o, f32(dB), lr, k, m, r, row_scales=row_scales)
    assert np.array_equal(u8(idx), idx_o)
    assert np.array_equal(bits32(f32(layer.dbuf)), bits32(dbuf_o))
    got = u8(layer.wq)
    assert np.array_equal(got, wq_o), f"{int((got != wq_o).sum())} codes differ"
    assert fq.last_device_status() == 0
    n_fixed = int(fixed.item())
    if want_sums and k > 0:
        d_after_opt = (np.float32(-lr) * f32(dB).astype(np.float64) + dbuf_before.astype(np.float64)).astype(np.float32)  # one fma each
        dprime = d_after_opt[idx_o]
        if per_row:
            coef = (row_scales[idx_o] / row_scales[m]).astype(np.float32)
            dprime = (dprime * coef[:, None]).astype(np.float32)
        worst = _check_sums(orc, f32(sums), idx_o, wq_before, dprime, m, r)
        print(f"[exact merge m={m} n={n} r={r} k={k}] worst |S - exact| / eps = {worst:.4f}, exact path {n_fixed} of {k * n}")
        assert worst < 0.5, f"accumulated sums use {worst:.3f} of the guard band"
    return n_fixed, k * n


@pytest.mark.parametrize("m,n,r,k", [(256, 128, 16, 40), (272, 208, 8, 272), (144, 400, 24, 17), (512, 256, 256, 64),
                                     (1040, 528, 72, 1), (640, 1280, 64, 133)])
def test_exact_merge_matches_the_oracle(fq, orc, m, n, r, k):
    fixed, total = _run(fq, orc, 61, m, n, r, k, 2e-2)
    # the guard band grows with r and with the size of the DeltaBuffer entries (these are 100x a training step's)
    assert fixed <= (0.25 if r > 128 else 0.05) * total + 16, f"{fixed} of {total} elements took the exact path"


@pytest.mark.parametrize("m,n,r,k", [(640, 1280, 64, 33), (272, 208, 8, 100)])
def test_exact_merge_per_row_scales(fq, orc, m, n, r, k):
    _run(fq, orc, 62, m, n, r, k, 2e-2, per_row=True)


def test_ties_tiny_terms_and_saturation_take_the_exact_path(fq, orc):
    """Sums that sit exactly on rounding boundaries, terms of 2^-140 that decide them, rows with entries below the
    smallest limb, and sums far beyond +-448."""
    m, n, r = 128, 64, 8
    enc = lambda v: orc.encode(float(v), orc.E4M3)
    wq = np.zeros((m + r, n), dtype=np.uint8)
    wq[:m, 0::2] = enc(8.0)
    wq[:m, 1::2] = enc(9.0)
    wq[m:] = enc(1.0)                                  # every A~ entry is 1: sum = w + sum_j d_j
    wq[m + 1, 1::4] = enc(-1.5)
    dbuf = np.zeros((m, r), dtype=np.float32)
    dbuf[0::4, 0] = 0.5                                # 8.5, 9.5: ties
    dbuf[1::4, 0] = 0.5; dbuf[1::4, 2] = 2.0 ** -140   # tie broken upwards by a term fp32 cannot add
    dbuf[2::4, 0] = -0.5; dbuf[2::4, 3] = -2.0 ** -149
    dbuf[3::4, 0] = 3.0e4; dbuf[3::4, 1] = -1.0e-3     # saturation (and for columns with -1.5: mixed signs)
    dbuf[5, :] = [2.0 ** 60, -2.0 ** 60, 0.75, 0, 0, 0, 0, 0]
    s_w = torch.ones(1, dtype=torch.float32, device=DEV)
    layer = fq.Layer(torch.from_numpy(wq).to(DEV), s_w, torch.from_numpy(dbuf).to(DEV), r)
    wq_o, dbuf_o = wq.copy(), dbuf.copy()
    idx, fixed, _ = fq.proxy_update_exact(layer, None, 0.0, m)
    idx_o, _ = orc.proxy_update_exact(wq_o, dbuf_o, None, 0.0, m, m, r)
    assert np.array_equal(u8(idx), idx_o) and np.array_equal(u8(layer.wq), wq_o)
    assert not f32(layer.dbuf).any()
    assert int(fixed.item()) >= (m // 4) * n * 3 - n   # the tie rows and the tiny-term rows cannot be decided in fp32
    # spot values: 8.5 -> 8 (even), 9.5 -> 10, 8.5 + 2^-140 -> 9
    out = u8(layer.wq)
    assert out[0, 0] == enc(8.0) and out[0, 3] == enc(10.0) and out[1, 0] == enc(9.0)


@pytest.mark.parametrize("name,n,m,r,k", [("q", 4096, 4096, 64, 256), ("gate, largest sweep point", 4096, 11008, 128, 4096)])
def test_exact_merge_full_size(fq, orc, name, n, m, r, k):
    fixed, total = _run(fq, orc, 63, m, n, r, k, 2e-4, dbuf_scale=1e-3, want_sums=False)
    assert fixed <= 0.02 * total, f"{fixed} of {total} elements took the exact path"


@pytest.mark.parametrize("prepared", [True, False])
def test_batched_exact_equals_per_layer_calls_and_the_oracle(fq, orc, prepared):
    """falqon_proxy_update_batched_exact: layers of different shapes, ranks, granularities and k (one with k = 0, one with
    adversarially large DeltaBuffer entries so that many elements take the exact path) in one call, twice in a row (the
    second call reuses the prepared copy of A~): bit-identical to the per-layer falqon_proxy_update_exact calls and to the
    oracle's exact merge."""
    specs = [(512, 384, 16, 40, False, 0.05), (272, 528, 64, 0, False, 0.05), (1024, 256, 128, 300, True, 0.05),
             (384, 640, 8, 384, False, 5.0)]
    lr = 0.05
    per, bat, dBs, ks, oracle_state = [], [], [], [], []
    for i, (m, n, r, k, per_row, scale) in enumerate(specs):
        W, A, _, _ = layer_inputs(61, i, m, n, r, 16, 0)
        if per_row:
            W = synth.backbone(61, i, m, n, heavy_tailed=True)
        a = fq.setup_layer(W.to(DEV), A.to(DEV), None, 1.0, per_row=per_row)
        a.dbuf.copy_(synth.normal_bf16(61, 50 + i, (m, r), scale).float().to(DEV) * 1.0009765625)
        b = fq.Layer(a.wq.clone(), a.s_w.clone(), a.dbuf.clone(), r)
        per.append(a); bat.append(b); ks.append(k)
        oracle_state.append((u8(a.wq).copy(), f32(a.dbuf).copy(), f32(a.s_w) if per_row else None))
    batch = None
    for call in range(2):
        dBs = [(synth.normal_bf16(61, 70 + 10 * call + i, (L.m, L.r), 1.0).float() * 0.337).to(DEV) for i, L in enumerate(per)]
        idx_per = [fq.proxy_update_exact(L, dB, lr, k, want_count=False)[0] for L, dB, k in zip(per, dBs, ks)]
        if batch is None:
            batch = fq.ProxyBatch(bat, dBs, ks)
            batch.prepare_exact()
        else:
            batch = fq.ProxyBatch(bat, dBs, ks)
            batch.scratch, batch.c_scratch, batch.c_scratch_bytes = keep
        keep = (batch.scratch, batch.c_scratch, batch.c_scratch_bytes)
        idx_bat = batch.run_exact(lr, prepared=prepared)
        torch.cuda.synchronize()
        for i, (La, Lb, ia, ib) in enumerate(zip(per, bat, idx_per, idx_bat)):
            assert (ia is None and ib is None) or torch.equal(ia, ib), f"layer {i} call {call}: selected rows"
            assert torch.equal(La.wq, Lb.wq), f"layer {i} call {call}: {int((La.wq != Lb.wq).sum())} codes differ"
            assert torch.equal(La.dbuf.view(torch.int32), Lb.dbuf.view(torch.int32))
            wq_o, dbuf_o, rs = oracle_state[i]
            orc.proxy_update_exact(wq_o, dbuf_o, f32(dBs[i]), lr, ks[i], La.m, La.r, row_scales=rs)
            assert np.array_equal(u8(Lb.wq), wq_o) and np.array_equal(bits32(f32(Lb.dbuf)), bits32(dbuf_o))
    assert fq.last_device_status() == 0
