"""GPU parity of the decoder-shaped chain of melded layers (the "32-layer stack" configuration).

The element-wise chain kernels are checked against the same formulas in fp32 on the CPU.  Every checked
projection inside the chain is teacher-forced like the single-layer tests: the oracle is fed the tensors the GPU
actually saw at that point of the step (captured copies), so each stage is compared in isolation.  Outputs
inside the chain are bf16, so tensor-core results are compared with the oracle's fp32 result at bf16 resolution:
within one bf16 step of it, and equal to its bf16 rounding on all but a small fraction of elements.
"""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, product_close, rel_fro, u8
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def fq():
    from paper_2510_24061_b200 import binding
    return binding


@pytest.fixture(scope="module")
def st():
    from paper_2510_24061_b200 import stack
    return stack


@pytest.fixture(scope="module")
def orc():
    from oracle import falqon_oracle
    return falqon_oracle


def _bf16_steps(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """Distance between two bf16 tensors in representable steps (monotone integer mapping of the bit patterns)."""
    def key(t):
        i = t.contiguous().view(torch.int16).to(torch.int32)
        return torch.where(i < 0, -(i & 0x7FFF), i)
    return (key(a) - key(b)).abs()


def test_chain_elementwise_kernels(st):
    torch.manual_seed(0)
    n = 8 * 4099
    a, b, c, d = [(torch.randn(n) * s).to(torch.bfloat16) for s in (1.0, 0.5, 2.0, 0.1)]
    ad, bd, cd, dd = [t.to(DEV) for t in (a, b, c, d)]
    out = torch.empty_like(ad)
    amax = torch.zeros(4, dtype=torch.float32, device=DEV)
    st.combine(out, ad, 0.5, bd, -1.25, cd, 3.0 ** -0.5, dd, 1.0, amax=amax[0:1])
    assert float(amax[0]) == float(out.float().abs().max())
    acc = a.double() * np.float32(0.5)
    for s, t in ((np.float32(-1.25), b), (np.float32(3.0 ** -0.5), c), (np.float32(1.0), d)):
        acc = (acc.float().double() + float(s) * t.double())      # fp32 fma chain: one rounding per step
    ref = acc.float().to(torch.bfloat16)
    assert int(_bf16_steps(out.cpu(), ref).max()) <= 1 and float((out.cpu() != ref).float().mean()) < 1e-3
    st.combine(out, ad, 2.0 ** -0.5)
    assert torch.equal(out.cpu(), (a.float() * np.float32(2.0 ** -0.5)).to(torch.bfloat16))
    z = torch.empty_like(ad)
    st.silu_mul(z, ad, bd, amax=amax[1:2])
    assert float(amax[1]) == float(z.float().abs().max())
    ref = (a.float() * torch.sigmoid(a.float()) * b.float()).to(torch.bfloat16)
    assert int(_bf16_steps(z.cpu(), ref).max()) <= 1 and float((z.cpu() != ref).float().mean()) < 2e-2
    dg, du = torch.empty_like(ad), torch.empty_like(ad)
    st.silu_mul_grad(dg, du, ad, bd, cd, amax[2:3], amax[3:4])
    assert float(amax[2]) == float(dg.float().abs().max()) and float(amax[3]) == float(du.float().abs().max())
    s = torch.sigmoid(a.float())
    ref_u = (c.float() * a.float() * s).to(torch.bfloat16)
    ref_g = (c.float() * b.float() * s * (1 + a.float() * (1 - s))).to(torch.bfloat16)
    for got, ref in ((du, ref_u), (dg, ref_g)):
        assert int(_bf16_steps(got.cpu(), ref).max()) <= 1 and float((got.cpu() != ref).float().mean()) < 2e-2


def test_chain_rmsnorm_and_its_gradient(st):
    torch.manual_seed(1)
    rows, cols = 37, 8 * 131
    x = (torch.randn(rows, cols) * 3.0).to(torch.bfloat16)
    dy = torch.randn(rows, cols).to(torch.bfloat16)
    y, inv = torch.empty_like(x, device=DEV), torch.empty(rows, dtype=torch.float32, device=DEV)
    amax = torch.zeros(1, dtype=torch.float32, device=DEV)
    st.rmsnorm(y, inv, x.to(DEV), amax=amax)
    assert float(amax[0]) == float(y.float().abs().max())
    xf = x.double()
    inv_ref = 1.0 / torch.sqrt((xf * xf).mean(dim=1) + st.NORM_EPS)
    assert torch.allclose(inv.cpu().double(), inv_ref, rtol=1e-5)
    ref = (xf * inv_ref[:, None]).float().to(torch.bfloat16)
    assert int(_bf16_steps(y.cpu(), ref).max()) <= 1 and float((y.cpu() != ref).float().mean()) < 1e-2
    dx = torch.empty_like(y)
    st.rmsnorm_grad(dx, dy.to(DEV), x.to(DEV), inv)
    xh = xf * inv_ref[:, None]
    ref = (inv_ref[:, None] * (dy.double() - xh * (dy.double() * xh).mean(dim=1, keepdim=True))).float().to(torch.bfloat16)
    assert int(_bf16_steps(dx.cpu(), ref).max()) <= 1 and float((dx.cpu() != ref).float().mean()) < 1e-2
    # against autograd of the same function
    xa = x.double().requires_grad_(True)
    (xa / torch.sqrt((xa * xa).mean(dim=1, keepdim=True) + st.NORM_EPS) * dy.double()).sum().backward()
    assert torch.allclose(dx.cpu().double(), xa.grad, rtol=2e-2, atol=1e-3)


def test_fused_chain_kernels_equal_the_separate_ones_bit_for_bit(st):
    """combine + rmsnorm in one pass, and sum + rmsnorm gradient + residual in one pass, against the kernels they replace
    (which the tests above check against the formulas): identical bits, identical absmax hand-over."""
    torch.manual_seed(3)
    rows, cols = 53, 8 * 77
    mk = lambda scale=1.0: (torch.randn(rows, cols) * scale).to(torch.bfloat16).to(DEV)
    a, b, c, x, res = mk(2.0), mk(0.5), mk(), mk(3.0), mk()
    s1, y1, s2, y2 = (torch.empty_like(a) for _ in range(4))
    inv1, inv2 = (torch.empty(rows, dtype=torch.float32, device=DEV) for _ in range(2))
    am1, am2 = (torch.zeros(1, dtype=torch.float32, device=DEV) for _ in range(2))
    st.combine(s1, a, st.INV_SQRT2, b, st.INV_SQRT2)
    st.rmsnorm(y1, inv1, s1, amax=am1)
    st.combine_rmsnorm(s2, y2, inv2, a, st.INV_SQRT2, b, st.INV_SQRT2, amax=am2)
    assert torch.equal(s1.view(torch.int16), s2.view(torch.int16)) and torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    assert torch.equal(inv1.view(torch.int32), inv2.view(torch.int32)) and float(am1) == float(am2)
    for dys in ([a, b], [a, b, c]):
        t, g, o1, o2 = (torch.empty_like(a) for _ in range(4))
        am1.zero_(); am2.zero_()
        st.combine(t, dys[0], 1.0, dys[1], 1.0, dys[2] if len(dys) == 3 else None, 1.0)
        st.rmsnorm_grad(g, t, x, inv1)
        st.combine(o1, res, st.INV_SQRT2, g, 1.0, amax=am1)
        st.rmsnorm_grad_combine(o2, dys, x, inv1, res, st.INV_SQRT2, amax=am2)
        assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and float(am1) == float(am2)
        # in place on the residual, as the stack does not, and on a gradient operand, as it may
        o3 = dys[0].clone()
        st.rmsnorm_grad_combine(o3, [o3, *dys[1:]], x, inv1, res, st.INV_SQRT2)
        assert torch.equal(o1.view(torch.int16), o3.view(torch.int16))


def test_stack_with_fused_chain_equals_the_unfused_stack(fq, st):
    """Three narrow blocks, one step each way: outputs, input gradient, every backbone and DeltaBuffer identical."""
    H, F, T, r, k = 256, 512, 300, 16, 24
    dev = torch.device(DEV)
    h0 = synth.normal_bf16(5, 9001, (T, H), 1.0, dev)
    G = synth.normal_bf16(5, 9002, (T, H), 1.0e-2, dev)
    outs = []
    for fuse in (False, True):
        stack = st.Stack(3, H, F, T, r, k, seed=5, device=dev, lr=2e-2, fuse_chain=fuse, fuse_cast=False)
        h = stack.forward(h0).clone()
        dh = stack.backward(G).clone()
        torch.cuda.synchronize()
        outs.append((h, dh, [(L.wq.clone(), L.dbuf.clone()) for blk in stack.layers for L in (blk.values() if isinstance(blk, dict) else blk)]))
    (h_a, dh_a, la), (h_b, dh_b, lb) = outs
    assert torch.equal(h_a.view(torch.int16), h_b.view(torch.int16)) and torch.equal(dh_a.view(torch.int16), dh_b.view(torch.int16))
    for (wa, da), (wb, db) in zip(la, lb):
        assert torch.equal(wa, wb) and torch.equal(da.view(torch.int32), db.view(torch.int32))
    assert fq.last_device_status() == 0


def _close_bf16(gpu: torch.Tensor, ref_f32: np.ndarray, what: str):
    """A bf16 tensor-core output against the oracle's fp32 result: every element within one bf16 step of the
    oracle's value (plus a floor of 2e-5 of the tensor's rms for elements that cancel to almost nothing), and
    the whole tensor within the rounding noise of bf16."""
    got = gpu.detach().float().cpu().numpy().astype(np.float64)
    ref = ref_f32.astype(np.float64)
    rms = np.sqrt(np.mean(ref * ref))
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 2e-5 * rms), f"{what}: element out of tolerance"
    assert np.linalg.norm(got - ref) <= 2.0 ** -8 * np.linalg.norm(ref), f"{what}: tensor out of tolerance"
    ref16 = torch.from_numpy(np.ascontiguousarray(ref_f32)).to(torch.bfloat16)
    assert float((gpu.detach().cpu() != ref16).float().mean()) < 0.02, f"{what}: too many elements differ from the rounded oracle"


def _check_projection(fq, orc, cap, layer, name, T, r, k, lr, n_rows):
    """cap: what the GPU saw for this projection (X, Y, OA, dY, dX, dB, wq and dbuf before its update)."""
    m, n = layer.m, layer.n
    wq, s_w = u8(cap["wq"]), np.float32(f32(layer.s_w)[0])
    rng = np.random.default_rng(5)
    tsel = np.sort(rng.choice(T, min(n_rows, T), replace=False))
    tdev = torch.from_numpy(tsel).to(DEV)
    # S1 + S2 (for k, v, up the codes came from the neighbouring projection's cast of the same X)
    xq_o, s_x_o, _ = orc.quantize(f32(cap["X"]), orc.E4M3)
    rows_o = orc.forward_gemm(xq_o, s_x_o, wq, s_w, m, r, tsel=tsel)
    _close_bf16(cap["Y"][tdev], rows_o[:, :m], f"{name} Y")
    assert product_close(f32(cap["OA"][tdev]), rows_o[:, m:], 2e-5), f"{name} OA"
    # S3 + S4 + S5
    gq_o, s_g_o, _ = orc.quantize(f32(cap["dY"]), orc.E5M2)
    _close_bf16(cap["dX"][tdev], orc.dx_gemm(gq_o, s_g_o, wq, s_w, m, tsel=tsel), f"{name} dX")
    oaq_o, s_oa_o, _ = orc.quantize(f32(cap["OA"]), orc.E4M3)
    isel = np.sort(rng.choice(m, min(2 * n_rows, m), replace=False))
    dB_o = orc.db_gemm(gq_o, s_g_o, oaq_o, s_oa_o, isel=isel)
    dB_g = f32(cap["dB"][torch.from_numpy(isel).to(DEV)])
    assert product_close(dB_g, dB_o, 2e-5), f"{name} dB"
    # S6..S8, fed the GPU's own dB: bit-exact
    wq_o, dbuf_o = wq.copy(), f32(cap["dbuf"]).copy()
    orc.proxy_update(wq_o, dbuf_o, f32(cap["dB"]), lr, k, m, r)
    assert np.array_equal(u8(layer.wq), wq_o), f"{name} merged rows"
    assert np.array_equal(bits32(f32(layer.dbuf)), bits32(dbuf_o)), f"{name} DeltaBuffer"


def _run_and_check(fq, st, orc, n_layers, H, F, T, r, k, check_blocks, n_rows, producer_amax=True, fuse_cast=False):
    stack = st.Stack(n_layers, H, F, T, r, k, seed=7, device=DEV, lr=2e-2, producer_amax=producer_amax,
                     batched_proxy=producer_amax,   # the second variant also keeps the per-projection proxy updates
                     fuse_cast=fuse_cast)
    h0 = synth.normal_bf16(7, 9001, (T, H), 1.0, DEV)
    G = synth.normal_bf16(7, 9002, (T, H), 1.0e-2, DEV)
    stack.capture = {(l, p): {} for l in check_blocks for p in st.PROJ}
    # the layer state each checked projection starts from (one step: a layer is updated once, after its backward)
    for (l, p), cap in stack.capture.items():
        cap["wq"] = stack.layers[l][p].wq.clone()
        cap["dbuf"] = stack.layers[l][p].dbuf.clone()
    h = stack.step(h0, G)
    torch.cuda.synchronize()
    assert fq.last_device_status() == 0
    assert bool(torch.isfinite(h.float()).all())
    for (l, p), cap in stack.capture.items():
        _check_projection(fq, orc, cap, stack.layers[l][p], f"block {l} {p}", T, r, k, 2e-2, n_rows)
    return stack


@pytest.mark.parametrize("producer_amax", [True, False])
def test_small_stack_every_projection(fq, st, orc, producer_amax):
    """Three blocks of a narrow chain, every projection of every block checked on all token rows; with the chain
    kernels handing the absmax of their outputs to the layers (single-pass input casts) and without."""
    _run_and_check(fq, st, orc, 3, 256, 640, 192, 16, 8, check_blocks=[0, 1, 2], n_rows=192, producer_amax=producer_amax)


def test_small_stack_with_the_casts_inside_the_chain_kernels(fq, st, orc):
    """The same chain with every layer input and output gradient leaving its producing kernel as FP8 codes: every
    projection against the oracle (the captured bf16 tensors are the ones the codes were made from), and the whole step
    bit for bit the step of the stack with separate casts."""
    _run_and_check(fq, st, orc, 3, 256, 640, 192, 16, 8, check_blocks=[0, 1, 2], n_rows=192, fuse_cast=True)
    H, F, T, r, k = 256, 512, 300, 16, 24
    dev = torch.device(DEV)
    h0 = synth.normal_bf16(5, 9001, (T, H), 1.0, dev)
    G = synth.normal_bf16(5, 9002, (T, H), 1.0e-2, dev)
    outs = []
    for fuse in (False, True):
        stack = st.Stack(3, H, F, T, r, k, seed=5, device=dev, lr=2e-2, fuse_cast=fuse)
        for _ in range(2):        # two steps: the second runs on updated backbones and reuses the kernels' scratch
            h = stack.step(h0, G).clone()
        dh = stack.dh.clone()
        torch.cuda.synchronize()
        outs.append((h, dh, [(L.wq.clone(), L.dbuf.clone()) for blk in stack.layers for L in blk.values()]))
    (h_a, dh_a, la), (h_b, dh_b, lb) = outs
    assert torch.equal(h_a.view(torch.int16), h_b.view(torch.int16)) and torch.equal(dh_a.view(torch.int16), dh_b.view(torch.int16))
    for (wa, da), (wb, db) in zip(la, lb):
        assert torch.equal(wa, wb) and torch.equal(da.view(torch.int32), db.view(torch.int32))
    assert fq.last_device_status() == 0


def test_stack_7b_shapes_sampled(fq, st, orc):
    """The 7B shapes (hidden 4096, MLP 11008, 4096 tokens, rank 64, top-256), 32 blocks in one step: the first, the
    last and two other blocks are checked on sampled rows."""
    stack = _run_and_check(fq, st, orc, 32, 4096, 11008, 4096, 64, 256, check_blocks=[0, 11, 22, 31], n_rows=24)
    assert stack.flops_per_step() == pytest.approx(107.41e12, rel=1e-3)


def test_stack_7b_shapes_sampled_with_the_casts_inside_the_chain_kernels(fq, st, orc):
    """The same at full size with the quantizing chain kernels (x1, a, x2 stay in shared memory across the grid barrier; z,
    dg and du mostly pass through memory)."""
    _run_and_check(fq, st, orc, 32, 4096, 11008, 4096, 64, 256, check_blocks=[0, 17, 31], n_rows=24, fuse_cast=True)


def test_small_stack_with_adamw(fq, st, orc):
    """Two steps of a narrow three-block chain with AdamW on every DeltaBuffer (one batched AdamW update per block): the
    first projection of every block is followed on the CPU from the captured gradients (oracle AdamW step, then the
    oracle's selection and merge), bit for bit."""
    n_layers, H, F, T, r, k = 3, 256, 640, 192, 16, 8
    hp = dict(beta1=0.9, beta2=0.99, eps=1e-8, weight_decay=0.01)
    stack = st.Stack(n_layers, H, F, T, r, k, seed=11, device=DEV, lr=3e-3, adamw=hp)
    h0 = synth.normal_bf16(11, 9001, (T, H), 1.0, DEV)
    G = synth.normal_bf16(11, 9002, (T, H), 1.0e-2, DEV)
    follow = {l: dict(wq=u8(stack.layers[l]["q"].wq).copy(), dbuf=f32(stack.layers[l]["q"].dbuf).copy(),
                      ea=np.zeros((H, r), np.float32), es=np.zeros((H, r), np.float32)) for l in range(n_layers)}
    for step in (1, 2):
        stack.capture = {(l, "q"): {} for l in range(n_layers)}
        h = stack.step(h0, G)
        torch.cuda.synchronize()
        assert bool(torch.isfinite(h.float()).all())
        for l in range(n_layers):
            o = follow[l]
            orc.adamw_step(o["dbuf"], f32(stack.capture[(l, "q")]["dB"]), o["ea"], o["es"], 3e-3, hp["beta1"], hp["beta2"],
                           hp["eps"], hp["weight_decay"], step)
            orc.proxy_update(o["wq"], o["dbuf"], None, 0.0, k, H, r)
            layer = stack.layers[l]["q"]
            assert np.array_equal(u8(layer.wq), o["wq"]), f"block {l} step {step}: backbone"
            assert np.array_equal(bits32(f32(layer.dbuf)), bits32(o["dbuf"])), f"block {l} step {step}: DeltaBuffer"
            assert np.array_equal(bits32(f32(stack.exp_avg[l][0])), bits32(o["ea"])), f"block {l} step {step}: exp_avg"
            assert np.array_equal(bits32(f32(stack.exp_avg_sq[l][0])), bits32(o["es"])), f"block {l} step {step}: exp_avg_sq"
    assert fq.last_device_status() == 0
