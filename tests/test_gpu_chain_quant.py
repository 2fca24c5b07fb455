"""The quantizing chain calls (the cast fused into the kernel that produces the tensor) against the plain chain call
followed by the oracle's per-tensor cast: the bf16 values must be those of the plain kernel bit for bit, the scale the
oracle's scale bit for bit, every code the oracle's code.  Sizes cover tensors that stay in shared memory, ragged
counts, fewer rows than SMs, and tensors large enough that most of each CTA's share passes through memory.
"""
import numpy as np
import pytest
import torch

from helpers import bits32, f32, u8

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
POISON = 0xAB


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


def _rand(shape, scale, seed):
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(shape, generator=g) * scale
    t.view(-1)[:: 997] *= 9.0          # a few large values, so that the absmax is not a typical element
    return t.to(torch.bfloat16).to(DEV)


def _check_codes(orc, fmt, plain16, codes, scale, what):
    """codes / scale against the oracle's cast of the plain kernel's bf16 output."""
    ofmt = orc.E4M3 if fmt == 0 else orc.E5M2
    want, s, _ = orc.quantize(f32(plain16).reshape(1, -1), ofmt)
    assert bits32(f32(scale))[0] == bits32(s).reshape(-1)[0], (what, float(scale), float(s))
    got = u8(codes).reshape(-1)[: plain16.numel()]
    want = want.reshape(-1)
    assert np.array_equal(got, want), (what, int((got != want).sum()), np.flatnonzero(got != want)[:8])


def _bufs(count):
    codes = torch.full((count + 64,), POISON, dtype=torch.uint8, device=DEV)
    scale = torch.zeros(1, dtype=torch.float32, device=DEV)
    out16 = torch.empty(count, dtype=torch.bfloat16, device=DEV)
    return codes, scale, out16


@pytest.mark.parametrize("count", [8, 8 * 511, 8 * 4099, 1024 * 1024, 8 * (148 * 14336 + 1000)])
@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("keep16", [False, True])
def test_combine_quantize(fq, st, orc, count, fmt, keep16):
    if count > 8 * 1024 * 1024 and keep16 and fmt == 0:
        pytest.skip("one large keep16 case is enough")
    a, b, c = _rand(count, 1.0, 1), _rand(count, 0.5, 2), _rand(count, 2.0, 3)
    plain = torch.empty_like(a)
    st.combine(plain, a, 0.5, b, -1.25, c, 3.0 ** -0.5)
    codes, scale, out16 = _bufs(count)
    scratch = st.chain_scratch(DEV)
    st.combine_quantize(codes, scale, fmt, out16, keep16, scratch, a, 0.5, b, -1.25, c, 3.0 ** -0.5)
    torch.cuda.synchronize()
    _check_codes(orc, fmt, plain, codes, scale, "combine")
    assert bool((codes[count:] == POISON).all())
    if keep16:
        assert torch.equal(out16.view(torch.int16), plain.view(torch.int16))
    assert int(scratch.view(torch.int32)[:2].abs().sum()) == 0          # the barrier's counters are back at zero
    # a second call on the same scratch, one input only (the scaled copy the backward uses)
    st.combine(plain, a, 2.0 ** -0.5)
    st.combine_quantize(codes, scale, fmt, out16, keep16, scratch, a, 2.0 ** -0.5)
    torch.cuda.synchronize()
    _check_codes(orc, fmt, plain, codes, scale, "scaled copy")
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("count", [8 * 77, 8 * 70001, 8 * (148 * 14336 + 4096 * 5 + 3)])
def test_silu_mul_quantize_and_its_gradient(fq, st, orc, count):
    g, u, dz = _rand(count, 1.5, 4), _rand(count, 1.0, 5), _rand(count, 0.01, 6)
    scratch = st.chain_scratch(DEV)
    z = torch.empty_like(g)
    st.silu_mul(z, g, u)
    codes, scale, out16 = _bufs(count)
    st.silu_mul_quantize(codes, scale, 0, out16, False, scratch, g, u)
    torch.cuda.synchronize()
    _check_codes(orc, 0, z, codes, scale, "silu_mul")
    # gradient: two tensors, two scales (E5M2)
    dg, du = torch.empty_like(g), torch.empty_like(g)
    st.silu_mul_grad(dg, du, g, u, dz)
    cg, sg, g16 = _bufs(count)
    cu, su, u16 = _bufs(count)
    for keep16 in (False, True):
        cg.fill_(POISON)
        cu.fill_(POISON)
        st.silu_mul_grad_quantize(cg, cu, sg, su, 1, g16, u16, keep16, scratch, g, u, dz)
        torch.cuda.synchronize()
        _check_codes(orc, 1, dg, cg, sg, "dg")
        _check_codes(orc, 1, du, cu, su, "du")
        assert bool((cg[count:] == POISON).all()) and bool((cu[count:] == POISON).all())
        if keep16:
            assert torch.equal(g16.view(torch.int16), dg.view(torch.int16).view(-1))
            assert torch.equal(u16.view(torch.int16), du.view(torch.int16).view(-1))
    assert int(scratch.view(torch.int32)[:2].abs().sum()) == 0
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("rows,cols", [(1, 8), (5, 1000), (149, 4096), (4096, 4096), (300, 16384), (6000, 4096), (1000, 11008)])
def test_rmsnorm_quantize(fq, st, orc, rows, cols):
    a, b = _rand((rows, cols), 1.0, 7), _rand((rows, cols), 0.7, 8)
    scratch = st.chain_scratch(DEV)
    count = rows * cols
    # plain normalisation
    y = torch.empty_like(a)
    inv = torch.empty(rows, dtype=torch.float32, device=DEV)
    st.rmsnorm(y, inv, a)
    codes, scale, y16 = _bufs(count)
    inv2 = torch.zeros_like(inv)
    st.rmsnorm_quantize(codes, scale, 0, y16.view(rows, cols), False, scratch, inv2, a)
    torch.cuda.synchronize()
    _check_codes(orc, 0, y, codes, scale, "rmsnorm")
    assert torch.equal(inv.view(torch.int32), inv2.view(torch.int32))
    assert bool((codes[count:] == POISON).all())
    # residual sum + normalisation, with the bf16 result kept
    s1, s2 = torch.empty_like(a), torch.empty_like(a)
    st.combine_rmsnorm(s1, y, inv, a, 2.0 ** -0.5, b, 2.0 ** -0.5)
    inv2.zero_()
    st.rmsnorm_quantize(codes, scale, 0, y16.view(rows, cols), True, scratch, inv2, a, sum_out=s2, sa=2.0 ** -0.5, b=b, sb=2.0 ** -0.5)
    torch.cuda.synchronize()
    _check_codes(orc, 0, y, codes, scale, "combine_rmsnorm")
    assert torch.equal(s1.view(torch.int16), s2.view(torch.int16))
    assert torch.equal(y16.view(torch.int16), y.view(torch.int16).view(-1))
    assert torch.equal(inv.view(torch.int32), inv2.view(torch.int32))
    assert int(scratch.view(torch.int32)[:2].abs().sum()) == 0
    assert fq.last_device_status() == 0


@pytest.mark.parametrize("rows,cols,three", [(3, 64, False), (149, 4096, True), (4096, 4096, False), (200, 16384, True), (5000, 4096, True)])
def test_rmsnorm_grad_combine_quantize(fq, st, orc, rows, cols, three):
    x, res = _rand((rows, cols), 1.0, 9), _rand((rows, cols), 0.01, 10)
    dys = [_rand((rows, cols), 0.01, 11 + i) for i in range(3 if three else 2)]
    inv = torch.empty(rows, dtype=torch.float32, device=DEV)
    st.rmsnorm(torch.empty_like(x), inv, x)
    plain = torch.empty_like(x)
    st.rmsnorm_grad_combine(plain, dys, x, inv, res, 2.0 ** -0.5)
    count = rows * cols
    codes, scale, out = _bufs(count)
    scratch = st.chain_scratch(DEV)
    st.rmsnorm_grad_combine_quantize(codes, scale, 1, out.view(rows, cols), scratch, dys, x, inv, res, 2.0 ** -0.5)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), plain.view(torch.int16).view(-1))
    _check_codes(orc, 1, plain, codes, scale, "rmsnorm_grad_combine")
    assert bool((codes[count:] == POISON).all())
    assert int(scratch.view(torch.int32)[:2].abs().sum()) == 0
    assert fq.last_device_status() == 0


def test_all_zero_tensor_and_argument_checks(fq, st, orc):
    count = 8 * 1000
    a = torch.zeros(count, dtype=torch.bfloat16, device=DEV)
    codes, scale, out16 = _bufs(count)
    scratch = st.chain_scratch(DEV)
    st.combine_quantize(codes, scale, 0, out16, False, scratch, a, 1.0)
    torch.cuda.synchronize()
    _check_codes(orc, 0, a, codes, scale, "zeros")          # the oracle's reading of an all-zero tensor (scale 1, zero codes)
    lib = st.lib
    bad = lib.falqon_chain_combine_quantize(codes.data_ptr(), scale.data_ptr(), 2, out16.data_ptr(), 0, a.data_ptr(), 1.0, None, 1.0,
                                            None, 1.0, None, 1.0, count, scratch.data_ptr(), None)
    assert bad == -1                                          # unknown format
    bad = lib.falqon_chain_combine_quantize(codes.data_ptr(), scale.data_ptr(), 0, out16.data_ptr(), 0, a.data_ptr(), 1.0, None, 1.0,
                                            None, 1.0, None, 1.0, count + 4, scratch.data_ptr(), None)
    assert bad == -1                                          # count not a multiple of 8
    bad = lib.falqon_chain_rmsnorm_quantize(codes.data_ptr(), scale.data_ptr(), 0, out16.data_ptr(), 0, scale.data_ptr(), None,
                                            a.data_ptr(), 1.0, a.data_ptr(), 1.0, 10, 800, 1e-6, scratch.data_ptr(), None)
    assert bad == -1                                          # a second input without a place for the sum
