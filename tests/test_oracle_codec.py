"""Pins for the oracle's software FP8 codec and quantizer (CPU only).

Independent references used here: PyTorch's CPU float8 casts (a different
implementation of the same formats), hand-worked code tables under
tests/golden/, and closed-form properties of the formats.
"""
import os

import numpy as np
import pytest
import torch

from oracle import falqon_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FMTS = [(orc.E4M3, torch.float8_e4m3fn, 448.0), (orc.E5M2, torch.float8_e5m2, 57344.0)]


def _torch_decode(fmt_dtype):
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    return codes.view(fmt_dtype).to(torch.float32).numpy().astype(np.float64)


def _torch_encode_clamped(values_f32: np.ndarray, fmt_dtype, fmax: float) -> np.ndarray:
    # torch's cast rounds to nearest even but does not saturate, so clamp first.
    t = torch.from_numpy(values_f32).clamp(-fmax, fmax)
    return t.to(fmt_dtype).view(torch.uint8).numpy()


@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_decode_matches_library_tables(fmt, tdt, fmax):
    ours = orc.decode_array(np.arange(256, dtype=np.uint8), fmt)
    ref = _torch_decode(tdt)
    finite = np.isfinite(ref)
    assert np.array_equal(np.isnan(ours), np.isnan(ref))
    assert np.array_equal(ours[finite], ref[finite])
    assert np.nanmax(np.where(np.isfinite(ours), ours, np.nan)) == fmax  # the maxima the paper states


def test_format_structure_closed_forms():
    # E4M3: min subnormal 2^-9, min normal 2^-6, 1.0 = 0x38; E5M2: 2^-16, 2^-14, 1.0 = 0x3C.
    assert orc.decode(0x01, orc.E4M3) == 2.0 ** -9 and orc.decode(0x08, orc.E4M3) == 2.0 ** -6
    assert orc.decode(0x38, orc.E4M3) == 1.0 and orc.decode(0x7E, orc.E4M3) == 448.0
    assert np.isnan(orc.decode(0x7F, orc.E4M3)) and np.isnan(orc.decode(0xFF, orc.E4M3))
    assert orc.decode(0x01, orc.E5M2) == 2.0 ** -16 and orc.decode(0x04, orc.E5M2) == 2.0 ** -14
    assert orc.decode(0x3C, orc.E5M2) == 1.0 and orc.decode(0x7B, orc.E5M2) == 57344.0
    assert orc.decode(0x7C, orc.E5M2) == np.inf and orc.decode(0xFC, orc.E5M2) == -np.inf
    assert np.isnan(orc.decode(0x7D, orc.E5M2))
    # adjacent normal codes differ by 2^(e-M): 1.0 -> 1.125 (E4M3), 1.0 -> 1.25 (E5M2)
    assert orc.decode(0x39, orc.E4M3) == 1.125 and orc.decode(0x3D, orc.E5M2) == 1.25


def test_golden_code_table():
    names = {"e4m3": orc.E4M3, "e5m2": orc.E5M2}
    count = 0
    with open(os.path.join(GOLDEN, "fp8_codes.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            fmt, expr, code = line.split()
            value = float(eval(expr, {"__builtins__": {}}))
            assert orc.encode(value, names[fmt]) == int(code, 16), line
            count += 1
    assert count == 33


@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_roundtrip_monotonic_midpoints(fmt, tdt, fmax):
    vals = orc.decode_array(np.arange(128, dtype=np.uint8), fmt)
    finite = np.isfinite(vals)
    codes = np.arange(128)[finite]
    v = vals[finite]
    assert np.all(np.diff(v) > 0)  # positive codes are strictly increasing in value
    for c, x in zip(codes, v):
        assert orc.encode(x, fmt) == c            # encode(decode(c)) == c
        assert orc.encode(-x, fmt) == (c | 0x80)  # and the sign bit carries over (incl. -0)
    # exact midpoints of neighbours go to the even code; a hair to either side goes to the nearer one
    for c in range(len(v) - 1):
        mid = np.float32((v[c] + v[c + 1]) / 2)
        assert float(mid) == (v[c] + v[c + 1]) / 2
        even = codes[c] if codes[c] % 2 == 0 else codes[c + 1]
        assert orc.encode(mid, fmt) == even
        assert orc.encode(np.nextafter(mid, np.float32(0)), fmt) == codes[c]
        assert orc.encode(np.nextafter(mid, np.float32(np.inf)), fmt) == codes[c + 1]


@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_saturation_and_specials(fmt, tdt, fmax):
    max_code = orc.encode(fmax, fmt)
    assert orc.decode(max_code, fmt) == fmax
    for x in [np.nextafter(np.float32(fmax), np.float32(np.inf)), fmax * 1.03, fmax * 1.2, 1e30, np.inf]:
        assert orc.encode(x, fmt) == max_code
        assert orc.encode(-x, fmt) == (max_code | 0x80)
    assert orc.encode(np.nan, fmt) == 0x7F
    assert orc.encode(1e-45, fmt) == 0x00 and orc.encode(-1e-45, fmt) == 0x80  # fp32 subnormal input


@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_encode_exhaustive_bf16_inputs_vs_library(fmt, tdt, fmax):
    bits = np.arange(1 << 16, dtype=np.uint32) << 16
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    ours = orc.encode_array(x, fmt)
    ref = _torch_encode_clamped(x, tdt, fmax)
    assert np.array_equal(ours, ref)


@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_encode_random_fp32_and_near_ties_vs_library(fmt, tdt, fmax):
    rng = np.random.default_rng(123)
    expo = rng.integers(-22, 18, size=1 << 20)
    x = (rng.standard_normal(1 << 20) * np.exp2(expo)).astype(np.float32)
    # values one fp32 ulp around every code midpoint, both signs
    v = orc.decode_array(np.arange(128, dtype=np.uint8), fmt)
    v = v[np.isfinite(v)]
    mids = ((v[:-1] + v[1:]) / 2).astype(np.float32)
    near = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf))])
    x = np.concatenate([x, near, -near])
    assert np.array_equal(orc.encode_array(x, fmt), _torch_encode_clamped(x, tdt, fmax))


# ---------------- quantizer: Q_fp8 = amax -> scale -> cast (Eq. quantize) ----------------

@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_quantize_scale_and_full_range(fmt, tdt, fmax):
    rng = np.random.default_rng(7)
    x = rng.standard_normal((37, 53)).astype(np.float32) * 3.7
    q, s, amax = orc.quantize(x, fmt)
    assert amax == np.abs(x).max()
    assert s.view(np.uint32) == (np.float32(fmax) / amax).view(np.uint32)  # one fp32 division, to the bit
    assert np.abs(orc.decode_array(q, fmt)).max() == fmax                  # the largest element fills the range
    # library cross-check of the whole array: clamp(x*s) cast by torch
    assert np.array_equal(q, _torch_encode_clamped(x * s, tdt, fmax))


@pytest.mark.parametrize("fmt,tdt,fmax", FMTS)
def test_quantize_idempotent_on_representable_values(fmt, tdt, fmax):
    rng = np.random.default_rng(8)
    x = rng.standard_normal((16, 64)).astype(np.float32)
    q, s, _ = orc.quantize(x, fmt)
    dq = orc.decode_array(q, fmt).astype(np.float32)   # representable values in the scaled domain
    q2, _, _ = orc.quantize(dq, fmt, scale_in=np.float32(1.0))
    assert np.array_equal(q, q2)


def test_quantize_exact_power_of_two_case():
    # amax = 448 * 2^-5 -> s = 32 exactly; every element is (an E4M3 value) * 2^-5 -> exact codes.
    codes = np.array([[0x7E, 0x01, 0x38, 0xB9], [0x00, 0x80, 0x45, 0xFE]], dtype=np.uint8)
    x = (orc.decode_array(codes, orc.E4M3) * 2.0 ** -5).astype(np.float32)
    q, s, amax = orc.quantize(x, orc.E4M3)
    assert s == 32.0 and amax == 14.0
    assert np.array_equal(q, codes)


def test_quantize_zero_tensor_and_bf16_input():
    q, s, amax = orc.quantize(np.zeros((3, 5), np.float32), orc.E4M3)
    assert s == 1.0 and amax == 0.0 and not q.any()
    x = torch.randn(8, 24, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    qa, sa, _ = orc.quantize(bits, orc.E4M3, src_is_bf16_bits=True)
    qb, sb, _ = orc.quantize(x.float().numpy(), orc.E4M3)
    assert sa == sb and np.array_equal(qa, qb)
    assert np.array_equal(orc.bf16_bits(x.float().numpy()), bits)


def test_quantize_given_scale_premul_and_saturation():
    # A~ = Q(gamma*A; s_W) (Eq. A_integ): two rounded fp32 multiplies, then a saturating cast.
    a = np.array([[0.03125, -0.02, 0.5, -0.75]], dtype=np.float32)
    s_w = np.float32(4600.0)
    q, s, _ = orc.quantize(a, orc.E4M3, scale_in=s_w, premul=2.0)
    assert s == s_w
    expect = _torch_encode_clamped((np.float32(2.0) * a) * s_w, torch.float8_e4m3fn, 448.0)
    assert np.array_equal(q, expect)
    assert q[0, 2] == 0x7E and q[0, 3] == 0xFE  # 4600 and -6900 saturate to +-448


def test_quantize_per_row():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((5, 40)).astype(np.float32) * np.array([[1], [10], [0.1], [100], [1e-3]], np.float32)
    q, s, amax = orc.quantize(x, orc.E4M3, gran=orc.PER_ROW)
    for i in range(5):
        qi, si, ai = orc.quantize(x[i:i + 1], orc.E4M3)
        assert si == s[i] and ai == amax[i] and np.array_equal(qi[0], q[i])


def test_f32_to_bf16_rounding_matches_library_cast():
    """The oracle's fp32 -> bf16 rounding (nearest, ties to even) against PyTorch's CPU cast, an independent
    implementation: every exact tie between two bf16 neighbours and its two fp32 neighbours for a spread of exponents,
    hand-worked cases, and random values."""
    import torch
    from oracle import falqon_oracle as orc
    cases = {1.0: 0x3F80, -1.0: 0xBF80, 0.0: 0x0000, 1.00390625: 0x3F80,    # 1 + 2^-8: tie, even mantissa below
             1.01171875: 0x3F82,                                            # 1 + 3*2^-8: tie, rounds up to the even code
             1.0078125: 0x3F81, 3.3895313892515355e38: 0x7F7F}              # largest finite bf16
    for v, code in cases.items():
        assert orc.f32_to_bf16_bits(v) == code, v
    rng = np.random.default_rng(3)
    hi = rng.integers(0x0080, 0x7F00, size=4000, dtype=np.uint32)           # positive normal bf16 patterns
    vals = []
    for h in hi:
        tie = (int(h) << 16) | 0x8000
        vals += [tie - 1, tie, tie + 1]
    bits = np.array(vals, dtype=np.uint32)
    bits = np.concatenate([bits, bits | 0x80000000, rng.integers(0, 0x7F800000, size=20000, dtype=np.uint32)])
    x = bits.view(np.float32)
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([orc.f32_to_bf16_bits(v) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
