"""Pins for the oracle's format layer: value tables, rounding, decoder (CPU only).

Each test ties an oracle function to something outside the oracle: values the paper
prints (tests/golden), a library cast, exact rational arithmetic, or enumeration.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import torch

from oracle import razer_oracle as ro

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_fp4_value_set_matches_paper():
    mags = [float(v) for v in _rows("fp4_value_set.txt")[0]]
    got = sorted(ro.fp4_value(c) for c in range(16))
    want = sorted([-m for m in mags] + mags)
    assert got == want
    # the two zero codes are 0b0000 and 0b1000 (sign bit only differs)
    assert ro.fp4_value(0) == 0.0 and ro.fp4_value(8) == 0.0
    # sign bit is the nibble's top bit; magnitude order follows the low three bits
    for c in range(8):
        assert ro.fp4_value(c) == mags[c]
        assert ro.fp4_value(c | 8) == -mags[c]


def test_e4m3_landmarks_and_torch_cast():
    for e, m, v in _rows("e4m3_landmarks.txt"):
        assert ro.e4m3_value((int(e) << 3) | int(m)) == float(v)
    # every 7-bit code agrees with the library's float8_e4m3fn decoding (same OCP format)
    codes = torch.arange(0, 127, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    mine = np.array([ro.e4m3_value(c) for c in range(127)])
    assert np.array_equal(lib, mine)
    # the weight scale format is the 64-code prefix with maximum 1.875
    g = ro.scale_grid(ro.SCALE_E3M3_META2)
    assert len(g) == 64 and g[-1] == 1.875 and g[1] == 2.0 ** -9
    assert np.all(np.diff(ro.scale_grid(ro.SCALE_E4M3_META1)) > 0)
    assert ro.scale_max(ro.SCALE_E4M3_META1) == 448.0


def test_scale_rounding_matches_library_cast():
    rng = np.random.default_rng(1)
    t = np.concatenate([
        np.abs(rng.standard_normal(20000)).astype(np.float32) * 3.0,
        np.exp(rng.uniform(np.log(2.0 ** -11), np.log(447.0), 20000)).astype(np.float32),
        np.array([0.0, 2.0 ** -10, 2.0 ** -9, 448.0], dtype=np.float32),
    ])
    # all midpoints between neighbouring grid values (ties) as well
    g = ro.scale_grid(ro.SCALE_E4M3_META1)
    t = np.concatenate([t, ((g[:-1] + g[1:]) / 2).astype(np.float32)])
    t = t[t <= 448.0]
    lib = torch.from_numpy(t).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = ro.round_to_scale(t, ro.SCALE_E4M3_META1)
    assert np.array_equal(lib, mine)
    # saturation above the maximum, and the 6-bit format saturating at 1.875
    assert ro.round_to_scale(np.array([1e9]), ro.SCALE_E4M3_META1)[0] == 126
    assert ro.round_to_scale(np.array([5.0]), ro.SCALE_E3M3_META2)[0] == 63
    small = t[t <= 1.875]
    assert np.array_equal(ro.round_to_scale(small, ro.SCALE_E3M3_META2),
                          torch.from_numpy(small).to(torch.float8_e4m3fn).view(torch.uint8).numpy())


def test_fp4_rounding_nearest_and_ties():
    mags = [float(v) for v in _rows("fp4_value_set.txt")[0]]
    rng = np.random.default_rng(2)
    x = rng.uniform(-7.5, 7.5, 5000)
    idx = ro.round_to_fp4(x)
    for xi, ii in zip(x, idx):
        d = [abs(abs(xi) - m) for m in mags]
        assert d[ii] == min(d)          # nearest (random reals: no ties)
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for t, want in ties.items():
        assert mags[ro.round_to_fp4(np.array([t]))[0]] == want
        assert mags[ro.round_to_fp4(np.array([-t]))[0]] == want
    assert mags[ro.round_to_fp4(np.array([100.0]))[0]] == 6.0


def test_offset_decoder_example_and_range():
    for reg, off, mag, sign, sv in _rows("offset_decoder_example.txt"):
        assert ro.offset_decoder_sv(int(reg, 2), int(sign)) == float(sv)
        assert abs(ro.offset_decoder_sv(int(reg, 2), 0)) == float(mag)
        assert ro.offset_decoder_sv(int(reg, 2), 0) - 6.0 == float(off)
    # the register spans [-3.5, 3.5] in steps of 0.5 => magnitudes 2.5 .. 9.5
    mags = sorted({ro.offset_decoder_sv(r, 0) for r in range(16)})
    assert mags[0] == 2.5 and mags[-1] == 9.5
    assert all(abs((b - a) - 0.5) < 1e-12 for a, b in zip(mags, mags[1:]))
    # metadata order for weights: sign bit then pair selector
    assert ro.sv_candidates((5.0, 8.0), ro.SCALE_E3M3_META2) == [5.0, 8.0, -5.0, -8.0]
    assert ro.sv_candidates((5.0, 5.0), ro.SCALE_E4M3_META1) == [5.0, -5.0]


def test_two_pass_value_list_by_enumeration():
    listed = [float(v) for v in _rows("two_pass_special_values.txt")[0]]
    assert tuple(listed) == ro.ALLOWED_SV_MAGNITUDES
    fp4 = sorted({abs(ro.fp4_value(c)) for c in range(16)} - {0.0})
    sums = {a + b for a, b in itertools.product(fp4, fp4)} - set(fp4)
    assert sorted(sums) == listed
    # every allowed special value times every block scale is exact in bf16 (<= 8 significant bits)
    for m in listed:
        for c in range(1, 127):
            v = Fraction(m) * Fraction(ro.e4m3_value(c))
            num = v.numerator
            while num % 2 == 0:
                num //= 2
            assert num < 256


def test_two_pass_split_reconstructs():
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 256, (8, 32), dtype=np.uint8)
    scales = (rng.integers(0, 4, (8, 4)) << 6 | rng.integers(1, 64, (8, 4))).astype(np.uint8)
    q, _ = ro.decode_block_values(codes, scales)
    main, comp, split = ro.two_pass_split(codes, scales)
    assert np.array_equal(main + comp, q)
    for mag, a, b in _rows("two_pass_example.txt"):
        assert split[float(mag)] == (float(a), float(b))
    is_sv = ro.unpack_codes(codes) == 0x8
    assert np.all(comp[~is_sv] == 0) and np.all(main[~is_sv] == q[~is_sv])
    fp4 = {ro.fp4_value(c) for c in range(16)}
    assert set(np.unique(main)) <= fp4 and set(np.unique(comp)) <= fp4


def test_decode_plain_nvfp4_when_no_special_code():
    """With no remapped code present the decode is plain NVFP4: value table x E4M3 scale,
    checked against torch's own float8 decoding of the scale byte."""
    rng = np.random.default_rng(4)
    c = rng.integers(0, 16, (16, 64), dtype=np.uint8)
    c[c == 8] = 0
    codes = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    scales = rng.integers(1, 127, (16, 4), dtype=np.uint8)           # activation format, meta 0
    d1 = ro.dequant_d1(codes, scales, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0,))
    s = torch.from_numpy(scales).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    tab = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, 0, -.5, -1, -1.5, -2, -3, -4, -6])
    assert np.array_equal(d1.astype(np.float64), tab[c] * np.repeat(s, 16, axis=1))


def test_decode_special_value_and_zero_convention_involution():
    rng = np.random.default_rng(5)
    c = rng.integers(0, 16, (32, 64), dtype=np.uint8)
    codes = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    scales = (rng.integers(0, 4, (32, 4)) << 6 | rng.integers(1, 64, (32, 4))).astype(np.uint8)
    q, s = ro.decode_block_values(codes, scales, sv_mag=(5.0, 8.0), remap_code=0x8)
    meta = np.repeat(scales >> 6, 16, axis=1)
    want_sv = np.array([5.0, 8.0, -5.0, -8.0])[meta]
    assert np.array_equal(q[c == 8], want_sv[c == 8])
    assert np.all(q[c == 0] == 0)
    # swapping which zero code is remapped == XOR 0x8 on the zero-magnitude nibbles
    c2 = np.where((c & 7) == 0, c ^ 8, c).astype(np.uint8)
    codes2 = (c2[:, 0::2] | (c2[:, 1::2] << 4)).astype(np.uint8)
    q2, _ = ro.decode_block_values(codes2, scales, sv_mag=(5.0, 8.0), remap_code=0x0)
    assert np.array_equal(q, q2)
    # activation format: one metadata bit in bit 7, seven scale bits
    sa = (rng.integers(0, 2, (32, 4)) << 7 | rng.integers(1, 127, (32, 4))).astype(np.uint8)
    qa, s_a = ro.decode_block_values(codes, sa, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0,))
    sign = np.repeat(sa >> 7, 16, axis=1)
    assert np.array_equal(qa[c == 8], np.where(sign == 1, -5.0, 5.0)[c == 8])
    assert np.array_equal(s_a, np.vectorize(ro.e4m3_value)(sa & 0x7F))


def test_f64_to_bf16_direct_rounding_exact_rational():
    rng = np.random.default_rng(6)
    x = np.concatenate([rng.standard_normal(3000) * np.exp(rng.uniform(-30, 30, 3000)),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38,
                                  1e39, -1e39, 2.0 ** -133, 2.0 ** -134, 1.5 * 2.0 ** -133])])
    bits = ro.f64_to_bf16_bits(x)
    back = ro.bf16_bits_to_f64(bits)
    for xi, bi, yi in zip(x, bits, back):
        if not np.isfinite(yi):
            assert abs(xi) >= (2.0 ** 127) * (2 - 2.0 ** -8)       # beyond the last midpoint
            continue
        # neighbours on the bf16 grid via the integer bit pattern
        mag = int(bi) & 0x7FFF
        cands = [m for m in (mag - 1, mag, mag + 1) if 0 <= m < 0x7F80]
        vals = [Fraction(float(ro.bf16_bits_to_f64(np.array([m], dtype=np.uint16))[0])) for m in cands]
        errs = [abs(Fraction(abs(float(xi))) - v) for v in vals]
        k = cands.index(mag)
        assert errs[k] == min(errs)
        if errs.count(min(errs)) > 1:                                # tie -> even pattern
            assert mag % 2 == 0
        assert (int(bi) >> 15) == int(np.signbit(xi))
    # a case where rounding through FP32 first would go wrong (double rounding)
    tricky = 1.0 + 2.0 ** -8 + 2.0 ** -30          # just above the bf16 midpoint 1 + 2^-8
    assert ro.bf16_bits_to_f64(ro.f64_to_bf16_bits(np.array([tricky])))[0] == 1.0 + 2.0 ** -7
