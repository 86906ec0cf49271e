"""Pins for the oracle's encoder (Eq. 1-3, Eq. 6-7) and matmul (CPU only).

The encoder is an algorithm, so it is pinned by invariants, special cases and brute
force rather than by a second copy of itself.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import razer_oracle as ro
from paper_2501_04052_b200 import inputs

FP4 = np.array([ro.fp4_value(c) for c in range(16)])


def _weights(n, k, seed, outliers=0.001):
    return inputs.student_t_weights(n, k, seed, outlier_frac=outliers).numpy()


def test_tensor_and_block_scale_follow_eq1_eq2():
    w = _weights(64, 256, 0)
    codes, scales, d32 = ro.quantize_weight(w)
    amax = np.max(np.abs(w)).astype(np.float64)
    # Eq. 1 with Qmax_FP8 = 1.875 (6-bit scale) and Qmax_FP4 = 6
    assert abs(float(d32) - amax / (1.875 * 6.0)) <= 1e-6 * amax
    # Eq. 2: the stored scale is the nearest grid value to bmax / (D32 * 6)
    grid = ro.scale_grid(ro.SCALE_E3M3_META2)
    bmax = np.max(np.abs(w.reshape(64, 16, 16)), axis=2).astype(np.float64)
    t = bmax / (float(d32) * 6.0)
    sc = scales & 0x3F
    nearest = np.min(np.abs(grid[None, None, 1:] - t[:, :, None]), axis=2)   # code 0 is not allowed
    got = np.abs(grid[sc] - t)
    assert np.all(got <= nearest * (1 + 1e-5) + 1e-12)
    # the block holding the tensor maximum uses the top of the scale range
    r, b = np.unravel_index(np.argmax(bmax), bmax.shape)
    assert sc[r, b] == 63
    # activations: Qmax_FP8 = 448
    x = inputs.activations(8, 256, 1)
    _, sa, d32a = ro.quantize_act(inputs.bf16_to_bits(x))
    ax = np.max(np.abs(x.float().numpy())).astype(np.float64)
    assert abs(float(d32a) - ax / (448.0 * 6.0)) <= 1e-6 * ax
    assert np.max(sa & 0x7F) == 126


def test_all_zero_and_zero_block():
    w = np.zeros((4, 64), dtype=np.float32)
    codes, scales, d32 = ro.quantize_weight(w)
    assert d32 == 1.0 and not codes.any() and not scales.any()
    w[1, 5] = 0.3
    codes, scales, d32 = ro.quantize_weight(w)
    assert scales[0].sum() == 0 and scales[1, 0] != 0 and scales[1, 1:].sum() == 0
    d2 = ro.dequant_d2(codes, scales, d32)
    assert np.count_nonzero(d2) == 1 and abs(d2[1, 5] - 0.3) < 1e-6


def test_razer_error_never_above_plain_fp4_and_argmin():
    w = _weights(128, 512, 2)
    codes, scales, d32, dbg = ro.quantize_weight(w, return_debug=True)
    e = dbg["errs64"]
    assert np.all(e <= dbg["err_fp4"][None] + 1e-12)              # Q subset of Q + {v}
    chosen = np.take_along_axis(e, dbg["meta"][None].astype(np.int64), axis=0)[0]
    ok = chosen <= e.min(axis=0) * (1 + 1e-5) + 1e-12
    assert np.all(ok | dbg["near_tie"])
    # the achieved error is what the decoded block actually has against xs
    q, s = ro.decode_block_values(codes, scales)
    xs = dbg["xs"].reshape(128, 512).astype(np.float64)
    achieved = np.sum(((q - xs) ** 2).reshape(128, 32, 16), axis=2)
    assert np.allclose(achieved, chosen, rtol=1e-9, atol=1e-12)


def test_special_code_only_where_strictly_closer_and_single_zero():
    w = _weights(64, 512, 3)
    codes, scales, d32, dbg = ro.quantize_weight(w, return_debug=True)
    c = ro.unpack_codes(codes)
    q, s = ro.decode_block_values(codes, scales)
    xs = dbg["xs"].reshape(64, 512).astype(np.float64)
    sv = c == 8
    assert sv.any()
    # where the special code is used it is strictly closer than every FP4 value
    d_sv = np.abs(xs - q)
    d_fp4 = np.min(np.abs(xs[..., None] - FP4[None, None, :]), axis=2)
    assert np.all(d_sv[sv] < d_fp4[sv])
    # where it is not used the element is the nearest FP4 value
    assert np.allclose(np.abs(xs - q)[~sv], d_fp4[~sv], rtol=0, atol=1e-7)
    # true zeros use the non-remapped zero code only
    assert np.all(c[(q == 0)] == 0)


def test_round_trip_requantize_returns_same_codes():
    w = _weights(64, 256, 4)
    codes, scales, d32 = ro.quantize_weight(w)
    d2 = ro.dequant_d2(codes, scales, d32)
    codes2, scales2, d32_2 = ro.quantize_weight(d2, tensor_scale=d32)
    q1, s1 = ro.decode_block_values(codes, scales)
    q2, s2 = ro.decode_block_values(codes2, scales2)
    # same scales wherever the block maximum was kept (always: the max element maps to itself)
    same = (scales & 0x3F) == (scales2 & 0x3F)
    assert same.mean() > 0.98
    m = np.repeat(same, 16, axis=1)
    assert np.array_equal((q1 * np.repeat(s1, 16, axis=1))[m], (q2 * np.repeat(s2, 16, axis=1))[m])


def test_scale_exponent_bias_invariance():
    """A different exponent bias for the 6-bit scale is absorbed by the tensor scale:
    identical codes and an identical dequantized tensor."""
    w = _weights(32, 256, 5)
    c0, s0, d0 = ro.quantize_weight(w)
    c1, s1, d1 = ro.quantize_weight(w, scale_bias_shift=4)       # bias 3: max 30
    assert np.array_equal(c0, c1) and np.array_equal(s0, s1)
    assert float(d1) * 16.0 == float(d0)
    a = ro.dequant_d2(c0, s0, d0)
    b = (np.float32(d1) * (ro.dequant_d1(c1, s1) * np.float32(16.0))).astype(np.float32)
    assert np.array_equal(a, b)


def test_zero_code_convention_gives_same_values():
    w = _weights(32, 256, 6)
    c8, s8, d8 = ro.quantize_weight(w, remap_code=0x8)
    c0, s0, d0 = ro.quantize_weight(w, remap_code=0x0)
    assert np.array_equal(s8, s0) and d8 == d0
    assert np.array_equal(ro.dequant_d2(c8, s8, d8, remap_code=0x8),
                          ro.dequant_d2(c0, s0, d0, remap_code=0x0))
    u8, u0 = ro.unpack_codes(c8), ro.unpack_codes(c0)
    assert np.array_equal(np.where((u8 & 7) == 0, u8 ^ 8, u8), u0)


@pytest.mark.parametrize("block", [2, 3])
def test_brute_force_tiny_blocks(block):
    """Enumerate every code vector and every metadata value of a tiny block and check
    that the encoder's choice attains the minimum of Eq. 6 (given its scales)."""
    rng = np.random.default_rng(7 + block)
    w = (rng.standard_t(5, size=(40, block * 4)) * 0.02).astype(np.float32)
    w[0, :block] = [0.5, -0.41][:block] + [0.1] * (block - 2)     # a block near +-5 after scaling
    codes, scales, d32, dbg = ro.quantize(w, ro.SCALE_E3M3_META2, (5.0, 8.0), 0x8, block=block,
                                           return_debug=True)
    q, s = ro.decode_block_values(codes, scales, block=block)
    xs = dbg["xs"].astype(np.float64)                               # [R, nb, block]
    qb = q.reshape(xs.shape)
    cands = ro.sv_candidates((5.0, 8.0), ro.SCALE_E3M3_META2)
    for r in range(xs.shape[0]):
        for b in range(xs.shape[1]):
            best = np.inf
            for v in cands:
                vals = np.array([ro.fp4_value(c) if c != 8 else v for c in range(16)])
                for vec in itertools.product(range(16), repeat=block):
                    e = float(np.sum((vals[list(vec)] - xs[r, b]) ** 2))
                    best = min(best, e)
            got = float(np.sum((qb[r, b] - xs[r, b]) ** 2))
            assert got <= best * (1 + 1e-9) + 1e-15


def test_activation_double_quantization_picks_better_sign():
    x = inputs.activations(16, 512, 8, outlier_channel_frac=0.01)
    bits = inputs.bf16_to_bits(x)
    codes, scales, d32, dbg = ro.quantize_act(bits, return_debug=True)
    assert dbg["errs64"].shape[0] == 2
    better = np.argmin(dbg["errs64"], axis=0)
    assert np.all((better == (scales >> 7)) | dbg["near_tie"] | ((scales & 0x7F) == 0))
    # a supplied tensor scale is used as given
    c2, s2, d2 = ro.quantize_act(bits, tensor_scale=np.float32(2.0) * d32)
    assert d2 == np.float32(2.0) * d32
    assert np.max(s2 & 0x7F) < np.max(scales & 0x7F)


def test_sv_pair_5_minimises_error_on_student_t():
    """Sec. 4.2: with a single pair of special values the error is lowest at +-5."""
    w = _weights(256, 1024, 9, outliers=0.0)
    tot = {}
    for m in (3.5, 4.5, 5.0, 5.5, 7.0, 8.0):
        codes, scales, d32 = ro.quantize_weight(w, sv_mag=(m, m))
        d2 = ro.dequant_d2(codes, scales, d32)
        tot[m] = float(np.sum((d2.astype(np.float64) - w) ** 2))
    plain = ro.quantize(w, ro.SCALE_E3M3_META2, (6.0, 6.0), 0x8)   # 6 is already an FP4 value: no gain
    tot_plain = float(np.sum((ro.dequant_d2(plain[0], plain[1], plain[2], sv_mag=(6.0, 6.0)) - w) ** 2))
    assert min(tot, key=tot.get) == 5.0
    assert tot[5.0] < 0.95 * tot_plain


def test_matmul_matches_library_on_plain_codes():
    """With only standard codes the product is an ordinary matmul of the decoded bf16 weights."""
    rng = np.random.default_rng(10)
    c = rng.integers(0, 16, (48, 256), dtype=np.uint8)
    c[c == 8] = 0
    codes = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    scales = rng.integers(24, 56, (48, 16), dtype=np.uint8)
    x = inputs.activations(5, 256, 11)
    y = ro.matmul_w4a16(inputs.bf16_to_bits(x), codes, scales, np.float32(0.37))
    d1 = torch.from_numpy(ro.dequant_d1(codes, scales))
    assert torch.equal(d1.to(torch.bfloat16).float(), d1)              # D1 fits bf16 exactly
    ref = 0.37 * (x.double() @ d1.double().T)
    got = torch.from_numpy(ro.bf16_bits_to_f64(y))
    assert torch.allclose(got, ref, rtol=2 ** -8, atol=1e-6)
    # rounding to bf16 once costs about 1.7e-3 relative Frobenius error against the unrounded result
    y64 = ro.matmul_w4a16(inputs.bf16_to_bits(x), codes, scales, np.float32(0.37), round_output=False)
    rel = np.linalg.norm(ro.bf16_bits_to_f64(y) - y64) / np.linalg.norm(y64)
    assert 5e-4 < rel < 3e-3


def test_matmul_linear_in_special_value_term():
    """sum_k x*q = sum over standard codes + sv * sum of x at the remapped positions."""
    rng = np.random.default_rng(12)
    codes = rng.integers(0, 256, (16, 64), dtype=np.uint8)
    scales = np.full((16, 8), (2 << 6) | 56, dtype=np.uint8)           # scale 1.0, meta 2 -> -5
    x = inputs.activations(3, 128, 13)
    xb = inputs.bf16_to_bits(x)
    y = ro.matmul_w4a16(xb, codes, scales, np.float32(1.0), round_output=False)
    c = ro.unpack_codes(codes)
    std = np.where(c == 8, 0.0, FP4[c])
    xf = x.double().numpy()
    want = xf @ std.T + (-5.0) * (xf @ (c == 8).astype(np.float64).T)
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)


def test_w4a4_matmul_against_dequantized_product():
    w = _weights(32, 256, 14)
    x = inputs.activations(6, 256, 15, outlier_channel_frac=0.01)
    wc, ws, wd = ro.quantize_weight(w)
    ac, as_, ad = ro.quantize_act(inputs.bf16_to_bits(x))
    y = ro.matmul_w4a4(ac, as_, ad, wc, ws, wd, round_output=False)
    a2 = ro.dequant_d2(ac, as_, ad, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0,)).astype(np.float64)
    w2 = ro.dequant_d2(wc, ws, wd).astype(np.float64)
    assert np.allclose(y, a2 @ w2.T, rtol=1e-5, atol=1e-7)
    # and the quantized product approximates the real one
    ref = x.double().numpy() @ w.astype(np.float64).T
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 0.2


# --------------------------------------------------------------------------
# block sizes 32 / 64 / 128 (the block-size study of Sec. 5; Sec. 4.3 deploys 128)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("block", [32, 64, 128])
def test_larger_blocks_scale_and_error_invariants(block):
    """One scale and one special value per `block` elements: the scale follows Eq. 2 on the block's maximum, the
    error with the special value never exceeds plain FP4 at the same scale (Q is a subset of Q + {v}), the decoded
    block attains the error the encoder reported, and element-wise optimality holds given (scale, v): every code is
    the nearest member of Q + {v}."""
    w = _weights(64, 1024, 30 + block)
    codes, scales, d32, dbg = ro.quantize(w, ro.SCALE_E3M3_META2, (5.0, 8.0), 0x8, block=block, return_debug=True)
    nb = 1024 // block
    assert scales.shape == (64, nb)
    bmax = np.abs(w).reshape(64, nb, block).max(axis=2)
    t = (bmax / np.float32(d32 * np.float32(6.0))).astype(np.float32)
    want = ro.round_to_scale(t, ro.SCALE_E3M3_META2)
    want = np.where((bmax > 0) & (want == 0), 1, want)
    assert np.array_equal(scales & 0x3F, want)
    e = dbg["errs64"]
    assert np.all(e <= dbg["err_fp4"][None] + 1e-12)
    chosen = np.take_along_axis(e, dbg["meta"][None].astype(np.int64), axis=0)[0]
    assert np.all((chosen <= e.min(axis=0) * (1 + 1e-5) + 1e-12) | dbg["near_tie"])
    q, s = ro.decode_block_values(codes, scales, block=block)
    xs = dbg["xs"].reshape(64, 1024).astype(np.float64)
    achieved = np.sum(((q - xs) ** 2).reshape(64, nb, block), axis=2)
    assert np.allclose(achieved, chosen, rtol=1e-9, atol=1e-12)
    # nearest member of Q + {v}, element by element (brute force over the 16 values)
    sv = np.repeat(np.array(ro.sv_candidates((5.0, 8.0), ro.SCALE_E3M3_META2))[dbg["meta"]], block, axis=1)
    fp4 = np.array(sorted({ro.fp4_value(c) for c in range(16)}))
    d_best = np.minimum(np.min(np.abs(xs[:, :, None] - fp4[None, None, :]), axis=2), np.abs(xs - sv))
    assert np.allclose(np.abs(q - xs), d_best, rtol=0, atol=1e-12)


@pytest.mark.parametrize("block", [32, 64, 128])
def test_larger_blocks_decode_equals_block16_with_repeated_scale_bytes(block):
    """A block of 16 k elements with one scale byte decodes exactly like k blocks of 16 that carry the same byte:
    this is what lets the packed form keep one byte per 16 elements for every block size."""
    w = _weights(32, 512, 40 + block)
    codes, scales, d32 = ro.quantize(w, ro.SCALE_E3M3_META2, (5.0, 9.0), 0x0, block=block)
    a = ro.dequant_d2(codes, scales, d32, sv_mag=(5.0, 9.0), remap_code=0x0, block=block)
    b = ro.dequant_d2(codes, np.repeat(scales, block // 16, axis=1), d32, sv_mag=(5.0, 9.0), remap_code=0x0)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    # and a larger block can only do worse than (or as well as) its 16-element sub-blocks quantized on their own
    c16, s16, d16 = ro.quantize(w, ro.SCALE_E3M3_META2, (5.0, 9.0), 0x0, block=16, tensor_scale=d32)
    e_big = np.sum((a.astype(np.float64) - w) ** 2)
    e_16 = np.sum((ro.dequant_d2(c16, s16, d16, sv_mag=(5.0, 9.0), remap_code=0x0).astype(np.float64) - w) ** 2)
    assert e_16 <= e_big * 1.02


# --------------------------------------------------------------------------
# scale-aware special-value selection (Eq. 6-7 with the scale of Eq. 2 chosen together with v)
# --------------------------------------------------------------------------

def _err_in_tensor_units(w, codes, scales, d32, **kw):
    d2 = ro.dequant_d2(codes, scales, d32, **kw).astype(np.float64)
    return ((d2 - w.astype(np.float64)) ** 2).reshape(w.shape[0], -1, 16).sum(axis=2)


def test_scale_aware_reaches_a_special_value_beyond_six_exactly():
    """A block that is exactly s * [8, 1, -2, 3, 0.5, ...]: with Eq. 2's Qmax = 6 the 8 cannot be hit (the scale
    makes it 6 and the rest moves off the grid); with the scale chosen for v = 8 the block is reproduced exactly."""
    vals = np.array([8, 1, -2, 3, 0.5, -1.5, 4, 6, 0, -0.5, 2, -3, 1, 1.5, -4, 0.5], dtype=np.float32)
    s = np.float32(ro.e4m3_value(20))                              # a scale in the middle of the E3M3 grid
    w = np.stack([vals * s, -vals * s]).astype(np.float32)
    d32 = np.float32(1.0)
    c, sc, _ = ro.quantize_scale_aware(w, tensor_scale=d32)
    assert np.array_equal(ro.dequant_d2(c, sc, d32), w)            # exact, for +8 and for -8
    assert list(sc >> 6) == [[1], [3]] and list(sc & 0x3F) == [[20], [20]]
    c0, s0, _ = ro.quantize_weight(w, tensor_scale=d32)
    assert _err_in_tensor_units(w, c0, s0, d32).min() > 0          # the plain selection cannot


def test_scale_aware_never_worse_and_identical_without_large_special_values():
    w = _weights(96, 512, 50)
    c1, s1, d1, dbg = ro.quantize_scale_aware(w, return_debug=True)
    c0, s0, d0 = ro.quantize_weight(w)
    assert d0 == d1
    e1, e0 = _err_in_tensor_units(w, c1, s1, d1), _err_in_tensor_units(w, c0, s0, d0)
    assert np.all((e1 <= e0 * (1 + 1e-5) + 1e-18) | dbg["near_tie"])      # a superset of candidates
    assert e1.sum() < e0.sum()                                           # and +-8 now does get used
    used8 = ((s1 >> 6) & 1) == 1
    assert used8.mean() > ((s0 >> 6) & 1).mean()
    # the reported minimum is what the decoded block has
    got = np.take_along_axis(dbg["errs64"], dbg["pick"][None], axis=0)[0]
    assert np.allclose(e1, got, rtol=1e-4, atol=1e-16)     # xs is rounded to FP32 on the way
    # no special value beyond 6: the candidate list is the plain one, the result identical
    a = ro.quantize_scale_aware(w, sv_mag=(2.5, 5.0))
    b = ro.quantize_weight(w, sv_mag=(2.5, 5.0))
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_scale_aware_brute_force_over_its_candidates_on_tiny_blocks():
    """Blocks of two elements: for every (special value, scale) candidate the method allows, enumerate all 256 code
    vectors; the encoder's choice attains the minimum of the reconstruction error over all of them."""
    rng = np.random.default_rng(11)
    w = (rng.standard_t(5, size=(30, 8)) * 0.02).astype(np.float32)
    c, s, d32 = ro.quantize_scale_aware(w, block=2)
    q, sv = ro.decode_block_values(c, s, block=2)
    got = (((q * np.repeat(sv, 2, axis=1) * float(d32)) - w) ** 2).reshape(30, 4, 2).sum(axis=2)
    cands = ro.sv_candidates((5.0, 8.0), ro.SCALE_E3M3_META2)
    grid = ro.scale_grid(ro.SCALE_E3M3_META2)
    wb = w.reshape(30, 4, 2).astype(np.float64)
    for r in range(30):
        for b in range(4):
            bmax = np.abs(wb[r, b]).max()
            top_neg = wb[r, b][np.argmax(np.abs(wb[r, b]))] < 0
            best = np.inf
            for v in cands:
                for qmax in ([6.0, abs(v)] if abs(v) > 6 and (v < 0) == top_neg else [6.0]):
                    t = np.float32(np.float32(bmax) / np.float32(d32 * np.float32(qmax)))
                    sc = max(int(ro.round_to_scale(np.array([t]), ro.SCALE_E3M3_META2)[0]), 1)
                    step = float(np.float32(d32 * np.float32(grid[sc])))
                    vals = np.array([ro.fp4_value(k) if k != 8 else v for k in range(16)]) * step
                    e = (vals[:, None] - wb[r, b][None, :]) ** 2       # [16 values, 2 elements]
                    best = min(best, e[:, 0].min() + e[:, 1].min())
            assert got[r, b] <= best * (1 + 1e-4) + 1e-18      # midpoint decisions are taken on FP32-rounded xs


# --------------------------------------------------------------------------
# plain NVFP4 (Sec. 3, Eq. 1-3): the activation format of the two-pass realization (App. D.3)
# --------------------------------------------------------------------------

def test_plain_nvfp4_is_eq_1_to_3_alone():
    x = inputs.activations(6, 512, 31, outlier_channel_frac=0.02)
    xb = inputs.bf16_to_bits(x)
    c, s, d32, dbg = ro.quantize_act(xb, sv_mag=None, return_debug=True)
    # no special-value code, no metadata bit; decoding it as RaZeR or as NVFP4 is the same thing
    nib = ro.unpack_codes(c)
    assert not np.any(nib == 0x8) and not np.any(s & 0x80)
    xf = ro.bf16_bits_to_f32(xb).astype(np.float64)
    # Eq. 3 by brute force: every element is the nearest point of the FP4 grid to xs (ties aside)
    grid = np.array(sorted({ro.fp4_value(k) for k in range(16)}))
    xs = dbg["xs"].astype(np.float64).reshape(6, 512)
    q, sv = ro.decode_block_values(c, s, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0, 5.0))
    nearest = np.abs(xs[..., None] - grid).min(axis=-1)
    assert np.all(np.abs(xs - q) <= nearest + 1e-6)
    # Eq. 6's invariant: adding a special value never raises a block's error at the same scale
    c2, s2, d2, dbg2 = ro.quantize_act(xb, sv_mag=(5.0,), return_debug=True)
    assert d2 == d32 and np.array_equal(s & 0x7F, s2 & 0x7F)
    assert np.all(dbg2["errs64"].min(axis=0) <= dbg["err_fp4"] + 1e-12)
    # re-quantizing the dequantized tensor with the same tensor scale returns the same codes
    d2v = ro.dequant_d2(c, s, d32, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0, 5.0)).astype(np.float32)
    c3, s3, _ = ro.quantize(d2v, ro.SCALE_E4M3_META1, None, tensor_scale=d32)
    assert np.array_equal(c3, c) and np.array_equal(s3, s)
    assert np.linalg.norm(d2v - xf) / np.linalg.norm(xf) < 0.12


# --------------------------------------------------------------------------
# deployment variant of Sec. 4.3: block 128, FP16 block scale carrying the metadata (oracle only)
# --------------------------------------------------------------------------

def test_fp16_block_scale_variant_bits_and_exact_cases():
    """Sec. 4.3: the FP16 scale's sign bit and most significant exponent bit hold the metadata.  A block that is an
    FP16 scale times grid values (special value included) is reproduced exactly, for each of the four special values;
    the stored scale always has bit 14 clear once the metadata is masked off."""
    rng = np.random.default_rng(5)
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
    rows = []
    svs = [5.0, 4.5, -5.0, -4.5]                       # both magnitudes below 6, so that Eq. 2's scale lets them be hit
    for v in svs:
        q = rng.choice(grid, size=128) * rng.choice([-1.0, 1.0], size=128)
        q[0] = 6.0 if v > 0 else -6.0                   # pins the scale: bmax / 6 = s exactly
        q[1:9] = v                                     # eight special values: no other candidate can match
        rows.append(q * 0.0123291015625)               # an FP16-representable scale (101 * 2^-13)
    w = np.array(rows, dtype=np.float32)
    codes, s16 = ro.quantize_fp16_block(w, sv_mag=(5.0, 4.5))
    assert [int(v) for v in (s16[:, 0] >> 14) & 3] == [0, 1, 2, 3]          # [sign | select] = metadata order +m0 +m1 -m0 -m1
    assert np.all((s16 & 0x3FFF).view(np.float16).astype(np.float64) == 0.0123291015625)
    assert np.array_equal(ro.dequant_fp16_block(codes, s16, sv_mag=(5.0, 4.5)), w.astype(np.float64))
    # random weights: metadata-free scale is a positive FP16 below 2, Eq. 6 invariant, idempotent re-quantization
    w = _weights(64, 1024, 60)
    codes, s16, dbg = ro.quantize_fp16_block(w, return_debug=True)
    sval = (s16 & 0x3FFF).view(np.float16).astype(np.float64)
    assert np.all((sval > 0) & (sval < 2)) and np.all(((s16 & 0x3FFF) >> 14) == 0)
    assert np.all(dbg["errs64"].min(axis=0) <= dbg["err_fp4"] + 1e-12)
    d = ro.dequant_fp16_block(codes, s16)
    c2, s2 = ro.quantize_fp16_block(d.astype(np.float32))
    assert np.array_equal(s2 & 0x3FFF, s16 & 0x3FFF)
    assert np.allclose(ro.dequant_fp16_block(c2, s2), d, rtol=0, atol=0) or np.mean(c2 == codes) > 0.999
    assert np.linalg.norm(d - w) / np.linalg.norm(w) < 0.15


def test_fp16_block_scale_variant_brute_force_on_tiny_blocks():
    """Eq. 6-7 by enumeration on blocks of two elements: the encoder's reconstruction error equals the minimum over
    the four special values and all 256 code vectors at the block's FP16 scale."""
    rng = np.random.default_rng(12)
    w = (rng.standard_t(5, size=(40, 4)) * 0.02).astype(np.float32)
    codes, s16 = ro.quantize_fp16_block(w, block=2)
    got = ((ro.dequant_fp16_block(codes, s16, block=2) - w.astype(np.float64)) ** 2).reshape(40, 2, 2).sum(axis=2)
    cands = ro.sv_candidates((5.0, 8.0), ro.SCALE_E3M3_META2)
    sval = (s16 & 0x3FFF).view(np.float16).astype(np.float64)
    wb = w.reshape(40, 2, 2).astype(np.float64)
    for r in range(40):
        for b in range(2):
            best = np.inf
            for v in cands:
                vals = np.array([ro.fp4_value(k) if k != 8 else v for k in range(16)]) * sval[r, b]
                e = (vals[:, None] - wb[r, b][None, :]) ** 2
                best = min(best, e[:, 0].min() + e[:, 1].min())
            assert got[r, b] <= best * (1 + 1e-4) + 1e-18
