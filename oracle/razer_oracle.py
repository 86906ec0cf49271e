"""RaZeR reference oracle (TEST INFRASTRUCTURE, not a product path).

A plain, slow, obviously-correct CPU statement of what the RaZeR matmul path
computes, written from the paper (arXiv 2501.04052).  Only the tests, the
smoke check and the benchmark's cpu-baseline leg may import this module; the
CUDA library never does, and the two share no code.

What is here, with the passage each function follows:

  fp4_value            Eq. 5   (FP4-E2M1 element value)
  e4m3_value           Eq. 4   (FP8-E4M3 value, sign ignored: Sec. 4.1)
  scale_grid           Sec. 4.1 (E4M3 7-bit activation scale, E3M3 6-bit weight scale)
  round_to_scale       Eq. 2's rounding onto the scale grid
  round_to_fp4         Eq. 3's rounding onto the FP4 set
  offset_decoder_sv    Sec. 4.4 (offset-register special-value decoder)
  quantize             Eq. 1-3 + Eq. 6-7 (tensor scale, block scale, special-value argmin)
  quantize_scale_aware Eq. 6-7 with the block scale of Eq. 2 chosen together with the special value
  decode_block_values  Sec. 4.2 + Sec. 4.4 (code -> value with the remapped zero)
  dequant_d1/_d2       the dequantization product Delta32 * Delta8 * Xbar (Sec. 3)
  matmul_w4a16/_w4a4   definition: FP64-accumulated product rounded once to bf16
  two_pass_split       App. D.3 (B_main / B_comp decomposition)
  quantize_fp16_block / dequant_fp16_block   Sec. 4.3 (deployment variant: block 128, FP16 block scale whose sign
                       bit and top exponent bit carry the metadata); oracle only, no CUDA counterpart

Floating point: the encoder works in FP32 in the operation order stated in each
docstring (numpy float32 ops are IEEE, one rounding per op, never fused); the
matmul accumulates in FP64.  bf16 tensors are carried as uint16 bit patterns.

Parity status: every function below is pinned by tests/test_oracle_*.py against
values the paper prints, library casts, closed forms or brute force.  What stays
"parity unpinned" is the set of conventions the paper leaves open (tie-breaks,
clamps, bit positions inside the bytes): those are this build's readings and can
not be checked against the authors' code.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# Formats
# --------------------------------------------------------------------------

BLOCK = 16
SCALE_E3M3_META2 = 0   # weights: 6-bit scale, 2 metadata bits (Sec. 4.1, 4.2)
SCALE_E4M3_META1 = 1   # activations: 7-bit scale, 1 metadata bit

# Special values expressible as a sum of two FP4 values (App. D.3, "Generality").
ALLOWED_SV_MAGNITUDES = (2.5, 3.5, 4.5, 5.0, 5.5, 6.5, 7.0, 7.5, 8.0, 9.0, 10.0, 12.0)


def fp4_value(code: int) -> float:
    """Eq. 5: nibble S E1 E0 M -> (-1)^S 2^(E-1) (1+M/2) if E != 0 else (-1)^S M/2."""
    s = (code >> 3) & 1
    e = (code >> 1) & 3
    m = code & 1
    mag = (2.0 ** (e - 1)) * (1.0 + m / 2.0) if e != 0 else m / 2.0
    return -mag if s else mag


def e4m3_value(code: int) -> float:
    """Eq. 4 without the sign (block scales are never negative, Sec. 4.1).

    code = E3 E2 E1 E0 M2 M1 M0 (7 bits): 2^(E-7) (1+M/8) if E != 0 else 2^-6 M/8.
    """
    e = (code >> 3) & 0xF
    m = code & 7
    return (2.0 ** (e - 7)) * (1.0 + m / 8.0) if e != 0 else (2.0 ** -6) * (m / 8.0)


def scale_grid(scale_fmt: int) -> np.ndarray:
    """All representable block-scale values, indexed by scale code (ascending).

    E4M3 (activations): codes 0..126; code 127 (E=15, M=7) is the NaN encoding of
    the OCP E4M3 format the paper cites and is never produced, so the maximum is 448.
    E3M3 (weights): the 6-bit format of Sec. 4.1, read as the low six bits of an
    E4M3 byte with the top exponent bit zero: codes 0..63, maximum 1.875.
    """
    n = 127 if scale_fmt == SCALE_E4M3_META1 else 64
    return np.array([e4m3_value(c) for c in range(n)], dtype=np.float64)


def scale_max(scale_fmt: int) -> float:
    return float(scale_grid(scale_fmt)[-1])


def meta_bits(scale_fmt: int) -> int:
    return 1 if scale_fmt == SCALE_E4M3_META1 else 2


def round_to_scale(t: np.ndarray, scale_fmt: int) -> np.ndarray:
    """Round non-negative FP32 values to scale codes (the rounding in Eq. 2).

    Round to nearest, ties to the code with an even mantissa, saturate at the
    format's maximum.  (Clamping a positive value that rounds to zero is done by
    the caller, which knows whether the block is empty.)
    """
    grid = scale_grid(scale_fmt)
    t64 = np.asarray(t, dtype=np.float64)
    hi = np.searchsorted(grid, t64, side="left")          # first grid value >= t
    hi = np.clip(hi, 0, len(grid) - 1)
    lo = np.clip(hi - 1, 0, len(grid) - 1)
    d_lo = t64 - grid[lo]
    d_hi = grid[hi] - t64
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo)
    code = np.where(t64 >= grid[-1], len(grid) - 1, code)
    code = np.where(t64 <= 0, 0, code)
    return code.astype(np.uint8)


_FP4_MAGS = np.array([fp4_value(c) for c in range(8)], dtype=np.float64)  # 0 .5 1 1.5 2 3 4 6


def round_to_fp4(xs: np.ndarray) -> np.ndarray:
    """The rounding of Eq. 3: nearest FP4 magnitude index (0..7) for |xs|.

    Round to nearest; a value halfway between two FP4 values goes to the one whose
    mantissa bit is 0 (0.25->0, 0.75->1, 1.25->1, 1.75->2, 2.5->2, 3.5->4, 5->4);
    magnitudes above 6 saturate to 6.  Returns the magnitude index; the sign is
    kept by the caller.
    """
    a = np.abs(np.asarray(xs, dtype=np.float64))
    hi = np.clip(np.searchsorted(_FP4_MAGS, a, side="left"), 0, 7)
    lo = np.clip(hi - 1, 0, 7)
    d_lo = a - _FP4_MAGS[lo]
    d_hi = _FP4_MAGS[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    idx = np.where(pick_hi, hi, lo)
    idx = np.where(a >= 6.0, 7, idx)
    return idx.astype(np.uint8)


def offset_decoder_sv(offset_reg: int, sign_bit: int) -> float:
    """Sec. 4.4: a 4-bit sign-magnitude fixed-point offset (1 sign, 2 integer, 1
    fraction bit) is added to 6.0 to give the magnitude; the metadata sign bit is
    then attached."""
    s = (offset_reg >> 3) & 1
    mag = ((offset_reg >> 1) & 3) + 0.5 * (offset_reg & 1)
    off = -mag if s else mag
    v = 6.0 + off
    return -v if sign_bit else v


def sv_candidates(sv_mag, scale_fmt: int):
    """Allowed special values in metadata order (Sec. 4.2, Sec. 4.4).

    Weights (2 bits): meta = sign*2 + select -> [+m0, +m1, -m0, -m1].
    Activations (1 bit): meta = sign -> [+m0, -m0].
    """
    if scale_fmt == SCALE_E4M3_META1:
        return [float(sv_mag[0]), -float(sv_mag[0])]
    return [float(sv_mag[0]), float(sv_mag[1]), -float(sv_mag[0]), -float(sv_mag[1])]


# --------------------------------------------------------------------------
# bf16 helpers (bf16 carried as uint16 patterns)
# --------------------------------------------------------------------------

def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round FP64 directly to bf16 (nearest, ties to even), with no FP32 step in
    between.  Overflow gives infinity; results below the bf16 normal range are
    rounded on the subnormal grid (quantum 2^-133)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    sign = np.signbit(x)
    a = np.abs(x)
    # normal range: keep 8 significant bits
    finite = np.isfinite(a)
    af = np.where(finite, a, 1.0)
    with np.errstate(over="ignore"):
        _, ex = np.frexp(af)                           # af = m * 2^ex, m in [0.5, 1)
        e = np.maximum(ex.astype(np.int64) - 1, -126)  # subnormal grid below 2^-126
        q = np.ldexp(1.0, e - 7)                       # quantum: 7 fraction bits
        r = np.rint(af / q) * q                        # np.rint = ties to even; af/q is exact
    r = np.where(finite, r, a)
    r32 = r.astype(np.float32)                          # exact: r has <= 8 significant bits (or inf)
    r32 = np.where(r >= 2.0 ** 128, np.float32(np.inf), r32)
    bits = (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    out[...] = bits | (sign.astype(np.uint16) << np.uint16(15))
    return out


# --------------------------------------------------------------------------
# Encoder (Eq. 1-3, Eq. 6-7)
# --------------------------------------------------------------------------

def quantize(x: np.ndarray, scale_fmt: int = SCALE_E3M3_META2, sv_mag=(5.0, 8.0),
             remap_code: int = 0x8, block: int = BLOCK, tensor_scale=None,
             scale_bias_shift: int = 0, return_debug: bool = False):
    """RaZeR-quantize a 2-D FP32 tensor, blocks of `block` elements along the last axis.

    Steps (FP32, one rounding per operation, in this order):
      1. Eq. 1: amax = max|x|; D32 = amax / fl32(Smax*6).  amax == 0 -> D32 = 1 and
         every code is zero.  A caller-supplied `tensor_scale` replaces step 1.
      2. Eq. 2: per block bmax = max|x_i|; t = bmax / fl32(D32*6); s = round(t) on the
         scale grid, saturating; bmax > 0 with s == 0 is clamped to the smallest
         positive scale; bmax == 0 gives scale code 0 and zero codes.
      3. xs_j = x_ij / fl32(D32 * s)                      (the X^Scaled of Eq. 6)
      4. Eq. 6: for every allowed special value v, q_j(v) = v if |xs_j - v| is strictly
         smaller than |xs_j - r(xs_j)| else r(xs_j), r = round_to_fp4 with sign;
         err(v) = sum_j (q_j(v) - xs_j)^2, FP32, ascending j.  The block takes the v
         with the smallest err; equal errors go to the smallest metadata value.
      5. Eq. 7: emit codes with Q + {v}: the special value is the remapped zero code,
         a true zero is always the other zero code; the scale byte carries the
         metadata in its top bit(s).

    `scale_bias_shift` = b rescales the scale grid by 2^b (an exponent-bias change of
    the 6/7-bit scale format); it is used only by the bias-invariance test.

    Returns (codes [R, C/2] uint8 with element 2j in the low nibble, scales [R, C/block]
    uint8, D32 float32) and, if `return_debug`, a dict with xs, the per-candidate FP32
    and FP64 errors and the plain-FP4 error.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 2 and x.shape[1] % block == 0
    assert remap_code in (0x0, 0x8)
    R, C = x.shape
    nb = C // block
    f32 = np.float32
    grid = scale_grid(scale_fmt) * (2.0 ** scale_bias_shift)
    smax = f32(grid[-1])
    cands = sv_candidates(sv_mag, scale_fmt) if sv_mag is not None else []   # None: plain NVFP4, Eq. 1-3 alone
    mbits = meta_bits(scale_fmt)
    shift = 8 - mbits

    if tensor_scale is None:
        amax = f32(np.max(np.abs(x))) if x.size else f32(0)
        d32 = f32(1.0) if amax == 0 else f32(amax / f32(smax * f32(6.0)))
    else:
        d32 = f32(tensor_scale)

    xb = x.reshape(R, nb, block)
    bmax = np.max(np.abs(xb), axis=2).astype(np.float32)
    t = (bmax / f32(d32 * f32(6.0))).astype(np.float32)
    # rounding on the (possibly bias-shifted) grid: divide out the exact power of two
    scode = round_to_scale((t.astype(np.float64) / (2.0 ** scale_bias_shift)), scale_fmt)
    scode = np.where((bmax > 0) & (scode == 0), 1, scode).astype(np.uint8)
    scode = np.where(bmax == 0, 0, scode).astype(np.uint8)
    sval = grid[scode].astype(np.float32)                     # exact in FP32
    denom = (d32 * sval).astype(np.float32)                   # fl32(D32 * s)
    safe = np.where(denom == 0, f32(1.0), denom)
    xs = (xb / safe[:, :, None]).astype(np.float32)
    xs = np.where(denom[:, :, None] == 0, f32(0.0), xs)

    ridx = round_to_fp4(xs)                                    # magnitude index 0..7
    rval = (np.where(np.signbit(xs), -1.0, 1.0) * _FP4_MAGS[ridx]).astype(np.float32)
    d_r = np.abs(xs - rval).astype(np.float32)

    errs32 = np.empty((len(cands), R, nb), dtype=np.float32)
    errs64 = np.empty((len(cands), R, nb), dtype=np.float64)
    use_sv = np.empty((len(cands), R, nb, block), dtype=bool)
    for ci, v in enumerate(cands):
        d_v = np.abs(xs - f32(v)).astype(np.float32)
        take = d_v < d_r
        q = np.where(take, f32(v), rval).astype(np.float32)
        diff = (q - xs).astype(np.float32)
        sq = (diff * diff).astype(np.float32)
        acc = np.zeros((R, nb), dtype=np.float32)
        for j in range(block):                                 # ascending j, FP32, no fusion
            acc = (acc + sq[:, :, j]).astype(np.float32)
        errs32[ci] = acc
        d64 = q.astype(np.float64) - xs.astype(np.float64)
        errs64[ci] = np.sum(d64 * d64, axis=2)
        use_sv[ci] = take
    if cands:
        meta = np.argmin(errs32, axis=0).astype(np.uint8)      # first minimum = smallest meta
        take = np.take_along_axis(use_sv, meta[None, :, :, None].astype(np.int64), axis=0)[0]
    else:                                                      # no special value: every element keeps r(xs)
        meta = np.zeros((R, nb), dtype=np.uint8)
        take = np.zeros((R, nb, block), dtype=bool)

    other_zero = remap_code ^ 0x8
    std_code = (ridx | (np.signbit(xs).astype(np.uint8) << 3)).astype(np.uint8)
    std_code = np.where(ridx == 0, other_zero, std_code).astype(np.uint8)   # one zero only
    code = np.where(take, np.uint8(remap_code), std_code).astype(np.uint8)
    code = np.where((scode == 0)[:, :, None], np.uint8(other_zero), code)
    code = code.reshape(R, C)
    packed = (code[:, 0::2] | (code[:, 1::2] << 4)).astype(np.uint8)
    sbyte = ((meta.astype(np.uint16) << shift) | scode).astype(np.uint8)
    sbyte = np.where(scode == 0, 0, sbyte).astype(np.uint8)
    if return_debug:
        d0 = rval.astype(np.float64) - xs.astype(np.float64)
        dbg = dict(xs=xs, errs32=errs32, errs64=errs64, err_fp4=np.sum(d0 * d0, axis=2),
                   meta=meta, scode=scode,
                   near_tie=_near_ties(errs64) if len(cands) > 1 else np.zeros((R, nb), dtype=bool))
        return packed, sbyte, d32, dbg
    return packed, sbyte, d32


def quantize_scale_aware(x: np.ndarray, scale_fmt: int = SCALE_E3M3_META2, sv_mag=(5.0, 8.0),
                         remap_code: int = 0x8, block: int = BLOCK, tensor_scale=None,
                         return_debug: bool = False):
    """Eq. 6-7 with the block scale chosen together with the special value.

    Eq. 2 scales a block so that its largest magnitude lands on Qmax = 6, whatever v is
    (Eq. 1-2 do not mention v), so a special value beyond 6 can only be reached where the
    scale clamps.  Here a special value v with |v| > 6 whose sign is that of the block's
    largest element also brings a scale of its own: Eq. 2 with Qmax replaced by |v|, the
    largest magnitude of Q + {v} on that side.  Candidates, in this order:
      0..n-1  the special values in metadata order with the scale of Eq. 2 (as `quantize`)
      n..     for every such v (metadata order) the pair (v, scale of Eq. 2 with Qmax = |v|)
    Each candidate's scaled-domain error e = sum_j (q_j - xs_j)^2 is formed exactly as in
    `quantize` (FP32, ascending j) and compared in the tensor's own units as
    fl32(fl32(d * d) * e) with d = fl32(D32 * s) the candidate's dequantization step; the
    first minimum wins.  D32 stays Eq. 1's.  The output format is unchanged (codes, scale
    byte = metadata | scale code), so every decoder reads it as it stands.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    assert x.ndim == 2 and x.shape[1] % block == 0 and remap_code in (0x0, 0x8)
    R, C = x.shape
    nb = C // block
    f32 = np.float32
    grid = scale_grid(scale_fmt)
    cands = sv_candidates(sv_mag, scale_fmt)
    shift = 8 - meta_bits(scale_fmt)
    if tensor_scale is None:
        amax = f32(np.max(np.abs(x))) if x.size else f32(0)
        d32 = f32(1.0) if amax == 0 else f32(amax / f32(f32(grid[-1]) * f32(6.0)))
    else:
        d32 = f32(tensor_scale)
    xb = x.reshape(R, nb, block)
    absx = np.abs(xb)
    bmax = np.max(absx, axis=2).astype(np.float32)
    top = np.take_along_axis(xb, np.argmax(absx, axis=2)[:, :, None], axis=2)[:, :, 0]   # first largest element
    top_neg = np.signbit(top)

    def scale_for(qmax):
        t = (bmax / f32(d32 * f32(qmax))).astype(np.float32)
        sc = round_to_scale(t, scale_fmt)
        sc = np.where((bmax > 0) & (sc == 0), 1, sc)
        return np.where(bmax == 0, 0, sc).astype(np.uint8)

    def evaluate(v, scode):
        sval = grid[scode].astype(np.float32)
        denom = (d32 * sval).astype(np.float32)
        safe = np.where(denom == 0, f32(1.0), denom)
        xs = (xb / safe[:, :, None]).astype(np.float32)
        xs = np.where(denom[:, :, None] == 0, f32(0.0), xs)
        ridx = round_to_fp4(xs)
        rval = (np.where(np.signbit(xs), -1.0, 1.0) * _FP4_MAGS[ridx]).astype(np.float32)
        take = np.abs(xs - f32(v)).astype(np.float32) < np.abs(xs - rval).astype(np.float32)
        q = np.where(take, f32(v), rval).astype(np.float32)
        diff = (q - xs).astype(np.float32)
        sq = (diff * diff).astype(np.float32)
        acc = np.zeros((R, nb), dtype=np.float32)
        for j in range(block):
            acc = (acc + sq[:, :, j]).astype(np.float32)
        err32 = ((denom * denom).astype(np.float32) * acc).astype(np.float32)
        d64 = (q.astype(np.float64) - xs.astype(np.float64)) * denom.astype(np.float64)[:, :, None]
        other_zero = remap_code ^ 0x8
        std = (ridx | (np.signbit(xs).astype(np.uint8) << 3)).astype(np.uint8)
        std = np.where(ridx == 0, other_zero, std).astype(np.uint8)
        code = np.where(take, np.uint8(remap_code), std).astype(np.uint8)
        code = np.where((scode == 0)[:, :, None], np.uint8(other_zero), code)
        return err32, np.sum(d64 * d64, axis=2), code

    s6 = scale_for(6.0)
    options = [(ci, v, s6, np.ones((R, nb), dtype=bool)) for ci, v in enumerate(cands)]
    for ci, v in enumerate(cands):
        if abs(v) > 6.0:
            options.append((ci, v, scale_for(abs(v)), (top_neg == (v < 0)) & (bmax > 0)))
    errs32 = np.empty((len(options), R, nb), dtype=np.float32)
    errs64 = np.empty((len(options), R, nb), dtype=np.float64)
    codes_all = np.empty((len(options), R, nb, block), dtype=np.uint8)
    for oi, (ci, v, sc, ok) in enumerate(options):
        e32, e64, code = evaluate(v, sc)
        errs32[oi] = np.where(ok, e32, np.float32(np.inf))
        errs64[oi] = np.where(ok, e64, np.inf)
        codes_all[oi] = code
    pick = np.argmin(errs32, axis=0)                                     # first minimum
    code = np.take_along_axis(codes_all, pick[None, :, :, None], axis=0)[0].reshape(R, C)
    meta = np.array([o[0] for o in options], dtype=np.uint8)[pick]
    scode = np.take_along_axis(np.stack([o[2] for o in options]), pick[None], axis=0)[0]
    packed = (code[:, 0::2] | (code[:, 1::2] << 4)).astype(np.uint8)
    sbyte = ((meta.astype(np.uint16) << shift) | scode).astype(np.uint8)
    sbyte = np.where(scode == 0, 0, sbyte).astype(np.uint8)
    if return_debug:
        return packed, sbyte, d32, dict(errs32=errs32, errs64=errs64, pick=pick, n_standard=len(cands),
                                        near_tie=_near_ties(np.where(np.isfinite(errs64), errs64, 1e300)))
    return packed, sbyte, d32


def _near_ties(errs64: np.ndarray) -> np.ndarray:
    """Blocks whose two best candidates are within 1e-6 relative in FP64: there either
    choice minimises Eq. 6 up to rounding, so an independent implementation may differ."""
    s = np.sort(errs64, axis=0)
    return (s[1] - s[0]) <= 1e-6 * np.maximum(s[1], 1e-300)


def quantize_weight(w, sv_mag=(5.0, 8.0), remap_code=0x8, **kw):
    """Offline weight quantization (Sec. 4.2): E3M3 block scale, four special values."""
    return quantize(w, SCALE_E3M3_META2, sv_mag, remap_code, **kw)


def quantize_act(x_bf16_bits, sv_mag=(5.0,), remap_code=0x8, tensor_scale=None, **kw):
    """Online activation quantization (Sec. 4.2, "double quantization"): bf16 input
    widened to FP32, E4M3 block scale, two special values +-sv_mag[0].  sv_mag = None
    gives plain NVFP4 (Sec. 3, Eq. 1-3), the activation format of the two-pass tensor-core
    realization (App. D.3)."""
    x = bf16_bits_to_f32(x_bf16_bits)
    return quantize(x, SCALE_E4M3_META1, None if sv_mag is None else (sv_mag[0], sv_mag[0]), remap_code,
                    tensor_scale=tensor_scale, **kw)


# --------------------------------------------------------------------------
# Decoder
# --------------------------------------------------------------------------

def unpack_codes(codes: np.ndarray) -> np.ndarray:
    codes = np.asarray(codes, dtype=np.uint8)
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 0xF
    out[:, 1::2] = codes >> 4
    return out


def decode_block_values(codes, scales, scale_fmt=SCALE_E3M3_META2, sv_mag=(5.0, 8.0),
                        remap_code=0x8, block=BLOCK):
    """Code -> element value q and scale byte -> block scale s (both FP64, exact).

    The remapped zero code takes the block's special value (Sec. 4.2); the metadata
    in the scale byte's top bit(s) picks it: sign bit, then pair selector (Sec. 4.4).
    """
    c = unpack_codes(codes)
    R, C = c.shape
    scales = np.asarray(scales, dtype=np.uint8)
    mb = meta_bits(scale_fmt)
    meta = scales >> (8 - mb)
    scode = scales & ((1 << (8 - mb)) - 1)
    s = np.array([e4m3_value(v) for v in range(128)], dtype=np.float64)[scode]
    cands = np.array(sv_candidates(sv_mag if len(sv_mag) > 1 else (sv_mag[0], sv_mag[0]),
                                   scale_fmt), dtype=np.float64)
    sv = cands[meta]                                            # [R, nb]
    table = np.array([fp4_value(k) for k in range(16)], dtype=np.float64)
    q = table[c]
    q = np.where(c == (remap_code ^ 0x8), 0.0, q)
    svb = np.repeat(sv, block, axis=1)
    q = np.where(c == remap_code, svb, q)
    return q, s


def dequant_d1(codes, scales, **kw):
    """D1 = q * Delta8 (exact; fits bf16).  Returned as float32.  A zero product is
    written as +0 (the sign of a zero carries no information in the format)."""
    block = kw.get("block", BLOCK)
    q, s = decode_block_values(codes, scales, **kw)
    return (q * np.repeat(s, block, axis=1) + 0.0).astype(np.float32)


def dequant_d2(codes, scales, tensor_scale, **kw):
    """D2 = fl32(Delta32 * D1): the dequantized tensor, one FP32 rounding."""
    return (np.float32(tensor_scale) * dequant_d1(codes, scales, **kw)).astype(np.float32)


# --------------------------------------------------------------------------
# Matmul (definition)
# --------------------------------------------------------------------------

def matmul_w4a16(x_bf16_bits, codes, scales, tensor_scale, round_output=True, **kw):
    """Y[m,n] = bf16( D32 * sum_k x[m,k] * D1[n,k] ), FP64 accumulation, one rounding."""
    x = bf16_bits_to_f64(x_bf16_bits)
    d1 = dequant_d1(codes, scales, **kw).astype(np.float64)
    y = float(np.float32(tensor_scale)) * (x @ d1.T)
    return f64_to_bf16_bits(y) if round_output else y


def matmul_w4a4(a_codes, a_scales, a_tensor_scale, w_codes, w_scales, w_tensor_scale,
                sv_mag_w=(5.0, 8.0), sv_mag_a=(5.0,), remap_code=0x8, round_output=True):
    """Y = bf16( D32w * D32a * sum_k D1a[m,k] * D1w[n,k] ), FP64 accumulation."""
    da = dequant_d1(a_codes, a_scales, scale_fmt=SCALE_E4M3_META1, sv_mag=sv_mag_a,
                    remap_code=remap_code).astype(np.float64)
    dw = dequant_d1(w_codes, w_scales, scale_fmt=SCALE_E3M3_META2, sv_mag=sv_mag_w,
                    remap_code=remap_code).astype(np.float64)
    y = (float(np.float32(w_tensor_scale)) * float(np.float32(a_tensor_scale))) * (da @ dw.T)
    return f64_to_bf16_bits(y) if round_output else y


def rel_frobenius(a_bits, b_bits) -> float:
    a = bf16_bits_to_f64(a_bits)
    b = bf16_bits_to_f64(b_bits)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


# --------------------------------------------------------------------------
# Two-pass decomposition (App. D.3)
# --------------------------------------------------------------------------

def two_pass_split(codes, scales, sv_mag=(5.0, 8.0), remap_code=0x8):
    """B_main: the remapped zero becomes a signed FP4 base value, everything else is
    unchanged.  B_comp: the remapped zero becomes the signed FP4 remainder, everything
    else is zero.  Returns the two element-value arrays (FP64) and the base/remainder
    pair chosen for each magnitude."""
    fp4 = sorted(set(abs(fp4_value(c)) for c in range(16)) - {0.0})
    pairs = {float(m): [(a, m - a) for a in fp4 if (m - a) in fp4] for m in sv_mag}
    for m, p in pairs.items():
        if not p:
            raise ValueError(f"{m} is not a sum of two FP4 values")
    # B_main holds one base per block whatever the selector says, so prefer the largest
    # base shared by all magnitudes (4 for {5, 8}: 4+1 and 4+4, the paper's example);
    # without a shared base each magnitude takes its own largest one.
    common = set.intersection(*[{a for a, _ in p} for p in pairs.values()])
    split = {}
    for m, p in pairs.items():
        a = max(common) if common else max(a for a, _ in p)
        split[m] = (a, m - a)
    q, _ = decode_block_values(codes, scales, SCALE_E3M3_META2, sv_mag, remap_code)
    c = unpack_codes(codes)
    is_sv = c == remap_code
    base = np.zeros_like(q)
    rem = np.zeros_like(q)
    for m, (a, b) in split.items():
        sel = is_sv & (np.abs(q) == m)
        base = np.where(sel, np.sign(q) * a, base)
        rem = np.where(sel, np.sign(q) * b, rem)
    main = np.where(is_sv, base, q)
    comp = np.where(is_sv, rem, 0.0)
    return main, comp, split


# --------------------------------------------------------------------------
# Deployment variant of the weight-only kernel (Sec. 4.3): block 128, FP16 block scale
# --------------------------------------------------------------------------

def quantize_fp16_block(w: np.ndarray, sv_mag=(5.0, 8.0), remap_code: int = 0x8, block: int = 128,
                        return_debug: bool = False):
    """Sec. 4.3: one FP16 scale per block of `block` weights; its sign bit (bit 15) and most
    significant exponent bit (bit 14) are redundant (a scale is positive and, for weights,
    far below 2) and carry the 2-bit metadata (bit 15 = sign of the special value, bit 14 =
    which magnitude, as in the 8-bit format).  There is no tensor scale.

    Steps (FP32 unless stated): bmax = max|w| of the block; s = fl16(bmax / 6) (round to
    nearest even onto FP16, then clamped into [2^-24, 2 - 2^-10] so that bit 14 stays
    clear and a non-empty block keeps a positive scale); xs = w / fl32(s); Eq. 6-7 over
    the whole block exactly as `quantize` does (candidates in metadata order, FP32 error
    sums in ascending element order, first minimum).  Returns (codes [R, C/2] uint8,
    scales [R, C/block] uint16).
    """
    w = np.ascontiguousarray(w, dtype=np.float32)
    assert w.ndim == 2 and w.shape[1] % block == 0 and remap_code in (0x0, 0x8)
    R, C = w.shape
    nb = C // block
    f32 = np.float32
    wb = w.reshape(R, nb, block)
    bmax = np.max(np.abs(wb), axis=2).astype(np.float32)
    s16 = (bmax / f32(6.0)).astype(np.float32).astype(np.float16)
    s16 = np.clip(s16, np.float16(2.0 ** -24), np.float16(2.0 - 2.0 ** -10)).astype(np.float16)
    s16 = np.where(bmax == 0, np.float16(0), s16).astype(np.float16)
    sval = s16.astype(np.float32)
    safe = np.where(sval == 0, f32(1.0), sval)
    xs = (wb / safe[:, :, None]).astype(np.float32)
    xs = np.where(sval[:, :, None] == 0, f32(0.0), xs)
    ridx = round_to_fp4(xs)
    rval = (np.where(np.signbit(xs), -1.0, 1.0) * _FP4_MAGS[ridx]).astype(np.float32)
    d_r = np.abs(xs - rval).astype(np.float32)
    cands = sv_candidates(sv_mag, SCALE_E3M3_META2)
    errs32 = np.empty((len(cands), R, nb), dtype=np.float32)
    errs64 = np.empty((len(cands), R, nb), dtype=np.float64)
    use_sv = np.empty((len(cands), R, nb, block), dtype=bool)
    for ci, v in enumerate(cands):
        take = np.abs(xs - f32(v)).astype(np.float32) < d_r
        q = np.where(take, f32(v), rval).astype(np.float32)
        diff = (q - xs).astype(np.float32)
        sq = (diff * diff).astype(np.float32)
        acc = np.zeros((R, nb), dtype=np.float32)
        for j in range(block):
            acc = (acc + sq[:, :, j]).astype(np.float32)
        errs32[ci] = acc
        d64 = q.astype(np.float64) - xs.astype(np.float64)
        errs64[ci] = np.sum(d64 * d64, axis=2)
        use_sv[ci] = take
    meta = np.argmin(errs32, axis=0).astype(np.uint16)
    take = np.take_along_axis(use_sv, meta[None, :, :, None].astype(np.int64), axis=0)[0]
    other_zero = remap_code ^ 0x8
    std = (ridx | (np.signbit(xs).astype(np.uint8) << 3)).astype(np.uint8)
    std = np.where(ridx == 0, other_zero, std).astype(np.uint8)
    code = np.where(take, np.uint8(remap_code), std).astype(np.uint8)
    code = np.where((sval == 0)[:, :, None], np.uint8(other_zero), code).reshape(R, C)
    packed = (code[:, 0::2] | (code[:, 1::2] << 4)).astype(np.uint8)
    # metadata order +m0, +m1, -m0, -m1: sign = meta >> 1 -> bit 15, select = meta & 1 -> bit 14
    sbits = s16.view(np.uint16) | ((meta >> 1) << 15) | ((meta & 1) << 14)
    sbits = np.where(sval == 0, 0, sbits).astype(np.uint16)
    if return_debug:
        d0 = rval.astype(np.float64) - xs.astype(np.float64)
        return packed, sbits, dict(xs=xs, errs64=errs64, err_fp4=np.sum(d0 * d0, axis=2), meta=meta,
                                   near_tie=_near_ties(errs64))
    return packed, sbits


def dequant_fp16_block(codes, scales16, sv_mag=(5.0, 8.0), remap_code: int = 0x8, block: int = 128):
    """Dequantized weights of the FP16-scale variant, FP64: fl16 scale (bits 13:0 of the stored
    word, i.e. sign and top exponent bit cleared) x element value, the special value given
    by bits 15 (sign) and 14 (magnitude select)."""
    scales16 = np.asarray(scales16, dtype=np.uint16)
    s = (scales16 & np.uint16(0x3FFF)).view(np.float16).astype(np.float64)
    sign = np.where((scales16 >> 15) & 1, -1.0, 1.0)
    mag = np.where((scales16 >> 14) & 1, float(sv_mag[1]), float(sv_mag[0]))
    sv = np.repeat(sign * mag, block, axis=1)
    c = unpack_codes(codes)
    vals = np.array([fp4_value(k) for k in range(16)], dtype=np.float64)[c]
    other_zero = remap_code ^ 0x8
    q = np.where(c == remap_code, sv, np.where(c == other_zero, 0.0, vals))
    return q * np.repeat(s, block, axis=1)
