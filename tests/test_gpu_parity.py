"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on identical seeded inputs.

Bars: dequantized weights and quantized activation codes bit-exact; matmul outputs within
1e-3 relative Frobenius error, both sides rounded to bf16 (accumulating 16-bit products in
FP32 instead of FP64 moves a result across a bf16 rounding boundary only rarely; one such
flip costs 2^-8 relative on one element).
"""
import numpy as np
import pytest
import torch

from oracle import razer_oracle as ro
from paper_2501_04052_b200 import inputs

from _util import (elementwise_report, oracle_quantized_weights, oracle_reference, rel_fro_bits, rows_with_edge_tiles,
                   sample_rows, to_dev)

pytestmark = pytest.mark.gpu
TOL = 1e-3


@pytest.fixture(scope="module")
def b():
    from paper_2501_04052_b200 import binding
    return binding


def _pack(b, codes, scales, d32, sv_mag=(5.0, 8.0), remap_code=0x8):
    N, K = codes.shape[0], codes.shape[1] * 2
    desc = b.make_desc(N, K, d32, sv_mag=sv_mag, remap_code=remap_code)
    packed = b.razer_pack_layout(desc, to_dev(codes), to_dev(scales))
    return desc, packed


# ------------------------------------------------------------------ dequant (bit-exact)

@pytest.mark.parametrize("N,K,seed", [(1024, 1024, 0), (200, 80, 3), (1, 16, 4), (129, 4160, 5)])
def test_dequant_bit_exact_oracle_quantized(b, N, K, seed):
    w, codes, scales, d32 = oracle_quantized_weights(N, K, seed)
    desc, packed = _pack(b, codes, scales, d32)
    d1 = b.razer_dequant(desc, packed, fp32=False).cpu()
    d2 = b.razer_dequant(desc, packed, fp32=True).cpu().numpy()
    want1 = ro.dequant_d1(codes, scales)
    want2 = ro.dequant_d2(codes, scales, np.float32(d32))
    assert np.array_equal(inputs.bf16_to_bits(d1), ro.f64_to_bf16_bits(want1.astype(np.float64)))
    assert np.array_equal(d2.view(np.uint32), want2.view(np.uint32))


@pytest.mark.parametrize("remap_code", [0x8, 0x0])
@pytest.mark.parametrize("sv_mag", [(5.0, 8.0), (5.0, 7.0), (5.0, 9.0), (2.5, 12.0)])
def test_dequant_bit_exact_random_codes(b, remap_code, sv_mag):
    """Uniform random codes and metadata exercise every special value, both zero codes,
    subnormal scales and zero blocks."""
    N, K = 300, 1104
    codes, scales = inputs.random_codes(N, K, seed=11, scale_lo=0, scale_hi=64, zero_block_frac=0.05)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.0123, sv_mag=sv_mag, remap_code=remap_code)
    d1 = b.razer_dequant(desc, packed, fp32=False).cpu()
    d2 = b.razer_dequant(desc, packed, fp32=True).cpu().numpy()
    want1 = ro.dequant_d1(codes, scales, sv_mag=sv_mag, remap_code=remap_code)
    want2 = ro.dequant_d2(codes, scales, np.float32(0.0123), sv_mag=sv_mag, remap_code=remap_code)
    assert np.array_equal(inputs.bf16_to_bits(d1), ro.f64_to_bf16_bits(want1.astype(np.float64)))
    assert np.array_equal(d2.view(np.uint32), want2.view(np.uint32))


# ------------------------------------------------------------------ GEMV / skinny GEMM

def _check_matmul(b, fn, desc, packed, codes, scales, d32, x, rows=None, **kw):
    """Two calls on one workspace must agree bit for bit; the result must meet the relative Frobenius bar and,
    element by element, lie within half a bf16 unit of the exact value plus the FP32 accumulation allowance."""
    op = b.OP_GEMV if fn is b.razer_gemv else b.OP_GEMM
    ws = b.alloc_workspace(desc, x.shape[0], op, "cuda")
    y = fn(desc, packed, x.cuda(), workspace=ws)
    b.razer_workspace_status(ws)            # synchronizes; raises if a device wait gave up
    y2 = fn(desc, packed, x.cuda(), workspace=ws)   # the workspace is left ready for the next call
    b.razer_workspace_status(ws)
    assert torch.equal(y, y2), "second call with the same workspace differs"
    xb = inputs.bf16_to_bits(x)
    if rows is None:
        ref, y64, mag = oracle_reference(xb, codes, scales, np.float32(d32), **kw)
        got = y
    else:
        ref, y64, mag = oracle_reference(xb, codes[rows], scales[rows], np.float32(d32), **kw)
        got = y[:, torch.from_numpy(rows).cuda()]
    err = rel_fro_bits(got, ref)
    assert err <= TOL, f"relative Frobenius error {err:.3e}"
    bad, differ, total = elementwise_report(got, ref, y64, mag)
    print(f"[parity] {tuple(x.shape)} x {tuple(codes.shape)}: rel fro {err:.2e}, {differ} of {total} outputs differ from "
          f"the oracle's bf16, {bad} outside the element-wise bound")
    assert bad == 0, f"{bad} of {total} outputs outside 2^-8 |y| + 2^-20 sum|x w|"
    return err


def test_gemv_config1_student_t(b):
    """Workload config 1: N=K=1024, Student-t x 0.02 weights from seed 0, M=1."""
    w, codes, scales, d32 = oracle_quantized_weights(1024, 1024, 0, outliers=0.0)
    desc, packed = _pack(b, codes, scales, d32)
    x = inputs.activations(1, 1024, 0)
    _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, d32, x)


@pytest.mark.parametrize("N,K", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_gemv_config2_llama7b_shapes(b, N, K):
    w, codes, scales, d32 = oracle_quantized_weights(N, K, 1)
    desc, packed = _pack(b, codes, scales, d32)
    x = inputs.activations(1, K, 1)
    _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, d32, x)


@pytest.mark.parametrize("M", [1, 2, 3, 4, 7, 16, 33, 64])
def test_gemv_ragged_shapes_random_codes(b, M):
    N, K = 333, 2064                      # N not a multiple of the row tile, K not of the k chunk
    codes, scales = inputs.random_codes(N, K, seed=20 + M, zero_block_frac=0.02)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.004)
    x = inputs.activations(M, K, 20 + M)
    _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, 0.004, x)


@pytest.mark.parametrize("sv_mag,remap_code", [((5.0, 7.0), 0x8), ((5.0, 9.0), 0x0), ((2.5, 12.0), 0x8)])
def test_gemv_other_special_values(b, sv_mag, remap_code):
    N, K = 256, 1024
    codes, scales = inputs.random_codes(N, K, seed=31)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.01, sv_mag=sv_mag, remap_code=remap_code)
    x = inputs.activations(4, K, 31)
    _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, 0.01, x, sv_mag=sv_mag, remap_code=remap_code)


@pytest.mark.parametrize("M,N,K", [(4, 8192, 8192), (16, 8192, 8192), (64, 8192, 8192),
                                   (4, 28672, 8192), (16, 28672, 8192), (4, 8192, 28672), (16, 8192, 28672),
                                   (64, 8192, 28672)])
def test_skinny_config3_full_size_sampled_rows(b, M, N, K):
    """Workload config 3 (skinny GEMM) at full size: random RaZeR codes, a sample of output columns checked
    one by one against the oracle."""
    codes, scales = inputs.random_codes(N, K, seed=40)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.002)
    x = inputs.activations(M, K, 40 + M)
    rows = rows_with_edge_tiles(N, 192, 41)
    _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, 0.002, x, rows=rows)


def test_skinny_config3_full_size_every_output(b):
    """M = 64 against 28672 x 8192: every one of the 1.8 M outputs of the full-size launch is compared with the
    oracle (computed in chunks of weight rows), so every CTA stripe and tile boundary is covered."""
    M, N, K = 64, 28672, 8192
    codes, scales = inputs.random_codes(N, K, seed=42)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.002)
    x = inputs.activations(M, K, 43)
    _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, 0.002, x)


def test_skinny_config3_oracle_quantized(b):
    w, codes, scales, d32 = oracle_quantized_weights(2048, 8192, 2)
    desc, packed = _pack(b, codes, scales, d32)
    for M in (4, 16, 64):
        x = inputs.activations(M, 8192, 50 + M)
        _check_matmul(b, b.razer_gemv, desc, packed, codes, scales, d32, x)


# ------------------------------------------------------------------ prefill GEMM

@pytest.mark.parametrize("M,N,K", [(256, 512, 1024), (130, 200, 464), (2048, 1024, 4096), (100, 300, 1040),
                                   (128, 640, 2048), (65, 129, 4160)])
def test_gemm_oracle_quantized(b, M, N, K):
    w, codes, scales, d32 = oracle_quantized_weights(N, K, 3, outliers=0.0)
    desc, packed = _pack(b, codes, scales, d32)
    x = inputs.activations(M, K, 60, outlier_channel_frac=0.01)
    _check_matmul(b, b.razer_gemm, desc, packed, codes, scales, d32, x)


@pytest.mark.parametrize("N,K", [(14336, 4096), (4096, 14336)])
def test_gemm_config4_full_size_sampled_rows(b, N, K):
    codes, scales = inputs.random_codes(N, K, seed=70)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.002)
    x = inputs.activations(2048, K, 70, outlier_channel_frac=0.01)
    rows = rows_with_edge_tiles(N, 96, 71)
    _check_matmul(b, b.razer_gemm, desc, packed, codes, scales, 0.002, x, rows=rows)


def test_gemm_config4_full_size_every_output(b):
    """M = 2048 against 4096 x 14336 (the shape whose stripes cut every output tile): all 8.4 M outputs."""
    M, N, K = 2048, 4096, 14336
    codes, scales = inputs.random_codes(N, K, seed=72)
    codes, scales = codes.numpy(), scales.numpy()
    desc, packed = _pack(b, codes, scales, 0.002)
    x = inputs.activations(M, K, 73, outlier_channel_frac=0.01)
    _check_matmul(b, b.razer_gemm, desc, packed, codes, scales, 0.002, x)


# ------------------------------------------------------------------ activation quantization / W4A4

@pytest.mark.parametrize("M,K,seed", [(256, 8192, 80), (7, 48, 81), (33, 1040, 82)])
def test_quant_act_bit_exact(b, M, K, seed):
    x = inputs.activations(M, K, seed, outlier_channel_frac=0.01)
    codes, scales, ts = b.razer_quant_act(x.cuda())
    torch.cuda.synchronize()
    want_c, want_s, want_d, dbg = ro.quantize_act(inputs.bf16_to_bits(x), return_debug=True)
    assert np.float32(ts.item()) == want_d
    got_s, got_c = scales.cpu().numpy(), codes.cpu().numpy()
    assert np.array_equal(got_s & 0x7F, want_s & 0x7F)
    # metadata and codes must agree except where the two candidates' errors tie within rounding
    blk_ok = (got_s == want_s) & np.all((got_c == want_c).reshape(M, K // 16, 8), axis=2)
    assert np.all(blk_ok | dbg["near_tie"])
    assert blk_ok.mean() > 0.999
    # the decode kernel inverts the GPU's own codes exactly like the oracle's decoder
    d1 = b.razer_decode_act(codes, scales).cpu()
    want1 = ro.dequant_d1(got_c, got_s, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0,))
    assert np.array_equal(inputs.bf16_to_bits(d1), ro.f64_to_bf16_bits(want1.astype(np.float64)))


def test_quant_act_given_scale_and_zero_input(b):
    x = inputs.activations(8, 256, 83)
    given = torch.tensor([0.05], dtype=torch.float32)
    codes, scales, ts = b.razer_quant_act(x.cuda(), tensor_scale=given.cuda())
    want_c, want_s, want_d = ro.quantize_act(inputs.bf16_to_bits(x), tensor_scale=np.float32(0.05))
    assert ts.item() == np.float32(0.05)
    assert np.array_equal(scales.cpu().numpy(), want_s) and np.array_equal(codes.cpu().numpy(), want_c)
    z = torch.zeros((4, 64), dtype=torch.bfloat16)
    codes, scales, ts = b.razer_quant_act(z.cuda())
    assert ts.item() == 1.0 and not codes.any() and not scales.any()


@pytest.mark.parametrize("N,K,seed,sv_mag,remap_code", [(1024, 1024, 0, (5.0, 8.0), 0x8), (200, 80, 3, (5.0, 8.0), 0x8),
                                                         (129, 4160, 5, (5.0, 9.0), 0x0), (300, 528, 6, (2.5, 12.0), 0x8)])
def test_quant_weight_bit_exact(b, N, K, seed, sv_mag, remap_code):
    """GPU weight quantizer against the oracle's (Sec. 4.2: E3M3 block scale, four special values): tensor scale,
    scale codes, metadata and element codes, bit for bit except where two candidates' errors tie within rounding."""
    w = inputs.student_t_weights(N, K, seed, outlier_frac=0.001)
    codes, scales, ts = b.razer_quant_weight(w.cuda(), sv_mag=sv_mag, remap_code=remap_code)
    torch.cuda.synchronize()
    want_c, want_s, want_d, dbg = ro.quantize_weight(w.numpy(), sv_mag=sv_mag, remap_code=remap_code, return_debug=True)
    assert np.float32(ts.item()) == want_d
    got_s, got_c = scales.cpu().numpy(), codes.cpu().numpy()
    assert np.array_equal(got_s & 0x3F, want_s & 0x3F)
    blk_ok = (got_s == want_s) & np.all((got_c == want_c).reshape(N, K // 16, 8), axis=2)
    assert np.all(blk_ok | dbg["near_tie"])
    assert blk_ok.mean() > 0.999
    # the GPU's codes go through the pack and dequant kernels like any others
    desc, packed = _pack(b, got_c, got_s, float(ts.item()), sv_mag=sv_mag, remap_code=remap_code)
    d2 = b.razer_dequant(desc, packed, fp32=True).cpu().numpy()
    want2 = ro.dequant_d2(got_c, got_s, np.float32(ts.item()), sv_mag=sv_mag, remap_code=remap_code)
    assert np.array_equal(d2.view(np.uint32), want2.view(np.uint32))
    # and the quantization error is the format's: a few percent of the tensor's norm
    assert np.linalg.norm(d2 - w.numpy()) / np.linalg.norm(w.numpy()) < 0.12


@pytest.mark.parametrize("block", [32, 64, 128])
def test_larger_blocks_quantize_pack_and_multiply(b, block):
    """Block sizes 32 / 64 / 128 (Sec. 5's block-size study, Sec. 4.3's deployment size): the GPU weight quantizer
    against the oracle's bit for bit (near-ties aside), the packed form's dequantization bit-exact, the decode
    GEMV and the tensor-core GEMM within the matmul bars."""
    N, K = 260, 2048
    w = inputs.student_t_weights(N, K, 160 + block, outlier_frac=0.001)
    codes, scales, ts = b.razer_quant_weight(w.cuda(), block=block)
    torch.cuda.synchronize()
    want_c, want_s, want_d, dbg = ro.quantize_weight(w.numpy(), block=block, return_debug=True)
    assert np.float32(ts.item()) == want_d and tuple(scales.shape) == (N, K // block)
    got_s, got_c = scales.cpu().numpy(), codes.cpu().numpy()
    assert np.array_equal(got_s & 0x3F, want_s & 0x3F)
    blk_ok = (got_s == want_s) & np.all((got_c == want_c).reshape(N, K // block, block // 2), axis=2)
    assert np.all(blk_ok | dbg["near_tie"]) and blk_ok.mean() > 0.999
    desc = b.make_desc(N, K, float(ts.item()), block=block)
    packed = b.razer_pack_layout(desc, codes, scales)
    d2 = b.razer_dequant(desc, packed, fp32=True).cpu().numpy()
    want2 = ro.dequant_d2(got_c, got_s, np.float32(ts.item()), block=block)
    assert np.array_equal(d2.view(np.uint32), want2.view(np.uint32))
    for M, fn in ((1, b.razer_gemv), (40, b.razer_gemv), (130, b.razer_gemm)):
        x = inputs.activations(M, K, 170 + M)
        _check_matmul(b, fn, desc, packed, got_c, got_s, float(ts.item()), x, block=block)


@pytest.mark.parametrize("N,K,seed,sv_mag,block", [(512, 1024, 21, (5.0, 8.0), 16), (200, 2048, 22, (7.0, 10.0), 32),
                                                    (130, 528, 23, (2.5, 5.0), 16)])
def test_quant_weight_scale_aware_bit_exact(b, N, K, seed, sv_mag, block):
    """Scale-aware special-value selection (Eq. 6-7 with the scale of Eq. 2 chosen together with v) on the GPU
    against the oracle's: same scale codes and metadata, same element codes, near-ties aside; the result decodes
    through the unchanged kernels and is no worse than the plain selection's."""
    w = inputs.student_t_weights(N, K, seed, outlier_frac=0.001)
    codes, scales, ts = b.razer_quant_weight(w.cuda(), sv_mag=sv_mag, block=block, scale_aware=True)
    torch.cuda.synchronize()
    want_c, want_s, want_d, dbg = ro.quantize_scale_aware(w.numpy(), sv_mag=sv_mag, block=block, return_debug=True)
    assert np.float32(ts.item()) == want_d
    got_s, got_c = scales.cpu().numpy(), codes.cpu().numpy()
    blk_ok = (got_s == want_s) & np.all((got_c == want_c).reshape(N, K // block, block // 2), axis=2)
    assert np.all(blk_ok | dbg["near_tie"]) and blk_ok.mean() > 0.999
    desc = b.make_desc(N, K, float(ts.item()), sv_mag=sv_mag, block=block)
    packed = b.razer_pack_layout(desc, codes, scales)
    d2 = b.razer_dequant(desc, packed, fp32=True).cpu().numpy()
    want2 = ro.dequant_d2(got_c, got_s, np.float32(ts.item()), sv_mag=sv_mag, block=block)
    assert np.array_equal(d2.view(np.uint32), want2.view(np.uint32))
    c0, s0, t0 = b.razer_quant_weight(w.cuda(), sv_mag=sv_mag, block=block)
    plain = ro.dequant_d2(c0.cpu().numpy(), s0.cpu().numpy(), np.float32(t0.item()), sv_mag=sv_mag, block=block)
    e_aware, e_plain = np.linalg.norm(d2 - w.numpy()), np.linalg.norm(plain - w.numpy())
    if max(sv_mag) > 6.0:
        assert e_aware < e_plain
    else:
        assert np.array_equal(got_c, c0.cpu().numpy()) and np.array_equal(got_s, s0.cpu().numpy())
    x = inputs.activations(3, K, seed + 100)
    _check_matmul(b, b.razer_gemv, desc, packed, got_c, got_s, float(ts.item()), x, sv_mag=sv_mag, block=block)


def test_quant_weight_given_scale_and_zero_input(b):
    w = inputs.student_t_weights(16, 256, 7)
    given = torch.tensor([0.01], dtype=torch.float32)
    codes, scales, ts = b.razer_quant_weight(w.cuda(), tensor_scale=given.cuda())
    want_c, want_s, want_d = ro.quantize_weight(w.numpy(), tensor_scale=np.float32(0.01))
    assert ts.item() == np.float32(0.01)
    assert np.array_equal(scales.cpu().numpy(), want_s) and np.array_equal(codes.cpu().numpy(), want_c)
    z = torch.zeros((4, 64), dtype=torch.float32)
    codes, scales, ts = b.razer_quant_weight(z.cuda())
    assert ts.item() == 1.0 and not codes.any() and not scales.any()
    codes, scales, ts = b.razer_quant_weight(z.cuda(), remap_code=0x0)      # the true zero is then code 0x8
    assert ts.item() == 1.0 and bool((codes == 0x88).all()) and not scales.any()
    with pytest.raises(b.RazerError) as e:
        b.razer_quant_weight(w.cuda(), sv_mag=(5.0, 6.0))                   # 6 is an FP4 value, not an allowed special value
    assert e.value.code == b.ERR_UNSUPPORTED


@pytest.mark.parametrize("M,N,K", [(256, 1024, 8192), (17, 200, 464), (8, 300, 2048), (13, 520, 1040)])
def test_w4a4_oracle_quantized(b, M, N, K):
    """Workload config 5, W4A4 (rows of N sampled down to keep the oracle quantizer quick)."""
    w, wc, ws, wd = oracle_quantized_weights(N, K, 4)
    desc, packed = _pack(b, wc, ws, wd)
    x = inputs.activations(M, K, 90, outlier_channel_frac=0.01)
    ac, as_, ats = b.razer_quant_act(x.cuda())
    y = b.razer_gemm_w4a4(desc, packed, ac, as_, ats)
    torch.cuda.synchronize()
    ref = ro.matmul_w4a4(ac.cpu().numpy(), as_.cpu().numpy(), np.float32(ats.item()), wc, ws, np.float32(wd))
    err = rel_fro_bits(y, ref)
    assert err <= TOL, f"relative Frobenius error {err:.3e}"


def _w4a4_native_check(b, desc, packed, wc, ws, wd, ac, as_, ats, rows=None, **kw):
    """Two-pass block-scaled FP4 path against the oracle's W4A4 matmul: relative Frobenius bar and the
    element-wise bound of the other matmul kernels (FP32 accumulation of exact products)."""
    M = ac.shape[0]
    wsb = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
    y = b.razer_gemm_w4a4(desc, packed, ac, as_, ats, workspace=wsb, use_native_fp4=True)
    b.razer_workspace_status(wsb)
    y2 = b.razer_gemm_w4a4(desc, packed, ac, as_, ats, workspace=wsb, use_native_fp4=True)
    b.razer_workspace_status(wsb)
    assert torch.equal(y, y2), "second call with the same workspace differs"
    acn, asn = ac.cpu().numpy(), as_.cpu().numpy()
    if rows is not None:
        wc, ws, y = wc[rows], ws[rows], y[:, torch.from_numpy(rows).cuda()]
    da = ro.dequant_d1(acn, asn, scale_fmt=ro.SCALE_E4M3_META1, sv_mag=(5.0, 5.0)).astype(np.float64)
    dw = ro.dequant_d1(wc, ws, **kw).astype(np.float64)
    scale = float(np.float32(wd)) * float(np.float32(ats.item()))
    y64 = scale * (da @ dw.T)
    mag = abs(scale) * (np.abs(da) @ np.abs(dw).T)
    ref = ro.f64_to_bf16_bits(y64)
    if kw.get("remap_code", 0x8) == 0x8:            # (the oracle's W4A4 matmul takes one remapped code for both operands)
        assert np.array_equal(ref, ro.matmul_w4a4(acn, asn, np.float32(ats.item()), wc, ws, np.float32(wd),
                                                  sv_mag_w=kw.get("sv_mag", (5.0, 8.0))))
    err = rel_fro_bits(y, ref)
    bad, differ, total = elementwise_report(y, ref, y64, mag)
    print(f"[parity] native FP4 {tuple(ac.shape)} x {tuple(wc.shape)}: rel fro {err:.2e}, {differ} of {total} differ, {bad} out of bound")
    assert err <= TOL and bad == 0


@pytest.mark.parametrize("M,N,K,sv_mag,remap_code", [(256, 512, 8192, (5.0, 8.0), 0x8), (17, 200, 464, (5.0, 8.0), 0x8),
                                                    (130, 300, 2048, (2.5, 12.0), 0x0), (13, 520, 1040, (7.0, 10.0), 0x8),
                                                    (300, 260, 272, (5.0, 8.0), 0x8)])
def test_w4a4_native_fp4_two_pass(b, M, N, K, sv_mag, remap_code):
    """App. D.3: RaZeR weights as B_main + B_comp on the block-scaled FP4 tensor-core path, activations in plain
    NVFP4 (quantized on the GPU with no special value, checked against the oracle's Eq. 1-3)."""
    w = inputs.student_t_weights(N, K, 300 + M, outlier_frac=0.001).numpy()
    wc, ws, wd = ro.quantize_weight(w, sv_mag=sv_mag, remap_code=remap_code)
    desc = b.make_desc(N, K, float(wd), sv_mag=sv_mag, remap_code=remap_code)
    packed = b.razer_pack_layout(desc, torch.from_numpy(wc).cuda(), torch.from_numpy(ws).cuda())
    x = inputs.activations(M, K, 301, outlier_channel_frac=0.01)
    ac, as_, ats = b.razer_quant_act(x.cuda(), sv_mag=0.0)
    torch.cuda.synchronize()
    want_c, want_s, want_d = ro.quantize_act(inputs.bf16_to_bits(x), sv_mag=None)
    assert np.float32(ats.item()) == want_d
    assert np.array_equal(ac.cpu().numpy(), want_c) and np.array_equal(as_.cpu().numpy(), want_s)
    _w4a4_native_check(b, desc, packed, wc, ws, wd, ac, as_, ats, sv_mag=sv_mag, remap_code=remap_code)


@pytest.mark.parametrize("nt,M", [(128, 300), (256, 40), (256, 300)])
def test_w4a4_native_fp4_forced_token_tile(b, monkeypatch, nt, M):
    """Both token-tile widths of the FP4 kernel at token counts the host would give to the other one."""
    monkeypatch.setenv("RAZER_FP4_NT", str(nt))
    N, K = 390, 2320                                                   # ragged row tile, 9.06 stages
    w = inputs.student_t_weights(N, K, 310 + nt, outlier_frac=0.001).numpy()
    wc, ws, wd = ro.quantize_weight(w)
    desc = b.make_desc(N, K, float(wd))
    packed = b.razer_pack_layout(desc, torch.from_numpy(wc).cuda(), torch.from_numpy(ws).cuda())
    x = inputs.activations(M, K, 311, outlier_channel_frac=0.01)
    ac, as_, ats = b.razer_quant_act(x.cuda(), sv_mag=0.0)
    _w4a4_native_check(b, desc, packed, wc, ws, wd, ac, as_, ats)


@pytest.mark.parametrize("M,N,K", [(256, 512, 8192), (17, 200, 464), (300, 260, 1040), (130, 390, 2320)])
def test_w4a4_fp4_prepared_operand_matches_the_interchange_route(b, M, N, K):
    """razer_quant_act_fp4 + razer_gemm_w4a4_fp4 (the quantizer writes the tensor core's operand layout itself)
    against razer_quant_act(sv_mag = 0) + razer_gemm_w4a4(use_native_fp4): same tensor scale, bit-identical outputs,
    and the outputs within the matmul bars of the oracle's W4A4 result.  The operand buffer starts as garbage: the
    quantizer has to write its padding too."""
    w = inputs.student_t_weights(N, K, 320 + M, outlier_frac=0.001).numpy()
    wc, ws, wd = ro.quantize_weight(w)
    desc = b.make_desc(N, K, float(wd))
    packed = b.razer_pack_layout(desc, torch.from_numpy(wc).cuda(), torch.from_numpy(ws).cuda())
    x = inputs.activations(M, K, 321, outlier_channel_frac=0.01).cuda()
    ac, as_, ats = b.razer_quant_act(x, sv_mag=0.0)
    wsb = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
    y_ref = b.razer_gemm_w4a4(desc, packed, ac, as_, ats, workspace=wsb, use_native_fp4=True).clone()
    b.razer_workspace_status(wsb)
    buf = torch.full((b.razer_fp4_act_bytes(M, K),), 0xA5, dtype=torch.uint8, device="cuda")
    act, ats2 = b.razer_quant_act_fp4(x, act_fp4=buf)
    assert ats2.item() == ats.item()
    wsb2 = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
    y = b.razer_gemm_w4a4_fp4(desc, packed, act, ats2, M, workspace=wsb2)
    b.razer_workspace_status(wsb2)
    assert torch.equal(y, y_ref)
    given = torch.tensor([0.01], dtype=torch.float32, device="cuda")          # a given tensor scale: no grid rendezvous
    act3, ats3 = b.razer_quant_act_fp4(x, tensor_scale=given)
    ac3, as3, _ = b.razer_quant_act(x, sv_mag=0.0, tensor_scale=given)
    y3 = b.razer_gemm_w4a4_fp4(desc, packed, act3, ats3, M, workspace=wsb2)
    y3_ref = b.razer_gemm_w4a4(desc, packed, ac3, as3, ats3, workspace=wsb, use_native_fp4=True)
    assert torch.equal(y3, y3_ref)
    _w4a4_native_check(b, desc, packed, wc, ws, wd, ac, as_, ats)


def test_w4a4_native_fp4_decodes_bit_exactly(b):
    """One-hot NVFP4 activations (code 1.0, block scale 1.0) through the two-pass path: y[m, n] is the tensor
    scale times one decoded weight, exact whatever the accumulation order, so main + comp is checked bit for bit."""
    N, K, TS = 300, 1104, 0.25
    for remap_code, sv_mag, seed in [(0x8, (5.0, 8.0), 211), (0x0, (2.5, 12.0), 212)]:
        codes, scales = inputs.random_codes(N, K, seed=seed, scale_lo=0, scale_hi=64, zero_block_frac=0.05)
        codes, scales = codes.numpy(), scales.numpy()
        want = ro.dequant_d1(codes, scales, sv_mag=sv_mag, remap_code=remap_code).astype(np.float64) * TS
        want_bits = ro.f64_to_bf16_bits(want)
        desc = b.make_desc(N, K, TS, sv_mag=sv_mag, remap_code=remap_code)
        packed = b.razer_pack_layout(desc, torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda())
        M = 160                                                        # two token tiles, the second ragged
        wsb = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
        one = torch.ones(1, dtype=torch.float32, device="cuda")
        got = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        as_ = torch.full((M, K // 16), 0x38, dtype=torch.uint8, device="cuda")      # E4M3 1.0 everywhere
        ar = torch.arange(M, device="cuda")
        for k0 in range(0, K, M):
            m = min(M, K - k0)
            ac = torch.zeros((M, K // 2), dtype=torch.uint8, device="cuda")
            kk = k0 + ar[:m]
            ac[ar[:m], kk // 2] = torch.where(kk % 2 == 0, 0x02, 0x20).to(torch.uint8)   # FP4 code of 1.0
            y = b.razer_gemm_w4a4(desc, packed, ac, as_, one, workspace=wsb, use_native_fp4=True)
            got[:, k0:k0 + m] = y[:m].t()
        b.razer_workspace_status(wsb)
        got_bits = inputs.bf16_to_bits(got.cpu())
        g = np.where((got_bits & 0x7FFF) == 0, 0, got_bits)
        wv = np.where((want_bits & 0x7FFF) == 0, 0, want_bits)
        bad = np.argwhere(g != wv)
        assert bad.size == 0, (remap_code, sv_mag, len(bad), bad[:5].tolist())


def test_w4a4_native_fp4_config5_full_size_sampled_rows(b):
    M, N, K = 256, 8192, 8192
    wc, ws = inputs.random_codes(N, K, seed=97)
    wc, ws = wc.numpy(), ws.numpy()
    desc, packed = _pack(b, wc, ws, 0.002)
    x = inputs.activations(M, K, 97, outlier_channel_frac=0.01)
    ac, as_, ats = b.razer_quant_act(x.cuda(), sv_mag=0.0)
    _w4a4_native_check(b, desc, packed, wc, ws, 0.002, ac, as_, ats, rows=sample_rows(N, 128, 98))


def test_w4a4_config5_full_size_sampled_rows(b):
    M, N, K = 256, 8192, 8192
    wc, ws = inputs.random_codes(N, K, seed=95)
    wc, ws = wc.numpy(), ws.numpy()
    desc, packed = _pack(b, wc, ws, 0.002)
    x = inputs.activations(M, K, 95, outlier_channel_frac=0.01)
    ac, as_, ats = b.razer_quant_act(x.cuda())
    y = b.razer_gemm_w4a4(desc, packed, ac, as_, ats)
    torch.cuda.synchronize()
    rows = sample_rows(N, 128, 96)
    ref = ro.matmul_w4a4(ac.cpu().numpy(), as_.cpu().numpy(), np.float32(ats.item()), wc[rows], ws[rows],
                         np.float32(0.002))
    err = rel_fro_bits(y[:, torch.from_numpy(rows).cuda()], ref)
    assert err <= TOL, f"relative Frobenius error {err:.3e}"


@pytest.mark.parametrize("M,N,K", [(2048, 14336, 4096), (64, 11008, 4096), (24, 4096, 11008), (128, 11008, 4096)])
def test_repeated_launches_are_bit_identical(b, M, N, K):
    """The same call repeated many times must return the same bits.  The tcgen05 kernel once let a dequant
    group mistake a weight load that was still in flight for the next load of the same stage (the loads of a
    ring complete in any order, and a group does not watch the stages of the items it skips): about one launch
    in a thousand of the first shape then produced a wrong partial tile at the start of a CTA's stripe."""
    codes, scales = inputs.random_codes(N, K, seed=140)
    desc, packed = _pack(b, codes.numpy(), scales.numpy(), 0.002)
    x = inputs.activations(M, K, 141, outlier_channel_frac=0.01).cuda()
    op, fn = (b.OP_GEMV, b.razer_gemv) if M <= 64 else (b.OP_GEMM, b.razer_gemm)
    ws = b.alloc_workspace(desc, M, op, "cuda")
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    fn(desc, packed, x, y, ws)
    first = y.clone()
    differing = 0
    for _ in range(1500):
        fn(desc, packed, x, y, ws)
        differing += int(not torch.equal(y, first))
    b.razer_workspace_status(ws)
    assert differing == 0, f"{differing} of 1500 launches differ from the first"
    rows = sample_rows(N, 64, 142)
    ref = ro.matmul_w4a16(inputs.bf16_to_bits(x.cpu()), codes.numpy()[rows], scales.numpy()[rows], np.float32(0.002))
    assert rel_fro_bits(first[:, torch.from_numpy(rows).cuda()], ref) <= TOL


@pytest.mark.parametrize("M,N,K", [(256, 8192, 8192), (2048, 4096, 4096), (100, 11008, 4096)])
def test_repeated_fp4_launches_are_bit_identical(b, M, N, K):
    """The block-scaled FP4 matmul repeated many times on one workspace must return the same bits: three rings, two
    producer warps, sixteen remap warps and partial tiles combined across CTAs leave room for a rare ordering fault."""
    codes, scales = inputs.random_codes(N, K, seed=150)
    desc, packed = _pack(b, codes.numpy(), scales.numpy(), 0.002)
    x = inputs.activations(M, K, 151, outlier_channel_frac=0.01).cuda()
    act, ats = b.razer_quant_act_fp4(x)
    ws = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    b.razer_gemm_w4a4_fp4(desc, packed, act, ats, M, y=y, workspace=ws)
    first = y.clone()
    differing = 0
    for _ in range(1000):
        b.razer_gemm_w4a4_fp4(desc, packed, act, ats, M, y=y, workspace=ws)
        differing += int(not torch.equal(y, first))
    b.razer_workspace_status(ws)
    assert differing == 0, f"{differing} of 1000 launches differ from the first"


# ------------------------------------------------------------------ host-buffer entry point, errors

@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("M,N,K", [(2, 512, 1024), (40, 300, 528)])
def test_gemv_host_entry_point(b, pinned, M, N, K):
    """Host x in, host y out.  Pinned y takes the kernel's stores directly, pageable y goes through the staging
    buffer; (2, 512, 1024) runs on the register-fragment kernel, (40, 300, 528) on the tcgen05 kernel."""
    codes, scales = inputs.random_codes(N, K, seed=97)
    desc, packed = _pack(b, codes.numpy(), scales.numpy(), 0.01)
    x = inputs.activations(M, K, 97)
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16)
    if pinned:
        x, y = x.pin_memory(), y.pin_memory()
    xs = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    ys = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws = b.alloc_workspace(desc, M, b.OP_GEMV, "cuda")
    for _ in range(2):
        b.razer_gemv_host(desc, packed, x, y, xs, ys, ws)
        y_dev = b.razer_gemv(desc, packed, x.cuda())
        assert torch.equal(y, y_dev.cpu())
        y.fill_(float("nan"))


def test_workspace_too_small_is_an_error(b):
    N, K = 512, 4096
    codes, scales = inputs.random_codes(N, K, seed=98)
    desc, packed = _pack(b, codes.numpy(), scales.numpy(), 0.01)
    need = b.razer_workspace_bytes(desc, 1, b.OP_GEMV)
    if need > 256:
        x = inputs.activations(1, K, 98).cuda()
        tiny = torch.empty(256, dtype=torch.uint8, device="cuda")
        with pytest.raises(b.RazerError) as e:
            b.razer_gemv(desc, packed, x, workspace=tiny)
        assert e.value.code == b.ERR_WORKSPACE


def test_weights_written_just_ahead_of_the_matmul_are_seen(b):
    """Stream-ordering contract of the header: the matmul kernels start reading the packed weights before the kernel
    directly ahead of them is known to have finished (programmatic dependent launch).  What is guaranteed: weights
    written by razer_pack_layout or by a device-to-device copy queued directly ahead of the matmul are the ones read.
    Two different tensors go alternately into ONE packed buffer, each time followed at once by the GEMV."""
    N, K = 4096, 4096
    desc = b.make_desc(N, K, 0.002)
    sets, want = [], []
    x = inputs.activations(1, K, 7).cuda()
    ws = b.alloc_workspace(desc, 1, b.OP_GEMV, "cuda")
    for s in range(2):
        c, sc = inputs.random_codes(N, K, seed=400 + s)
        sets.append((c.cuda(), sc.cuda()))
        p = b.razer_pack_layout(desc, *sets[-1])
        want.append(b.razer_gemv(desc, p, x, workspace=ws).clone())
    assert not torch.equal(want[0], want[1])
    packed = torch.empty_like(p)
    y = torch.empty_like(want[0])
    keep = [b.razer_pack_layout(desc, *sets[s]) for s in range(2)]
    bad = 0
    for i in range(300):
        s = i & 1
        if i % 3 == 0:
            packed.copy_(keep[s])                                       # device-to-device copy
        else:
            b.razer_pack_layout(desc, sets[s][0], sets[s][1], packed)   # the library's own writer
        b.razer_gemv(desc, packed, x, y, ws)
        bad += int(not torch.equal(y, want[s]))
    b.razer_workspace_status(ws)
    assert bad == 0, f"{bad} of 300 launches read stale weights"


# ------------------------------------------------------------------ alternative kernels (chosen by environment)

_ALT_KERNEL_CHECK = r"""
import sys, numpy as np, torch
sys.path.insert(0, sys.argv[1])
from oracle import razer_oracle as ro
from paper_2501_04052_b200 import binding as b, inputs
for (M, N, K, seed) in [(1, 1000, 4160, 1), (5, 333, 2064, 2), (16, 640, 1024, 3), (8, 384, 8192, 4), (2, 6000, 1088, 5),
                        (1, 4096, 4096, 6), (3, 8200, 1024, 7), (2, 11008, 2048, 8), (1, 50, 16, 9), (8, 5000, 144, 10)]:
    codes, scales = inputs.random_codes(N, K, seed=seed, scale_lo=0, scale_hi=64, zero_block_frac=0.02)
    codes, scales = codes.numpy(), scales.numpy()
    desc = b.make_desc(N, K, 0.004, sv_mag=(5.0, 9.0))
    packed = b.razer_pack_layout(desc, torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda())
    x = inputs.activations(M, K, seed)
    ws = b.alloc_workspace(desc, M, b.OP_GEMV, "cuda")
    y = b.razer_gemv(desc, packed, x.cuda(), workspace=ws)
    b.razer_workspace_status(ws)
    ref = ro.matmul_w4a16(inputs.bf16_to_bits(x), codes, scales, np.float32(0.004), sv_mag=(5.0, 9.0))
    err = ro.rel_frobenius(inputs.bf16_to_bits(y.cpu()), ref)
    assert err <= 1e-3, (M, N, K, err)
print("ok")
"""


@pytest.mark.parametrize("kernel,extra_env", [
    ("umma", {}), ("simt", {}), ("stream", {}),
    # the decode kernel's partitions, each forced on every shape: whole units only / units cut along K and combined
    # through the workspace, with one or two 16-row strips per unit
    ("stream", {"RAZER_STREAM_SPLIT": "0", "RAZER_STREAM_TM": "1"}),
    ("stream", {"RAZER_STREAM_SPLIT": "0", "RAZER_STREAM_TM": "2"}),
    ("stream", {"RAZER_STREAM_SPLIT": "1", "RAZER_STREAM_TM": "1"}),
    ("stream", {"RAZER_STREAM_SPLIT": "1", "RAZER_STREAM_TM": "2"}),
])
def test_alternative_kernels_match_the_oracle(kernel, extra_env):
    """RAZER_KERNEL pins the matmul entry points to one kernel (the tcgen05 kernel, the TMA-fed
    register-fragment kernel wherever it can run (M <= 8), or the CUDA-core kernel) instead of the
    per-shape choice; it is read once per process, so the check runs in a child process."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, RAZER_KERNEL=kernel, **extra_env)
    r = subprocess.run([sys.executable, "-c", _ALT_KERNEL_CHECK, root], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout + r.stderr


def test_back_to_back_dependent_launches(b):
    """The matmul kernels start their weight stream while the preceding kernel of the stream still runs
    (programmatic dependent launch) and must read activations, workspace and outputs only after it has
    finished.  A chain y1 = W1 x, y2 = W2 y1, y3 = W1 y2 with shared workspace, launched back to back many
    times, is compared with the same chain computed by the oracle."""
    N = K = 2048
    M = 3
    c1, s1 = inputs.random_codes(N, K, seed=131)
    c2, s2 = inputs.random_codes(N, K, seed=132)
    c1, s1, c2, s2 = c1.numpy(), s1.numpy(), c2.numpy(), s2.numpy()
    d1, p1 = _pack(b, c1, s1, 0.002)
    d2, p2 = _pack(b, c2, s2, 0.002)
    x = inputs.activations(M, K, 133)
    ws = b.alloc_workspace(d1, M, b.OP_GEMV, "cuda")
    xd = x.cuda()
    bufs = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    outs = []
    for rep in range(20):
        b.razer_gemv(d1, p1, xd, bufs[0], ws)
        b.razer_gemv(d2, p2, bufs[0], bufs[1], ws)
        b.razer_gemv(d1, p1, bufs[1], bufs[2], ws)
        outs.append(bufs[2].clone())
    b.razer_workspace_status(ws)
    y1 = ro.matmul_w4a16(inputs.bf16_to_bits(x), c1, s1, np.float32(0.002))
    y2 = ro.matmul_w4a16(y1, c2, s2, np.float32(0.002))
    y3 = ro.matmul_w4a16(y2, c1, s1, np.float32(0.002))
    for o in outs:
        assert torch.equal(o, outs[0]), "a repetition of the chain differs"
    # three chained bf16 roundings: allow a few times the single-product bar
    assert rel_fro_bits(outs[0], y3) <= 5e-3
    assert rel_fro_bits(bufs[0], y1) <= TOL
