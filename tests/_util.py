"""Helpers shared by the GPU parity tests: oracle-side references for sampled rows."""
import numpy as np
import torch

from oracle import razer_oracle as ro
from paper_2501_04052_b200 import inputs


def oracle_quantized_weights(N, K, seed, outliers=0.001, sv_mag=(5.0, 8.0), remap_code=0x8):
    w = inputs.student_t_weights(N, K, seed, outlier_frac=outliers).numpy()
    codes, scales, d32 = ro.quantize_weight(w, sv_mag=sv_mag, remap_code=remap_code)
    return w, codes, scales, float(d32)


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def rel_fro_bits(y_gpu: torch.Tensor, y_ref_bits: np.ndarray) -> float:
    return ro.rel_frobenius(inputs.bf16_to_bits(y_gpu.cpu()), y_ref_bits)


def sample_rows(N, n, seed):
    rng = np.random.default_rng(seed)
    rows = np.unique(np.concatenate([rng.integers(0, N, n), [0, N - 1, min(N - 1, 127), min(N - 1, 128)]]))
    return rows


def rows_with_edge_tiles(N, n, seed, tile=128):
    """Random rows plus every row of the first and of the last 128-row tile."""
    rng = np.random.default_rng(seed)
    first = np.arange(0, min(tile, N))
    last = np.arange(max(0, (N - 1) // tile * tile), N)
    return np.unique(np.concatenate([rng.integers(0, N, n), first, last]))


def oracle_reference(x_bits, codes, scales, tensor_scale, chunk_rows=2048, **kw):
    """Oracle outputs for all rows of (codes, scales), computed chunk by chunk over the weight rows to bound
    memory: (bf16 bits [M, n], unrounded FP64 result [M, n], tensor_scale * sum_k |x * D1| [M, n])."""
    x = ro.bf16_bits_to_f64(x_bits)
    ts = float(np.float32(tensor_scale))
    n = codes.shape[0]
    y64 = np.empty((x.shape[0], n), dtype=np.float64)
    mag = np.empty_like(y64)
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        y64[:, r0:r1] = ro.matmul_w4a16(x_bits, codes[r0:r1], scales[r0:r1], tensor_scale, round_output=False, **kw)
        d1 = np.abs(ro.dequant_d1(codes[r0:r1], scales[r0:r1], **kw).astype(np.float64))
        mag[:, r0:r1] = ts * (np.abs(x) @ d1.T)
    return ro.f64_to_bf16_bits(y64), y64, mag


def elementwise_report(y_gpu: torch.Tensor, ref_bits, y64, mag):
    """Per-element check of a bf16 GPU result against the oracle.  Every output must lie within half a bf16
    unit of the exact result (2^-8 relative) plus what FP32 accumulation of the exact products can add
    (2^-20 of the sum of the products' magnitudes).  Returns (violations, elements whose bf16 bits differ from the
    oracle's, total)."""
    got_bits = inputs.bf16_to_bits(y_gpu.cpu())
    got = ro.bf16_bits_to_f64(got_bits)
    bound = 2.0 ** -8 * np.abs(y64) + 2.0 ** -20 * mag
    bad = int(np.count_nonzero(~(np.abs(got - y64) <= bound)))
    differ = int(np.count_nonzero((got_bits != ref_bits) & ~((got == 0) & (ro.bf16_bits_to_f64(ref_bits) == 0))))
    return bad, differ, got_bits.size
