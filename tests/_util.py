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
