"""Bit-exact dequantization THROUGH the matmul kernels (Sec. 3 dequantization; Sec. 4.2 / 4.4 remapped zero).

razer_dequant has a scalar decoder of its own; the matmul kernels decode with packed-bf16 bit tricks and
shared-memory tables.  To check that decoder bit for bit, the activations are rows of the identity: token m
is 1.0 at column k0 + m and 0 elsewhere, the tensor scale is a power of two, so

    y[m, n] = bf16( ts * D1[n, k0 + m] )

with a single non-zero product: exact whatever the accumulation order, and exactly representable.  Sweeping k0
over all of K recovers the whole decoded tensor from the kernel's outputs; it must equal the oracle's
dequant_d1 bit for bit (a zero's sign carries no information and is not compared).

RAZER_KERNEL pins the kernel and is read once per process, so every case runs in a child process.  M picks the
kernel's configuration (token-tile width).
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

_CHILD = r"""
import sys, numpy as np, torch
sys.path.insert(0, sys.argv[1])
from oracle import razer_oracle as ro
from paper_2501_04052_b200 import binding as b, inputs
Ms = [int(v) for v in sys.argv[2].split(",")]
N, K = 300, 1104                               # three row tiles (the last ragged), 17.25 k chunks
TS = 0.25
for remap_code, sv_mag, seed in [(0x8, (5.0, 8.0), 201), (0x0, (2.5, 12.0), 202)]:
    codes, scales = inputs.random_codes(N, K, seed=seed, scale_lo=0, scale_hi=64, zero_block_frac=0.05)
    codes, scales = codes.numpy(), scales.numpy()
    want = ro.dequant_d1(codes, scales, sv_mag=sv_mag, remap_code=remap_code).astype(np.float64) * TS
    want_bits = ro.f64_to_bf16_bits(want)
    assert np.array_equal(ro.bf16_bits_to_f64(want_bits), want)          # exactly representable
    desc = b.make_desc(N, K, TS, sv_mag=sv_mag, remap_code=remap_code)
    packed = b.razer_pack_layout(desc, torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda())
    for M in Ms:
        fn, op = (b.razer_gemv, b.OP_GEMV) if M <= 64 else (b.razer_gemm, b.OP_GEMM)
        ws = b.alloc_workspace(desc, M, op, "cuda")
        got = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        ar = torch.arange(M, device="cuda")
        for k0 in range(0, K, M):
            x = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
            m = min(M, K - k0)
            x[ar[:m], k0 + ar[:m]] = 1.0
            y = fn(desc, packed, x, workspace=ws)
            got[:, k0:k0 + m] = y[:m].t()
        b.razer_workspace_status(ws)
        got_bits = inputs.bf16_to_bits(got.cpu())
        g = np.where((got_bits & 0x7FFF) == 0, 0, got_bits)               # -0 and +0 are the same zero
        w = np.where((want_bits & 0x7FFF) == 0, 0, want_bits)
        bad = np.argwhere(g != w)
        assert bad.size == 0, (M, remap_code, sv_mag, len(bad), bad[:5].tolist())
print("ok")
"""


def _run(kernel, Ms):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ)
    env.pop("RAZER_KERNEL", None)
    if kernel:
        env["RAZER_KERNEL"] = kernel
    r = subprocess.run([sys.executable, "-c", _CHILD, root, ",".join(str(m) for m in Ms)], env=env,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


@pytest.mark.parametrize("kernel,Ms", [
    ("", (1, 8, 16, 64)),                 # the kernels the library picks by itself for these sizes
    ("stream", (1, 3, 8)),                # TMA-fed register-fragment kernel (M <= 8)
    ("umma", (16, 32, 64, 128, 256)),     # tcgen05 kernel: token tiles 16 (group issue), 32, 64, 128, 256
    ("simt", (1, 4)),                     # CUDA-core kernel
])
def test_matmul_kernels_decode_bit_exactly(kernel, Ms):
    _run(kernel, Ms)
