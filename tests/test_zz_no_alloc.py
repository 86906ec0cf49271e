"""razer_gemv_static: the GEMV entry point for callers that may not allocate device memory.

A plug-in inside another framework's memory pool, or a loop that must stay out of the CUDA
allocator, cannot hand razer_gemv a workspace.  razer_gemv_static takes its scratch from an
array inside the library, so these checks call it through the C ABI with caller-owned inputs
and outputs only.  Its results are compared with the CPU oracle (the same bar as every other
matmul test) and with razer_gemv, which may run a different kernel for the same shape.  Two
calls in a row on different inputs show that what one call leaves in the shared array does
not leak into the next.  This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import razer_oracle as ro
from paper_2501_04052_b200 import inputs

pytestmark = pytest.mark.gpu
TOL = 1e-3      # the relative Frobenius bar of the other matmul tests


def _rel_fro(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm().clamp_min(1e-300))


def test_gemv_static_matches_the_oracle_on_two_calls_in_a_row():
    from paper_2501_04052_b200 import binding as b
    N, K = 1000, 4160                         # ragged in both dimensions; several stripes share tiles
    codes, scales = inputs.random_codes(N, K, seed=120, zero_block_frac=0.02)
    desc = b.make_desc(N, K, 0.004)
    packed = b.razer_pack_layout(desc, codes.cuda(), scales.cuda())
    cn, sn = codes.numpy(), scales.numpy()

    def check(M, seed):
        x = inputs.activations(M, K, seed)
        y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        b.razer_gemv_static(desc, packed, x.cuda(), y)
        other = b.razer_gemv(desc, packed, x.cuda())
        torch.cuda.synchronize()
        assert torch.isfinite(y.float()).all()
        ref = ro.matmul_w4a16(inputs.bf16_to_bits(x), cn, sn, np.float32(0.004))
        assert ro.rel_frobenius(inputs.bf16_to_bits(y.cpu()), ref) <= TOL
        assert _rel_fro(y, other) <= TOL      # the entry point with a caller-owned workspace agrees too
        return y

    first = check(1, 120)
    check(16, 121)                            # second call: other inputs, other M, same built-in scratch
    again = check(1, 120)                     # and the first inputs once more: nothing depends on what ran before
    assert torch.equal(first, again)


def test_gemv_static_rejects_what_does_not_fit():
    from paper_2501_04052_b200 import binding as b
    N, K = 256, 256
    codes, scales = inputs.random_codes(N, K, seed=121)
    desc = b.make_desc(N, K, 0.01)
    packed = b.razer_pack_layout(desc, codes.cuda(), scales.cuda())
    x = inputs.activations(17, K, 121).cuda()
    y = torch.empty((17, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.RazerError) as e:
        b.razer_gemv_static(desc, packed, x, y)
    assert e.value.code == b.ERR_INVALID_ARG
    huge = b.make_desc(200_000_000, 16, 0.01)   # scratch need far beyond the built-in array; nothing is launched
    with pytest.raises(b.RazerError) as e:
        b._check(b.lib().razer_gemv_static(__import__("ctypes").byref(huge), packed.data_ptr(), x.data_ptr(), 1,
                                           y.data_ptr(), None))
    assert e.value.code == b.ERR_UNSUPPORTED
    assert "scratch" in str(e.value)
