"""The C-ABI library loads without a GPU, exports every function the header declares, and
rejects bad arguments on the host before any CUDA work."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2501_04052_b200 import build
    build.build()
    from paper_2501_04052_b200 import binding as b
    return b


def _declared():
    src = open(os.path.join(ROOT, "include", "razer.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(razer_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_exported(binding):
    names = _declared()
    assert len(names) >= 12 and "razer_gemv" in names and "razer_pack_layout" in names
    for n in names:
        assert hasattr(binding.lib(), n), f"{n} declared in razer.h but not exported"
    assert sorted(binding.EXPORTS) == names
    assert binding.razer_version() >= 100


def test_desc_struct_matches_header(binding):
    assert ctypes.sizeof(binding.RazerDesc) == 32
    assert binding.RazerDesc.sv_mag.offset == 20 and binding.RazerDesc.tensor_scale.offset == 28


def test_host_side_validation(binding):
    b = binding
    good = b.make_desc(256, 512, 0.01)
    assert b.razer_packed_bytes(good) == 2 * 8 * 4608           # 2 row tiles x 8 k-chunks
    assert b.razer_packed_bytes(b.make_desc(256, 512, 0.01, block=128)) == 2 * 8 * 4608   # one byte per 16 elements whatever the block
    assert b.razer_packed_bytes(b.make_desc(1, 16, 1.0)) == 4608  # padded to one tile-chunk
    for bad, code in [
        (b.make_desc(256, 520, 0.01), b.ERR_INVALID_ARG),                   # K % 16
        (b.make_desc(0, 512, 0.01), b.ERR_INVALID_ARG),
        (b.make_desc(256, 512, 0.01, block=48), b.ERR_UNSUPPORTED),
        (b.make_desc(256, 544, 0.01, block=64), b.ERR_INVALID_ARG),                 # K % block
        (b.make_desc(256, 512, 0.01, sv_mag=(5.0, 8.5)), b.ERR_UNSUPPORTED),  # 8.5 is not exact in bf16 products
        (b.make_desc(256, 512, 0.01, remap_code=3), b.ERR_INVALID_ARG),
        (b.make_desc(256, 512, 0.0), b.ERR_INVALID_ARG),
        (b.make_desc(256, 512, 0.01, scale_fmt=b.SCALE_E4M3_META1), b.ERR_UNSUPPORTED),
    ]:
        with pytest.raises(b.RazerError) as e:
            b.razer_packed_bytes(bad)
        assert e.value.code == code and b.last_error()
    with pytest.raises(b.RazerError) as e:
        b.razer_workspace_bytes(good, 65, b.OP_GEMV)
    assert e.value.code == b.ERR_INVALID_ARG
    assert b.razer_workspace_bytes(good, 1, b.OP_GEMV) % 256 == 0
    # null / misaligned pointers are refused before any launch
    n = ctypes.c_size_t()
    assert b.lib().razer_packed_bytes(None, ctypes.byref(n)) == b.ERR_INVALID_ARG
    assert b.lib().razer_pack_layout(ctypes.byref(good), None, None, None, None) == b.ERR_INVALID_ARG
    assert b.lib().razer_gemv(ctypes.byref(good), 24, 16, 1, 16, None, 0, None) == b.ERR_INVALID_ARG  # packed misaligned
    assert b.lib().razer_quant_act(None, 4, 64, 5.0, None, None, None, None, None, None) == b.ERR_INVALID_ARG
    assert b.lib().razer_quant_act(16, 4, 72, 5.0, None, None, None, None, None, None) == b.ERR_INVALID_ARG
    # the block-scaled FP4 path checks its workspace before it launches anything
    assert b.lib().razer_gemm_w4a4(ctypes.byref(good), 16, 16, 16, 16, 5.0, 4, 16, 256, 1 << 10, 1, None) == b.ERR_WORKSPACE
