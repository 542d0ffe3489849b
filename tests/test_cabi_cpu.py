"""Host-side checks that need no GPU: the CUDA library builds, loads, exports
every symbol the header declares, validates arguments before touching a
device, and refuses to run without one (there is no fallback)."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2608_14560_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(moe_fp8_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = C.CDLL(path)
    declared = _declared_functions()
    assert len(declared) >= 9
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= set(declared)


def test_strerror_and_null_arguments():
    lib = binding.load_library()
    assert lib.moe_fp8_strerror(0) == b"ok"
    assert b"no fallback" in lib.moe_fp8_strerror(binding.ERR_ARCH)
    assert lib.moe_fp8_create(None, None) == binding.ERR_BAD_ARG
    assert lib.moe_fp8_destroy(None) == binding.ERR_BAD_ARG
    assert lib.moe_fp8_workspace_bytes(None) == 0
    assert lib.moe_fp8_set_workspace(None, None, 0) == binding.ERR_BAD_ARG
    assert lib.moe_fp8_last_launch_count(None) == 0


@pytest.mark.parametrize("field,value,rc", [
    ("hidden", 7000, binding.ERR_UNSUPPORTED_DIMS),
    ("intermediate", 100, binding.ERR_UNSUPPORTED_DIMS),
    ("num_experts", 128, binding.ERR_UNSUPPORTED_DIMS),
    ("top_k", 6, binding.ERR_UNSUPPORTED_DIMS),
    ("num_local_experts", 300, binding.ERR_UNSUPPORTED_DIMS),
    ("num_local_experts", 0, binding.ERR_BAD_ARG),
    ("max_tokens", -1, binding.ERR_BAD_ARG),
    ("hidden_scale_layout", 2, binding.ERR_UNSUPPORTED_DIMS),
])
def test_create_rejects_bad_shapes_before_touching_the_device(field, value, rc):
    lib = binding.load_library()
    cfg = binding.Config(7168, 2048, 256, 32, 8, 4, 8, 64, 0, 1)
    setattr(cfg, field, value)
    h = C.c_void_p()
    assert lib.moe_fp8_create(C.byref(cfg), C.byref(h)) == rc
    assert not h.value


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU behaviour")
def test_no_device_means_loud_failure_not_a_fallback():
    with pytest.raises(binding.MoeFp8Error):
        binding.MoeFp8(device="cpu")


def test_binding_constants_agree_with_the_header():
    import re
    from paper_2608_14560_b200 import binding
    text = open(os.path.join(ROOT, "include", "moe_fp8.h")).read()
    defs = {m.group(1): int(m.group(2).strip("()")) for m in re.finditer(r"#define (MOE_FP8_\w+) (\(?-?\d+\)?)", text)}
    assert defs["MOE_FP8_STATIC_HISTOGRAM_MAX_TOKENS"] == binding.STATIC_HISTOGRAM_MAX_TOKENS
    assert defs["MOE_FP8_ERR_STATIC_LIMIT"] == binding.ERR_STATIC_LIMIT
    assert (defs["MOE_FP8_ERR_BAD_ARG"], defs["MOE_FP8_ERR_UNSUPPORTED_DIMS"], defs["MOE_FP8_ERR_NO_WORKSPACE"],
            defs["MOE_FP8_ERR_CUDA"], defs["MOE_FP8_ERR_ARCH"]) == (
        binding.ERR_BAD_ARG, binding.ERR_UNSUPPORTED_DIMS, binding.ERR_NO_WORKSPACE, binding.ERR_CUDA, binding.ERR_ARCH)
