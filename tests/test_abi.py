"""Host-only checks of the C-ABI library: it loads, exports every function the header
declares, and its pure-host helpers (sizes, status strings, workspace sizing) behave."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2308_14352_b200 import build, binding

    build.build()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "emoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(emoe_[a-z0-9_]+)\s*\(", text)))


def test_header_functions_are_exported(lib):
    from paper_2308_14352_b200 import binding

    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/emoe.h but not exported"
    assert set(binding.EXPORTS) == set(names)
    for n in names:  # the Python binding carries the same names
        assert hasattr(binding, n) or n in ("emoe_status_string",)


def test_size_helpers(lib):
    from paper_2308_14352_b200 import binding as B

    assert B.emoe_packed_bytes(3072, 768, 4) == 3072 * 768 // 2
    assert B.emoe_packed_bytes(3072, 768, 2) == 3072 * 768 // 4
    assert B.emoe_packed_bytes(4096, 14336, 8) == 4096 * 14336
    assert B.emoe_packed_bytes(8, 8, 3) == 0
    assert B.emoe_packed_bytes(1, 3, 2) == 0          # 6 bits: not a whole byte
    assert B.emoe_scales_bytes(3072, 768, 128, B.DTYPE_F16) == 3072 * 6 * 2
    assert B.emoe_scales_bytes(3072, 768, 0, B.DTYPE_F32) == 3072 * 4
    assert B.emoe_scales_bytes(3072, 768, 100, B.DTYPE_F16) == 0
    assert B.emoe_scales_bytes(3072, 768, 128, B.DTYPE_BF16) == 0


def test_status_strings(lib):
    from paper_2308_14352_b200 import binding as B

    seen = set()
    for code in (B.OK, B.ERR_INVALID_ARG, B.ERR_UNSUPPORTED, B.ERR_ALIGNMENT, B.ERR_WORKSPACE, B.ERR_CUDA,
                 B.ERR_DEVICE_CHECK):
        s = B.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 7
    assert B.status_string(-99) == "unknown status"


def test_workspace_sizing(lib):
    from paper_2308_14352_b200 import binding as B, inputs, layer

    w = inputs.WORKLOADS["mixtral_decode"]
    desc = layer.make_desc(w.shape)
    small, big = B.emoe_workspace_bytes(desc, 1), B.emoe_workspace_bytes(desc, 32)
    assert 0 < small < big
    # at least the hidden vectors and one copy of the expert outputs must fit
    assert big >= 32 * 2 * (14336 * 2 + 4096 * 4)
    bad = layer.make_desc(w.shape)
    bad.top_k = 9
    assert B.emoe_workspace_bytes(bad, 4) == 0
    assert B.emoe_workspace_bytes(desc, 0) == 0


def test_null_context_is_rejected_without_touching_a_gpu(lib):
    from paper_2308_14352_b200 import binding as B

    assert lib.emoe_destroy(None) == B.ERR_INVALID_ARG
    assert lib.emoe_set_ffn_path(None, 0) == B.ERR_INVALID_ARG
    assert lib.emoe_pack_expert(None, None, 1, 1, 4, 0, 0, None, None, None) == B.ERR_INVALID_ARG
    assert lib.emoe_last_cuda_error(None) == 0
