"""The C-ABI library loads and exports every symbol include/losa.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2608_12032_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "losa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(losa_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert set(names) >= set(binding.EXPORTS)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_mirrors_the_header_names():
    for n in declared_symbols():
        if n == "losa_last_cuda_error":
            continue  # surfaced through LosaError
        assert hasattr(binding, n), n


def test_workspace_sizing_and_status_strings_need_no_gpu():
    p = binding.Problem(1, 12, 32760, 128, 128, 128, 12 * 32760 * 128, 32760 * 128, 128, 0.0)
    assert binding.losa_workspace_bytes(binding.LOSA_OP_BLOCK_MASS, p) > 0
    assert binding.losa_workspace_bytes(binding.LOSA_OP_SELECT, p) > 0
    # counter + one partial-result slot per persistent CTA: independent of N
    assert 0 < binding.losa_workspace_bytes(binding.LOSA_OP_ATTN, p) <= 32 << 20
    bad = binding.Problem(1, 1, 128, 96, 128, 128, 128 * 96, 128 * 96, 96, 0.0)
    assert binding.losa_workspace_bytes(binding.LOSA_OP_BLOCK_MASS, bad) == 0
    assert binding.losa_status_string(0) == "LOSA_OK"
    assert binding.losa_status_string(-6) == "LOSA_ERR_TIMEOUT"
