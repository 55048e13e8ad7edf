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
    # block geometries: query blocks of 128 rows go with key blocks of 128, 64 or 32 (the paper's own),
    # query blocks of 64 rows with key blocks of 64 only
    for R, C, ok in [(128, 128, True), (128, 64, True), (128, 32, True), (64, 64, True), (64, 32, False),
                     (32, 32, False), (128, 16, False), (64, 128, False)]:
        g = binding.Problem(1, 2, 1000, 128, R, C, 2 * 1000 * 128, 1000 * 128, 128, 0.0)
        for op in (binding.LOSA_OP_BLOCK_MASS, binding.LOSA_OP_SPARSE_ATTN, binding.LOSA_OP_ATTN,
                   binding.LOSA_OP_ATTN_MASS):
            assert (binding.losa_workspace_bytes(op, g) > 0) == ok, (R, C, op)
    # the sparse forward also holds the merged tile lists of all work units: grows with N / C
    small = binding.Problem(1, 12, 32760, 128, 128, 128, 12 * 32760 * 128, 32760 * 128, 128, 0.0)
    fine = binding.Problem(1, 12, 32760, 128, 128, 32, 12 * 32760 * 128, 32760 * 128, 128, 0.0)
    assert (binding.losa_workspace_bytes(binding.LOSA_OP_SPARSE_ATTN, fine)
            > binding.losa_workspace_bytes(binding.LOSA_OP_SPARSE_ATTN, small)
            > binding.losa_workspace_bytes(binding.LOSA_OP_ATTN, small))
    assert binding.losa_status_string(0) == "LOSA_OK"
    assert binding.losa_status_string(-6) == "LOSA_ERR_TIMEOUT"
