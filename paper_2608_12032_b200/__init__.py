"""LoSA attention hot path for B200: block-mass pass, retained-mass selection, block-sparse
attention and the library's own dense attention, as hand-written sm_100a CUDA kernels behind a
C-ABI shared library (``liblosa.so``) with a ctypes binding of the same names."""
from . import inputs  # noqa: F401  (seeded synthetic workloads; no method arithmetic)
from .binding import (  # noqa: F401
    LosaError,
    Problem,
    check_async,
    losa_async_status,
    losa_attn,
    losa_attn_mass,
    losa_block_mass,
    losa_debug_stall_next_launch,
    losa_select,
    losa_select_noalloc,
    losa_select_topk,
    losa_row_recall,
    losa_sparse_attn,
    losa_sparse_attn_batched,
    losa_status_string,
    losa_validate_csr,
    losa_work_slots,
    losa_workspace_bytes,
    losa_workspace_bytes_batched,
    make_problem,
)
