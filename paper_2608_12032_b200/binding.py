"""ctypes binding of liblosa.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  PyTorch supplies device
memory and the current stream.  There is no CPU fallback: if the library cannot be
loaded the import of a function from here raises.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# (LOSA_LIBRARY selects another build of the same library, e.g. the checked build of the kernels)
LIB_PATH = os.environ.get("LOSA_LIBRARY") or os.path.join(_PKG, "liblosa.so")

LOSA_OP_BLOCK_MASS, LOSA_OP_SELECT, LOSA_OP_SPARSE_ATTN, LOSA_OP_ATTN, LOSA_OP_ATTN_MASS = 0, 1, 2, 3, 4
LOSA_DTYPE_BF16, LOSA_DTYPE_F32 = 0, 1

EXPORTS = (
    "losa_workspace_bytes", "losa_block_mass", "losa_select", "losa_sparse_attn", "losa_attn",
    "losa_attn_mass", "losa_select_topk", "losa_row_recall",
    "losa_select_noalloc", "losa_validate_csr", "losa_async_status", "losa_status_string", "losa_last_cuda_error",
    "losa_debug_stall_next_launch", "losa_sparse_attn_batched", "losa_workspace_bytes_batched",
    "losa_work_slots",
)


class LosaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        lib = _lib()
        name = lib.losa_status_string(code).decode()
        detail = lib.losa_last_cuda_error().decode()
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail and code == -5 else ""))


class Problem(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("D", ctypes.c_int32),
        ("R", ctypes.c_int32), ("C", ctypes.c_int32),
        ("sb", ctypes.c_int64), ("sh", ctypes.c_int64), ("sn", ctypes.c_int64),
        ("scale", ctypes.c_float),
    ]


class Layer(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("offsets", ctypes.c_void_p), ("kv_idx", ctypes.c_void_p), ("o", ctypes.c_void_p),
    ]


_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_12032_b200.build` "
                "(there is no fallback path)"
            )
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        pp = ctypes.POINTER(Problem)
        lib.losa_workspace_bytes.restype = sz
        lib.losa_workspace_bytes.argtypes = [ctypes.c_int, pp]
        lib.losa_block_mass.restype = ctypes.c_int
        lib.losa_block_mass.argtypes = [pp, vp, vp, vp, vp, vp, sz, vp]
        lib.losa_select.restype = ctypes.c_int
        lib.losa_select.argtypes = [i32, i32, i32, i32, vp, ctypes.c_double, vp, vp, i64, vp, sz, vp]
        lib.losa_select_topk.restype = ctypes.c_int
        lib.losa_select_topk.argtypes = [i32, i32, i32, i32, vp, i32, vp, vp, i64, vp, sz, vp]
        lib.losa_row_recall.restype = ctypes.c_int
        lib.losa_row_recall.argtypes = [i32, i32, vp, vp, vp, vp, vp, vp]
        lib.losa_select_noalloc.restype = ctypes.c_int
        lib.losa_select_noalloc.argtypes = [i32, i32, i32, i32, vp, ctypes.c_double, vp, vp, i64, vp, vp]
        lib.losa_sparse_attn.restype = ctypes.c_int
        lib.losa_sparse_attn.argtypes = [pp, vp, vp, vp, vp, vp, vp, ctypes.c_int, vp, sz, vp]
        lib.losa_sparse_attn_batched.restype = ctypes.c_int
        lib.losa_sparse_attn_batched.argtypes = [pp, i32, ctypes.POINTER(Layer), ctypes.c_int, vp, sz, vp]
        lib.losa_workspace_bytes_batched.restype = sz
        lib.losa_workspace_bytes_batched.argtypes = [ctypes.c_int, pp, i32]
        lib.losa_work_slots.restype = i32
        lib.losa_work_slots.argtypes = [ctypes.c_int, pp]
        lib.losa_attn.restype = ctypes.c_int
        lib.losa_attn.argtypes = [pp, vp, vp, vp, vp, ctypes.c_int, vp, sz, vp]
        lib.losa_attn_mass.restype = ctypes.c_int
        lib.losa_attn_mass.argtypes = [pp, vp, vp, vp, vp, ctypes.c_int, vp, vp, vp, sz, vp]
        lib.losa_validate_csr.restype = ctypes.c_int
        lib.losa_validate_csr.argtypes = [i32, i32, vp, vp, vp]
        lib.losa_async_status.restype = ctypes.c_int
        lib.losa_async_status.argtypes = [vp]
        lib.losa_debug_stall_next_launch.restype = ctypes.c_int
        lib.losa_debug_stall_next_launch.argtypes = [ctypes.c_uint32]
        lib.losa_status_string.restype = ctypes.c_char_p
        lib.losa_status_string.argtypes = [ctypes.c_int]
        lib.losa_last_cuda_error.restype = ctypes.c_char_p
        lib.losa_last_cuda_error.argtypes = []
        _LIB = lib
    return _LIB


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise LosaError(rc, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def make_problem(q: torch.Tensor, R: int, C: int, scale: Optional[float] = None) -> Problem:
    if q.dim() != 4 or q.stride(3) != 1:
        raise ValueError("expected [B, H, N, D] with a contiguous last dimension")
    B, H, N, D = q.shape
    return Problem(B, H, N, D, R, C, q.stride(0), q.stride(1), q.stride(2),
                   0.0 if scale is None else float(scale))


def _same_layout(ref: torch.Tensor, *others: torch.Tensor) -> None:
    for t in others:
        if t.shape != ref.shape or t.stride() != ref.stride():
            raise ValueError("q, k, v (and o) must share shape and strides")
        if t.device != ref.device:
            raise ValueError("tensors must live on the same device")


def losa_workspace_bytes(op: int, problem: Problem) -> int:
    return int(_lib().losa_workspace_bytes(op, ctypes.byref(problem)))


def losa_work_slots(op: int, problem: Problem) -> int:
    """Work slots (persistent CTAs, or pairs of them) an attention call of this kind occupies."""
    return int(_lib().losa_work_slots(op, ctypes.byref(problem)))


def _workspace(op: int, problem: Problem, device, ws: Optional[torch.Tensor]) -> Tuple[Optional[torch.Tensor], int]:
    need = losa_workspace_bytes(op, problem)
    if ws is None and need > 0:
        ws = torch.empty(need, dtype=torch.uint8, device=device)
    return ws, (0 if ws is None else ws.numel() * ws.element_size())


def losa_block_mass(q: torch.Tensor, k: torch.Tensor, R: int, C: int, scale: Optional[float] = None,
                    return_lse: bool = False, ws: Optional[torch.Tensor] = None,
                    mass: Optional[torch.Tensor] = None):
    """mass[B, H, nQb, nKb] (fp32) of one dense attention step; optionally the rows' log-sum-exp."""
    _same_layout(q, k)
    prob = make_problem(q, R, C, scale)
    B, H, N, _ = q.shape
    nQb, nKb = -(-N // R), -(-N // C)
    if mass is None:
        mass = torch.empty((B, H, nQb, nKb), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if return_lse else None
    ws, ws_bytes = _workspace(LOSA_OP_BLOCK_MASS, prob, q.device, ws)
    _check(_lib().losa_block_mass(ctypes.byref(prob), _ptr(q), _ptr(k), _ptr(mass), _ptr(lse),
                                  _ptr(ws), ws_bytes, _stream()), "losa_block_mass")
    return (mass, lse) if return_lse else mass


def losa_select(mass: torch.Tensor, tau: float, kv_capacity: Optional[int] = None,
                ws: Optional[torch.Tensor] = None,
                out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None):
    """(offsets[rows + 1], kv_idx[kv_capacity]) int32; kv_idx is valid up to offsets[-1]."""
    if mass.dim() != 4 or not mass.is_contiguous() or mass.dtype != torch.float32:
        raise ValueError("mass must be a contiguous fp32 [B, H, nQb, nKb] tensor")
    B, H, nQb, nKb = mass.shape
    rows = B * H * nQb
    if out is None:
        cap = rows * nKb if kv_capacity is None else int(kv_capacity)
        offsets = torch.empty(rows + 1, dtype=torch.int32, device=mass.device)
        kv_idx = torch.empty(max(cap, 1), dtype=torch.int32, device=mass.device)
    else:
        offsets, kv_idx = out
        cap = kv_idx.numel() if kv_capacity is None else int(kv_capacity)
    ws_need = _select_workspace_bytes(B, H, nQb, nKb)
    if ws is None:
        ws = torch.empty(ws_need, dtype=torch.uint8, device=mass.device)
    _check(_lib().losa_select(B, H, nQb, nKb, _ptr(mass), float(tau), _ptr(offsets), _ptr(kv_idx),
                              cap, _ptr(ws), ws.numel(), _stream()), "losa_select")
    return offsets, kv_idx


def losa_select_topk(mass: torch.Tensor, k: int, ws: Optional[torch.Tensor] = None):
    """Fixed-ratio selection: (offsets, kv_idx) keeping the k heaviest blocks of every row."""
    if mass.dim() != 4 or not mass.is_contiguous() or mass.dtype != torch.float32:
        raise ValueError("mass must be a contiguous fp32 [B, H, nQb, nKb] tensor")
    B, H, nQb, nKb = mass.shape
    rows = B * H * nQb
    offsets = torch.empty(rows + 1, dtype=torch.int32, device=mass.device)
    kv_idx = torch.empty(max(rows * int(k), 1), dtype=torch.int32, device=mass.device)
    if ws is None:
        ws = torch.empty(_select_workspace_bytes(B, H, nQb, nKb), dtype=torch.uint8, device=mass.device)
    _check(_lib().losa_select_topk(B, H, nQb, nKb, _ptr(mass), int(k), _ptr(offsets), _ptr(kv_idx),
                                   kv_idx.numel(), _ptr(ws), ws.numel(), _stream()), "losa_select_topk")
    return offsets, kv_idx


def losa_row_recall(mass: torch.Tensor, offsets: torch.Tensor, kv_idx: torch.Tensor):
    """(retained, total) fp64 per row: Recall (Eq. 2) is retained.sum() / total.sum()."""
    if not mass.is_contiguous() or mass.dtype != torch.float32:
        raise ValueError("mass must be a contiguous fp32 tensor")
    nKb = mass.shape[-1]
    rows = mass.numel() // nKb
    retained = torch.empty(rows, dtype=torch.float64, device=mass.device)
    total = torch.empty(rows, dtype=torch.float64, device=mass.device)
    _check(_lib().losa_row_recall(rows, nKb, _ptr(mass), _ptr(offsets), _ptr(kv_idx), _ptr(retained),
                                  _ptr(total), _stream()), "losa_row_recall")
    return retained, total


def losa_select_noalloc(mass: torch.Tensor, tau: float, offsets: torch.Tensor, kv_idx: torch.Tensor,
                        device_status: Optional[torch.Tensor] = None) -> None:
    """losa_select without any allocation: for callers that own no allocator.

    The caller passes every output (``offsets`` [rows + 1], ``kv_idx`` [capacity], optionally a
    one-element int32 ``device_status``); the scratch memory is a fixed array inside the library.
    This wrapper itself allocates nothing either.  Calls that may overlap on the GPU share that
    array and must be serialised by the caller.
    """
    if mass.dim() != 4 or not mass.is_contiguous() or mass.dtype != torch.float32:
        raise ValueError("mass must be a contiguous fp32 [B, H, nQb, nKb] tensor")
    B, H, nQb, nKb = mass.shape
    _check(_lib().losa_select_noalloc(B, H, nQb, nKb, _ptr(mass), float(tau), _ptr(offsets),
                                      _ptr(kv_idx), kv_idx.numel(), _ptr(device_status), _stream()),
           "losa_select_noalloc")


def _select_workspace_bytes(B: int, H: int, nQb: int, nKb: int) -> int:
    # losa_workspace_bytes(LOSA_OP_SELECT) reads B, H and ceil(N/R), ceil(N/C): describe the
    # mass matrix as N = nQb * nKb tokens with R = nKb and C = nQb.
    prob = Problem(B, H, nQb * nKb, 64, nKb, nQb, 0, 0, 0, 0.0)
    return losa_workspace_bytes(LOSA_OP_SELECT, prob)


def losa_sparse_attn(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, offsets: torch.Tensor,
                     kv_idx: torch.Tensor, R: int, C: int, scale: Optional[float] = None,
                     out_dtype: torch.dtype = torch.bfloat16, out: Optional[torch.Tensor] = None,
                     ws: Optional[torch.Tensor] = None):
    """Block-sparse attention over the frozen CSR pattern; rows >= N do not exist."""
    _same_layout(q, k, v)
    prob = make_problem(q, R, C, scale)
    o = _alloc_out(q, out_dtype, out)
    ws, ws_bytes = _workspace(LOSA_OP_SPARSE_ATTN, prob, q.device, ws)
    _check(_lib().losa_sparse_attn(ctypes.byref(prob), _ptr(q), _ptr(k), _ptr(v), _ptr(offsets),
                                   _ptr(kv_idx), _ptr(o), _dtype_code(o.dtype), _ptr(ws), ws_bytes,
                                   _stream()),
           "losa_sparse_attn")
    return o


def losa_workspace_bytes_batched(op: int, problem: Problem, n_layers: int) -> int:
    return int(_lib().losa_workspace_bytes_batched(op, ctypes.byref(problem), int(n_layers)))


def losa_sparse_attn_batched(layers, R: int, C: int, scale: Optional[float] = None,
                             out_dtype: torch.dtype = torch.bfloat16, outs=None,
                             ws: Optional[torch.Tensor] = None):
    """Block-sparse attention of several problems of one shape in one launch.

    ``layers`` is a sequence of ``(q, k, v, offsets, kv_idx)``; returns the list of outputs."""
    q0 = layers[0][0]
    prob = make_problem(q0, R, C, scale)
    arr = (Layer * len(layers))()
    result = []
    for i, (q, k, v, offsets, kv_idx) in enumerate(layers):
        _same_layout(q0, q, k, v)
        o = _alloc_out(q, out_dtype, None if outs is None else outs[i])
        result.append(o)
        arr[i] = Layer(_ptr(q), _ptr(k), _ptr(v), _ptr(offsets), _ptr(kv_idx), _ptr(o))
    need = losa_workspace_bytes_batched(LOSA_OP_SPARSE_ATTN, prob, len(layers))
    if ws is None:
        ws = torch.empty(max(need, 1), dtype=torch.uint8, device=q0.device)
    _check(_lib().losa_sparse_attn_batched(ctypes.byref(prob), len(layers), arr,
                                           _dtype_code(result[0].dtype), _ptr(ws), ws.numel(), _stream()),
           "losa_sparse_attn_batched")
    return result


def losa_attn(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, R: int = 128, C: int = 128,
              scale: Optional[float] = None, out_dtype: torch.dtype = torch.bfloat16,
              out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None):
    """Dense softmax attention with the library's own kernel."""
    _same_layout(q, k, v)
    prob = make_problem(q, R, C, scale)
    o = _alloc_out(q, out_dtype, out)
    ws, ws_bytes = _workspace(LOSA_OP_ATTN, prob, q.device, ws)
    _check(_lib().losa_attn(ctypes.byref(prob), _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                            _dtype_code(o.dtype), _ptr(ws), ws_bytes, _stream()), "losa_attn")
    return o


def losa_attn_mass(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, R: int, C: int,
                   scale: Optional[float] = None, out_dtype: torch.dtype = torch.bfloat16,
                   return_lse: bool = False, out: Optional[torch.Tensor] = None,
                   mass: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None):
    """The construction step in one kernel: (o, mass[, lse]) = dense attention + block masses."""
    _same_layout(q, k, v)
    prob = make_problem(q, R, C, scale)
    B, H, N, _ = q.shape
    o = _alloc_out(q, out_dtype, out)
    if mass is None:
        mass = torch.empty((B, H, -(-N // R), -(-N // C)), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if return_lse else None
    ws, ws_bytes = _workspace(LOSA_OP_ATTN_MASS, prob, q.device, ws)
    _check(_lib().losa_attn_mass(ctypes.byref(prob), _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                 _dtype_code(o.dtype), _ptr(mass), _ptr(lse), _ptr(ws), ws_bytes,
                                 _stream()), "losa_attn_mass")
    return (o, mass, lse) if return_lse else (o, mass)


def losa_validate_csr(offsets: torch.Tensor, kv_idx: torch.Tensor, nKb: int) -> None:
    _check(_lib().losa_validate_csr(offsets.numel() - 1, nKb, _ptr(offsets), _ptr(kv_idx), _stream()),
           "losa_validate_csr")


def losa_async_status() -> int:
    """Synchronises the current stream and returns (and clears) the device-side status."""
    return int(_lib().losa_async_status(_stream()))


def losa_debug_stall_next_launch(polls: int = 2048) -> None:
    """Arms one diagnostic attention launch whose waits all run out (LOSA_ERR_TIMEOUT)."""
    _check(_lib().losa_debug_stall_next_launch(int(polls)), "losa_debug_stall_next_launch")


def losa_status_string(code: int) -> str:
    return _lib().losa_status_string(code).decode()


def check_async(where: str = "liblosa") -> None:
    code = losa_async_status()
    if code != 0:
        raise LosaError(code, where)


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return LOSA_DTYPE_BF16
    if dt == torch.float32:
        return LOSA_DTYPE_F32
    raise ValueError("output dtype must be bfloat16 or float32")


def _alloc_out(q: torch.Tensor, dtype: torch.dtype, out: Optional[torch.Tensor]) -> torch.Tensor:
    if out is not None:
        if out.shape != q.shape or out.stride() != q.stride():
            raise ValueError("o must share q's shape and strides")
        return out
    return torch.empty_strided(q.shape, q.stride(), dtype=dtype, device=q.device)


def default_scale(D: int) -> float:
    return 1.0 / math.sqrt(D)
