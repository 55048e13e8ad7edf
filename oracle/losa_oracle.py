"""ctypes front end of the fp64 CPU oracle (``losa_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg import this module.  It shares no code with the CUDA library
and never imports it.

Inputs are numpy float32 arrays that hold the bf16 input values exactly
(``tensor.float().numpy()``), laid out ``[B, H, N, D]``.  All results are
float64 / int32 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "losa_oracle.c")
_LIB = None


def _cpu_flags() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    fl = set(line.split(":", 1)[1].split())
                    if "avx2" in fl and "fma" in fl:
                        return "avx2"
                    break
    except OSError:
        pass
    return "generic"


def lib_path() -> str:
    return os.path.join(_HERE, f"liblosa_oracle_{_cpu_flags()}.so")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc + OpenMP into this directory."""
    out = lib_path()
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
        return out
    flags = ["-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-fno-fast-math"]
    if _cpu_flags() == "avx2":
        flags += ["-mavx2", "-mfma"]
    tmp = out + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", *flags, "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, out)
    return out


def _lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(build())
        _LIB.losa_oracle_threads.restype = ctypes.c_int
    return _LIB


def threads() -> int:
    return int(_lib().losa_oracle_threads())


def _f32(x) -> np.ndarray:
    a = np.ascontiguousarray(x, dtype=np.float32)
    if a.ndim != 4:
        raise ValueError("expected [B, H, N, D]")
    return a


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _rows(row_ids: Optional[Sequence[int]], total: int) -> Tuple[Optional[np.ndarray], int]:
    if row_ids is None:
        return None, total
    r = np.ascontiguousarray(row_ids, dtype=np.int32)
    return r, int(r.size)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def dense_attn(q, k, v, scale: Optional[float] = None) -> np.ndarray:
    """Dense softmax attention, fp64, [B, H, N, D]."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, N, D = q.shape
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    o = np.empty((B, H, N, D), dtype=np.float64)
    _check(
        _lib().losa_oracle_dense_attn(
            _ptr(q), _ptr(k), _ptr(v), B, H, N, D, ctypes.c_double(scale), _ptr(o)
        ),
        "dense_attn",
    )
    return o


def block_mass(q, k, R: int, C: int, scale: Optional[float] = None,
               row_ids: Optional[Sequence[int]] = None, return_lse: bool = False):
    """Block attention mass (Eq. 1, averaged over the query block's valid rows).

    Returns ``mass [n_rows, nKb]`` (and ``lse [n_rows, R]``, natural log) for the
    query blocks in ``row_ids`` (flattened ``(b*H + h)*nQb + i``; None = all).
    """
    q, k = _f32(q), _f32(k)
    B, H, N, D = q.shape
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    nQb, nKb = -(-N // R), -(-N // C)
    rid, n = _rows(row_ids, B * H * nQb)
    mass = np.empty((n, nKb), dtype=np.float64)
    lse = np.empty((n, R), dtype=np.float64) if return_lse else None
    _check(
        _lib().losa_oracle_block_mass(
            _ptr(q), _ptr(k), B, H, N, D, R, C, ctypes.c_double(scale), n, _ptr(rid),
            _ptr(mass), _ptr(lse)
        ),
        "block_mass",
    )
    return (mass, lse) if return_lse else mass


class Selection:
    """Result of the retained-mass selection (Eq. 3) on ``rows`` query blocks."""

    def __init__(self, order, cum, count, kept, tau):
        self.order = order      # [rows, nKb] pi: blocks by decreasing mass, ties by lower index
        self.cum = cum          # [rows, nKb] cumulative mass along pi
        self.count = count      # [rows] s
        self.kept = kept        # [rows, nKb] ascending kept indices, -1 padded
        self.tau = tau

    @property
    def offsets(self) -> np.ndarray:
        off = np.zeros(self.count.size + 1, dtype=np.int64)
        np.cumsum(self.count, out=off[1:])
        return off.astype(np.int32)

    @property
    def kv_idx(self) -> np.ndarray:
        return self.kept[self.kept >= 0].astype(np.int32)

    def boundary_distance(self) -> np.ndarray:
        """Per row: min(|cum_s - tau|, |cum_{s-1} - tau|) — how close the decision was."""
        r = np.arange(self.count.size)
        s = self.count
        d = np.abs(self.cum[r, s - 1] - self.tau)
        prev = np.where(s >= 2, np.abs(self.cum[r, np.maximum(s - 2, 0)] - self.tau), np.inf)
        return np.minimum(d, prev)


def select(mass, tau: float) -> Selection:
    """Smallest prefix of the mass-sorted blocks whose cumulative mass reaches tau."""
    m = np.ascontiguousarray(mass, dtype=np.float64)
    if m.ndim != 2:
        raise ValueError("expected [rows, nKb]")
    rows, nKb = m.shape
    order = np.empty((rows, nKb), dtype=np.int32)
    cum = np.empty((rows, nKb), dtype=np.float64)
    count = np.empty((rows,), dtype=np.int32)
    kept = np.empty((rows, nKb), dtype=np.int32)
    _check(
        _lib().losa_oracle_select(
            _ptr(m), rows, nKb, ctypes.c_double(tau), _ptr(order), _ptr(cum), _ptr(count),
            _ptr(kept)
        ),
        "select",
    )
    return Selection(order, cum, count, kept, float(tau))


def select_topk(mass, k: int):
    """Fixed-ratio rule of the paper's ablation: (offsets, kv_idx) keeping the k heaviest blocks per row."""
    m = np.ascontiguousarray(mass, dtype=np.float64)
    rows, nKb = m.shape
    kept = np.empty((rows, k), dtype=np.int32)
    _check(_lib().losa_oracle_select_topk(_ptr(m), rows, nKb, int(k), _ptr(kept)), "select_topk")
    offsets = (np.arange(rows + 1, dtype=np.int64) * k).astype(np.int32)
    return offsets, kept.reshape(-1)


def row_recall(mass, offsets, kv_idx):
    """Per row: (retained mass, total mass) under the CSR pattern (Eq. 2 before the outer sums)."""
    m = np.ascontiguousarray(mass, dtype=np.float64)
    rows, nKb = m.shape
    off = np.ascontiguousarray(offsets, dtype=np.int32)
    idx = np.ascontiguousarray(kv_idx, dtype=np.int32)
    ret = np.empty(rows, dtype=np.float64)
    tot = np.empty(rows, dtype=np.float64)
    _check(_lib().losa_oracle_row_recall(_ptr(m), rows, nKb, _ptr(off), _ptr(idx), _ptr(ret), _ptr(tot)),
           "row_recall")
    return ret, tot


def sparse_attn(q, k, v, R: int, C: int, offsets, kv_idx, scale: Optional[float] = None,
                row_ids: Optional[Sequence[int]] = None) -> np.ndarray:
    """Attention restricted to the retained key blocks (Eq. 4): ``[n_rows, R, D]`` fp64."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, N, D = q.shape
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    nQb = -(-N // R)
    off = np.ascontiguousarray(offsets, dtype=np.int32)
    idx = np.ascontiguousarray(kv_idx, dtype=np.int32)
    if off.size != B * H * nQb + 1:
        raise ValueError("offsets must have B*H*nQb + 1 entries")
    rid, n = _rows(row_ids, B * H * nQb)
    o = np.empty((n, R, D), dtype=np.float64)
    _check(
        _lib().losa_oracle_sparse_attn(
            _ptr(q), _ptr(k), _ptr(v), B, H, N, D, R, C, ctypes.c_double(scale), _ptr(off),
            _ptr(idx), n, _ptr(rid), _ptr(o)
        ),
        "sparse_attn",
    )
    return o


def blocks_to_tokens(o_blocks: np.ndarray, B: int, H: int, N: int) -> np.ndarray:
    """[B*H*nQb, R, D] (all query blocks, in order) -> [B, H, N, D]."""
    rows, R, D = o_blocks.shape
    nQb = rows // (B * H)
    return o_blocks.reshape(B, H, nQb * R, D)[:, :, :N, :]


def recall(mass, offsets, kv_idx) -> float:
    """Retained fraction of the dense block mass (Eq. 2)."""
    m = np.asarray(mass, dtype=np.float64)
    rows, _ = m.shape
    off = np.asarray(offsets, dtype=np.int64)
    idx = np.asarray(kv_idx, dtype=np.int64)
    row_of = np.repeat(np.arange(rows), np.diff(off))
    return float(m[row_of, idx].sum() / m.sum())


def coverage(offsets, nKb: int) -> float:
    """Kept fraction of the block area (the paper's Coverage; uniform over heads)."""
    off = np.asarray(offsets, dtype=np.int64)
    rows = off.size - 1
    return float(off[-1]) / float(rows * nKb)


if __name__ == "__main__":
    print(build(force=True))
