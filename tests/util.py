"""Shared helpers of the GPU parity tests (test code only)."""
import numpy as np
import torch

from oracle import losa_oracle as orc

MAX_ABS_TOL = 1e-2   # output tolerance against fp64, bf16 inputs / fp32 accumulation
MEAN_ABS_TOL = 1e-3
MASS_TOL = 1e-5      # masses lie in [0, 1]
NEAR_TAU = 1e-6      # rows whose cumulative mass is this close to tau may differ at the boundary


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().contiguous().numpy()


def rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator("cpu").manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).bfloat16()


def random_csr(rows, nKb, seed, keep_prob=0.5):
    """Random ascending block lists with at least one block per row."""
    rng = np.random.default_rng(seed)
    offs = [0]
    idx = []
    for _ in range(rows):
        keep = np.nonzero(rng.random(nKb) < keep_prob)[0]
        if keep.size == 0:
            keep = np.array([rng.integers(nKb)])
        idx.extend(keep.tolist())
        offs.append(len(idx))
    return np.asarray(offs, np.int32), np.asarray(idx, np.int32)


def all_blocks_csr(rows, nKb):
    return (np.arange(rows + 1, dtype=np.int32) * nKb,
            np.tile(np.arange(nKb, dtype=np.int32), rows))


def csr_rows(offsets, kv_idx):
    return [tuple(kv_idx[offsets[r]:offsets[r + 1]].tolist()) for r in range(len(offsets) - 1)]


def compare_csr(gpu_off, gpu_idx, sel: "orc.Selection"):
    """Bit-exact comparison of a GPU CSR with the oracle's; returns (mismatching rows outside the
    near-threshold exemption, number of exempt rows that differ)."""
    go = np.asarray(gpu_off)
    gi = np.asarray(gpu_idx)[: go[-1]]
    mine = csr_rows(go, gi)
    ref = csr_rows(sel.offsets, sel.kv_idx)
    dist = sel.boundary_distance()
    bad, exempt = [], 0
    for r, (a, b) in enumerate(zip(mine, ref)):
        if a != b:
            if dist[r] < NEAR_TAU:
                exempt += 1
            else:
                bad.append(r)
    return bad, exempt


def assert_output_close(o_gpu: torch.Tensor, o_ref: np.ndarray, what=""):
    diff = np.abs(to_np(o_gpu).astype(np.float64) - o_ref)
    assert np.isfinite(diff).all(), f"{what}: non-finite output"
    assert diff.max() <= MAX_ABS_TOL, f"{what}: max-abs {diff.max():.3e}"
    assert diff.mean() <= MEAN_ABS_TOL, f"{what}: mean-abs {diff.mean():.3e}"
    return diff.max(), diff.mean()
