"""Seeded random problems across every supported geometry, head dimension and mode against the
fp64 oracle: small sizes (one to a dozen tiles), ragged lengths, and index lists that range from a
single block to all blocks within one problem."""
import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu

GEOMETRIES = [(64, 64), (128, 128), (128, 64), (128, 32)]


def random_lists(rng, rows, nKb):
    offs, idx = [0], []
    for _ in range(rows):
        kind = rng.integers(5)
        if kind == 0:
            keep = np.array([rng.integers(nKb)])
        elif kind == 1:
            keep = np.arange(nKb)
        elif kind == 2:
            keep = np.sort(rng.choice(nKb, size=max(1, nKb // 3), replace=False))
        else:
            keep = np.nonzero(rng.random(nKb) < rng.random())[0]
        if keep.size == 0:
            keep = np.array([nKb - 1])
        idx.extend(keep.tolist())
        offs.append(len(idx))
    return np.asarray(offs, np.int32), np.asarray(idx, np.int32)


@pytest.mark.parametrize("seed", range(24))
def test_random_problem(seed):
    import paper_2608_12032_b200 as losa

    rng = np.random.default_rng(1000 + seed)
    R, C = GEOMETRIES[seed % 4]
    D = (64, 128)[(seed // 4) % 2]
    B, H = int(rng.integers(1, 3)), int(rng.integers(1, 5))
    N = int(rng.integers(1, 1400))
    q = util.rand_bf16((B, H, N, D), 3 * seed, 1.5)
    k = util.rand_bf16((B, H, N, D), 3 * seed + 1, 1.5)
    v = util.rand_bf16((B, H, N, D), 3 * seed + 2, 1.0)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    nQb, nKb = -(-N // R), -(-N // C)
    tag = f"seed {seed}: B{B} H{H} N{N} D{D} R{R} C{C}"

    off, idx = random_lists(rng, B * H * nQb, nKb)
    o = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(), R, C,
                              out_dtype=torch.float32)
    assert losa.losa_async_status() == 0, tag
    ref = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, R, C, off, idx), B, H, N)
    util.assert_output_close(o, ref, f"sparse, {tag}")

    o_f, mass = losa.losa_attn_mass(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0, tag
    dense = orc.dense_attn(qn, kn, vn)
    util.assert_output_close(o_f, dense, f"fused o, {tag}")
    ref_m = orc.block_mass(qn, kn, R, C)
    assert np.abs(mass.cpu().numpy().reshape(ref_m.shape) - ref_m).max() <= util.MASS_TOL, tag
    mass2 = losa.losa_block_mass(qd, kd, R, C)
    assert losa.losa_async_status() == 0, tag
    assert np.abs(mass2.cpu().numpy().reshape(ref_m.shape) - ref_m).max() <= util.MASS_TOL, tag
    o_d = losa.losa_attn(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0, tag
    util.assert_output_close(o_d, dense, f"dense, {tag}")
