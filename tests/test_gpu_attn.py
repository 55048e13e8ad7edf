"""Dense attention, block-sparse attention and the block-mass pass on the GPU against the fp64
oracle, element by element, through the C ABI.  Sizes span several tiles, odd tile counts, both
block geometries and ragged tails."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc
from paper_2608_12032_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu

# (B, H, N, D, BLK): several 128-row tiles, odd numbers of tiles, short last blocks
SHAPES = [
    (1, 1, 128, 128, 128),
    (1, 2, 256, 64, 64),
    (1, 2, 300, 128, 128),
    (2, 2, 1000, 64, 64),
    (1, 3, 777, 128, 64),
    (1, 2, 650, 64, 128),
    (1, 1, 1500, 128, 128),
]


def lib():
    import paper_2608_12032_b200 as losa
    return losa


def make(B, H, N, D, seed, scale=1.0):
    """q, k ~ N(0, scale^2) (scale > 1 sharpens the softmax), v ~ N(0, 1) as in the workloads."""
    return (util.rand_bf16((B, H, N, D), seed, scale), util.rand_bf16((B, H, N, D), seed + 1, scale),
            util.rand_bf16((B, H, N, D), seed + 2, 1.0))


@pytest.mark.parametrize("shape", SHAPES)
def test_dense_attention_matches_oracle(shape):
    losa = lib()
    B, H, N, D, BLK = shape
    q, k, v = make(B, H, N, D, 11, 1.5)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    o = losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
    o16 = losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=torch.bfloat16)
    assert losa.losa_async_status() == 0
    ref = orc.dense_attn(util.to_np(q), util.to_np(k), util.to_np(v))
    # the fp32 output carries the tolerance; the bf16 output is the same value rounded once
    util.assert_output_close(o, ref, f"dense {shape}")
    assert torch.equal(o16, o.bfloat16())
    assert np.all(np.abs(util.to_np(o16) - ref) <= util.MAX_ABS_TOL + np.abs(ref) * 2.0 ** -8)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("keep_prob", [0.15, 0.6])
def test_sparse_attention_matches_oracle_on_random_patterns(shape, keep_prob):
    losa = lib()
    B, H, N, D, BLK = shape
    q, k, v = make(B, H, N, D, 21, 1.5)
    nQb = nKb = -(-N // BLK)
    off, idx = util.random_csr(B * H * nQb, nKb, 5 + N, keep_prob)
    o = losa.losa_sparse_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(off).cuda(),
                              torch.from_numpy(idx).cuda(), BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    ref = orc.blocks_to_tokens(
        orc.sparse_attn(util.to_np(q), util.to_np(k), util.to_np(v), BLK, BLK, off, idx), B, H, N)
    util.assert_output_close(o, ref, f"sparse {shape}")


@pytest.mark.parametrize("shape", SHAPES)
def test_sparse_with_all_blocks_equals_own_dense(shape):
    losa = lib()
    B, H, N, D, BLK = shape
    q, k, v = (t.cuda() for t in make(B, H, N, D, 31))
    nb = -(-N // BLK)
    off, idx = util.all_blocks_csr(B * H * nb, nb)
    o_s = losa.losa_sparse_attn(q, k, v, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(),
                                BLK, BLK, out_dtype=torch.float32)
    o_d = losa.losa_attn(q, k, v, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    assert torch.equal(o_s, o_d)  # same tiles in the same order: bit-identical


@pytest.mark.parametrize("shape", SHAPES)
def test_block_mass_matches_oracle(shape):
    losa = lib()
    B, H, N, D, BLK = shape
    q, k, _ = make(B, H, N, D, 41, 1.5)
    mass, lse = losa.losa_block_mass(q.cuda(), k.cuda(), BLK, BLK, return_lse=True)
    assert losa.losa_async_status() == 0
    ref, ref_lse = orc.block_mass(util.to_np(q), util.to_np(k), BLK, BLK, return_lse=True)
    got = mass.cpu().numpy().reshape(ref.shape).astype(np.float64)
    assert np.abs(got - ref).max() <= util.MASS_TOL
    assert np.abs(got.sum(1) - 1.0).max() <= util.MASS_TOL
    nQb = -(-N // BLK)
    lse_ref = ref_lse.reshape(B, H, nQb * BLK)[:, :, :N]
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 1e-3


@pytest.mark.parametrize("shape", SHAPES)
def test_fused_construction_step_matches_oracle_and_the_separate_calls(shape):
    """losa_attn_mass = dense attention + block masses in one pass (the paper's construction kernel)."""
    losa = lib()
    B, H, N, D, BLK = shape
    q, k, v = make(B, H, N, D, 71, 1.5)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    o, mass, lse = losa.losa_attn_mass(qd, kd, vd, BLK, BLK, out_dtype=torch.float32, return_lse=True)
    o_sep = losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    util.assert_output_close(o, orc.dense_attn(qn, kn, vn), f"fused o {shape}")
    # same tiles and arithmetic; the separate call may cut its last work items into parts of the key
    # range and merge them, which changes the summation order, not the result beyond rounding: two
    # approximations, each within the tolerance of the exact result
    assert (o - o_sep).abs().max().item() <= 2 * util.MAX_ABS_TOL
    assert (o - o_sep).abs().mean().item() <= 2 * util.MEAN_ABS_TOL  # no systematic difference
    ref, ref_lse = orc.block_mass(qn, kn, BLK, BLK, return_lse=True)
    got = mass.cpu().numpy().reshape(ref.shape).astype(np.float64)
    assert np.abs(got - ref).max() <= util.MASS_TOL
    assert np.abs(got.sum(1) - 1.0).max() <= util.MASS_TOL
    nQb = -(-N // BLK)
    assert np.abs(lse.cpu().numpy() - ref_lse.reshape(B, H, nQb * BLK)[:, :, :N]).max() <= 1e-3


@pytest.mark.parametrize("name,taus", [("tiny", (0.5, 0.75, 0.9, 0.99)), ("small", (0.9, 0.99, 1.0))])
def test_chain_mass_select_sparse_on_named_workloads(name, taus):
    """mass -> select -> sparse on the generator's tensors: strict selection parity on the GPU's
    own masses, chain differences explained by the mass error, output parity on the oracle CSR."""
    losa = lib()
    wl = inputs.WORKLOADS[name]
    q, k, v = inputs.make_qkv(wl, 0)
    qn, kn, vn = (util.to_np(t) for t in (q, k, v))
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    mass = losa.losa_block_mass(qd, kd, wl.R, wl.C)
    ref_mass = orc.block_mass(qn, kn, wl.R, wl.C)
    gm = mass.cpu().numpy().reshape(ref_mass.shape)
    mass_err = np.abs(gm - ref_mass).max()
    assert mass_err <= util.MASS_TOL
    for tau in taus:
        off, idx = losa.losa_select(mass, tau)
        assert losa.losa_async_status() == 0
        off_h, idx_h = off.cpu().numpy(), idx.cpu().numpy()
        # strict: the oracle's rule on the very same fp32 masses
        strict = orc.select(gm.astype(np.float64), tau)
        bad, _ = util.compare_csr(off_h, idx_h, strict)
        assert not bad
        # chain: oracle masses -> oracle selection; differences only where the decision was
        # closer to tau than the mass error allows
        chain = orc.select(ref_mass, tau)
        mine, ref = util.csr_rows(off_h, idx_h[: off_h[-1]]), util.csr_rows(chain.offsets, chain.kv_idx)
        dist = chain.boundary_distance()
        for r, (a, b) in enumerate(zip(mine, ref)):
            if a != b:
                assert dist[r] <= mass_err * wl.nKb + util.NEAR_TAU
        # output parity with the same CSR on both sides (the oracle's)
        o = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(chain.offsets).cuda(),
                                  torch.from_numpy(chain.kv_idx).cuda(), wl.R, wl.C,
                                  out_dtype=torch.float32)
        ref_o = orc.blocks_to_tokens(
            orc.sparse_attn(qn, kn, vn, wl.R, wl.C, chain.offsets, chain.kv_idx), wl.B, wl.H, wl.N)
        util.assert_output_close(o, ref_o, f"{name} tau={tau}")
        assert orc.recall(ref_mass, off_h, idx_h[: off_h[-1]]) >= tau - 1e-4
    assert losa.losa_async_status() == 0


def test_two_guidance_branches_in_one_batch_keep_their_own_patterns():
    """The two classifier-free-guidance branches travel as B = 2 and each (b, h, query block) row
    of the CSR is its own pattern: one batched pass over both branches must equal the two
    single-branch passes bit for bit in masses and CSR, and in the output up to the rounding of P
    (a launch with fewer work units cuts them into more parts, each with its own reference, so the
    bf16 weights round differently), and each branch must match the oracle on its own pattern.
    The branches get differently sharp scores, so their patterns differ."""
    losa = lib()
    H, N, D, BLK, tau = 2, 900, 128, 128, 0.9
    q0, k0, v0 = make(1, H, N, D, 71, 1.0)
    q1, k1, v1 = make(1, H, N, D, 81, 2.0)
    q, k, v = (torch.cat(p) for p in ((q0, q1), (k0, k1), (v0, v1)))
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    mass = losa.losa_block_mass(qd, kd, BLK, BLK)
    off, idx = losa.losa_select(mass, tau)
    o = losa.losa_sparse_attn(qd, kd, vd, off, idx, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    off_h, idx_h = off.cpu().numpy(), idx.cpu().numpy()
    nQb = -(-N // BLK)
    rows = H * nQb
    per_branch = []
    for b in range(2):
        qb, kb, vb = (t[b:b + 1].contiguous() for t in (qd, kd, vd))
        mb = losa.losa_block_mass(qb, kb, BLK, BLK)
        ob_, ib_ = losa.losa_select(mb, tau)
        o_b = losa.losa_sparse_attn(qb, kb, vb, ob_, ib_, BLK, BLK, out_dtype=torch.float32)
        assert torch.equal(mb.reshape(-1), mass[b].reshape(-1))
        lo, hi = off_h[b * rows], off_h[(b + 1) * rows]
        assert np.array_equal(ob_.cpu().numpy(), off_h[b * rows:(b + 1) * rows + 1] - lo)
        assert np.array_equal(ib_.cpu().numpy()[: hi - lo], idx_h[lo:hi])
        assert (o_b[0] - o[b]).abs().max().item() <= util.MAX_ABS_TOL
        per_branch.append(util.csr_rows(ob_.cpu().numpy(), ib_.cpu().numpy()[: hi - lo]))
        # against the oracle, branch by branch
        qn, kn, vn = (util.to_np(t[b:b + 1]) for t in (q, k, v))
        sel = orc.select(mb.cpu().numpy().reshape(rows, -1).astype(np.float64), tau)
        bad, _ = util.compare_csr(ob_.cpu().numpy(), ib_.cpu().numpy(), sel)
        assert not bad
        ref = orc.blocks_to_tokens(
            orc.sparse_attn(qn, kn, vn, BLK, BLK, sel.offsets, sel.kv_idx), 1, H, N)
        util.assert_output_close(o[b:b + 1], ref, f"branch {b}")
    assert per_branch[0] != per_branch[1]


def test_strided_heads_layout():
    """[B, N, H, D] storage viewed as [B, H, N, D]: strides come from the problem description."""
    losa = lib()
    B, H, N, D, BLK = 1, 3, 400, 64, 64
    base = [util.rand_bf16((B, N, H, D), 51 + i) for i in range(3)]
    q, k, v = (t.cuda().permute(0, 2, 1, 3) for t in base)
    assert not q.is_contiguous()
    o = losa.losa_attn(q, k, v, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0 and o.stride() == q.stride()
    qn, kn, vn = (util.to_np(t.permute(0, 2, 1, 3)) for t in base)
    util.assert_output_close(o, orc.dense_attn(qn, kn, vn), "strided")


def test_bad_block_index_is_reported_and_skipped():
    losa = lib()
    B, H, N, D, BLK = 1, 1, 512, 64, 64
    q, k, v = (t.cuda() for t in make(B, H, N, D, 61))
    off, idx = util.random_csr(8, 8, 1, 0.5)
    good = idx.copy()
    bad = idx.copy()
    victim = int(off[3])
    bad[victim] = 99  # out of range: must be skipped, not dereferenced
    o = losa.losa_sparse_attn(q, k, v, torch.from_numpy(off).cuda(), torch.from_numpy(bad).cuda(),
                              BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_status_string(losa.losa_async_status()) == "LOSA_ERR_BAD_INDEX"
    assert torch.isfinite(o).all()
    # the other rows are unaffected
    o_good = losa.losa_sparse_attn(q, k, v, torch.from_numpy(off).cuda(),
                                   torch.from_numpy(good).cuda(), BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    keep = torch.ones(N, dtype=torch.bool)
    keep[3 * BLK:4 * BLK] = False
    assert torch.equal(o[0, 0, keep.cuda()], o_good[0, 0, keep.cuda()])


def test_host_side_argument_errors():
    losa = lib()
    q = torch.zeros(1, 1, 128, 96, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(losa.LosaError) as e:
        losa.losa_attn(q, q, q, 128, 128)
    assert e.value.code == -2
    q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(losa.LosaError) as e:
        losa.losa_attn(q, q, q, 64, 32)  # query blocks of 64 rows go with key blocks of 64 only
    assert e.value.code == -2
    with pytest.raises(losa.LosaError) as e:
        losa.losa_block_mass(q, q, 64, 64, ws=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3


def test_kernels_are_deterministic():
    losa = lib()
    wl = dataclasses.replace(inputs.WORKLOADS["small"], H=2)
    q, k, v = (t.cuda() for t in inputs.make_qkv(wl, 3))
    m1 = losa.losa_block_mass(q, k, wl.R, wl.C)
    m2 = losa.losa_block_mass(q, k, wl.R, wl.C)
    o1 = losa.losa_attn(q, k, v, wl.R, wl.C)
    o2 = losa.losa_attn(q, k, v, wl.R, wl.C)
    assert losa.losa_async_status() == 0
    assert torch.equal(m1, m2) and torch.equal(o1, o2)


@pytest.mark.parametrize("D,BLK,H,tiles", [(64, 64, 5, 65), (128, 128, 7, 47)])
def test_last_wave_items_cut_into_parts_and_merged(D, BLK, H, tiles):
    """More work items than SMs, with a remainder: the items of the last, partly filled wave are
    processed as parts of their key-block lists whose partial results a second kernel merges.
    Checks query blocks of those items (and of whole items) against the oracle, for a sparse
    pattern with very uneven lists and for dense attention, in both output types."""
    losa = lib()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    B, N = 1, tiles * 128 - 37
    items = H * ((tiles + 1) // 2)
    assert items > sms and items % sms != 0, "shape no longer exercises the split on this GPU"
    q, k, v = make(B, H, N, D, 91, 1.5)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    nQb = nKb = -(-N // BLK)
    rows = B * H * nQb
    rng = np.random.default_rng(17)
    # uneven lists: some rows keep one block, some half, some all
    offs, idx = [0], []
    for r in range(rows):
        mode = rng.integers(4)
        if mode == 0:
            keep = np.array([rng.integers(nKb)])
        elif mode == 1:
            keep = np.arange(nKb)
        else:
            keep = np.nonzero(rng.random(nKb) < 0.4)[0]
            if keep.size == 0:
                keep = np.array([0])
        idx.extend(keep.tolist())
        offs.append(len(idx))
    off, idx = np.asarray(offs, np.int32), np.asarray(idx, np.int32)
    # the last items in scheduling order are the last query blocks of the last head
    ids = np.array(sorted({rows - 1, rows - 2, rows - 3, rows - nQb // 4, rows - nQb // 3, 0, 1,
                           nQb - 1, rows // 2}), dtype=np.int32)
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)

    def gather(o):
        out = np.zeros((len(ids), BLK, D))
        oh = o.float().cpu().numpy().reshape(B * H, N, D)
        for n, r in enumerate(ids):
            bh, i = divmod(int(r), nQb)
            blk = oh[bh, i * BLK:min((i + 1) * BLK, N)]
            out[n, :blk.shape[0]] = blk
        return out

    ref_s = orc.sparse_attn(qn, kn, vn, BLK, BLK, off, idx, row_ids=ids)
    doff, didx = util.all_blocks_csr(rows, nKb)
    ref_d = orc.sparse_attn(qn, kn, vn, BLK, BLK, doff, didx, row_ids=ids)
    for dt in (torch.float32, torch.bfloat16):
        tol = util.MAX_ABS_TOL if dt == torch.float32 else util.MAX_ABS_TOL + 2.0 ** -7
        o = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(),
                                  BLK, BLK, out_dtype=dt)
        assert losa.losa_async_status() == 0
        d = np.abs(gather(o) - ref_s)
        assert d.max() <= tol and d.mean() <= util.MEAN_ABS_TOL, (dt, d.max(), d.mean())
        o = losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=dt)
        assert losa.losa_async_status() == 0
        d = np.abs(gather(o) - ref_d)
        assert d.max() <= tol and d.mean() <= util.MEAN_ABS_TOL, (dt, d.max(), d.mean())


# (B, H, N, D, R, C): query blocks of 128 rows with finer key blocks (the paper's own geometry is
# R = 128, C = 32): 128 / C key blocks are gathered into one 128-key tile; N is chosen so that the
# number of key blocks is not a multiple of 128 / C and the last block is ragged
GEOMETRIES = [
    (1, 2, 128 * 3 + 45, 128, 128, 32),
    (1, 3, 128 * 5 - 19, 64, 128, 32),
    (2, 1, 128 * 4 + 70, 128, 128, 64),
    (1, 2, 128 * 2 + 33, 64, 128, 64),
    (1, 1, 32 * 3, 128, 128, 32),
]


@pytest.mark.parametrize("shape", GEOMETRIES)
def test_rectangular_blocks_match_oracle(shape):
    """R != C: dense and sparse attention, block mass, the fused pass and the selection chain."""
    losa = lib()
    B, H, N, D, R, C = shape
    q, k, v = make(B, H, N, D, 131, 1.5)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    nQb, nKb = -(-N // R), -(-N // C)
    rows = B * H * nQb

    # dense
    o = losa.losa_attn(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o, orc.dense_attn(qn, kn, vn), f"dense {shape}")

    # block mass (Eq. 1) with rectangular blocks, and the fused pass
    mass, lse = losa.losa_block_mass(qd, kd, R, C, return_lse=True)
    assert losa.losa_async_status() == 0
    ref, ref_lse = orc.block_mass(qn, kn, R, C, return_lse=True)
    got = mass.cpu().numpy().reshape(ref.shape).astype(np.float64)
    assert got.shape == (rows, nKb)
    assert np.abs(got - ref).max() <= util.MASS_TOL
    assert np.abs(got.sum(1) - 1.0).max() <= util.MASS_TOL
    assert np.abs(lse.cpu().numpy() - ref_lse.reshape(B, H, nQb * R)[:, :, :N]).max() <= 1e-3
    o_f, mass_f = losa.losa_attn_mass(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o_f, orc.dense_attn(qn, kn, vn), f"fused o {shape}")
    assert np.abs(mass_f.cpu().numpy().reshape(ref.shape) - ref).max() <= util.MASS_TOL

    # selection on the GPU masses, bit-exact against the oracle's rule on the same masses
    off, idx = losa.losa_select(mass, 0.9)
    assert losa.losa_async_status() == 0
    sel = orc.select(mass.cpu().numpy().reshape(rows, nKb).astype(np.float64), 0.9)
    bad, _ = util.compare_csr(off.cpu().numpy(), idx.cpu().numpy(), sel)
    assert not bad

    # sparse attention over that pattern and over random patterns (uneven lists)
    for name, (o_h, i_h) in {
        "selected": (off.cpu().numpy(), idx.cpu().numpy()[: int(off[-1])]),
        "random 0.2": util.random_csr(rows, nKb, 7 + N, 0.2),
        "random 0.7": util.random_csr(rows, nKb, 9 + N, 0.7),
    }.items():
        o_s = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(np.ascontiguousarray(o_h)).cuda(),
                                    torch.from_numpy(np.ascontiguousarray(i_h)).cuda(), R, C,
                                    out_dtype=torch.float32)
        assert losa.losa_async_status() == 0
        ref_o = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, R, C, o_h.astype(np.int32),
                                                     i_h.astype(np.int32)), B, H, N)
        util.assert_output_close(o_s, ref_o, f"sparse {name} {shape}")


@pytest.mark.parametrize("D,BLK", [(128, 128), (64, 64), (64, 128)])
@pytest.mark.parametrize("jump", [6.0, 35.0, 110.0])
def test_scores_that_jump_far_above_the_first_tiles(D, BLK, jump):
    """The attention kernels exponentiate against a reference that only moves when a tile's row sums
    leave the safe range.  Scores that rise by `jump` nats after the first key tiles (p would reach
    2^(jump * 1.44): within range, beyond 2^40, beyond fp32) must give the exact softmax all the
    same, for dense and sparse attention and for the fused pass."""
    losa = lib()
    B, H, N = 1, 2, 128 * 5 + 40
    g = torch.Generator("cpu").manual_seed(5)
    q = torch.randn(B, H, N, D, generator=g) * 0.3 + 1.0   # q . ones(D) is about D
    k = torch.randn(B, H, N, D, generator=g) * 0.3
    # keys from 256 on: an added component along ones(D) that lifts q.k / sqrt(D) by about `jump`,
    # rising in two steps (at 256 and at 448) so that the reference has to move more than once
    lift = jump * (D ** 0.5) / D
    k[:, :, 256:] += 0.5 * lift
    k[:, :, 448:] += 0.5 * lift
    v = torch.randn(B, H, N, D, generator=g)
    q, k, v = q.bfloat16(), k.bfloat16(), v.bfloat16()
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    ref = orc.dense_attn(qn, kn, vn)
    o = losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    assert torch.isfinite(o).all()
    util.assert_output_close(o, ref, f"dense jump {jump}")
    o_f, mass = losa.losa_attn_mass(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o_f, ref, f"fused jump {jump}")
    ref_m = orc.block_mass(qn, kn, BLK, BLK)
    assert np.abs(mass.cpu().numpy().reshape(ref_m.shape) - ref_m).max() <= util.MASS_TOL
    nb = -(-N // BLK)
    off, idx = util.random_csr(B * H * nb, nb, 3, 0.6)
    o_s = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(),
                                BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    ref_s = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, BLK, BLK, off, idx), B, H, N)
    util.assert_output_close(o_s, ref_s, f"sparse jump {jump}")


@pytest.mark.parametrize("R,C", [(64, 64), (128, 128), (128, 64), (128, 32)])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("scale", [2.0, 4.0])
def test_sharp_scores_stay_within_the_stated_tolerance(R, C, D, scale):
    """q, k ~ N(0, scale^2): the scores have a standard deviation of scale^2 nats (4 and 16), so
    most rows are dominated by one or two keys.  That is where rounding P to bf16 shows most: the
    output is a weighted mean of V with weights off by up to 2^-8 each, and it stays inside the
    tolerance only because it is normalised by the sum of the ROUNDED weights (a row that a single
    key dominates is then exact).  Dense, sparse and fused forward at the stated 1e-2 / 1e-3."""
    losa = lib()
    B, H, N = 2, 3, 128 * 7 + 77
    q, k, v = make(B, H, N, D, 211 + int(scale), scale)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    nQb, nKb = -(-N // R), -(-N // C)
    dense = orc.dense_attn(qn, kn, vn)
    o = losa.losa_attn(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o, dense, f"dense scale {scale}")
    o_f, mass = losa.losa_attn_mass(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o_f, dense, f"fused scale {scale}")
    ref_m = orc.block_mass(qn, kn, R, C)
    assert np.abs(mass.cpu().numpy().reshape(ref_m.shape) - ref_m).max() <= util.MASS_TOL
    off, idx = util.random_csr(B * H * nQb, nKb, 17 + D, 0.5)
    o_s = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(),
                                R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    ref_s = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, R, C, off, idx), B, H, N)
    util.assert_output_close(o_s, ref_s, f"sparse scale {scale}")


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("col", [2, 3, 19, 5])
def test_block_mass_with_one_key_far_above_the_reference(D, col):
    """The mass pass with 128-key blocks exponentiates against a reference that moves only when a
    tile's row sums leave the safe range, and computes the exponentials of columns 2 and 3 (mod 16)
    with a polynomial.  One key 100 nats above everything else, in a later tile, at such a column
    (and at an ordinary one): its block must get mass ~1, exactly as the oracle says."""
    losa = lib()
    B, H, N, BLK = 1, 2, 128 * 4 + 50, 128
    g = torch.Generator("cpu").manual_seed(9 + col)
    q = torch.randn(B, H, N, D, generator=g) * 0.3 + 1.0
    k = torch.randn(B, H, N, D, generator=g) * 0.3
    v = torch.randn(B, H, N, D, generator=g)
    k[:, :, 2 * 128 + col] += 100.0 * (D ** 0.5) / D  # q . k / sqrt(D) rises by about 100
    q, k, v = q.bfloat16(), k.bfloat16(), v.bfloat16()
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    ref = orc.block_mass(qn, kn, BLK, BLK)
    assert ref[:, 2].min() > 0.999
    mass = losa.losa_block_mass(q.cuda(), k.cuda(), BLK, BLK)
    assert losa.losa_async_status() == 0
    got = mass.cpu().numpy().reshape(ref.shape).astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= util.MASS_TOL
    o_f, mass_f = losa.losa_attn_mass(q.cuda(), k.cuda(), v.cuda(), BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    assert np.abs(mass_f.cpu().numpy().reshape(ref.shape) - ref).max() <= util.MASS_TOL
    util.assert_output_close(o_f, orc.dense_attn(qn, kn, vn), "fused o with an outlier key")


@pytest.mark.parametrize("D,BLK", [(128, 128), (64, 64)])
def test_rows_that_outgrow_their_reference_in_whole_and_cut_work_units(D, BLK):
    """The forward keeps, per work unit, the reference of the unit's first tile; a unit whose scores
    rise far above it is handed to a second launch that moves the reference.  More work items than
    SMs, so that some units are whole items and the last ones are parts; half of the heads carry
    keys 60 nats above the rest from the third tile on, the other half do not (their units must
    not be touched by the second launch: compared with the oracle all the same)."""
    losa = lib()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    B, N = 1, 128 * 7 + 50
    H = sms // 4 + 6                       # 4 pairs of query tiles per head: more items than SMs
    assert H * 4 > sms
    g = torch.Generator("cpu").manual_seed(77)
    q = torch.randn(B, H, N, D, generator=g) * 0.3 + 1.0
    k = torch.randn(B, H, N, D, generator=g) * 0.3
    k[:, ::2, 300:] += 60.0 * (D ** 0.5) / D
    v = torch.randn(B, H, N, D, generator=g)
    q, k, v = q.bfloat16(), k.bfloat16(), v.bfloat16()
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    o = losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o, orc.dense_attn(qn, kn, vn), "dense, some heads outgrow the reference")
    nb = -(-N // BLK)
    off, idx = util.random_csr(B * H * nb, nb, 9, 0.7)
    o_s = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(),
                                BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    ref_s = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, BLK, BLK, off, idx), B, H, N)
    util.assert_output_close(o_s, ref_s, "sparse, some heads outgrow the reference")
    o_f, mass = losa.losa_attn_mass(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    util.assert_output_close(o_f, orc.dense_attn(qn, kn, vn), "fused, some heads outgrow the reference")
    ref_m = orc.block_mass(qn, kn, BLK, BLK)
    assert np.abs(mass.cpu().numpy().reshape(ref_m.shape) - ref_m).max() <= util.MASS_TOL
