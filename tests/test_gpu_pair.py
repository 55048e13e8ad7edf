"""The forward at head dimension 128 with 128-row query blocks runs on pairs of CTAs, one query tile
of a work item per CTA, both multiplying every key tile of the union of the two tiles' lists.
Patterns built to reach what that design adds: key tiles that only one of the two query tiles lists
(the other CTA must contribute nothing), a first listed tile that falls on either of the two
alternating softmax groups (the row reference is handed from one group to the other), query tiles
whose only key tile comes last, an odd number of query tiles, and launches with whole and cut
work units.  All against the fp64 oracle (Eq. 4)."""
import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu

D, R = 128, 128


def lib():
    import paper_2608_12032_b200 as losa
    return losa


def csr_from(lists):
    offs, idx = [0], []
    for row in lists:
        row = sorted(set(int(j) for j in row))
        assert row, "every query block keeps at least one key block (Eq. 3 with tau > 0)"
        idx.extend(row)
        offs.append(len(idx))
    return np.asarray(offs, np.int32), np.asarray(idx, np.int32)


def patterns(nQb, nKb, kind, seed):
    rng = np.random.default_rng(seed)
    rows = []
    for g in range(nQb):
        if kind == "disjoint_singletons":
            # consecutive query blocks never share a key block: every key tile has one taker
            rows.append([(2 * g + (g % 2) * 3) % nKb] if nKb > 1 else [0])
        elif kind == "late_only_tile":
            # the even query tile lists everything, the odd one only a block near the end, so its
            # first (and only) tile is met late, by the group that the position's parity selects
            rows.append(range(nKb) if g % 2 == 0 else [nKb - 1 - (g // 2) % 2])
        elif kind == "odd_position_first":
            # the odd query tile lists a few early blocks, the even one starts later
            rows.append(range(min(3, nKb)) if g % 2 == 1 else range(min(1 + (g // 2) % 2, nKb - 1), nKb))
        elif kind == "interleaved":
            rows.append([j for j in range(nKb) if (j + g) % 2 == 0] or [0])
        else:
            keep = np.nonzero(rng.random(nKb) < 0.4)[0]
            rows.append(keep if keep.size else [int(rng.integers(nKb))])
    return rows


@pytest.mark.parametrize("C", [128, 64, 32])
@pytest.mark.parametrize("kind", ["disjoint_singletons", "late_only_tile", "odd_position_first", "interleaved", "random"])
@pytest.mark.parametrize("tiles", [6, 7])
def test_crafted_patterns_match_oracle(C, kind, tiles):
    losa = lib()
    B, H = 1, 2
    N = 128 * tiles - 37  # a ragged last query tile and key block; 7 tiles: the last pair has one tile
    nQb, nKb = -(-N // R), -(-N // C)
    q = util.rand_bf16((B, H, N, D), 900 + tiles, 2.0)
    k = util.rand_bf16((B, H, N, D), 901 + tiles, 2.0)
    v = util.rand_bf16((B, H, N, D), 902 + tiles)
    lists = []
    for bh in range(B * H):
        lists += patterns(nQb, nKb, kind, 17 + bh)
    off, idx = csr_from(lists)
    o = losa.losa_sparse_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(off).cuda(),
                              torch.from_numpy(idx).cuda(), R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    ref = orc.blocks_to_tokens(
        orc.sparse_attn(util.to_np(q), util.to_np(k), util.to_np(v), R, C, off, idx), B, H, N)
    util.assert_output_close(o, ref, f"{kind} C={C} tiles={tiles}")


@pytest.mark.parametrize("C", [128, 64, 32])
def test_whole_and_cut_work_units_in_one_launch(C):
    """More work items than pairs of CTAs fit at once, and not a multiple of them: the first waves
    run whole items, the last one is cut into parts and merged."""
    losa = lib()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    slots = min(sms, 160) // 2
    tiles = 4                              # two work items per head
    H = slots // 2 + 3                     # slots + 6 items: one whole wave, six items cut
    B, N = 1, 128 * tiles - 50
    nQb, nKb = -(-N // R), -(-N // C)
    q = util.rand_bf16((B, H, N, D), 1000, 1.5)
    k = util.rand_bf16((B, H, N, D), 1001, 1.5)
    v = util.rand_bf16((B, H, N, D), 1002)
    off, idx = util.random_csr(B * H * nQb, nKb, 5, 0.6)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    o = losa.losa_sparse_attn(qd, kd, vd, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda(), R, C,
                              out_dtype=torch.float32)
    od = losa.losa_attn(qd, kd, vd, R, C, out_dtype=torch.float32)
    assert losa.losa_async_status() == 0
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    ref = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, R, C, off, idx), B, H, N)
    util.assert_output_close(o, ref, f"sparse C={C}")
    a_off, a_idx = util.all_blocks_csr(B * H * nQb, nKb)
    ref_d = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, R, C, a_off, a_idx), B, H, N)
    util.assert_output_close(od, ref_d, f"dense C={C}")


def test_same_call_twice_gives_the_same_bits():
    losa = lib()
    B, H, N, C = 1, 5, 128 * 9 + 11, 128
    nQb, nKb = -(-N // R), -(-N // C)
    q, k, v = (util.rand_bf16((B, H, N, D), 1100 + i, 1.5).cuda() for i in range(3))
    off, idx = util.random_csr(B * H * nQb, nKb, 9, 0.5)
    offd, idxd = torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda()
    first = losa.losa_sparse_attn(q, k, v, offd, idxd, R, C, out_dtype=torch.float32)
    for _ in range(5):
        again = losa.losa_sparse_attn(q, k, v, offd, idxd, R, C, out_dtype=torch.float32)
        assert torch.equal(first, again)
    assert losa.losa_async_status() == 0


@pytest.mark.parametrize("Dh,Rq,Ck", [(128, 128, 128), (64, 64, 64)])
def test_two_streams_with_their_own_workspaces_do_not_disturb_each_other(Dh, Rq, Ck):
    """Calls on different streams may overlap on the GPU when each has its own workspace and output
    (the header's rule): persistent kernels of two launches then share the SMs.  Each stream's results
    must equal, bit for bit, what the same calls give alone."""
    losa = lib()
    B, H, N = 1, 6, 128 * 11 + 40
    nQb, nKb = -(-N // Rq), -(-N // Ck)
    data = []
    for i in range(2):
        q, k, v = (util.rand_bf16((B, H, N, Dh), 1200 + 10 * i + j, 1.5).cuda() for j in range(3))
        off, idx = util.random_csr(B * H * nQb, nKb, 40 + i, 0.5)
        data.append((q, k, v, torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda()))
    alone = []
    for q, k, v, off, idx in data:
        alone.append((losa.losa_sparse_attn(q, k, v, off, idx, Rq, Ck, out_dtype=torch.float32),
                      losa.losa_attn(q, k, v, Rq, Ck, out_dtype=torch.float32)))
    torch.cuda.synchronize()
    assert losa.losa_async_status() == 0
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    results = [[], []]
    for rep in range(4):
        for i, (q, k, v, off, idx) in enumerate(data):
            with torch.cuda.stream(streams[i]):
                results[i].append((losa.losa_sparse_attn(q, k, v, off, idx, Rq, Ck, out_dtype=torch.float32),
                                   losa.losa_attn(q, k, v, Rq, Ck, out_dtype=torch.float32)))
    torch.cuda.synchronize()
    assert losa.losa_async_status() == 0
    for i in range(2):
        for o_s, o_d in results[i]:
            assert torch.equal(o_s, alone[i][0]) and torch.equal(o_d, alone[i][1])
