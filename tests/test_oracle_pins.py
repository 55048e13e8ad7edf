"""Pins for the fp64 CPU oracle: closed forms, brute force, library special cases.

None of these tests calls the CUDA path.  Each checks the oracle against
something other than itself: the paper's definitions written out on a
materialised attention matrix (numpy, inside this file), torch's fp64
attention, closed-form inputs, and subset enumeration.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked.txt")


def bf16_exact(shape, seed, scale=1.0):
    g = torch.Generator("cpu").manual_seed(seed)
    x = torch.randn(shape, generator=g) * scale
    return x.bfloat16().float().numpy()


def dense_probs(q, k, scale):
    """Materialised A = softmax(Q K^T * scale) in fp64 (the definition, numpy)."""
    s = np.einsum("bhqd,bhkd->bhqk", q.astype(np.float64), k.astype(np.float64)) * scale
    s -= s.max(-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(-1, keepdims=True)


def brute_mass(A, R, C):
    B, H, N, _ = A.shape
    nQb, nKb = -(-N // R), -(-N // C)
    out = np.zeros((B, H, nQb, nKb))
    for i in range(nQb):
        rows = slice(i * R, min((i + 1) * R, N))
        nv = rows.stop - rows.start
        for j in range(nKb):
            cols = slice(j * C, min((j + 1) * C, N))
            out[:, :, i, j] = A[:, :, rows, cols].sum((-1, -2)) / nv
    return out.reshape(B * H * nQb, nKb)


# ---------------------------------------------------------------- dense attention

@pytest.mark.parametrize("N,D", [(37, 8), (200, 64)])
def test_dense_matches_torch_sdpa_fp64(N, D):
    q, k, v = (bf16_exact((2, 3, N, D), s) for s in (1, 2, 3))
    o = orc.dense_attn(q, k, v)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).double(), torch.from_numpy(k).double(), torch.from_numpy(v).double()
    ).numpy()
    assert np.abs(o - ref).max() < 1e-12


def test_dense_uniform_when_keys_zero():
    q, v = bf16_exact((1, 1, 50, 16), 4), bf16_exact((1, 1, 50, 16), 5)
    k = np.zeros_like(q)
    o = orc.dense_attn(q, k, v)
    assert np.abs(o - v.astype(np.float64).mean(2, keepdims=True)).max() < 1e-13


# ---------------------------------------------------------------------- block mass

@pytest.mark.parametrize("N,R,C", [(256, 64, 64), (200, 64, 64), (130, 32, 16), (97, 128, 32)])
def test_mass_matches_materialised_definition(N, R, C):
    q, k = bf16_exact((1, 2, N, 32), 10), bf16_exact((1, 2, N, 32), 11)
    scale = 1.0 / math.sqrt(32)
    mass, lse = orc.block_mass(q, k, R, C, return_lse=True)
    A = dense_probs(q, k, scale)
    assert np.abs(mass - brute_mass(A, R, C)).max() < 1e-13
    # every query block's masses sum to one (each row of A sums to one)
    assert np.abs(mass.sum(1) - 1.0).max() < 1e-13
    # log-sum-exp against the definition
    s = np.einsum("bhqd,bhkd->bhqk", q.astype(np.float64), k.astype(np.float64)) * scale
    ref_lse = np.log(np.exp(s - s.max(-1, keepdims=True)).sum(-1)) + s.max(-1)
    nQb = -(-N // R)
    padded = np.zeros((1, 2, nQb * R))
    padded[:, :, :N] = ref_lse
    assert np.abs(lse - padded.reshape(2 * nQb, R)).max() < 1e-12


def test_mass_uniform_attention_closed_form_with_ragged_tail():
    # K = 0  =>  A(q,k) = 1/N  =>  mass(i,j) = |B^K_j| / N, short last block included
    N, R, C = 150, 64, 64
    q = bf16_exact((1, 1, N, 16), 20)
    k = np.zeros_like(q)
    mass = orc.block_mass(q, k, R, C)
    expect = np.array([64, 64, 22], dtype=np.float64) / N
    assert mass.shape == (3, 3)
    assert np.abs(mass - expect[None, :]).max() < 1e-15


def test_mass_block_one_hot_closed_form():
    # Q = K = lam * e_block(token): scores are lam^2*scale inside the own block, 0 elsewhere.
    nB, Cb, D, lam = 4, 16, 8, 4.0
    N = nB * Cb
    x = np.zeros((1, 1, N, D), dtype=np.float32)
    for n in range(N):
        x[0, 0, n, n // Cb] = lam
    scale = 1.0 / math.sqrt(D)
    mass = orc.block_mass(x, x, Cb, Cb, scale=scale)
    a = lam * lam * scale
    diag = Cb * math.exp(a) / (Cb * math.exp(a) + N - Cb)
    off = Cb / (Cb * math.exp(a) + N - Cb)
    expect = np.full((nB, nB), off)
    np.fill_diagonal(expect, diag)
    assert np.abs(mass - expect).max() < 1e-14


def test_mass_key_block_permutation_equivariance():
    N, R, C = 128, 32, 32
    q, k = bf16_exact((1, 1, N, 16), 30), bf16_exact((1, 1, N, 16), 31)
    perm = np.array([2, 0, 3, 1])
    kp = k.reshape(1, 1, 4, C, 16)[:, :, perm].reshape(1, 1, N, 16)
    m0 = orc.block_mass(q, k, R, C)
    m1 = orc.block_mass(q, kp, R, C)
    assert np.abs(m1 - m0[:, perm]).max() < 1e-14


def test_mass_row_subset_matches_full():
    q, k = bf16_exact((1, 3, 200, 16), 40), bf16_exact((1, 3, 200, 16), 41)
    full = orc.block_mass(q, k, 64, 64)
    ids = [11, 0, 5, 7]
    sub = orc.block_mass(q, k, 64, 64, row_ids=ids)
    assert np.array_equal(sub, full[ids])


# ----------------------------------------------------------------------- selection

def random_mass(rows, nKb, seed, tail=3.0):
    rng = np.random.default_rng(seed)
    m = np.exp(tail * rng.standard_normal((rows, nKb)))
    return m / m.sum(1, keepdims=True)


@pytest.mark.parametrize("tau", [0.5, 0.9, 0.99])
def test_select_is_minimal_prefix(tau):
    m = random_mass(64, 37, 1)
    sel = orc.select(m, tau)
    for r in range(m.shape[0]):
        s = sel.count[r]
        kept = sel.kept[r, :s]
        assert np.all(np.diff(kept) > 0) and np.all(sel.kept[r, s:] == -1)
        assert set(kept) == set(sel.order[r, :s])
        assert m[r, kept].sum() >= tau - 1e-15
        # dropping the smallest kept block falls below tau
        if s > 1:
            assert m[r, kept].sum() - m[r, kept].min() < tau
        # order really is by decreasing mass
        assert np.all(np.diff(m[r, sel.order[r]]) <= 0)


@pytest.mark.parametrize("nKb", [1, 2, 5, 9, 12])
def test_select_brute_force_subsets(nKb):
    m = random_mass(6, nKb, 100 + nKb, tail=1.5)
    for tau in (0.3, 0.6, 0.9, 0.97):
        sel = orc.select(m, tau)
        for r in range(m.shape[0]):
            s = int(sel.count[r])
            best_smaller = 0.0
            for size in range(1, s):
                best_smaller = max(
                    best_smaller, max(m[r, list(c)].sum() for c in itertools.combinations(range(nKb), size))
                )
            assert best_smaller < tau  # no smaller subset reaches tau
            best_same = max(m[r, list(c)].sum() for c in itertools.combinations(range(nKb), s))
            got = m[r, sel.kept[r, :s]].sum()
            assert got >= tau - 1e-15 or s == nKb
            assert abs(got - best_same) < 1e-15  # the prefix is the heaviest set of its size


def test_select_uniform_masses_lower_index_first():
    nKb = 10
    m = np.full((3, nKb), 1.0 / nKb)
    sel = orc.select(m, 0.75)  # 0.75 is away from multiples of 0.1
    assert np.all(sel.count == 8)
    assert np.array_equal(sel.kept[:, :8], np.tile(np.arange(8), (3, 1)))
    assert np.array_equal(sel.order, np.tile(np.arange(nKb), (3, 1)))


def test_select_ties_broken_by_lower_index():
    m = np.array([[0.1, 0.3, 0.3, 0.1, 0.2]])
    sel = orc.select(m, 0.55)
    assert list(sel.order[0]) == [1, 2, 4, 0, 3]
    assert sel.count[0] == 2 and list(sel.kept[0, :2]) == [1, 2]
    sel = orc.select(m, 0.85)  # 0.3+0.3+0.2 = 0.8 < 0.85 -> needs block 0 (tie with 3)
    assert sel.count[0] == 4 and list(sel.kept[0, :4]) == [0, 1, 2, 4]


def test_select_threshold_is_inclusive():
    """Eq. 3 keeps the shortest prefix whose mass is >= tau: a prefix that lands exactly on tau
    already suffices.  Masses and thresholds are exactly representable, so equality is exact."""
    m = np.array([[0.5, 0.25, 0.25], [0.25, 0.25, 0.5], [0.125, 0.5, 0.375]])
    sel = orc.select(m, 0.75)
    # row 0: 0.5 + 0.25 == 0.75 -> two blocks, the tie goes to the lower index
    assert sel.count[0] == 2 and list(sel.kept[0, :2]) == [0, 1]
    # row 1: order (2, 0, 1) with the tie by index; 0.5 + 0.25 == 0.75 -> {0, 2}
    assert list(sel.order[1]) == [2, 0, 1]
    assert sel.count[1] == 2 and list(sel.kept[1, :2]) == [0, 2]
    # row 2: 0.5 + 0.375 = 0.875 >= 0.75 -> {1, 2}
    assert sel.count[2] == 2 and list(sel.kept[2, :2]) == [1, 2]
    assert np.all(sel.cum[:2, 1] == 0.75)
    # a single block that equals tau suffices; one ulp more does not
    sel = orc.select(np.array([[0.5, 0.25, 0.25]]), 0.5)
    assert sel.count[0] == 1 and sel.kept[0, 0] == 0
    sel = orc.select(np.array([[0.5, 0.25, 0.25]]), np.nextafter(0.5, 1.0))
    assert sel.count[0] == 2
    # uniform masses on a multiple of 1/nKb: 8 * 0.125 == 1.0 exactly, 6 * 0.125 == 0.75
    sel = orc.select(np.full((1, 8), 0.125), 0.75)
    assert sel.count[0] == 6 and list(sel.kept[0, :6]) == list(range(6))


def test_select_one_hot_and_tau_one():
    m = np.zeros((2, 7))
    m[0, 4] = 1.0
    m[1, 0] = 1.0
    sel = orc.select(m, 0.99)
    assert list(sel.count) == [1, 1] and sel.kept[0, 0] == 4 and sel.kept[1, 0] == 0
    m = random_mass(5, 9, 3)
    sel = orc.select(m, 1.0)
    assert np.all(sel.count == 9)
    assert np.array_equal(sel.kept, np.tile(np.arange(9), (5, 1)))


def test_select_monotone_in_tau_and_recall():
    m = random_mass(40, 50, 7)
    prev = None
    for tau in (0.5, 0.8, 0.9, 0.99, 0.999):
        sel = orc.select(m, tau)
        cur = [set(sel.kept[r, : sel.count[r]]) for r in range(m.shape[0])]
        if prev is not None:
            assert all(a <= b for a, b in zip(prev, cur))
        prev = cur
        # retained mass reaches tau in every row, hence overall (the guarantee at t0)
        assert orc.recall(m, sel.offsets, sel.kv_idx) >= tau - 1e-12
        assert 0 < orc.coverage(sel.offsets, 50) <= 1


def test_select_against_numpy_argsort_cumsum():
    m = random_mass(30, 64, 9)
    tau = 0.95
    sel = orc.select(m, tau)
    order = np.argsort(-m, axis=1, kind="stable")
    cum = np.cumsum(np.take_along_axis(m, order, 1), axis=1)
    s = (cum >= tau).argmax(1) + 1
    assert np.array_equal(sel.order, order)
    assert np.array_equal(sel.count, s)
    assert np.abs(sel.cum - cum).max() < 1e-15


def test_topk_against_numpy_and_heaviest_subset():
    m = random_mass(12, 11, 21, tail=1.5)
    m[3, 2] = m[3, 7]  # a tie: the lower index wins when only one of the two fits
    for k in (1, 4, 11):
        off, idx = orc.select_topk(m, k)
        assert list(off) == [r * k for r in range(13)]
        order = np.argsort(-m, axis=1, kind="stable")[:, :k]
        assert np.array_equal(idx.reshape(12, k), np.sort(order, axis=1))
        for r in range(12):
            best = max(m[r, list(c)].sum() for c in itertools.combinations(range(11), k))
            assert abs(m[r, idx.reshape(12, k)[r]].sum() - best) < 1e-15
    with pytest.raises(RuntimeError):
        orc.select_topk(m, 0)


def test_row_recall_against_the_definition():
    m = random_mass(20, 17, 22)
    sel = orc.select(m, 0.9)
    ret, tot = orc.row_recall(m, sel.offsets, sel.kv_idx)
    for r in range(20):
        kept = sel.kept[r, : sel.count[r]]
        assert abs(ret[r] - m[r, kept].sum()) < 1e-15 and abs(tot[r] - m[r].sum()) < 1e-15
    assert abs(ret.sum() / tot.sum() - orc.recall(m, sel.offsets, sel.kv_idx)) < 1e-15
    assert np.all(ret >= 0.9 - 1e-12)  # the guarantee of Eq. 3 at the construction step


def test_select_rejects_bad_tau():
    with pytest.raises(RuntimeError):
        orc.select(np.ones((1, 2)) / 2, 0.0)


# ---------------------------------------------------------------- sparse attention

def all_blocks_csr(rows, nKb):
    off = np.arange(rows + 1, dtype=np.int32) * nKb
    idx = np.tile(np.arange(nKb, dtype=np.int32), rows)
    return off, idx


@pytest.mark.parametrize("N,R,C", [(200, 64, 64), (96, 32, 16)])
def test_sparse_with_all_blocks_is_dense(N, R, C):
    q, k, v = (bf16_exact((1, 2, N, 16), s) for s in (50, 51, 52))
    nQb, nKb = -(-N // R), -(-N // C)
    off, idx = all_blocks_csr(2 * nQb, nKb)
    o = orc.blocks_to_tokens(orc.sparse_attn(q, k, v, R, C, off, idx), 1, 2, N)
    assert np.abs(o - orc.dense_attn(q, k, v)).max() < 1e-14


def test_sparse_matches_masked_sdpa_and_renormalisation_identity():
    N, R, C, D = 200, 64, 32, 16
    q, k, v = (bf16_exact((1, 2, N, D), s, 1.5) for s in (60, 61, 62))
    scale = 1.0 / math.sqrt(D)
    nQb, nKb = -(-N // R), -(-N // C)
    mass = orc.block_mass(q, k, R, C)
    sel = orc.select(mass, 0.8)
    assert sel.count.min() < nKb  # the pattern really is sparse
    o = orc.blocks_to_tokens(orc.sparse_attn(q, k, v, R, C, sel.offsets, sel.kv_idx), 1, 2, N)
    # boolean token mask expanded from the block indices
    mask = np.zeros((1, 2, N, N), dtype=bool)
    for r in range(2 * nQb):
        h, i = divmod(r, nQb)
        for j in sel.kept[r, : sel.count[r]]:
            mask[0, h, i * R : (i + 1) * R, j * C : (j + 1) * C] = True
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).double(), torch.from_numpy(k).double(), torch.from_numpy(v).double(),
        attn_mask=torch.from_numpy(mask),
    ).numpy()
    assert np.abs(o - ref).max() < 1e-12
    # Eq. 4 is the dense row restricted to the kept keys and renormalised by its kept mass rho
    A = dense_probs(q, k, scale)
    rho = (A * mask).sum(-1, keepdims=True)
    ident = np.einsum("bhqk,bhkd->bhqd", A * mask, v.astype(np.float64)) / rho
    assert np.abs(o - ident).max() < 1e-12
    dense = orc.dense_attn(q, k, v)
    bound = 2 * (1 - rho) * np.abs(v).max()
    assert np.all(np.abs(o - dense) <= bound + 1e-12)


def test_sparse_constant_values_and_single_block():
    N, R, C, D = 128, 32, 32, 8
    q, k = bf16_exact((1, 1, N, D), 70), bf16_exact((1, 1, N, D), 71)
    v = np.full((1, 1, N, D), 0.75, dtype=np.float32)
    off = np.array([0, 1, 3, 4, 6], dtype=np.int32)
    idx = np.array([3, 0, 2, 1, 0, 3], dtype=np.int32)
    o = orc.sparse_attn(q, k, v, R, C, off, idx)
    assert np.abs(o - 0.75).max() < 1e-15
    # single kept block: plain attention of query block i on key block j alone
    v = bf16_exact((1, 1, N, D), 72)
    o = orc.sparse_attn(q, k, v, R, C, off, idx, row_ids=[0, 2])
    for slot, (i, j) in enumerate([(0, 3), (2, 1)]):
        sub = orc.dense_attn(
            q[:, :, i * R : (i + 1) * R], k[:, :, j * C : (j + 1) * C], v[:, :, j * C : (j + 1) * C]
        )
        assert np.abs(o[slot] - sub[0, 0]).max() < 1e-14


def test_sparse_rejects_empty_row():
    q = bf16_exact((1, 1, 32, 8), 80)
    with pytest.raises(RuntimeError):
        orc.sparse_attn(q, q, q, 16, 16, np.array([0, 0, 1], np.int32), np.array([0], np.int32))


# ------------------------------------------------------------- hand-worked fixture

def read_golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = [float(x) for x in vals]
    return out


def test_hand_worked_example():
    g = read_golden()
    q = np.ones((1, 1, 4, 1), dtype=np.float32)
    k = np.log(np.arange(1, 5, dtype=np.float64)).astype(np.float32).reshape(1, 1, 4, 1)
    v = np.array([10, 20, 30, 40], dtype=np.float32).reshape(1, 1, 4, 1)
    mass = orc.block_mass(q, k, 1, 1, scale=1.0)
    assert np.abs(mass - np.array(g["mass"])[None, :]).max() < 1e-6
    sel = orc.select(mass, g["tau"][0])
    assert list(sel.order[0]) == g["order"] and sel.count[0] == g["count"][0]
    assert list(sel.kept[0, :2]) == g["kept"]
    assert orc.select(mass, g["tau2"][0]).count[0] == g["count2"][0]
    o = orc.sparse_attn(q, k, v, 1, 1, sel.offsets, sel.kv_idx, scale=1.0)
    assert np.abs(o - g["sparse_o"][0]).max() < 1e-5
    assert np.abs(orc.dense_attn(q, k, v, scale=1.0) - g["dense_o"][0]).max() < 1e-5
