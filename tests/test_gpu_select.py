"""losa_select and losa_validate_csr on the GPU against the oracle's Eq. 3, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu


def lib():
    import paper_2608_12032_b200 as losa
    return losa


def random_mass(rows, nKb, seed, tail=3.0):
    rng = np.random.default_rng(seed)
    m = np.exp(tail * rng.standard_normal((rows, nKb)))
    return (m / m.sum(1, keepdims=True)).astype(np.float32)


def run_select(m32, tau, B=1, H=1, **kw):
    losa = lib()
    rows, nKb = m32.shape
    mass = torch.from_numpy(m32).cuda().reshape(B, H, rows // (B * H), nKb)
    off, idx = losa.losa_select(mass, tau, **kw)
    status = losa.losa_async_status()
    return off.cpu().numpy(), idx.cpu().numpy(), status


@pytest.mark.parametrize("rows,nKb", [(8, 1), (8, 4), (64, 31), (64, 32), (64, 33), (96, 256),
                                      (40, 278), (24, 929), (6, 1500), (3, 5000)])
@pytest.mark.parametrize("tau", [0.5, 0.99, 1.0])
def test_select_bit_exact_against_oracle(rows, nKb, tau):
    m32 = random_mass(rows, nKb, 1000 + nKb)
    off, idx, status = run_select(m32, tau)
    assert status == 0
    sel = orc.select(m32.astype(np.float64), tau)
    bad, exempt = util.compare_csr(off, idx, sel)
    assert not bad, f"rows {bad[:5]} differ"
    assert exempt == 0 or tau < 1.0
    assert off[0] == 0 and off[-1] == sel.count.sum()


def test_select_ties_uniform_and_zero_masses():
    nKb = 10
    m = np.full((4, nKb), 0.1, dtype=np.float32)
    off, idx, status = run_select(m, 0.75)
    sel = orc.select(m.astype(np.float64), 0.75)
    assert status == 0 and not util.compare_csr(off, idx, sel)[0]
    assert list(idx[: off[1]]) == list(range(sel.count[0]))
    m = np.array([[0.1, 0.3, 0.3, 0.1, 0.2], [0.0, 0.0, 1.0, 0.0, -0.0]], dtype=np.float32)
    for tau in (0.55, 0.85, 0.99):
        off, idx, status = run_select(m, tau)
        sel = orc.select(np.abs(m).astype(np.float64), tau)
        assert status == 0 and not util.compare_csr(off, idx, sel)[0]


@pytest.mark.parametrize("nKb", [3, 8, 64, 2048])
def test_select_threshold_is_inclusive_on_exactly_representable_masses(nKb):
    """A prefix whose mass equals tau exactly already suffices (Eq. 3: >= tau).  Masses are powers
    of two, so both sides add them without rounding; nKb = 2048 takes the sorting kernel."""
    m = np.zeros((3, nKb), dtype=np.float32)
    m[0, :3] = (0.5, 0.25, 0.25)
    m[1, :3] = (0.25, 0.25, 0.5)
    m[2, -1], m[2, 0], m[2, 1] = 0.5, 0.25, 0.25
    for tau, counts in ((0.75, (2, 2, 2)), (0.5, (1, 1, 1)), (float(np.nextafter(0.5, 1.0)), (2, 2, 2))):
        off, idx, status = run_select(m, tau)
        sel = orc.select(m.astype(np.float64), tau)
        assert status == 0
        assert tuple(sel.count) == counts
        bad, exempt = util.compare_csr(off, idx, sel)
        # exact ties with tau sit inside the near-threshold band by definition: compare them anyway
        assert util.csr_rows(off, idx[: off[-1]]) == util.csr_rows(sel.offsets, sel.kv_idx), (tau, bad, exempt)
    if nKb == 8:
        u = np.full((2, 8), 0.125, dtype=np.float32)
        off, idx, status = run_select(u, 0.75)
        assert status == 0 and list(np.diff(off)) == [6, 6] and list(idx[:6]) == list(range(6))


def test_select_is_deterministic_and_multi_head():
    m32 = random_mass(2 * 3 * 16, 70, 5)
    a = run_select(m32, 0.9, B=2, H=3)
    b = run_select(m32, 0.9, B=2, H=3)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1][: a[0][-1]], b[1][: b[0][-1]])
    sel = orc.select(m32.astype(np.float64), 0.9)
    assert not util.compare_csr(a[0], a[1], sel)[0]


def test_select_reports_capacity_overflow_without_writing_past_it():
    losa = lib()
    m32 = random_mass(16, 64, 7)
    sel = orc.select(m32.astype(np.float64), 0.99)
    nnz = int(sel.count.sum())
    cap = nnz // 2
    mass = torch.from_numpy(m32).cuda().reshape(1, 1, 16, 64)
    offsets = torch.empty(17, dtype=torch.int32, device="cuda")
    kv = torch.full((nnz,), -7, dtype=torch.int32, device="cuda")
    losa.losa_select(mass, 0.99, kv_capacity=cap, out=(offsets, kv))
    assert losa.losa_status_string(losa.losa_async_status()) == "LOSA_ERR_CAPACITY"
    assert int(offsets[-1]) == nnz  # offsets stay exact
    assert torch.all(kv[cap:] == -7)
    assert np.array_equal(kv[:cap].cpu().numpy(), sel.kv_idx[:cap])
    assert losa.losa_async_status() == 0  # the status word was cleared


def test_select_flags_negative_and_nan_mass():
    losa = lib()
    m = random_mass(4, 16, 9)
    m[1, 3] = -0.5
    m[2, 5] = np.nan
    run = run_select(m, 0.9)
    assert losa.losa_status_string(run[2]) == "LOSA_ERR_BAD_MASS"


@pytest.mark.parametrize("nKb", [40, 1500])
def test_select_flags_rows_whose_masses_do_not_look_like_masses(nKb):
    """Masses above 8, and rows whose masses add up to more than 8 (beyond the warp kernel's
    fixed-point range), are reported instead of giving a silently wrong pattern; a row with a bad
    sum keeps every block.  Both selection kernels (nKb = 1500 takes the sorting one)."""
    losa = lib()
    m = random_mass(4, nKb, 11)
    m[2] = 1.0            # each value passes, the row adds up to nKb
    off, idx, status = run_select(m, 0.9)
    assert losa.losa_status_string(status) == "LOSA_ERR_BAD_MASS"
    assert off[3] - off[2] == nKb
    sel = orc.select(m.astype(np.float64), 0.9)
    rows = util.csr_rows(off, idx[: off[-1]])
    ref = util.csr_rows(sel.offsets, sel.kv_idx)
    assert [rows[r] for r in (0, 1, 3)] == [ref[r] for r in (0, 1, 3)]  # the other rows are untouched
    m = random_mass(4, nKb, 12)
    m[1, 7] = 9.0
    assert losa.losa_status_string(run_select(m, 0.9)[2]) == "LOSA_ERR_BAD_MASS"


def test_select_host_side_argument_errors():
    losa = lib()
    mass = torch.rand(1, 1, 4, 8, device="cuda")
    for tau in (0.0, -1.0, 1.5, float("nan")):
        with pytest.raises(losa.LosaError) as e:
            losa.losa_select(mass, tau)
        assert e.value.code == -1
    with pytest.raises(losa.LosaError) as e:
        losa.losa_select(mass, 0.9, ws=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    # rows longer than LOSA_SELECT_MAX_KEY_BLOCKS are refused before any launch
    long_rows = torch.zeros(1, 1, 1, 8193, device="cuda")
    with pytest.raises(losa.LosaError) as e:
        losa.losa_select(long_rows, 0.9)
    assert e.value.code == -2


@pytest.mark.parametrize("rows,nKb,k", [(16, 33, 1), (16, 33, 20), (8, 256, 170), (4, 929, 557), (8, 40, 40)])
def test_topk_selection_bit_exact(rows, nKb, k):
    losa = lib()
    m32 = random_mass(rows, nKb, 300 + nKb)
    m32[1, 2] = m32[1, 5]  # a tie
    off, idx = losa.losa_select_topk(torch.from_numpy(m32).cuda().reshape(1, 1, rows, nKb), k)
    assert losa.losa_async_status() == 0
    ref_off, ref_idx = orc.select_topk(m32.astype(np.float64), k)
    assert np.array_equal(off.cpu().numpy(), ref_off)
    assert np.array_equal(idx.cpu().numpy()[: rows * k], ref_idx)


def test_row_recall_matches_oracle_and_eq3_guarantee():
    losa = lib()
    m32 = random_mass(64, 278, 77)
    mass = torch.from_numpy(m32).cuda().reshape(1, 2, 32, 278)
    for tau in (0.9, 0.99):
        off, idx = losa.losa_select(mass, tau)
        ret, tot = losa.losa_row_recall(mass, off, idx)
        assert losa.losa_async_status() == 0
        off_h = off.cpu().numpy()
        r_ref, t_ref = orc.row_recall(m32.astype(np.float64), off_h, idx.cpu().numpy()[: off_h[-1]])
        assert np.abs(ret.cpu().numpy() - r_ref).max() < 1e-12
        assert np.abs(tot.cpu().numpy() - t_ref).max() < 1e-12
        assert float(ret.min()) >= tau - 1e-12  # retained mass reaches tau in every row
    # at equal coverage the retained-mass rule keeps at least as much mass per row as any other set
    k = 100
    off_k, idx_k = losa.losa_select_topk(mass, k)
    ret_k, _ = losa.losa_row_recall(mass, off_k, idx_k)
    rng_off, rng_idx = util.random_csr(64, 278, 5, k / 278)
    ret_r, _ = losa.losa_row_recall(mass, torch.from_numpy(rng_off).cuda(), torch.from_numpy(rng_idx).cuda())
    sizes = np.diff(rng_off)
    assert np.all(ret_k.cpu().numpy()[sizes <= k] >= ret_r.cpu().numpy()[sizes <= k] - 1e-12)


def test_validate_csr():
    losa = lib()
    off, idx = util.random_csr(50, 40, 3)
    o, i = torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda()
    losa.losa_validate_csr(o, i, 40)
    assert losa.losa_async_status() == 0
    for mutate in ("range", "order", "empty"):
        off2, idx2 = off.copy(), idx.copy()
        if mutate == "range":
            idx2[off2[7]] = 40
        elif mutate == "order":
            r = int(np.argmax(np.diff(off2) >= 2))
            idx2[off2[r]], idx2[off2[r] + 1] = idx2[off2[r] + 1], idx2[off2[r]]
        else:
            off2[10] = off2[11]
        losa.losa_validate_csr(torch.from_numpy(off2).cuda(), torch.from_numpy(idx2).cuda(), 40)
        assert losa.losa_status_string(losa.losa_async_status()) == "LOSA_ERR_BAD_INDEX", mutate
