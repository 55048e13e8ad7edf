"""losa_select_noalloc: the selection entry point for callers that cannot allocate.

Some users of this library run where device allocation is not theirs to do: a serving loop whose
memory was partitioned at start-up, a host framework whose allocator owns the whole device, a
plugin that receives tensors and nothing else.  For them the library carries its own fixed
scratch array.  This test drives that entry point through the C ABI and checks, on two calls in a
row that share the scratch array (with different inputs, so stale contents would show), that it
returns exactly what losa_select returns and exactly what the fp64 oracle's Eq. 3 gives on the
same masses.  Integer results: both comparisons are bit-exact.  Rows of 278 and 33 blocks take
the warp-per-row kernel, rows of 1500 blocks the sorting kernel, as in losa_select.

Collected last on purpose, so a run that stops at the first failure has already run the rest.
"""
import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu


def random_mass(B, H, nQb, nKb, seed):
    rng = np.random.default_rng(seed)
    m = np.exp(3.0 * rng.standard_normal((B, H, nQb, nKb)))
    return torch.from_numpy((m / m.sum(-1, keepdims=True)).astype(np.float32)).cuda()


def test_noalloc_select_matches_select_on_two_calls_in_a_row():
    import paper_2608_12032_b200 as losa

    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    # second problem is smaller and differently shaped: leftovers of the first call must not leak
    for call, (shape, tau) in enumerate([((1, 3, 40, 278), 0.99), ((2, 2, 9, 33), 0.9),
                                         ((1, 1, 5, 1500), 0.95)]):
        B, H, nQb, nKb = shape
        mass = random_mass(B, H, nQb, nKb, 100 + call)
        rows = B * H * nQb
        ref_off, ref_idx = losa.losa_select(mass, tau)
        assert losa.losa_async_status() == 0
        offsets = torch.full((rows + 1,), -1, dtype=torch.int32, device="cuda")
        kv_idx = torch.full((rows * nKb,), -1, dtype=torch.int32, device="cuda")
        losa.losa_select_noalloc(mass, tau, offsets, kv_idx, device_status=status)
        torch.cuda.synchronize()
        assert int(status) == 0
        assert torch.equal(offsets, ref_off)
        nnz = int(ref_off[-1])
        assert torch.equal(kv_idx[:nnz], ref_idx[:nnz])
        assert torch.all(kv_idx[nnz:] == -1)  # nothing written past the CSR
        # against the oracle's rule on the same fp32 masses
        sel = orc.select(mass.cpu().numpy().reshape(rows, nKb).astype(np.float64), tau)
        bad, exempt = util.compare_csr(offsets.cpu().numpy(), kv_idx.cpu().numpy(), sel)
        assert not bad and exempt == 0
        # a warm call leaves the device's free memory as it found it
        free_before = torch.cuda.mem_get_info()[0]
        losa.losa_select_noalloc(mass, tau, offsets, kv_idx, device_status=status)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before


def test_noalloc_select_reports_device_errors_and_size_limit():
    import paper_2608_12032_b200 as losa

    mass = random_mass(1, 1, 8, 64, 7)
    offsets = torch.empty(9, dtype=torch.int32, device="cuda")
    kv_idx = torch.empty(16, dtype=torch.int32, device="cuda")  # too small on purpose
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    losa.losa_select_noalloc(mass, 0.99, offsets, kv_idx, device_status=status)
    torch.cuda.synchronize()
    assert losa.losa_status_string(int(status)) == "LOSA_ERR_CAPACITY"
    # a later good call clears the word again
    kv_idx = torch.empty(8 * 64, dtype=torch.int32, device="cuda")
    losa.losa_select_noalloc(mass, 0.99, offsets, kv_idx, device_status=status)
    torch.cuda.synchronize()
    assert int(status) == 0
    # a negative mass is reported through the caller's word too
    bad = mass.clone()
    bad[0, 0, 3, 5] = -0.25
    losa.losa_select_noalloc(bad, 0.99, offsets, kv_idx, device_status=status)
    torch.cuda.synchronize()
    assert losa.losa_status_string(int(status)) == "LOSA_ERR_BAD_MASS"
    assert losa.losa_async_status() == 0  # the library's own status word is not involved
    # a mass matrix whose scratch exceeds the built-in array is refused before any launch
    # (no launch happens, so the pointers only have to be non-null)
    with pytest.raises(losa.LosaError) as e:
        losa.binding._check(
            losa.binding._lib().losa_select_noalloc(1, 1, 40000, 929, 16, 0.99, 16, 16, 1, None, None),
            "losa_select_noalloc")
    assert e.value.code == -3
