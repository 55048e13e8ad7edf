"""Failure detection on the GPU without harming it: a device-side wait that runs out, and canary
words behind every workspace.

The time-out test never hangs, traps or faults the GPU.  It arms the library's one-shot diagnostic
launch, in which the role that publishes the tile lists publishes nothing and every wait is
limited to a few thousand polls: no copy and no tensor-core instruction is issued, every role's
first wait runs out, the CTAs leave through the common teardown, and the status word reports
LOSA_ERR_TIMEOUT.  The context stays usable: the next ordinary call must pass parity."""
import numpy as np
import pytest
import torch

from oracle import losa_oracle as orc
from tests import util

pytestmark = pytest.mark.gpu


def lib():
    import paper_2608_12032_b200 as losa
    return losa


@pytest.mark.parametrize("mode", ["dense", "sparse", "mass", "fused"])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_fine(mode):
    losa = lib()
    B, H, N, D, BLK = 1, 2, 700, 128, 128
    q = util.rand_bf16((B, H, N, D), 1, 1.5)
    k = util.rand_bf16((B, H, N, D), 2, 1.5)
    v = util.rand_bf16((B, H, N, D), 3)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    nb = -(-N // BLK)
    off, idx = util.random_csr(B * H * nb, nb, 5, 0.5)
    offd, idxd = torch.from_numpy(off).cuda(), torch.from_numpy(idx).cuda()

    def call():
        if mode == "dense":
            return losa.losa_attn(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)
        if mode == "sparse":
            return losa.losa_sparse_attn(qd, kd, vd, offd, idxd, BLK, BLK, out_dtype=torch.float32)
        if mode == "mass":
            return losa.losa_block_mass(qd, kd, BLK, BLK)
        return losa.losa_attn_mass(qd, kd, vd, BLK, BLK, out_dtype=torch.float32)

    assert losa.losa_async_status() == 0
    losa.losa_debug_stall_next_launch(2048)
    call()
    assert losa.losa_status_string(losa.losa_async_status()) == "LOSA_ERR_TIMEOUT"
    assert losa.losa_async_status() == 0  # reading the status cleared it
    # the diagnostic armed exactly one launch: the same call again is an ordinary one
    out = call()
    assert losa.losa_async_status() == 0
    qn, kn, vn = util.to_np(q), util.to_np(k), util.to_np(v)
    if mode == "mass":
        ref = orc.block_mass(qn, kn, BLK, BLK)
        assert np.abs(out.cpu().numpy().reshape(ref.shape) - ref).max() <= util.MASS_TOL
    elif mode == "sparse":
        ref = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, BLK, BLK, off, idx), B, H, N)
        util.assert_output_close(out, ref, "sparse after a timed-out launch")
    else:
        o = out if mode == "dense" else out[0]
        util.assert_output_close(o, orc.dense_attn(qn, kn, vn), f"{mode} after a timed-out launch")


def test_stall_diagnostic_rejects_bad_limits():
    losa = lib()
    for polls in (0, 1 << 17):
        with pytest.raises(losa.LosaError) as e:
            losa.losa_debug_stall_next_launch(polls)
        assert e.value.code == -1


CANARY = 0xA5


def guarded(nbytes):
    """A workspace of exactly `nbytes` usable bytes followed by 4 KiB of canary bytes."""
    buf = torch.full((nbytes + 4096,), CANARY, dtype=torch.uint8, device="cuda")
    return buf, buf[:nbytes]


def intact(buf, nbytes):
    return bool(torch.all(buf[nbytes:] == CANARY))


@pytest.mark.parametrize("R,C,D,N", [(128, 128, 128, 128 * 9 + 5), (64, 64, 64, 64 * 21 + 9), (128, 32, 128, 128 * 6 + 40)])
def test_no_call_writes_past_the_workspace_it_asked_for(R, C, D, N):
    """Every call gets exactly losa_workspace_bytes() bytes; the bytes behind them must survive.
    H is chosen so that the attention kernels cut their last work items into parts (the partial
    results and the tile lists are the largest users of the workspace)."""
    losa = lib()
    B, H = 1, 5
    q = util.rand_bf16((B, H, N, D), 4, 1.5).cuda()
    k = util.rand_bf16((B, H, N, D), 5, 1.5).cuda()
    v = util.rand_bf16((B, H, N, D), 6).cuda()
    prob = losa.make_problem(q, R, C)
    nQb, nKb = -(-N // R), -(-N // C)
    rows = B * H * nQb
    from paper_2608_12032_b200 import binding

    need = {op: losa.losa_workspace_bytes(op, prob) for op in range(5)}
    need[binding.LOSA_OP_SELECT] = binding._select_workspace_bytes(B, H, nQb, nKb)

    buf, ws = guarded(need[binding.LOSA_OP_BLOCK_MASS])
    mass = losa.losa_block_mass(q, k, R, C, ws=ws)
    assert losa.losa_async_status() == 0 and intact(buf, ws.numel())

    buf, ws = guarded(need[binding.LOSA_OP_SELECT])
    off, idx = losa.losa_select(mass, 0.9, ws=ws)
    assert losa.losa_async_status() == 0 and intact(buf, ws.numel())
    buf, ws = guarded(need[binding.LOSA_OP_SELECT])
    losa.losa_select_topk(mass, max(1, nKb // 2), ws=ws)
    assert losa.losa_async_status() == 0 and intact(buf, ws.numel())

    # the longest tile lists: every row keeps every block
    all_off, all_idx = util.all_blocks_csr(rows, nKb)
    for o_h, i_h in ((off, idx), (torch.from_numpy(all_off).cuda(), torch.from_numpy(all_idx).cuda())):
        buf, ws = guarded(need[binding.LOSA_OP_SPARSE_ATTN])
        losa.losa_sparse_attn(q, k, v, o_h, i_h, R, C, ws=ws)
        assert losa.losa_async_status() == 0 and intact(buf, ws.numel())

    buf, ws = guarded(need[binding.LOSA_OP_ATTN])
    losa.losa_attn(q, k, v, R, C, ws=ws)
    assert losa.losa_async_status() == 0 and intact(buf, ws.numel())

    buf, ws = guarded(need[binding.LOSA_OP_ATTN_MASS])
    losa.losa_attn_mass(q, k, v, R, C, ws=ws)
    assert losa.losa_async_status() == 0 and intact(buf, ws.numel())
