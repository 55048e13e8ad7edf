"""Head sharding across ranks, on CPU: two gloo ranks each take their heads of one layer, run the
whole path on them (here with the fp64 oracle standing in for the GPU kernels - the partition is
what is under test) and the reassembled masses, pattern and output must equal the one-rank result
exactly.  No collective runs inside the path; the only exchange is the gather of the results."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_12032_b200 import sharding  # noqa: E402

B, H, N, D, R, C, TAU = 2, 5, 200, 16, 32, 16, 0.9


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _layer():
    g = torch.Generator("cpu").manual_seed(3)
    return tuple((torch.randn(B, H, N, D, generator=g) * s).bfloat16() for s in (1.5, 1.5, 1.0))


def _path(q, k, v):
    """mass -> select -> sparse attention on a [B, h, N, D] problem; numpy results."""
    from oracle import losa_oracle as orc

    qn, kn, vn = (t.float().contiguous().numpy() for t in (q, k, v))
    b, h = qn.shape[:2]
    mass = orc.block_mass(qn, kn, R, C)                       # [b*h*nQb, nKb]
    sel = orc.select(mass, TAU)
    o = orc.blocks_to_tokens(orc.sparse_attn(qn, kn, vn, R, C, sel.offsets, sel.kv_idx), b, h, N)
    return mass, sel.offsets, sel.kv_idx, o


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q, k, v = _layer()
    mine = _path(*(sharding.shard_heads(t, rank, world) for t in (q, k, v)))
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)                    # results only; nothing inside the path
    if rank == 0:
        out["parts"] = gathered
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_by_heads_reassemble_to_the_one_rank_result():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        parts = out["parts"]
    q, k, v = _layer()
    mass, off, idx, o = _path(q, k, v)
    nQb, nKb = -(-N // R), -(-N // C)
    # heads 0-1 went to rank 0, heads 2-4 to rank 1
    assert [sharding.head_range(H, r, world) for r in range(world)] == [(0, 2), (2, 5)]
    got_o = sharding.gather_heads([torch.from_numpy(p[3]) for p in parts]).numpy()
    assert np.array_equal(got_o, o)
    got_mass = sharding.gather_heads(
        [torch.from_numpy(p[0]).reshape(B, -1, nQb, nKb) for p in parts]).numpy().reshape(-1, nKb)
    assert np.array_equal(got_mass, mass)
    got_off, got_idx = sharding.gather_csr(
        [(torch.from_numpy(p[1]), torch.from_numpy(p[2])) for p in parts], B, nQb)
    assert np.array_equal(got_off.numpy(), off) and np.array_equal(got_idx.numpy(), idx)
    # slicing the full pattern gives each rank the pattern it built itself
    for r in range(world):
        s_off, s_idx = sharding.shard_csr(torch.from_numpy(off), torch.from_numpy(idx), B, H, nQb, r, world)
        assert np.array_equal(s_off.numpy(), parts[r][1]) and np.array_equal(s_idx.numpy(), parts[r][2])


def test_head_ranges_cover_all_heads_once():
    for heads in (1, 5, 12, 24, 48):
        for world in (1, 2, 4, 8):
            if world > heads:
                with pytest.raises(ValueError):
                    sharding.head_range(heads, 0, world)
                continue
            spans = [sharding.head_range(heads, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == heads
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1
    with pytest.raises(ValueError):
        sharding.head_range(4, 4, 4)
