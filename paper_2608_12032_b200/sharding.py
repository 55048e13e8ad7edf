"""Head sharding of one attention layer across GPUs: bookkeeping only, no method arithmetic.

Every (batch, head) is independent in all of the library's calls, and a CSR row belongs to one
(batch, head, query block), so a layer is split across ranks by heads: rank r of W takes the heads
[h0, h1) = [r * H // W, (r + 1) * H // W), its rows of the mass matrix and of the CSR follow, and
nothing is exchanged inside the path (one process per GPU; the surrounding model gathers the
outputs, or re-shards them by sequence, outside this library).  These helpers slice tensors and
patterns for a rank and put per-rank results back in head order; they work on CPU and CUDA tensors
alike.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch


def head_range(H: int, rank: int, world: int) -> Tuple[int, int]:
    """Heads [h0, h1) of rank `rank` out of `world`: contiguous, sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    if world > H:
        raise ValueError(f"{world} ranks cannot share {H} heads: a rank would be left without work")
    return (rank * H) // world, ((rank + 1) * H) // world


def shard_heads(t: torch.Tensor, rank: int, world: int) -> torch.Tensor:
    """The rank's heads of a [B, H, ...] tensor, as a view (the library takes the strides as they are)."""
    h0, h1 = head_range(t.shape[1], rank, world)
    return t[:, h0:h1]


def shard_csr(offsets: torch.Tensor, kv_idx: torch.Tensor, B: int, H: int, nQb: int, rank: int,
              world: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """The rank's rows of a CSR pattern over all heads: (offsets [B*(h1-h0)*nQb + 1], kv_idx).

    Rows are numbered (b * H + h) * nQb + i; the rank's rows are one run per batch entry.  The new
    offsets start at zero; the block indices are copied unchanged (key blocks are per head)."""
    h0, h1 = head_range(H, rank, world)
    off = offsets.to(torch.int64)
    starts = [(b * H + h0) * nQb for b in range(B)]
    stops = [(b * H + h1) * nQb for b in range(B)]
    counts = torch.cat([off[s + 1:e + 1] - off[s:e] for s, e in zip(starts, stops)])
    new_off = torch.zeros(counts.numel() + 1, dtype=torch.int64, device=offsets.device)
    torch.cumsum(counts, 0, out=new_off[1:])
    bounds = [(int(off[s]), int(off[e])) for s, e in zip(starts, stops)]
    new_idx = torch.cat([kv_idx[a:b] for a, b in bounds])
    return new_off.to(torch.int32), new_idx.contiguous()


def gather_heads(parts: Sequence[torch.Tensor]) -> torch.Tensor:
    """Per-rank [B, h_r, ...] results, in rank order, back to [B, H, ...]."""
    return torch.cat(list(parts), dim=1)


def gather_csr(parts: Sequence[Tuple[torch.Tensor, torch.Tensor]], B: int, nQb: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """Per-rank CSR patterns, in rank order, back to one pattern over all heads (the inverse of
    shard_csr): rows are re-interleaved batch entry by batch entry."""
    counts_per_rank: List[torch.Tensor] = []
    for off, _ in parts:
        o = off.to(torch.int64)
        counts_per_rank.append((o[1:] - o[:-1]).reshape(B, -1))  # [B, h_r * nQb]
    counts = torch.cat(counts_per_rank, dim=1).reshape(-1)
    new_off = torch.zeros(counts.numel() + 1, dtype=torch.int64, device=counts.device)
    torch.cumsum(counts, 0, out=new_off[1:])
    pieces = []
    for b in range(B):
        for (off, idx), cnt in zip(parts, counts_per_rank):
            rows = cnt.shape[1]
            o = off.to(torch.int64)
            pieces.append(idx[int(o[b * rows]):int(o[(b + 1) * rows])])
    return new_off.to(torch.int32), torch.cat(pieces).contiguous()
