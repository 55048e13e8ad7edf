"""Seeded synthetic Q/K/V for LoSA's attention hot path.

This module only *draws inputs*; it holds none of the method's arithmetic (no
softmax, no block mass, no selection).  Both the CUDA path and the CPU oracle
are fed from here, so the two never exchange data with each other.

The tensors stand in for the query/key/value activations of self-attention
layers in video diffusion transformers (the paper's Wan2.1, HunyuanVideo and
CogVideoX-like workloads, "Experiments" section): tokens lie on a 3D
(frame, height, width) grid, optionally preceded by text tokens, and queries
and keys carry a shared sinusoidal position component so that attention mass
is concentrated on spatio-temporally close blocks with a long low-mass tail
(the property the paper's "Motivation" section measures).

Recipe
------
* token index n <-> (t, h, w) with n = n_text + (t * Hh + h) * W + w (w fastest);
  text tokens come first and carry a zero position component.
* PE(t, h, w) in R^d = concat(PE_t, PE_h, PE_w); d_h = d_w = 2 * floor(d / 6),
  d_t = d - d_h - d_w; PE_a(p) = [sin(w_i p)]_i || [cos(w_i p)]_i with
  w_i = base ** (-2 i / d_a), i < d_a / 2.
* Q = N(0,1) + pe_scale * PE, K = N(0,1) + pe_scale * PE (independent noise,
  same PE for every head), V = N(0,1); drawn in fp32 from
  ``torch.Generator('cpu').manual_seed(seed)`` in the order Q, K, V, then
  rounded to bf16 (round-to-nearest-even).
* reuse draw t (t >= 1): x_t = x_0 (fp32, before the cast) + noise * rms(x_0) * eps_t
  with eps_t ~ N(0,1) from seed t, for each of Q, K, V, then cast to bf16.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Tuple

import torch

PE_BASE = 400.0
PE_SCALE = 2.0


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one attention layer's problem."""

    name: str
    B: int
    H: int
    D: int
    grid: Tuple[int, int, int]  # (T, Hh, W) video token grid
    n_text: int
    R: int  # query block size
    C: int  # key/value block size
    tau: float = 0.99
    pe_base: float = PE_BASE
    pe_scale: float = PE_SCALE

    @property
    def N(self) -> int:
        t, h, w = self.grid
        return self.n_text + t * h * w

    @property
    def nQb(self) -> int:
        return -(-self.N // self.R)

    @property
    def nKb(self) -> int:
        return -(-self.N // self.C)

    @property
    def rows(self) -> int:
        return self.B * self.H * self.nQb

    def dense_flop(self) -> float:
        return 4.0 * self.N * self.N * self.D * self.H * self.B


WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 1, 2, 64, (4, 8, 8), 0, 64, 64),
    "small": Workload("small", 1, 4, 64, (8, 16, 16), 0, 64, 64),
    "cogvideox": Workload("cogvideox", 1, 48, 64, (13, 30, 45), 226, 64, 64),
    "wan": Workload("wan", 1, 12, 128, (21, 30, 52), 0, 128, 128),
    "hunyuan": Workload("hunyuan", 1, 24, 128, (33, 45, 80), 0, 128, 128),
    # the Wan-shaped layer with the paper's own block geometry (query blocks of 128, key blocks of 32)
    "wan_r128c32": Workload("wan_r128c32", 1, 12, 128, (21, 30, 52), 0, 128, 32),
}


def _axis_pe(pos: torch.Tensor, d_a: int, base: float) -> torch.Tensor:
    half = d_a // 2
    i = torch.arange(half, dtype=torch.float64)
    omega = base ** (-2.0 * i / d_a)
    ang = pos.to(torch.float64)[:, None] * omega[None, :]
    return torch.cat([torch.sin(ang), torch.cos(ang)], dim=1)


def position_component(wl: Workload) -> torch.Tensor:
    """[N, D] fp32 position component (zero rows for text tokens)."""
    T, Hh, W = wl.grid
    d = wl.D
    d_h = d_w = 2 * (d // 6)
    d_t = d - d_h - d_w
    n = torch.arange(T * Hh * W)
    w = n % W
    h = (n // W) % Hh
    t = n // (W * Hh)
    pe = torch.cat(
        [_axis_pe(t, d_t, wl.pe_base), _axis_pe(h, d_h, wl.pe_base), _axis_pe(w, d_w, wl.pe_base)],
        dim=1,
    )
    out = torch.zeros(wl.N, d, dtype=torch.float64)
    out[wl.n_text:] = pe
    return out.to(torch.float32)


def _base_fp32(wl: Workload, seed: int):
    g = torch.Generator("cpu").manual_seed(seed)
    shape = (wl.B, wl.H, wl.N, wl.D)
    pe = position_component(wl) * wl.pe_scale
    q = torch.randn(shape, generator=g, dtype=torch.float32)
    q += pe
    k = torch.randn(shape, generator=g, dtype=torch.float32)
    k += pe
    v = torch.randn(shape, generator=g, dtype=torch.float32)
    return q, k, v


def make_qkv(wl: Workload, seed: int = 0):
    """Step-0 tensors: contiguous bf16 CPU tensors q, k, v of shape [B, H, N, D]."""
    q, k, v = _base_fp32(wl, seed)
    return q.bfloat16(), k.bfloat16(), v.bfloat16()


def make_base_fp32(wl: Workload, seed: int = 0):
    """The fp32 tensors before the bf16 cast (what the reuse draws perturb)."""
    return _base_fp32(wl, seed)


def make_reuse_draw(wl: Workload, draw: int, base_seed: int = 0, noise: float = 0.05, base=None):
    """Later-step tensors: the step-0 fp32 tensors perturbed by `noise` * rms Gaussian noise.

    Stands in for the later denoising steps on which the frozen pattern is
    reused (the paper recomputes Q/K/V from the current hidden states at each
    step and keeps the block indices fixed).  `base` may carry the result of
    make_base_fp32(wl, base_seed) to avoid drawing it again.
    """
    if draw < 1:
        raise ValueError("reuse draws are numbered from 1")
    if base is None:
        base = _base_fp32(wl, base_seed)
    g = torch.Generator("cpu").manual_seed(draw)
    out = []
    for x in base:
        rms = float(x.double().pow(2).mean().sqrt())
        eps = torch.randn(x.shape, generator=g, dtype=torch.float32)
        out.append((x + (noise * rms) * eps).bfloat16())
    return tuple(out)


def default_scale(D: int) -> float:
    return 1.0 / math.sqrt(D)
