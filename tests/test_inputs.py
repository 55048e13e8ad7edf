"""The synthetic input generator: shapes, determinism, and the locality it is meant to create."""
import numpy as np
import torch

from paper_2608_12032_b200 import inputs


def test_workload_shapes_match_the_named_configs():
    w = inputs.WORKLOADS
    assert (w["tiny"].N, w["tiny"].nQb, w["tiny"].nKb) == (256, 4, 4)
    assert (w["small"].N, w["small"].nQb) == (2048, 32)
    assert (w["cogvideox"].N, w["cogvideox"].nKb, w["cogvideox"].N - 277 * 64) == (17776, 278, 48)
    assert (w["wan"].N, w["wan"].nKb, w["wan"].N - 255 * 128) == (32760, 256, 120)
    assert (w["hunyuan"].N, w["hunyuan"].nKb, w["hunyuan"].N - 928 * 128) == (118800, 929, 16)


def test_generator_is_seeded_and_bf16():
    wl = inputs.WORKLOADS["tiny"]
    a = inputs.make_qkv(wl, 0)
    b = inputs.make_qkv(wl, 0)
    c = inputs.make_qkv(wl, 1)
    for x, y in zip(a, b):
        assert x.dtype == torch.bfloat16 and x.shape == (1, 2, 256, 64) and x.is_contiguous()
        assert torch.equal(x, y)
    assert not torch.equal(a[0], c[0])


def test_position_component_layout():
    wl = inputs.Workload("t", 1, 1, 64, (2, 3, 4), 5, 16, 16)
    pe = inputs.position_component(wl)
    assert pe.shape == (5 + 24, 64)
    assert torch.all(pe[:5] == 0)  # text tokens carry no position
    # token (t,h,w) = (0,0,0): sines are 0, cosines are 1
    first = pe[5]
    assert torch.allclose(first[:12], torch.zeros(12)) and torch.allclose(first[12:24], torch.ones(12))
    # w is the fastest axis: tokens 5 and 6 differ only in the w part (last 20 dims)
    assert torch.equal(pe[5, :44], pe[6, :44]) and not torch.equal(pe[5, 44:], pe[6, 44:])
    # each axis part has unit-norm (sin, cos) pairs -> squared norm = d/2
    assert abs(float(pe[17].pow(2).sum()) - 32.0) < 1e-4


def test_reuse_draw_is_a_small_perturbation():
    wl = inputs.WORKLOADS["tiny"]
    q0, _, _ = inputs.make_qkv(wl, 0)
    q1, _, _ = inputs.make_reuse_draw(wl, 1)
    q1b, _, _ = inputs.make_reuse_draw(wl, 1)
    q2, _, _ = inputs.make_reuse_draw(wl, 2)
    assert torch.equal(q1, q1b) and not torch.equal(q1, q2)
    rel = float((q1.float() - q0.float()).pow(2).mean().sqrt() / q0.float().pow(2).mean().sqrt())
    assert 0.03 < rel < 0.07
