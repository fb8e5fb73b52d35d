"""The seeded input generators: shapes, reproducibility, stream statistics."""
import math

import numpy as np
import pytest
import torch

from paper_2605_04711_b200 import workloads as W


def test_shape_counts():
    want = {"toy": (12, 1_049_856), "resnet50": (161, 25_557_032), "gpt2_small": (148, 124_439_808),
            "llama_1b": (146, 1_139_345_408)}
    for name, (n, p) in want.items():
        wl = W.make_workload(name)
        assert (len(wl.blocks), wl.numel) == (n, p), name
    unet = W.make_workload("unet")
    assert abs(unet.numel / 860e6 - 1.0) < 0.02
    assert [W.make_workload(n).window for n in W.WORKLOADS] == [8, 32, 32, 32, 64]


def test_streams_are_reproducible_and_block_local():
    wl = W.make_workload("toy", seed=0)
    a = W.block_grad(wl, 2, 3)
    b = W.block_grad(W.make_workload("toy", seed=0), 2, 3)
    assert a.dtype == torch.bfloat16 and torch.equal(a, b)
    assert not torch.equal(a, W.block_grad(wl, 2, 4))
    assert not torch.equal(a, W.block_grad(W.make_workload("toy", seed=1), 2, 3))
    assert torch.equal(W.block_param(wl, 1), W.block_param(wl, 1))


def test_expected_cosine_is_close_to_stability():
    wl = W.make_workload("toy", seed=0)
    i = 1                                          # 512 x 512
    wl.blocks[i].tau = 0.0                         # equal per-coordinate scales: E cos = a exactly
    g1 = W.block_grad(wl, i, 1).double()
    g2 = W.block_grad(wl, i, 2).double()
    cos = float(g1 @ g2 / (g1.norm() * g2.norm()))
    assert abs(cos - wl.blocks[i].stability) < 0.02


def test_heavy_tail_blocks_and_levels():
    wl = W.make_workload("gpt2_small")
    assert wl.blocks[0].heavy_tail and not wl.blocks[-1].heavy_tail
    un = W.make_workload("unet")
    scales = sorted({round(b.scale, 9) for b in un.blocks})
    assert len(scales) == 4 and abs(scales[-1] / scales[0] - 100.0) < 1e-6


def test_time_ratio_table_and_layout():
    wl = W.make_workload("resnet50")
    t = W.time_ratio_table(wl, [1.0, 1.25, 0.8, 1.5, 0.7])
    assert t.shape == (161, 5) and torch.all(t[:, 0] >= 0.9) and torch.all(t[:, 0] <= 1.1)
    offs, total = W.flat_layout(wl, 128)
    assert all(o % 128 == 0 for o in offs) and total >= wl.numel
    assert all(offs[k + 1] - offs[k] >= wl.blocks[k].numel for k in range(len(offs) - 1))
