"""The seeded generator: shapes, determinism, and that needles really are planted as the recipe says."""
import math

import torch

from paper_2609_20971_b200.synth import SynthConfig, make_inputs, paper_configs, to_f64


def test_shapes_dtype_determinism():
    cfg = SynthConfig("t", L=2, N=512, Hq=4, Hkv=2, B=64, sigma=(0.1, 1.0), seed=7)
    Q, K, V = make_inputs(cfg)
    assert Q.shape == (2, 512, 4, 128) and K.shape == V.shape == (2, 512, 2, 128)
    assert Q.dtype == K.dtype == V.dtype == torch.bfloat16 and Q.is_contiguous()
    Q2, K2, V2 = make_inputs(cfg)
    assert torch.equal(Q, Q2) and torch.equal(K, K2) and torch.equal(V, V2)
    cfg.seed = 8
    assert not torch.equal(make_inputs(cfg)[1], K)


def test_needles_have_the_stated_norm_and_rate():
    cfg = SynthConfig("t", N=64 * 256, Hq=2, Hkv=1, B=64, sigma=0.3, p_needle=0.10, seed=9)
    _, K, _ = make_inputs(cfg)
    norms = torch.from_numpy(to_f64(K))[0, :, 0].norm(dim=1).view(cfg.M, cfg.B)
    target = cfg.nu * math.sqrt(cfg.d)            # typical key norm is ~ sqrt(d (1 + sigma^2)) < target
    n_needles = ((norms - target).abs() < 0.1).sum(dim=1)
    assert n_needles.max() <= 1
    assert 0.04 < (n_needles > 0).float().mean().item() < 0.18


def test_paper_configs_cover_the_named_shapes():
    c = paper_configs()
    assert (c["q30b_128k"].N, c["q30b_128k"].Hq, c["q30b_128k"].Hkv, c["q30b_128k"].B) == (131072, 32, 4, 128)
    assert (c["q32b_128k_8l"].L, c["q32b_128k_8l"].Hq, c["q32b_128k_8l"].Hkv) == (8, 64, 8)
    assert c["tiny"].M == 64
