"""The Quest-style comparison selector (Sec. 4.2; App. D.2) through the C ABI against the oracle: box statistics from
the shared read of K (exact: minima and maxima of bf16 values), the choice of query block i's ceil(delta (i + 1)) best
blocks outside a 1e-3 band around the last kept score, the union with the forced blocks, density bookkeeping."""
import math

import numpy as np
import pytest
import torch

from oracle import rbs_oracle as orc
from paper_2609_20971_b200 import rbs_block_stats, rbs_block_stats_box, rbs_device_status, rbs_select_box, rbs_sparse_prefill
from paper_2609_20971_b200.synth import SynthConfig, make_inputs, to_f64

pytestmark = pytest.mark.gpu

CASES = {
    "b128": SynthConfig("box_b128", L=2, N=128 * 150 + 37, Hq=4, Hkv=2, B=128, sigma=(0.1, 1.0), seed=81, n_sink=2, n_local=2),
    "b64": SynthConfig("box_b64", N=64 * 300, Hq=2, Hkv=1, B=64, sigma=(0.1, 1.0), sigma_ln=0.4, seed=82),
}


def _bits(mask, M):
    words = mask.cpu().numpy().view(np.uint32)
    return np.unpackbits(words.view(np.uint8), axis=-1, bitorder="little")[..., :M].astype(bool)


@pytest.mark.parametrize("name", list(CASES))
def test_box_selector_parity(name):
    cfg = CASES[name]
    delta = 0.0405 if name == "b128" else 0.11
    Q, K, V = make_inputs(cfg)
    dev = torch.device("cuda:0")
    Qg, Kg = Q.to(dev), K.to(dev)
    stats, lo, hi = rbs_block_stats_box(Kg, cfg.B)
    plain = rbs_block_stats(Kg, cfg.B)
    mask, dens, chosen = rbs_select_box(Qg, lo, hi, cfg.B, delta, cfg.n_sink, cfg.n_local, cfg.n_recent, debug=True)
    torch.cuda.synchronize()
    assert rbs_device_status() == 0
    # the box variant of the statistics kernel gives the same centroids and radii as the plain one
    assert torch.equal(stats.centroid, plain.centroid) and torch.equal(stats.radius, plain.radius)
    M, G = cfg.M, cfg.Hq // cfg.Hkv
    got, got_c = _bits(mask, M), _bits(chosen, M)
    pairs = M * (M + 1) // 2
    for l in range(cfg.L):
        for hk in range(cfg.Hkv):
            olo, ohi = orc.box_stats(to_f64(K[l, :, hk]), cfg.B)
            assert np.array_equal(lo[l, hk].cpu().numpy().astype(np.float64), olo)      # exact: extrema of bf16 values
            assert np.array_equal(hi[l, hk].cpu().numpy().astype(np.float64), ohi)
            for h in range(hk * G, (hk + 1) * G):
                sel = orc.select_head_box(to_f64(Q[l, :, h]), olo, ohi, cfg.B, delta, cfg.n_sink, cfg.n_local, cfg.n_recent)
                near = sel.margin <= 1e-3
                assert not ((got_c[l, h] != sel.chosen) & ~near).any()
                assert not ((got[l, h] != sel.final) & ~near).any()
                assert np.array_equal(got[l, h], got_c[l, h] | sel.forced) and not np.triu(got[l, h], 1).any()
                # every row keeps at least its quota, and more only through ties inside the band
                quota = np.array([min(i + 1, max(1, math.ceil(delta * (i + 1)))) for i in range(M)])
                assert np.all(got_c[l, h].sum(1) >= quota) and np.all(got_c[l, h].sum(1) <= quota + near.sum(1))
                assert float(dens[l, h]) == np.float32(got[l, h].sum() / pairs)
    # the mask drives the attention kernel like any other
    O = rbs_sparse_prefill(Qg, Kg, V.to(dev), mask, cfg.B)
    torch.cuda.synchronize()
    i = M - 3
    ref, _ = orc.masked_attention_block(to_f64(Q[0, :, 1]), to_f64(K[0, :, 1 // G]), to_f64(V[0, :, 1 // G]), got[0, 1, i], i, cfg.B)
    err = np.abs(O[0, i * cfg.B:(i + 1) * cfg.B, 1].float().cpu().numpy() - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3


def test_box_selector_rejects_what_it_does_not_support():
    from paper_2609_20971_b200.binding import RbsError
    cfg = SynthConfig("box_b256", N=256 * 4, Hq=2, Hkv=1, B=256, sigma=0.5, seed=83)
    Q, K, _ = make_inputs(cfg)
    stats, lo, hi = rbs_block_stats_box(K.cuda(), cfg.B)        # the statistics exist for every block size
    olo, ohi = orc.box_stats(to_f64(K[0, :, 0]), cfg.B)
    assert np.array_equal(lo[0, 0].cpu().numpy().astype(np.float64), olo) and np.array_equal(hi[0, 0].cpu().numpy().astype(np.float64), ohi)
    with pytest.raises(RbsError, match="UNSUPPORTED"):
        rbs_select_box(Q.cuda(), lo, hi, cfg.B)
    with pytest.raises(RbsError, match="INVALID"):
        rbs_select_box(Q.cuda(), lo, hi, cfg.B, density_param=0.0)
