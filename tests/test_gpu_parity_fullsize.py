"""Parity at the benchmark's full size (128K tokens, 32 query / 4 KV heads, block 128) in the launch configuration
bench.py times: the whole path runs once on the GPU and sampled outputs are recomputed one by one by the fp64 oracle
(statistics of one KV head, complete mask rows of sampled (head, query block) pairs, attention rows of sampled tiles,
dense rows).  Same tolerances as the small cases."""
import numpy as np
import pytest
import torch

from oracle import rbs_oracle as orc
from paper_2609_20971_b200 import rbs_block_stats, rbs_device_status, rbs_select, rbs_sparse_prefill
from paper_2609_20971_b200.synth import make_inputs, paper_configs, to_f64

pytestmark = pytest.mark.gpu


def _row_bits(mask, l, h, i, M):
    words = mask[l, h, i].cpu().numpy().view(np.uint32)
    return (((words[:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[:M]).astype(bool)


@pytest.fixture(scope="module")
def full():
    cfg = paper_configs()["q30b_128k"]
    Q, K, V = make_inputs(cfg)
    dev = torch.device("cuda:0")
    Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
    stats = rbs_block_stats(Kg, cfg.B)
    mask, dens, mb, mr = rbs_select(Qg, stats, cfg.B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local,
                                    cfg.n_recent, debug=True)
    O, lse = rbs_sparse_prefill(Qg, Kg, Vg, mask, cfg.B, return_lse=True)
    Od = rbs_sparse_prefill(Qg, Kg, Vg, None, cfg.B)
    torch.cuda.synchronize()
    assert rbs_device_status() == 0
    return dict(cfg=cfg, Q=Q, K=K, V=V, stats=stats, mask=mask, dens=dens, mb=mb, mr=mr, O=O, lse=lse, Od=Od)


def test_fullsize_stats_and_selection(full):
    cfg = full["cfg"]
    M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
    rng = np.random.default_rng(5)
    for hk in (0, cfg.Hkv - 1):
        K64 = to_f64(full["K"][0, :, hk])
        c, r = orc.block_stats(K64, B)
        beta, lo, hi = orc.rescue_coefficient(r)
        st = full["stats"]
        assert np.allclose(st.centroid[0, hk].cpu().numpy(), c, rtol=2e-5, atol=2e-6)
        assert np.allclose(st.radius[0, hk].cpu().numpy(), r, rtol=2e-5)
        assert np.allclose(st.rq[0, hk].cpu().numpy(), [lo, hi], rtol=5e-5)
        assert np.allclose(st.beta[0, hk].cpu().numpy(), beta, atol=2e-4)
        h = hk * G + int(rng.integers(0, G))
        rows = sorted({0, 1, 127, 128, M - 1, M - 2} | {int(x) for x in rng.integers(0, M, size=10)})
        sel = orc.select_head(to_f64(full["Q"][0, :, h]), c, r, beta, B, cfg.alpha_base, cfg.alpha_rescue,
                              cfg.n_sink, cfg.n_local, cfg.n_recent, rows=rows)
        for i in rows:
            near_b, near_r = sel.margin_base[i] <= 1e-3, sel.margin_rescue[i] <= 1e-3
            assert not ((_row_bits(full["mb"], 0, h, i, M) != sel.base[i]) & ~near_b).any()
            assert not ((_row_bits(full["mr"], 0, h, i, M) != sel.rescue[i]) & ~near_r).any()
            got = _row_bits(full["mask"], 0, h, i, M)
            assert not ((got != sel.final[i]) & ~(near_b | near_r)).any()
            assert not got[i + 1:].any() and got[i] and got[0]
    # density bookkeeping over the whole mask: popcount of every head's words
    words = full["mask"].cpu().numpy().view(np.uint32)
    pop = np.unpackbits(words.view(np.uint8)).reshape(1, cfg.Hq, -1).sum(-1)
    assert np.array_equal(full["dens"].cpu().numpy(), (pop / (M * (M + 1) / 2)).astype(np.float32))


def test_fullsize_whole_mask(full):
    """Every row of every head of the 128K mask (32 x 1,024 rows; base, rescue and final) against the selector oracle
    run in full: identical outside the 1e-3 band around each branch threshold, and the number of differing decisions
    inside the band stays small."""
    cfg = full["cfg"]
    M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
    words = {k: full[k].cpu().numpy().view(np.uint32)[0] for k in ("mask", "mb", "mr")}       # [Hq, M, W]

    def bits(w):   # [M, W] uint32 -> [M, M] bool
        return np.unpackbits(w.view(np.uint8), axis=1, bitorder="little")[:, :M].astype(bool)
    n_mismatch = 0
    for hk in range(cfg.Hkv):
        c, r = orc.block_stats(to_f64(full["K"][0, :, hk]), B)
        beta, _, _ = orc.rescue_coefficient(r)
        for h in range(hk * G, (hk + 1) * G):
            sel = orc.select_head(to_f64(full["Q"][0, :, h]), c, r, beta, B, cfg.alpha_base, cfg.alpha_rescue,
                                  cfg.n_sink, cfg.n_local, cfg.n_recent)
            near_b, near_r = sel.margin_base <= 1e-3, sel.margin_rescue <= 1e-3
            got, got_b, got_r = bits(words["mask"][h]), bits(words["mb"][h]), bits(words["mr"][h])
            assert not ((got_b != sel.base) & ~near_b).any(), h
            assert not ((got_r != sel.rescue) & ~near_r).any(), h
            assert not ((got != sel.final) & ~(near_b | near_r)).any(), h
            assert np.array_equal(got, got_b | got_r | sel.forced)      # the union is exact on the GPU's own branches
            assert not np.triu(got, 1).any()
            n_mismatch += int((got != sel.final).sum())
            assert abs(float(full["dens"][0, h]) - sel.density) <= (int((near_b | near_r).sum()) + 0.5) / (M * (M + 1) / 2)
    assert n_mismatch <= int(2e-3 * cfg.Hq * M * (M + 1) // 2)


def test_fullsize_attention_rows(full):
    cfg = full["cfg"]
    M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
    rng = np.random.default_rng(6)
    got, want, got_l, want_l = [], [], [], []
    for h in (0, 13, cfg.Hq - 1):
        hk = h // G
        Q64, K64, V64 = to_f64(full["Q"][0, :, h]), to_f64(full["K"][0, :, hk]), to_f64(full["V"][0, :, hk])
        for i in sorted({0, 1, M - 1} | {int(x) for x in rng.integers(2, M - 1, size=4)}):
            bits = _row_bits(full["mask"], 0, h, i, M)
            o, l = orc.masked_attention_block(Q64, K64, V64, bits, i, B)
            want.append(o); want_l.append(l)
            got.append(full["O"][0, i * B:(i + 1) * B, h].float().cpu().numpy())
            got_l.append(full["lse"][0, h, i * B:(i + 1) * B].cpu().numpy())
        # one dense row in the middle of the sequence
        i = M // 2 + h
        o, _ = orc.masked_attention_block(Q64, K64, V64, np.ones(M, bool), i, B)
        err = np.abs(full["Od"][0, i * B:(i + 1) * B, h].float().cpu().numpy() - o)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3
    err = np.abs(np.concatenate(got) - np.concatenate(want))
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    assert np.allclose(np.concatenate(got_l), np.concatenate(want_l), atol=2e-3, rtol=1e-4)


def test_maximum_block_count():
    """The largest block count the library accepts (M = 8192; here 512K tokens at block 64, one head): statistics of
    the whole sequence, complete mask rows of sampled query blocks and their attention rows against the oracle; one
    block more is refused before anything is launched."""
    from paper_2609_20971_b200.binding import RbsError
    from paper_2609_20971_b200.synth import SynthConfig
    cfg = SynthConfig("max_blocks", N=8192 * 64, Hq=1, Hkv=1, B=64, sigma=0.5, seed=88)
    M, B = cfg.M, cfg.B
    assert M == 8192
    Q, K, V = make_inputs(cfg)
    dev = torch.device("cuda:0")
    Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
    stats = rbs_block_stats(Kg, B)
    mask, dens, mb, mr = rbs_select(Qg, stats, B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local,
                                    cfg.n_recent, debug=True)
    O = rbs_sparse_prefill(Qg, Kg, Vg, mask, B)
    torch.cuda.synchronize()
    assert rbs_device_status() == 0
    K64 = to_f64(K[0, :, 0])
    c, r = orc.block_stats(K64, B)
    beta, lo, hi = orc.rescue_coefficient(r)
    assert np.allclose(stats.centroid[0, 0].cpu().numpy(), c, rtol=2e-5, atol=2e-6)
    assert np.allclose(stats.radius[0, 0].cpu().numpy(), r, rtol=2e-5)
    assert np.allclose(stats.beta[0, 0].cpu().numpy(), beta, atol=2e-4)
    rows = [0, 63, 4097, M - 2, M - 1]
    Q64, V64 = to_f64(Q[0, :, 0]), to_f64(V[0, :, 0])
    sel = orc.select_head(Q64, c, r, beta, B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local, cfg.n_recent,
                          rows=rows)
    for i in rows:
        near = (sel.margin_base[i] <= 1e-3) | (sel.margin_rescue[i] <= 1e-3)
        got = _row_bits(mask, 0, 0, i, M)
        assert not ((got != sel.final[i]) & ~near).any()
        assert not got[i + 1:].any()
    for i in (63, 4097, M - 2):      # M - 1 is the dense (recent) row: 8192 blocks, left to the smaller cases
        bits = _row_bits(mask, 0, 0, i, M)
        o, _ = orc.masked_attention_block(Q64, K64, V64, bits, i, B)
        err = np.abs(O[0, i * B:(i + 1) * B, 0].float().cpu().numpy() - o)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3
    words = mask.cpu().numpy().view(np.uint32)
    pop = int(np.unpackbits(words.view(np.uint8)).sum())
    assert abs(float(dens[0, 0]) - pop / (M * (M + 1) / 2)) <= 1e-7
    # one block more than the maximum
    one_more = torch.empty(1, (M + 1) * B, 1, 128, dtype=torch.bfloat16, device=dev)
    with pytest.raises(RbsError, match="UNSUPPORTED"):
        rbs_block_stats(one_more, B)


def _sampled_config_check(cfg, layers, heads_per_layer, n_rows, seed):
    """One pass of the whole path over `cfg` on the GPU; statistics of sampled KV heads, complete mask rows and
    attention tiles of sampled (layer, head, query block) triples are recomputed by the oracle."""
    M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
    Q, K, V = make_inputs(cfg)
    dev = torch.device("cuda:0")
    Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
    stats = rbs_block_stats(Kg, B)
    mask, dens, mb, mr = rbs_select(Qg, stats, B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local,
                                    cfg.n_recent, debug=True)
    O, lse = rbs_sparse_prefill(Qg, Kg, Vg, mask, B, return_lse=True)
    torch.cuda.synchronize()
    assert rbs_device_status() == 0
    del Qg, Kg, Vg
    rng = np.random.default_rng(seed)
    rq_seen = set()
    for l in layers:
        for h in sorted({0, cfg.Hq - 1} | {int(x) for x in rng.integers(0, cfg.Hq, size=heads_per_layer)}):
            hk = h // G
            K64 = to_f64(K[l, :, hk])
            c, r = orc.block_stats(K64, B)
            beta, lo, hi = orc.rescue_coefficient(r)
            assert np.allclose(stats.centroid[l, hk].cpu().numpy(), c, rtol=2e-5, atol=2e-6)
            assert np.allclose(stats.radius[l, hk].cpu().numpy(), r, rtol=2e-5)
            assert np.allclose(stats.rq[l, hk].cpu().numpy(), [lo, hi], rtol=5e-5)
            assert np.allclose(stats.beta[l, hk].cpu().numpy(), beta, atol=2e-4)
            rq_seen.add((round(lo, 6), round(hi, 6)))
            rows = sorted({0, 1, M - 1} | {int(x) for x in rng.integers(0, M, size=n_rows)})
            Q64, V64 = to_f64(Q[l, :, h]), to_f64(V[l, :, hk])
            sel = orc.select_head(Q64, c, r, beta, B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local,
                                  cfg.n_recent, rows=rows)
            got_o, want_o, got_l, want_l = [], [], [], []
            for i in rows:
                near_b, near_r = sel.margin_base[i] <= 1e-3, sel.margin_rescue[i] <= 1e-3
                assert not ((_row_bits(mb, l, h, i, M) != sel.base[i]) & ~near_b).any()
                assert not ((_row_bits(mr, l, h, i, M) != sel.rescue[i]) & ~near_r).any()
                got = _row_bits(mask, l, h, i, M)
                assert not ((got != sel.final[i]) & ~(near_b | near_r)).any()
                assert not got[i + 1:].any()
                if i == M - 1 and M > 1024:
                    continue                      # the dense last row of a very long sequence: covered at 128K / B 128
                o, ls = orc.masked_attention_block(Q64, K64, V64, got, i, B)
                want_o.append(o); want_l.append(ls)
                t0, t1 = i * B, min(cfg.N, (i + 1) * B)
                got_o.append(O[l, t0:t1, h].float().cpu().numpy()); got_l.append(lse[l, h, t0:t1].cpu().numpy())
            err = np.abs(np.concatenate(got_o) - np.concatenate(want_o))
            assert err.max() <= 2e-2 and err.mean() <= 2e-3, (l, h, err.max(), err.mean())
            assert np.allclose(np.concatenate(got_l), np.concatenate(want_l), atol=2e-3, rtol=1e-4)
    # density bookkeeping over the whole mask
    words = mask.cpu().numpy().view(np.uint32)
    pop = np.unpackbits(words.view(np.uint8)).reshape(cfg.L, cfg.Hq, -1).sum(-1)
    assert np.array_equal(dens.cpu().numpy(), (pop / (M * (M + 1) / 2)).astype(np.float32))
    return rq_seen


def test_fullsize_64k_lognormal_norms():
    """The 64K workload: needles at 5 % of the blocks and log-normal key norms (sigma 0.5), which put the radii of all
    blocks far above the needle scale -- the case that stresses the rescue branch."""
    _sampled_config_check(paper_configs()["q30b_64k"], layers=[0], heads_per_layer=3, n_rows=8, seed=11)


def test_fullsize_two_layers_of_the_64_head_shape():
    """Two consecutive layers of the 64-query / 8-KV-head shape at 128K in one call chain (batch = 2): every
    (layer, KV head) has its own key-noise level, hence its own radius quantiles and rescue coefficients."""
    import dataclasses
    cfg = dataclasses.replace(paper_configs()["q32b_128k_8l"], name="q32b_128k_2l", L=2)
    rq_seen = _sampled_config_check(cfg, layers=[0, 1], heads_per_layer=2, n_rows=5, seed=12)
    assert len(rq_seen) >= 4            # distinct (r_low, r_high) per sampled (layer, KV head)
