"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Tolerances (from the build's target statement):
  * integer / bit work (mask words, density bookkeeping): exact, except that a (query block, key block)
    decision may differ from the oracle where the oracle's score is within 1e-3 (relative) of that
    branch's threshold;
  * attention output, bf16 inputs with fp32 accumulation: max-abs <= 2e-2 and mean-abs <= 2e-3;
  * statistics (fp32 sums of <= 256 bf16 values): rtol 2e-5 against fp64.
"""
import math

import numpy as np
import pytest
import torch

from oracle import rbs_oracle as orc
from paper_2609_20971_b200 import rbs_block_stats, rbs_mask_group_union, rbs_select, rbs_sparse_prefill
from paper_2609_20971_b200.synth import SynthConfig, make_inputs, paper_configs, to_f64

pytestmark = pytest.mark.gpu

MASK_MARGIN = 1e-3
OUT_MAX_ABS = 2e-2
OUT_MEAN_ABS = 2e-3


@pytest.fixture(autouse=True)
def no_wait_gave_up():
    """Every kernel wait is bounded; a wait that ran out would leave a code in the device status word."""
    yield
    from paper_2609_20971_b200 import rbs_device_status
    assert rbs_device_status(clear=True) == 0


def unpack_mask(mask: torch.Tensor, M: int) -> np.ndarray:
    """[L, Hq, M, W] int32 words -> bool [L, Hq, M, M]."""
    words = mask.cpu().numpy().view(np.uint32)
    bits = (words[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1
    return bits.reshape(*words.shape[:-1], -1)[..., :M].astype(bool)


def pack_mask(dense: np.ndarray) -> torch.Tensor:
    """bool [L, Hq, M, M] -> int32 words [L, Hq, M, W]."""
    L, H, M, _ = dense.shape
    W = (M + 31) // 32
    padded = np.zeros((L, H, M, W * 32), dtype=np.uint32)
    padded[..., :M] = dense
    words = (padded.reshape(L, H, M, W, 32) << np.arange(32, dtype=np.uint32)).sum(-1).astype(np.uint32)
    return torch.from_numpy(words.view(np.int32))


CASES = {
    # name: config.  Sizes span several 128-row centroid tiles with a ragged tail and both block sizes.
    "tiny_iid": paper_configs()["tiny_iid"],
    "tiny": paper_configs()["tiny"],
    "ragged_b64": SynthConfig("ragged_b64", N=64 * 300, Hq=2, Hkv=1, B=64, sigma=(0.1, 1.0), seed=31),
    "gqa_b128": SynthConfig("gqa_b128", L=2, N=128 * 150, Hq=4, Hkv=2, B=128, sigma=(0.1, 1.0), seed=32,
                            n_sink=2, n_local=3, n_recent=2),
    "gqa_b256": SynthConfig("gqa_b256", N=256 * 37, Hq=4, Hkv=2, B=256, sigma=(0.1, 1.0), seed=34, n_sink=1, n_local=2,
                            n_recent=1),
    # sequence lengths that are not a multiple of the block: short last key / query block
    "ragged_n_b128": SynthConfig("ragged_n_b128", N=128 * 21 + 37, Hq=4, Hkv=2, B=128, sigma=(0.1, 1.0), seed=35),
    "ragged_n_b64": SynthConfig("ragged_n_b64", N=64 * 45 + 63, Hq=2, Hkv=1, B=64, sigma=0.5, seed=36),
    "ragged_n_b256": SynthConfig("ragged_n_b256", N=256 * 9 + 100, Hq=2, Hkv=2, B=256, sigma=0.5, seed=37),
    "lognormal_b128": SynthConfig("lognormal_b128", N=128 * 40, Hq=2, Hkv=2, B=128, sigma=0.5, sigma_ln=0.5,
                                  p_needle=0.05, seed=33),
    # a last block of 256 whose SECOND half of 128 tokens is the short one, an odd group size, and coherent queries
    # of large norm: logits beyond the range in which the norm bounds can serve as log-sum-exp shifts
    "ragged_n2_b256": SynthConfig("ragged_n2_b256", N=256 * 6 + 200, Hq=3, Hkv=1, B=256, sigma=(0.1, 1.0), s_q=3.5,
                                  seed=38),
    "hot_b128": SynthConfig("hot_b128", N=128 * 19 + 5, Hq=4, Hkv=2, B=128, sigma=(0.1, 1.0), s_q=3.5, sigma_ln=0.3,
                            seed=39),
}


@pytest.fixture(scope="module", params=list(CASES))
def case(request):
    cfg = CASES[request.param]
    Q, K, V = make_inputs(cfg)
    dev = torch.device("cuda:0")
    Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
    stats = rbs_block_stats(Kg, cfg.B)
    mask, density, mb, mr = rbs_select(Qg, stats, cfg.B, cfg.alpha_base, cfg.alpha_rescue,
                                       cfg.n_sink, cfg.n_local, cfg.n_recent, debug=True)
    torch.cuda.synchronize()
    Q64, K64 = to_f64(Q), to_f64(K)
    ref = orc.select_all(Q64, K64, cfg.B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local, cfg.n_recent)
    return dict(cfg=cfg, Q=Q, K=K, V=V, Qg=Qg, Kg=Kg, Vg=Vg, stats=stats, mask=mask, density=density,
                mb=mb, mr=mr, ref=ref, Q64=Q64, K64=K64, V64=to_f64(V))


def test_block_stats_parity(case):
    st, ref = case["stats"], case["ref"]
    c = st.centroid.cpu().numpy().astype(np.float64)
    r = st.radius.cpu().numpy().astype(np.float64)
    assert np.allclose(c, ref.centroid, rtol=2e-5, atol=2e-6)
    assert np.allclose(r, ref.radius, rtol=2e-5)


def test_rescue_coefficient_parity(case):
    st, ref = case["stats"], case["ref"]
    assert np.allclose(st.rq.cpu().numpy(), ref.rq, rtol=5e-5)
    assert np.allclose(st.beta.cpu().numpy(), ref.beta, atol=2e-4)
    # plateaus are exact: beta == 0 at or below the median radius, == 1 at or above the 0.9 quantile
    beta = st.beta.cpu().numpy()
    lo, hi = ref.rq[..., 0:1], ref.rq[..., 1:2]
    assert np.all(beta[ref.radius < lo * (1 - 1e-4)] == 0) and np.all(beta[ref.radius > hi * (1 + 1e-4)] == 1)


def test_mask_parity(case):
    cfg, ref = case["cfg"], case["ref"]
    M = cfg.M
    final = unpack_mask(case["mask"], M)
    base = unpack_mask(case["mb"], M)
    rescue = unpack_mask(case["mr"], M)
    n_mismatch = 0
    for l in range(cfg.L):
        for h in range(cfg.Hq):
            s = ref.selection[l][h]
            near_b = s.margin_base <= MASK_MARGIN
            near_r = s.margin_rescue <= MASK_MARGIN
            assert not ((base[l, h] != s.base) & ~near_b).any()
            assert not ((rescue[l, h] != s.rescue) & ~near_r).any()
            bad = (final[l, h] != s.final) & ~(near_b | near_r)
            assert not bad.any()
            n_mismatch += int((final[l, h] != s.final).sum())
            # the union is exact on the GPU's own branch masks, forced blocks always present, nothing above the diagonal
            assert np.array_equal(final[l, h], base[l, h] | rescue[l, h] | s.forced)
            assert not np.triu(final[l, h], 1).any()
    pairs = M * (M + 1) // 2
    assert n_mismatch <= max(2, int(2e-3 * pairs * cfg.L * cfg.Hq))   # near-threshold blocks are rare


def test_group_union_of_masks(case):
    """Group-shared variant: bit-exact union of the GPU's own per-head masks inside each KV group, density of it."""
    cfg = case["cfg"]
    M, G = cfg.M, cfg.Hq // cfg.Hkv
    per_head = unpack_mask(case["mask"], M)
    mask = case["mask"].clone()
    dens = torch.empty_like(case["density"])
    rbs_mask_group_union(mask, dens, cfg.Hkv, cfg.B, cfg.N)
    torch.cuda.synchronize()
    got = unpack_mask(mask, M)
    dens = dens.cpu().numpy()
    for l in range(cfg.L):
        for hk in range(cfg.Hkv):
            want = orc.group_union([per_head[l, hk * G + g] for g in range(G)])
            for g in range(G):
                assert np.array_equal(got[l, hk * G + g], want)
                assert abs(dens[l, hk * G + g] - orc.density(want)) <= 1e-6
    # words past the last block column stay untouched (zero)
    assert np.array_equal(mask.cpu().numpy()[..., (M + 31) // 32:], case["mask"].cpu().numpy()[..., (M + 31) // 32:])


def test_density_parity(case):
    cfg, ref = case["cfg"], case["ref"]
    M = cfg.M
    final = unpack_mask(case["mask"], M)
    dens = case["density"].cpu().numpy()
    pairs = M * (M + 1) // 2
    for l in range(cfg.L):
        for h in range(cfg.Hq):
            assert dens[l, h] == np.float32(final[l, h].sum() / pairs)         # exact bookkeeping
            allowed = ((ref.selection[l][h].margin_base <= MASK_MARGIN) |
                       (ref.selection[l][h].margin_rescue <= MASK_MARGIN)).sum()
            assert abs(dens[l, h] - ref.density[l, h]) <= (allowed + 0.5) / pairs


def _check_output(O_gpu, O_ref):
    err = np.abs(O_gpu - O_ref)
    assert err.max() <= OUT_MAX_ABS, err.max()
    assert err.mean() <= OUT_MEAN_ABS, err.mean()


def _rows_to_check(cfg, n=12, seed=0):
    M = cfg.M
    rows = {0, 1, M - 1, M // 2}
    rng = np.random.default_rng(seed)
    rows |= {int(x) for x in rng.integers(0, M, size=n)}
    return sorted(r for r in rows if 0 <= r < M)


def test_sparse_attention_parity(case):
    cfg = case["cfg"]
    M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
    O, lse = rbs_sparse_prefill(case["Qg"], case["Kg"], case["Vg"], case["mask"], B, return_lse=True)
    torch.cuda.synchronize()
    O = O.float().cpu().numpy().astype(np.float64)
    lse = lse.cpu().numpy().astype(np.float64)
    final = unpack_mask(case["mask"], M)     # the oracle attends over the mask the GPU kernel was given
    every_row = M <= 64
    for l in range(cfg.L):
        for h in range(cfg.Hq):
            hk = h // G
            rows = range(M) if every_row else _rows_to_check(cfg, seed=l * 131 + h)
            got, want, got_lse, want_lse = [], [], [], []
            for i in rows:
                o_ref, lse_ref = orc.masked_attention_block(case["Q64"][l, :, h], case["K64"][l, :, hk],
                                                            case["V64"][l, :, hk], final[l, h, i], i, B)
                want.append(o_ref); want_lse.append(lse_ref)
                got.append(O[l, i * B:min(cfg.N, (i + 1) * B), h]); got_lse.append(lse[l, h, i * B:min(cfg.N, (i + 1) * B)])
            _check_output(np.concatenate(got), np.concatenate(want))
            assert np.allclose(np.concatenate(got_lse), np.concatenate(want_lse), atol=2e-3, rtol=1e-4)


def test_dense_attention_parity(case):
    cfg = case["cfg"]
    if cfg.N > 8192:
        pytest.skip("dense oracle rows are checked on the small cases; large cases check sampled rows below")
    B, G = cfg.B, cfg.Hq // cfg.Hkv
    O = rbs_sparse_prefill(case["Qg"], case["Kg"], case["Vg"], None, B)
    torch.cuda.synchronize()
    O = O.float().cpu().numpy().astype(np.float64)
    for l in range(cfg.L):
        for h in range(cfg.Hq):
            ref, _ = orc.dense_causal_attention(case["Q64"][l, :, h], case["K64"][l, :, h // G], case["V64"][l, :, h // G])
            _check_output(O[l, :, h], ref)


def test_dense_attention_sampled_rows(case):
    cfg = case["cfg"]
    if cfg.N <= 8192:
        pytest.skip("covered in full by test_dense_attention_parity")
    M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
    O = rbs_sparse_prefill(case["Qg"], case["Kg"], case["Vg"], None, B)
    torch.cuda.synchronize()
    O = O.float().cpu().numpy().astype(np.float64)
    full = np.ones(M, dtype=bool)
    l, h = cfg.L - 1, cfg.Hq - 1
    got, want = [], []
    for i in (0, 1, M // 3, M - 1):
        o_ref, _ = orc.masked_attention_block(case["Q64"][l, :, h], case["K64"][l, :, h // G], case["V64"][l, :, h // G], full, i, B)
        want.append(o_ref); got.append(O[l, i * B:min(cfg.N, (i + 1) * B), h])
    _check_output(np.concatenate(got), np.concatenate(want))


# ------------------------------------------------------------------------------------------ edge cases
def _small(B=64, M=5, Hq=2, Hkv=1, seed=40):
    cfg = SynthConfig("edge", N=B * M, Hq=Hq, Hkv=Hkv, B=B, sigma=0.4, seed=seed)
    Q, K, V = make_inputs(cfg)
    return cfg, Q, K, V


@pytest.mark.parametrize("B", [64, 128, 256])
def test_single_block_sequence(B):
    cfg, Q, K, V = _small(B=B, M=1)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    stats = rbs_block_stats(Kg, B)
    mask, dens = rbs_select(Qg, stats, B)
    assert unpack_mask(mask, 1).all() and np.all(dens.cpu().numpy() == 1.0)
    assert np.all(stats.beta.cpu().numpy() == 0)            # one radius: degenerate quantiles
    O = rbs_sparse_prefill(Qg, Kg, Vg, mask, B).float().cpu().numpy()
    for h in range(cfg.Hq):
        ref, _ = orc.dense_causal_attention(to_f64(Q)[0, :, h], to_f64(K)[0, :, 0], to_f64(V)[0, :, 0])
        _check_output(O[0, :, h], ref)


def test_hand_built_mask_empty_rows_and_bits_above_diagonal():
    cfg, Q, K, V = _small(B=64, M=6)
    M, B = cfg.M, cfg.B
    dense = np.zeros((1, cfg.Hq, M, M), dtype=bool)
    dense[0, 0] = np.tril(np.random.default_rng(1).random((M, M)) < 0.5)
    dense[0, 0, 2, :] = False                     # an empty row
    dense[0, 0, 3, :] = False
    dense[0, 0, 3, 3] = True                      # diagonal only
    dense[0, 1] = np.tril(np.ones((M, M), bool))
    given = dense.copy()
    given[0, 1, 1, 4] = True                      # bits with b > i must be ignored
    given[0, 0, 2, 5] = True
    mask = pack_mask(given).cuda()
    O, lse = rbs_sparse_prefill(Q.cuda(), K.cuda(), V.cuda(), mask, B, return_lse=True)
    O = O.float().cpu().numpy().astype(np.float64)
    lse = lse.cpu().numpy()
    for h in range(cfg.Hq):
        for i in range(M):
            ref, lref = orc.masked_attention_block(to_f64(Q)[0, :, h], to_f64(K)[0, :, 0], to_f64(V)[0, :, 0], dense[0, h, i], i, B)
            _check_output(O[0, i * B:(i + 1) * B, h], ref)
            if not dense[0, h, i].any():
                assert not O[0, i * B:(i + 1) * B, h].any() and np.all(np.isneginf(lse[0, h, i * B:(i + 1) * B]))


def test_branch_disable_and_degenerate_radii():
    cfg, Q, K, V = _small(B=64, M=40, seed=41)
    Qg, Kg = Q.cuda(), K.cuda()
    stats = rbs_block_stats(Kg, cfg.B)
    Q64, K64 = to_f64(Q), to_f64(K)
    # rescue branch disabled (alpha > 1): final == base-branch mask, no forced blocks
    mask, _, mb, mr = rbs_select(Qg, stats, cfg.B, 0.22, 2.0, 0, 0, 0, debug=True)
    assert torch.equal(mask, mb) and not mr.any()
    ref = orc.select_all(Q64, K64, cfg.B, 0.22, 2.0, 0, 0, 0)
    for h in range(cfg.Hq):
        s = ref.selection[0][h]
        assert not ((unpack_mask(mask, cfg.M)[0, h] != s.final) & (s.margin_base > MASK_MARGIN)).any()
    # both disabled: forced blocks only, density closed form 1 + 2 (M - 2) + M over M (M + 1) / 2
    mask, dens = rbs_select(Qg, stats, cfg.B, 1.5, 1.5, 1, 1, 1)
    M = cfg.M
    assert np.allclose(dens.cpu().numpy(), (1 + 2 * (M - 2) + M) / (M * (M + 1) / 2))
    # equal radii => beta == 0 => both branches score identically
    stats.radius.fill_(3.0)
    mask, _, mb, mr = rbs_select(Qg, stats, cfg.B, 0.2, 0.2, 0, 0, 0, debug=True)
    assert not stats.beta.any() and torch.equal(mb, mr)


def test_strided_views_of_a_packed_qkv_buffer():
    cfg, Q, K, V = _small(B=128, M=9, Hq=4, Hkv=2, seed=42)
    L, N, d = 1, cfg.N, cfg.d
    packed = torch.empty(L, N, cfg.Hq + 2 * cfg.Hkv, d, dtype=torch.bfloat16, device="cuda")
    packed[:, :, :cfg.Hq] = Q.cuda()
    packed[:, :, cfg.Hq:cfg.Hq + cfg.Hkv] = K.cuda()
    packed[:, :, cfg.Hq + cfg.Hkv:] = V.cuda()
    Qv, Kv, Vv = packed[:, :, :cfg.Hq], packed[:, :, cfg.Hq:cfg.Hq + cfg.Hkv], packed[:, :, cfg.Hq + cfg.Hkv:]
    s1 = rbs_block_stats(Kv, cfg.B)
    s2 = rbs_block_stats(K.cuda(), cfg.B)
    assert torch.equal(s1.centroid, s2.centroid) and torch.equal(s1.radius, s2.radius)
    m1, d1 = rbs_select(Qv, s1, cfg.B)
    m2, d2 = rbs_select(Q.cuda(), s2, cfg.B)
    assert torch.equal(m1, m2) and torch.equal(d1, d2)
    o1 = rbs_sparse_prefill(Qv, Kv, Vv, m1, cfg.B)
    o2 = rbs_sparse_prefill(Q.cuda(), K.cuda(), V.cuda(), m2, cfg.B)
    assert torch.equal(o1, o2)


def test_select_is_deterministic_and_reusable_workspace():
    cfg, Q, K, V = _small(B=64, M=33, seed=43)
    Qg, Kg = Q.cuda(), K.cuda()
    stats = rbs_block_stats(Kg, cfg.B)
    m1, d1 = rbs_select(Qg, stats, cfg.B)
    m2, d2 = rbs_select(Qg, stats, cfg.B)
    assert torch.equal(m1, m2) and torch.equal(d1, d2)


def test_selector_variants_match_the_oracle_with_fixed_beta():
    """Centroid-only (beta = 0, one threshold) and Full-L2 (beta = 1, one threshold) through rbs_select_variant."""
    from paper_2609_20971_b200.binding import SELECTOR_CENTROID_ONLY, SELECTOR_FULL_L2
    cfg, Q, K, V = _small(B=128, M=140, Hq=2, Hkv=1, seed=44)
    Qg, Kg = Q.cuda(), K.cuda()
    stats = rbs_block_stats(Kg, cfg.B)
    Q64, K64 = to_f64(Q), to_f64(K)
    c, r = orc.block_stats(K64[0, :, 0], cfg.B)
    for selector, beta, ab, ar in ((SELECTOR_CENTROID_ONLY, np.zeros_like(r), 0.194, 2.0),
                                   (SELECTOR_FULL_L2, np.ones_like(r), 2.0, 0.022)):
        mask, dens = rbs_select(Qg, stats, cfg.B, ab if ab < 1 else 0.5, ar if ar < 1 else 0.5, 1, 1, 1, selector=selector)
        assert np.array_equal(stats.beta.cpu().numpy()[0, 0], beta.astype(np.float32))
        got = unpack_mask(mask, cfg.M)
        for h in range(cfg.Hq):
            s = orc.select_head(Q64[0, :, h], c, r, beta, cfg.B, ab, ar, 1, 1, 1)
            near = (s.margin_base <= MASK_MARGIN) if ab < 1 else (s.margin_rescue <= MASK_MARGIN)
            assert not ((got[0, h] != s.final) & ~near).any()


@pytest.mark.parametrize("B,Mtot,cuts", [(128, 23, (0, 7, 16)), (64, 40, (0, 13)), (256, 9, (0, 4))])
def test_chunked_calls_reproduce_the_whole_sequence(B, Mtot, cuts):
    """Queries processed in chunks (a KV prefix plus new query blocks) give bit-identical masks and outputs."""
    from paper_2609_20971_b200 import rbs_select_chunk, rbs_sparse_prefill_chunk
    cfg = SynthConfig("chunk", N=B * Mtot - 19, Hq=4, Hkv=2, B=B, sigma=(0.1, 1.0), seed=45, n_recent=2)
    Q, K, V = make_inputs(cfg)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    stats = rbs_block_stats(Kg, B)
    mask, dens = rbs_select(Qg, stats, B, 0.22, 0.18, 1, 1, 2)
    O, lse = rbs_sparse_prefill(Qg, Kg, Vg, mask, B, return_lse=True)
    Od = rbs_sparse_prefill(Qg, Kg, Vg, None, B)
    bounds = list(cuts) + [cfg.M]
    kept = 0.0
    for q0, q1 in zip(bounds[:-1], bounds[1:]):
        t0, t1 = q0 * B, min(cfg.N, q1 * B)
        Qc = Qg[:, t0:t1]                                        # a strided view: no copy
        mc, dc = rbs_select_chunk(Qc, stats, B, cfg.N, q0, 0.22, 0.18, 1, 1, 2)
        assert torch.equal(mc, mask[:, :, q0:q1])
        pairs = sum(i + 1 for i in range(q0, q1))
        kept += float(dc[0, 0]) * pairs
        oc, lc = rbs_sparse_prefill_chunk(Qc, Kg, Vg, mc, B, q0, return_lse=True)
        assert torch.equal(oc, O[:, t0:t1]) and torch.equal(lc, lse[:, :, t0:t1])
        od = rbs_sparse_prefill_chunk(Qc, Kg, Vg, None, B, q0)
        if B == 64 and q0 % 2 == 1:
            # dense attention with blocks of 64 runs on the 128-row tensor-core kernel when the chunk starts on a
            # 128-token boundary and on the 64-row kernel otherwise: same values to rounding, not the same bits
            assert (od.float() - Od[:, t0:t1].float()).abs().max().item() <= OUT_MAX_ABS
        else:
            assert torch.equal(od, Od[:, t0:t1])
    assert abs(kept / (cfg.M * (cfg.M + 1) / 2) - float(dens[0, 0])) < 1e-6


def test_host_pipeline_matches_device_resident_calls():
    from paper_2609_20971_b200.host import HostPrefill
    cfg = SynthConfig("host", L=1, N=128 * 37 + 50, Hq=4, Hkv=2, B=128, sigma=(0.1, 1.0), seed=46)
    Q, K, V = make_inputs(cfg)
    Qh, Kh, Vh = Q.pin_memory(), K.pin_memory(), V.pin_memory()
    Oh = torch.empty_like(Qh).pin_memory()
    hp = HostPrefill(1, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.B, "cuda:0", chunk_blocks=8)
    for _ in range(2):                       # second run reuses buffers and streams
        Oh.zero_()
        hp.run(Qh, Kh, Vh, Oh)
        hp.wait()
        torch.cuda.synchronize()
        Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
        stats = rbs_block_stats(Kg, cfg.B)
        mask, _ = rbs_select(Qg, stats, cfg.B)
        O = rbs_sparse_prefill(Qg, Kg, Vg, mask, cfg.B)
        assert torch.equal(Oh.cuda(), O) and torch.equal(hp.mask(), mask)


def test_varlen_batch_equals_one_call_per_prompt():
    """Prompts of different lengths packed back to back: each is selected and attended on its own (Sec. 4.1:
    requests are not concatenated), so the packed call must reproduce the single-prompt calls bit for bit, and the
    oracle's attention on sampled rows."""
    from paper_2609_20971_b200.host import prefill_varlen
    dev = torch.device("cuda:0")
    B, Hq, Hkv = 128, 4, 2
    lens = [128 * 9 + 17, 128 * 3, 100, 128 * 14 + 127]
    parts = [make_inputs(SynthConfig(f"varlen{k}", N=n, Hq=Hq, Hkv=Hkv, B=B, sigma=0.5, seed=70 + k)) for k, n in enumerate(lens)]
    Qp, Kp, Vp = (torch.cat([p[j][0] for p in parts], dim=0).to(dev) for j in range(3))
    cu = np.concatenate([[0], np.cumsum(lens)])
    streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    O, dens = prefill_varlen(Qp, Kp, Vp, cu, B, streams=streams)
    torch.cuda.synchronize()
    for k, (Q, K, V) in enumerate(parts):
        Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
        stats = rbs_block_stats(Kg, B)
        mask, d1 = rbs_select(Qg, stats, B)
        O1 = rbs_sparse_prefill(Qg, Kg, Vg, mask, B)
        torch.cuda.synchronize()
        assert torch.equal(O[cu[k]:cu[k + 1]], O1[0])
        assert torch.equal(dens[k], d1)
    # the same batch through the library's own varlen entry point (one call, one workspace)
    from paper_2609_20971_b200.binding import rbs_prefill_varlen
    O2, dens2 = rbs_prefill_varlen(Qp, Kp, Vp, cu, B)
    torch.cuda.synchronize()
    assert torch.equal(O2, O) and all(torch.equal(dens2[k:k + 1], dens[k]) for k in range(len(lens)))
    # oracle check on the shortest prompt (one short block: dense causal attention over 100 tokens)
    k = 2
    Q64, K64, V64 = (to_f64(t) for t in parts[k])
    ref, _ = orc.dense_causal_attention(Q64[0, :, 0], K64[0, :, 0], V64[0, :, 0])
    got = O[cu[k]:cu[k + 1], 0].float().cpu().numpy()
    assert np.abs(got - ref).max() <= OUT_MAX_ABS


@pytest.mark.parametrize("pos", [10, 100])
def test_logit_jump_inside_a_block(pos):
    """One key far out of scale (its logit exceeds everything before it by about 115 in log2 units) in the first or
    the second half of a late key block: the running maximum has to be replaced in the middle of the block and O
    rescaled, for the rows that see the key and only for them."""
    dev = torch.device("cuda:0")
    B, N, d = 128, 128 * 6, 128
    g = torch.Generator().manual_seed(91 + pos)
    u = torch.ones(d) / math.sqrt(d)
    Q = (3.0 * u + 0.5 * torch.randn(N, d, generator=g)).to(torch.bfloat16).view(1, N, 1, d)
    K = (0.1 * torch.randn(N, d, generator=g))
    t_big = 3 * B + pos
    K[t_big] = 300.0 * u
    K = K.to(torch.bfloat16).view(1, N, 1, d)
    V = torch.randn(N, d, generator=g).to(torch.bfloat16).view(1, N, 1, d)
    O, lse = rbs_sparse_prefill(Q.to(dev), K.to(dev), V.to(dev), None, B, return_lse=True)
    torch.cuda.synchronize()
    ref, ref_lse = orc.dense_causal_attention(to_f64(Q[0, :, 0]), to_f64(K[0, :, 0]), to_f64(V[0, :, 0]))
    err = np.abs(O[0, :, 0].float().cpu().numpy() - ref)
    assert err.max() <= OUT_MAX_ABS and err.mean() <= OUT_MEAN_ABS, (err.max(), err.mean())
    assert np.allclose(lse[0, 0].cpu().numpy(), ref_lse, atol=2e-3, rtol=1e-4)
    # rows from the big key on are its value row (to bf16 rounding); earlier rows are not
    assert np.abs(O[0, t_big + 5, 0].float().cpu().numpy() - V[0, t_big, 0].float().numpy()).max() <= 2e-2


def test_whole_path_is_bitwise_repeatable():
    """Statistics, selection and attention (sparse and dense) give bit-identical results launch after launch:
    nothing in the path depends on the order in which CTAs happen to run."""
    dev = torch.device("cuda:0")
    cfg = SynthConfig("repeat", N=128 * 37 + 55, Hq=8, Hkv=2, B=128, sigma=(0.1, 1.0), seed=5)
    Q, K, V = (t.to(dev) for t in make_inputs(cfg))
    ref = None
    for _ in range(25):
        st = rbs_block_stats(K, cfg.B)
        mask, dens = rbs_select(Q, st, cfg.B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local, cfg.n_recent)
        O = rbs_sparse_prefill(Q, K, V, mask, cfg.B)
        Od = rbs_sparse_prefill(Q, K, V, None, cfg.B)
        torch.cuda.synchronize()
        cur = (st.centroid, st.radius, st.beta, mask, dens, O, Od)
        if ref is None:
            ref = cur
        else:
            assert all(torch.equal(a, b) for a, b in zip(ref, cur))


def test_batch_stride_beyond_32_bits():
    """Two layers whose data sit more than 2^31 elements apart inside one buffer (strided views, nothing copied):
    every kernel must carry the batch offset in 64 bits.  Checked bit for bit against the same data held contiguously."""
    dev = torch.device("cuda:0")
    B, N, Hq, Hkv, d = 128, 128 * 9 + 40, 4, 2, 128
    SB = (1 << 31) + (1 << 20)                       # batch stride in elements
    nq, nk = N * Hq * d, N * Hkv * d
    big = torch.empty(SB + 2 * nq + 2 * nk, dtype=torch.bfloat16, device=dev)

    def view(off, H):
        return torch.as_strided(big, (2, N, H, d), (SB, H * d, d, 1), off)
    Qv, Ov = view(0, Hq), view(nq, Hq)
    Kv, Vv = view(2 * nq, Hkv), view(2 * nq + nk, Hkv)
    cfg = SynthConfig("stride", L=2, N=N, Hq=Hq, Hkv=Hkv, B=B, sigma=(0.1, 1.0), seed=77)
    Q, K, V = (t.to(dev) for t in make_inputs(cfg))
    Qv.copy_(Q); Kv.copy_(K); Vv.copy_(V)
    st_v = rbs_block_stats(Kv, B)
    mask_v, dens_v = rbs_select(Qv, st_v, B)
    rbs_sparse_prefill(Qv, Kv, Vv, mask_v, B, out=Ov)
    st = rbs_block_stats(K, B)
    mask, dens = rbs_select(Q, st, B)
    O = rbs_sparse_prefill(Q, K, V, mask, B)
    torch.cuda.synchronize()
    assert torch.equal(st_v.centroid, st.centroid) and torch.equal(st_v.radius, st.radius)
    assert torch.equal(mask_v, mask) and torch.equal(dens_v, dens)
    assert torch.equal(Ov, O)
    assert not torch.equal(O[0], O[1])               # the two layers really differ


@pytest.mark.parametrize("B,M,tail", [(128, 300, 77), (256, 140, 0)])
def test_long_rows_are_split_and_merged(B, M, tail):
    """Rows of more than 256 key tiles of 128 are cut into parts that run as separate CTAs and are merged afterwards
    (here the dense "recent" rows and a hand-made long row): outputs and lse against the oracle, bit-identical results
    when the same rows are computed by chunked calls, and a second launch gives the same bits."""
    from paper_2609_20971_b200 import rbs_sparse_prefill_chunk
    cfg = SynthConfig("split", N=B * (M - 1) + (tail or B), Hq=4, Hkv=2, B=B, sigma=(0.1, 1.0), seed=61, n_recent=2)
    Q, K, V = make_inputs(cfg)
    dev = torch.device("cuda:0")
    Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
    stats = rbs_block_stats(Kg, B)
    mask, _ = rbs_select(Qg, stats, B, cfg.alpha_base, cfg.alpha_rescue, 1, 1, cfg.n_recent)
    dense = unpack_mask(mask, cfg.M)
    dense[0, 1, cfg.M - 5, : cfg.M - 4] = True          # one more long row, not at the end, for one head only
    dense[0, 1, cfg.M - 5, 3:40:2] = False              # with holes
    mask = pack_mask(dense).to(dev)
    from paper_2609_20971_b200.binding import prefill_workspace_bytes
    ws = torch.empty(prefill_workspace_bytes(1, cfg.N, cfg.Hq, cfg.Hkv, B), dtype=torch.uint8, device=dev)
    O, lse = rbs_sparse_prefill(Qg, Kg, Vg, mask, B, return_lse=True, workspace=ws)
    O2 = rbs_sparse_prefill(Qg, Kg, Vg, mask, B, workspace=ws)
    O_plain = rbs_sparse_prefill(Qg, Kg, Vg, mask, B)          # no workspace: every row whole
    torch.cuda.synchronize()
    assert torch.equal(O, O2)
    assert (O.float() - O_plain.float()).abs().max().item() <= OUT_MAX_ABS
    short = slice(0, 200 * 128)                                  # rows that are not cut give the same bits either way
    assert torch.equal(O[:, short], O_plain[:, short])
    Q64, K64, V64 = to_f64(Q), to_f64(K), to_f64(V)
    for h, i in ((0, cfg.M - 1), (3, cfg.M - 2), (1, cfg.M - 5), (1, cfg.M - 6), (2, 5)):
        ref, lref = orc.masked_attention_block(Q64[0, :, h], K64[0, :, h // 2], V64[0, :, h // 2], dense[0, h, i], i, B)
        t0, t1 = i * B, min(cfg.N, (i + 1) * B)
        _check_output(O[0, t0:t1, h].float().cpu().numpy(), ref)
        assert np.allclose(lse[0, h, t0:t1].cpu().numpy(), lref, atol=2e-3, rtol=1e-4)
    # the last query blocks again as a chunk of their own: the same rows are cut the same way
    q0 = cfg.M - 7
    oc, lc = rbs_sparse_prefill_chunk(Qg[:, q0 * B:], Kg, Vg, mask[:, :, q0:].contiguous(), B, q0, return_lse=True,
                                      workspace=ws)
    assert torch.equal(oc, O[:, q0 * B:]) and torch.equal(lc, lse[:, :, q0 * B:])


def test_grouped_attention_under_group_shared_masks():
    """Head-packed query tiles: with the masks of a KV group made identical (rbs_mask_group_union) two heads of the group
    share one stream of K/V tiles.  Against the oracle (attention over the oracle's union of the GPU's per-head masks) and
    against the one-head-per-CTA kernel on the same mask."""
    from paper_2609_20971_b200 import rbs_sparse_prefill_grouped
    for cfg in (SynthConfig("grouped", L=2, N=128 * 45 + 50, Hq=8, Hkv=2, B=128, sigma=(0.1, 1.0), seed=62),
                SynthConfig("grouped256", N=256 * 21, Hq=4, Hkv=2, B=256, sigma=0.6, seed=63)):
        Q, K, V = make_inputs(cfg)
        dev = torch.device("cuda:0")
        Qg, Kg, Vg = Q.to(dev), K.to(dev), V.to(dev)
        stats = rbs_block_stats(Kg, cfg.B)
        mask, dens = rbs_select(Qg, stats, cfg.B, cfg.alpha_base, cfg.alpha_rescue, 1, 1, 1)
        per_head = unpack_mask(mask, cfg.M)
        rbs_mask_group_union(mask, dens, cfg.Hkv, cfg.B, cfg.N)
        O, lse = rbs_sparse_prefill_grouped(Qg, Kg, Vg, mask, cfg.B, return_lse=True)
        O1, lse1 = rbs_sparse_prefill(Qg, Kg, Vg, mask, cfg.B, return_lse=True)
        torch.cuda.synchronize()
        assert (O.float() - O1.float()).abs().max().item() <= OUT_MAX_ABS
        assert torch.allclose(lse, lse1, atol=2e-3, rtol=1e-4)
        M, B, G = cfg.M, cfg.B, cfg.Hq // cfg.Hkv
        Q64, K64, V64 = to_f64(Q), to_f64(K), to_f64(V)
        Onp, lnp = O.float().cpu().numpy(), lse.cpu().numpy()
        for l in range(cfg.L):
            for h in (0, 3, cfg.Hq - 1):
                hk = h // G
                want_mask = orc.group_union([per_head[l, hk * G + g] for g in range(G)])
                for i in (0, 1, M // 2, M - 1):
                    ref, lref = orc.masked_attention_block(Q64[l, :, h], K64[l, :, hk], V64[l, :, hk], want_mask[i], i, B)
                    t0, t1 = i * B, min(cfg.N, (i + 1) * B)
                    _check_output(Onp[l, t0:t1, h], ref)
                    assert np.allclose(lnp[l, h, t0:t1], lref, atol=2e-3, rtol=1e-4)
