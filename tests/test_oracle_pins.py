"""Pins for the fp64 oracle: every check compares it with something other than itself --
values the paper prints, closed forms, brute force in pure Python, library routines on special
cases, and invariants the paper states.  CPU only."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import rbs_oracle as orc

GOLDEN = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "appendix_d_examples.json")))


def rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- Sec. 3.1 statistics
def test_centroid_radius_closed_form_symmetric_pairs():
    # keys = mu_b +/- delta_j  =>  centroid = mu_b exactly, radius = max ||delta_j||
    g = rng(1)
    B, d, M = 8, 5, 3
    K, mus, rads = [], [], []
    for b in range(M):
        mu = g.normal(size=d)
        deltas = g.normal(size=(B // 2, d)) * (b + 1)
        K.append(np.concatenate([mu + deltas, mu - deltas]))
        mus.append(mu)
        rads.append(np.sqrt((deltas ** 2).sum(1)).max())
    c, r = orc.block_stats(np.concatenate(K), B)
    assert np.allclose(c, np.stack(mus), atol=1e-13)
    assert np.allclose(r, rads, rtol=1e-13)


def test_centroid_radius_bruteforce_pure_python():
    g = rng(2)
    B, d, M = 4, 3, 5
    K = g.normal(size=(B * M, d))
    c, r = orc.block_stats(K, B)
    for b in range(M):
        rows = [list(map(float, K[b * B + t])) for t in range(B)]
        cen = [math.fsum(row[j] for row in rows) / B for j in range(d)]
        best = 0.0
        for row in rows:
            best = max(best, math.sqrt(math.fsum((row[j] - cen[j]) ** 2 for j in range(d))))
        assert np.allclose(c[b], cen, atol=1e-14)
        assert abs(r[b] - best) < 1e-13


def test_radius_is_distance_to_centroid_not_to_origin_or_pairwise():
    # one block: 3 keys at 0 and one at (4,0): centroid (1,0), farthest key is (4,0) at distance 3
    K = np.array([[0.0, 0], [0, 0], [0, 0], [4, 0]])
    c, r = orc.block_stats(K, 4)
    assert np.allclose(c[0], [1, 0]) and r[0] == pytest.approx(3.0)


def test_short_last_block_divides_by_its_own_size():
    K = np.array([[1.0, 1], [3, 3], [10, 0], [10, 4], [7, 7]])  # B=2 -> blocks of 2, 2, 1
    c, r = orc.block_stats(K, 2)
    assert c.shape == (3, 2)
    assert np.allclose(c[2], [7, 7]) and r[2] == 0.0
    assert np.allclose(c[1], [10, 2]) and r[1] == pytest.approx(2.0)


def test_quantile_closed_form_and_library():
    r = np.arange(11.0)
    assert orc.quantile_linear(r, 0.5) == pytest.approx(5.0)
    assert orc.quantile_linear(r, 0.9) == pytest.approx(9.0)
    r = np.arange(1024.0)[::-1]  # order must not matter; position p*(M-1)
    assert orc.quantile_linear(r, 0.9) == pytest.approx(0.9 * 1023)
    assert orc.quantile_linear(np.array([3.0]), 0.9) == 3.0
    assert orc.quantile_linear(np.array([1.0, 2.0]), 0.5) == pytest.approx(1.5)
    x = rng(3).lognormal(size=257)
    for p in (0.5, 0.9, 0.0, 1.0, 0.123):
        assert orc.quantile_linear(x, p) == pytest.approx(float(np.quantile(x, p)), rel=1e-13)


def test_beta_closed_form_and_plateaus():
    r = np.arange(11.0)                       # r_low = 5, r_high = 9
    beta, lo, hi = orc.rescue_coefficient(r)
    assert (lo, hi) == (pytest.approx(5.0), pytest.approx(9.0))
    assert np.allclose(beta, [0, 0, 0, 0, 0, 0, .25, .5, .75, 1, 1])
    x = rng(4).lognormal(size=1000)
    beta, lo, hi = orc.rescue_coefficient(x)
    assert np.all(beta[x <= lo] == 0) and np.all(beta[x >= hi] == 1)        # Eq. beta plateaus
    assert (beta == 0).sum() >= 500 and (beta == 1).sum() >= 100
    inside = (x > lo) & (x < hi)
    assert np.all((beta[inside] > 0) & (beta[inside] < 1))
    # monotone in the radius
    order = np.argsort(x)
    assert np.all(np.diff(beta[order]) >= 0)


def test_beta_degenerate_quantiles_give_zero():
    beta, lo, hi = orc.rescue_coefficient(np.full(16, 2.5))
    assert lo == hi == 2.5 and np.all(beta == 0)


def test_metadata_closed_form_fixes_record_per_block():
    m = GOLDEN["metadata_mib"]
    per_layer = m["blocks"] * m["kv_heads"]
    mib = 1024.0 * 1024.0
    assert round(per_layer * m["d"] * 2 / mib, 3) == m["centroid_only"]
    assert round(per_layer * (m["d"] * 2 + 4) / mib, 3) == m["with_radius"]
    assert round(per_layer * (m["d"] * 2 + 8) / mib, 3) == m["with_radius_and_beta"]
    # 1,024 blocks at the default block size is the 128K context of the headline result
    assert orc.n_blocks(131072, GOLDEN["defaults"]["block"]) == m["blocks"]
    assert (orc.P_LOW, orc.P_HIGH) == (GOLDEN["defaults"]["p_low"], GOLDEN["defaults"]["p_high"])


# ----------------------------------------------------------------------------- App. D worked examples
def test_worked_example_antipodal_pair():
    ex = GOLDEN["antipodal_pair"]
    g = rng(5)
    u = g.normal(size=6)
    u /= np.linalg.norm(u)
    keys = np.stack([-u, u])
    c, r = orc.block_stats(keys, 2)
    assert np.linalg.norm(c[0]) == pytest.approx(ex["centroid_norm"], abs=1e-15)
    assert r[0] == pytest.approx(ex["radius"])
    for beta in (0.0, 0.3, 1.0):
        lb, lr = orc.branch_logits(u[None, :], c, r, np.array([beta]))
        assert lb[0, 0] == pytest.approx(ex["base_logit"], abs=1e-15)
        assert lr[0, 0] == pytest.approx(beta * ex["rescue_logit_over_beta"])
    assert (keys @ u).max() == pytest.approx(ex["max_token_logit"])


def test_worked_example_cross_polytope_and_thin_box():
    ex = GOLDEN["cross_polytope"]
    keys, q = np.array(ex["keys"], float), np.array(ex["q"], float)
    c, r = orc.block_stats(keys, 4)
    assert np.allclose(c[0], ex["centroid"]) and r[0] == pytest.approx(ex["radius"])
    assert orc.l2_upper_bound(q, keys) == pytest.approx(ex["U_L2"])
    assert orc.box_upper_bound(q, keys) == pytest.approx(ex["U_box"])
    # beta = 1 makes the rescue logit equal the full L2 bound (Sec. 3.2)
    _, lr = orc.branch_logits(q[None, :], c, r, np.ones(1))
    assert lr[0, 0] == pytest.approx(ex["U_L2"])
    ex = GOLDEN["thin_box"]
    e = ex["eps"]
    keys = np.array([[1, 0], [-1, 0], [0, e], [0, -e]], float)
    q = np.array(ex["q"], float)
    _, r = orc.block_stats(keys, 4)
    assert r[0] == pytest.approx(ex["radius"])
    assert orc.l2_upper_bound(q, keys) == pytest.approx(ex["U_L2"])
    assert orc.box_upper_bound(q, keys) == pytest.approx(e * ex["U_box_over_eps"])


def test_cauchy_schwarz_bound_with_beta_one_and_logit_order():
    g = rng(6)
    B, d, M = 8, 16, 12
    K = g.normal(size=(B * M, d)) * g.uniform(0.2, 3.0, size=(B * M, 1))
    Q = g.normal(size=(B, d)) * 2
    c, r = orc.block_stats(K, B)
    lb, lr = orc.branch_logits(Q, c, r, np.ones(M))
    token_max = np.stack([(Q @ K[b * B:(b + 1) * B].T).max(axis=1) for b in range(M)], axis=1)
    assert np.all(lr >= token_max - 1e-12)              # Eq. full_l2_bound
    beta, _, _ = orc.rescue_coefficient(r)
    lb2, lr2 = orc.branch_logits(Q, c, r, beta)
    assert np.all(lr2 >= lb2) and np.array_equal(lb2, lb)      # rescue logits >= base logits
    assert np.all(np.exp(lr2 / math.sqrt(d)).sum(0) >= np.exp(lb2 / math.sqrt(d)).sum(0))


# ----------------------------------------------------------------------------- Sec. 3.2 selection
def _scene(x, radii, d=16, B=4):
    """All queries equal sqrt(d) e1; block b holds keys c_b +/- r_b e2 with c_b = x_b e1.
    Then l_base/sqrt(d) = x_b and l_rescue/sqrt(d) = x_b + r_b beta_b for every token."""
    M = len(x)
    K = np.zeros((M * B, d))
    for b in range(M):
        K[b * B:(b + 1) * B, 0] = x[b]
        K[b * B:(b + 1) * B:2, 1] = radii[b]
        K[b * B + 1:(b + 1) * B:2, 1] = -radii[b]
    Q = np.zeros((M * B, d))
    Q[:, 0] = math.sqrt(d)
    return Q, K


def test_threshold_rule_closed_form_scene():
    # With identical tokens S_b = B exp(z_b - m): b is kept iff z_b >= z_max + ln(alpha).
    B, d = 4, 16
    x = np.array([0.0, -1.0, -2.0, 0.5, -0.2, -3.0, 0.4, -1.4])
    radii = np.array([0.1, 0.1, 3.0, 0.1, 0.1, 5.0, 0.1, 0.1])       # median .1, q90 = 3.6
    M = len(x)
    Q, K = _scene(x, radii, d, B)
    c, r = orc.block_stats(K, B)
    assert np.allclose(r, radii) and np.allclose(c[:, 0], x)
    beta, lo, hi = orc.rescue_coefficient(r)
    exp_beta = np.clip((radii - lo) / (hi - lo), 0, 1)
    assert np.allclose(beta, exp_beta) and beta[5] == 1.0 and 0 < beta[2] < 1
    a_b, a_r = 0.3, 0.2
    sel = orc.select_head(Q, c, r, beta, B, a_b, a_r, 0, 0, 0)
    y = x + radii * exp_beta
    for i in range(M):
        zb, zr = x[:i + 1], y[:i + 1]
        assert np.array_equal(sel.base[i, :i + 1], zb >= zb.max() + math.log(a_b))
        assert np.array_equal(sel.rescue[i, :i + 1], zr >= zr.max() + math.log(a_r))
        assert not sel.base[i, i + 1:].any() and not sel.rescue[i, i + 1:].any()
        # the margins that define the tolerance band of the GPU mask tests: the relative distance of a score from its
        # branch threshold alpha * max S (Eq. branch_thresholds); here S_b / max S = exp(z_b - z_max) exactly, so
        # margin = |exp(z_b - z_max) / alpha - 1|.  (Dividing by max S instead of alpha * max S would fail this.)
        assert np.allclose(sel.margin_base[i, :i + 1], np.abs(np.exp(zb - zb.max()) / a_b - 1.0), rtol=1e-12, atol=1e-14)
        assert np.allclose(sel.margin_rescue[i, :i + 1], np.abs(np.exp(zr - zr.max()) / a_r - 1.0), rtol=1e-12, atol=1e-14)
        assert np.all(np.isinf(sel.margin_base[i, i + 1:])) and np.all(np.isinf(sel.margin_rescue[i, i + 1:]))
    assert not sel.forced.any()
    assert np.array_equal(sel.final, sel.base | sel.rescue)
    # the scene has rows where the rescue mask does not contain the base mask and vice versa
    assert (sel.base & ~sel.rescue).any() and (sel.rescue & ~sel.base).any()


def test_threshold_is_inclusive_and_keeps_argmax():
    S = np.array([1.0, 0.5, 0.25, 0.125])
    assert list(orc.threshold_branch(S, 0.25)) == [True, True, True, False]
    assert list(orc.threshold_branch(S, 1.0)) == [True, False, False, False]


def test_aggregation_sums_tokens_not_means_or_maxes():
    # two tokens, two blocks: logits/sqrt(d) = [[0, ln 3], [ln 4, 0]]  ->  S proportional to [1+4, 3+1]
    d = 4
    z = np.array([[0.0, math.log(3.0)], [math.log(4.0), 0.0]])
    S = orc.aggregate(z * math.sqrt(d), d)
    assert S[0] / S[1] == pytest.approx(5.0 / 4.0)
    assert S.max() <= 2.0 + 1e-12          # shifted by the row-global max: every term <= 1
    L = orc.aggregate_local_lse(z * math.sqrt(d), d)
    assert math.exp(L[0] - L[1]) == pytest.approx(5.0 / 4.0)


def _random_head(seed, M=24, B=8, d=16, s_q=1.0):
    g = rng(seed)
    mu = g.normal(size=(M, 1, d))
    K = (mu + g.uniform(0.1, 1.0) * g.normal(size=(M, B, d)))
    hot = g.random(M) < 0.2
    K[hot, 0] = 4.0 * g.normal(size=(hot.sum(), d))
    K = K.reshape(M * B, d)
    Q = (s_q * g.normal(size=(M, 1, d)) + g.normal(size=(M, B, d))).reshape(M * B, d)
    V = g.normal(size=(M * B, d))
    return Q, K, V


@pytest.mark.parametrize("seed", [10, 11, 12])
def test_union_forced_and_argmax_invariants(seed):
    B = 8
    Q, K, _ = _random_head(seed, B=B)
    c, r = orc.block_stats(K, B)
    beta, _, _ = orc.rescue_coefficient(r)
    M = c.shape[0]
    sel = orc.select_head(Q, c, r, beta, B, 0.22, 0.18, 2, 2, 3)
    assert np.array_equal(sel.final, sel.base | sel.rescue | sel.forced)
    assert not np.triu(sel.final, 1).any()
    for i in range(M):
        want = {b for b in range(i + 1) if b < 2 or b > i - 2 or i >= M - 3}
        assert {int(b) for b in np.nonzero(sel.forced[i])[0]} == want
        assert want <= {int(b) for b in np.nonzero(sel.final[i])[0]}
        assert sel.base[i].any() and sel.rescue[i].any()          # arg-max block is always kept
    assert list(np.nonzero(sel.final[0])[0]) == [0]
    assert sel.density == pytest.approx(sel.final.sum() / (M * (M + 1) / 2))


def test_density_closed_form_forced_only():
    # both branches disabled (alpha > 1): only forced blocks remain.  M = 8, sink/local/recent = 1/1/1:
    # row 0 -> {0}; rows 1..6 -> {0, i}; row 7 -> all 8  => 1 + 12 + 8 = 21 of 36 pairs.
    B = 4
    Q, K, _ = _random_head(13, M=8, B=B)
    c, r = orc.block_stats(K, B)
    beta, _, _ = orc.rescue_coefficient(r)
    sel = orc.select_head(Q, c, r, beta, B, 1.5, 1.5, 1, 1, 1)
    assert not sel.base.any() and not sel.rescue.any()
    assert sel.final.sum() == 21 and sel.density == pytest.approx(21 / 36)


@pytest.mark.parametrize("seed", [20, 21])
def test_reduces_to_centroid_selector(seed):
    B = 8
    Q, K, _ = _random_head(seed, B=B)
    c, r = orc.block_stats(K, B)
    beta, _, _ = orc.rescue_coefficient(r)
    # (a) rescue branch disabled: final == base-branch mask of a selector that never sees radii
    a = orc.select_head(Q, c, r, beta, B, 0.22, 2.0, 0, 0, 0)
    b = orc.select_head(Q, c, np.zeros_like(r), np.zeros_like(r), B, 0.22, 2.0, 0, 0, 0)
    assert np.array_equal(a.final, b.base) and np.array_equal(a.final, a.base)
    # (b) beta == 0 everywhere: both branches score identically, union = centroid mask at min(alpha)
    z = orc.select_head(Q, c, r, np.zeros_like(r), B, 0.22, 0.18, 0, 0, 0)
    lo = orc.select_head(Q, c, r, np.zeros_like(r), B, 0.18, 2.0, 0, 0, 0)
    assert np.array_equal(z.final, lo.base)
    # (c) equal radii => degenerate quantiles => beta = 0
    beta_eq, _, _ = orc.rescue_coefficient(np.full_like(r, 3.0))
    assert not beta_eq.any()


def test_monotone_in_each_alpha():
    B = 8
    Q, K, _ = _random_head(22, B=B)
    c, r = orc.block_stats(K, B)
    beta, _, _ = orc.rescue_coefficient(r)
    prev = None
    for a in (0.9, 0.5, 0.22, 0.1, 0.01):
        sel = orc.select_head(Q, c, r, beta, B, a, a, 1, 1, 1)
        if prev is not None:
            assert not (prev.base & ~sel.base).any() and not (prev.rescue & ~sel.rescue).any()
            assert sel.density >= prev.density
        prev = sel
    full = orc.select_head(Q, c, r, beta, B, 1e-300, 1e-300, 0, 0, 0)
    assert full.density == 1.0


def test_mask_does_not_depend_on_the_shift():
    B, d = 8, 16
    Q, K, _ = _random_head(23, B=B, d=d)
    c, r = orc.block_stats(K, B)
    beta, _, _ = orc.rescue_coefficient(r)
    sel = orc.select_head(Q, c, r, beta, B, 0.22, 0.18, 0, 0, 0)
    M = c.shape[0]
    for i in range(M):
        lb, lr = orc.branch_logits(Q[i * B:(i + 1) * B], c[:i + 1], r[:i + 1], beta[:i + 1])
        for logits, alpha, mask, margin in ((lb, 0.22, sel.base, sel.margin_base),
                                            (lr, 0.18, sel.rescue, sel.margin_rescue)):
            L = orc.aggregate_local_lse(logits, d)
            alt = L >= math.log(alpha) + L.max()
            clear = margin[i, :i + 1] > 1e-9
            assert np.array_equal(alt[clear], mask[i, :i + 1][clear])


def test_rotation_invariance():
    B, d = 8, 16
    Q, K, V = _random_head(24, B=B, d=d)
    R, _ = np.linalg.qr(rng(25).normal(size=(d, d)))
    c, r = orc.block_stats(K, B)
    c2, r2 = orc.block_stats(K @ R, B)
    assert np.allclose(r, r2, rtol=1e-12) and np.allclose(c @ R, c2, atol=1e-12)
    beta, _, _ = orc.rescue_coefficient(r)
    beta2, _, _ = orc.rescue_coefficient(r2)
    s1 = orc.select_head(Q, c, r, beta, B, 0.22, 0.18, 1, 1, 1)
    s2 = orc.select_head(Q @ R, c2, r2, beta2, B, 0.22, 0.18, 1, 1, 1)
    clear = (s1.margin_base > 1e-9) & (s1.margin_rescue > 1e-9)
    assert np.array_equal(s1.final[clear], s2.final[clear])
    i = 7
    o1, _ = orc.masked_attention_block(Q, K, V, s1.final[i], i, B)
    o2, _ = orc.masked_attention_block(Q @ R, K @ R, V, s1.final[i], i, B)
    assert np.allclose(o1, o2, atol=1e-11)


# ----------------------------------------------------------------------------- Sec. 3.3 attention
def test_dense_attention_matches_library_routine():
    g = rng(30)
    N, d = 96, 16
    Q, K, V = g.normal(size=(3, N, d))
    O, lse = orc.dense_causal_attention(Q, K, V)
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0, 0].numpy()
    assert np.allclose(O, ref, atol=1e-12)
    s = torch.from_numpy(Q @ K.T / math.sqrt(d)).masked_fill(torch.triu(torch.ones(N, N, dtype=torch.bool), 1), -math.inf)
    assert np.allclose(lse, torch.logsumexp(s, dim=1).numpy(), atol=1e-12)


def test_full_mask_equals_dense():
    g = rng(31)
    N, d, B = 64, 8, 8
    Q, K, V = g.normal(size=(3, N, d))
    Od, lsed = orc.dense_causal_attention(Q, K, V)
    for i in range(N // B):
        O, lse = orc.masked_attention_block(Q, K, V, np.ones(N // B, bool), i, B)
        assert np.allclose(O, Od[i * B:(i + 1) * B], atol=1e-13)
        assert np.allclose(lse, lsed[i * B:(i + 1) * B], atol=1e-13)


def test_masked_attention_bruteforce_pure_python():
    g = rng(32)
    N, d, B = 16, 3, 4
    Q, K, V = g.normal(size=(3, N, d))
    selected = np.array([True, False, True, True])
    i = 3
    O, lse = orc.masked_attention_block(Q, K, V, selected, i, B)
    for r, t in enumerate(range(i * B, (i + 1) * B)):
        keys = [j for j in range(N) if j <= t and selected[j // B]]
        s = [math.fsum(Q[t, a] * K[j, a] for a in range(d)) / math.sqrt(d) for j in keys]
        w = [math.exp(v) for v in s]
        z = math.fsum(w)
        for a in range(d):
            assert O[r, a] == pytest.approx(math.fsum(wj * V[j, a] for wj, j in zip(w, keys)) / z, abs=1e-13)
        assert lse[r] == pytest.approx(math.log(z), abs=1e-13)


def test_masked_attention_closed_form_block_masses():
    # keys of block b all equal kappa_b * sqrt(d) e1, queries e1: every retained visible key of block b
    # has weight exp(kappa_b).  V = one-hot(block)  =>  O_t[b] = n_b(t) exp(kappa_b) / Z.
    B, M, d = 4, 5, 8
    kappa = np.array([0.3, -1.0, 2.0, 0.0, 1.1])
    K = np.zeros((M * B, d))
    K[:, 0] = np.repeat(kappa, B) * math.sqrt(d)
    Q = np.zeros((M * B, d))
    Q[:, 0] = 1.0
    V = np.zeros((M * B, d))
    V[np.arange(M * B), np.arange(M * B) // B] = 1.0
    selected = np.array([True, False, True, False, True])
    i = 4
    O, lse = orc.masked_attention_block(Q, K, V, selected, i, B)
    for r in range(B):
        n = np.array([B, 0, B, 0, r + 1], float)          # visible retained keys per block
        w = n * np.exp(kappa)
        assert np.allclose(O[r, :M], w / w.sum(), atol=1e-14)
        assert lse[r] == pytest.approx(math.log(w.sum()))
    # blocks beyond i in the mask are ignored; an empty selection gives zeros and -inf
    O2, _ = orc.masked_attention_block(Q, K, V, np.array([True, False, True, False, False]), 2, B)
    assert np.allclose(O2[:, :3].sum(1), 1.0)
    O3, lse3 = orc.masked_attention_block(Q, K, V, np.zeros(M, bool), 3, B)
    assert not O3.any() and np.all(np.isneginf(lse3))


def test_end_to_end_gqa_wrapper_uses_the_right_kv_head():
    g = rng(33)
    L, N, Hq, Hkv, d, B = 2, 64, 4, 2, 8, 8
    Q = g.normal(size=(L, N, Hq, d))
    K = g.normal(size=(L, N, Hkv, d)) * g.uniform(0.5, 2.0, size=(L, 1, Hkv, 1))
    ref = orc.select_all(Q, K, B, 0.22, 0.18, 1, 1, 1)
    for l in range(L):
        for h in range(Hq):
            hk = h // (Hq // Hkv)
            c, r = orc.block_stats(K[l, :, hk], B)
            beta, lo, hi = orc.rescue_coefficient(r)
            assert np.array_equal(ref.centroid[l, hk], c) and np.array_equal(ref.beta[l, hk], beta)
            assert tuple(ref.rq[l, hk]) == (lo, hi)
            one = orc.select_head(Q[l, :, h], c, r, beta, B, 0.22, 0.18, 1, 1, 1)
            assert np.array_equal(ref.selection[l][h].final, one.final)
            assert ref.density[l, h] == one.density


def test_short_last_block_selection_is_causal_and_uses_its_own_tokens():
    # cutting tokens off the end must not change any earlier query block's row (causality), and the short last
    # query block scores exactly like a direct evaluation of Eq. block_aggregation over its remaining tokens
    B, d = 8, 16
    Q, K, _ = _random_head(26, M=12, B=B, d=d)
    cut = 5
    Qs, Ks = Q[:-cut], K[:-cut]
    c, r = orc.block_stats(K, B)
    cs, rs = orc.block_stats(Ks, B)
    assert np.array_equal(c[:-1], cs[:-1]) and np.array_equal(r[:-1], rs[:-1])
    beta = np.linspace(0, 1, 12)                    # same beta on both sides: the quantiles see the changed last radius
    full = orc.select_head(Q, c, r, beta, B, 0.22, 0.18, 1, 1, 0)
    short = orc.select_head(Qs, cs, rs, beta, B, 0.22, 0.18, 1, 1, 0)
    assert np.array_equal(full.final[:-1, :-1], short.final[:-1, :-1])
    i = 11
    lb, lr = orc.branch_logits(Qs[i * B:], cs, rs, beta)
    Sb = np.exp(lb / math.sqrt(d)).sum(0)
    Sr = np.exp(lr / math.sqrt(d)).sum(0)
    want = (Sb >= 0.22 * Sb.max()) | (Sr >= 0.18 * Sr.max()) | orc.forced_blocks(i, 12, 1, 1, 0)
    assert np.array_equal(short.final[i], want)


def test_group_union_is_a_superset_with_additive_density_bound():
    """Union over a KV group's heads: contains every head's mask, adds nothing else, density between the
    largest per-head density and their sum."""
    rng = np.random.default_rng(5)
    M = 17
    causal = np.tril(np.ones((M, M), dtype=bool))
    heads = [(rng.random((M, M)) < 0.2) & causal for _ in range(4)]
    u = orc.group_union(heads)
    for f in heads:
        assert not (f & ~u).any()
    assert not (u & ~np.any(np.stack(heads), axis=0)).any()
    rho = [orc.density(f) for f in heads]
    assert max(rho) <= orc.density(u) <= sum(rho)
    assert np.array_equal(orc.group_union([heads[0]]), heads[0])


# ----------------------------------------------------------------------------- Sec. 4.2 / App. D.2: Quest-style box selector
def test_box_stats_and_bound_against_the_worked_examples_and_brute_force():
    ex = GOLDEN["cross_polytope"]
    keys, q = np.array(ex["keys"], float), np.array(ex["q"], float)
    lo, hi = orc.box_stats(keys, 4)
    assert np.array_equal(lo[0], [-1, -1]) and np.array_equal(hi[0], [1, 1])
    assert orc.box_logits(q[None, :], lo, hi)[0, 0] == pytest.approx(ex["U_box"])
    ex = GOLDEN["thin_box"]
    e = ex["eps"]
    keys = np.array([[1, 0], [-1, 0], [0, e], [0, -e]], float)
    lo, hi = orc.box_stats(keys, 4)
    assert orc.box_logits(np.array([ex["q"]], float), lo, hi)[0, 0] == pytest.approx(e * ex["U_box_over_eps"])
    # random blocks: per-coordinate extrema by pure Python; the bound dominates every token logit and equals
    # q.v + |q|.h with the box centre v and half-width h (App. D.2)
    g = rng(20)
    B, d, M = 6, 5, 4
    K = g.normal(size=(B * M, d)) * g.uniform(0.2, 2.0, size=(B * M, 1))
    Q = g.normal(size=(7, d))
    lo, hi = orc.box_stats(K, B)
    for b in range(M):
        rows = [list(map(float, K[b * B + t])) for t in range(B)]
        assert np.array_equal(lo[b], [min(r[j] for r in rows) for j in range(d)])
        assert np.array_equal(hi[b], [max(r[j] for r in rows) for j in range(d)])
    U = orc.box_logits(Q, lo, hi)
    token_max = np.stack([(Q @ K[b * B:(b + 1) * B].T).max(axis=1) for b in range(M)], axis=1)
    assert np.all(U >= token_max - 1e-12)
    v, h = (hi + lo) / 2, (hi - lo) / 2
    assert np.allclose(U, Q @ v.T + np.abs(Q) @ h.T, rtol=1e-13, atol=1e-13)
    # a short last block uses its own keys only
    lo2, hi2 = orc.box_stats(K[:B * M - 2], B)
    assert np.array_equal(lo2[-1], K[B * (M - 1):B * M - 2].min(0)) and np.array_equal(lo2[:-1], lo[:-1])


def test_top_fraction_counts_ties_and_extremes():
    S = np.array([5.0, 1.0, 3.0, 3.0, 2.0, 0.5, 4.0, 0.1])
    assert orc.top_fraction(S, 0.25).sum() == 2 and orc.top_fraction(S, 0.25)[[0, 6]].all()
    assert orc.top_fraction(S, 0.26).sum() == 4          # ceil(2.08) = 3, and the tie with the third score is kept
    assert orc.top_fraction(S, 1.0).all() and orc.top_fraction(S, 1e-9).sum() == 1
    assert orc.top_fraction(np.array([2.0]), 0.0405).all()


def test_box_selection_closed_form_scene_and_invariants():
    # identical queries sqrt(d) e1; block b holds keys x_b e1 +/- w_b e2: box logit / sqrt(d) = x_b exactly
    # (the queries have no e2 component), so row i keeps the ceil(delta (i + 1)) largest x_b, b <= i
    B, d = 4, 16
    x = np.array([0.0, -1.0, 2.0, 0.5, -0.2, 3.0, 0.4, -1.4, 1.0, 0.9])
    Q, K = _scene(x, np.linspace(0.1, 2.0, len(x)), d, B)
    lo, hi = orc.box_stats(K, B)
    M = len(x)
    sel = orc.select_head_box(Q, lo, hi, B, 0.3, 0, 0, 0)
    for i in range(M):
        k = int(math.ceil(0.3 * (i + 1)))
        want = np.zeros(i + 1, bool)
        want[np.argsort(-x[:i + 1], kind="stable")[:k]] = True
        assert np.array_equal(sel.final[i, :i + 1], want) and not sel.final[i, i + 1:].any()
        kth = np.sort(x[:i + 1])[::-1][k - 1]
        assert np.allclose(sel.margin[i, :i + 1], np.abs(np.exp(x[:i + 1] - kth) - 1.0), rtol=1e-12, atol=1e-14)
    assert sel.density == pytest.approx(sum(int(math.ceil(0.3 * (i + 1))) for i in range(M)) / (M * (M + 1) / 2))
    # forced blocks are united in; a larger density parameter never removes a block
    Qr, Kr, _ = _random_head(21, M=20, B=8)
    lo, hi = orc.box_stats(Kr, 8)
    a = orc.select_head_box(Qr, lo, hi, 8, 0.1, 1, 1, 1)
    b2 = orc.select_head_box(Qr, lo, hi, 8, 0.25, 1, 1, 1)
    assert np.array_equal(a.final, a.chosen | a.forced) and np.all(b2.final | ~a.final) and b2.density >= a.density
    assert a.final[-1, :].all() and a.final[:, 0].all() and np.diag(a.final).all()
