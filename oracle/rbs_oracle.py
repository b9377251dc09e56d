"""Plain fp64 CPU oracle for the RBS-Attention prefill path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of what
the path computes.  It is imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg, and by nothing else; the CUDA library never routes through it and
shares no code, tables or helpers with it.

Everything is float64 numpy.  Inputs are the bf16 values the GPU sees, widened exactly.
Each function names the passage of the paper it restates.  No blocking, fusion or
re-ordering beyond what the definitions say.

Readings taken where the paper is silent (each is an argument, so another reading is one
call-site change):
  * quantile = linear interpolation between order statistics at position p*(M-1)
    (Sec. 3.1 only says "quantile(r, 0.5)", "median and 90-th percentile");
  * r_high <= r_low  =>  beta = 0 for that head (Eq. beta is defined only for r_high > r_low);
  * 1/sqrt(d) scales the whole branch logit, radius term included (Eq. block_aggregation
    divides l_z by sqrt(d));
  * candidates C_i = {b <= i}, diagonal block scored with its full centroid;
  * threshold comparison is inclusive (>=), as printed in Eq. branch_thresholds;
  * sink / local / recent are counted in blocks: key blocks b < n_sink; key blocks
    i - n_local < b <= i; the last n_recent query blocks keep every causal key block;
  * masks are per query head; query head h uses the statistics of KV head h // (Hq/Hkv);
  * density denominator is M(M+1)/2 per head (Eq. actual_density, "valid causal block pairs").

Parity pins (tests/test_oracle_pins.py): worked examples of App. D, closed-form threshold
scenes, brute force on tiny inputs, reduction to the centroid selector, full mask == dense
causal attention == a library attention routine, invariances (shift, rotation, monotone in
alpha).  Parity unpinned (a reading only; nothing in the paper fixes them): the quantile
interpolation rule, per-query-head mask granularity under GQA, the meaning and units of
sink/local/recent, and scoring of the diagonal block.

The Quest-style comparison selector (Sec. 4.2; App. D.2, Eq. quest_box) is restated too: per-coordinate
minima / maxima per block (box_stats), the box upper bound as the block logit (box_logits; pinned by
the App. D.2 values and by "bound >= every token logit"), and block selection by a density parameter.
The paper only says the adaptation "uses per-dimension key minima/maxima and query-dependent block
selection" with "density parameter 0.0405" in "a shared prefill backend".  Reading taken, PARITY
UNPINNED: the box logit goes through the same aggregation over the query block's tokens as the
other selectors (Eq. block_aggregation); query block i keeps its ceil(delta * (i + 1)) best causal
blocks, ties with the last kept score included, united with the same forced blocks.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

P_LOW = 0.5   # Sec. 4.4: r_low  = quantile(r, 0.5)
P_HIGH = 0.9  # Sec. 4.4: r_high = quantile(r, 0.9)


def n_blocks(n_tokens: int, block: int) -> int:
    """M = ceil(N / B) (Sec. 3.3)."""
    return (n_tokens + block - 1) // block


# --------------------------------------------------------------------------------------
# Sec. 3.1: block statistics
# --------------------------------------------------------------------------------------
def block_stats(K: np.ndarray, block: int):
    """Centroid c_b = mean of the block's keys and radius r_b = max_k ||k - c_b||_2.

    Sec. 3.1 (centroid and maximum-radius equations), Algorithm 1 first loop.
    K: [N, d] keys of ONE KV head.  A short last block divides by its own size |K_b|.
    Returns (centroid [M, d], radius [M]).
    """
    K = np.asarray(K, dtype=np.float64)
    N, d = K.shape
    M = n_blocks(N, block)
    centroid = np.zeros((M, d), dtype=np.float64)
    radius = np.zeros(M, dtype=np.float64)
    for b in range(M):
        keys = K[b * block:min(N, (b + 1) * block)]
        c = keys.sum(axis=0) / keys.shape[0]
        diff = keys - c
        dist = np.sqrt((diff * diff).sum(axis=1))
        centroid[b] = c
        radius[b] = dist.max()
    return centroid, radius


def quantile_linear(values: np.ndarray, p: float) -> float:
    """quantile(r, p) with linear interpolation at position p*(M-1) of the sorted values."""
    s = np.sort(np.asarray(values, dtype=np.float64))
    M = s.shape[0]
    x = p * (M - 1)
    lo = int(math.floor(x))
    hi = min(lo + 1, M - 1)
    return float(s[lo] + (x - lo) * (s[hi] - s[lo]))


def rescue_coefficient(radius: np.ndarray, p_low: float = P_LOW, p_high: float = P_HIGH):
    """beta_b = clamp((r_b - r_low) / (r_high - r_low), 0, 1)   (Eq. beta).

    r_low / r_high are the p_low / p_high quantiles of this head's block radii.
    Returns (beta [M], r_low, r_high).  r_high <= r_low gives beta = 0.
    """
    radius = np.asarray(radius, dtype=np.float64)
    r_low = quantile_linear(radius, p_low)
    r_high = quantile_linear(radius, p_high)
    if r_high > r_low:
        beta = np.clip((radius - r_low) / (r_high - r_low), 0.0, 1.0)
    else:
        beta = np.zeros_like(radius)
    return beta, r_low, r_high


# --------------------------------------------------------------------------------------
# Sec. 3.2: branch logits, aggregation, thresholds, union
# --------------------------------------------------------------------------------------
def branch_logits(Qi: np.ndarray, centroid: np.ndarray, radius: np.ndarray, beta: np.ndarray):
    """Unscaled branch logits of every token of one query block against candidate blocks.

    l_base(q, b)   = q . c_b                      (Eq. base_score)
    l_rescue(q, b) = q . c_b + ||q||_2 r_b beta_b (Eq. rescue_score)
    Qi [T, d]; centroid [nb, d]; radius, beta [nb].  Returns (l_base, l_rescue), each [T, nb].
    """
    Qi = np.asarray(Qi, dtype=np.float64)
    l_base = Qi @ np.asarray(centroid, dtype=np.float64).T
    q_norm = np.sqrt((Qi * Qi).sum(axis=1))
    l_rescue = l_base + q_norm[:, None] * (np.asarray(radius) * np.asarray(beta))[None, :]
    return l_base, l_rescue


def aggregate(logits: np.ndarray, d: int) -> np.ndarray:
    """S_{i,b} = sum_t exp(l(q_t, b)/sqrt(d) - m_i),  m_i = max over b and t  (Eq. block_aggregation)."""
    z = logits / math.sqrt(d)
    m = z.max()
    return np.exp(z - m).sum(axis=0)


def aggregate_local_lse(logits: np.ndarray, d: int) -> np.ndarray:
    """The "local log-sum-exp" form the paper mentions after Eq. block_aggregation:
    per-block LSE over the tokens, returned in the log domain (no common shift)."""
    z = logits / math.sqrt(d)
    mb = z.max(axis=0)
    return mb + np.log(np.exp(z - mb[None, :]).sum(axis=0))


def threshold_branch(S: np.ndarray, alpha: float) -> np.ndarray:
    """{b : S_b >= alpha * max_b' S_b'}   (Eq. branch_thresholds)."""
    return S >= alpha * S.max()


def forced_blocks(i: int, M: int, n_sink: int, n_local: int, n_recent: int) -> np.ndarray:
    """M^{sink/window/last}_i as a bool vector over b = 0..i (Sec. 3.2, after the union equation)."""
    b = np.arange(i + 1)
    forced = (b < n_sink) | (b > i - n_local)
    if i >= M - n_recent:
        forced = np.ones(i + 1, dtype=bool)
    return forced


@dataclass
class HeadSelection:
    base: np.ndarray      # [M, M] bool, lower triangular
    rescue: np.ndarray    # [M, M] bool
    forced: np.ndarray    # [M, M] bool
    final: np.ndarray     # [M, M] bool = base | rescue | forced
    margin_base: np.ndarray    # [M, M] |S - alpha*max| / (alpha*max); +inf above the diagonal
    margin_rescue: np.ndarray  # [M, M]
    density: float        # Eq. actual_density for this head


def select_head(Q: np.ndarray, centroid: np.ndarray, radius: np.ndarray, beta: np.ndarray,
                block: int, alpha_base: float, alpha_rescue: float,
                n_sink: int, n_local: int, n_recent: int, rows=None) -> HeadSelection:
    """Algorithm 1, third loop, for ONE query head against its KV head's statistics.

    Q [N, d]; centroid [M, d]; radius, beta [M].  A short last query block aggregates over its own tokens.
    `rows` (optional) restricts the work to those query blocks; other rows stay empty and the
    returned density is then meaningless.
    """
    Q = np.asarray(Q, dtype=np.float64)
    N, d = Q.shape
    M = n_blocks(N, block)
    base = np.zeros((M, M), dtype=bool)
    rescue = np.zeros((M, M), dtype=bool)
    forced = np.zeros((M, M), dtype=bool)
    margin_base = np.full((M, M), np.inf)
    margin_rescue = np.full((M, M), np.inf)
    for i in (range(M) if rows is None else rows):
        Qi = Q[i * block:min(N, (i + 1) * block)]
        nb = i + 1  # causal candidates C_i = {0..i}
        l_base, l_rescue = branch_logits(Qi, centroid[:nb], radius[:nb], beta[:nb])
        S_base = aggregate(l_base, d)
        S_rescue = aggregate(l_rescue, d)
        base[i, :nb] = threshold_branch(S_base, alpha_base)
        rescue[i, :nb] = threshold_branch(S_rescue, alpha_rescue)
        forced[i, :nb] = forced_blocks(i, M, n_sink, n_local, n_recent)
        tb = alpha_base * S_base.max()
        tr = alpha_rescue * S_rescue.max()
        margin_base[i, :nb] = np.abs(S_base - tb) / tb
        margin_rescue[i, :nb] = np.abs(S_rescue - tr) / tr
    final = base | rescue | forced
    return HeadSelection(base, rescue, forced, final, margin_base, margin_rescue, density(final))


def density(final: np.ndarray) -> float:
    """rho = selected causal block pairs / all causal block pairs (Eq. actual_density)."""
    M = final.shape[0]
    causal = np.tril(np.ones((M, M), dtype=bool))
    return float((final & causal).sum()) / float(M * (M + 1) // 2)


def group_union(finals) -> np.ndarray:
    """Group-shared mask under grouped-query attention: a pair is kept for the whole KV group when any of the
    group's query heads keeps it.  `finals` are the [M, M] masks of the heads of one group.  (A variant: the
    paper's selector, Sec. 3.2, is per query head and has no such step.)"""
    out = np.zeros_like(np.asarray(finals[0], dtype=bool))
    for f in finals:
        out = out | np.asarray(f, dtype=bool)
    return out


# --------------------------------------------------------------------------------------
# Sec. 3.3: attention over the retained blocks; Eq. (1): dense causal attention
# --------------------------------------------------------------------------------------
def masked_attention_block(Q: np.ndarray, K: np.ndarray, V: np.ndarray, selected: np.ndarray,
                           i: int, block: int, scale: float | None = None):
    """Output rows of query block i when only key blocks {b <= i : selected[b]} are retained.

    Token t attends to keys j <= t inside retained blocks; softmax is normalised over those
    keys only (Sec. 3.3).  A token with no retained key gets a zero row and lse = -inf.
    Q, K, V: [N, d] of one (query head, its KV head).  Returns (O [T, d], lse [T]).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N, d = Q.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    t0, t1 = i * block, min(N, (i + 1) * block)
    O = np.zeros((t1 - t0, V.shape[1]), dtype=np.float64)
    lse = np.full(t1 - t0, -np.inf)
    blocks = [b for b in range(i + 1) if selected[b]]
    if not blocks:
        return O, lse
    key_idx = np.concatenate([np.arange(b * block, min(N, (b + 1) * block)) for b in blocks])
    s = (Q[t0:t1] @ K[key_idx].T) * scale
    tok = np.arange(t0, t1)
    visible = key_idx[None, :] <= tok[:, None]          # causal mask inside retained tiles
    s = np.where(visible, s, -np.inf)
    has_key = visible.any(axis=1)
    m = np.where(has_key, s.max(axis=1), 0.0)
    p = np.exp(s - m[:, None])                          # exp(-inf) = 0 for hidden keys
    denom = p.sum(axis=1)
    pv = p @ V[key_idx]
    O[has_key] = pv[has_key] / denom[has_key, None]
    lse[has_key] = m[has_key] + np.log(denom[has_key])
    return O, lse


def dense_causal_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float | None = None):
    """Eq. (1), token by token; never looks at a mask.  Q, K, V [N, d]. Returns (O, lse)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N, d = Q.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    O = np.zeros((N, V.shape[1]), dtype=np.float64)
    lse = np.zeros(N, dtype=np.float64)
    for t in range(N):
        s = (K[:t + 1] @ Q[t]) * scale
        m = s.max()
        p = np.exp(s - m)
        denom = p.sum()
        O[t] = (p @ V[:t + 1]) / denom
        lse[t] = m + math.log(denom)
    return O, lse


# --------------------------------------------------------------------------------------
# App. D: the two geometric upper bounds (used by the worked-example pins)
# --------------------------------------------------------------------------------------
def l2_upper_bound(q: np.ndarray, keys: np.ndarray) -> float:
    """U^L2(q) = q.c + ||q||_2 r   (Eq. full_l2_bound)."""
    c, r = block_stats(np.asarray(keys, dtype=np.float64), len(keys))
    q = np.asarray(q, dtype=np.float64)
    return float(q @ c[0] + math.sqrt(float(q @ q)) * r[0])


def box_upper_bound(q: np.ndarray, keys: np.ndarray) -> float:
    """U^box(q) = sum_j max(q_j a_j, q_j u_j), a/u the per-coordinate min/max (Eq. quest_box)."""
    keys = np.asarray(keys, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    a = keys.min(axis=0)
    u = keys.max(axis=0)
    return float(np.maximum(q * a, q * u).sum())


# --------------------------------------------------------------------------------------
# Sec. 4.2 / App. D.2: the Quest-style comparison selector
# --------------------------------------------------------------------------------------
def box_stats(K: np.ndarray, block: int):
    """a_b = per-coordinate minimum, u_b = per-coordinate maximum of the block's keys (App. D.2).
    K [N, d] of one KV head.  Returns (lo [M, d], hi [M, d])."""
    K = np.asarray(K, dtype=np.float64)
    N, d = K.shape
    M = n_blocks(N, block)
    lo = np.zeros((M, d))
    hi = np.zeros((M, d))
    for b in range(M):
        keys = K[b * block:min(N, (b + 1) * block)]
        lo[b] = keys.min(axis=0)
        hi[b] = keys.max(axis=0)
    return lo, hi


def box_logits(Qi: np.ndarray, lo: np.ndarray, hi: np.ndarray) -> np.ndarray:
    """U_b^box(q) = sum_j max(q_j a_bj, q_j u_bj) for every token of Qi [T, d] and block (Eq. quest_box),
    coordinate by coordinate as printed.  Returns [T, nb]."""
    Qi = np.asarray(Qi, dtype=np.float64)
    out = np.zeros((Qi.shape[0], lo.shape[0]))
    for b in range(lo.shape[0]):
        out[:, b] = np.maximum(Qi * lo[b][None, :], Qi * hi[b][None, :]).sum(axis=1)
    return out


def top_fraction(S: np.ndarray, delta: float) -> np.ndarray:
    """Keeps the ceil(delta * n) largest of the n scores; scores equal to the last kept one are kept too."""
    n = S.shape[0]
    k = min(n, max(1, int(math.ceil(delta * n))))
    kth = np.sort(S)[n - k]
    return S >= kth


@dataclass
class BoxSelection:
    chosen: np.ndarray    # [M, M] bool: the density-parameter choice alone
    forced: np.ndarray    # [M, M] bool
    final: np.ndarray     # [M, M] bool = chosen | forced
    margin: np.ndarray    # [M, M] |S - S_kth| / S_kth, the k-th largest score of the row; +inf above the diagonal
    density: float


def select_head_box(Q: np.ndarray, lo: np.ndarray, hi: np.ndarray, block: int, delta: float,
                    n_sink: int, n_local: int, n_recent: int, rows=None) -> BoxSelection:
    """Quest-style selection for ONE query head against its KV head's boxes (see the module header for the
    reading): S_{i,b} = sum_t exp(U_b^box(q_t)/sqrt(d) - m_i), keep the ceil(delta (i + 1)) best b <= i."""
    Q = np.asarray(Q, dtype=np.float64)
    N, d = Q.shape
    M = n_blocks(N, block)
    chosen = np.zeros((M, M), dtype=bool)
    forced = np.zeros((M, M), dtype=bool)
    margin = np.full((M, M), np.inf)
    for i in (range(M) if rows is None else rows):
        Qi = Q[i * block:min(N, (i + 1) * block)]
        nb = i + 1
        S = aggregate(box_logits(Qi, lo[:nb], hi[:nb]), d)
        chosen[i, :nb] = top_fraction(S, delta)
        forced[i, :nb] = forced_blocks(i, M, n_sink, n_local, n_recent)
        k = min(nb, max(1, int(math.ceil(delta * nb))))
        kth = np.sort(S)[nb - k]
        margin[i, :nb] = np.abs(S - kth) / kth
    final = chosen | forced
    return BoxSelection(chosen, forced, final, margin, density(final))


# --------------------------------------------------------------------------------------
# Algorithm 1 end to end, GQA layout [L, N, H, d]
# --------------------------------------------------------------------------------------
@dataclass
class PrefillReference:
    centroid: np.ndarray  # [L, Hkv, M, d]
    radius: np.ndarray    # [L, Hkv, M]
    beta: np.ndarray      # [L, Hkv, M]
    rq: np.ndarray        # [L, Hkv, 2]  (r_low, r_high)
    selection: list       # [L][Hq] of HeadSelection
    density: np.ndarray   # [L, Hq]


def stats_all(K: np.ndarray, block: int):
    """Block statistics and rescue coefficients for K [L, N, Hkv, d] (Algorithm 1, loops 1-2)."""
    L, N, Hkv, d = K.shape
    M = n_blocks(N, block)
    centroid = np.zeros((L, Hkv, M, d))
    radius = np.zeros((L, Hkv, M))
    beta = np.zeros((L, Hkv, M))
    rq = np.zeros((L, Hkv, 2))
    for l in range(L):
        for hk in range(Hkv):
            c, r = block_stats(K[l, :, hk, :], block)
            bt, lo, hi = rescue_coefficient(r)
            centroid[l, hk], radius[l, hk], beta[l, hk], rq[l, hk] = c, r, bt, (lo, hi)
    return centroid, radius, beta, rq


def select_all(Q: np.ndarray, K: np.ndarray, block: int, alpha_base: float, alpha_rescue: float,
               n_sink: int, n_local: int, n_recent: int, heads=None) -> PrefillReference:
    """Statistics + selection for every (l, query head) (or the listed `heads` only)."""
    L, N, Hq, d = Q.shape
    Hkv = K.shape[2]
    G = Hq // Hkv
    centroid, radius, beta, rq = stats_all(K, block)
    sel = [[None] * Hq for _ in range(L)]
    dens = np.full((L, Hq), np.nan)
    for l in range(L):
        for h in (range(Hq) if heads is None else heads):
            hk = h // G
            sel[l][h] = select_head(Q[l, :, h, :], centroid[l, hk], radius[l, hk], beta[l, hk], block,
                                    alpha_base, alpha_rescue, n_sink, n_local, n_recent)
            dens[l, h] = sel[l][h].density
    return PrefillReference(centroid, radius, beta, rq, sel, dens)
