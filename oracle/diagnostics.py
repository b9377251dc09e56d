"""Selector diagnostics of the paper's motivation figure (Sec. 2, Fig. 1) on synthetic inputs, from the fp64 oracle.

TEST INFRASTRUCTURE ONLY, like the rest of this package: a report for a reader, not part of the CUDA path.

The figure itself is not reproduced (its data are model activations on benchmark prompts); what it measures is:
  (a) attention-mass coverage at a given selected-block ratio: the share of a query block's dense causal attention mass
      that falls into the blocks a selector keeps when it may keep a fraction `budget` of the causal candidates,
      next to the ceiling reached by ranking blocks by that mass itself;
  (b) rank underestimation by radius quintile: of the blocks that are in the top 5 % by attention mass and lie in radius
      quintile Q, the share a selector ranks outside its own top 5 %;
  (c) where the top-5 % blocks lie: their share per radius quintile (20 % each if radius did not matter).
The paper does not print formulas for (a)-(c); these definitions are this module's reading of the captions.
Selectors are turned into rankings by the score they threshold: the centroid score S_base, the full-L2 score
(beta = 1), the box score, and for RBS the larger of its two branch scores each divided by its own threshold
alpha_z max S_z (a block is kept exactly when that ratio reaches 1, and scaling both thresholds by one factor moves
the budget along this ranking).
"""
from __future__ import annotations

import json
import math

import numpy as np

from . import rbs_oracle as orc


def block_attention_mass(Q: np.ndarray, K: np.ndarray, i: int, block: int) -> np.ndarray:
    """Mean over the tokens of query block i of the dense causal softmax mass that falls into each key block b <= i."""
    N, d = Q.shape
    t0, t1 = i * block, min(N, (i + 1) * block)
    s = (Q[t0:t1] @ K[:t1].T) / math.sqrt(d)
    tok = np.arange(t0, t1)
    s = np.where(np.arange(t1)[None, :] <= tok[:, None], s, -np.inf)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    nb = i + 1
    pad = nb * block - t1
    if pad:
        p = np.concatenate([p, np.zeros((p.shape[0], pad))], axis=1)
    return p.reshape(p.shape[0], nb, block).sum(axis=2).mean(axis=0)


def selector_scores(Qi: np.ndarray, stats: dict, nb: int, alpha_base: float, alpha_rescue: float) -> dict:
    """Ranking score of every candidate block b < nb under each selector."""
    d = Qi.shape[1]
    c, r, beta = stats["centroid"][:nb], stats["radius"][:nb], stats["beta"][:nb]
    lb, lr = orc.branch_logits(Qi, c, r, beta)
    _, lfull = orc.branch_logits(Qi, c, r, np.ones(nb))
    S_b, S_r = orc.aggregate(lb, d), orc.aggregate(lr, d)
    return {
        "centroid": S_b,
        "full_l2": orc.aggregate(lfull, d),
        "box": orc.aggregate(orc.box_logits(Qi, stats["lo"][:nb], stats["hi"][:nb]), d),
        "rbs": np.maximum(S_b / (alpha_base * S_b.max()), S_r / (alpha_rescue * S_r.max())),
    }


def report(Q: np.ndarray, K: np.ndarray, block: int, rows, budgets=(0.02, 0.05, 0.10, 0.20), top: float = 0.05,
           alpha_base: float = 0.22, alpha_rescue: float = 0.18) -> dict:
    """Diagnostics (a)-(c) for ONE (query head, KV head) pair, averaged over the query blocks `rows`."""
    Q, K = np.asarray(Q, np.float64), np.asarray(K, np.float64)
    c, r = orc.block_stats(K, block)
    beta, r_low, r_high = orc.rescue_coefficient(r)
    lo, hi = orc.box_stats(K, block)
    stats = dict(centroid=c, radius=r, beta=beta, lo=lo, hi=hi)
    quintile = np.minimum(4, (np.argsort(np.argsort(r)) * 5) // len(r))          # radius quintile of every block
    names = ["centroid", "full_l2", "box", "rbs"]
    cover = {n: {b: [] for b in budgets} for n in names + ["ceiling"]}
    top_in_q = np.zeros(5)
    missed = {n: np.zeros(5) for n in names}
    for i in rows:
        nb = i + 1
        mass = block_attention_mass(Q, K, i, block)
        scores = selector_scores(Q[i * block:min(len(Q), (i + 1) * block)], stats, nb, alpha_base, alpha_rescue)
        scores["ceiling"] = mass
        for n, s in scores.items():
            order = np.argsort(-s, kind="stable")
            for b in budgets:
                k = max(1, int(math.ceil(b * nb)))
                cover[n][b].append(float(mass[order[:k]].sum()))
        k = max(1, int(math.ceil(top * nb)))
        top_blocks = np.argsort(-mass, kind="stable")[:k]
        np.add.at(top_in_q, quintile[top_blocks], 1)
        for n in names:
            kept = set(np.argsort(-scores[n], kind="stable")[:k].tolist())
            for b in top_blocks:
                if int(b) not in kept:
                    missed[n][quintile[b]] += 1
    return {
        "rows": list(map(int, rows)), "blocks": int(len(r)), "r_low": r_low, "r_high": r_high,
        "coverage": {n: {str(b): float(np.mean(v)) for b, v in per.items()} for n, per in cover.items()},
        "top_share_by_radius_quintile": (top_in_q / max(1.0, top_in_q.sum())).tolist(),
        "missed_top_by_radius_quintile": {n: (missed[n] / np.maximum(1.0, top_in_q)).tolist() for n in names},
    }


def main():
    import argparse

    from paper_2609_20971_b200.synth import make_inputs, paper_configs, to_f64
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--workload", default="q30b_32k")
    ap.add_argument("--head", type=int, default=0)
    ap.add_argument("--rows", type=int, default=24, help="query blocks sampled evenly over the second half of the sequence")
    args = ap.parse_args()
    cfg = paper_configs()[args.workload]
    Q, K, _ = make_inputs(cfg)
    G = cfg.Hq // cfg.Hkv
    rows = sorted({int(x) for x in np.linspace(cfg.M // 2, cfg.M - 1, args.rows)})
    out = report(to_f64(Q[0, :, args.head]), to_f64(K[0, :, args.head // G]), cfg.B, rows,
                 alpha_base=cfg.alpha_base, alpha_rescue=cfg.alpha_rescue)
    out["workload"] = cfg.name
    print(json.dumps(out, indent=1))


if __name__ == "__main__":
    main()
