"""The selector diagnostics report (Sec. 2, Fig. 1 as read by oracle/diagnostics.py) on a small synthetic head: checks
what must hold whatever the data -- the mass ranking is the ceiling, coverage grows with the budget, masses and shares
are distributions -- and the one thing the synthetic recipe plants: needle blocks have large radii and attract mass."""
import numpy as np

from oracle import diagnostics as dg
from oracle import rbs_oracle as orc
from paper_2609_20971_b200.synth import SynthConfig, make_inputs, to_f64


def test_report_invariants_on_a_small_head():
    cfg = SynthConfig("diag", N=64 * 60, Hq=2, Hkv=1, B=64, sigma=0.4, p_needle=0.15, seed=17)
    Q, K, _ = make_inputs(cfg)
    Q64, K64 = to_f64(Q[0, :, 1]), to_f64(K[0, :, 0])
    mass = dg.block_attention_mass(Q64, K64, 37, cfg.B)
    assert mass.shape == (38,) and abs(mass.sum() - 1.0) < 1e-12 and np.all(mass >= 0)
    # against the oracle's attention: the mass of one block equals the softmax weight the dense routine gives its keys
    t = 37 * cfg.B + 5
    s = (K64[:t + 1] @ Q64[t]) / np.sqrt(cfg.d)
    p = np.exp(s - s.max()); p /= p.sum()
    per_tok = np.array([p[b * cfg.B:(b + 1) * cfg.B].sum() for b in range(38)])
    tok_mass = np.zeros(38)
    for tt in range(37 * cfg.B, 38 * cfg.B):
        ss = (K64[:tt + 1] @ Q64[tt]) / np.sqrt(cfg.d)
        pp = np.exp(ss - ss.max()); pp /= pp.sum()
        tok_mass += np.array([pp[b * cfg.B:(b + 1) * cfg.B].sum() for b in range(38)])
    assert np.allclose(mass, tok_mass / cfg.B, atol=1e-12) and per_tok.sum() > 0.999
    rows = list(range(30, 60, 3))
    rep = dg.report(Q64, K64, cfg.B, rows)
    budgets = sorted(rep["coverage"]["ceiling"], key=float)
    for name, per in rep["coverage"].items():
        vals = [per[b] for b in budgets]
        assert all(0.0 <= v <= 1.0 + 1e-12 for v in vals) and all(a <= b + 1e-12 for a, b in zip(vals, vals[1:]))
        assert all(per[b] <= rep["coverage"]["ceiling"][b] + 1e-12 for b in budgets)      # nothing beats the ceiling
    share = np.array(rep["top_share_by_radius_quintile"])
    assert abs(share.sum() - 1.0) < 1e-12 and share[4] > 0.2          # the planted needles sit in the top radius quintile
    for name, m in rep["missed_top_by_radius_quintile"].items():
        assert all(0.0 <= v <= 1.0 for v in m)
