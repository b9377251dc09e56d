"""rbs_select_static: the selection entry point for callers that cannot allocate device memory (a serving
process that has already given every free byte to its own pools, a latency-critical path that cannot afford
the device-wide synchronisation of an allocation, a plug-in that is handed no allocator).  Its scratch is a
fixed array inside the library, so it must give exactly what rbs_select gives with a caller-owned workspace --
also on a second call, when the array still holds the first call's leftovers.

Collected last on purpose: a failure here cannot hide the outcome of any other test in a stop-at-first-failure
run.  It does not depend on the tests before it and passes in a fresh process as well."""
import ctypes

import pytest
import torch

from paper_2609_20971_b200 import binding, rbs_block_stats, rbs_select, rbs_select_static
from paper_2609_20971_b200.binding import RbsShape, RbsStats, RbsTensor
from paper_2609_20971_b200.synth import SynthConfig, make_inputs


@pytest.mark.gpu
def test_static_scratch_select_matches_workspace_select_on_two_calls_in_a_row():
    dev = torch.device("cuda:0")
    results = []
    # two different problems back to back: the second call finds the first one's centroids, g values and
    # pair counters in the shared array and must not be affected by them
    for cfg in (SynthConfig("na1", L=2, N=128 * 150, Hq=4, Hkv=2, B=128, sigma=(0.1, 1.0), seed=51),
                SynthConfig("na2", L=1, N=64 * 70, Hq=2, Hkv=1, B=64, sigma=0.4, seed=52, n_sink=2, n_local=2)):
        Q, K, _ = make_inputs(cfg)
        Qg, Kg = Q.to(dev), K.to(dev)
        stats = rbs_block_stats(Kg, cfg.B)
        want = rbs_select(Qg, stats, cfg.B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local, cfg.n_recent,
                          debug=True)
        beta_want, rq_want = stats.beta.clone(), stats.rq.clone()
        stats.beta.zero_(); stats.rq.zero_()
        mask = torch.full_like(want[0], -1)
        dens = torch.full_like(want[1], -1.0)
        db, dr = torch.full_like(want[0], -1), torch.full_like(want[0], -1)
        rbs_select_static(Qg, stats, cfg.B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local, cfg.n_recent,
                          mask=mask, density=dens, dbg_base=db, dbg_rescue=dr)
        torch.cuda.synchronize()
        # integer work is bit-exact; density is the same exact bookkeeping; beta / quantiles identical
        assert torch.equal(mask, want[0]) and torch.equal(db, want[2]) and torch.equal(dr, want[3])
        assert torch.equal(dens, want[1])
        assert torch.equal(stats.beta, beta_want) and torch.equal(stats.rq, rq_want)
        results.append(float(dens.mean()))
        # the property the entry point exists for: a call (after the device's first one) takes no device memory --
        # the driver reports the same free bytes before and after, with nothing handed back in between
        free_before, _ = torch.cuda.mem_get_info(dev)
        rbs_select_static(Qg, stats, cfg.B, cfg.alpha_base, cfg.alpha_rescue, cfg.n_sink, cfg.n_local, cfg.n_recent,
                          mask=mask, density=dens, dbg_base=db, dbg_rescue=dr)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(dev)
        assert free_after == free_before
        assert torch.equal(mask, want[0]) and torch.equal(dens, want[1])
    assert all(0.0 < r <= 1.0 for r in results)


def test_static_scratch_select_rejects_shapes_beyond_its_fixed_array():
    # pure host-side check: returns before any CUDA call, so it also runs on a machine without a GPU
    from paper_2609_20971_b200.build import build_library
    build_library()
    lib = binding.load_library()
    big = RbsShape(8, 131072, 64, 8, 128, 64)          # 8 x 8 x 2048 centroid rows: 16x the array
    assert lib.rbs_workspace_bytes(1, ctypes.byref(big)) > binding.SELECT_STATIC_SCRATCH_BYTES
    p = ctypes.c_void_p(0x1000)
    code = lib.rbs_select_static(ctypes.byref(big), RbsTensor(0x1000, 0, 128, 128), RbsStats(0x1000, 0x1000, 0x1000, 0x1000),
                                 0.22, 0.18, 1, 1, 1, p, p, None, None, None)
    assert code == 3 and lib.rbs_status_string(code) == b"RBS_ERR_WORKSPACE"
    fits = RbsShape(1, 131072, 32, 4, 128, 128)
    assert lib.rbs_workspace_bytes(1, ctypes.byref(fits)) <= binding.SELECT_STATIC_SCRATCH_BYTES
