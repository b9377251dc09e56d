"""The bounded-wait path on a real GPU, in the one harmless form: a single thread waits with a short limit on a
barrier that nothing arrives on.  The wait must run out, report its code, leave the context usable, and the next
ordinary call must still match the oracle."""
import numpy as np
import pytest
import torch

from oracle import rbs_oracle as orc
from paper_2609_20971_b200 import rbs_block_stats, rbs_device_status
from paper_2609_20971_b200.binding import rbs_selftest_wait_timeout
from paper_2609_20971_b200.synth import SynthConfig, make_inputs, to_f64

pytestmark = pytest.mark.gpu

WAIT_SELFTEST_CODE = 7


def test_wait_that_runs_out_reports_and_leaves_the_context_usable():
    assert rbs_device_status(clear=True) == 0
    flag = rbs_selftest_wait_timeout(4096)
    torch.cuda.synchronize()
    assert int(flag.item()) == 1                               # the wait gave up and the kernel returned
    assert rbs_device_status(clear=False) == WAIT_SELFTEST_CODE    # reported, and kept until cleared
    assert rbs_device_status(clear=True) == WAIT_SELFTEST_CODE
    assert rbs_device_status(clear=True) == 0
    # an ordinary call afterwards: statistics against the oracle
    cfg = SynthConfig("after_timeout", N=128 * 9 + 5, Hq=2, Hkv=2, B=128, sigma=0.5, seed=90)
    _, K, _ = make_inputs(cfg)
    st = rbs_block_stats(K.cuda(), cfg.B)
    torch.cuda.synchronize()
    for hk in range(cfg.Hkv):
        c, r = orc.block_stats(to_f64(K[0, :, hk]), cfg.B)
        assert np.allclose(st.centroid[0, hk].cpu().numpy(), c, rtol=2e-5, atol=2e-6)
        assert np.allclose(st.radius[0, hk].cpu().numpy(), r, rtol=2e-5)
    assert rbs_device_status(clear=True) == 0
