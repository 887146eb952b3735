"""What happens when a device-side wait runs out (needs a B200).

Every wait of the tcgen05 kernels is bounded: on expiry the kernel records LSA_ERR_TIMEOUT in the context's status
word, every other wait of the launch sees the word and stops, and the kernel ends normally.  The expiry is provoked
here in the one way that harms nothing: lsa_selftest_wait launches a block that waits, with a short budget, on a
barrier nobody arrives on.  No production kernel's budget is shortened and nothing faults or hangs.
"""
import pytest
import torch

from paper_2608_01662_b200.configs import CONFIGS
from paper_2608_01662_b200.workload import DecodeWorkload, PrefillWorkload

import parity_util as pu

pytestmark = pytest.mark.gpu

LSA_ERR_TIMEOUT = -5


def test_expired_wait_is_reported_and_the_context_recovers(cuda_device):
    cfg = CONFIGS["cfg3"].replace(name="fd_prefill", L=3000, M=8, Ksp=256, W=256, R=1, seed=31)
    wl = PrefillWorkload(cfg, cuda_device)
    wl.prepare()
    wl.step()
    assert wl.ctx.status() == 0
    idx0, out0 = wl.sparse_idx.clone(), wl.out[0].clone()

    wl.ctx.selftest_wait(1_000_000)                  # about half a millisecond of SM clock
    assert wl.ctx.status() == LSA_ERR_TIMEOUT        # reported ...
    assert wl.ctx.status() == 0                      # ... and cleared by the read

    # the word was raised while later launches were already queued: they give up at once and say so
    wl.ctx.selftest_wait(1_000_000)
    wl.step()
    assert wl.ctx.status() == LSA_ERR_TIMEOUT

    # after the status has been read the same context computes the same bits as before
    wl.sparse_idx.fill_(-9)
    wl.out[0].zero_()
    wl.step()
    assert wl.ctx.status() == 0
    assert torch.equal(wl.sparse_idx, idx0) and torch.equal(wl.out[0], out0)


def test_decode_context_recovers_after_an_expired_wait(cuda_device):
    cfg = CONFIGS["cfg4"].replace(name="fd_decode", batch=6, ctx_lo=1500, ctx_hi=6000, M=16, Ksp=512, R=2, seed=33)
    wl = DecodeWorkload(cfg, cuda_device)
    wl.prepare()
    wl.ctx.selftest_wait(200_000)
    assert wl.ctx.status() == LSA_ERR_TIMEOUT
    wl.step()
    assert wl.ctx.status() == 0
    m = pu.check_decode(wl, range(cfg.batch))
    m.assert_ok(pu.TOL_FP8)


def test_selftest_budget_is_checked_on_the_host(cuda_device):
    from paper_2608_01662_b200 import binding
    cfg = CONFIGS["cfg1"]
    wl = PrefillWorkload(cfg, cuda_device)
    for bad in (-1, (1 << 31) + 1):
        with pytest.raises(binding.LsaError) as e:
            wl.ctx.selftest_wait(bad)
        assert e.value.code == -1
    assert wl.ctx.status() == 0
