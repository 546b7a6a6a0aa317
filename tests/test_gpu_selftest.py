"""The give-up branch of the library's bounded device waits, taken on purpose and safely.

Every wait of the streaming kernels on an asynchronous copy has a cycle limit; when it runs out the
kernel raises an abort flag, drains, sets KVC_FLAG_WAIT_EXPIRED and returns.  Normal runs never get
there.  kvc_selftest_wait_expiry makes one CTA wait, with a limit of a millisecond, on a barrier that
nothing arrives on: the wait must give up (no thread may report success), the flag must show in the
status word, and the next ordinary launch must run clean and correct on the same context.
"""
import numpy as np
import pytest
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

import helpers as hp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_bounded_wait_gives_up_sets_the_flag_and_leaves_the_context_usable():
    kvc.kvc_status_reset()
    assert kvc.kvc_status_poll() == 0
    succeeded, abort, cycles = kvc.kvc_selftest_wait_expiry(1.0)
    assert succeeded == 0 and abort == 1
    khz = 1_965_000                                         # B200: SM clock at most 1965 MHz
    assert 0.2 * khz <= cycles <= 50 * khz, cycles          # about a millisecond of SM cycles, not seconds
    assert kvc.kvc_status_poll() & kvc.KVC_FLAG_WAIT_EXPIRED
    kvc.kvc_status_reset()
    assert kvc.kvc_status_poll() == 0
    # the next ordinary launch on this context: a small apply through the tensor-core path, against the oracle
    cfg = wl.CONFIGS["llama8b_8k"].scaled(name="after_expiry", L=1, H=2, T=300)
    src_cpu = hp.make_cache(cfg)
    st_cpu = hp.make_state(cfg, 1)
    shift = 37
    _, ref_k, ref_v = orc.apply(hp.oracle_cache(src_cpu), hp.oracle_state(st_cpu), shift, hp.inv_freq(cfg), want_ref=True)
    dst = hp.empty_dst(src_cpu, cfg, DEV)
    kvc.kvc_apply(hp.to_dev(src_cpu, DEV), hp.state_to_dev(st_cpu, DEV), shift, kvc.Rope(cfg.theta), dst)
    torch.cuda.synchronize()
    assert kvc.kvc_status_poll() == 0
    for which, ref in (("k", ref_k), ("v", ref_v)):
        assert hp.tol_ratio(hp.logical_bits(dst, which), ref) <= 1.0


def test_selftest_rejects_unbounded_limits():
    for bad in (0.0, -1.0, 1e4):
        with pytest.raises(kvc.KvcError):
            kvc.kvc_selftest_wait_expiry(bad)
