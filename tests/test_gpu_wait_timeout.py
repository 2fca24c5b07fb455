"""The bounded device-side waits: a wait that nothing ever satisfies gives up after its limit, the kernel returns, the
host reads FALQON_ERR_TIMEOUT from the status word, and the context is still usable.  Nothing here faults, traps or
hangs: the self-test kernel is one warp that polls a barrier for 20 ms and returns."""
import time

import numpy as np
import pytest
import torch

from helpers import u8
from paper_2510_24061_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    from paper_2510_24061_b200 import binding as fq
    from oracle import falqon_oracle as orc
    assert fq.last_device_status() == 0
    t0 = time.perf_counter()
    assert fq.lib.falqon_selftest_wait_timeout(20, None) == fq.OK
    assert fq.last_device_status() == fq.ERR_TIMEOUT              # synchronises, reads and clears the status word
    waited = time.perf_counter() - t0
    assert 0.015 < waited < 1.0, waited                           # it waited for its limit, not for the 2 s default
    assert fq.last_device_status() == 0                           # reported once
    x = synth.activations(3, 0, 64, 256, 2)
    codes, scale, _ = fq.quantize(x.to(DEV), fq.E4M3)             # and the library works as before
    q, s, _ = orc.quantize(x.float().numpy(), orc.E4M3)
    assert np.array_equal(u8(codes), q) and np.float32(scale.item()) == s
    assert fq.last_device_status() == 0
    assert fq.lib.falqon_selftest_wait_timeout(0, None) == fq.ERR_INVALID_ARG
    assert fq.lib.falqon_selftest_wait_timeout(5000, None) == fq.ERR_INVALID_ARG
