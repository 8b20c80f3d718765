"""The bounded device-side waits and the sticky status word, exercised without faulting or hanging anything:
a one-warp kernel waits, with a short limit, on a barrier that nothing arrives on; the wait runs out and the
kernel returns with the status word set."""
import numpy as np
import pytest
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200 import binding
from paper_2609_33586_b200.inputs import Workload, make_inputs

from parity_util import compare

pytestmark = pytest.mark.gpu

TIMEOUT = -7      # ATTN_ERR_TIMEOUT
SELFTEST_CODE = (7 << 8) | 0x7F


def test_an_expired_wait_sets_the_sticky_word_and_later_launches_store_nothing_until_reset():
    binding.device_status_reset()
    assert binding.device_status() == 0 and binding.device_status_code() == 0
    try:
        binding.selftest_wait(2_000_000)                       # about a millisecond
        assert binding.device_status() == TIMEOUT
        assert binding.device_status_code() == SELFTEST_CODE
        assert "wait" in binding.status_string(TIMEOUT)

        wl = Workload("after_timeout", 1, 2, 2, 300, 300, 128, True, "bf16", 81)
        inp = make_inputs(wl)
        q, k, v = inp.q.cuda(), inp.k.cuda(), inp.v.cuda()
        out = torch.full((wl.B, wl.Sq, wl.Hq, wl.D), 7.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.full((wl.B, wl.Hq, wl.Sq), -3.0, dtype=torch.float32, device="cuda")
        # the word is sticky: the call itself reports success (it is asynchronous), the kernel stores nothing
        binding.attn_fwd(q, k, v, causal=True, softmax_scale=wl.softmax_scale, weight_mode=orc.W_H15, out=out, lse=lse)
        torch.cuda.synchronize()
        assert torch.all(out == 7.0) and torch.all(lse == -3.0)
        assert binding.device_status() == TIMEOUT and binding.device_status_code() == SELFTEST_CODE   # the first code is kept
        # a second expiry does not replace the first code
        binding.selftest_wait(1_000)
        assert binding.device_status_code() == SELFTEST_CODE
    finally:
        binding.device_status_reset()
    assert binding.device_status() == 0
    # after the reset everything works again
    st = compare(wl, orc.W_H15, inp)
    assert st["ok"], st
    assert binding.device_status() == 0


def test_selftest_limits_are_checked():
    assert binding.lib().attn_selftest_wait(0, None) == -9
    assert binding.lib().attn_selftest_wait(3_000_000_000, None) == -9
    assert binding.device_status() == 0
