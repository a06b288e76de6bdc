"""A bounded device-side wait that actually runs out: the kernel returns normally, the status
word reads IBERT_ERR_TIMEOUT once, and the context keeps working afterwards."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import binding, synth

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_leaves_the_context_usable():
    c = ctx()
    c.check()
    c.ibert_selftest_wait_timeout(2000)                  # 2 ms on the GPU's timer
    assert c.ibert_last_status() == -7                   # IBERT_ERR_TIMEOUT
    assert c.ibert_last_status() == 0                    # reported once, then cleared
    # the same context, right after: a real operator still matches the oracle
    q, S, S_out = synth.gelu_inputs(4096 + 3, 1.0)
    got, _ = c.ibert_gelu_i(dev(q), S, S_out)
    c.check()
    want, _ = oracle.gelu(q, S, S_out)
    assert_same(host(got), want, "i-GELU after an expired wait")


def test_wait_limit_is_validated():
    c = ctx()
    for bad in (0, -5, 10 ** 6):
        with pytest.raises(binding.IbertError) as e:
            c.ibert_selftest_wait_timeout(bad)
        assert e.value.code == -1
    assert c.ibert_last_status() == 0
