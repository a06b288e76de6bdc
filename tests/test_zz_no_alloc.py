"""The allocation-free LayerNorm entry point gives the same bytes as the ordinary one.

Collected last on purpose (file name): if it failed, a run that stops at the first failure has
already exercised everything else.  Two calls in a row check that what the first call left in the
library's fixed device array does not leak into the second."""
import numpy as np
import pytest
import torch

from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import binding, synth

pytestmark = pytest.mark.gpu


def test_static_layernorm_matches_the_allocating_entry_point_twice():
    torch.cuda.set_device(0)
    cases = [(64, 768, 1.0, True), (33, 1024, 4.0, True)]       # second call: other C, scales, tables
    for rows, C, sigma, residual in cases:
        q, S, r, S_r, gamma, beta, S_out = synth.layernorm_inputs(rows, C, sigma, with_residual=residual)
        qd, rd = dev(q), dev(r)
        want, _ = ctx().ibert_layernorm_i(qd, S, rd, S_r, gamma, beta, S_out)
        ctx().check()
        got, S_ret = binding.ibert_layernorm_i_static(qd, S, rd, S_r, gamma, beta, S_out)
        torch.cuda.synchronize()
        assert S_ret == S_out
        assert_same(host(got), host(want), f"static layernorm C={C}")
    # sizes beyond the fixed tables are refused, not truncated
    with pytest.raises(binding.IbertError) as e:
        binding.ibert_layernorm_i_static(torch.zeros((1, 2048), dtype=torch.int32, device="cuda"), 1e-3, None, 0.0,
                                         np.ones(2048), np.zeros(2048), 0.02)
    assert e.value.code == -2
