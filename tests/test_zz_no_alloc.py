"""The LayerNorm entry point that allocates no device memory, against the CPU oracle and against
the ordinary entry point.

Collected last on purpose (file name): if it failed, a run that stops at the first failure has
already exercised everything else.  Consecutive calls with different widths, scales and tables
check that what one call left in the library's fixed device array does not leak into the next."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import binding, synth

pytestmark = pytest.mark.gpu

# (rows, C, sigma, residual): a vector-friendly width twice in a row with other tables, the
# largest width the fixed array takes, widths that are not multiples of 16 or of 4, no residual
CASES = [(64, 768, 1.0, True), (33, 1024, 4.0, True), (9, 2047, 1.0, True), (17, 770, 1.0, True),
         (5, 771, 4.0, True), (40, 768, 1.0, False), (3, 2047, 4.0, False)]


def test_static_layernorm_matches_the_oracle_and_the_allocating_entry_point():
    torch.cuda.set_device(0)
    for rows, C, sigma, residual in CASES:
        q, S, r, S_r, gamma, beta, S_out = synth.layernorm_inputs(rows, C, sigma, with_residual=residual)
        qd = dev(q)
        rd = dev(r) if residual else None
        got, S_ret = binding.ibert_layernorm_i_static(qd, S, rd, S_r, gamma, beta, S_out)
        torch.cuda.synchronize()
        assert S_ret == S_out
        want, _ = oracle.layernorm(q, S, r, S_r or 0.0, gamma, beta, S_out)
        assert_same(host(got), want, f"static layernorm vs oracle, C={C} residual={residual}")
        same, _ = ctx().ibert_layernorm_i(qd, S, rd, S_r, gamma, beta, S_out)
        ctx().check()
        assert_same(host(got), host(same), f"static layernorm vs ibert_layernorm_i, C={C}")
    assert binding.ibert_layernorm_i_static_status() == 0


def test_static_layernorm_refuses_what_its_fixed_array_cannot_hold():
    torch.cuda.set_device(0)
    with pytest.raises(binding.IbertError) as e:
        binding.ibert_layernorm_i_static(torch.zeros((1, 2048), dtype=torch.int32, device="cuda"), 1e-3, None, 0.0,
                                         np.ones(2048), np.zeros(2048), 0.02)
    assert e.value.code == -2
