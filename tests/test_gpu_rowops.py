"""GPU parity (bit-exact) of the standalone integer non-linearities against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [0, 1, 3, 5, 1000, 4096, 128 * 128 * 7 + 2, (1 << 20) + 3])
@pytest.mark.parametrize("sigma", [1.0, 4.0])
def test_gelu_matches_oracle(n, sigma):
    q, S, S_out = synth.gelu_inputs(max(n, 1), sigma)
    q = q[:n]
    out, S_ret = ctx().ibert_gelu_i(dev(q), S, S_out)
    ctx().check()
    want, _ = oracle.gelu(q, S, S_out)
    assert S_ret == S_out
    assert_same(host(out), want, "gelu")


def test_gelu_full_int32_range_and_odd_scales():
    rng = np.random.default_rng(3)
    q = np.concatenate([rng.integers(-2 ** 31, 2 ** 31, 50000), np.arange(-40000, 40000),
                        [2 ** 31 - 1, -2 ** 31, 0, 32767, -32767, 32768, -32768]]).astype(np.int32)
    for S, S_out in [(1e-3, 4 / 127), (1.2207e-4, 0.031), (1.5e-4, 0.002), (0.05, 1.0), (3e-6, 1e-3), (2.0, 0.5)]:
        out, _ = ctx().ibert_gelu_i(dev(q), S, S_out)
        want, _ = oracle.gelu(q, S, S_out)
        assert_same(host(out), want, f"gelu S={S}")
    ctx().check()


@pytest.mark.parametrize("rows,L", [(5, 1), (9, 7), (33, 64), (17, 65), (96 * 8, 128), (64, 256), (40, 512),
                                    (7, 1000), (12, 1024), (3, 130), (0, 128),
                                    (6, 4), (1, 128), (1027, 100), (2, 124)])   # short rows: four rows per warp
@pytest.mark.parametrize("p_max", [255, 127])
def test_softmax_matches_oracle(rows, L, p_max):
    for sigma in (1.0, 4.0):
        q, S = synth.softmax_inputs(max(rows, 1), L, sigma)
        q = q[:rows]
        out, S_ret = ctx().ibert_softmax_i(dev(q), S, p_max)
        ctx().check()
        assert S_ret == 1.0 / p_max
        if rows:
            want, _ = oracle.softmax(q, S, p_max)
            assert_same(host(out), want, f"softmax L={L}")


@pytest.mark.parametrize("rows,L", [(9, 7), (96 * 8, 128), (40, 512), (12, 1024), (3, 130)])
def test_softmax_with_exp_by_table_equals_the_integer_kernel(rows, L):
    """The table holds the integer function's own values, so the comparison variant agrees bit for bit."""
    for sigma, p_max in ((1.0, 255), (4.0, 127)):
        q, S = synth.softmax_inputs(rows, L, sigma)
        a, _ = ctx().ibert_softmax_lut_i(dev(q), S, p_max)
        ctx().check()
        assert_same(host(a), oracle.softmax(q, S, p_max)[0], f"softmax by table L={L}")
    rng = np.random.default_rng(L)
    q = rng.integers(-2 ** 31, 2 ** 31, (rows, L)).astype(np.int32)
    q[0] = 3
    for S in (1e-3, 2e-5, 1e-8, 0.69):
        a, _ = ctx().ibert_softmax_lut_i(dev(q), S, 255)
        assert_same(host(a), oracle.softmax(q, S, 255)[0], f"softmax by table S={S}")
    ctx().check()


def test_softmax_extreme_inputs_and_scales():
    rng = np.random.default_rng(5)
    L = 96
    q = rng.integers(-2 ** 31, 2 ** 31, (64, L)).astype(np.int32)
    q[0] = 7
    q[1] = np.arange(L) - 2 ** 31
    q[2, :] = -2 ** 31
    q[2, 5] = 2 ** 31 - 1
    q[3] = rng.integers(-50, 50, L)
    q[4:20] = rng.integers(-3000, 3000, (16, L))
    for S in (1e-3, 4.5e-5, 2e-5, 1e-8, 0.3, 0.69, 3.3e-7):
        out, _ = ctx().ibert_softmax_i(dev(q), S, 255)
        want, _ = oracle.softmax(q, S, 255)
        assert_same(host(out), want, f"softmax S={S}")
    ctx().check()


@pytest.mark.parametrize("rows,C", [(3, 8), (5, 17), (64, 768), (33, 1024), (4, 2047), (2, 1), (9, 260), (0, 768),
                                    (7, 1536)])
@pytest.mark.parametrize("residual", [True, False])
def test_layernorm_matches_oracle(rows, C, residual):
    for sigma in (1.0, 4.0):
        q, S, r, S_r, gamma, beta, S_out = synth.layernorm_inputs(max(rows, 1), C, sigma, with_residual=residual)
        q = q[:rows]
        r = None if r is None else r[:rows]
        gamma = gamma.copy()
        gamma[::5] *= -1.0
        out, S_ret = ctx().ibert_layernorm_i(dev(q), S, None if r is None else dev(r), S_r, gamma, beta, S_out)
        ctx().check()
        assert S_ret == S_out
        if rows:
            want, _ = oracle.layernorm(q, S, r, S_r or 0.0, gamma, beta, S_out)
            assert_same(host(out), want, f"layernorm C={C}")


@pytest.mark.parametrize("rows,C", [(3, 8), (5, 17), (64, 768), (33, 1024), (4, 2047), (2, 1), (9, 260), (0, 768),
                                    (7, 1536), (300, 512), (11, 774)])
@pytest.mark.parametrize("residual", [True, False])
def test_layernorm_on_int16_q16_matches_oracle(rows, C, residual):
    """ibert_layernorm_i16: the same Q16 values in an int16 container (every kernel variant: streamed
    rows, register rows with and without vector loads) against the same oracle."""
    for sigma in (1.0, 4.0):
        q, S, r, S_r, gamma, beta, S_out = synth.layernorm_inputs(max(rows, 1), C, sigma, with_residual=residual)
        q = q[:rows]
        r = None if r is None else r[:rows]
        assert np.abs(q).max(initial=0) <= 32767
        gamma = gamma.copy()
        gamma[::7] *= -1.0
        out, S_ret = ctx().ibert_layernorm_i(dev(q.astype(np.int16)), S, None if r is None else dev(r), S_r, gamma, beta,
                                             S_out)
        ctx().check()
        assert S_ret == S_out
        if rows:
            want, _ = oracle.layernorm(q, S, r, S_r or 0.0, gamma, beta, S_out)
            assert_same(host(out), want, f"layernorm int16 C={C}")


def test_layernorm_degenerate_rows():
    C = 64
    q = np.zeros((6, C), dtype=np.int32)
    q[0] = 1234                      # constant row: sigma clamps to 1
    q[1, 0] = 2 ** 20                # largest allowed magnitude
    q[2] = np.where(np.arange(C) % 2 == 0, 2 ** 20, -2 ** 20)
    q[3, :] = 1
    q[3, 0] = 0
    q[4] = np.arange(C) - 32
    q[5] = -2 ** 20
    gamma = np.linspace(-1.5, 1.5, C)
    beta = np.linspace(-1.0, 1.0, C)
    out, _ = ctx().ibert_layernorm_i(dev(q), 1e-4, None, 0.0, gamma, beta, 0.02)
    want, _ = oracle.layernorm(q, 1e-4, None, 0.0, gamma, beta, 0.02)
    assert_same(host(out), want, "layernorm degenerate")
    ctx().check()


def test_rowops_error_codes_on_device_context():
    from paper_2101_01321_b200.binding import IbertError
    q = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(IbertError) as e:
        ctx().ibert_softmax_i(q, 0.7)                 # q_ln2 would be 0
    assert e.value.code == -3
    with pytest.raises(IbertError) as e:
        ctx().ibert_softmax_i(torch.zeros((1, 1025), dtype=torch.int32, device="cuda"), 1e-3)
    assert e.value.code == -2
    with pytest.raises(IbertError) as e:
        ctx().ibert_gelu_i(q, -1.0, 0.03)
    assert e.value.code == -3
    with pytest.raises(IbertError) as e:
        ctx().ibert_gelu_i(q.view(-1)[1:], 1e-3, 0.03)  # misaligned
    assert e.value.code == -4
    with pytest.raises(IbertError) as e:
        ctx().ibert_layernorm_i(torch.zeros((1, 2048), dtype=torch.int32, device="cuda"), 1e-3, None, 0.0,
                                np.ones(2048), np.zeros(2048), 0.02)
    assert e.value.code == -2
    assert ctx().ibert_last_status() == 0
