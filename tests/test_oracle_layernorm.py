"""Pins for the oracle's i-LayerNorm with residual (Sec. 3.6, Eq. 16, Algorithm 4)."""
import numpy as np
import pytest

import oracle


def float_layernorm_int8(q, S, r, S_r, gamma, beta, S_out):
    x = q.astype(np.float64) * S
    if r is not None:
        x = x + r.astype(np.float64) * S_r
    mu = x.mean(axis=1, keepdims=True)
    sd = x.std(axis=1, ddof=0, keepdims=True)
    y = (x - mu) / sd * gamma + beta
    return np.clip(np.rint(y / S_out), -127, 127)


def _make(rows, C, seed, sigma=1.0, residual=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((rows, C)) * sigma + rng.standard_normal((rows, 1)) * sigma / 2
    res = rng.standard_normal((rows, C)) * sigma / 4 if residual else None
    tot = x + (res if residual else 0.0)
    S = np.abs(tot).max() / 32767.0
    q = np.rint(x / S).astype(np.int32)
    r = S_r = None
    if residual:
        S_r = np.abs(res).max() / 127.0
        r = np.rint(res / S_r).astype(np.int8)
    gamma = 1.0 + 0.1 * rng.standard_normal(C)
    beta = 0.1 * rng.standard_normal(C)
    gamma[::7] *= -1.0              # negative gains too
    return q, S, r, S_r, gamma, beta, 4.5 / 127.0


@pytest.mark.parametrize("C,residual,sigma", [(768, True, 1.0), (1024, True, 4.0), (768, False, 1.0),
                                              (17, True, 1.0), (2047, False, 1.0)])
def test_layernorm_within_one_step_of_float_layernorm(C, residual, sigma):
    q, S, r, S_r, gamma, beta, S_out = _make(48, C, 100 + C, sigma, residual)
    out, S_ret = oracle.layernorm(q, S, r, S_r or 0.0, gamma, beta, S_out)
    assert S_ret == S_out
    ref = float_layernorm_int8(q, S, r, S_r, gamma, beta, S_out)
    diff = np.abs(out.astype(np.int64) - ref)
    assert diff.max() <= 1
    assert (diff != 0).mean() < 0.015


def test_layernorm_constant_row_gives_requantized_beta():
    C = 64
    gamma = np.linspace(0.5, 1.5, C)
    beta = np.linspace(-1.0, 1.0, C)
    S_out = 0.02
    q = np.full((2, C), 1234, dtype=np.int32)
    q[1] = -77
    out, _ = oracle.layernorm(q, 1e-3, None, 0.0, gamma, beta, S_out)
    want = np.clip(np.floor(beta / S_out + 0.5), -127, 127)
    assert (out[0] == want).all() and (out[1] == want).all()


def test_layernorm_row_shift_invariance_is_exact():
    q, S, r, S_r, gamma, beta, S_out = _make(16, 768, 7, residual=False)
    a, _ = oracle.layernorm(q, S, None, 0.0, gamma, beta, S_out)
    k = np.arange(16, dtype=np.int32)[:, None] * 997 - 5000
    b, _ = oracle.layernorm(q + k, S, None, 0.0, gamma, beta, S_out)
    assert (a == b).all()


def test_layernorm_permutation_equivariance():
    q, S, r, S_r, gamma, beta, S_out = _make(8, 300, 8)
    perm = np.random.default_rng(0).permutation(300)
    a, _ = oracle.layernorm(q, S, r, S_r, gamma, beta, S_out)
    b, _ = oracle.layernorm(q[:, perm], S, r[:, perm], S_r, gamma[perm], beta[perm], S_out)
    assert (a[:, perm] == b).all()


def test_layernorm_residual_uses_the_dyadic_rescale():
    # residual at exactly 256x the main scale: r * 256 is added, nothing is rounded
    C = 32
    rng = np.random.default_rng(3)
    q = rng.integers(-20000, 20000, (4, C)).astype(np.int32)
    r = rng.integers(-60, 60, (4, C)).astype(np.int8)
    g, b = np.ones(C), np.zeros(C)
    a, _ = oracle.layernorm(q, 1e-4, r, 256e-4, g, b, 0.03)
    c, _ = oracle.layernorm(q + 256 * r.astype(np.int32), 1e-4, None, 0.0, g, b, 0.03)
    assert (a == c).all()


def test_layernorm_rejects_out_of_range_inputs():
    with pytest.raises(oracle.OracleError):
        oracle.layernorm(np.full((1, 8), 2 ** 20 + 1, np.int32), 1e-3, None, 0.0, np.ones(8), np.zeros(8), 0.02)
    with pytest.raises(oracle.OracleError):
        oracle.layernorm(np.zeros((1, 2048), np.int32), 1e-3, None, 0.0, np.ones(2048), np.zeros(2048), 0.02)
