"""Pins of the integer h-GELU (Eq. 6; the comparison function of Table 1 and Table 3): against the
float formula of Eq. 6, against GELU within the error the paper prints for h-GELU, and the exact
regions (zero below -3/1.702, identity above +3/1.702)."""
import math

import numpy as np
import pytest

import oracle

_erf = np.vectorize(math.erf)


def _float_hgelu(x):
    return x * np.clip(1.702 * x + 3.0, 0.0, 6.0) / 6.0


@pytest.mark.parametrize("S,S_out", [(8.0 * 0.56 / 32767, 4.0 / 127), (1e-3, 4.0 / 127), (2.5e-4, 0.05), (3e-5, 0.04)])
def test_integer_hgelu_follows_eq6_and_the_papers_error_figure(S, S_out):
    x = np.linspace(-4.0, 4.0, 20001)
    q = np.clip(np.rint(x / S), -32767, 32767).astype(np.int32)
    out, S_ret = oracle.hgelu(q, S, S_out)
    assert S_ret == S_out
    xr = q * S
    top = 127 * S_out
    h = np.clip(_float_hgelu(xr), -top, top)
    assert np.abs(out * S_out - h).max() <= S_out / 2 + 1e-3          # Eq. 6, to output rounding
    g = np.clip(xr * 0.5 * (1.0 + _erf(xr / math.sqrt(2.0))), -top, top)
    err = np.abs(out * S_out - g).max()
    assert err <= 0.0687 + S_out / 2 + 1e-3                           # Table 1: L-inf 0.068 for h-GELU
    assert err >= 0.05                                                # ... and it really is that far off
    assert not out[xr < -3.0 / 1.702 - 1e-9].any()                    # ReLU6 = 0: exact zeros
    assert out[q == 0].max(initial=0) == 0


def test_hgelu_is_the_identity_above_the_knee():
    S, S_out = 1e-4, 3.2 / 127
    q = np.arange(int(3.0 / 1.702 / S) + 2, 32767, 37, dtype=np.int32)
    out, _ = oracle.hgelu(q, S, S_out)
    assert np.abs(out * S_out - np.clip(q * S, None, 127 * S_out)).max() <= S_out / 2 + 1e-3


def test_hgelu_clamps_its_input_to_q16_and_rejects_bad_scales():
    S, S_out = 1e-4, 4.0 / 127
    a, _ = oracle.hgelu(np.array([40000, -40000, 2**31 - 1, -2**31], np.int32), S, S_out)
    b, _ = oracle.hgelu(np.array([32767, -32767, 32767, -32767], np.int32), S, S_out)
    assert np.array_equal(a, b)
    with pytest.raises(oracle.OracleError):
        oracle.hgelu(np.zeros(4, np.int32), 10.0, 1.0)               # 6 / (1.702 S) < 1
