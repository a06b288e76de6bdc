"""GPU parity (bit-exact) of linear + residual + i-LayerNorm as one operation against the oracle's
linear layer (Q16 output) followed by its i-LayerNorm (Sec. 3.6, Eq. 16).  Shapes with N a
multiple of 256 run the single cluster kernel; the others run the two kernels back to back."""
import numpy as np
import pytest

import oracle
from gpu_util import assert_same, ctx, dev, host

pytestmark = pytest.mark.gpu


def _problem(M, N, K, seed, res_ratio=0.5):
    rng = np.random.default_rng(seed)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-200000, 200000, N).astype(np.int32)
    res = rng.integers(-127, 128, (M, N)).astype(np.int8)
    S_w = rng.uniform(1e-4, 4e-4, N)
    S_x = 0.03
    amax = 127.0 * 127.0 * np.sqrt(K) * 1.2 * S_x * 2.5e-4       # a few standard deviations of the product
    S_mid = 1.5 * amax / 32767.0
    S_res = res_ratio * amax / 127.0
    gamma = 1.0 + 0.1 * rng.standard_normal(N)
    beta = 0.1 * rng.standard_normal(N)
    S_out = 4.5 / 127.0
    return x, w, bias, res, S_w, S_x, S_mid, S_res, gamma, beta, S_out


def _oracle(x, w, bias, res, S_w, S_x, S_mid, S_res, gamma, beta, S_out):
    mid = oracle.linear(x, S_x, w, S_w, bias, 1, S_mid)
    want, _ = oracle.layernorm(mid, S_mid, res, S_res, gamma, beta, S_out)
    return want


# (rows, channels, reduction): 1..7 CTAs per cluster, ragged row tiles, several tiles per cluster,
# reduction lengths that are not multiples of the 128-byte K block, and shapes the cluster kernel
# does not take (channels not a multiple of 256)
SHAPES = [(1, 256, 64), (127, 256, 128), (300, 512, 144), (129, 768, 768), (1000, 768, 3072), (260, 1024, 1024),
          (515, 1024, 4096), (70, 1280, 256), (40, 1792, 128), (20000, 256, 64), (9000, 768, 256),
          (77, 128, 64), (300, 320, 80), (0, 768, 768)]


@pytest.fixture(autouse=True)
def _restore_fusion_mode():
    yield
    ctx().ibert_set_fusion(0)


@pytest.mark.parametrize("mode", [1, 2, 0])       # cluster kernel forced, two kernels forced, by size
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_linear_layernorm_matches_oracle(M, N, K, mode):
    p = _problem(M, N, K, M + N + K)
    x, w, bias, res, S_w, S_x, S_mid, S_res, gamma, beta, S_out = p
    ctx().ibert_set_fusion(mode)
    out, S_ret = ctx().ibert_linear_layernorm_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, dev(res), S_res,
                                                 gamma, beta, S_out)
    ctx().check()
    assert S_ret == S_out
    if M:
        want = _oracle(*p)
        assert_same(host(out), want, f"linear+LN {M}x{N}x{K} mode {mode}")
        assert np.abs(want).max() > 20


def test_linear_layernorm_constant_rows_and_no_bias():
    """Rows whose pre-LayerNorm values are all equal (variance 0: the standard deviation floor of 1
    applies) and a call without bias."""
    M, N, K = 140, 512, 128
    p = list(_problem(M, N, K, 5))
    p[0][:70] = 0                       # x = 0 -> accumulators = bias
    p[2][:] = 1234                      # the same bias everywhere
    p[3][:70] = 7                       # constant residual
    p[4][:] = 2e-4                      # one weight scale: every channel requantizes alike
    x, w, bias, res, S_w, S_x, S_mid, S_res, gamma, beta, S_out = p
    ctx().ibert_set_fusion(1)
    out, _ = ctx().ibert_linear_layernorm_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, dev(res), S_res,
                                             gamma, beta, S_out)
    ctx().check()
    assert_same(host(out), _oracle(*p), "constant rows")
    p[2] = None
    out, _ = ctx().ibert_linear_layernorm_i8(dev(x), S_x, dev(w), S_w, None, S_mid, dev(res), S_res,
                                             gamma, beta, S_out)
    ctx().check()
    assert_same(host(out), _oracle(*p), "no bias")


def test_linear_layernorm_equals_the_two_separate_calls():
    M, N, K = 700, 768, 768
    x, w, bias, res, S_w, S_x, S_mid, S_res, gamma, beta, S_out = _problem(M, N, K, 11)
    c = ctx()
    c.ibert_set_fusion(1)
    fused, _ = c.ibert_linear_layernorm_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, dev(res), S_res,
                                           gamma, beta, S_out)
    mid, _ = c.ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 1, S_mid)
    two, _ = c.ibert_layernorm_i(mid, S_mid, dev(res), S_res, gamma, beta, S_out)
    c.check()
    assert_same(host(fused), host(two), "fused vs separate")
