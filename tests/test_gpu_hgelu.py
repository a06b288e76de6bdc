"""GPU parity (bit-exact) of the integer h-GELU (Eq. 6), standalone and as a GEMM epilogue."""
import numpy as np
import pytest

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,sigma", [(1 << 20, 1.0), (100003, 4.0), (5, 1.0), (0, 1.0)])
def test_hgelu_matches_oracle(n, sigma):
    q, S, S_out = synth.gelu_inputs(max(n, 1), sigma)
    q = q[:n]
    out, S_ret = ctx().ibert_hgelu_i(dev(q), S, S_out)
    ctx().check()
    assert S_ret == S_out
    if n:
        want, _ = oracle.hgelu(q, S, S_out)
        assert_same(host(out), want, "h-GELU")
        assert (n < 1000 or want.max() > 100) and want.min() <= 0


def test_hgelu_full_int32_range_and_odd_scales():
    rng = np.random.default_rng(2)
    q = np.concatenate([rng.integers(-2**31, 2**31, 100000), np.arange(-40000, 40000, 7),
                        [2**31 - 1, -2**31, 0, 1, -1, 32767, -32767, 32768, -32768]]).astype(np.int32)
    for S, S_out in [(1e-3, 4.0 / 127), (1.2207e-4, 0.03), (3.3e-5, 0.011), (0.02, 0.9)]:
        out, _ = ctx().ibert_hgelu_i(dev(q), S, S_out)
        ctx().check()
        assert_same(host(out), oracle.hgelu(q, S, S_out)[0], f"h-GELU S={S}")


@pytest.mark.parametrize("M,N,K", [(130, 272, 144), (300, 3072, 768), (2100, 512, 256)])
def test_linear_hgelu_matches_oracle(M, N, K):
    rng = np.random.default_rng(M + N)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-200000, 200000, N).astype(np.int32)
    S_w = rng.uniform(1e-4, 4e-4, N)
    S_x = 0.03
    amax = 127.0 * 127.0 * np.sqrt(K) * 1.2 * S_x * 2.5e-4
    S_mid, S_out = 2.0 * amax / 32767, amax / 127
    out, _ = ctx().ibert_linear_hgelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
    ctx().check()
    mid = oracle.linear(x, S_x, w, S_w, bias, 1, S_mid)
    want, _ = oracle.hgelu(mid, S_mid, S_out)
    assert_same(host(out), want.reshape(M, N), "linear + h-GELU")


@pytest.mark.parametrize("sigma", [1.0, 4.0])
def test_gelu_by_table_lookup_equals_the_integer_kernel(sigma):
    """The look-up table is built from the i-GELU kernel, so both entry points agree bit for bit
    (and with the oracle), for ordinary inputs and for the whole int32 range."""
    q, S, S_out = synth.gelu_inputs(300007, sigma)
    rng = np.random.default_rng(4)
    q = np.concatenate([q, rng.integers(-2**31, 2**31, 5000).astype(np.int32),
                        np.array([2**31 - 1, -2**31, 0, 32767, -32767, 32768, -32768], np.int32)])
    a, _ = ctx().ibert_gelu_lut_i(dev(q), S, S_out)
    b, _ = ctx().ibert_gelu_i(dev(q), S, S_out)
    ctx().check()
    assert_same(host(a), host(b), "table vs kernel")
    assert_same(host(a), oracle.gelu(q, S, S_out)[0], "table vs oracle")
    a2, _ = ctx().ibert_gelu_lut_i(dev(q), S, S_out)          # second call: cached table
    ctx().check()
    assert_same(host(a2), host(b), "cached table")


@pytest.mark.parametrize("split", [1, 4])
@pytest.mark.parametrize("S_mid,S_out", [(1.4e-3, 2.7e-4), (2.7e-3, 8e-4), (1.6e-3, 1e-4), (3e-4, 2e-5)])
def test_fused_gelu_kinds_with_a_final_multiplier_above_one_half(S_mid, S_out, split):
    """An output scale so fine that the final multiplier of the GELU epilogue does not fit the upper-word
    form while the per-channel ones do: the whole epilogue must then run in the generic form, on the
    plain (b, c) pairs.  (Found by a sweep over random scales: the per-channel table used to be
    converted regardless.)"""
    rng = np.random.default_rng(7)
    M, N, K = 130, 272, 144
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-2000, 2000, N).astype(np.int32)
    S_w, S_x = rng.uniform(1e-4, 4e-4, N), 0.02
    c = ctx()
    c.ibert_set_split_k(split)
    try:
        mid = oracle.linear(x, S_x, w, S_w, bias, 1, S_mid)
        out, _ = c.ibert_linear_hgelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
        assert_same(host(out), oracle.hgelu(mid, S_mid, S_out)[0], "linear + h-GELU")
        out, _ = c.ibert_linear_gelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
        assert_same(host(out), oracle.gelu(mid, S_mid, S_out)[0], "linear + i-GELU")
        c.check()
    finally:
        c.ibert_set_split_k(0)


def test_encoder_layer_with_a_fine_gelu_output_scale():
    """The same situation inside ibert_encoder_layer: S_go small enough that FFN1's final multiplier
    leaves the upper-word form (most outputs clamp; the bits still have to be the oracle's)."""
    B, L = 2, 64
    x, params = synth.make_model(0, B, layers=1, H=256, heads=4, F=1024, L=L)
    p = dict(params[0])
    p["S_go"] = p["S_go"] / 400.0
    layer = ctx().ibert_layer_create(p)
    out, _ = ctx().ibert_encoder_layer(layer, dev(x), B, L)
    ctx().check()
    assert_same(host(out), oracle.encoder_layer(p, x, B, L).out, "layer with a fine S_go")
    layer.close()


def test_table_caches_are_bounded_and_stay_correct_past_the_bound():
    """More distinct scale pairs than the 64 tables a context keeps, for both table look-up operators."""
    q, S, S_out = synth.gelu_inputs(5000, 1.0)
    sq, sS = synth.softmax_inputs(40, 96, 1.0)
    for i in range(80):
        f = 1.0 + 0.01 * i
        a, _ = ctx().ibert_gelu_lut_i(dev(q), S * f, S_out * f)
        assert_same(host(a), oracle.gelu(q, S * f, S_out * f)[0], f"gelu by table, scale pair {i}")
        p, _ = ctx().ibert_softmax_lut_i(dev(sq), sS * f, 255)
        assert_same(host(p), oracle.softmax(sq, sS * f, 255)[0], f"softmax by table, scale {i}")
    ctx().check()
