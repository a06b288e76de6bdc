"""GPU parity (bit-exact) of the tcgen05 INT8 GEMM and its fused epilogues against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host

pytestmark = pytest.mark.gpu


def _problem(M, N, K, seed, acc_scale=1.0):
    rng = np.random.default_rng(seed)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-200000, 200000, N).astype(np.int32)
    S_w = rng.uniform(1e-4, 4e-4, N)
    S_x = 0.03
    amax = 127.0 * 127.0 * np.sqrt(K) * 1.2 * S_x * 2.5e-4 * acc_scale
    return x, w, bias, S_w, S_x, amax


SHAPES = [(1, 16, 16), (7, 48, 80), (128, 128, 128), (130, 272, 144), (300, 768, 768), (257, 2304, 768),
          (129, 768, 3072), (1024, 1024, 1024), (4100, 512, 256), (2100, 2304, 768), (4800, 1024, 512), (19000, 256, 64), (0, 64, 64)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_linear_raw_accumulators(M, N, K):
    x, w, bias, S_w, S_x, _ = _problem(M, N, K, 1)
    out, S_ret = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 2)
    ctx().check()
    if M:
        assert_same(host(out), oracle.linear(x, S_x, w, S_w, bias, 2), "raw")
    assert np.array_equal(S_ret, S_x * S_w)
    out, _ = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, None, 2)
    ctx().check()
    if M:
        assert_same(host(out), oracle.linear(x, S_x, w, S_w, None, 2), "raw, no bias")


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("kind", [0, 1])
def test_linear_requantized(M, N, K, kind):
    x, w, bias, S_w, S_x, amax = _problem(M, N, K, 2)
    S_out = amax / (100.0 if kind == 0 else 20000.0)       # a few values clamp
    out, S_ret = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), kind, S_out)
    ctx().check()
    assert S_ret == S_out
    if M:
        want = oracle.linear(x, S_x, w, S_w, bias, kind, S_out)
        assert_same(host(out), want, f"kind {kind}")
        qmax = 127 if kind == 0 else 32767
        assert np.abs(want.astype(np.int64)).max() <= qmax


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_linear_q16_stored_as_int16(M, N, K):
    """out_kind 3: the Q16 values of out_kind 1 in an int16 container -- same oracle, narrower store.
    A generic (not upper-word) multiplier set and a forced split-K width are covered as well."""
    x, w, bias, S_w, S_x, amax = _problem(M, N, K, 5)
    for S_out in (amax / 20000.0, amax / 2.0e9):          # a few values clamp / multipliers >= 1: generic form
        out, S_ret = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 3, S_out)
        ctx().check()
        assert S_ret == S_out and out.dtype == torch.int16
        if M:
            want = oracle.linear(x, S_x, w, S_w, bias, 1, S_out)
            assert_same(host(out).astype(np.int32), want, f"kind 3, S_out={S_out}")
    if M and K > 128:
        ctx().ibert_set_split_k(2)
        try:
            out, _ = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 3, amax / 20000.0)
            ctx().check()
        finally:
            ctx().ibert_set_split_k(0)
        assert_same(host(out).astype(np.int32), oracle.linear(x, S_x, w, S_w, bias, 1, amax / 20000.0), "kind 3, split K")


def test_linear_int16_needs_rows_of_16_bytes():
    from paper_2101_01321_b200.binding import IbertError
    x, w, bias, S_w, S_x, amax = _problem(8, 20, 32, 6)
    with pytest.raises(IbertError) as e:
        ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 3, amax / 20000.0)
    assert e.value.code == -2


@pytest.mark.parametrize("M,N,K", [(7, 48, 80), (300, 768, 768), (257, 3072, 768), (1000, 4096, 1024), (2500, 3072, 768)])
def test_linear_with_fused_gelu(M, N, K, gelu_mode):
    x, w, bias, S_w, S_x, amax = _problem(M, N, K, 3)
    # scale the problem so the GELU input covers about [-6, 6]
    S_mid = 6.0 / 32767.0
    S_x = S_x * (6.0 / amax)
    S_out = 6.0 / 127.0
    out, S_ret = ctx().ibert_linear_gelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
    ctx().check()
    mid = oracle.linear(x, S_x, w, S_w, bias, 1, S_mid)
    want, _ = oracle.gelu(mid, S_mid, S_out)
    assert_same(host(out), want, "linear+gelu")
    assert np.abs(mid).max() > 8000 and want.max() > 60


@pytest.mark.parametrize("S_out,low_clamp_hit", [(0.17 / 126.0, False), (0.17 / 128.0, None), (0.17 / 400.0, True),
                                                 (6.0 / 127.0, False)])
def test_linear_with_fused_gelu_around_the_lower_clamp(S_out, low_clamp_hit, gelu_mode):
    """Output scales at which the negative lobe of GELU (minimum about -0.17) stays inside int8, just
    touches -127, or saturates: the epilogue without a lower clamp may only run where none is needed."""
    x, w, bias, S_w, S_x, amax = _problem(256, 256, 128, 5)
    S_mid = 6.0 / 32767.0
    S_x = S_x * (6.0 / amax)
    out, _ = ctx().ibert_linear_gelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
    ctx().check()
    mid = oracle.linear(x, S_x, w, S_w, bias, 1, S_mid)
    want, _ = oracle.gelu(mid, S_mid, S_out)
    assert_same(host(out), want, f"linear+gelu S_out={S_out}")
    if low_clamp_hit is not None:
        assert (want.min() == -127) == low_clamp_hit


def test_linear_odd_dyadic_shifts_and_negative_results():
    # multipliers >= 1 (small shifts) and a large-bias column block
    M, N, K = 64, 64, 64
    rng = np.random.default_rng(11)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-2 ** 28, 2 ** 28, N).astype(np.int32)
    S_w = np.geomspace(1e-6, 10.0, N)
    for kind, S_out in ((0, 1e-3), (1, 1e-5), (0, 50.0), (1, 0.2)):
        out, _ = ctx().ibert_linear_i8(dev(x), 0.5, dev(w), S_w, dev(bias), kind, S_out)
        assert_same(host(out), oracle.linear(x, 0.5, w, S_w, bias, kind, S_out), f"kind {kind} S_out {S_out}")
    ctx().check()


def test_linear_error_codes():
    from paper_2101_01321_b200.binding import IbertError
    x = torch.zeros((4, 24), dtype=torch.int8, device="cuda")
    w = torch.zeros((16, 24), dtype=torch.int8, device="cuda")
    with pytest.raises(IbertError) as e:
        ctx().ibert_linear_i8(x, 1.0, w, np.ones(16), None, 0, 1.0)      # K % 16 != 0
    assert e.value.code == -2
    x = torch.zeros((4, 32), dtype=torch.int8, device="cuda")
    w = torch.zeros((8, 32), dtype=torch.int8, device="cuda")
    with pytest.raises(IbertError) as e:
        ctx().ibert_linear_i8(x, 1.0, w, np.ones(8), None, 0, 1.0)       # int8 rows need N % 16 == 0
    assert e.value.code == -2
    w = torch.zeros((16, 32), dtype=torch.int8, device="cuda")
    with pytest.raises(IbertError) as e:
        ctx().ibert_linear_i8(x, 1.0, w, np.full(16, 1e30), None, 0, 1e-30)  # multiplier >= 2^31
    assert e.value.code == -3
    for bad in (-1, 2):                                                  # the table switch knows modes 0 and 1
        with pytest.raises(IbertError) as e:
            ctx().ibert_set_gelu_table(bad)
        assert e.value.code == -1
    for bad in (-1, 3):                                                  # the layout switch modes 0, 1 and 2
        with pytest.raises(IbertError) as e:
            ctx().ibert_set_qkv_layout(bad)
        assert e.value.code == -1
    assert ctx().ibert_last_status() == 0


def test_constant_table_cache_survives_its_own_trimming():
    """Every distinct scale set leaves constant tables in the context's cache (multipliers and shifts of
    a linear layer: two per call here), which is dropped once it holds more than 4096 entries.  The
    drop must not happen while a call still holds pointers into the cache: every result stays right
    across two such drops, the second met with the other parity of the table count."""
    M, N, K = 8, 16, 16
    rng = np.random.default_rng(3)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-2000, 2000, N).astype(np.int32)
    base = rng.uniform(1e-3, 1.4e-3, N)
    xd, wd, bd = dev(x), dev(w), dev(bias)

    def scales(i, eps):
        # bit j of i doubles channel j's scale: a different shift table for every i;
        # the factor makes the multiplier table different as well
        return base * np.array([2.0 if (i >> j) & 1 else 1.0 for j in range(N)]) * (1.0 + eps)

    for i in range(4800):
        S_w = scales(i, 1e-5 * i)
        out, _ = ctx().ibert_linear_i8(xd, 0.03, wd, S_w, bd, 0, 0.05)
        assert_same(host(out), oracle.linear(x, 0.03, w, S_w, bias, 0, 0.05), f"call {i}")
        if i == 3000:       # same shifts as the call before, new multipliers: one table more, parity flips
            S_w = scales(i, 0.5)
            out, _ = ctx().ibert_linear_i8(xd, 0.03, wd, S_w, bd, 0, 0.05)
            assert_same(host(out), oracle.linear(x, 0.03, w, S_w, bias, 0, 0.05), "odd call")
    ctx().check()
