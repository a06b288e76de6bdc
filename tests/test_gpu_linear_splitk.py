"""GPU parity (bit-exact) of the split-K cluster GEMM: every epilogue kind, both cluster widths forced,
ragged M / N / K, K ranges that leave a CTA of the cluster without a block, and the size rule."""
import numpy as np
import pytest

import oracle
from gpu_util import assert_same, ctx, dev, host

pytestmark = pytest.mark.gpu

# (M, N, K): K = 144 / 272 leave ranks of a 4-wide cluster without a K block
SHAPES = [(1, 16, 144), (7, 48, 272), (128, 128, 512), (130, 272, 400), (300, 768, 768), (129, 768, 3072),
          (257, 1024, 1024), (128, 2304, 768), (100, 3072, 768), (520, 320, 4096)]


def _problem(M, N, K, seed):
    rng = np.random.default_rng(seed)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-200000, 200000, N).astype(np.int32)
    S_w = rng.uniform(1e-4, 4e-4, N)
    S_x = 0.03
    amax = 127.0 * 127.0 * np.sqrt(K) * 1.2 * S_x * 2.5e-4
    return x, w, bias, S_w, S_x, amax


@pytest.fixture
def split(request):
    c = ctx()
    c.ibert_set_split_k(request.param)
    yield request.param
    c.ibert_set_split_k(0)


@pytest.mark.parametrize("split", [2, 4], indirect=True)
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_split_k_raw_q16_int8(M, N, K, split):
    x, w, bias, S_w, S_x, amax = _problem(M, N, K, split)
    out, _ = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 2)
    assert_same(host(out), oracle.linear(x, S_x, w, S_w, bias, 2), "raw")
    for kind, S_out in ((0, amax / 100.0), (1, amax / 20000.0)):
        out, _ = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), kind, S_out)
        assert_same(host(out), oracle.linear(x, S_x, w, S_w, bias, kind, S_out), f"kind {kind}")
    ctx().check()


@pytest.mark.parametrize("split", [2, 4], indirect=True)
@pytest.mark.parametrize("M,N,K", [(7, 48, 272), (300, 768, 768), (129, 3072, 768), (257, 1024, 1024)])
def test_split_k_fused_gelu_and_hgelu(M, N, K, split):
    x, w, bias, S_w, S_x, amax = _problem(M, N, K, 3)
    S_mid, S_x, S_out = 6.0 / 32767.0, S_x * (6.0 / amax), 6.0 / 127.0
    mid = oracle.linear(x, S_x, w, S_w, bias, 1, S_mid)
    out, _ = ctx().ibert_linear_gelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
    assert_same(host(out), oracle.gelu(mid, S_mid, S_out)[0], "linear+gelu")
    out, _ = ctx().ibert_linear_hgelu_i8(dev(x), S_x, dev(w), S_w, dev(bias), S_mid, S_out)
    assert_same(host(out), oracle.hgelu(mid, S_mid, S_out)[0], "linear+hgelu")
    ctx().check()


@pytest.mark.parametrize("split", [4], indirect=True)
def test_split_k_generic_dyadic_form(split):
    """Multipliers >= 1 and large biases: the epilogue with the 64-bit product instead of the upper-word form."""
    M, N, K = 64, 64, 256
    rng = np.random.default_rng(11)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-2 ** 28, 2 ** 28, N).astype(np.int32)
    S_w = np.geomspace(1e-6, 10.0, N)
    for kind, S_out in ((0, 1e-3), (1, 1e-5), (0, 50.0), (1, 0.2)):
        out, _ = ctx().ibert_linear_i8(dev(x), 0.5, dev(w), S_w, dev(bias), kind, S_out)
        assert_same(host(out), oracle.linear(x, 0.5, w, S_w, bias, kind, S_out), f"kind {kind} S_out {S_out}")
    ctx().check()


@pytest.mark.parametrize("split", [0, 1], indirect=True)
def test_size_rule_and_unsplit_agree(split):
    """Mode 0 picks the width by size (these shapes split), mode 1 never splits: same bits."""
    for M, N, K in ((128, 768, 3072), (1024, 768, 768), (100, 2304, 768)):
        x, w, bias, S_w, S_x, amax = _problem(M, N, K, 5)
        out, _ = ctx().ibert_linear_i8(dev(x), S_x, dev(w), S_w, dev(bias), 1, amax / 20000.0)
        assert_same(host(out), oracle.linear(x, S_x, w, S_w, bias, 1, amax / 20000.0), f"mode {split} {M}x{N}x{K}")
    ctx().check()


def test_split_k_mode_argument_is_checked():
    from paper_2101_01321_b200.binding import IbertError
    with pytest.raises(IbertError) as e:
        ctx().ibert_set_split_k(3)
    assert e.value.code == -1
    ctx().ibert_set_split_k(0)
