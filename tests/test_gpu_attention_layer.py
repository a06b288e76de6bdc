"""GPU parity (bit-exact) of the fused attention kernel and the whole encoder layer."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,L,heads", [(1, 16, 1), (2, 37, 2), (1, 128, 12), (3, 128, 2), (2, 200, 2), (1, 256, 3),
                                       (1, 512, 2), (2, 1, 1), (1, 33, 1), (1, 300, 1), (0, 64, 1), (1, 130, 1), (1, 384, 2),
                                       (2, 480, 1), (40, 160, 8), (20, 290, 8), (30, 128, 12), (16, 100, 12), (38, 64, 4),
                                       (25, 256, 8), (10, 384, 16)])
@pytest.mark.parametrize("p_max", [255, 127])
def test_attention_matches_oracle(B, L, heads, p_max):
    H = heads * 64
    rng = np.random.default_rng(L * 7 + heads)
    qkv = np.clip(np.rint(rng.standard_normal((max(B, 1) * L, 3 * H)) * 40), -127, 127).astype(np.int8)[:B * L]
    S_q = S_k = 0.02
    S_v, S_ctx = 0.02, 0.006
    out, S_ret = ctx().ibert_attention_i8(dev(qkv), B, L, H, heads, S_q, S_k, S_v, S_ctx, p_max)
    ctx().check()
    assert S_ret == S_ctx
    if B:
        want = oracle.attention(qkv, B, L, H, heads, S_q, S_k, S_v, S_ctx, p_max)
        assert_same(host(out), want, f"attention L={L}")
        assert np.abs(want).max() > 5


def test_attention_peaked_and_uniform_rows():
    B, L, heads = 1, 128, 2
    H = heads * 64
    rng = np.random.default_rng(0)
    qkv = rng.integers(-127, 128, (L, 3 * H)).astype(np.int8)       # full-range scores: one-hot rows
    qkv[:, 64:128] = 0                                              # head 1: q = 0 -> uniform rows
    for S_qk in (0.05, 0.004):
        out, _ = ctx().ibert_attention_i8(dev(qkv), B, L, H, heads, S_qk, S_qk, 0.02, 0.01, 255)
        want = oracle.attention(qkv, B, L, H, heads, S_qk, S_qk, 0.02, 0.01, 255)
        assert_same(host(out), want, "attention peaked")
    ctx().check()


@pytest.mark.parametrize("L", [100, 200])
@pytest.mark.parametrize("S_qk", [1.5, 2.0])
def test_attention_coarse_score_scale(L, S_qk):
    """Score scales so coarse that q_ln2 <= 2: the kernel with the clamped i-exp quotient runs."""
    B, heads = 2, 2
    H = heads * 64
    rng = np.random.default_rng(L)
    qkv = rng.integers(-3, 4, (B * L, 3 * H)).astype(np.int8)
    qkv[:, 2 * H:] = rng.integers(-127, 128, (B * L, H))
    out, _ = ctx().ibert_attention_i8(dev(qkv), B, L, H, heads, S_qk, S_qk, 0.02, 0.01, 255)
    want = oracle.attention(qkv, B, L, H, heads, S_qk, S_qk, 0.02, 0.01, 255)
    assert_same(host(out), want, f"attention coarse L={L}")
    assert np.abs(want).max() > 5
    ctx().check()


def _run_layers(x, params, B, L, fusion=0):
    c = ctx()
    c.ibert_set_fusion(fusion)
    h = dev(x)
    outs = []
    for p in params:
        layer = c.ibert_layer_create(p)
        h, S = c.ibert_encoder_layer(layer, h, B, L)
        assert S == p["S_out"]
        outs.append(host(h))
        c.check()
        layer.close()
    c.ibert_set_fusion(0)
    return outs


@pytest.mark.parametrize("fusion", [0, 1])      # linear + LayerNorm: by size (two kernels here) / cluster kernel
@pytest.mark.parametrize("B,L,H,heads,F", [(2, 16, 128, 2, 256), (1, 37, 64, 1, 64), (3, 128, 256, 4, 1024),
                                           (2, 100, 768, 12, 3072)])
def test_small_encoder_layers_match_oracle(B, L, H, heads, F, fusion, qkv_layout):
    x, params = synth.make_model(0, B, layers=2, H=H, heads=heads, F=F, L=L)
    outs = _run_layers(x, params, B, L, fusion)
    h = x
    for p, got in zip(params, outs):
        h = oracle.encoder_layer(p, h, B, L).out
        assert_same(got, h, "encoder layer")


def test_config0_roberta_base_layer_matches_oracle(gelu_mode):
    x, params = synth.make_model(0, 1)
    got = _run_layers(x, params, 1, 128)[0]
    want = oracle.encoder_layer(params[0], x, 1, 128).out
    assert_same(got, want, "config 0")
    assert want.std() > 20


def test_config2_three_layers_batch8_match_oracle(qkv_layout):
    B, L = 8, 128
    x, params = synth.make_model(2, B, layers=3)
    outs = _run_layers(x, params, B, L)
    h = x
    for p, got in zip(params, outs):
        h = oracle.encoder_layer(p, h, B, L).out
        assert_same(got, h, "config 2 layer")


def test_large_shapes_one_layer_L256_and_L512(gelu_mode, qkv_layout):
    for cfg, B in ((3, 2), (4, 1)):
        L = synth.CONFIGS[cfg].L
        x, params = synth.make_model(cfg, B, layers=1)
        got = _run_layers(x, params, B, L)[0]
        want = oracle.encoder_layer(params[0], x, B, L).out
        assert_same(got, want, f"config {cfg}")


def test_layer_error_codes():
    from paper_2101_01321_b200.binding import IbertError
    x, params = synth.make_model(0, 1, layers=1, H=128, heads=2, F=256, L=16)
    bad = dict(params[0])
    bad["S_q"] = -1.0
    with pytest.raises(IbertError) as e:
        ctx().ibert_layer_create(bad)
    assert e.value.code == -3
    bad = dict(params[0])
    bad["heads"] = 3
    with pytest.raises(IbertError) as e:
        ctx().ibert_layer_create(bad)
    assert e.value.code == -2
    layer = ctx().ibert_layer_create(params[0])
    with pytest.raises(IbertError) as e:
        ctx().ibert_encoder_layer(layer, dev(x), 1, 513)
    assert e.value.code == -2
    layer.close()
    assert ctx().ibert_last_status() == 0


@pytest.mark.parametrize("B,L,heads", [(2, 128, 3), (3, 100, 2), (2, 256, 2), (1, 512, 1), (2, 37, 1)])
def test_attention_power_of_two_score_scale(B, L, heads):
    """Score scale exactly ln2 / 2^k: the kernel takes quotient and remainder of i-exp by shift and
    mask; the oracle is the ordinary one at that scale."""
    H = heads * 64
    rng = np.random.default_rng(L)
    qkv = np.clip(np.rint(rng.standard_normal((B * L, 3 * H)) * 40), -127, 127).astype(np.int8)
    S_k = 0.02
    S_q = synth.snap_q_scale(0.02, S_k)
    q_ln2 = oracle.exp_consts((S_q * S_k) / 8.0)["q_ln2"]
    assert q_ln2 & (q_ln2 - 1) == 0
    out, _ = ctx().ibert_attention_i8(dev(qkv), B, L, H, heads, S_q, S_k, 0.02, 0.006, 255)
    ctx().check()
    assert_same(host(out), oracle.attention(qkv, B, L, H, heads, S_q, S_k, 0.02, 0.006, 255), f"pow2 attention L={L}")
    lens = np.array([L, 1, max(L // 2, 1)][:B], np.int32)
    out, _ = ctx().ibert_attention_masked_i8(dev(qkv), B, L, H, heads, dev(lens), S_q, S_k, 0.02, 0.006, 255)
    ctx().check()
    assert_same(host(out), oracle.attention(qkv, B, L, H, heads, S_q, S_k, 0.02, 0.006, 255, lens=lens),
                f"pow2 masked attention L={L}")


def test_encoder_layers_with_power_of_two_score_scales():
    B, L, H, heads, F = 2, 128, 256, 4, 1024
    x, params = synth.make_model(0, B, layers=2, H=H, heads=heads, F=F, L=L, pow2_scores=True)
    outs = _run_layers(x, params, B, L)
    h = x
    for p, got in zip(params, outs):
        h = oracle.encoder_layer(p, h, B, L).out
        assert_same(got, h, "pow2-score layer")


@pytest.mark.parametrize("shrink,S_go_scale", [(2.0, 1.0), (3.5, 1.0), (6.0, 1.0), (3.5, 0.004)])
def test_layer_with_ffn1_multipliers_of_one_half_and_more(shrink, S_go_scale, gelu_mode):
    """A finer GELU-input scale makes the per-channel multipliers S_h1 S_w[n] / S_gi reach 1/2 and go
    beyond 1: the FFN1 epilogue then takes the wide upper-word form (multiplier split into an integer
    part and a 32-bit fraction), with and without the lower output clamp; many values clamp at Q16."""
    B, L, H, heads, F = 5, 96, 256, 4, 1024
    x, params = synth.make_model(0, B, layers=1, H=H, heads=heads, F=F, L=L)
    p = dict(params[0])
    p["S_gi"] = p["S_gi"] / shrink
    p["S_go"] = p["S_go"] * S_go_scale
    m = p["S_h1"] * np.asarray(p["S_w_f1"]) / p["S_gi"]
    assert m.max() >= 0.5
    c = ctx()
    layer = c.ibert_layer_create(p)
    try:
        out, _ = c.ibert_encoder_layer(layer, dev(x), B, L)
        c.check()
    finally:
        layer.close()
    res = oracle.encoder_layer(p, x, B, L, want_taps=True)
    assert_same(host(out), res.out, f"layer with FFN1 multipliers up to {m.max():.2f}")
    assert np.abs(np.asarray(res.taps["g"]).astype(int)).max() > 20
