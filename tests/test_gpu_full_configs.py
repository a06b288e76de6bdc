"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The encoder never mixes sequences, so the oracle recomputes a sample of whole sequences through
every layer and the GPU rows of those sequences (taken from the full-batch run) must match bit
for bit.  The standalone sweeps of config 1 are compared in full."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu


def _full_model_check(config_id, B, sample, scales="analytic"):
    cfg = synth.CONFIGS[config_id]
    L = cfg.L
    x, params = synth.make_model(config_id, B, scales=scales)
    c = ctx()
    layers = [c.ibert_layer_create(p) for p in params]
    h = dev(x)
    bufs = [torch.empty_like(h), torch.empty_like(h)]
    for i, ly in enumerate(layers):
        h, _ = c.ibert_encoder_layer(ly, h, B, L, out=bufs[i & 1])
    c.check()
    got = host(h).reshape(B, L, cfg.H)
    for ly in layers:
        ly.close()
    for s in sample:
        ref = x.reshape(B, L, cfg.H)[s].reshape(L, cfg.H)
        for p in params:
            ref = oracle.encoder_layer(p, ref, 1, L).out
        assert_same(got[s], ref, f"config {config_id}, sequence {s}")
    assert got.std() > 12                      # the stack stays well scaled through all layers


def test_config2_twelve_layers_batch128_sampled_sequences(gelu_mode):
    _full_model_check(2, 128, sample=(0, 77, 127))


def test_config2_small_batches():
    for B in (1, 8, 32):
        _full_model_check(2, B, sample=(0, B - 1))


def test_config3_large_24_layers_L256_batch32_sampled_sequences(qkv_layout):
    _full_model_check(3, 32, sample=(0, 5, 31))


def test_config4_large_24_layers_L512_batch64_sampled_sequences():
    _full_model_check(4, 64, sample=(0, 31, 63))


def test_config2_layers_with_ragged_token_count(qkv_layout):
    """37 sequences of 112 tokens: 4144 tokens = 32 full 128-token tiles and a 48-token tail, large
    enough for the transposed intermediates (Q|K|V and the FFN1 result) where the layout switch allows them."""
    cfg = synth.CONFIGS[2]
    B, L = 37, 112
    x, params = synth.make_model(2, B)
    x, params = np.ascontiguousarray(x[:B * L]), params[:2]
    c = ctx()
    layers = [c.ibert_layer_create(p) for p in params]
    h = dev(x)
    for ly in layers:
        h, _ = c.ibert_encoder_layer(ly, h, B, L)
    c.check()
    got = host(h).reshape(B, L, cfg.H)
    for ly in layers:
        ly.close()
    for s in (0, 36):                          # the last sequence ends in the ragged tile
        ref = x.reshape(B, L, cfg.H)[s]
        for p in params:
            ref = oracle.encoder_layer(p, ref, 1, L).out
        assert_same(got[s], ref, f"ragged batch, sequence {s}")


def test_config2_with_oracle_calibrated_scales():
    """The same stack with the static scales calibrated from each site's max|x| (the stored blob)."""
    _full_model_check(2, 128, sample=(3, 100), scales="calibrated")


def test_config3_with_oracle_calibrated_scales():
    _full_model_check(3, 32, sample=(17,), scales="calibrated")


@pytest.mark.parametrize("config_id,B,L", [(2, 128, 128), (3, 32, 256)])
def test_full_config_packed_sentence_mix(config_id, B, L):
    """Bench-size packed batch (the sentence-length mix without its padding): sampled sequences
    against the oracle run on each sequence alone."""
    cfg = synth.CONFIGS[config_id]
    x, params = synth.make_model(config_id, B)
    lens = synth.make_lengths(config_id, B, L)
    rows = np.concatenate([np.arange(b * L, b * L + n) for b, n in enumerate(lens)])
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    c = ctx()
    layers = [c.ibert_layer_create(p) for p in params]
    h, cu_d = dev(np.ascontiguousarray(x[rows])), dev(cu)
    bufs = [torch.empty_like(h), torch.empty_like(h)]
    for i, ly in enumerate(layers):
        h, _ = c.ibert_encoder_layer_packed(ly, h, cu_d, L, out=bufs[i & 1])
    c.check()
    got = host(h)
    for ly in layers:
        ly.close()
    for s in (0, B // 2, B - 1):
        n = int(lens[s])
        ref = x[s * L:s * L + n]
        for p in params:                       # a sequence alone, at its own length: no padding, no mask
            ref = oracle.encoder_layer(p, ref, 1, n).out
        assert_same(got[cu[s]:cu[s] + n], ref, f"config {config_id} packed, sequence {s} ({n} tokens)")


@pytest.mark.parametrize("sigma", [1.0, 4.0])
def test_config1_gelu_16m_elements(sigma):
    q, S, S_out = synth.gelu_inputs(1 << 24, sigma)
    out, _ = ctx().ibert_gelu_i(dev(q), S, S_out)
    ctx().check()
    assert_same(host(out), oracle.gelu(q, S, S_out)[0], "gelu 16M")


@pytest.mark.parametrize("rows,L", [(96 * 128, 128), (384 * 512, 512)])
def test_config1_softmax_score_tensors(rows, L):
    for sigma in (1.0, 4.0):
        q, S = synth.softmax_inputs(rows, L, sigma)
        out, _ = ctx().ibert_softmax_i(dev(q), S, 255)
        ctx().check()
        assert_same(host(out), oracle.softmax(q, S, 255)[0], f"softmax [{rows},{L}]")


@pytest.mark.parametrize("rows,C", [(4096, 768), (16384, 1024)])
def test_config1_layernorm_rows(rows, C):
    for sigma in (1.0, 4.0):
        q, S, r, S_r, gamma, beta, S_out = synth.layernorm_inputs(rows, C, sigma)
        out, _ = ctx().ibert_layernorm_i(dev(q), S, dev(r), S_r, gamma, beta, S_out)
        ctx().check()
        assert_same(host(out), oracle.layernorm(q, S, r, S_r, gamma, beta, S_out)[0], f"layernorm [{rows},{C}]")
