"""GPU parity (bit-exact) of the pieces around the plain layer -- attention and the encoder layer
with a key-padding mask, the INT8 embedding + i-LayerNorm, the first-token classifier -- against
the oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu

SC = dict(S_q=0.02, S_k=0.02, S_v=0.02, S_ctx=0.006)


def _lens(B, L, seed):
    """A length mix with the edge cases in it: full, one key, none, 32-multiples and neighbours."""
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, L + 1, B).astype(np.int32)
    special = [L, 1, 0, min(32, L), min(33, L), max(L - 1, 0), min(128, L), min(129, L)]
    lens[:min(B, len(special))] = special[:min(B, len(special))]
    return lens


@pytest.mark.parametrize("B,L,heads", [(8, 128, 2), (9, 100, 1), (8, 37, 3), (10, 256, 2), (8, 200, 1), (9, 512, 1),
                                       (8, 384, 2), (40, 160, 8)])
@pytest.mark.parametrize("p_max", [255, 127])
def test_masked_attention_matches_oracle(B, L, heads, p_max):
    H = heads * 64
    rng = np.random.default_rng(L + heads)
    qkv = np.clip(np.rint(rng.standard_normal((B * L, 3 * H)) * 40), -127, 127).astype(np.int8)
    lens = _lens(B, L, L)
    out, _ = ctx().ibert_attention_masked_i8(dev(qkv), B, L, H, heads, dev(lens), SC["S_q"], SC["S_k"], SC["S_v"],
                                             SC["S_ctx"], p_max)
    ctx().check()
    want = oracle.attention(qkv, B, L, H, heads, **SC, p_max=p_max, lens=lens)
    assert_same(host(out), want, f"masked attention L={L}")
    assert np.abs(want).max() > 5


def test_masked_attention_with_full_lengths_equals_the_unmasked_call():
    B, L, heads = 5, 128, 4
    H = heads * 64
    qkv = np.random.default_rng(0).integers(-60, 61, (B * L, 3 * H)).astype(np.int8)
    c = ctx()
    a, _ = c.ibert_attention_i8(dev(qkv), B, L, H, heads, 0.02, 0.02, 0.02, 0.006)
    b, _ = c.ibert_attention_masked_i8(dev(qkv), B, L, H, heads, dev(np.full(B, L, np.int32)), 0.02, 0.02, 0.02, 0.006)
    c.check()
    assert_same(host(a), host(b), "full lengths")


def test_masked_attention_coarse_score_scale():
    B, L, heads = 4, 150, 2
    H = heads * 64
    rng = np.random.default_rng(3)
    qkv = rng.integers(-3, 4, (B * L, 3 * H)).astype(np.int8)
    qkv[:, 2 * H:] = rng.integers(-127, 128, (B * L, H))
    lens = np.array([150, 0, 77, 1], np.int32)
    out, _ = ctx().ibert_attention_masked_i8(dev(qkv), B, L, H, heads, dev(lens), 1.5, 1.5, 0.02, 0.01)
    ctx().check()
    assert_same(host(out), oracle.attention(qkv, B, L, H, heads, 1.5, 1.5, 0.02, 0.01, lens=lens), "coarse, masked")


@pytest.mark.parametrize("B,L,H,heads,F", [(4, 48, 256, 4, 512), (3, 128, 128, 2, 256)])
def test_masked_encoder_layers_match_oracle(B, L, H, heads, F, qkv_layout):
    x, params = synth.make_model(0, B, layers=2, H=H, heads=heads, F=F, L=L)
    lens = _lens(B, L, 7)
    c = ctx()
    h = dev(x)
    want = x
    for p in params:
        layer = c.ibert_layer_create(p)
        h, S = c.ibert_encoder_layer_masked(layer, h, B, L, dev(lens))
        c.check()
        layer.close()
        want = oracle.encoder_layer(p, want, B, L, lens=lens).out
        assert_same(host(h), want, "masked layer")


@pytest.mark.parametrize("B,L,H,V", [(3, 17, 96, 300), (16, 128, 768, 5000), (1, 1, 16, 2), (0, 8, 64, 10)])
def test_embedding_matches_oracle(B, L, H, V):
    rng = np.random.default_rng(H + L)
    P = L + 3
    word = rng.integers(-127, 128, (V, H)).astype(np.int8)
    pos = rng.integers(-127, 128, (P, H)).astype(np.int8)
    ids = rng.integers(0, V, B * L).astype(np.int32)
    gamma, beta = 1.0 + 0.1 * rng.standard_normal(H), 0.1 * rng.standard_normal(H)
    S_word, S_pos, S_out = 0.011, 0.004, 4.5 / 127
    out, S_ret = ctx().ibert_embedding_i8(dev(ids), L, dev(word), S_word, dev(pos), S_pos, gamma, beta, S_out)
    ctx().check()
    assert S_ret == S_out
    if B:
        assert_same(host(out), oracle.embedding(ids, L, word, S_word, pos, S_pos, gamma, beta, S_out), "embedding")


def test_embedding_reports_an_id_outside_the_table():
    from paper_2101_01321_b200.binding import IbertError
    rng = np.random.default_rng(1)
    word = rng.integers(-127, 128, (10, 32)).astype(np.int8)
    pos = rng.integers(-127, 128, (4, 32)).astype(np.int8)
    ids = np.array([1, 2, 10, 3], np.int32)
    c = ctx()
    c.ibert_embedding_i8(dev(ids), 4, dev(word), 0.01, dev(pos), 0.01, np.ones(32), np.zeros(32), 0.03)
    with pytest.raises(IbertError):
        c.check()
    c.check()       # the status is cleared by reading it


@pytest.mark.parametrize("B,L,H,N", [(5, 12, 64, 16), (128, 128, 768, 4), (1, 3, 1024, 8)])
def test_classifier_matches_oracle(B, L, H, N):
    rng = np.random.default_rng(B + N)
    x = rng.integers(-127, 128, (B * L, H)).astype(np.int8)
    w = rng.integers(-127, 128, (N, H)).astype(np.int8)
    bias = rng.integers(-5000, 5000, N).astype(np.int32)
    S_w = rng.uniform(1e-3, 2e-3, N)
    out, S_ret = ctx().ibert_classifier_i8(dev(x), B, L, 0.03, dev(w), S_w, dev(bias))
    ctx().check()
    assert_same(host(out), oracle.classifier(x, B, L, 0.03, w, S_w, bias), "classifier")
    assert np.array_equal(S_ret, 0.03 * S_w)
