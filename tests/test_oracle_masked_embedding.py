"""Pins of the oracle functions around the plain layer: attention with a key-padding mask, the
encoder layer on padded sequences, the INT8 embedding + i-LayerNorm and the first-token classifier.

The paper defines none of these beyond "the Embedding is kept at INT8" (implementation appendix);
each is a composition of functions pinned elsewhere, so the pins here check the composition against
definitions that do not go through the function under test: attention / layers of the truncated
sequences, numpy gathers, an int64 numpy matmul."""
import numpy as np
import pytest

import oracle
from paper_2101_01321_b200 import synth

SC = dict(S_q=0.02, S_k=0.02, S_v=0.02, S_ctx=0.01)


def _qkv(B, L, H, seed):
    rng = np.random.default_rng(seed)
    return np.clip(np.rint(rng.standard_normal((B * L, 3 * H)) * 40), -127, 127).astype(np.int8)


def test_mask_with_full_lengths_is_the_plain_attention():
    B, L, heads = 3, 50, 2
    H = heads * 64
    qkv = _qkv(B, L, H, 1)
    plain = oracle.attention(qkv, B, L, H, heads, **SC)
    masked = oracle.attention(qkv, B, L, H, heads, **SC, lens=np.full(B, L, np.int32))
    assert np.array_equal(plain, masked)


@pytest.mark.parametrize("p_max", [255, 127])
def test_valid_rows_equal_attention_of_the_truncated_sequence(p_max):
    B, L, heads = 4, 70, 2
    H = heads * 64
    qkv = _qkv(B, L, H, 2)
    lens = np.array([70, 33, 1, 64], np.int32)
    ctx, probs = oracle.attention(qkv, B, L, H, heads, **SC, p_max=p_max, want_probs=True, lens=lens)
    for b, n in enumerate(lens):
        seq = qkv[b * L:(b + 1) * L]
        want = oracle.attention(seq[:n], 1, int(n), H, heads, **SC, p_max=p_max)
        assert np.array_equal(ctx[b * L:b * L + n], want), b
        assert probs[b, :, :, n:].max(initial=0) == 0                    # masked keys: probability 0
        rows = probs[b, :, :, :n].astype(np.int64).sum(-1)
        assert rows.max() <= p_max and rows.min() >= p_max - n           # floors lose < 1 per key


def test_padded_query_rows_attend_to_the_valid_keys():
    """A padded query's context depends only on its q vector and the valid K, V: moving that q
    vector into row 0 of the truncated sequence must reproduce it."""
    B, L, heads = 1, 40, 1
    H = 64
    qkv = _qkv(B, L, H, 3)
    n = 13
    ctx = oracle.attention(qkv, B, L, H, heads, **SC, lens=np.array([n], np.int32))
    for i in (n, 25, L - 1):
        trunc = qkv[:n].copy()
        trunc[0, :H] = qkv[i, :H]
        want = oracle.attention(trunc, 1, n, H, heads, **SC)
        assert np.array_equal(ctx[i], want[0]), i


def test_sequence_without_valid_keys_gives_zero_context():
    B, L, heads = 2, 20, 1
    qkv = _qkv(B, L, 64, 4)
    ctx = oracle.attention(qkv, B, L, 64, heads, **SC, lens=np.array([0, 20], np.int32))
    assert not ctx[:L].any()
    assert np.array_equal(ctx[L:], oracle.attention(qkv[L:], 1, L, 64, heads, **SC))


def test_masked_layer_valid_rows_equal_the_layer_on_truncated_sequences():
    B, L, H, heads, F = 3, 24, 64, 1, 128
    x, params = synth.make_model(0, B, layers=1, H=H, heads=heads, F=F, L=L)
    p = params[0]
    lens = np.array([24, 9, 16], np.int32)
    got = oracle.encoder_layer(p, x, B, L, lens=lens).out
    assert np.array_equal(oracle.encoder_layer(p, x, B, L, lens=np.full(B, L, np.int32)).out,
                          oracle.encoder_layer(p, x, B, L).out)
    for b, n in enumerate(lens):
        want = oracle.encoder_layer(p, x[b * L:b * L + n], 1, int(n)).out
        assert np.array_equal(got[b * L:b * L + n], want), b


def test_embedding_is_gather_plus_layernorm():
    rng = np.random.default_rng(5)
    V, P, H, B, L = 300, 40, 96, 3, 17
    word = rng.integers(-127, 128, (V, H)).astype(np.int8)
    pos = rng.integers(-127, 128, (P, H)).astype(np.int8)
    ids = rng.integers(0, V, B * L).astype(np.int32)
    gamma, beta = 1.0 + 0.1 * rng.standard_normal(H), 0.1 * rng.standard_normal(H)
    S_word, S_pos, S_out = 0.011, 0.004, 4.5 / 127
    got = oracle.embedding(ids, L, word, S_word, pos, S_pos, gamma, beta, S_out)
    a = word[ids].astype(np.int32)
    r = pos[np.arange(B * L) % L]
    want, _ = oracle.layernorm(a, S_word, r, S_pos, gamma, beta, S_out)
    assert np.array_equal(got, want)
    assert np.abs(got).max() > 60
    with pytest.raises(oracle.OracleError):
        oracle.embedding(np.array([V], np.int32), 1, word, S_word, pos, S_pos, gamma, beta, S_out)


def test_classifier_is_an_int64_matmul_on_the_first_tokens():
    rng = np.random.default_rng(6)
    B, L, H, N = 5, 12, 64, 16
    x = rng.integers(-127, 128, (B * L, H)).astype(np.int8)
    w = rng.integers(-127, 128, (N, H)).astype(np.int8)
    bias = rng.integers(-5000, 5000, N).astype(np.int32)
    S_w = rng.uniform(1e-3, 2e-3, N)
    got = oracle.classifier(x, B, L, 0.03, w, S_w, bias)
    want = x[::L].astype(np.int64) @ w.astype(np.int64).T + bias
    assert np.array_equal(got.astype(np.int64), want)
