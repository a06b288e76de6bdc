"""GPU parity (bit-exact) of the packed-batch calls -- sequences of different lengths stored without
padding -- against the oracle's masked operators on the padded batch, restricted to the valid rows
(valid rows of a masked layer depend on valid rows of their own sequence only)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import binding, synth

pytestmark = pytest.mark.gpu

SC = dict(S_q=0.02, S_k=0.02, S_v=0.02, S_ctx=0.006)


def _lens(B, L, seed, allow_empty=True):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, L + 1, B).astype(np.int32)
    special = [L, 1, 0 if allow_empty else 2, min(32, L), min(33, L), max(L - 1, 1), min(128, L), min(129, L)]
    lens[:min(B, len(special))] = special[:min(B, len(special))]
    return lens


def _pack(padded, lens, L):
    """[B*L, C] padded rows -> [sum lens, C] valid rows in sequence order."""
    rows = np.concatenate([np.arange(b * L, b * L + n) for b, n in enumerate(lens)]) if lens.sum() else np.zeros(0, int)
    return np.ascontiguousarray(padded[rows]), rows


def _cu(lens):
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)


@pytest.mark.parametrize("B,L,heads", [(8, 128, 2), (9, 100, 1), (8, 37, 3), (10, 256, 2), (8, 200, 1), (9, 512, 1),
                                       (8, 384, 2), (40, 160, 8), (300, 64, 1)])
@pytest.mark.parametrize("p_max", [255, 127])
def test_packed_attention_matches_masked_oracle_on_valid_rows(B, L, heads, p_max):
    H = heads * 64
    rng = np.random.default_rng(L + heads)
    qkv = np.clip(np.rint(rng.standard_normal((B * L, 3 * H)) * 40), -127, 127).astype(np.int8)
    lens = _lens(B, L, L + 1)
    packed, rows = _pack(qkv, lens, L)
    out, S_ret = ctx().ibert_attention_packed_i8(dev(packed), dev(_cu(lens)), L, H, heads, **SC, p_max=p_max)
    ctx().check()
    assert S_ret == SC["S_ctx"]
    want = oracle.attention(qkv, B, L, H, heads, **SC, p_max=p_max, lens=lens)[rows]
    assert_same(host(out), want, f"packed attention L={L}")
    assert np.abs(want).max() > 5


@pytest.mark.parametrize("B,L,H,heads,F", [(6, 64, 256, 4, 1024), (9, 128, 768, 12, 3072), (5, 200, 128, 2, 256),
                                           (40, 128, 768, 12, 3072), (3, 300, 1024, 16, 512)])
@pytest.mark.parametrize("fusion", [0, 1, 2])
def test_packed_encoder_layer_matches_masked_oracle_on_valid_rows(B, L, H, heads, F, fusion):
    x, params = synth.make_model(0, B, layers=1, H=H, heads=heads, F=F, L=L)
    lens = _lens(B, L, B + L)
    packed, rows = _pack(x, lens, L)
    c = ctx()
    layer = c.ibert_layer_create(params[0])
    c.ibert_set_fusion(fusion)
    try:
        out, S_out = c.ibert_encoder_layer_packed(layer, dev(packed), dev(_cu(lens)), L)
        c.check()
    finally:
        c.ibert_set_fusion(0)
        layer.close()
    want = oracle.encoder_layer(params[0], x, B, L, lens=lens).out[rows]
    assert S_out == params[0]["S_out"]
    assert_same(host(out), want, f"packed layer B={B} L={L} H={H} fusion={fusion}")


def test_packed_model_embedding_layers_classifier():
    B, L, H, heads, F = 12, 96, 256, 4, 512
    m = synth.make_full_model(2, B, layers=2, H=H, heads=heads, F=F, L=L, vocab=1000)
    lens = _lens(B, L, 5, allow_empty=False)
    ids_packed, rows = _pack(m["ids"].reshape(-1, 1), lens, L)
    ids_packed = ids_packed.reshape(-1)
    cu = dev(_cu(lens))
    e, hd = m["emb"], m["head"]
    c = ctx()
    layers = [c.ibert_layer_create(p) for p in m["layers"]]
    try:
        h, _ = c.ibert_embedding_packed_i8(dev(ids_packed), cu, L, dev(e["word"]), e["S_word"], dev(e["pos"]), e["S_pos"],
                                           e["gamma"], e["beta"], e["S_out"])
        emb_got = host(h)
        for ly in layers:
            h, _ = c.ibert_encoder_layer_packed(ly, h, cu, L)
        logits, S_log = c.ibert_classifier_packed_i8(h, cu, m["layers"][-1]["S_out"], dev(hd["w"]), hd["S_w"], dev(hd["bias"]))
        c.check()
    finally:
        for ly in layers:
            ly.close()
    # oracle on the padded batch: position of a token = its index inside the sequence
    ho = oracle.embedding(m["ids"], L, e["word"], e["S_word"], e["pos"], e["S_pos"], e["gamma"], e["beta"], e["S_out"])
    assert_same(emb_got, ho[rows], "packed embedding")
    for p in m["layers"]:
        ho = oracle.encoder_layer(p, ho, B, L, lens=lens).out
    assert_same(host(h), ho[rows], "packed layers")
    want = oracle.classifier(ho, B, L, m["layers"][-1]["S_out"], hd["w"], hd["S_w"], hd["bias"])
    assert_same(host(logits), want, "packed classifier")


def test_packed_calls_validate_their_arguments():
    c = ctx()
    H = 64
    qkv = torch.zeros((10, 3 * H), dtype=torch.int8, device="cuda")
    cu = dev(np.array([0, 4, 10], np.int32))
    with pytest.raises(binding.IbertError) as e:
        c.ibert_attention_packed_i8(qkv, cu, 4, H, 1, **SC)            # 10 rows > B * max_len
    assert e.value.code == -2
    # a sequence longer than max_len is reported through the status word
    out, _ = c.ibert_attention_packed_i8(qkv, cu, 5, H, 1, **SC)
    assert c.ibert_last_status() == -8
    assert c.ibert_last_status() == 0
