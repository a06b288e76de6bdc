"""Tensors with more than 2^31 elements or bytes: index arithmetic beyond 32 bits in every kernel
class.  The inputs are drawn on the device; the oracle checks sampled rows / sequences (rows of a
linear layer and of LayerNorm, and sequences of attention, are independent of one another)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu


def _rows(M, n=96):
    g = np.random.default_rng(M)
    return np.unique(np.concatenate([np.arange(0, 40), np.arange(M - 40, M), g.integers(0, M, n),
                                     np.arange(2 ** 31 // 768 - 3, 2 ** 31 // 768 + 3)]).clip(0, M - 1))


def test_linear_with_more_than_2_31_output_elements():
    M, N, K = 2_900_000, 768, 768                      # 2.23e9 outputs
    gen = torch.Generator(device="cuda").manual_seed(1)
    x = torch.randint(-127, 128, (M, K), generator=gen, dtype=torch.int8, device="cuda")
    rng = np.random.default_rng(1)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-200000, 200000, N).astype(np.int32)
    S_w, S_x = rng.uniform(1e-4, 4e-4, N), 0.03
    S_out = 127.0 * 127.0 * np.sqrt(K) * 1.2 * S_x * 2.5e-4 / 100.0
    rows = _rows(M)
    xs = host(x[torch.from_numpy(rows).cuda()])
    for kind in (0, 1):                                # int8 (2.2 GB) and Q16 in int32 (8.9 GB)
        out, _ = ctx().ibert_linear_i8(x, S_x, dev(w), S_w, dev(bias), kind, S_out if kind == 0 else S_out / 200.0)
        ctx().check()
        got = host(out[torch.from_numpy(rows).cuda()])
        del out
        assert_same(got, oracle.linear(xs, S_x, w, S_w, bias, kind, S_out if kind == 0 else S_out / 200.0), f"kind {kind}")


def test_layernorm_with_more_than_2_31_elements():
    rows_n, C = 2_900_000, 768
    q0, S, r0, S_r, gamma, beta, S_out = synth.layernorm_inputs(4096, C, 1.0)
    reps = (rows_n + 4095) // 4096
    q = dev(q0).repeat(reps, 1)[:rows_n].contiguous()           # 8.9 GB of int32
    r = dev(r0).repeat(reps, 1)[:rows_n].contiguous()
    shift = torch.arange(rows_n, device="cuda", dtype=torch.int32) % 977    # rows differ from their copies
    q += shift[:, None]
    out, _ = ctx().ibert_layernorm_i(q, S, r, S_r, gamma, beta, S_out)
    ctx().check()
    rows = _rows(rows_n)
    idx = torch.from_numpy(rows).cuda()
    want, _ = oracle.layernorm(host(q[idx]), S, host(r[idx]), S_r, gamma, beta, S_out)
    assert_same(host(out[idx]), want, "layernorm rows")


def test_attention_with_more_than_2_31_input_bytes():
    B, L, heads = 1400, 512, 16                        # qkv: 716800 tokens x 3072 bytes = 2.2e9
    H = heads * 64
    gen = torch.Generator(device="cuda").manual_seed(2)
    qkv = (torch.randn((B * L, 3 * H), generator=gen, device="cuda") * 40).round().clamp(-127, 127).to(torch.int8)
    out, _ = ctx().ibert_attention_i8(qkv, B, L, H, heads, 0.02, 0.02, 0.02, 0.006, 255)
    ctx().check()
    for b in (0, 681, 683, B - 1):                     # around byte offset 2^31 and at both ends
        seq = host(qkv[b * L:(b + 1) * L])
        want = oracle.attention(seq, 1, L, H, heads, 0.02, 0.02, 0.02, 0.006, 255)
        assert_same(host(out[b * L:(b + 1) * L]), want, f"sequence {b}")


def test_linear_layernorm_cluster_kernel_with_more_than_2_31_output_elements():
    T, H, K = 2_900_000, 768, 256
    gen = torch.Generator(device="cuda").manual_seed(3)
    x = torch.randint(-127, 128, (T, K), generator=gen, dtype=torch.int8, device="cuda")
    res = torch.randint(-127, 128, (T, H), generator=gen, dtype=torch.int8, device="cuda")
    rng = np.random.default_rng(3)
    w = rng.integers(-127, 128, (H, K)).astype(np.int8)
    bias = rng.integers(-20000, 20000, H).astype(np.int32)
    S_w, S_x = rng.uniform(1e-4, 4e-4, H), 0.03
    S_mid = 127.0 * 127.0 * np.sqrt(K) * 1.2 * S_x * 2.5e-4 / 8000.0
    S_res = S_mid * 100.0
    gamma, beta, S_out = rng.normal(1, 0.1, H), rng.normal(0, 0.1, H), 4.0 / 127.0
    out, _ = ctx().ibert_linear_layernorm_i8(x, S_x, dev(w), S_w, dev(bias), S_mid, res, S_res, gamma, beta, S_out)
    ctx().check()
    rows = _rows(T)
    idx = torch.from_numpy(rows).cuda()
    mid = oracle.linear(host(x[idx]), S_x, w, S_w, bias, 1, S_mid)
    want, _ = oracle.layernorm(mid, S_mid, host(res[idx]), S_res, gamma, beta, S_out)
    assert_same(host(out[idx]), want, "linear + layernorm rows")


def test_encoder_layer_on_2_9_million_tokens():
    """One RoBERTa-Base shaped layer on 22656 sequences of 128 tokens: every activation of the layer
    (the FFN one is 8.9e9 bytes) is indexed beyond 2^31.  Sequences are independent: the oracle runs
    the first, the last and two in between."""
    B, L = 22656, 128
    x8, params = synth.make_model(2, 8, layers=1)
    p = params[0]
    gen = torch.Generator(device="cuda").manual_seed(4)
    x = (torch.randn((B * L, p["H"]), generator=gen, device="cuda") * 40).round().clamp(-127, 127).to(torch.int8)
    layer = ctx().ibert_layer_create(p)
    out, _ = ctx().ibert_encoder_layer(layer, x, B, L)
    ctx().check()
    for b in (0, 5461, 16383, B - 1):
        seq = host(x[b * L:(b + 1) * L])
        assert_same(host(out[b * L:(b + 1) * L]), oracle.encoder_layer(p, seq, 1, L).out, f"sequence {b}")
    layer.close()
