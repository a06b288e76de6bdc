"""Pins for the oracle's INT8 MatMul + requant, attention head and encoder layer."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2101_01321_b200 import synth


def _requant_np(acc, S_x, S_w, S_out, qmax):
    out = np.empty(acc.shape, dtype=np.int64)
    for n in range(acc.shape[1]):
        b, c = oracle.dyadic((S_x * S_w[n]) / S_out[n])
        for m in range(acc.shape[0]):
            v = math.floor(Fraction(int(acc[m, n]) * b, 2 ** c) + Fraction(1, 2))
            out[m, n] = max(-qmax, min(qmax, v))
    return out


@pytest.mark.parametrize("M,N,K", [(5, 7, 16), (33, 20, 48), (128, 96, 80)])
def test_linear_equals_numpy_int64_matmul_and_exact_requant(M, N, K):
    rng = np.random.default_rng(M * N)
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    bias = rng.integers(-50000, 50000, N).astype(np.int32)
    S_w = rng.uniform(1e-4, 1e-3, N)
    S_x = 0.03
    acc = x.astype(np.int64) @ w.astype(np.int64).T + bias
    raw = oracle.linear(x, S_x, w, S_w, bias, 2)
    assert raw.dtype == np.int32 and (raw == acc).all()
    # non-symmetric operands: a transposed weight would fail this
    assert not (raw == (x.astype(np.int64) @ w.astype(np.int64)[:, ::-1].T + bias)).all()
    S_o8 = np.full(N, np.abs(acc * S_x * S_w).max() / 300.0)       # some values clamp
    got8 = oracle.linear(x, S_x, w, S_w, bias, 0, S_o8[0])
    assert got8.dtype == np.int8 and (got8 == _requant_np(acc, S_x, S_w, S_o8, 127)).all()
    assert np.abs(got8.astype(np.int64)).max() == 127
    S_o16 = np.full(N, np.abs(acc * S_x * S_w).max() / 32767.0)
    got16 = oracle.linear(x, S_x, w, S_w, bias, 1, S_o16[0])
    assert got16.dtype == np.int32 and (got16 == _requant_np(acc, S_x, S_w, S_o16, 32767)).all()
    # per-column output scales
    S_cols = rng.uniform(0.5, 2.0, N) * S_o8
    gotc = oracle.linear(x, S_x, w, S_w, bias, 0, 0.0, S_cols)
    assert (gotc == _requant_np(acc, S_x, S_w, S_cols, 127)).all()
    # no bias
    assert (oracle.linear(x, S_x, w, S_w, None, 2) == acc - bias).all()


def test_linear_tracks_the_float_product():
    rng = np.random.default_rng(9)
    M, N, K = 64, 48, 256
    x = rng.integers(-127, 128, (M, K)).astype(np.int8)
    w = rng.integers(-127, 128, (N, K)).astype(np.int8)
    S_w = rng.uniform(1e-4, 2e-4, N)
    S_x = 0.03
    real = (x * S_x) @ (w * S_w[:, None]).T
    S_out = np.abs(real).max() / 127.0
    got = oracle.linear(x, S_x, w, S_w, None, 0, S_out)
    assert np.abs(got * S_out - real).max() <= S_out * (0.5 + 1e-6)


def _attention_by_parts(qkv, B, L, H, heads, S_q, S_k, S_v, S_ctx, M):
    T = B * L
    q3 = qkv.reshape(B, L, 3, heads, 64).astype(np.int64)
    ctx = np.empty((B, L, heads, 64), dtype=np.int64)
    b, c = oracle.dyadic(((1.0 / M) * S_v) / S_ctx)
    for bi in range(B):
        for h in range(heads):
            s = q3[bi, :, 0, h] @ q3[bi, :, 1, h].T
            p, _ = oracle.softmax(s.astype(np.int32), (S_q * S_k) / 8.0, M)
            acc = p.astype(np.int64) @ q3[bi, :, 2, h]
            for i in range(L):
                for t in range(64):
                    ctx[bi, i, h, t] = oracle.requant(int(acc[i, t]), b, c, 127)
    return ctx.reshape(T, H)


@pytest.mark.parametrize("B,L,heads,M", [(2, 16, 2, 255), (1, 37, 1, 127)])
def test_attention_is_matmul_softmax_matmul_requant(B, L, heads, M):
    H = heads * 64
    rng = np.random.default_rng(L)
    qkv = rng.integers(-127, 128, (B * L, 3 * H)).astype(np.int8)
    S_q = S_k = 0.02
    S_v, S_ctx = 0.015, 0.004
    ctx, probs = oracle.attention(qkv, B, L, H, heads, S_q, S_k, S_v, S_ctx, M, want_probs=True)
    assert (ctx == _attention_by_parts(qkv, B, L, H, heads, S_q, S_k, S_v, S_ctx, M)).all()
    sums = probs.astype(np.int64).sum(axis=-1)
    assert (sums <= M).all() and (sums > M - L).all()


def test_attention_tracks_float_attention():
    B, L, heads = 1, 64, 2
    H = heads * 64
    rng = np.random.default_rng(5)
    S_q = S_k = 0.03
    S_v = 0.02
    qkv = np.clip(np.rint(rng.standard_normal((L, 3 * H)) * 30), -127, 127).astype(np.int8)
    f = qkv.reshape(L, 3, heads, 64).astype(np.float64)
    real = np.empty((L, heads, 64))
    for h in range(heads):
        s = (f[:, 0, h] * S_q) @ (f[:, 1, h] * S_k).T / 8.0
        e = np.exp(s - s.max(axis=1, keepdims=True))
        real[:, h] = (e / e.sum(axis=1, keepdims=True)) @ (f[:, 2, h] * S_v)
    S_ctx = np.abs(real).max() / 127.0
    ctx = oracle.attention(qkv, B, L, H, heads, S_q, S_k, S_v, S_ctx, 255)
    # probabilities are floored to 1/255 steps: each row loses < L/255 of its mass
    err = np.abs(ctx.reshape(L, heads, 64) * S_ctx - real)
    assert err.max() <= 0.5 * S_ctx + (L / 255.0 + 3e-3) * np.abs(f[:, 2] * S_v).max()
    assert np.corrcoef(ctx.reshape(-1), real.reshape(-1))[0, 1] > 0.97


def _small_layer(B=2, L=16, H=128, heads=2, F=256, seed_cfg=0):
    x, S_x = synth.make_input(seed_cfg, B, L, H)
    p = synth.make_layer(seed_cfg, 0, H, heads, F, L, S_x)
    return x, p


def test_encoder_layer_is_the_composition_of_its_pinned_ops():
    B, L = 2, 16
    x, p = _small_layer(B, L)
    H, F = p["H"], p["F"]
    res = oracle.encoder_layer(p, x, B, L, want_taps=True)
    t = res.taps
    so = np.concatenate([np.full(H, p["S_q"]), np.full(H, p["S_k"]), np.full(H, p["S_v"])])
    qkv = oracle.linear(x, p["S_x"], p["w_qkv"], p["S_w_qkv"], p["bias_qkv"], 0, 0.0, so)
    assert (t["qkv"] == qkv).all()
    ctx = oracle.attention(qkv, B, L, H, p["heads"], p["S_q"], p["S_k"], p["S_v"], p["S_ctx"], p["p_max"])
    assert (t["ctx"] == ctx).all()
    r1 = oracle.linear(ctx, p["S_ctx"], p["w_o"], p["S_w_o"], p["bias_o"], 1, p["S_r1"])
    assert (t["r1"] == r1).all()
    h1, _ = oracle.layernorm(r1, p["S_r1"], x, p["S_x"], p["gamma1"], p["beta1"], p["S_h1"])
    assert (t["h1"] == h1).all()
    gi = oracle.linear(h1, p["S_h1"], p["w_f1"], p["S_w_f1"], p["bias_f1"], 1, p["S_gi"])
    g, _ = oracle.gelu(gi, p["S_gi"], p["S_go"])
    assert (t["g"] == g).all()
    r2 = oracle.linear(g, p["S_go"], p["w_f2"], p["S_w_f2"], p["bias_f2"], 1, p["S_r2"])
    assert (t["r2"] == r2).all()
    out, _ = oracle.layernorm(r2, p["S_r2"], h1, p["S_h1"], p["gamma2"], p["beta2"], p["S_out"])
    assert (res.out == out).all()


def _float_layer_taps(p, x, B, L, mistake=None):
    """float64 post-LN encoder layer (Fig. 1 left) on the dequantized parameters, with its intermediate
    tensors.  `mistake` plants one plausible wiring error, to show that the comparison below notices it."""
    H, heads = p["H"], p["heads"]
    erf = np.vectorize(math.erf)
    W = {n: p[f"w_{n}"].astype(np.float64) * p[f"S_w_{n}"][:, None] for n in ("qkv", "o", "f1", "f2")}
    sx = {"qkv": p["S_x"], "o": p["S_ctx"], "f1": p["S_h1"], "f2": p["S_go"]}
    bf = {n: p[f"bias_{n}"] * sx[n] * p[f"S_w_{n}"] for n in W}
    if mistake == "no_bias":
        bf = {n: 0.0 * v for n, v in bf.items()}
    xf = x.astype(np.float64) * p["S_x"]
    qkv2 = xf @ W["qkv"].T + bf["qkv"]
    qkv = qkv2.reshape(B, L, 3, heads, 64)
    iq, ik, iv = (0, 2, 1) if mistake == "k_and_v_swapped" else (0, 1, 2)
    ctx = np.empty((B, L, heads, 64))
    for b in range(B):
        for h in range(heads):
            s = qkv[b, :, iq, h] @ qkv[b, :, ik, h].T / (1.0 if mistake == "no_sqrt_d" else 8.0)
            e = np.exp(s - s.max(axis=1, keepdims=True))
            ctx[b, :, h] = (e / e.sum(axis=1, keepdims=True)) @ qkv[b, :, iv, h]
    if mistake == "heads_interleaved":
        ctx = ctx.transpose(0, 1, 3, 2)
    ctx2 = ctx.reshape(B * L, H)
    o = ctx2 @ W["o"].T + bf["o"]

    def ln(v, g, be):
        if mistake == "ln_without_variance":
            return (v - v.mean(1, keepdims=True)) * g + be
        return (v - v.mean(1, keepdims=True)) / v.std(1, keepdims=True) * g + be
    g1, b1, g2, b2 = p["gamma1"], p["beta1"], p["gamma2"], p["beta2"]
    if mistake == "layernorms_swapped":
        g1, b1, g2, b2 = g2, b2, g1, b1
    h1 = ln((0.0 if mistake == "no_residual_1" else xf) + o, g1, b1)
    z = h1 @ W["f1"].T + bf["f1"]
    gz = np.maximum(z, 0.0) if mistake == "relu" else z * 0.5 * (1.0 + erf(z / math.sqrt(2.0)))
    res2 = {"no_residual_2": 0.0, "residual_2_from_x": xf}.get(mistake, h1)
    out = ln(res2 + gz @ W["f2"].T + bf["f2"], g2, b2)
    return {"qkv": qkv2, "ctx": ctx2, "h1": h1, "g": gz, "out": out}


# mean / 99th percentile of |integer tap - float tap| in steps of the tap's scale: about twice what
# the correct wiring shows on this input (0.25/0.49, 1.49/4.91, 0.25/0.54, 0.69/1.58, 0.35/1.03)
_TAP_BOUNDS = {"qkv": (0.5, 1.0), "ctx": (3.0, 10.0), "h1": (0.5, 1.1), "g": (1.4, 3.2), "out": (0.7, 2.1)}


def _tap_errors(p, x, B, L, res, mistake=None):
    H = p["H"]
    scales = {"qkv": np.concatenate([np.full(H, p["S_q"]), np.full(H, p["S_k"]), np.full(H, p["S_v"])]),
              "ctx": p["S_ctx"], "h1": p["S_h1"], "g": p["S_go"], "out": p["S_out"]}
    ft = _float_layer_taps(p, x, B, L, mistake)
    errs = {}
    for name, S in scales.items():
        got = (res.out if name == "out" else res.taps[name]).astype(np.float64)
        e = np.abs(got - np.clip(ft[name] / S, -127, 127))
        errs[name] = (e.mean(), np.percentile(e, 99))
    return errs


def test_encoder_layer_tracks_a_float_layer_tap_by_tap():
    """The pin of the composed layer against something that is not the oracle: a float64 textbook
    post-LN encoder layer on the dequantized parameters.  Every intermediate tensor of the integer
    layer stays within quantization noise of its float counterpart, and the static scales of the
    synthetic recipe clamp almost nothing."""
    B, L = 2, 32
    x, p = _small_layer(B, L, H=256, heads=4, F=1024)
    res = oracle.encoder_layer(p, x, B, L, want_taps=True)
    for name, (mean, p99) in _tap_errors(p, x, B, L, res).items():
        assert mean < _TAP_BOUNDS[name][0] and p99 < _TAP_BOUNDS[name][1], (name, mean, p99)
    for name, qmax in (("qkv", 127), ("ctx", 127), ("h1", 127), ("g", 127), ("r1", 32767), ("r2", 32767)):
        frac = (np.abs(res.taps[name]) >= qmax).mean()
        assert frac < 0.01, (name, frac)
        if qmax == 127:       # (r1, r2 hold one addend at the scale of the residual *sum*)
            assert np.abs(res.taps[name]).max() > 60, name          # and the range is used


@pytest.mark.parametrize("mistake", ["no_sqrt_d", "k_and_v_swapped", "heads_interleaved", "no_residual_1",
                                     "no_residual_2", "residual_2_from_x", "layernorms_swapped", "relu",
                                     "ln_without_variance", "no_bias"])
def test_the_float_comparison_notices_a_wiring_mistake(mistake):
    """Each plausible mistake, planted in the float layer, pushes at least one tap outside the bounds
    the correct wiring meets -- so the same mistake inside the oracle would fail the test above."""
    B, L = 2, 32
    x, p = _small_layer(B, L, H=256, heads=4, F=1024)
    res = oracle.encoder_layer(p, x, B, L, want_taps=True)
    errs = _tap_errors(p, x, B, L, res, mistake)
    assert any(mean > _TAP_BOUNDS[n][0] or p99 > _TAP_BOUNDS[n][1] for n, (mean, p99) in errs.items()), errs


def test_layers_chain_through_their_scales():
    x, params = synth.make_model(2, 1, layers=2, H=128, heads=2, F=256, L=16)
    assert params[1]["S_x"] == params[0]["S_out"]
    h = x
    for p in params:
        h = oracle.encoder_layer(p, h, 1, 16).out
    assert h.dtype == np.int8 and np.abs(h).max() <= 127 and h.std() > 10
