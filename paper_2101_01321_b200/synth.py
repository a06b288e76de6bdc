"""Seeded synthetic inputs for the integer-only encoder layer.

This module only *makes inputs*: random tensors of the shapes and
distributions the workloads call for, quantized once to integers with
Eq. 1 (uniform symmetric, ``S = alpha / (2^(b-1) - 1)``), and the static
activation scales of a layer (Sec. 3.1: fixed offline).  None of the
method's integer arithmetic (requantization, i-exp, i-GELU, i-LayerNorm)
lives here, so the CPU oracle and the CUDA path can both be fed from it.

Generators are ``numpy.random.Generator(PCG64(seed))`` with
``seed = 21010000 + 1000*config + 10*layer + tensor_id``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from pathlib import Path

import numpy as np

SEED_BASE = 21010000

# tensor ids inside one layer
_T_X, _T_WQKV, _T_BQKV, _T_WO, _T_BO, _T_WF1, _T_BF1, _T_WF2, _T_BF2 = range(9)
# gamma1, beta1, gamma2, beta2 share id 9 (drawn in that order from one stream)
_T_LN = 9


@dataclass(frozen=True)
class ModelConfig:
    name: str
    H: int
    heads: int
    F: int
    layers: int
    L: int
    config_id: int


CONFIGS = {
    0: ModelConfig("roberta-base-1layer", 768, 12, 3072, 1, 128, 0),
    2: ModelConfig("roberta-base-12layer", 768, 12, 3072, 12, 128, 2),
    3: ModelConfig("roberta-large-24layer-L256", 1024, 16, 4096, 24, 256, 3),
    4: ModelConfig("roberta-large-24layer-L512", 1024, 16, 4096, 24, 512, 4),
}


def rng_for(config_id: int, layer: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(SEED_BASE + 1000 * config_id + 10 * layer + tensor_id))


def quantize_sym(x: np.ndarray, S, qmax: int) -> np.ndarray:
    """Eq. 1 with Int = round-to-nearest-even and clip to +-qmax."""
    return np.clip(np.rint(x / S), -qmax, qmax)


def _quantize_weight(rng: np.random.Generator, n_out: int, n_in: int, std: float = 0.02):
    """W ~ N(0, std^2), per-output-channel symmetric int8."""
    W = rng.standard_normal((n_out, n_in), dtype=np.float32).astype(np.float64) * std
    S_w = np.abs(W).max(axis=1) / 127.0
    w = quantize_sym(W, S_w[:, None], 127).astype(np.int8)
    return w, S_w


def _quantize_bias(rng: np.random.Generator, S_x: float, S_w: np.ndarray, std: float = 0.02):
    """float bias ~ N(0, std^2) held as int32 at scale S_x * S_w[n]."""
    bias = rng.standard_normal(S_w.shape[0]) * std
    return np.rint(bias / (S_x * S_w)).astype(np.int32)


def _gelu_second_moment(sigma: float) -> float:
    """E[GELU(z)^2] for z ~ N(0, sigma^2), by a plain Riemann sum."""
    z = np.linspace(-8.0 * sigma, 8.0 * sigma, 20001)
    erf = np.vectorize(math.erf)
    g = z * 0.5 * (1.0 + erf(z / math.sqrt(2.0)))
    pdf = np.exp(-0.5 * (z / sigma) ** 2) / (sigma * math.sqrt(2.0 * math.pi))
    return float(np.sum(g * g * pdf) * (z[1] - z[0]))


def static_activation_scales(H: int, F: int, L: int, S_x: float, w_std: float = 0.02) -> dict:
    """The 11 static activation scales of a layer, from the input distributions.

    The layer input has (close to) unit variance -- N(0,1) for the first
    layer, a LayerNorm output with gamma ~ N(1, 0.1^2), beta ~ N(0, 0.1^2)
    afterwards -- so every site's standard deviation follows from the weight
    distribution.  int8 sites clip at 4 (context: 5) standard deviations,
    Q16 sites (held in int32) at 8.
    """
    ln_var = 1.0 * (1.0 + 0.1 ** 2) + 0.1 ** 2            # E[(gamma n + beta)^2], n ~ N(0,1)
    sd_qkv = w_std * math.sqrt(H * 1.0 + 1.0)
    sd_ctx = w_std * math.sqrt(H / L + 1.0)                # ~ mean of L value rows (+ bias)
    sd_o = w_std * math.sqrt(H * sd_ctx ** 2 + 1.0)
    sd_f1 = w_std * math.sqrt(H * ln_var + 1.0)
    sd_f2 = w_std * math.sqrt(F * _gelu_second_moment(sd_f1) + 1.0)
    s = {
        "S_x": float(S_x),
        "S_q": 4.0 * sd_qkv / 127.0,
        "S_k": 4.0 * sd_qkv / 127.0,
        "S_v": 4.0 * sd_qkv / 127.0,
        "S_ctx": 5.0 * sd_ctx / 127.0,
        "S_r1": 8.0 * math.sqrt(ln_var + sd_o ** 2) / 32767.0,
        "S_h1": 4.0 * math.sqrt(ln_var) / 127.0,
        "S_gi": 8.0 * sd_f1 / 32767.0,
        "S_go": 4.0 * sd_f1 / 127.0,
        "S_r2": 8.0 * math.sqrt(ln_var + sd_f2 ** 2) / 32767.0,
        "S_out": 4.0 * math.sqrt(ln_var) / 127.0,
    }
    return s


def snap_q_scale(S_q: float, S_k: float) -> float:
    """The smallest S_q' >= S_q for which the score scale S_q' S_k / 8 is ln2 / 2^k for an integer
    k <= 14 (a static-quantization choice: the query scale is free as long as it covers the range).
    With such a scale the i-exp quotient floor(d / q_ln2) has q_ln2 = 2^k exactly."""
    ln2 = 0.6931471805599453
    k = min(int(math.floor(math.log2(8.0 * ln2 / (S_q * S_k)))), 14)
    S = 8.0 * ln2 / (2.0 ** k * S_k)
    for _ in range(64):                       # a few ulps down until floor(ln2 / score scale) is 2^k
        if math.floor(ln2 / ((S * S_k) / 8.0)) == 2 ** k:
            break
        S = float(np.nextafter(S, 0.0))
    assert S >= S_q * (1.0 - 1e-12) and math.floor(ln2 / ((S * S_k) / 8.0)) == 2 ** k
    return S


def make_input(config_id: int, B: int, L: int, H: int, shard: int = 0):
    """x ~ N(0,1) as int8 with S_x = max|x| / 127.  Returns (x_q [B*L, H], S_x).

    `shard` selects the slice of a data-parallel global batch (one seeded stream per shard,
    tensor id 100*shard).  The static scale S_x is always the one of shard 0, so every rank
    quantizes with the same scale (later shards clip the few values beyond it)."""
    x0 = rng_for(config_id, 0, _T_X).standard_normal((B * L, H), dtype=np.float32).astype(np.float64)
    S_x = float(np.abs(x0).max() / 127.0)
    if shard == 0:
        x = x0
    else:
        x = rng_for(config_id, 0, _T_X + 100 * shard).standard_normal((B * L, H), dtype=np.float32).astype(np.float64)
    return quantize_sym(x, S_x, 127).astype(np.int8), S_x


CALIBRATED_SCALES_FILE = Path(__file__).resolve().parent.parent / "tests" / "golden" / "calibrated_scales.json"
_calibrated = None


def calibrated_scales(config_id: int, layer: int) -> dict:
    """The ten static activation scales S_q .. S_out of one layer as calibrated offline: each site's
    max|x| on the first sequences of the seeded input (Sec. 3.1: scales are fixed before inference).
    The file is written by tests/golden/make_calibrated_scales.py; this module only reads it."""
    global _calibrated
    if _calibrated is None:
        import json
        if not CALIBRATED_SCALES_FILE.exists():
            raise FileNotFoundError(f"{CALIBRATED_SCALES_FILE} is missing (run tests/golden/make_calibrated_scales.py)")
        _calibrated = json.loads(CALIBRATED_SCALES_FILE.read_text())
    layers = _calibrated["configs"][str(config_id)]["layers"]
    if layer >= len(layers):
        raise ValueError(f"no calibrated scales for config {config_id}, layer {layer}")
    return {k: float(v) for k, v in layers[layer].items()}


def make_layer(config_id: int, layer: int, H: int, heads: int, F: int, L: int, S_x: float,
               p_max: int = 255, pow2_scores: bool = False, scales: dict | None = None) -> dict:
    """One layer's integer parameters and static scales (a plain dict of numpy arrays).
    pow2_scores: the query scale is raised (by less than 2x) so that the score scale is ln2 / 2^k.
    scales: the activation scales S_q .. S_out to use instead of the closed-form ones."""
    assert H == heads * 64
    p = {"H": H, "heads": heads, "F": F, "p_max": p_max}
    p.update(static_activation_scales(H, F, L, S_x))
    if scales:
        p.update({k: float(v) for k, v in scales.items() if k != "S_x"})
    if pow2_scores:
        p["S_q"] = snap_q_scale(p["S_q"], p["S_k"])
    in_scale = {"qkv": p["S_x"], "o": p["S_ctx"], "f1": p["S_h1"], "f2": p["S_go"]}
    shapes = {"qkv": (3 * H, H), "o": (H, H), "f1": (F, H), "f2": (H, F)}
    tids = {"qkv": (_T_WQKV, _T_BQKV), "o": (_T_WO, _T_BO), "f1": (_T_WF1, _T_BF1), "f2": (_T_WF2, _T_BF2)}
    for nm in ("qkv", "o", "f1", "f2"):
        w, S_w = _quantize_weight(rng_for(config_id, layer, tids[nm][0]), *shapes[nm])
        p[f"w_{nm}"] = w
        p[f"S_w_{nm}"] = S_w
        p[f"bias_{nm}"] = _quantize_bias(rng_for(config_id, layer, tids[nm][1]), in_scale[nm], S_w)
    rng = rng_for(config_id, layer, _T_LN)
    p["gamma1"] = 1.0 + 0.1 * rng.standard_normal(H)
    p["beta1"] = 0.1 * rng.standard_normal(H)
    p["gamma2"] = 1.0 + 0.1 * rng.standard_normal(H)
    p["beta2"] = 0.1 * rng.standard_normal(H)
    return p


def make_model(config_id: int, B: int, layers: int | None = None, H: int | None = None,
               heads: int | None = None, F: int | None = None, L: int | None = None, shard: int = 0,
               pow2_scores: bool = False, scales: str = "analytic"):
    """Input and per-layer parameters of one of the encoder configs (0, 2, 3, 4).
    Layer l+1 consumes layer l's int8 output, so its S_x is layer l's S_out.
    scales: "analytic" (closed-form, any shape) or "calibrated" (the stored per-layer scales of
    the config's own shape)."""
    cfg = CONFIGS[config_id]
    H = H or cfg.H
    heads = heads or cfg.heads
    F = F or cfg.F
    L = L or cfg.L
    layers = layers or cfg.layers
    x, S_x = make_input(config_id, B, L, H, shard)
    params = []
    s_in = S_x
    for l in range(layers):
        cal = calibrated_scales(config_id, l) if scales == "calibrated" else None
        p = make_layer(config_id, l, H, heads, F, L, s_in, pow2_scores=pow2_scores, scales=cal)
        params.append(p)
        s_in = p["S_out"]
    return x, params


# ---------------------------------------------------------------------------
# standalone non-linearity sweeps (config 1)
# ---------------------------------------------------------------------------

def gelu_inputs(n: int, sigma: float, tensor_id: int = 0):
    """x ~ N(0, sigma^2) as Q16 held in int32; S = max|x|/32767, S_out = max|x|/127."""
    rng = rng_for(1, 0, tensor_id)
    x = rng.standard_normal(n, dtype=np.float32).astype(np.float64) * sigma
    amax = float(np.abs(x).max())
    S = amax / 32767.0
    return quantize_sym(x, S, 32767).astype(np.int32), S, amax / 127.0


def softmax_inputs(rows: int, L: int, sigma: float, tensor_id: int = 1):
    """score-like int32 rows: x ~ N(0, sigma^2), S = sigma/16384 (|q| up to ~2^17)."""
    rng = rng_for(1, 1, tensor_id)
    x = rng.standard_normal((rows, L), dtype=np.float32).astype(np.float64) * sigma
    S = sigma / 16384.0
    return np.rint(x / S).astype(np.int32), S


def layernorm_inputs(rows: int, C: int, sigma: float, tensor_id: int = 2, with_residual: bool = True):
    """Q16 rows with a per-row offset, an int8 residual, gamma/beta and an output scale.

    x ~ N(0, sigma^2) + row offset N(0, (sigma/2)^2); S = max|x|/32767.
    The residual is N(0, (sigma/4)^2) as int8.  S_out covers 4.5 standard
    deviations of the normalized, affine-transformed output.
    """
    rng = rng_for(1, 2, tensor_id)
    x = rng.standard_normal((rows, C), dtype=np.float32).astype(np.float64) * sigma
    x += rng.standard_normal((rows, 1)) * (sigma / 2.0)
    gamma = 1.0 + 0.1 * rng.standard_normal(C)
    beta = 0.1 * rng.standard_normal(C)
    r = S_r = None
    total = x
    if with_residual:
        res = rng.standard_normal((rows, C), dtype=np.float32).astype(np.float64) * (sigma / 4.0)
        S_r = float(np.abs(res).max() / 127.0)
        r = quantize_sym(res, S_r, 127).astype(np.int8)
        total = x + res
    S = float(np.abs(total).max() / 32767.0)
    q = quantize_sym(x, S, 32767).astype(np.int32)
    S_out = 4.5 * math.sqrt(1.0 * (1.0 + 0.1 ** 2) + 0.1 ** 2) / 127.0
    return q, S, r, S_r, gamma, beta, S_out


# ---------------------------------------------------------------------------
# the model around the layers: padded batches, INT8 embedding, classifier head
# ---------------------------------------------------------------------------
_T_IDS, _T_LENS, _T_WORD, _T_POS, _T_EMB_LN, _T_HEAD_W, _T_HEAD_B = 20, 21, 22, 23, 24, 25, 26
VOCAB = 50265          # RoBERTa's vocabulary size
N_LABELS = 4           # label dimension of the head, padded to a multiple of 4


def make_lengths(config_id: int, B: int, L: int, shard: int = 0) -> np.ndarray:
    """Valid tokens per sequence, a sentence-length mix: half the batch uniform in [L/8, L/2],
    the other half uniform in [L/2, L] (mean ~0.53 L), at least one sequence of full length."""
    rng = rng_for(config_id, 0, _T_LENS + 100 * shard)
    short = rng.integers(max(L // 8, 1), L // 2 + 1, B)
    long_ = rng.integers(L // 2, L + 1, B)
    lens = np.where(rng.random(B) < 0.5, short, long_).astype(np.int32)
    lens[0] = L
    return lens


def make_full_model(config_id: int, B: int, layers: int | None = None, H: int | None = None,
                    heads: int | None = None, F: int | None = None, L: int | None = None,
                    vocab: int = VOCAB, shard: int = 0, scales: str = "analytic") -> dict:
    """Token ids, lengths, INT8 embedding tables, encoder layers and a first-token classifier.
    Word / position rows ~ N(0, 0.02^2)-like tables quantized with one symmetric int8 scale per
    table (Eq. 1); the embedding LayerNorm has gamma ~ N(1, 0.1), beta ~ N(0, 0.1) and an output
    scale covering 4 standard deviations, which is the first layer's S_x."""
    cfg = CONFIGS[config_id]
    H = H or cfg.H
    heads = heads or cfg.heads
    F = F or cfg.F
    L = L or cfg.L
    layers = layers or cfg.layers
    ids = rng_for(config_id, 0, _T_IDS + 100 * shard).integers(0, vocab, B * L).astype(np.int32)
    lens = make_lengths(config_id, B, L, shard)
    word_f = rng_for(config_id, 0, _T_WORD).standard_normal((vocab, H), dtype=np.float32).astype(np.float64) * 0.02
    pos_f = rng_for(config_id, 0, _T_POS).standard_normal((L + 2, H), dtype=np.float32).astype(np.float64) * 0.02
    S_word = float(np.abs(word_f).max() / 127.0)
    S_pos = float(np.abs(pos_f).max() / 127.0)
    rng = rng_for(config_id, 0, _T_EMB_LN)
    emb = {"word": quantize_sym(word_f, S_word, 127).astype(np.int8), "S_word": S_word,
           "pos": quantize_sym(pos_f, S_pos, 127).astype(np.int8), "S_pos": S_pos,
           "gamma": 1.0 + 0.1 * rng.standard_normal(H), "beta": 0.1 * rng.standard_normal(H),
           "S_out": 4.0 * math.sqrt(1.0 * (1.0 + 0.1 ** 2) + 0.1 ** 2) / 127.0}
    params = []
    s_in = emb["S_out"]
    for l in range(layers):
        cal = calibrated_scales(config_id, l) if scales == "calibrated" else None
        p = make_layer(config_id, l, H, heads, F, L, s_in, scales=cal)
        params.append(p)
        s_in = p["S_out"]
    w, S_w = _quantize_weight(rng_for(config_id, 0, _T_HEAD_W), N_LABELS, H)
    head = {"w": w, "S_w": S_w, "bias": _quantize_bias(rng_for(config_id, 0, _T_HEAD_B), s_in, S_w)}
    return {"ids": ids, "lens": lens, "emb": emb, "layers": params, "head": head, "B": B, "L": L, "H": H}
