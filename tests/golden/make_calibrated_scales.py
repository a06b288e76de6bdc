#!/usr/bin/env python
"""Writes tests/golden/calibrated_scales.json: the static activation scales of every layer of the
encoder configurations, calibrated progressively with the CPU oracle.

Static quantization (Sec. 3.1 of the paper) fixes every activation scale before inference.  Here
each site's scale is S = max|x| / qmax (Eq. 1 with alpha = the largest magnitude seen) over the
exact pre-requantization values of that site on the first sequences of the seeded input, site by
site and layer by layer: a site is calibrated on the integer tensors the already calibrated sites
before it produce.  int8 sites use qmax = 127, the Q16 sites (residual sums, GELU input) 32767.

Only `oracle/` (integer operators) and `synth` (seeded inputs) are used, plus numpy for the
real-valued statistics: the scale of an integer tensor times its values, a float LayerNorm and a
float GELU of those values.  Nothing of the CUDA path is imported.

    python tests/golden/make_calibrated_scales.py [--configs 0 2 3 4] [--sequences 8]
"""
from __future__ import annotations

import argparse
import json
import math
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent.parent
sys.path.insert(0, str(ROOT))

import oracle  # noqa: E402
from paper_2101_01321_b200 import synth  # noqa: E402

OUT = Path(__file__).resolve().parent / "calibrated_scales.json"
_erf = np.vectorize(math.erf)


def _gelu(x):
    return x * 0.5 * (1.0 + _erf(x / math.sqrt(2.0)))


def _float_layernorm(v, gamma, beta):
    mu = v.mean(axis=1, keepdims=True)
    sd = v.std(axis=1, keepdims=True)
    return (v - mu) / np.maximum(sd, 1e-12) * gamma + beta


def calibrate_layer(cfg_id, layer, cfg, x, S_x, n_seq):
    """Returns (scales of this layer, its int8 output)."""
    H, F, L, heads = cfg.H, cfg.F, cfg.L, cfg.heads
    p = synth.make_layer(cfg_id, layer, H, heads, F, L, S_x)          # weights, gamma / beta; scales replaced below
    s = {}

    def bias_for(nm, S_in):
        return synth._quantize_bias(synth.rng_for(cfg_id, layer, {"qkv": synth._T_BQKV, "o": synth._T_BO,
                                                                  "f1": synth._T_BF1, "f2": synth._T_BF2}[nm]),
                                    S_in, p[f"S_w_{nm}"])

    # QKV projection: raw accumulators -> real values -> one scale per column block
    b_qkv = bias_for("qkv", S_x)
    raw = oracle.linear(x, S_x, p["w_qkv"], p["S_w_qkv"], b_qkv, 2)
    real = raw.astype(np.float64) * (S_x * p["S_w_qkv"])[None, :]
    s["S_q"], s["S_k"], s["S_v"] = (float(np.abs(real[:, i * H:(i + 1) * H]).max() / 127.0) for i in range(3))
    so = np.repeat([s["S_q"], s["S_k"], s["S_v"]], H)
    qkv = oracle.linear(x, S_x, p["w_qkv"], p["S_w_qkv"], b_qkv, 0, S_out_cols=so)
    # context: integer probabilities times values, before requantization
    q3 = qkv.reshape(n_seq, L, 3, heads, 64).astype(np.int64)
    amax = 0.0
    for b in range(n_seq):
        for h in range(heads):
            sc = q3[b, :, 0, h] @ q3[b, :, 1, h].T
            pr, S_p = oracle.softmax(sc.astype(np.int32), (s["S_q"] * s["S_k"]) / 8.0, 255)
            ctx_int = pr.astype(np.int64) @ q3[b, :, 2, h]
            amax = max(amax, float(np.abs(ctx_int).max()) * S_p * s["S_v"])
    s["S_ctx"] = amax / 127.0
    ctx = oracle.attention(qkv, n_seq, L, H, heads, s["S_q"], s["S_k"], s["S_v"], s["S_ctx"], 255)
    # output projection + residual: scale of the SUM, so that both addends fit
    b_o = bias_for("o", s["S_ctx"])
    raw = oracle.linear(ctx, s["S_ctx"], p["w_o"], p["S_w_o"], b_o, 2)
    total = raw.astype(np.float64) * (s["S_ctx"] * p["S_w_o"])[None, :] + x.astype(np.float64) * S_x
    s["S_r1"] = float(np.abs(total).max() / 32767.0)
    s["S_h1"] = float(np.abs(_float_layernorm(total, p["gamma1"], p["beta1"])).max() / 127.0)
    r1 = oracle.linear(ctx, s["S_ctx"], p["w_o"], p["S_w_o"], b_o, 1, s["S_r1"])
    h1, _ = oracle.layernorm(r1, s["S_r1"], x, S_x, p["gamma1"], p["beta1"], s["S_h1"])
    # FFN1 and GELU
    b_f1 = bias_for("f1", s["S_h1"])
    raw = oracle.linear(h1, s["S_h1"], p["w_f1"], p["S_w_f1"], b_f1, 2)
    real = raw.astype(np.float64) * (s["S_h1"] * p["S_w_f1"])[None, :]
    s["S_gi"] = float(np.abs(real).max() / 32767.0)
    s["S_go"] = float(np.abs(_gelu(real)).max() / 127.0)
    gi = oracle.linear(h1, s["S_h1"], p["w_f1"], p["S_w_f1"], b_f1, 1, s["S_gi"])
    g, _ = oracle.gelu(gi, s["S_gi"], s["S_go"])
    # FFN2 + residual
    b_f2 = bias_for("f2", s["S_go"])
    raw = oracle.linear(g, s["S_go"], p["w_f2"], p["S_w_f2"], b_f2, 2)
    total = raw.astype(np.float64) * (s["S_go"] * p["S_w_f2"])[None, :] + h1.astype(np.float64) * s["S_h1"]
    s["S_r2"] = float(np.abs(total).max() / 32767.0)
    s["S_out"] = float(np.abs(_float_layernorm(total, p["gamma2"], p["beta2"])).max() / 127.0)
    r2 = oracle.linear(g, s["S_go"], p["w_f2"], p["S_w_f2"], b_f2, 1, s["S_r2"])
    out, _ = oracle.layernorm(r2, s["S_r2"], h1, s["S_h1"], p["gamma2"], p["beta2"], s["S_out"])
    # the operators above, composed, are the layer: the oracle's own layer must agree
    pc = synth.make_layer(cfg_id, layer, H, heads, F, L, S_x, scales=s)
    whole = oracle.encoder_layer(pc, x, n_seq, L).out
    assert np.array_equal(whole, out), "site-by-site composition differs from the oracle's layer"
    return s, out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", type=int, nargs="*", default=[0, 2, 3, 4])
    ap.add_argument("--sequences", type=int, default=8)
    args = ap.parse_args()
    blob = json.loads(OUT.read_text()) if OUT.exists() else {"configs": {}}
    blob["how"] = ("S = max|x| / qmax per site on the first sequences of the seeded input, progressively through the "
                   "layers with the CPU oracle (tests/golden/make_calibrated_scales.py)")
    for cid in args.configs:
        cfg = synth.CONFIGS[cid]
        n_seq = args.sequences
        x, S_x = synth.make_input(cid, n_seq, cfg.L, cfg.H)
        layers = []
        t0 = time.time()
        for l in range(cfg.layers):
            s, x = calibrate_layer(cid, l, cfg, x, S_x, n_seq)
            layers.append(s)
            S_x = s["S_out"]
            print(f"config {cid} layer {l}: " + " ".join(f"{k}={v:.4g}" for k, v in s.items()) +
                  f"  ({time.time() - t0:.0f} s)", flush=True)
        blob["configs"][str(cid)] = {"sequences": n_seq, "seq_len": cfg.L, "layers": layers}
        OUT.write_text(json.dumps(blob, indent=1) + "\n")


if __name__ == "__main__":
    main()
