"""The stored oracle-calibrated activation scales: present for every encoder configuration,
positive, and doing their job -- on the calibration input no site clamps (the scale covers the
largest value seen) and the integer layer stays close to a float layer."""
import json

import numpy as np

import oracle
from paper_2101_01321_b200 import synth

SITES = ("S_q", "S_k", "S_v", "S_ctx", "S_r1", "S_h1", "S_gi", "S_go", "S_r2", "S_out")


def test_blob_covers_every_layer_of_every_config():
    blob = json.loads(synth.CALIBRATED_SCALES_FILE.read_text())
    for cid in (0, 2, 3, 4):
        layers = blob["configs"][str(cid)]["layers"]
        assert len(layers) == synth.CONFIGS[cid].layers
        for sc in layers:
            assert set(sc) == set(SITES)
            assert all(np.isfinite(v) and v > 0 for v in sc.values())
    # the calibrated scales differ from the closed-form ones but stay in their neighbourhood
    a = synth.make_model(2, 1, layers=1)[1][0]
    c = synth.make_model(2, 1, layers=1, scales="calibrated")[1][0]
    for k in SITES:
        assert 0.2 < c[k] / a[k] < 5.0 and c[k] != a[k], k


def test_calibrated_layer_does_not_clamp_on_its_calibration_input():
    """Config 0 was calibrated on 8 sequences: on those, every int8 / Q16 tensor of the layer stays
    strictly inside its range except where the maximum itself sits (it maps to the last code)."""
    cfg = synth.CONFIGS[0]
    x, params = synth.make_model(0, 8, scales="calibrated")
    res = oracle.encoder_layer(params[0], x, 8, cfg.L, want_taps=True)
    taps = res.taps
    for name, qmax in (("qkv", 127), ("ctx", 127), ("h1", 127), ("g", 127)):
        t = np.asarray(taps[name]).astype(np.int64)
        assert np.abs(t).max() <= qmax
        assert (np.abs(t) == qmax).mean() < 1e-4, name        # only the extreme value(s) reach the last code
    out = np.asarray(res.out).astype(np.int64)
    assert 100 <= np.abs(out).max() <= 127
