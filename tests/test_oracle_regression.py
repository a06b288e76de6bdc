"""The oracle still produces the stored vectors (written by golden/make_regression_vectors.py
from the oracle itself: a change guard, not a pin)."""
import json
from pathlib import Path

import numpy as np

import oracle

V = json.loads((Path(__file__).parent / "golden" / "regression_vectors.json").read_text())


def test_scalar_vectors():
    for m, bc in V["dyadic"].items():
        assert list(oracle.dyadic(float(m))) == bc
    for n, r in V["isqrt"].items():
        assert list(oracle.isqrt(int(n))) == r
    for S, k in V["exp_consts"].items():
        assert oracle.exp_consts(float(S)) == k
    for S, k in V["gelu_consts"].items():
        assert oracle.gelu_consts(float(S)) == k


def test_tensor_vectors():
    g = V["gelu"]
    assert oracle.gelu_raw(np.array(g["q"]), g["S"])[0].tolist() == g["g"]
    assert oracle.gelu(np.array(g["q"]), g["S"], g["S_out"])[0].tolist() == g["out"]
    assert oracle.softmax(np.array([[0, -693, -1000, -5000, 300, 299]]), 1e-3, 255)[0][0].tolist() == V["softmax"]["1e-3"]["255"]
    assert oracle.softmax(np.array([[0, -34657, -100000, -3000000, 12345]]), 2e-5, 127)[0][0].tolist() == V["softmax"]["2e-5"]["127"]
    assert oracle.layernorm(np.array([[1000, -2000, 3000, -500]]), 1e-4, np.array([[127, -127, 5, 0]]), 0.03,
                            [1, 1, 1, 1], [0, 0, 0, 0], 0.02)[0][0].tolist() == V["layernorm"]["residual"]
