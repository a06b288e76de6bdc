"""Writes ``regression_vectors.json`` next to this file from the CPU oracle alone.

These vectors are NOT pins (they restate the oracle); they only guard the oracle's
arithmetic against accidental change.  Run:  python tests/golden/make_regression_vectors.py
"""
import json
import sys
from pathlib import Path

import numpy as np

sys.path.insert(0, str(Path(__file__).resolve().parents[2]))
import oracle  # noqa: E402


def main():
    v = {}
    v["dyadic"] = {repr(m): oracle.dyadic(m) for m in (9e-4, 258.0, -0.37, 1.0, 0.5, 3e-10, 2.0 ** 30)}
    v["isqrt"] = {str(n): oracle.isqrt(n) for n in (0, 1, 2, 3, 4, 15, 16, 17, 2 ** 31 - 1, 2 ** 32 - 1,
                                                     16785408, 2 ** 42 + 12345)}
    v["exp_consts"] = {repr(S): oracle.exp_consts(S) for S in (1e-3, 4.5e-5, 2e-5)}
    rows = {"1e-3": ([0, -693, -1000, -5000, 300, 299], 1e-3), "2e-5": ([0, -34657, -100000, -3000000, 12345], 2e-5)}
    v["softmax"] = {k: {str(M): oracle.softmax(np.array([q]), S, M)[0][0].tolist() for M in (255, 127)}
                    for k, (q, S) in rows.items()}
    v["gelu_consts"] = {repr(S): oracle.gelu_consts(S) for S in (1e-3, 1.5e-4)}
    q = [0, 1, -1, 500, -500, 1000, -1000, 2349, -2349, 2502, 2503, 4000, -4000, 32767, -32768, 100000]
    v["gelu"] = {"q": q, "S": 1e-3, "S_out": 4 / 127,
                 "g": oracle.gelu_raw(np.array(q), 1e-3)[0].tolist(),
                 "out": oracle.gelu(np.array(q), 1e-3, 4 / 127)[0].tolist()}
    v["layernorm"] = {
        "plain": oracle.layernorm(np.array([[1000, -2000, 3000, -500, 0, 250, -4000, 1500]]), 1.0, None, 0.0,
                                  [1.0, 0.9, 1.1, -1.0, 1.0, 1.0, 0.5, 1.2],
                                  [0, 0.1, -0.1, 0, 0.05, 0, 0, -0.2], 0.025)[0][0].tolist(),
        "residual": oracle.layernorm(np.array([[1000, -2000, 3000, -500]]), 1e-4, np.array([[127, -127, 5, 0]]),
                                     0.03, [1, 1, 1, 1], [0, 0, 0, 0], 0.02)[0][0].tolist()}
    out = Path(__file__).with_name("regression_vectors.json")
    out.write_text(json.dumps(v, indent=1, sort_keys=True) + "\n")
    print("wrote", out)


if __name__ == "__main__":
    main()
