"""Writes ``tiny_layer.json``: one small seeded case of the layer, inputs and the oracle's
outputs.  Calls only the CPU oracle.  The paper prints no worked numeric example, so this
fixture is a regression anchor for the oracle itself (its independent pins are the tests
in ``test_oracle_pins.py``), not a value taken from the paper.

Run from the repository root:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle import arl2_oracle  # noqa: E402


def main():
    rng = np.random.default_rng(16579)
    B, L, H, D = 1, 3, 2, 4
    r = lambda *s: np.round(rng.standard_normal(s), 3)  # noqa: E731  (short decimals)
    q, k, v, g = r(B, L, H, D), r(B, L, H, D), r(B, L, H, D), r(B, L, H)
    kc, vc, a = r(B, L, H, D), r(B, L, H, D), r(B, H)
    S0 = r(B, H, D, D)
    wq, wk, wv = r(H, D, D), r(H, D, D), r(H, D, D)
    ang = np.round(rng.uniform(0, 3, (L, D // 2)), 3)
    cos, sin = np.cos(ang), np.sin(ang)
    out = arl2_oracle.step(q, k, v, g, S0, wq, cos, sin, eps=1e-6)
    S1 = arl2_oracle.commit(kc, vc, a, S0, wk, wv, cos, sin, eps=1e-6)
    doc = {
        "note": "oracle outputs (float64) for a tiny seeded case; Eq. 2-8 and Algorithm 1",
        "B": B, "L": L, "H": H, "D": D, "eps": 1e-6,
        "q": q.tolist(), "k": k.tolist(), "v": v.tolist(), "g": g.tolist(),
        "kc": kc.tolist(), "vc": vc.tolist(), "a": a.tolist(), "S0": S0.tolist(),
        "wq": wq.tolist(), "wk": wk.tolist(), "wv": wv.tolist(), "angle": ang.tolist(),
        "out": out.tolist(), "S1": S1.tolist(),
    }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_layer.json")
    with open(path, "w") as f:
        json.dump(doc, f, indent=0)
    print("wrote", path)


if __name__ == "__main__":
    main()
