"""Writes tests/golden/tiny_block.json: outputs of the CPU oracle on one tiny seeded block.

The paper prints no worked numeric example, so there is nothing of the paper's to store.  This file
pins the oracle to itself over time instead: it is produced by the oracle alone (no GPU code is
imported), and tests/test_oracle_golden.py fails when a later edit of the oracle changes a value.
What makes the stored values trustworthy in the first place are the pins in tests/test_oracle_pins.py
and tests/test_oracle_stack.py (invertibility, finite differences, closed forms, a library cross-check).

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import revffn_oracle as orc                      # noqa: E402
from workloads import BlockConfig, make_streams, make_weights  # noqa: E402

CFG = dict(name="golden", tokens=5, d_model=16, n_experts=5, top_k=2, d_expert=12, d_shared=10, weight_dtype="f32")
SEED, SCALE = 4, 8.0


def compute():
    cfg = BlockConfig(**CFG)
    p = make_weights(cfg, SEED)
    for n in p:
        if n != "norm_gamma":
            p[n] = p[n] * SCALE
    s = make_streams(cfg, SEED)
    y2, info = orc.forward(p, s["y1"], s["x2"], cfg.top_k)
    x2, _ = orc.inverse(p, s["y1"], y2, cfg.top_k)
    g = orc.backward(p, s["y1"], s["dy2"], cfg.top_k)
    return {
        "config": CFG, "seed": SEED, "weight_scale": SCALE,
        "source": "oracle/revffn_oracle.py: forward (Eq. 2), inverse (Sec. 3.1), backward (Sec. 2, Sec. 3.1)",
        "idx": info["idx"].tolist(), "gates": info["gates"].tolist(), "F": info["F"].tolist(),
        "y2": y2.tolist(), "max_abs_reconstruction_error": float(np.max(np.abs(x2 - s["x2"]))),
        "dy1": g["dy1"].tolist(),
        "grad_sums": {n: float(np.sum(v)) for n, v in g.items() if n in p},
        "grad_abs_sums": {n: float(np.sum(np.abs(v))) for n, v in g.items() if n in p},
    }


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_block.json")
    with open(out, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", out)
