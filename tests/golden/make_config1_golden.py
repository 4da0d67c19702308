"""Writes tests/golden/config1_oracle.json from the fp64 oracle alone (no CUDA code is touched).

Config 1: tiny fp32 layer, seed 0, step 0 (dense, nothing cached yet) then step 1 at tau = 0.1 with
26 of 128 positions redrawn and the rest perturbed by N(0, (1e-3)^2); modes KV, O and both.
The stored values freeze the oracle + generator so that a later, unintended change to either shows up.
Run:  python tests/golden/make_config1_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import dare_oracle as orc                     # noqa: E402
from paper_2605_08134_b200 import workloads as wl         # noqa: E402

SAMPLE = [(0, 0, 0), (0, 5, 17), (0, 63, 255), (0, 64, 1), (0, 100, 128), (0, 127, 255)]


def build():
    shape = wl.TINY_F32
    w, x0, x1, changed = wl.two_step_case(shape, 26)
    out = {"tau": 0.1, "planned": np.nonzero(changed.reshape(-1))[0].tolist(), "modes": {}}
    for name, mode in (("kv", 1), ("o", 2), ("both", 3)):
        lay = orc.OracleLayer(shape.d_model, shape.n_heads, shape.head_dim, shape.batch, shape.seq,
                              shape.rope_theta, shape.rms_eps, w["w_q"], w["w_k"], w["w_v"], w["w_o"], w["rms_gain"])
        y0 = lay.step(x0, mode, 0.1)
        y1 = lay.step(x1, mode, 0.1)
        out["modes"][name] = {
            "idx": lay.last_idx.tolist(),
            "score_min_selected": float(lay.last_scores[lay.last_idx].min()),
            "score_max_reused": float(np.delete(lay.last_scores, lay.last_idx).max()),
            "y0_samples": [float(y0[s]) for s in SAMPLE],
            "y1_samples": [float(y1[s]) for s in SAMPLE],
            "y1_rms": float(np.sqrt(np.mean(y1 ** 2))),
            "y1_sum": float(y1.sum()),
            "k_cache_sum": float(lay.k_cache.sum()),
            "o_cache_sum": float(lay.o_cache.sum()),
        }
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_oracle.json")
    with open(path, "w") as f:
        json.dump(build(), f, indent=1)
    print("wrote", path)
