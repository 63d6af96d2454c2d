"""Writes tests/golden/tiny_layer.json: one small seeded layer and what the CPU oracle makes of it.

The paper prints no worked numerical example of a compressed cache, so this fixture is a
regression pin of the oracle (it calls nothing but oracle/ and the seeded input generator):
a later change to the oracle's arithmetic shows up as a diff of this file.

  python tests/golden/make_tiny_layer.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import chunkkv_oracle as ora  # noqa: E402
from workloads import CONFIGS, make_layer, scaled  # noqa: E402

WL = dict(Hq=4, Hkv=2, d=64, L=96, w=8, c=5, budget=33, seed=7, planted_count=2, sink_tokens=0)


def build():
    wl = scaled(CONFIGS[1], **WL)
    x = make_layer(wl)
    t = ora.token_scores(x.q_obs, x.K, wl.Hq, wl.Hkv, wl.w)
    s = ora.chunk_scores(t, wl.c)
    idx = ora.select(s, wl.L, wl.w, wl.c, wl.budget)
    return {
        "workload": WL,
        "planted_chunks": [int(v) for v in x.planted],
        "chunk_scores": [[float(f"{v:.12e}") for v in row] for row in s],
        "token_score_sums": [float(f"{v:.12e}") for v in t.sum(axis=1)],
        "idx": [[int(v) for v in row] for row in idx],
    }


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_layer.json")
    with open(out, "w") as f:
        json.dump(build(), f, indent=1)
        f.write("\n")
    print("wrote", out)
