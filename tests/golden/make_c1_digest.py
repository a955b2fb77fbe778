"""Writes c1_oracle_digest.json from the CPU oracle alone (never from the CUDA path).

Run:  python tests/golden/make_c1_digest.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from mka_inputs import CONFIGS, make_tensor  # noqa: E402
from oracle import mka_oracle as orc  # noqa: E402


def digest():
    cfg = CONFIGS["c1"]
    t = {n: make_tensor(cfg, n).double().numpy() for n in ("X", "W_r", "Q", "K1", "V1", "K2", "V2", "K3", "V3")}
    gate, _ = orc.router(t["X"], t["W_r"])
    K, V = [t["K1"], t["K2"], t["K3"]], [t["V1"], t["V2"], t["V3"]]
    O, LSE = orc.fwd(t["Q"], K, V, gate, cfg.W)
    Of, _ = orc.fwd(t["Q"], K, V, gate, cfg.W, mode="full")
    pick = [(0, 0, 0, 0), (0, 1, 63, 5), (0, 2, 64, 17), (0, 3, 255, 63)]
    return {
        "config": "c1 (fp32 B=1 H=4 d=64 D=256 T=256 W=64 N3=128, seed 0)",
        "gate_sum": float(gate.sum()),
        "gate_t0": [float(x) for x in gate[0, 0]],
        "O_fast": {str(p): float(O[p]) for p in pick},
        "O_full": {str(p): float(Of[p]) for p in pick},
        "LSE": {str(p[:3]): float(LSE[p[:3]]) for p in pick},
        "O_fast_abs_sum": float(np.abs(O).sum()),
    }


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_oracle_digest.json")
    with open(out, "w") as f:
        json.dump(digest(), f, indent=1)
    print("wrote", out)
