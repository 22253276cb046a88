"""Writes tests/golden/l2_digest.json: digests of every integer tensor and
sums of the floating-point outputs of the SSDi8 oracle on two small seeded
workloads.  It calls only the oracle and the input generator; nothing here
comes from the CUDA path.  The fixture guards the oracle's arithmetic against
accidental change (the paper itself prints no worked example to store)."""
import hashlib
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
sys.path.insert(0, os.path.dirname(HERE))

from oracle import oracle as orc  # noqa: E402
from paper_2608_21952_b200 import inputs  # noqa: E402
from helpers import TWO_BLOCK  # noqa: E402


def digest(cfg):
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    y, fin, taps = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"],
                                 q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], None,
                                 taps=tuple(orc.TAP_SPECS))
    out = {k: hashlib.sha256(np.ascontiguousarray(v).tobytes()).hexdigest()[:16]
           for k, v in sorted(taps.items())}
    for k in ("xq", "Bq", "Cq", "s_x", "s_xs", "s_cb", "s_h"):
        out["in_" + k] = hashlib.sha256(np.ascontiguousarray(q[k]).tobytes()).hexdigest()[:16]
    out["final"] = hashlib.sha256(fin.tobytes()).hexdigest()[:16]
    out["y_sum"] = float(y.sum())
    out["y_abs_sum"] = float(np.abs(y).sum())
    return out


def main():
    res = {"cfg0": digest(inputs.CONFIGS["cfg0"]), "two_block": digest(TWO_BLOCK)}
    with open(os.path.join(HERE, "l2_digest.json"), "w") as f:
        json.dump(res, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main()
