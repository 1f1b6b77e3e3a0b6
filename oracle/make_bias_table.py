"""Writes paper_2412_00876_b200/workload_bias.json: the second-layer bias b2 of each
synthetic predictor, fixed once so that about `keep_rate` of N(0,1) rows get a positive
logit (image predictors are centred on the median; their b2 does not change a ranking).

Calls only the oracle and the seeded generators.  Run:  python -m oracle.make_bias_table
"""
import json
import os

import numpy as np

from oracle import dl_oracle as orc
from paper_2412_00876_b200 import workloads as wl

CALIB_ROWS = 4096


def main():
    table = {}
    for cid, cfg in wl.CONFIGS.items():
        for which in ("img", "txt"):
            key = f"{cid}:{which}:{cfg.hidden}:{cfg.pred_hidden}"
            p = wl.make_predictor(cfg, which, b2=0.0)
            x = wl.host_normal(cfg, wl.S_X_TXT, (CALIB_ROWS, cfg.hidden), sub=99)
            s = orc.predictor_logits(x, p.w1, p.b1, p.w2, 0.0)
            rate = cfg.keep_rate if which == "txt" else 0.5
            b2 = -float(np.quantile(s, 1.0 - rate))
            table[key] = float(np.float32(b2))
            print(key, "b2 =", table[key], "logit std =", float(s.std()))
    out = os.path.join(os.path.dirname(os.path.abspath(wl.__file__)), "workload_bias.json")
    with open(out, "w") as f:
        json.dump(table, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main()
