"""Writes synth/thresholds.json: per workload, the log-confidence thresholds at the stated quantiles.

Run from the repository root:  python -m oracle.calibrate_thresholds
For each workload, 4096 synthetic (drafter row, drafted token) pairs from a counter range disjoint
from the step inputs are scored with the oracle's log-confidence; the nearest-rank quantiles
(q_lo, q_hi) of those scores become (log_tau_lo, log_tau_hi), so that the lowest q_lo of drafted
tokens go to the full verifier, the top 1 - q_hi are accepted directly and the rest go to the slim
verifier (App. B, regions A/B/C).  Only oracle code computes the stored values.
"""
import json
import os

import numpy as np

from synth import workloads as W
from oracle import tiers


def main() -> None:
    out, memo = {}, {}
    for name, wl in W.WORKLOADS.items():
        k = (wl.seed, wl.shape.vocab, wl.logit_sigma, wl.plant, wl.quantiles)
        if k not in memo:
            d = []
            V = wl.shape.vocab
            for c in range(0, 4096, 512):                       # chunks bound host memory
                logits, tok = W.calibration_rows(wl, 512, first=c)
                d += [tiers.log_confidence(logits[i], int(tok[i])) for i in range(512)]
            lo, hi = tiers.quantile_thresholds(np.array(d, dtype=np.float32), *wl.quantiles)
            memo[k] = {"log_tau_lo": float(lo), "log_tau_hi": float(hi), "quantiles": list(wl.quantiles),
                       "samples": len(d)}
        out[name] = memo[k]
        print(name, out[name])
    path = os.path.join(os.path.dirname(os.path.abspath(W.__file__)), "thresholds.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main()
