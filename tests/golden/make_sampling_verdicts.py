"""Writes tests/golden/sampling_verdicts.json: the sampling-soundness check of the oracle (oracle/sampling_check.py)
on the three large benchmark configurations, 10^5 seeded samples per box on every box.  It takes tens of minutes of
host time, so it is run once and its verdict kept; tests/test_oracle_pins.py checks the stored verdict against the
oracle's current source and repeats the check on a subsample.  Calls only oracle/ and the input generators.

    python tests/golden/make_sampling_verdicts.py [config indices, default 2 3 4]
"""
import hashlib
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import deeppoly_oracle as orc  # noqa: E402
from oracle import sampling_check as sc  # noqa: E402
from paper_2507_20055_b200 import workloads as wl  # noqa: E402

OUT = os.path.join(ROOT, "tests", "golden", "sampling_verdicts.json")
M = 100_000


def oracle_sha():
    with open(os.path.join(ROOT, "oracle", "deeppoly_oracle.c"), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def main():
    configs = [int(x) for x in sys.argv[1:]] or [2, 3, 4]
    verdicts = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for idx in configs:
        w = wl.make_config(idx)
        t0 = time.time()
        r = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
        l0, u0 = sc.box(w.centers, w.eps, w.clip_lo, w.clip_hi)
        viol, slack = 0, np.inf
        for b in range(w.batch):
            v, s = sc.check_box(w.layers, r["lb"][b], r["ub"][b], l0[b], u0[b], M, seed=1000 * idx + b)
            viol += v
            slack = min(slack, s)
        verdicts[w.name] = {"config": idx, "boxes": w.batch, "samples_per_box": M, "violations": viol,
                            "smallest_slack": slack, "oracle_source_sha256_16": oracle_sha(),
                            "seconds": round(time.time() - t0, 1),
                            "passage": "Section 2 (soundness of the abstract shape); Appendix C, DeepPoly listing"}
        print(w.name, verdicts[w.name], flush=True)
        with open(OUT, "w") as f:
            json.dump(verdicts, f, indent=1, sort_keys=True)


if __name__ == "__main__":
    main()
