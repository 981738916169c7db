"""Writes ``topk_cfg3.json``, ``topk_cfg4.json`` and ``topk_cfg5.json``: the oracle's full-pool top
lists for the workloads whose pools are large.

Calls only the CPU oracle and the seeded input generator (never the CUDA library).  For each
workload every pool (1,048,576 candidates; 64 pools of 65,536 for the batched workload) is scored in
FP64 and, per GP, the 4k best candidates (index, EI) are stored together with the pool's maximum EI,
so that a test can apply the top-k rule: set equality when the oracle's gap at rank k exceeds the
tolerance, otherwise every chosen candidate within tolerance of the oracle's rank-k value.

    python tests/golden/make_topk_golden.py [3] [4] [5]  # a minute for 3, several minutes each for 4 and 5
"""
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import gp_oracle as o  # noqa: E402
from paper_2604_11109_b200 import workloads as w  # noqa: E402


def top_list(c, g, t0):
    f = o.fit(g["X"], g["y"], g["ell"], g["sf2"], g["sn2"])
    ei = np.empty(c.m)
    step = 65536
    for s in range(0, c.m, step):
        ei[s:s + step] = o.score(f, g["Xcand"][s:s + step])[2]
        if c.batch == 1:
            print(f"{c.name}: {min(s + step, c.m)}/{c.m} candidates, {time.time() - t0:.0f} s", flush=True)
    idx, val = o.topk(ei, 4 * c.k)
    return {
        "ei_max": repr(float(ei.max())),
        "gap_rank_k_to_next": repr(float(val[c.k - 1] - val[c.k])),
        "idx": [int(i) for i in idx],
        "ei": [repr(float(v)) for v in val],
    }


def main(cfgs):
    for cfg in cfgs:
        c = w.get_config(cfg)
        t0 = time.time()
        out = {
            "_source": "CPU oracle over the full seeded pool; see make_topk_golden.py",
            "cfg": cfg, "m": c.m, "n": c.n, "d": c.d, "k": c.k, "seed": c.seed,
        }
        if c.batch == 1:
            out.update(top_list(c, w.generate_gp(c, 0), t0))
        else:   # one list per GP
            out["batch"] = c.batch
            out["gps"] = []
            for q in range(c.batch):
                out["gps"].append(top_list(c, w.generate_gp(c, q), t0))
                print(f"{c.name}: GP {q + 1}/{c.batch}, {time.time() - t0:.0f} s", flush=True)
        path = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"topk_{c.name}.json")
        with open(path, "w") as fh:
            json.dump(out, fh, indent=0)
        print("wrote", path, f"{time.time() - t0:.0f} s")


if __name__ == "__main__":
    main([int(a) for a in sys.argv[1:]] or [3, 4, 5])
