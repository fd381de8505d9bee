"""Writes tests/golden/checksums.json: word checksums of what the CPU oracle computes on the seeded
workloads. The paper prints no worked example for these kernels, so the stored values are the
oracle's own (this script calls nothing but `oracle/` and the seeded input generator); they pin the
oracle and the input generator against silent drift, and give the GPU tests expected values at
sizes where running the oracle again would only repeat this computation.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle                                                     # noqa: E402
from paper_2510_00932_b200 import inputs                          # noqa: E402

CASES = [("c1", None), ("c2", 1 << 22), ("c3", 1 << 22), ("c4", 1 << 22)]     # (workload, length override)
SHMEM = [((1 << 20) + 77, 600), ((1 << 18) + 4099, 1500), (3 * 8192 + 5, 7)]


def compute():
    oracle.build()
    out = {"numpy": np.__version__, "chain": {}, "shmem_mix": {}}
    for name, n in CASES:
        w = inputs.WORKLOADS[name]
        a, b, c = inputs.make_arrays(w, n)
        entry = {"n": int(a.size), "inputs": [inputs.checksum(v) for v in (a, b, c)]}
        a, b, c, d = oracle.chain(a, b, c, w.scalar)
        entry["after_one_pass"] = [inputs.checksum(v) for v in (a, b, c)]
        entry["dot"] = float(d).hex()
        out["chain"][name] = entry
    for n, rounds in SHMEM:
        x = inputs.make_words(n)
        out["shmem_mix"][f"{n}x{rounds}"] = {"input": inputs.checksum(x), "output": inputs.checksum(oracle.shmem_mix(x, rounds))}
    return out


if __name__ == "__main__":
    with open(os.path.join(HERE, "checksums.json"), "w") as f:
        json.dump(compute(), f, indent=1)
        f.write("\n")
    print("wrote checksums.json")
