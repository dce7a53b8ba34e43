#!/usr/bin/env python
"""Writes tests/golden/fullsize_digests.json: the CPU oracle's result for every class of the full-size
int8 configurations (C2: 10 classes x 5000 samples, C5: 1000 classes x 1300 samples), as one digest per class.

Calls only the oracle (Algorithm 1 with a coverage vector per block, shown identical to the plain-definition
variant on small inputs by the CPU tests) and the seeded input generator.  Nothing here touches the CUDA
library.  Classes are independent in Algorithm 1, so each class is run by itself, one per thread.

A digest covers, for one class: the block of every sample (class-local order), the class-local indices of the
samples in pick order, and the W block values f(A_j).  The inputs are keyed by a digest of the generated
features, labels and capacities, so a drift of the generator shows up as a key mismatch, not as a parity failure.

    python tests/golden/make_fullsize_golden.py [C2] [C5] [--threads 8]

Takes about 10 minutes per configuration on 8 cores.
"""
from __future__ import annotations

import hashlib
import json
import os
import sys
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

OUT = os.path.join(HERE, "fullsize_digests.json")


def class_digest(assign_local: np.ndarray, order_local: np.ndarray, fvals: np.ndarray) -> str:
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(assign_local, dtype=np.int32).tobytes())
    h.update(np.ascontiguousarray(order_local, dtype=np.int32).tobytes())
    h.update(np.ascontiguousarray(fvals, dtype=np.int64).tobytes())
    return h.hexdigest()[:32]


def input_digest(wl) -> str:
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(wl.features).tobytes())
    h.update(np.ascontiguousarray(wl.labels, dtype=np.int32).tobytes())
    h.update(np.ascontiguousarray(wl.capacities, dtype=np.float64).tobytes())
    return h.hexdigest()[:32]


def run_config(name: str, threads: int) -> dict:
    from oracle import rcd_oracle as orc
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name)
    groups = orc.split_by_label(wl.labels, wl.L)

    def one(l):
        ids = groups[l]
        q = orc.quotas(len(ids), wl.capacities)
        S = orc.similarity(wl.features[ids])
        assign, oj, ov, fv = orc.partition_class(S, q, "incremental")
        assert len(ov) == len(ids) and np.array_equal(assign[ov], oj)
        return class_digest(assign, ov, fv), int(fv.sum())

    t0 = time.time()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        outs = list(ex.map(one, range(wl.L)))
    return {"inputs": input_digest(wl), "L": wl.L, "N": wl.N, "W": wl.W,
            "total_objective": int(sum(o[1] for o in outs)),
            "class_digests": [o[0] for o in outs], "oracle_seconds": round(time.time() - t0, 1), "threads": threads}


def main():
    args = sys.argv[1:]
    threads = os.cpu_count() or 1
    if "--threads" in args:
        at = args.index("--threads")
        threads = int(args[at + 1])
        del args[at:at + 2]
    names = args or ["C2", "C5"]
    data = json.load(open(OUT)) if os.path.exists(OUT) else {
        "_source": "Written by tests/golden/make_fullsize_golden.py from the CPU oracle alone (Algorithm 1, facility "
                   "location, readings as in the oracle's header); one digest per class of the full-size int8 configurations."}
    for name in names:
        data[name] = run_config(name, threads)
        json.dump(data, open(OUT, "w"), indent=0)
        print(name, "done in", data[name]["oracle_seconds"], "s")


if __name__ == "__main__":
    main()
