"""Write tests/golden/full_size.npz: the CPU oracle's top-k (indices and scores) for EVERY problem
of the full-size configurations, so that the GPU parity tests can compare all P rows without
recomputing the oracle (minutes of host time per configuration) on every run.

Calls only `oracle/` and the seeded generators. Per case the file also keeps a checksum of the
generated inputs and model; a test that finds a different checksum (the generators drifted)
ignores the stored rows and recomputes them.

    python -m tests.golden.make_full_size [case ...]      # default: every case
"""
from __future__ import annotations

import os
import sys
import time
import zlib

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2609_35587_b200 import workloads as wl  # noqa: E402

PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "full_size.npz")

# name -> (config, threshold law or None, problems or None = all of the config)
CASES = {
    "cfg1_pernode": (1, "pernode", None),
    "cfg1_hist256": (1, "hist256", None),
    "cfg1_slots128": (1, "slots128", None),
    "cfg2_pernode": (2, "pernode", None),
    "cfg3_pernode": (3, "pernode", 1000),   # the first 1,000 calls of the latency stream
    "cfg4": (4, None, None),
}


def workload(name: str) -> wl.Workload:
    cfg, law, P = CASES[name]
    return wl.make_workload(cfg, P=P, law=law or wl.DEFAULT_LAW)


def checksum(w: wl.Workload) -> int:
    """CRC of everything the ranking depends on."""
    c = 0
    parts = [w.problems, w.candidates, w.desc]
    if w.seg_offsets is not None:
        parts += [w.seg_offsets, w.seg_index]
    if w.gbdt is not None:
        parts += [w.gbdt[0], w.gbdt[1], np.float32(w.gbdt[2])]
    if w.mlp is not None:
        parts += list(w.mlp["weights"]) + list(w.mlp["biases"]) + [w.mlp["mu"], w.mlp["sigma"]]
    for a in parts:
        c = zlib.crc32(np.ascontiguousarray(a).tobytes(), c)
    return c


def oracle_topk(w: wl.Workload):
    return oracle.select(w.problems, w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp,
                         seg_off=w.seg_offsets, seg_idx=w.seg_index)


def load() -> dict:
    if not os.path.exists(PATH):
        return {}
    with np.load(PATH) as z:
        return {k: z[k] for k in z.files}


def main(names) -> None:
    store = load()
    for name in names or list(CASES):
        w = workload(name)
        t0 = time.time()
        idx, sc = oracle_topk(w)
        store[f"{name}_idx"], store[f"{name}_score"] = idx, sc
        store[f"{name}_crc"] = np.array([checksum(w)], dtype=np.uint32)
        print(f"{name}: {idx.shape} in {time.time() - t0:.0f} s on {oracle.threads()} threads", flush=True)
        np.savez_compressed(PATH, **store)
    print("wrote", PATH, os.path.getsize(PATH), "bytes")


if __name__ == "__main__":
    main(sys.argv[1:])
