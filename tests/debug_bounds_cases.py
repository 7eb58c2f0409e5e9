"""Small parity cases run against the checked build of the library (KS_LIBRARY points at
libks_debug.so): every case must match the oracle AND leave the bounds word at 0. Run as a
script by tests/test_gpu_debug_bounds.py in a process of its own, because the library is chosen
when the binding is imported."""
import sys

import numpy as np
import torch

import oracle
from paper_2609_35587_b200 import binding as ks
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import topk_accept


def main() -> int:
    assert ks.debug_bounds_line() == 0, "not the checked build, or a stale violation"
    desc = wl.gpu_desc()
    dev = torch.device("cuda", 0)
    ctx = ks.Context(desc, 0)
    cases = []
    for P, C, k, trees, depth in ((1, 1, 5, 3, 1), (2, 7, 10, 5, 2), (3, 70, 32, 9, 2), (3, 69, 5, 4, 1),
                                  (2, 1030, 10, 40, 6), (33, 40, 10, 12, 5)):
        for law in ("slots128", "pernode"):
            cases.append((f"P{P} C{C} k{k} T{trees} D{depth} {law}", wl.make_workload(1, P=P, C=C, trees=trees, depth=depth, law=law), k))
    # every tile geometry at full ensemble size, segments, mixed element types
    cases.append(("cfg1 pernode", wl.make_workload(1, P=2, C=2100, law="pernode"), 10))
    cases.append(("cfg2 pernode segments", wl.make_workload(2, P=3, seg=1100, law="pernode"), 10))
    cases.append(("cfg2 memo", wl.make_workload(2, P=40, seg=90, trees=30, depth=6), 10))
    # more (problem, candidate block) items than SMs: the launch form in which a CTA serves many items
    cases.append(("many items", wl.make_workload(1, P=90, C=2100, trees=24, depth=8, law="pernode"), 10))
    for name, w, k in cases:
        model = ctx.model_create_gbdt(*w.gbdt)
        assert "select_fast_kernel" in model.describe(), (name, model.describe())
        P, C = len(w.problems), len(w.candidates)
        d_so = None if w.seg_offsets is None else ks.to_device(w.seg_offsets, dev)
        d_si = None if w.seg_index is None else ks.to_device(w.seg_index, dev)
        idx, sc = ctx.select(ks.to_device(w.problems, dev), P, ks.to_device(w.candidates, dev), C, model, k,
                             d_so, d_si, w.pairs)
        torch.cuda.synchronize()
        idx, sc = idx.cpu().numpy(), sc.cpu().numpy()
        for i in range(P):
            if w.seg_offsets is None:
                pool = np.arange(C, dtype=np.int32)
                so = si = None
            else:
                pool = w.seg_index[w.seg_offsets[i]:w.seg_offsets[i + 1]]
                so, si = np.array([0, len(pool)], np.int64), pool
            _, _, allsc = oracle.select(w.problems[i:i + 1], w.candidates, desc, k, gbdt=w.gbdt, seg_off=so, seg_idx=si,
                                        want_scores=True)
            ok, msg = topk_accept(idx[i], sc[i], allsc, pool, k, 1e-5)
            assert ok, f"{name}, problem {i}: {msg}"
        if w.seg_offsets is None:
            hi, hs = ctx.select_one(w.problems[:1], ks.to_device(w.candidates, dev), C, model, k)
            assert np.array_equal(hi.numpy(), idx[0]), name
            x = oracle.featurize(w.problems[:1], w.candidates, desc)
            s = ctx.score(ks.to_device(x, dev), model).cpu().numpy()
            rs = oracle.score_gbdt(x, *w.gbdt)
            assert np.all(np.abs(s - rs) <= 1e-5 * np.maximum(1, np.abs(rs))), name
        line = ks.debug_bounds_line()
        assert line == 0, f"{name}: index out of range at ks_gbdt_fast.cu line {line}"
    print("checked build: %d cases, no index out of range" % len(cases))
    return 0


if __name__ == "__main__":
    sys.exit(main())
