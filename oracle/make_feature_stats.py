"""Write paper_2609_35587_b200/data/feature_stats.npz: per workload, per feature column, the
128 split-threshold slots (sample quantiles of the column, each placed midway between two
adjacent distinct sample values), the column's empirical distribution over the sample (its
distinct values with cumulative counts, from which the generator takes any quantile), and the
standardisation constants (mu, sigma) used by the synthetic tree ensembles and MLPs. The
feature values come from the CPU oracle only.

Run from the repository root:  python -m oracle.make_feature_stats
"""
from __future__ import annotations

import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import oracle  # noqa: E402
from paper_2609_35587_b200 import workloads as wl  # noqa: E402

SAMPLE = 65536
# columns holding categorical codes / flags: left unscaled (section "Model B")
CATEGORICAL = (3, 4, 5, 8, 9, 17, 18, 19, 36, 51)
LOG2_COLS = (0, 1, 2)


def slots_from_values(vals: np.ndarray, n_slots: int) -> np.ndarray:
    s = np.sort(vals.astype(np.float32))
    d = np.unique(s)
    out = np.empty(n_slots, dtype=np.float32)
    for j in range(n_slots):
        q = 0.05 + 0.9 * (j + 0.5) / n_slots
        v0 = s[int(np.floor(q * (len(s) - 1)))]
        i = int(np.searchsorted(d, v0))
        if i + 1 < len(d):
            lo, hi = d[i], d[i + 1]
        elif i >= 1:
            lo, hi = d[i - 1], d[i]
        else:
            out[j] = np.float32(v0 + np.float32(0.5))
            continue
        t = np.float32((np.float64(lo) + np.float64(hi)) / 2.0)
        out[j] = hi if t <= lo else t
    return out


def stats_for(cfg: int) -> dict:
    prob, cand, _, _ = wl.make_inputs(cfg, seg=1) if cfg == 2 else wl.make_inputs(cfg)
    desc = wl.gpu_desc()
    seed = wl.BASE_SEED + 1000 * cfg
    n = min(SAMPLE, len(prob) * len(cand))
    idx = np.arange(n)
    if n == len(prob) * len(cand):
        pi, ci = idx // len(cand), idx % len(cand)
    else:
        pi = wl.randint(seed, wl._S_SAMPLE, idx, len(prob))
        ci = wl.randint(seed, wl._S_SAMPLE + 1, idx, len(cand))
    x = oracle.featurize(prob[pi], cand, desc, seg_off=np.arange(n + 1, dtype=np.int64),
                         seg_idx=ci.astype(np.int32))
    # log2 columns: every problem of the workload, so that a slot never sits within an ulp of
    # a value the workload can produce
    xp = oracle.featurize(prob, cand[:1], desc)
    thr = np.empty((wl.KS_F, wl.N_QUANTILE_SLOTS), dtype=np.float32)
    dval, dcum, doff = [], [], [0]
    for f in range(wl.KS_F):
        col = xp[:, f] if f in LOG2_COLS else x[:, f]
        thr[f] = slots_from_values(col, wl.N_QUANTILE_SLOTS)
        d, cnt = np.unique(col.astype(np.float32), return_counts=True)
        dval.append(d)
        dcum.append(np.cumsum(cnt))
        doff.append(doff[-1] + len(d))
    mu = x.astype(np.float64).mean(axis=0)
    sigma = x.astype(np.float64).std(axis=0)
    sigma[sigma < 1e-12] = 1.0
    for f in CATEGORICAL + (63,):
        mu[f], sigma[f] = 0.0, 1.0
    return {"thr": thr, "mu": mu.astype(np.float32), "sigma": sigma.astype(np.float32),
            "dval": np.concatenate(dval).astype(np.float32), "dcum": np.concatenate(dcum).astype(np.int32),
            "doff": np.asarray(doff, dtype=np.int32)}


def main() -> None:
    out = {}
    for cfg in (0, 1, 2):
        st = stats_for(cfg)
        for k, v in st.items():
            out[f"cfg{cfg}_{k}"] = v
        print(f"cfg{cfg}: thr {st['thr'].shape}, distinct thresholds per column "
              f"min {min(len(np.unique(r)) for r in st['thr'])} "
              f"max {max(len(np.unique(r)) for r in st['thr'])}")
    path = wl._STATS_PATH
    os.makedirs(os.path.dirname(path), exist_ok=True)
    np.savez_compressed(path, **out)
    print("wrote", path, os.path.getsize(path), "bytes")


if __name__ == "__main__":
    main()
