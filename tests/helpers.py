"""Small builders shared by the tests (records only; no method arithmetic)."""
import numpy as np

from paper_2609_35587_b200 import workloads as wl


def problem(m, n, k, layout=0, dtype_ab=0, dtype_d=0, epi_flags=0):
    p = np.zeros(1, wl.PROBLEM_DT)
    p["m"], p["n"], p["k"] = m, n, k
    p["layout"], p["dtype_ab"], p["dtype_d"], p["epi_flags"] = layout, dtype_ab, dtype_d, epi_flags
    return p


def candidate(tile_m, tile_n, tile_k, stages, cluster_m=1, cluster_n=1, kernel_sched=0, epi_sched=1,
              tile_sched=0, instr_n=None, instr_m=64, instr_k=16):
    c = np.zeros(1, wl.CANDIDATE_DT)
    c["tile_m"], c["tile_n"], c["tile_k"] = tile_m, tile_n, tile_k
    c["instr_n"] = tile_n if instr_n is None else instr_n
    c["stages"], c["cluster_m"], c["cluster_n"] = stages, cluster_m, cluster_n
    c["kernel_sched"], c["epi_sched"], c["tile_sched"] = kernel_sched, epi_sched, tile_sched
    c["instr_m"], c["instr_k"] = instr_m, instr_k
    return c


def read_worked_examples(path):
    """Parse tests/golden/worked_examples.txt -> list of (name, problem, candidate, pins)."""
    out = []
    cur = None
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("example"):
                head, tail = line.split("|")
                h = head.split()
                pv = [int(v) for v in h[2:]]
                cv = [int(v) for v in tail.split()]
                p = problem(*pv)
                c = candidate(cv[0], cv[1], cv[2], cv[4], cv[5], cv[6], cv[7], cv[8], cv[9],
                              instr_n=cv[3], instr_m=cv[10], instr_k=cv[11])
                cur = (h[1], p, c, [])
                out.append(cur)
            else:
                parts = line.split()
                col, val = int(parts[0]), float(parts[1])
                bits = int(parts[2], 16) if len(parts) > 2 else None
                cur[3].append((col, val, bits))
    return out


def topk_accept(gpu_idx, gpu_score, oracle_scores_row, pool_idx_row, k, tol):
    """Check one problem's top-k list against the oracle's scores of the same segment.

    Accepts iff no duplicates, every index is in the segment, every returned score matches the
    oracle's score of that candidate within tol, the j-th pick is as good as the oracle's j-th
    up to tol, and among exact ties the indices ascend. An exact tie is one on both sides: two
    candidates whose oracle scores are equal but whose returned scores differ (another order of
    the fp32 additions moved one of them by an ulp) are a tie within the tolerance, which may
    come out in either order. Returns (ok, message)."""
    n = len(oracle_scores_row)
    kk = min(k, n)
    order = np.lexsort((pool_idx_row, -oracle_scores_row.astype(np.float64)))
    best = oracle_scores_row[order[:kk]]
    pos = {int(pool_idx_row[i]): i for i in range(n)} if n <= 200000 else None
    seen = set()
    for j in range(k):
        gi = int(gpu_idx[j])
        if j >= kk:
            if gi != -1 or not np.isneginf(gpu_score[j]):
                return False, f"rank {j}: expected padding, got ({gi}, {gpu_score[j]})"
            continue
        if gi in seen:
            return False, f"rank {j}: duplicate index {gi}"
        seen.add(gi)
        if pos is not None:
            if gi not in pos:
                return False, f"rank {j}: index {gi} outside the segment"
            r = pos[gi]
        else:
            r = int(np.searchsorted(pool_idx_row, gi))
        so = float(oracle_scores_row[r])
        if abs(float(gpu_score[j]) - so) > tol * max(1.0, abs(so)):
            return False, f"rank {j}: score {gpu_score[j]} vs oracle {so} for index {gi}"
        if float(best[j]) - so > tol * max(1.0, abs(float(best[j]))):
            return False, f"rank {j}: picked {gi} (oracle {so}) but oracle's rank-{j} score is {best[j]}"
        if j > 0:
            prev = int(gpu_idx[j - 1])
            rp = pos[prev] if pos is not None else int(np.searchsorted(pool_idx_row, prev))
            if float(oracle_scores_row[rp]) == so and float(gpu_score[j - 1]) == float(gpu_score[j]) and prev > gi:
                return False, f"rank {j}: tie not in ascending index order ({prev} before {gi})"
    return True, ""
