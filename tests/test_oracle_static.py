"""Pins for the oracle's static sampling score (data-collection section: clusters n_c, cluster
waves W, score = n_c / (W S_SM c_M c_N) * S * sqrt(T_M T_N T_K)): hand-worked values, a
brute-force count of clusters and waves, the invariants the formula fixes, and the ranking
against numpy's sort."""
import os

import numpy as np

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import candidate, problem, read_worked_examples

DESC = wl.gpu_desc()
HERE = os.path.dirname(__file__)


def static_scores(prob, cand, k=1):
    idx, sc, allsc = oracle.select(prob, cand, DESC, k, static=True, want_scores=True)
    return idx, sc, allsc.reshape(len(prob), len(cand))


def test_hand_worked_values():
    ex = {name: (p, c) for name, p, c, _ in read_worked_examples(os.path.join(HERE, "golden", "worked_examples.txt"))}
    seen = 0
    with open(os.path.join(HERE, "golden", "static_score.txt")) as fh:
        for line in fh:
            if not line.strip() or line.startswith("#"):
                continue
            name, val, bits = line.split()
            p, c = ex[name]
            s = static_scores(p, c)[2][0, 0]
            assert abs(float(s) - float(val)) <= 1e-6 * float(val), (name, s)
            assert int(s.view(np.uint32)) == int(bits, 16), (name, hex(int(s.view(np.uint32))))
            seen += 1
    assert seen == 3


def count_clusters_and_waves(M, N, TM, TN, cM, cN, sms):
    """Lay the clusters over the output one by one, then hand them to the SMs wave by wave."""
    n_c = 0
    for _m0 in range(0, M, cM * TM):
        for _n0 in range(0, N, cN * TN):
            n_c += 1
    waves, left = 0, n_c
    while left > 0:
        left -= sms
        waves += 1
    return n_c, waves


def test_against_a_brute_force_count():
    rng = np.random.default_rng(5)
    sms = int(np.asarray(DESC["num_sms"]).reshape(-1)[0])
    for _ in range(200):
        M, N = (int(v) for v in rng.integers(1, 6000, 2))
        TM, TN, TK = (int(v) for v in rng.choice([64, 128, 192, 256], 3))
        cM, cN = (int(v) for v in rng.choice([1, 2, 4], 2))
        S = int(rng.integers(1, 9))
        p = problem(M, N, 777)
        c = candidate(TM, TN, TK, S, cM, cN)
        n_c, W = count_clusters_and_waves(M, N, TM, TN, cM, cN, sms)
        want = n_c / (W * sms * cM * cN) * S * np.sqrt(float(TM * TN * TK))
        got = float(static_scores(p, c)[2][0, 0])
        assert abs(got - want) <= 3e-7 * want, (M, N, TM, TN, TK, cM, cN, S, got, want)


def test_invariants():
    prob, cand, _, _ = wl.make_inputs(1, P=16, C=4000)
    _, _, s = static_scores(prob, cand)
    S = cand["stages"].astype(np.float64)
    vol = (cand["tile_m"].astype(np.float64) * cand["tile_n"] * cand["tile_k"])
    fill = s / (S * np.sqrt(vol))[None, :]
    # the wave-filling factor lies in (0, 1 / (c_M c_N)]
    cl = (cand["cluster_m"].astype(np.float64) * cand["cluster_n"])[None, :]
    assert np.all(fill > 0) and np.all(fill * cl <= 1 + 1e-6)
    # K does not enter; neither do layout, data types or the epilogue
    p2 = prob.copy()
    p2["k"] = 1 + (p2["k"] * 7) % 9973
    p2["layout"] = (p2["layout"] + 1) % 4
    assert np.array_equal(static_scores(p2, cand)[2], s)
    # twice the stages: exactly twice the score; four times tile_k: exactly twice the score
    c2 = cand.copy()
    c2["stages"] = c2["stages"] * 2
    assert np.array_equal(static_scores(prob, c2)[2], 2 * s)
    c4 = cand[cand["tile_k"] <= 64].copy()
    base = static_scores(prob, c4)[2]
    c4["tile_k"] = c4["tile_k"] * 4
    np.testing.assert_allclose(static_scores(prob, c4)[2], 2 * base, rtol=3e-7)
    # an exact multiple of full waves with 1x1 clusters fills perfectly
    p = problem(148 * 128, 3 * 128, 64)
    c = candidate(128, 128, 64, 1)
    assert static_scores(p, c)[2][0, 0] == np.float32(np.sqrt(np.float32(128 * 128 * 64)))


def test_ranking_matches_a_library_sort():
    prob, cand, so, si = wl.make_inputs(2, P=9, seg=700)
    k = 25
    idx, sc, _ = oracle.select(prob, cand, DESC, k, static=True, seg_off=so, seg_idx=si, want_scores=True)
    for i in range(len(prob)):
        pool = si[so[i]:so[i + 1]]
        s = static_scores(prob[i:i + 1], cand[pool])[2][0]
        order = np.lexsort((pool, -s.astype(np.float64)))[:k]
        assert np.array_equal(idx[i], pool[order]) and np.array_equal(sc[i], s[order])
