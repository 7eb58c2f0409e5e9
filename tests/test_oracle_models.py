"""Pins for the oracle's scorers and ranking: special cases with known answers, brute force on
tiny inputs, and library routines (torch CPU linear layers, numpy sorting)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import read_worked_examples

DESC = wl.gpu_desc()
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.txt")


def make_tree(records):
    """records: list of (feat or None, value, left)."""
    nd = np.zeros(len(records), wl.NODE_DT)
    for i, (f, v, left) in enumerate(records):
        nd[i]["feat"] = 0xFFFF if f is None else f
        nd[i]["v"] = v
        nd[i]["left"] = left
    return nd


def test_tiny_scoring_example():
    """Two depth-1 trees on the worked examples: T1 splits the wave count (column 30) at 3.5
    into (+0.1 | -0.2); T2 splits eta_last (column 31) at 0.5 into (-0.3 | +0.3).
    A: 7 waves, eta 0.988 -> -0.2 + 0.3; B: 1 wave, eta 0.108 -> 0.1 - 0.3; C: 1 wave,
    eta 0.541 -> 0.1 + 0.3; D: 1 wave, eta 0.065 -> 0.1 - 0.3."""
    ex = read_worked_examples(GOLDEN)
    x = np.concatenate([oracle.featurize(p, c, DESC) for _, p, c, _ in ex])
    t1 = make_tree([(30, 3.5, 1), (None, 0.1, 0), (None, -0.2, 0)])
    t2 = make_tree([(31, 0.5, 1), (None, -0.3, 0), (None, 0.3, 0)])
    nodes = np.concatenate([t1, t2])
    off = np.array([0, 3, 6])
    s, leaf = oracle.score_gbdt(x, off, nodes, want_leaf_idx=True)
    np.testing.assert_allclose(s, [0.1, -0.2, 0.4, -0.2], rtol=1e-6)
    assert leaf.tolist() == [[2, 2], [1, 1], [1, 2], [1, 1]]
    s2 = oracle.score_gbdt(x, off, nodes, base_score=1.5)
    np.testing.assert_allclose(s2, [1.6, 1.3, 1.9, 1.3], rtol=1e-6)


def test_depth0_trees_give_a_constant():
    x = np.random.default_rng(0).normal(size=(17, 64)).astype(np.float32)
    nodes = make_tree([(None, 0.25, 0), (None, -1.0, 0), (None, 0.5, 0)])
    s, leaf = oracle.score_gbdt(x, np.array([0, 1, 2, 3]), nodes, want_leaf_idx=True)
    assert np.all(s == np.float32(-0.25)) and np.all(leaf == 0)


def test_strict_less_than_goes_left():
    nodes = make_tree([(5, 2.0, 1), (None, 1.0, 0), (None, 2.0, 0)])
    x = np.zeros((3, 64), np.float32)
    x[:, 5] = [np.nextafter(np.float32(2.0), np.float32(0)), 2.0, np.nextafter(np.float32(2.0), np.float32(3))]
    s = oracle.score_gbdt(x, np.array([0, 3]), nodes)
    assert s.tolist() == [1.0, 2.0, 2.0]


def test_non_finite_values_at_a_numeric_split():
    """Model A sends a row left iff x < t: a NaN and +inf are not less than anything (right),
    -inf is less than every finite threshold (left)."""
    nodes = make_tree([(5, 2.0, 1), (None, 1.0, 0), (None, 2.0, 0)])
    x = np.zeros((3, 64), np.float32)
    x[:, 5] = [np.nan, np.inf, -np.inf]
    s = oracle.score_gbdt(x, np.array([0, 3]), nodes)
    assert s.tolist() == [2.0, 2.0, 1.0]


def brute_force_score(x, off, nodes, base=0.0):
    """Explicit loop evaluation, pure Python, fp64 sum in tree order."""
    out = []
    for r in range(len(x)):
        s = float(base)
        ids = []
        for t in range(len(off) - 1):
            i = 0
            tree = nodes[off[t]:off[t + 1]]
            while tree[i]["feat"] != 0xFFFF:
                i = int(tree[i]["left"]) + (0 if x[r, tree[i]["feat"]] < tree[i]["v"] else 1)
            ids.append(i)
            s += float(tree[i]["v"])
        out.append((np.float32(s), ids))
    return out


def test_gbdt_brute_force_and_level_order_leaf_index():
    w = wl.make_workload(0, P=3, C=40, trees=7, depth=4)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    off, nodes, base = w.gbdt
    s, leaf = oracle.score_gbdt(x, off, nodes, base, want_leaf_idx=True)
    ref = brute_force_score(x, off, nodes, base)
    assert np.array_equal(s, np.array([r[0] for r in ref], np.float32))
    assert leaf.tolist() == [r[1] for r in ref]
    # complete tree in level order: leaf index = 2^D - 1 + path bits (1 = went right)
    D = 4
    for r in range(0, len(x), 7):
        for t in range(len(off) - 1):
            tree = nodes[off[t]:off[t + 1]]
            i, bits = 0, 0
            for _ in range(D):
                right = 0 if x[r, tree[i]["feat"]] < tree[i]["v"] else 1
                bits = 2 * bits + right
                i = 2 * i + 1 + right
            assert leaf[r, t] == (1 << D) - 1 + bits
    assert len(np.unique(leaf)) > 4  # the thresholds really split the data


def test_gbdt_unbalanced_tree():
    # root -> (leaf | node) ; node -> (leaf | leaf)
    nodes = make_tree([(1, 0.0, 1), (None, -1.0, 0), (2, 10.0, 3), (None, 5.0, 0), (None, 7.0, 0)])
    x = np.zeros((3, 64), np.float32)
    x[:, 1] = [-1, 1, 1]
    x[:, 2] = [0, 0, 20]
    s, leaf = oracle.score_gbdt(x, np.array([0, 5]), nodes, want_leaf_idx=True)
    assert s.tolist() == [-1.0, 5.0, 7.0] and leaf[:, 0].tolist() == [1, 3, 4]


def bf16_bits_to_f32(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


def test_mlp_zero_weights_give_last_bias():
    mlp = wl.mlp_xavier(1, [64, 64, 1], np.zeros(64), np.ones(64))
    mlp["weights"] = [np.zeros_like(w) for w in mlp["weights"]]
    x = np.random.default_rng(1).normal(size=(9, 64)).astype(np.float32)
    s = oracle.score_mlp(x, mlp)
    assert np.all(s == mlp["biases"][-1][0])


def test_mlp_matches_torch_linear_on_bf16_rounded_tensors():
    """Same rounding points evaluated with torch CPU linear layers in fp64."""
    w = wl.make_workload(4, P=4, C=64)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    mlp = w.mlp
    s = oracle.score_mlp(x, mlp)
    xt = torch.from_numpy(x.copy())
    xt = torch.where(torch.isfinite(xt), xt, torch.zeros_like(xt))
    h = (xt - torch.from_numpy(mlp["mu"])) / torch.from_numpy(mlp["sigma"])
    h[:, 63] = 0
    h = h.to(torch.bfloat16).to(torch.float64)
    L = len(mlp["weights"])
    for l in range(L):
        W = torch.from_numpy(bf16_bits_to_f32(mlp["weights"][l]).astype(np.float64))
        b = torch.from_numpy(mlp["biases"][l].astype(np.float64))
        h = torch.nn.functional.linear(h, W, b).to(torch.float32)
        if l < L - 1:
            h = torch.relu(h).to(torch.bfloat16).to(torch.float64)
    ref = h[:, 0].numpy()
    np.testing.assert_allclose(s, ref, rtol=1e-6, atol=1e-7)
    assert np.std(s) > 1e-3
    # against an evaluation with no bf16 rounding of the activations: within the 2e-2 budget
    h = ((xt - torch.from_numpy(mlp["mu"])) / torch.from_numpy(mlp["sigma"])).to(torch.float64)
    h[:, 63] = 0
    for l in range(L):
        W = torch.from_numpy(bf16_bits_to_f32(mlp["weights"][l]).astype(np.float64))
        h = torch.nn.functional.linear(h, W, torch.from_numpy(mlp["biases"][l].astype(np.float64)))
        if l < L - 1:
            h = torch.relu(h)
    full = h[:, 0].numpy()
    assert np.max(np.abs(s - full) / np.maximum(1.0, np.abs(full))) < 2e-2


def test_mlp_non_finite_inputs_become_zero():
    mlp = wl.mlp_xavier(3, [64, 128, 1], np.full(64, 0.5), np.full(64, 2.0))
    x = np.random.default_rng(2).normal(size=(4, 64)).astype(np.float32)
    y = x.copy()
    y[0, 3], y[1, 10], y[2, 62] = np.nan, np.inf, -np.inf
    z = x.copy()
    z[0, 3], z[1, 10], z[2, 62] = 0, 0, 0
    assert np.array_equal(oracle.score_mlp(y, mlp), oracle.score_mlp(z, mlp))
    # column 63 is ignored
    y = x.copy()
    y[:, 63] = 1e9
    assert np.array_equal(oracle.score_mlp(y, mlp), oracle.score_mlp(x, mlp))


def test_topk_against_numpy_sort():
    rng = np.random.default_rng(5)
    P, n, k = 7, 300, 10
    s = rng.normal(size=P * n).astype(np.float32)
    s[rng.integers(0, P * n, 200)] = 0.5  # ties
    idx, sc = oracle.topk(s, P, k, rows_per_problem=n)
    for i in range(P):
        row = s[i * n:(i + 1) * n]
        order = np.lexsort((np.arange(n), -row.astype(np.float64)))[:k]
        assert idx[i].tolist() == order.tolist()
        assert np.array_equal(sc[i], row[order])
    one, _ = oracle.topk(s, P, 1, rows_per_problem=n)
    for i in range(P):
        row = s[i * n:(i + 1) * n]
        assert one[i, 0] == int(np.argmax(row))  # k = 1 is the argmax rule (first maximum)


def test_topk_padding_ties_and_segments():
    s = np.array([1, 3, 2, 9, 9, 9, 9], np.float32)
    so = np.array([0, 3, 3, 7])
    si = np.array([4, 8, 15, 2, 5, 7, 11], np.int32)
    idx, sc = oracle.topk(s, 3, 5, seg_off=so, seg_idx=si)
    assert idx[0].tolist() == [8, 15, 4, -1, -1]
    assert sc[0, :3].tolist() == [3, 2, 1] and np.all(np.isneginf(sc[0, 3:]))
    assert idx[1].tolist() == [-1] * 5 and np.all(np.isneginf(sc[1]))
    assert idx[2].tolist() == [2, 5, 7, 11, -1]  # all-equal scores: ascending pool index


def test_select_is_the_composition_of_its_steps():
    w = wl.make_workload(0, P=5, C=300, trees=20, depth=5)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    s = oracle.score_gbdt(x, *w.gbdt)
    ridx, rsc = oracle.topk(s, 5, w.k, rows_per_problem=300)
    idx, sc, allsc = oracle.select(w.problems, w.candidates, DESC, w.k, gbdt=w.gbdt, want_scores=True)
    assert np.array_equal(idx, ridx) and np.array_equal(sc, rsc) and np.array_equal(allsc, s)
    w2 = wl.make_workload(2, P=4, C=400, seg=64, trees=10, depth=4)
    x = oracle.featurize(w2.problems, w2.candidates, DESC, w2.seg_offsets, w2.seg_index)
    s = oracle.score_gbdt(x, *w2.gbdt)
    ridx, rsc = oracle.topk(s, 4, 10, seg_off=w2.seg_offsets, seg_idx=w2.seg_index)
    idx, sc = oracle.select(w2.problems, w2.candidates, DESC, 10, gbdt=w2.gbdt,
                            seg_off=w2.seg_offsets, seg_idx=w2.seg_index)
    assert np.array_equal(idx, ridx) and np.array_equal(sc, rsc)
    w4 = wl.make_workload(4, P=2, C=100)
    x = oracle.featurize(w4.problems, w4.candidates, DESC)
    s = oracle.score_mlp(x, w4.mlp)
    ridx, _ = oracle.topk(s, 2, 10, rows_per_problem=100)
    idx, _ = oracle.select(w4.problems, w4.candidates, DESC, 10, mlp=w4.mlp)
    assert np.array_equal(idx, ridx)


def test_one_layer_model_is_the_linear_scorer():
    """n_layers = 1: s = w . bf16((x - mu) / sigma) + b, against a numpy dot product in fp64."""
    st = wl.feature_stats("cfg1")
    prob, cand, _, _ = wl.make_inputs(1, P=2, C=40)
    x = oracle.featurize(prob, cand, DESC)
    m = wl.mlp_xavier(21, [64, 1], st["mu"], st["sigma"])
    s = oracle.score_mlp(x, m)
    xs = ((x - m["mu"]) / m["sigma"]).astype(np.float32)
    xs[:, 63] = 0
    xs = torch.from_numpy(xs).to(torch.bfloat16).to(torch.float64).numpy()
    wv = bf16_bits_to_f32(m["weights"][0]).astype(np.float64)[0]
    ref = xs @ wv + float(m["biases"][0][0])
    np.testing.assert_allclose(s, ref, rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------------------------------------
# partition splits on categorical fields (native categorical handling)
# ---------------------------------------------------------------------------------------------

def cat_node(feat, mask, left):
    nd = np.zeros(1, wl.NODE_DT)
    nd["feat"], nd["kind"], nd["left"] = feat, 1, left
    nd["v"] = np.array([mask], np.uint32).view(np.float32)
    return nd


def test_partition_split_membership_goes_right():
    """kernel_sched (column 17) has codes 0..3; members of the set go right."""
    x = np.zeros((4, 64), np.float32)
    x[:, 17] = [0, 1, 2, 3]
    leaves = make_tree([(None, -1.0, 0), (None, 2.0, 0)])
    for mask in range(1, 15):
        nodes = np.concatenate([cat_node(17, mask, 1), leaves])
        s, leaf = oracle.score_gbdt(x, np.array([0, 3]), nodes, want_leaf_idx=True)
        want = [2.0 if (mask >> c) & 1 else -1.0 for c in range(4)]
        assert s.tolist() == want and leaf[:, 0].tolist() == [2 if v > 0 else 1 for v in want]


def test_partition_split_of_an_upper_set_equals_a_numeric_split():
    """The set {c, c+1, ...} is the numeric split x < c: same leaves on real feature rows."""
    prob, cand, _, _ = wl.make_inputs(1, P=3, C=400)
    x = oracle.featurize(prob, cand, DESC)
    rng = np.random.default_rng(3)
    for col, levels in wl.CATEGORICAL_LEVELS.items():
        for c in range(1, levels):
            upper = sum(1 << v for v in range(c, levels))
            leaves = make_tree([(None, float(rng.normal()), 0), (None, float(rng.normal()), 0)])
            numeric = np.concatenate([make_tree([(col, float(c), 1)]), leaves])
            part = np.concatenate([cat_node(col, upper, 1), leaves])
            a = oracle.score_gbdt(x, np.array([0, 3]), numeric)
            b = oracle.score_gbdt(x, np.array([0, 3]), part)
            assert np.array_equal(a, b), (col, c)


def test_partition_ensemble_against_nested_ifs():
    prob, cand, _, _ = wl.make_inputs(2, P=2, seg=150)
    x = oracle.featurize(prob, cand[:150], DESC)
    off, nodes = wl.gbdt_complete(17, 40, 4, wl.feature_stats("cfg2"), 0.1)
    pnodes = wl.with_partition_splits(5, nodes)
    assert pnodes["kind"].sum() > 20 and np.array_equal(pnodes["feat"], nodes["feat"])
    got = oracle.score_gbdt(x, off, pnodes, base_score=0.25)
    want = np.empty(len(x))
    for r in range(len(x)):
        s = 0.25
        for t in range(len(off) - 1):
            tree = pnodes[off[t]:off[t + 1]]
            i = 0
            while tree[i]["feat"] != 0xFFFF:
                f, v = int(tree[i]["feat"]), tree[i]["v"]
                if tree[i]["kind"] & 1:
                    right = (int(np.float32(v).view(np.uint32)) >> int(x[r, f])) & 1
                else:
                    right = not (x[r, f] < v)
                i = int(tree[i]["left"]) + (1 if right else 0)
            s += float(tree[i]["v"])
        want[r] = s
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-6)
    # complementing a set and swapping the children changes nothing
    flipped = pnodes.copy()
    for t in range(len(off) - 1):
        lo = off[t]
        for i in range(lo, off[t + 1]):
            if flipped[i]["kind"] & 1:
                levels = wl.CATEGORICAL_LEVELS[int(flipped[i]["feat"])]
                m = int(flipped["v"][i:i + 1].view(np.uint32)[0]) ^ ((1 << levels) - 1)
                flipped["v"][i] = np.array([m], np.uint32).view(np.float32)[0]
                l = lo + int(flipped[i]["left"])
                if flipped[l]["feat"] == 0xFFFF and flipped[l + 1]["feat"] == 0xFFFF:
                    flipped[[l, l + 1]] = flipped[[l + 1, l]]
                else:  # only leaf pairs can be swapped in place; undo the complement here
                    flipped["v"][i] = pnodes["v"][i]
    np.testing.assert_allclose(oracle.score_gbdt(x, off, flipped, base_score=0.25), got, rtol=1e-6, atol=1e-6)


# ---------------------------------------------------------------------------------------------
# one-hot input of the ranker (width 80)
# ---------------------------------------------------------------------------------------------

def onehot_numpy(x):
    """The 80-wide input built with numpy indexing: kept columns, then np.eye rows per field."""
    keep = [j for j in range(63) if j not in (5, 9, 17, 18)]
    parts = [x[:, keep]]
    for col, levels in wl.ONEHOT_FIELDS:
        parts.append(np.eye(levels, dtype=np.float32)[x[:, col].astype(np.int64)])
    y = np.concatenate(parts, axis=1)
    return np.concatenate([y, np.zeros((len(x), 80 - y.shape[1]), np.float32)], axis=1)


def test_onehot_mlp_matches_torch_linear_on_the_expanded_input():
    prob, cand, _, _ = wl.make_inputs(2, P=3, seg=120)
    x = oracle.featurize(prob, cand[:120], DESC)
    st = wl.feature_stats("cfg2")
    mu, sg = wl.onehot_stats(st["mu"], st["sigma"])
    mlp = wl.mlp_xavier(21, [80, 128, 64, 1], mu, sg)
    s = oracle.score_mlp(x, mlp)
    y = onehot_numpy(x)
    assert y.shape == (360, 80) and np.all(y[:, 59:73].sum(axis=1) == 4) and np.all(y[:, 73:] == 0)
    h = (torch.from_numpy(y) - torch.from_numpy(mu)) / torch.from_numpy(sg)
    h[:, 73:] = 0
    h = h.to(torch.bfloat16).to(torch.float64)
    L = len(mlp["weights"])
    for l in range(L):
        W = torch.from_numpy(bf16_bits_to_f32(mlp["weights"][l]).astype(np.float64))
        h = torch.nn.functional.linear(h, W, torch.from_numpy(mlp["biases"][l].astype(np.float64)))
        h = h.to(torch.float32)
        if l < L - 1:
            h = torch.relu(h).to(torch.bfloat16).to(torch.float64)
    np.testing.assert_allclose(s, h[:, 0].numpy(), rtol=2e-6, atol=2e-6)


def test_onehot_ridge_with_level_proportional_weights_equals_the_ordinal_ridge():
    """A linear scorer whose indicator weights are level x w reproduces the ordinal-code scorer
    (codes enter unscaled: mu = 0, sigma = 1), when level x w is exact in bf16."""
    prob, cand, _, _ = wl.make_inputs(1, P=4, C=300)
    x = oracle.featurize(prob, cand, DESC)
    st = wl.feature_stats("cfg1")
    mu, sg = st["mu"].copy(), st["sigma"].copy()
    for col, _ in wl.ONEHOT_FIELDS:
        mu[col], sg[col] = 0.0, 1.0
    rng = np.random.default_rng(8)
    w64 = (rng.integers(-8, 9, 64) / 16.0).astype(np.float32)      # few mantissa bits
    w64[63] = 0
    ordinal = {"widths": np.array([64, 1], np.int32), "weights": [wl.float_to_bf16_bits(w64).reshape(1, 64)],
               "biases": [np.array([0.375], np.float32)], "mu": mu, "sigma": sg}
    keep = [j for j in range(63) if j not in (5, 9, 17, 18)]
    w80 = np.zeros(80, np.float32)
    w80[:59] = w64[keep]
    p = 59
    for col, levels in wl.ONEHOT_FIELDS:
        for l in range(levels):
            w80[p] = l * w64[col]
            p += 1
    mu80, sg80 = wl.onehot_stats(mu, sg)
    onehot = {"widths": np.array([80, 1], np.int32), "weights": [wl.float_to_bf16_bits(w80).reshape(1, 80)],
              "biases": [np.array([0.375], np.float32)], "mu": mu80, "sigma": sg80}
    np.testing.assert_allclose(oracle.score_mlp(x, onehot), oracle.score_mlp(x, ordinal), rtol=1e-6, atol=1e-6)
