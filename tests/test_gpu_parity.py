"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on
seeded inputs that span several tiles and a ragged tail, plus the edge cases of the method.

Bars: integer-valued features, leaf indices and top-k indices bit-exact (top-k up to
tolerance ties); float features bit-exact expected, gate 1e-5 relative; tree-ensemble scores
1e-5 * max(1, |s|); MLP scores 2e-2 * max(1, |s|)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import candidate, problem, topk_accept

pytestmark = pytest.mark.gpu

DESC = wl.gpu_desc()
TOL_GBDT, TOL_MLP = 1e-5, 2e-2


@pytest.fixture(scope="module")
def ks():
    from paper_2609_35587_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(ks):
    c = ks.Context(DESC, 0)
    yield c
    c.close()


def dev(ks, a):
    return ks.to_device(a, torch.device("cuda", 0))


def gpu_features(ks, ctx, prob, cand, so=None, si=None):
    pairs = len(prob) * len(cand) if so is None else int(so[-1])
    out = ctx.featurize(dev(ks, prob), len(prob), dev(ks, cand), len(cand),
                        None if so is None else dev(ks, so), None if si is None else dev(ks, si), pairs)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def assert_features_equal(got, ref):
    assert got.shape == ref.shape
    same = got.view(np.uint32) == ref.view(np.uint32)
    if not same.all():
        r, c = np.argwhere(~same)[0]
        raise AssertionError(f"feature [{r}, {c}]: gpu {got[r, c]!r} oracle {ref[r, c]!r} "
                             f"({(~same).sum()} of {same.size} differ)")


# ---------------------------------------------------------------------------------------------
# ks_featurize
# ---------------------------------------------------------------------------------------------

def test_featurize_config0_bit_exact(ks, ctx):
    prob, cand, _, _ = wl.make_inputs(0)
    assert_features_equal(gpu_features(ks, ctx, prob, cand), oracle.featurize(prob, cand, DESC))


def test_featurize_cross_precision_segments_bit_exact(ks, ctx):
    prob, cand, so, si = wl.make_inputs(2, P=37, seg=333)
    got = gpu_features(ks, ctx, prob, cand, so, si)
    assert_features_equal(got, oracle.featurize(prob, cand, DESC, so, si))


def test_featurize_dense_mixed_element_types_bit_exact(ks, ctx):
    """Dense form with the element types changing from problem to problem: the candidate-only
    columns a lane keeps across problems are re-evaluated whenever the combination changes."""
    prob, cand, _, _ = wl.make_inputs(2, P=41, seg=64)
    cand = cand[:1500]
    assert len(np.unique(prob["dtype_ab"].astype(int) * 4 + prob["dtype_d"])) > 3
    assert_features_equal(gpu_features(ks, ctx, prob, cand), oracle.featurize(prob, cand, DESC))


def test_featurize_stream_problems_and_ragged_sizes(ks, ctx):
    prob, cand, _, _ = wl.make_inputs(3, P=301, C=70)
    assert_features_equal(gpu_features(ks, ctx, prob, cand), oracle.featurize(prob, cand, DESC))
    for C in (1, 255, 256, 257):
        prob, cand, _, _ = wl.make_inputs(1, P=3, C=C)
        assert_features_equal(gpu_features(ks, ctx, prob, cand), oracle.featurize(prob, cand, DESC))


def test_featurize_extreme_dimensions_and_wide_knobs(ks, ctx):
    prob = np.concatenate([problem(1, 1, 1), problem(1 << 19, 1 << 19, 1 << 19, 3, 3, 3, 5),
                           problem(524287, 3, 99991, 1, 2, 1, 4), problem(7, 524288, 13, 2, 1, 1, 1)])
    cand = np.concatenate([candidate(64, 16, 32, 2), candidate(256, 256, 512, 12, 16, 1, 2, 2, 1),
                           candidate(192, 80, 256, 9, 1, 16, 1, 1, 0), candidate(128, 48, 64, 5, 4, 4, 3, 0, 0)])
    assert_features_equal(gpu_features(ks, ctx, prob, cand), oracle.featurize(prob, cand, DESC))


def test_featurize_empty_and_uneven_segments(ks, ctx):
    prob, cand, _, _ = wl.make_inputs(2, P=5, seg=1)
    so = np.array([0, 0, 600, 601, 601, 1300], np.int64)
    si = (np.arange(1300) * 7 % len(cand)).astype(np.int32)
    assert_features_equal(gpu_features(ks, ctx, prob, cand, so, si), oracle.featurize(prob, cand, DESC, so, si))


# ---------------------------------------------------------------------------------------------
# ks_score
# ---------------------------------------------------------------------------------------------

def test_score_gbdt_leaf_indices_and_scores(ks, ctx):
    w = wl.make_workload(0, P=16, C=700)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    rs, rleaf = oracle.score_gbdt(x, *w.gbdt, want_leaf_idx=True)
    model = ctx.model_create_gbdt(*w.gbdt)
    s, leaf = ctx.score(dev(ks, x), model, want_leaf_idx=True)
    torch.cuda.synchronize()
    assert np.array_equal(leaf.cpu().numpy().view(np.uint16), rleaf)
    s = s.cpu().numpy()
    assert np.all(np.abs(s - rs) <= TOL_GBDT * np.maximum(1, np.abs(rs)))
    assert len(np.unique(rleaf)) > 32


def test_score_gbdt_unbalanced_and_stump_trees(ks, ctx):
    nodes = np.zeros(9, wl.NODE_DT)
    # tree 0: root -> (leaf | node -> (leaf | leaf)); tree 1: a single leaf; tree 2: depth 1
    recs = [(1, 0.0, 1), (None, -1.0, 0), (2, 10.0, 3), (None, 5.0, 0), (None, 7.0, 0),
            (None, 0.25, 0), (0, 3.0, 1), (None, 100.0, 0), (None, 200.0, 0)]
    for i, (f, v, left) in enumerate(recs):
        nodes[i] = (v, 0xFFFF if f is None else f, 0, left)
    off = np.array([0, 5, 6, 9])
    x = np.zeros((300, 64), np.float32)
    rng = np.random.default_rng(0)
    x[:, :3] = rng.normal(0, 8, size=(300, 3)).astype(np.float32)
    x[0, 0] = 3.0  # exactly on the threshold: not strictly less, goes right
    rs, rleaf = oracle.score_gbdt(x, off, nodes, 0.5, want_leaf_idx=True)
    model = ctx.model_create_gbdt(off, nodes, 0.5)
    s, leaf = ctx.score(dev(ks, x), model, want_leaf_idx=True)
    torch.cuda.synchronize()
    assert np.array_equal(leaf.cpu().numpy().view(np.uint16), rleaf)
    assert np.array_equal(s.cpu().numpy(), rs)


def test_score_gbdt_quantised_path(ks, ctx):
    """Scores without leaf indices from a qualifying ensemble take the quantised walk on tiles
    built from the given rows: ragged row count, non-finite inputs (a NaN goes right at a numeric
    split, as x < t is false), partition splits."""
    w = wl.make_workload(1, P=5, C=3000, trees=60, depth=8)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    rng = np.random.default_rng(3)
    numeric = np.array([c for c in range(63) if c not in wl.CATEGORICAL_LEVELS])
    for v in (np.nan, np.inf, -np.inf):
        x[rng.integers(0, len(x), 200), numeric[rng.integers(0, len(numeric), 200)]] = v
    for gbdt in (w.gbdt, (w.gbdt[0], wl.with_partition_splits(5, w.gbdt[1]), w.gbdt[2])):
        rs = oracle.score_gbdt(x, *gbdt)
        model = ctx.model_create_gbdt(*gbdt)
        d_x = dev(ks, x)
        n0 = ctx.launch_count()
        s = ctx.score(d_x, model).cpu().numpy()
        assert ctx.launch_count() - n0 == 2          # tile launch + walk launch
        assert np.all(np.abs(s - rs) <= TOL_GBDT * np.maximum(1, np.abs(rs)))
        s2, leaf = ctx.score(d_x, model, want_leaf_idx=True)   # the general kernel
        _, rleaf = oracle.score_gbdt(x, *gbdt, want_leaf_idx=True)
        assert np.array_equal(leaf.cpu().numpy().view(np.uint16), rleaf)
        assert np.all(np.abs(s - s2.cpu().numpy()) <= TOL_GBDT * np.maximum(1, np.abs(rs)))
    for n in (1, 1023, 1024, 1025):
        s = ctx.score(dev(ks, x[:n]), model).cpu().numpy()
        assert np.all(np.abs(s - rs[:n]) <= TOL_GBDT * np.maximum(1, np.abs(rs[:n])))


def test_walk_floor_sums(ks, ctx):
    """The measurement form of the walk (ks_debug_walk_floor) walks real trees on real tiles:
    its sums are those of the ensemble's first two chunks, repeated as the header says."""
    import re
    w = wl.make_workload(1, P=1, C=2500, trees=60, depth=8)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    off, nodes, base = w.gbdt
    model = ctx.model_create_gbdt(off, nodes, base)
    m = re.search(r"threads=(\d+) block=1024 .*chunks=(\d+) chunk_trees=(\d+)", model.describe())
    assert m, model.describe()
    G, n_chunks, tpc = int(m.group(1)) // 256, int(m.group(2)), int(m.group(3))
    assert n_chunks >= 2 * G
    # tree group g walks chunks g, g + G, ...; its first two stay resident
    part = [oracle.score_gbdt(x, off[c * tpc:(c + 1) * tpc + 1] - off[c * tpc],
                              nodes[off[c * tpc]:off[(c + 1) * tpc]], 0.0).astype(np.float64) for c in range(2 * G)]
    d_x = dev(ks, x)
    for repeat in (1, 3):
        got = ctx.debug_walk_floor(d_x, model, repeat).cpu().numpy()
        want = np.full(len(x), np.float64(base))
        walks = 0
        for g in range(G):
            n = repeat * len(range(g, n_chunks, G))
            want += ((n + 1) // 2) * part[g] + (n // 2) * part[g + G]
            walks += n
        assert np.all(np.abs(got - want) <= 4 * TOL_GBDT * walks * np.maximum(1, np.abs(want)))
    assert np.std(part[0]) > 1e-2
    # an ensemble in another tile geometry or shape is refused
    w2 = wl.make_workload(0, P=1, C=300)
    model2 = ctx.model_create_gbdt(*w2.gbdt)
    with pytest.raises(ks.KsError) as e:
        ctx.debug_walk_floor(dev(ks, oracle.featurize(w2.problems, w2.candidates, DESC)), model2, 2)
    assert e.value.status == ks.KS_ERR_UNSUPPORTED


def test_score_mlp(ks, ctx):
    w = wl.make_workload(4, P=3, C=411)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    x[5, 7] = np.nan
    x[6, 40] = np.inf
    rs = oracle.score_mlp(x, w.mlp)
    model = ctx.model_create_mlp(w.mlp)
    s = ctx.score(dev(ks, x), model).cpu().numpy()
    assert np.all(np.isfinite(s))
    assert np.all(np.abs(s - rs) <= TOL_MLP * np.maximum(1, np.abs(rs)))
    assert np.std(rs) > 1e-2


def test_score_mlp_tensor_core_path(ks, ctx):
    """ks_score with a model the tensor-core kernel serves (ordinal input, one or two hidden layers
    of at most 256 units) runs there on the given rows: more tiles than CTAs with an uneven share,
    a ragged last tile, tiny inputs, padded shapes; the one-hot form and wider models take the
    general kernel."""
    w = wl.make_workload(4, P=8, C=5003)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    x[17, 3] = np.nan
    x[40001, 62] = -np.inf
    st = wl.feature_stats("cfg1")
    for shape in ([64, 256, 256, 1], [64, 128, 1], [64, 256, 64, 1]):
        mlp = w.mlp if shape == [64, 256, 256, 1] else wl.mlp_xavier(77, shape, st["mu"], st["sigma"])
        rs = oracle.score_mlp(x, mlp)
        model = ctx.model_create_mlp(mlp)
        d_x = dev(ks, x)
        n0 = ctx.launch_count()
        s = ctx.score(d_x, model).cpu().numpy()
        assert ctx.launch_count() - n0 == 2            # flag reset + the tensor-core kernel
        assert np.all(np.abs(s - rs) <= TOL_MLP * np.maximum(1, np.abs(rs)))
        for n in (1, 127, 128, 129, 148 * 128 + 5):
            s = ctx.score(dev(ks, x[:n]), model).cpu().numpy()
            assert np.all(np.abs(s - rs[:n]) <= TOL_MLP * np.maximum(1, np.abs(rs[:n])))


# ---------------------------------------------------------------------------------------------
# ks_select
# ---------------------------------------------------------------------------------------------

def check_select(w, idx, sc, tol, sample=None):
    """Compare [P, k] GPU results with the oracle (all problems, or the sampled ones)."""
    P = len(w.problems)
    probs = range(P) if sample is None else sample
    sel = np.array(list(probs))
    if w.seg_offsets is None:
        so = si = None
        sub_so = None
    else:
        so, si = w.seg_offsets, w.seg_index
    for i in sel:
        p1 = w.problems[i:i + 1]
        if so is None:
            _, _, allsc = oracle.select(p1, w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp, want_scores=True)
            pool = np.arange(len(w.candidates), dtype=np.int32)
        else:
            pool = si[so[i]:so[i + 1]]
            _, _, allsc = oracle.select(p1, w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp,
                                        seg_off=np.array([0, len(pool)], np.int64), seg_idx=pool,
                                        want_scores=True)
        ok, msg = topk_accept(idx[i], sc[i], allsc, pool, idx.shape[1], tol)
        assert ok, f"problem {i}: {msg}"


def run_select(ks, ctx, w, model, k=None):
    k = w.k if k is None else k
    P, C = len(w.problems), len(w.candidates)
    idx, sc = ctx.select(dev(ks, w.problems), P, dev(ks, w.candidates), C, model, k,
                         None if w.seg_offsets is None else dev(ks, w.seg_offsets),
                         None if w.seg_index is None else dev(ks, w.seg_index), w.pairs)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), sc.cpu().numpy()


def test_select_config0_matches_oracle_exactly(ks, ctx):
    w = wl.make_workload(0)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    ridx, rsc = oracle.select(w.problems, w.candidates, DESC, w.k, gbdt=w.gbdt)
    check_select(w, idx, sc, TOL_GBDT)
    # no tolerance tie occurs in this workload, so the index lists are simply equal
    assert np.array_equal(idx, ridx)
    assert np.all(np.abs(sc - rsc) <= TOL_GBDT * np.maximum(1, np.abs(rsc)))
    idx2, sc2 = run_select(ks, ctx, w, model)
    assert np.array_equal(idx, idx2) and np.array_equal(sc.view(np.uint32), sc2.view(np.uint32))


def test_select_segments_cross_precision(ks, ctx):
    w = wl.make_workload(2, P=24, seg=3000, trees=60, depth=8)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)


def test_select_full_space_shape_small(ks, ctx):
    w = wl.make_workload(1, P=6, C=5000, trees=50)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)
    ridx, _ = oracle.select(w.problems, w.candidates, DESC, w.k, gbdt=w.gbdt)
    assert np.array_equal(idx, ridx)


@pytest.mark.parametrize("C,k", [(1, 5), (3, 32), (33, 1), (257, 10), (2049, 32)])
def test_select_ragged_sizes_and_padding(ks, ctx, C, k):
    w = wl.make_workload(0, P=3, C=C, trees=9, depth=3)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model, k)
    x = oracle.featurize(w.problems, w.candidates, DESC)
    s = oracle.score_gbdt(x, *w.gbdt)
    ridx, rsc = oracle.topk(s, 3, k, rows_per_problem=C)
    for i in range(3):
        ok, msg = topk_accept(idx[i], sc[i], s[i * C:(i + 1) * C], np.arange(C, dtype=np.int32), k, TOL_GBDT)
        assert ok, msg
    if k > C:
        assert np.all(idx[:, C:] == -1) and np.all(np.isneginf(sc[:, C:]))


def test_select_all_equal_scores_returns_lowest_indices(ks, ctx):
    nodes = np.zeros(2, wl.NODE_DT)
    nodes[0] = (0.125, 0xFFFF, 0, 0)
    nodes[1] = (-0.5, 0xFFFF, 0, 0)
    prob, cand, _, _ = wl.make_inputs(0, P=4, C=1000)
    w = wl.Workload("ties", DESC, prob, cand, 7, gbdt=(np.array([0, 1, 2]), nodes, 0.0))
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    assert np.array_equal(idx, np.tile(np.arange(7, dtype=np.int32), (4, 1)))
    assert np.all(sc == np.float32(-0.375))


def test_select_empty_and_uneven_segments(ks, ctx):
    w = wl.make_workload(2, P=5, seg=1, trees=12, depth=4)
    w.seg_offsets = np.array([0, 0, 600, 601, 601, 5300], np.int64)
    w.seg_index = np.concatenate([np.sort(np.random.default_rng(i).choice(len(w.candidates), n, replace=False))
                                  for i, n in enumerate([0, 600, 1, 0, 4699])]).astype(np.int32)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    assert np.all(idx[0] == -1) and np.all(idx[3] == -1) and np.all(np.isneginf(sc[0]))
    assert idx[2, 0] == w.seg_index[600] and np.all(idx[2, 1:] == -1)
    check_select(w, idx, sc, TOL_GBDT)


def test_select_mlp(ks, ctx):
    w = wl.make_workload(4, P=3, C=1500)
    model = ctx.model_create_mlp(w.mlp)
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_MLP)


def test_select_mlp_segments_and_uneven_sizes(ks, ctx):
    """The tensor-core kernel on per-problem segments (uneven, one empty), and on sizes around
    its 4,096-row blocks, where CTAs of one problem walk different numbers of tiles."""
    w = wl.make_workload(2, P=6, seg=5000, trees=4, depth=2)
    w.mlp = wl.make_workload(4, P=1, C=16).mlp
    w.gbdt = None
    w.seg_offsets = np.array([0, 4097, 4097, 9000, 9001, 17193, 21500], np.int64)
    w.seg_index = np.concatenate([np.sort(np.random.default_rng(i).choice(len(w.candidates), n, replace=False))
                                  for i, n in enumerate(np.diff(w.seg_offsets))]).astype(np.int32)
    model = ctx.model_create_mlp(w.mlp)
    idx, sc = run_select(ks, ctx, w, model)
    assert np.all(idx[1] == -1) and np.all(np.isneginf(sc[1]))
    assert idx[3, 0] == w.seg_index[9000] and np.all(idx[3, 1:] == -1)
    check_select(w, idx, sc, TOL_MLP)
    for C in (4095, 4096, 4097, 8193):
        wd = wl.make_workload(4, P=2, C=C)
        idx, sc = run_select(ks, ctx, wd, ctx.model_create_mlp(wd.mlp))
        check_select(wd, idx, sc, TOL_MLP)


def test_select_mlp_every_score(ks, ctx):
    """k >= |segment| returns every pair's score: each one against the oracle, on sizes that
    cross the 128-row tile and the 2,048-row block of the tensor-core kernel."""
    for C in (1, 32, 127, 129):
        w = wl.make_workload(4, P=5, C=C)
        model = ctx.model_create_mlp(w.mlp)
        idx, sc = run_select(ks, ctx, w, model, 32)
        _, _, allsc = oracle.select(w.problems, w.candidates, DESC, 32, mlp=w.mlp, want_scores=True)
        for i in range(5):
            ref = allsc[i * C:(i + 1) * C]
            n = min(C, 32)
            got_idx = idx[i, :n]
            assert len(set(got_idx.tolist())) == n and got_idx.min() >= 0 and got_idx.max() < C
            err = np.abs(sc[i, :n] - ref[got_idx]) / np.maximum(1, np.abs(ref[got_idx]))
            assert err.max() < 5e-3, (C, i, err.max())
            assert np.all(idx[i, n:] == -1)
    w = wl.make_workload(4, P=2, C=4500)
    model = ctx.model_create_mlp(w.mlp)
    idx, sc = run_select(ks, ctx, w, model, 32)
    check_select(w, idx, sc, TOL_MLP)
    _, _, allsc = oracle.select(w.problems, w.candidates, DESC, 32, mlp=w.mlp, want_scores=True)
    for i in range(2):
        ref = allsc[i * 4500:(i + 1) * 4500]
        err = np.abs(sc[i] - ref[idx[i]]) / np.maximum(1, np.abs(ref[idx[i]]))
        assert err.max() < 5e-3
    # narrower layers and a single hidden layer run on the same kernel, padded with zero units
    # (and an identity second layer); three hidden layers stay on the general kernel
    st = wl.feature_stats("cfg1")
    ohm, ohs = wl.onehot_stats(st["mu"], st["sigma"])
    for widths in ([64, 128, 64, 1], [64, 64, 1], [64, 256, 128, 1], [80, 192, 1], [80, 64, 256, 1], [64, 128, 128, 64, 1]):
        mu, sg = (w.mlp["mu"], w.mlp["sigma"]) if widths[0] == 64 else (ohm, ohs)
        m2 = wl.mlp_xavier(11, widths, mu, sg)
        w2 = wl.Workload("mlp2", DESC, w.problems, w.candidates[:300], 32, mlp=m2)
        idx, sc = run_select(ks, ctx, w2, ctx.model_create_mlp(m2))
        check_select(w2, idx, sc, TOL_MLP)
        _, _, allsc = oracle.select(w2.problems, w2.candidates, DESC, 32, mlp=m2, want_scores=True)
        for i in range(2):
            ref = allsc[i * 300:(i + 1) * 300]
            err = np.abs(sc[i] - ref[idx[i]]) / np.maximum(1, np.abs(ref[idx[i]]))
            assert err.max() < 5e-3, (widths, err.max())


def test_select_one_and_select_host_agree_with_select(ks, ctx):
    w = wl.make_workload(3, P=4, C=3000, trees=30)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    d_c = dev(ks, w.candidates)
    for i in range(4):
        # the latency form adds the trees' leaves in a different (fixed) order: same ranking,
        # scores equal up to rounding
        hi, hs = ctx.select_one(w.problems[i:i + 1], d_c, len(w.candidates), model, w.k)
        assert np.array_equal(hi.numpy(), idx[i])
        assert np.all(np.abs(hs.numpy() - sc[i]) <= TOL_GBDT * np.maximum(1, np.abs(sc[i])))
        hi2, hs2 = ctx.select_one(w.problems[i:i + 1], d_c, len(w.candidates), model, w.k)
        assert np.array_equal(hi.numpy(), hi2.numpy()) and np.array_equal(hs.numpy(), hs2.numpy())
    hi, hs = ctx.select_host(w.problems, 4, w.candidates, len(w.candidates), model, w.k)
    assert np.array_equal(hi.numpy(), idx) and np.array_equal(hs.numpy(), sc)
    check_select(w, idx, sc, TOL_GBDT)
    w2 = wl.make_workload(2, P=6, seg=500, trees=10, depth=5)
    model2 = ctx.model_create_gbdt(*w2.gbdt)
    idx2, sc2 = run_select(ks, ctx, w2, model2)
    hi, hs = ctx.select_host(w2.problems, 6, w2.candidates, len(w2.candidates), model2, w2.k,
                             w2.seg_offsets, w2.seg_index, w2.pairs)
    assert np.array_equal(hi.numpy(), idx2) and np.array_equal(hs.numpy(), sc2)


def test_select_one_latency_stream_against_oracle(ks, ctx):
    """Single problems of the latency stream (arbitrary integer dimensions, decode-like M)
    against the full catalogue and the 500-tree ensemble, each checked against the oracle."""
    w = wl.make_workload(3, P=6)
    model = ctx.model_create_gbdt(*w.gbdt)
    d_c = dev(ks, w.candidates)
    C = len(w.candidates)
    for i in range(len(w.problems)):
        hi, hs = ctx.select_one(w.problems[i:i + 1], d_c, C, model, w.k)
        _, _, allsc = oracle.select(w.problems[i:i + 1], w.candidates, DESC, w.k, gbdt=w.gbdt, want_scores=True)
        ok, msg = topk_accept(hi.numpy(), hs.numpy(), allsc, np.arange(C, dtype=np.int32), w.k, TOL_GBDT)
        assert ok, f"call {i}: {msg}"
    for C2 in (1, 2047, 2049, 5000):
        hi, hs = ctx.select_one(w.problems[:1], d_c, C2, model, w.k)
        _, _, allsc = oracle.select(w.problems[:1], w.candidates[:C2], DESC, w.k, gbdt=w.gbdt, want_scores=True)
        ok, msg = topk_accept(hi.numpy(), hs.numpy(), allsc, np.arange(C2, dtype=np.int32), w.k, TOL_GBDT)
        assert ok, f"C={C2}: {msg}"


# ---------------------------------------------------------------------------------------------
# host-side error behaviour (status codes, never a fault)
# ---------------------------------------------------------------------------------------------

def test_invalid_arguments_return_status_codes(ks, ctx):
    w = wl.make_workload(0, P=2, C=64, trees=3, depth=2)
    model = ctx.model_create_gbdt(*w.gbdt)
    d_p, d_c = dev(ks, w.problems), dev(ks, w.candidates)
    for k in (0, -1, 33):
        with pytest.raises(ks.KsError) as e:
            ctx.select(d_p, 2, d_c, 64, model, k)
        assert e.value.status == ks.KS_ERR_INVALID_ARG
    with pytest.raises(ks.KsError):
        ctx.select(d_p, 2, d_c, 64, model, 5, pairs=127)  # pairs must equal P*C
    with pytest.raises(ks.KsError):
        ctx.select(None, 2, d_c, 64, model, 5)
    idx, sc = ctx.select(d_p, 0, d_c, 64, model, 5, out_idx=torch.zeros((1, 5), dtype=torch.int32, device="cuda"),
                         out_score=torch.zeros((1, 5), device="cuda"))  # P = 0 is a no-op
    bad = w.gbdt[1].copy()
    bad["feat"][0] = 63
    with pytest.raises(ks.KsError):
        ctx.model_create_gbdt(w.gbdt[0], bad)
    bad = w.gbdt[1].copy()
    bad["left"][0] = 0  # child index not after its parent
    with pytest.raises(ks.KsError):
        ctx.model_create_gbdt(w.gbdt[0], bad)
    bad = w.gbdt[1].copy()
    bad["v"][1] = np.nan
    with pytest.raises(ks.KsError):
        ctx.model_create_gbdt(w.gbdt[0], bad)
    bad = w.gbdt[1].copy()
    bad["left"][1] = 5  # two parents for node 5
    with pytest.raises(ks.KsError):
        ctx.model_create_gbdt(w.gbdt[0], bad)
    m4 = wl.make_workload(4, P=1, C=8).mlp
    m4["sigma"] = m4["sigma"].copy()
    m4["sigma"][3] = 0
    with pytest.raises(ks.KsError):
        ctx.model_create_mlp(m4)
    with pytest.raises(ks.KsError):
        ctx.select_one(problem(0, 5, 5), d_c, 64, model, 5)


# ---------------------------------------------------------------------------------------------
# model shapes that take the other code paths of the fused tree kernel
# ---------------------------------------------------------------------------------------------

def random_trees(seed, n_trees, max_depth, p_split, thresholds):
    """Random (unbalanced) trees in breadth-first order; thresholds(feat, rng) draws a split."""
    rng = np.random.default_rng(seed)
    nodes, offsets = [], [0]
    for _ in range(n_trees):
        tree = [None]            # records (feat or None, value, left)
        frontier = [(0, 0)]      # (node index, depth)
        while frontier:
            i, d = frontier.pop(0)
            if d < max_depth and (d == 0 or rng.random() < p_split):
                f = int(rng.integers(0, 63))
                left = len(tree)
                tree += [None, None]
                tree[i] = (f, float(thresholds(f, rng)), left)
                frontier += [(left, d + 1), (left + 1, d + 1)]
            else:
                tree[i] = (None, float(rng.normal(0, 0.1)), 0)
        nodes += tree
        offsets.append(len(nodes))
    nd = np.zeros(len(nodes), wl.NODE_DT)
    for i, (f, v, left) in enumerate(nodes):
        nd[i] = (np.float32(v), 0xFFFF if f is None else f, 0, left)
    return np.array(offsets, np.int64), nd


def slot_thresholds(stats_key):
    thr = wl.feature_stats(stats_key)["thr"]
    return lambda f, rng: thr[f, rng.integers(0, thr.shape[1])]


@pytest.mark.parametrize("case", ["unbalanced_depth8", "depth9", "depth10", "odd_tree_count", "deep_generic",
                                  "many_shallow_trees", "split_rows", "too_many_rows"])
def test_select_other_model_shapes(ks, ctx, case):
    prob, cand, _, _ = wl.make_inputs(1, P=5, C=3000)
    x = oracle.featurize(prob, cand, DESC)
    if case == "unbalanced_depth8":      # padded to complete trees on the quantised path
        off, nodes = random_trees(1, 40, 8, 0.7, slot_thresholds("cfg1"))
    elif case == "depth9":               # four trees per 16 KB chunk
        off, nodes = random_trees(6, 30, 9, 0.8, slot_thresholds("cfg1"))
    elif case == "depth10":              # two trees per chunk: each half of a CTA walks one
        off, nodes = random_trees(7, 21, 10, 0.8, slot_thresholds("cfg1"))
    elif case == "odd_tree_count":       # the last chunk is padded with empty trees
        off, nodes = random_trees(8, 13, 8, 0.8, slot_thresholds("cfg1"))
    elif case == "deep_generic":         # depth 12 > 10: generic kernel
        off, nodes = random_trees(2, 12, 12, 0.8, slot_thresholds("cfg1"))
    elif case == "many_shallow_trees":   # 2,500 trees: fewer top levels fit the constant bank
        off, nodes = random_trees(3, 2500, 3, 0.9, slot_thresholds("cfg1"))
    elif case == "split_rows":           # > 127 distinct thresholds on some columns: two rows each
        lo, hi = x.min(axis=0), x.max(axis=0)
        def thr(f, rng):
            if f in (27, 31, 39):
                return np.float32(lo[f] + (hi[f] - lo[f]) * (rng.integers(1, 300) / 300.0))
            return slot_thresholds("cfg1")(f, rng)
        off, nodes = random_trees(4, 120, 7, 0.85, thr)
    else:                                # continuous thresholds everywhere: too many rows, generic kernel
        lo, hi = x.min(axis=0), x.max(axis=0)
        off, nodes = random_trees(5, 150, 7, 0.9, lambda f, rng: np.float32(lo[f] + (hi[f] - lo[f]) * rng.random()))
    w = wl.Workload(case, DESC, prob, cand, 10, gbdt=(off, nodes, 0.25))
    model = ctx.model_create_gbdt(off, nodes, 0.25)
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)
    d_c = dev(ks, cand)
    hi_, hs_ = ctx.select_one(prob[2:3], d_c, len(cand), model, 10)
    assert np.array_equal(hi_.numpy(), idx[2])


@pytest.mark.parametrize("case", ["cfg1_slots128", "cfg1_hist256", "cfg1_pernode", "cfg2_pernode", "continuous"])
def test_select_tile_geometries(ks, ctx, case):
    """The quantised kernel's tile geometries, picked by the number of rows: the slot-table
    ensemble (<= 74 rows: two CTAs of 256 threads x 1,024 candidates per SM), the 256-bin and the
    quantile-per-node ensembles of config 1 (<= 156 rows: one CTA of 512 threads x 1,024
    candidates with 32 KB chunk buffers), the quantile-per-node ensemble of config 2 (<= 376 rows:
    one CTA of 512 threads x 512 candidates), and an ensemble with a continuous threshold at every node of 3,000 trees (more
    rows than any geometry holds: the general kernel). Each: a batch (ks_select), the single-problem call (tree slices
    over prepared tiles), the scoring call on given feature rows, and a batch of 33 problems or
    more that takes the per-(problem, class) memo."""
    if case == "continuous":
        prob, cand, _, _ = wl.make_inputs(1, P=3, C=2500)
        x = oracle.featurize(prob, cand, DESC)
        lo, hi = x.min(axis=0), x.max(axis=0)
        off, nodes = random_trees(5, 3000, 5, 0.95, lambda f, rng: np.float32(lo[f] + (hi[f] - lo[f]) * rng.random()))
        w = wl.Workload(case, DESC, prob, cand, 10, gbdt=(off, nodes, 0.0))
        want = "select_generic_kernel"
    elif case == "cfg2_pernode":
        w = wl.make_workload(2, P=6, seg=2500, law="pernode")
        want = "threads=512 block=512"
    else:
        law = case.split("_")[1]
        w = wl.make_workload(1, P=5, C=3000, law=law)
        want = "threads=256 block=1024" if law == "slots128" else "threads=512 block=1024"
    model = ctx.model_create_gbdt(*w.gbdt)
    assert want in model.describe(), model.describe()
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)
    if case == "continuous":
        return
    # single-problem call against the dense pool, and the scoring call on given rows
    C = min(len(w.candidates), 2600)
    cand = w.candidates[:C]
    d_c = dev(ks, cand)
    for i in (0, len(w.problems) - 1):
        hi_, hs_ = ctx.select_one(w.problems[i:i + 1], d_c, C, model, 10)
        _, _, allsc = oracle.select(w.problems[i:i + 1], cand, DESC, 10, gbdt=w.gbdt, want_scores=True)
        ok, msg = topk_accept(hi_.numpy(), hs_.numpy(), allsc, np.arange(C, dtype=np.int32), 10, TOL_GBDT)
        assert ok, msg
    x = oracle.featurize(w.problems[:2], cand, DESC)
    rs = oracle.score_gbdt(x, *w.gbdt)
    s = ctx.score(dev(ks, x), model).cpu().numpy()
    assert np.all(np.abs(s - rs) <= TOL_GBDT * np.maximum(1, np.abs(rs)))
    # memo path: 40 problems, few candidates
    cfg = 2 if case.startswith("cfg2") else 1
    wm = wl.make_workload(cfg, P=40, C=None if cfg == 2 else 700, seg=600 if cfg == 2 else None, law=w.meta["law"])
    idx, sc = run_select(ks, ctx, wm, model)
    check_select(wm, idx, sc, TOL_GBDT, sample=range(0, 40, 3))


@pytest.mark.parametrize("geometry", ["512,1024,32", "512,1024,16", "512,512,32", "512,512,16", "256,512,16", "256,1024,16"])
def test_select_forced_tile_geometry(ks, ctx, geometry, monkeypatch):
    """Every tile geometry on the same ensemble (config 1, a quantile per node, 143 rows), forced
    through KS_FAST_GEOMETRY = threads, candidates per CTA, chunk-buffer KiB."""
    monkeypatch.setenv("KS_FAST_GEOMETRY", geometry)
    w = wl.make_workload(1, P=4, C=2700, law="pernode")
    model = ctx.model_create_gbdt(*w.gbdt)
    t, c, _ = geometry.split(",")
    assert f"threads={t} block={c}" in model.describe(), model.describe()
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)
    hi_, hs_ = ctx.select_one(w.problems[1:2], dev(ks, w.candidates), len(w.candidates), model, 10)
    assert np.array_equal(hi_.numpy(), idx[1])


@pytest.mark.parametrize("geometry,segments", [("512,1024,32", False), ("512,512,16", False), ("512,512,32", True)])
def test_select_more_items_than_sms(ks, ctx, geometry, segments, monkeypatch):
    """The one-CTA-per-SM geometries launch one CTA per SM and let it serve many (problem,
    candidate block) items: here 330 to 660 items, not a multiple of the 148 CTAs, so that some
    CTAs take one item more than others, with a ragged last block per problem; dense catalogue
    (ranked in similarity order) and per-problem segments."""
    monkeypatch.setenv("KS_FAST_GEOMETRY", geometry)
    if segments:
        w = wl.make_workload(2, P=110, seg=1300, trees=24, depth=8, law="pernode")
    else:
        w = wl.make_workload(1, P=110, C=2700, trees=24, depth=8, law="pernode")
    model = ctx.model_create_gbdt(*w.gbdt)
    t, c, _ = geometry.split(",")
    assert f"threads={t} block={c}" in model.describe(), model.describe()
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT, sample=range(0, 110, 2))
    idx2, sc2 = run_select(ks, ctx, w, model)     # the barriers' parities carry over from call to call
    assert np.array_equal(idx, idx2) and np.array_equal(sc, sc2)
    if not segments:
        # a CTA keeps a candidate block's candidate-only rows from one problem to the next while
        # the element types stay the same: runs of equal types of every length, and switches
        rng = np.random.default_rng(11)
        w.problems = w.problems.copy()
        kinds = [(0, 0), (1, 1), (2, 1), (3, 3)]       # (dtype_ab, dtype_d)
        pick = np.repeat(rng.integers(0, 4, 40), rng.integers(1, 6, 40))[:110]
        w.problems["dtype_ab"] = [kinds[i][0] for i in pick]
        w.problems["dtype_d"] = [kinds[i][1] for i in pick]
        idx, sc = run_select(ks, ctx, w, model)
        check_select(w, idx, sc, TOL_GBDT, sample=range(0, 110, 3))


@pytest.mark.parametrize("law", ["slots128", "pernode"])
def test_select_one_prepared_catalogue(ks, ctx, law):
    """The single-problem call against a prepared catalogue (candidate-only rows and classes made
    once per catalogue and model): every call must give the oracle's ranking and the same result
    as the unprepared call; mixed element types use different slices of the prepared tables; a
    model the quantised path does not serve goes through the plain call."""
    w = wl.make_workload(3, P=12, C=7000, law=law)
    probs = w.problems.copy()
    probs["dtype_ab"][3:6] = [1, 2, 3]
    probs["dtype_d"][3:6] = [1, 1, 3]
    probs["epi_flags"][6:8] = [3, 4]
    model = ctx.model_create_gbdt(*w.gbdt)
    C = len(w.candidates)
    d_c = dev(ks, w.candidates)
    cat = ctx.catalogue_prepare(d_c, C, model)
    n0 = ctx.launch_count()
    hi, hs = ctx.select_one_prepared(cat, probs[:1], 10)
    assert ctx.launch_count() - n0 == 2   # the per-class table of the problem, then the fused walk + top-k
    for i in range(len(probs)):
        hi, hs = ctx.select_one_prepared(cat, probs[i:i + 1], 10)
        hi, hs = hi.numpy().copy(), hs.numpy().copy()
        _, _, allsc = oracle.select(probs[i:i + 1], w.candidates, DESC, 10, gbdt=w.gbdt, want_scores=True)
        ok, msg = topk_accept(hi, hs, allsc, np.arange(C, dtype=np.int32), 10, TOL_GBDT)
        assert ok, f"problem {i}: {msg}"
        pi, ps = ctx.select_one(probs[i:i + 1], d_c, C, model, 10)
        assert np.array_equal(pi.numpy(), hi) and np.array_equal(ps.numpy(), hs)
    call = ctx.select_one_caller(d_c, C, model, 10, catalogue=cat)
    ci, cs = call(ks.problem_structs(probs[2:3])[0])
    pi, ps = ctx.select_one(probs[2:3], d_c, C, model, 10)
    assert np.array_equal(ci.numpy(), pi.numpy())
    cat.close()
    # other k, a tiny pool (a single block: no slices, plain call), and an MLP
    small = ctx.catalogue_prepare(d_c, 40, model)
    hi, hs = ctx.select_one_prepared(small, probs[:1], 32)
    pi, ps = ctx.select_one(probs[:1], d_c, 40, model, 32)
    assert np.array_equal(hi.numpy(), pi.numpy())
    w4 = wl.make_workload(4, P=1, C=16)
    mlp = ctx.model_create_mlp(w4.mlp)
    mcat = ctx.catalogue_prepare(d_c, C, mlp)
    hi, hs = ctx.select_one_prepared(mcat, probs[:1], 10)
    pi, ps = ctx.select_one(probs[:1], d_c, C, mlp, 10)
    assert np.array_equal(hi.numpy(), pi.numpy())


def test_merge_topk_of_candidate_shares(ks, ctx):
    """The exchange step of the candidate-split form: three shares of a pool are ranked separately
    (per-share segments), their lists are concatenated as a gather would, and ks_merge_topk must
    give the ranking of the whole pool; plus padding entries and exact ties."""
    w = wl.make_workload(1, P=4, C=2000, trees=30, depth=6)
    model = ctx.model_create_gbdt(*w.gbdt)
    k, C, P = 10, 2000, 4
    d_p, d_c = dev(ks, w.problems), dev(ks, w.candidates)
    parts_i, parts_s = [], []
    for lo, hi in ((0, 700), (700, 707), (707, 2000)):   # the middle share has fewer than k members
        so = np.arange(P + 1, dtype=np.int64) * (hi - lo)
        si = np.tile(np.arange(lo, hi, dtype=np.int32), P)
        i, s = ctx.select(d_p, P, d_c, C, model, k, dev(ks, so), dev(ks, si), int(so[-1]))
        parts_i.append(i)
        parts_s.append(s)
    gi, gs = ctx.merge_topk(torch.cat(parts_i, dim=1).contiguous(), torch.cat(parts_s, dim=1).contiguous(), k)
    torch.cuda.synchronize()
    check_select(w, gi.cpu().numpy(), gs.cpu().numpy(), TOL_GBDT)
    # ties and padding against the plain definition
    rng = np.random.default_rng(5)
    idx = rng.permutation(400).astype(np.int32).reshape(2, 200)
    sc = rng.integers(0, 6, (2, 200)).astype(np.float32)
    idx[:, ::7] = -1
    gi, gs = ctx.merge_topk(dev(ks, idx), dev(ks, sc), 32)
    for r in range(2):
        live = idx[r] >= 0
        order = np.lexsort((idx[r][live], -sc[r][live]))[:32]
        assert np.array_equal(gi[r].cpu().numpy(), idx[r][live][order])
        assert np.array_equal(gs[r].cpu().numpy(), sc[r][live][order])
    few = ctx.merge_topk(dev(ks, idx[:, :7]), dev(ks, sc[:, :7]), 10)[0].cpu().numpy()
    assert np.all(few[:, 6:] == -1)


def test_select_memo_table_in_batches(ks, ctx):
    """The per-(problem, class) table holds 256 MiB of records; a batch of more problems than that
    is served in several launches that reuse it (here 80-byte records: 409 problems at a time)."""
    w = wl.make_workload(1, P=900, C=300, law="pernode")
    model = ctx.model_create_gbdt(*w.gbdt)
    n0 = ctx.launch_count()
    idx, sc = run_select(ks, ctx, w, model)
    # mask, candidate rows, compaction, the key kernel of the catalogue's similarity order (the sort
    # runs the library's kernels, not counted), 3 x (table, walk), merge
    assert ctx.launch_count() - n0 == 2 + 1 + 1 + 3 * 2 + 1
    check_select(w, idx, sc, TOL_GBDT, sample=list(range(0, 900, 37)) + [408, 409, 817, 818, 899])


def test_select_pair_row_memo_paths(ks, ctx):
    """Batches of 32 problems or more copy the per-pair tile rows from a per-(problem, class)
    table, a class being (T_M, T_N, T_K, S, c_M, c_N, resident blocks). Cases: mixed element
    types (one class table per combination), candidates whose fields do not fit the class key
    (evaluated directly), more classes than the table holds (the late ones evaluated directly),
    and segments."""
    # mixed element types, dense, a few candidates outside the key's range
    w = wl.make_workload(2, P=40, seg=64, trees=30, depth=6)
    cand = w.candidates[:2500].copy()
    cand["tile_m"][::97] = 4096 + 64
    cand["tile_k"][5::211] = 8192
    w = wl.Workload("memo_mixed", DESC, w.problems, cand, 10, gbdt=w.gbdt)
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)
    # more distinct classes than slots: 12,000 different tile shapes
    i = np.arange(12000)
    big = np.zeros(12000, wl.CANDIDATE_DT)
    big["tile_m"], big["tile_n"], big["tile_k"] = 16 * (1 + i % 16), 8 * (1 + (i // 16) % 32), 16 * (1 + (i // 512) % 32)
    big["instr_n"], big["instr_m"], big["instr_k"] = big["tile_n"], 64, 16
    big["stages"], big["cluster_m"], big["cluster_n"] = 2 + i % 3, 1 + (i // 7) % 2, 1
    big["kernel_sched"], big["epi_sched"], big["tile_sched"] = i % 4, i % 3, i % 2
    assert len(np.unique(big[["tile_m", "tile_n", "tile_k", "stages", "cluster_m"]])) > 8192
    w1 = wl.make_workload(1, P=33, C=10, trees=12, depth=5)
    wb = wl.Workload("memo_overflow", DESC, w1.problems, big, 10, gbdt=w1.gbdt)
    model = ctx.model_create_gbdt(*w1.gbdt)
    idx, sc = run_select(ks, ctx, wb, model)
    check_select(wb, idx, sc, TOL_GBDT)
    # segments over the pool
    ws = wl.make_workload(2, P=48, seg=700, trees=20, depth=5)
    model = ctx.model_create_gbdt(*ws.gbdt)
    idx, sc = run_select(ks, ctx, ws, model)
    check_select(ws, idx, sc, TOL_GBDT)


def test_select_ridge_and_paper_sized_models(ks, ctx):
    """The linear (ridge) scorer as a one-layer model, and models of the sizes the paper ships:
    916 trees of depth 7, and the largest MLP preset 64-1024-1024-512-256-1."""
    st = wl.feature_stats("cfg1")
    prob, cand, _, _ = wl.make_inputs(1, P=3, C=900)
    ridge = wl.mlp_xavier(21, [64, 1], st["mu"], st["sigma"])
    w = wl.Workload("ridge", DESC, prob, cand, 10, mlp=ridge)
    rmodel = ctx.model_create_mlp(ridge)
    idx, sc = run_select(ks, ctx, w, rmodel)
    check_select(w, idx, sc, TOL_MLP)
    # the fused linear kernel evaluates exact features: only the order of the sum differs
    ridx, rsc = oracle.select(prob, cand, DESC, 10, mlp=ridge)
    assert np.array_equal(idx, ridx) and np.all(np.abs(sc - rsc) <= 1e-4 * np.maximum(1, np.abs(rsc)))
    hi, hs = ctx.select_one(prob[1:2], dev(ks, cand), len(cand), rmodel, 10)
    assert np.array_equal(hi.numpy(), ridx[1])
    hi, hs = ctx.select_host(prob, 3, cand, len(cand), rmodel, 10)
    assert np.array_equal(hi.numpy(), ridx)
    # mixed element types and per-problem segments, ordinal and one-hot form
    w2 = wl.make_workload(2, P=9, seg=2500, trees=4, depth=2)
    for form in (64, 80):
        mu, sg = (st["mu"], st["sigma"]) if form == 64 else wl.onehot_stats(st["mu"], st["sigma"])
        r2 = wl.mlp_xavier(5, [form, 1], mu, sg)
        wr = wl.Workload("ridge_seg", DESC, w2.problems, w2.candidates, 10, seg_offsets=w2.seg_offsets,
                         seg_index=w2.seg_index, mlp=r2)
        idx2, sc2 = run_select(ks, ctx, wr, ctx.model_create_mlp(r2))
        check_select(wr, idx2, sc2, 1e-4)
    big = wl.mlp_xavier(22, [64, 1024, 1024, 512, 256, 1], st["mu"], st["sigma"])
    w = wl.Workload("mlp_big", DESC, prob[:1], cand[:200], 10, mlp=big)
    idx, sc = run_select(ks, ctx, w, ctx.model_create_mlp(big))
    check_select(w, idx, sc, TOL_MLP)
    off, nodes = wl.gbdt_complete(wl.BASE_SEED + 9, 916, 7, st, 0.1)
    w = wl.Workload("gbdt_916x7", DESC, prob, cand, 10, gbdt=(off, nodes, 0.0))
    idx, sc = run_select(ks, ctx, w, ctx.model_create_gbdt(off, nodes, 0.0))
    check_select(w, idx, sc, TOL_GBDT)


# ---------------------------------------------------------------------------------------------
# the static sampling score as a scorer (no learned model)
# ---------------------------------------------------------------------------------------------

def test_select_static_score_bit_exact(ks, ctx):
    model = ctx.model_create_static()
    # every score: k >= C returns all of them
    for C in (1, 31, 32):
        prob, cand, _, _ = wl.make_inputs(3, P=7, C=C)
        idx, sc = ctx.select(dev(ks, prob), 7, dev(ks, cand), C, model, 32)
        torch.cuda.synchronize()
        idx, sc = idx.cpu().numpy(), sc.cpu().numpy()
        ridx, rsc = oracle.select(prob, cand, DESC, 32, static=True)
        assert np.array_equal(idx, ridx)
        assert np.array_equal(sc[:, :C].view(np.uint32), rsc[:, :C].view(np.uint32))
        assert np.all(idx[:, C:] == -1) and np.all(np.isneginf(sc[:, C:]))
    # dense batch over several blocks with a ragged tail; equal scores rank by index
    prob, cand, _, _ = wl.make_inputs(1, P=5, C=9001)
    idx, sc = ctx.select(dev(ks, prob), 5, dev(ks, cand), 9001, model, 20)
    torch.cuda.synchronize()
    ridx, rsc = oracle.select(prob, cand, DESC, 20, static=True)
    assert np.array_equal(idx.cpu().numpy(), ridx)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), rsc.view(np.uint32))
    # segments (cross-precision shape), empty segment included
    prob, cand, so, si = wl.make_inputs(2, P=6, seg=1500)
    so = so.copy()
    so[1:] -= so[1]
    so[0] = 0
    pairs = int(so[-1])
    si = si[len(si) - pairs:] if pairs < len(si) else si
    idx, sc = ctx.select(dev(ks, prob), 6, dev(ks, cand), len(cand), model, 10, dev(ks, so), dev(ks, si), pairs)
    torch.cuda.synchronize()
    ridx, rsc = oracle.select(prob, cand, DESC, 10, static=True, seg_off=so, seg_idx=si)
    assert np.array_equal(idx.cpu().numpy(), ridx)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), rsc.view(np.uint32))
    assert np.all(ridx[0] == -1)
    # the single-problem and host-buffer forms
    prob, cand, _, _ = wl.make_inputs(3, P=3, C=5000)
    d_c = dev(ks, cand)
    ridx, rsc = oracle.select(prob, cand, DESC, 10, static=True)
    for i in range(3):
        hi, hs = ctx.select_one(prob[i:i + 1], d_c, 5000, model, 10)
        assert np.array_equal(hi.numpy(), ridx[i]) and np.array_equal(hs.numpy(), rsc[i])
    hi, hs = ctx.select_host(prob, 3, cand, 5000, model, 10)
    assert np.array_equal(hi.numpy(), ridx) and np.array_equal(hs.numpy(), rsc)
    # extreme dimensions
    prob = np.concatenate([problem(1, 1, 1), problem(1 << 19, 1 << 19, 1 << 19), problem(524287, 3, 5)])
    cand = np.concatenate([candidate(64, 8, 16, 1), candidate(256, 256, 256, 12, 4, 4), candidate(128, 64, 32, 3, 2, 1)])
    idx, sc = ctx.select(dev(ks, prob), 3, dev(ks, cand), 3, model, 3)
    torch.cuda.synchronize()
    ridx, rsc = oracle.select(prob, cand, DESC, 3, static=True)
    assert np.array_equal(idx.cpu().numpy(), ridx)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), rsc.view(np.uint32))
    # the score is a function of (p, c), not of a feature row
    x = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(ks.KsError) as ei:
        ctx.score(x, model)
    assert ei.value.status == ks.KS_ERR_UNSUPPORTED


# ---------------------------------------------------------------------------------------------
# partition splits on categorical fields (general tree kernel)
# ---------------------------------------------------------------------------------------------

def test_partition_split_ensembles(ks, ctx):
    # leaf indices and scores of the standalone scorer
    prob, cand, so, si = wl.make_inputs(2, P=5, seg=700)
    x = oracle.featurize(prob, cand, DESC, so, si)
    off, nodes = wl.gbdt_complete(23, 64, 6, wl.feature_stats("cfg2"), 0.1)
    pnodes = wl.with_partition_splits(9, nodes)
    assert pnodes["kind"].sum() > 100
    model = ctx.model_create_gbdt(off, pnodes, 0.5)
    sc, leaf = ctx.score(dev(ks, x), model, want_leaf_idx=True)
    torch.cuda.synchronize()
    rs, rleaf = oracle.score_gbdt(x, off, pnodes, 0.5, want_leaf_idx=True)
    assert np.array_equal(leaf.cpu().numpy(), rleaf)
    assert np.all(np.abs(sc.cpu().numpy() - rs) <= TOL_GBDT * np.maximum(1, np.abs(rs)))
    # the partitions matter: the same trees with numeric splits score differently
    assert not np.array_equal(oracle.score_gbdt(x, off, nodes, 0.5), rs)
    # the fused path, dense and segmented, against the oracle
    w = wl.Workload("partition", DESC, prob, cand, 10, gbdt=(off, pnodes, 0.5), seg_offsets=so, seg_index=si)
    idx, sc = run_select(ks, ctx, w, model)
    check_select(w, idx, sc, TOL_GBDT)
    w2 = wl.make_workload(1, P=3, C=3000, trees=40)
    pn2 = wl.with_partition_splits(4, w2.gbdt[1])
    w2.gbdt = (w2.gbdt[0], pn2, w2.gbdt[2])
    m2 = ctx.model_create_gbdt(*w2.gbdt)
    idx, sc = run_select(ks, ctx, w2, m2)
    check_select(w2, idx, sc, TOL_GBDT)
    hi, hs = ctx.select_one(w2.problems[:1], dev(ks, w2.candidates), len(w2.candidates), m2, w2.k)
    assert np.array_equal(hi.numpy(), idx[0])
    # every subset of the levels of a four-level field, the full set included, as the root of a
    # depth-2 tree (quantised kernel: rank rows, exchanged children, always-right)
    for mask in range(1, 16):
        nd = np.zeros(7, wl.NODE_DT)
        nd[0] = (np.array([mask], np.uint32).view(np.float32)[0], 17, 1, 1)
        nd[1] = (np.array([1], np.uint32).view(np.float32)[0], 19, 1, 3)
        nd[2] = (3.5, 10, 0, 5)
        for j, v in enumerate((0.25, -0.5, 1.0, -2.0)):
            nd[3 + j] = (v, 0xFFFF, 0, 0)
        w3 = wl.Workload("subset", DESC, w2.problems, w2.candidates[:2500], 10, gbdt=(np.array([0, 7]), nd, 0.0))
        idx, sc = run_select(ks, ctx, w3, ctx.model_create_gbdt(*w3.gbdt))
        check_select(w3, idx, sc, TOL_GBDT)
        _, rsc = oracle.select(w3.problems, w3.candidates, DESC, 10, gbdt=w3.gbdt)
        assert np.array_equal(sc, rsc), mask
    # an ensemble too deep for the quantised kernel keeps its partition splits on the general one
    off5, n5 = wl.gbdt_complete(31, 6, 11, wl.feature_stats("cfg1"), 0.1)
    p5 = wl.with_partition_splits(2, n5)
    w5 = wl.Workload("deep", DESC, w2.problems, w2.candidates[:1200], 10, gbdt=(off5, p5, 0.0))
    idx, sc = run_select(ks, ctx, w5, ctx.model_create_gbdt(*w5.gbdt))
    check_select(w5, idx, sc, TOL_GBDT)
    # validation: partition splits only on level-code columns, with a mask inside the levels
    def one(feat, mask, kind=1):
        nd = np.zeros(3, wl.NODE_DT)
        nd[0] = (np.array([mask], np.uint32).view(np.float32)[0], feat, kind, 1)
        nd[1] = (0.5, 0xFFFF, 0, 0)
        nd[2] = (-0.5, 0xFFFF, 0, 0)
        return np.array([0, 3]), nd
    ctx.model_create_gbdt(*one(17, 0b1010), 0.0)
    for feat, mask, kind in ((17, 0, 1), (17, 0b10000, 1), (19, 0b100, 1), (10, 1, 1), (17, 1, 2)):
        with pytest.raises(ks.KsError) as ei:
            ctx.model_create_gbdt(*one(feat, mask, kind), 0.0)
        assert ei.value.status == ks.KS_ERR_INVALID_ARG


# ---------------------------------------------------------------------------------------------
# one-hot input form of the ranker
# ---------------------------------------------------------------------------------------------

def test_onehot_mlp(ks, ctx):
    st = wl.feature_stats("cfg1")
    mu, sg = wl.onehot_stats(st["mu"], st["sigma"])
    prob, cand, _, _ = wl.make_inputs(1, P=4, C=900)
    x = oracle.featurize(prob, cand, DESC)
    for widths in ([80, 128, 64, 1], [80, 1], [80, 256, 256, 1]):
        mlp = wl.mlp_xavier(13, widths, mu, sg)
        model = ctx.model_create_mlp(mlp)
        sc = ctx.score(dev(ks, x), model)
        torch.cuda.synchronize()
        rs = oracle.score_mlp(x, mlp)
        assert np.all(np.abs(sc.cpu().numpy() - rs) <= 5e-3 * np.maximum(1, np.abs(rs))), widths
        w = wl.Workload("onehot", DESC, prob, cand, 10, mlp=mlp)
        idx, s2 = run_select(ks, ctx, w, model)
        check_select(w, idx, s2, TOL_MLP)
    # the 80-256-256-1 shape runs on the tensor-core kernel (problem-only inputs folded into a
    # per-CTA bias): every score, on problems of mixed element types and epilogues
    mlp = wl.mlp_xavier(17, [80, 256, 256, 1], mu, sg)
    model = ctx.model_create_mlp(mlp)
    prob2, cand2, _, _ = wl.make_inputs(2, P=12, seg=100)
    assert len(set(prob2["dtype_ab"].tolist())) > 1 and len(set((prob2["epi_flags"] >> 1).tolist())) > 1
    for C in (129, 4500):
        idx, s2 = ctx.select(dev(ks, prob2), 12, dev(ks, cand2[:C]), C, model, 32)
        torch.cuda.synchronize()
        idx, s2 = idx.cpu().numpy(), s2.cpu().numpy()
        _, _, allsc = oracle.select(prob2, cand2[:C], DESC, 32, mlp=mlp, want_scores=True)
        for i in range(12):
            ref = allsc[i * C:(i + 1) * C]
            assert len(set(idx[i].tolist())) == 32 and idx[i].min() >= 0 and idx[i].max() < C
            err = np.abs(s2[i] - ref[idx[i]]) / np.maximum(1, np.abs(ref[idx[i]]))
            assert err.max() < 5e-3, (C, i, err.max())
            ok, msg = topk_accept(idx[i], s2[i], ref, np.arange(C, dtype=np.int32), 32, TOL_MLP)
            assert ok, msg
    # the one-hot form reads its own positions: indicator weights change the score
    mlp = wl.mlp_xavier(13, [80, 1], mu, sg)
    base = oracle.score_mlp(x, mlp)
    w2 = {k: (v.copy() if isinstance(v, np.ndarray) else [a.copy() for a in v]) for k, v in mlp.items()}
    w2["weights"][0][0, 66:70] = wl.float_to_bf16_bits(np.array([1.0, -1.0, 0.5, -0.5], np.float32))
    m2 = ctx.model_create_mlp(w2)
    got = ctx.score(dev(ks, x), m2).cpu().numpy()
    ref = oracle.score_mlp(x, w2)
    assert np.all(np.abs(got - ref) <= 5e-3 * np.maximum(1, np.abs(ref))) and not np.allclose(ref, base)
    # invalid: another input width, or constants shorter than the width
    bad = dict(mlp)
    bad["widths"] = np.array([72, 1], np.int32)
    bad["weights"] = [mlp["weights"][0][:, :72].copy()]
    with pytest.raises(ks.KsError):
        ctx.model_create_mlp(bad)
