"""Full-size parity: the benchmark's workloads in the launch configuration bench.py times,
checked on sampled problems the oracle can rank one by one, plus properties that hold for
every problem."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import topk_accept

pytestmark = pytest.mark.gpu

TOL_GBDT, TOL_MLP = 1e-5, 2e-2


@pytest.fixture(scope="module")
def ks():
    from paper_2609_35587_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(ks):
    c = ks.Context(wl.gpu_desc(), 0)
    yield c
    c.close()


def run_full(ks, ctx, w, model):
    dev = torch.device("cuda", 0)
    P, C = len(w.problems), len(w.candidates)
    d_so = None if w.seg_offsets is None else ks.to_device(w.seg_offsets, dev)
    d_si = None if w.seg_index is None else ks.to_device(w.seg_index, dev)
    idx, sc = ctx.select(ks.to_device(w.problems, dev), P, ks.to_device(w.candidates, dev), C, model, w.k,
                         d_so, d_si, w.pairs)
    torch.cuda.synchronize()
    assert ctx.device_status() == ks.KS_OK
    return idx.cpu().numpy(), sc.cpu().numpy()


def check_properties(w, idx, sc):
    P = len(w.problems)
    assert idx.shape == (P, w.k) and np.all(np.isfinite(sc))
    assert np.all(np.diff(sc, axis=1) <= 0), "scores must be non-increasing along k"
    srt = np.sort(idx, axis=1)
    assert np.all(np.diff(srt, axis=1) > 0), "indices of a problem must be distinct"
    if w.seg_offsets is None:
        assert idx.min() >= 0 and idx.max() < len(w.candidates)
    else:
        for i in range(0, P, max(1, P // 64)):
            seg = w.seg_index[w.seg_offsets[i]:w.seg_offsets[i + 1]]
            assert np.all(np.isin(idx[i], seg))


def check_sampled(w, idx, sc, sample, tol):
    for i in sample:
        p1 = w.problems[i:i + 1]
        if w.seg_offsets is None:
            pool = np.arange(len(w.candidates), dtype=np.int32)
            _, _, allsc = oracle.select(p1, w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp, want_scores=True)
        else:
            pool = w.seg_index[w.seg_offsets[i]:w.seg_offsets[i + 1]]
            _, _, allsc = oracle.select(p1, w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp,
                                        seg_off=np.array([0, len(pool)], np.int64), seg_idx=pool,
                                        want_scores=True)
        ok, msg = topk_accept(idx[i], sc[i], allsc, pool, w.k, tol)
        assert ok, f"problem {i}: {msg}"


def test_config1_full_space(ks, ctx):
    w = wl.make_workload(1)
    assert w.pairs == 61_440_000
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_full(ks, ctx, w, model)
    check_properties(w, idx, sc)
    sample = wl.randint(7, 1, np.arange(12), len(w.problems))
    check_sampled(w, idx, sc, [0, len(w.problems) - 1] + sample.tolist(), TOL_GBDT)
    idx2, sc2 = run_full(ks, ctx, w, model)
    assert np.array_equal(idx, idx2) and np.array_equal(sc.view(np.uint32), sc2.view(np.uint32))


def test_config2_cross_precision(ks, ctx):
    w = wl.make_workload(2)
    assert w.pairs == 67_108_864
    model = ctx.model_create_gbdt(*w.gbdt)
    idx, sc = run_full(ks, ctx, w, model)
    check_properties(w, idx, sc)
    sample = wl.randint(7, 2, np.arange(10), len(w.problems))
    check_sampled(w, idx, sc, [0, len(w.problems) - 1] + sample.tolist(), TOL_GBDT)


def test_config4_neural_ranker(ks, ctx):
    w = wl.make_workload(4)
    assert w.pairs == 61_440_000
    model = ctx.model_create_mlp(w.mlp)
    idx, sc = run_full(ks, ctx, w, model)
    check_properties(w, idx, sc)
    check_sampled(w, idx, sc, [0, 517, len(w.problems) - 1], TOL_MLP)
    idx2, sc2 = run_full(ks, ctx, w, model)
    assert np.array_equal(idx, idx2) and np.array_equal(sc.view(np.uint32), sc2.view(np.uint32))


def test_config3_latency_stream_sample(ks, ctx):
    """Calls drawn from the 100,000-call stream (first, last and a few in between)."""
    w = wl.make_workload(3, P=100_000)
    model = ctx.model_create_gbdt(*w.gbdt)
    dev = torch.device("cuda", 0)
    d_c = ks.to_device(w.candidates, dev)
    C = len(w.candidates)
    for i in [0, 1, 49_999, 77_777, 99_999]:
        hi, hs = ctx.select_one(w.problems[i:i + 1], d_c, C, model, w.k)
        _, _, allsc = oracle.select(w.problems[i:i + 1], w.candidates, w.desc, w.k, gbdt=w.gbdt, want_scores=True)
        ok, msg = topk_accept(hi.numpy(), hs.numpy(), allsc, np.arange(C, dtype=np.int32), w.k, TOL_GBDT)
        assert ok, f"call {i}: {msg}"
    # the prepared caller (the form bench.py times) is the same call
    call = ctx.select_one_caller(d_c, C, model, w.k)
    structs = ks.problem_structs(w.problems[:300])
    for i in [0, 7, 299]:
        hi, hs = ctx.select_one(w.problems[i:i + 1], d_c, C, model, w.k)
        ci, cs = call(structs[i])
        assert np.array_equal(ci.numpy(), hi.numpy()) and np.array_equal(cs.numpy(), hs.numpy())


def test_full_size_paper_forms(ks, ctx):
    """The paper's own model forms at config-1 / config-4 size: partition splits on the
    categorical fields, the one-hot ranker input, and the linear ridge scorer."""
    w = wl.make_workload(1)
    w.gbdt = (w.gbdt[0], wl.with_partition_splits(3, w.gbdt[1]), w.gbdt[2])
    idx, sc = run_full(ks, ctx, w, ctx.model_create_gbdt(*w.gbdt))
    check_properties(w, idx, sc)
    check_sampled(w, idx, sc, [0, 333, len(w.problems) - 1], TOL_GBDT)
    st = wl.feature_stats("cfg1")
    mu, sg = wl.onehot_stats(st["mu"], st["sigma"])
    w4 = wl.make_workload(4)
    w4.mlp = wl.mlp_xavier(31, [80, 256, 256, 1], mu, sg)
    idx, sc = run_full(ks, ctx, w4, ctx.model_create_mlp(w4.mlp))
    check_properties(w4, idx, sc)
    check_sampled(w4, idx, sc, [0, 700], TOL_MLP)
    w4.mlp = wl.mlp_xavier(32, [64, 1], st["mu"], st["sigma"])
    idx, sc = run_full(ks, ctx, w4, ctx.model_create_mlp(w4.mlp))
    check_properties(w4, idx, sc)
    check_sampled(w4, idx, sc, [0, 511, len(w4.problems) - 1], 1e-4)


def test_score_rows_in_batches(ks, ctx):
    """ks_score on the quantised path takes 4,096 blocks of 1,024 rows per batch: more rows than
    one batch, with a ragged last block."""
    w = wl.make_workload(1, P=4, C=4000, trees=6, depth=5)
    x = oracle.featurize(w.problems, w.candidates, w.desc)
    rows = 4096 * 1024 + 777
    x = np.ascontiguousarray(np.resize(x, (rows, x.shape[1])))
    x[-1, 3] = np.nan
    rs = oracle.score_gbdt(x, *w.gbdt)
    model = ctx.model_create_gbdt(*w.gbdt)
    n0 = ctx.launch_count()
    s = ctx.score(ks.to_device(x, torch.device("cuda", 0)), model).cpu().numpy()
    assert ctx.launch_count() - n0 == 4
    assert np.all(np.abs(s - rs) <= TOL_GBDT * np.maximum(1, np.abs(rs)))
