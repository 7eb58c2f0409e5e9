"""The failure path of the bounded device-side waits, exercised on a healthy GPU: a test hook makes
a wait run out (the tree kernel arms its chunk barriers for more bytes than the copies bring, the
tensor-core kernel never copies its weights), with a probe budget of about a millisecond. The
kernels must set the status word and return, the call must report KS_ERR_TIMEOUT, nothing may
fault, and the next ordinary call on the same context must give the oracle's result."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35587_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DESC = wl.gpu_desc()


@pytest.fixture()
def ks():
    from paper_2609_35587_b200 import binding
    return binding


def dev(ks, a):
    return ks.to_device(a, torch.device("cuda", 0))


def assert_matches_oracle(w, idx, sc, tol):
    ridx, rsc = oracle.select(w.problems, w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp)
    if w.gbdt is not None:
        assert np.array_equal(idx, ridx)
    assert np.all(np.abs(sc - rsc) <= tol * np.maximum(1, np.abs(rsc)))


@pytest.mark.parametrize("law", ["slots128", "pernode"])
def test_tree_kernel_wait_runs_out(ks, law):
    ctx = ks.Context(DESC, 0)
    w = wl.make_workload(1, P=3, C=2500, trees=60, law=law)
    model = ctx.model_create_gbdt(*w.gbdt)
    assert "select_fast_kernel" in model.describe()
    d_p, d_c = dev(ks, w.problems), dev(ks, w.candidates)
    ctx.debug_set_wait(2000, True)
    # asynchronous batch call: the status word tells
    ctx.select(d_p, 3, d_c, 2500, model, w.k)
    assert ctx.device_status() == ks.KS_ERR_TIMEOUT
    assert ctx.device_status() == ks.KS_OK          # reported once, then cleared
    # host-buffer call and single-problem call (tree slices) report it themselves
    with pytest.raises(ks.KsError) as e:
        ctx.select_host(w.problems, 3, w.candidates, 2500, model, w.k)
    assert e.value.status == ks.KS_ERR_TIMEOUT
    with pytest.raises(ks.KsError) as e:
        ctx.select_one(w.problems[:1], d_c, 2500, model, w.k)
    assert e.value.status == ks.KS_ERR_TIMEOUT
    # scoring call on the same walk
    x = oracle.featurize(w.problems[:1], w.candidates, DESC)
    ctx.score(dev(ks, x), model)
    assert ctx.device_status() == ks.KS_ERR_TIMEOUT
    # back to normal: same context, same model
    ctx.debug_set_wait(0, False)
    idx, sc = ctx.select(d_p, 3, d_c, 2500, model, w.k)
    assert ctx.device_status() == ks.KS_OK
    assert_matches_oracle(w, idx.cpu().numpy(), sc.cpu().numpy(), 1e-5)
    hi, hs = ctx.select_one(w.problems[1:2], d_c, 2500, model, w.k)
    assert np.array_equal(hi.numpy(), idx[1].cpu().numpy())
    s = ctx.score(dev(ks, x), model).cpu().numpy()
    rs = oracle.score_gbdt(x, *w.gbdt)
    assert np.all(np.abs(s - rs) <= 1e-5 * np.maximum(1, np.abs(rs)))
    ctx.close()


def test_short_probe_budget_alone_does_not_fail(ks):
    """The budget used above (2,000 probes) is ample for a healthy copy: without the hook the same
    call succeeds."""
    ctx = ks.Context(DESC, 0)
    w = wl.make_workload(1, P=3, C=2500, trees=60)
    model = ctx.model_create_gbdt(*w.gbdt)
    ctx.debug_set_wait(2000, False)
    idx, sc = ctx.select(dev(ks, w.problems), 3, dev(ks, w.candidates), 2500, model, w.k)
    assert ctx.device_status() == ks.KS_OK
    assert_matches_oracle(w, idx.cpu().numpy(), sc.cpu().numpy(), 1e-5)
    ctx.close()


def test_tensor_core_kernel_wait_runs_out(ks):
    ctx = ks.Context(DESC, 0)
    w = wl.make_workload(4, P=2, C=1500)
    model = ctx.model_create_mlp(w.mlp)
    assert "select_mlp_tc_kernel" in model.describe()
    d_p, d_c = dev(ks, w.problems), dev(ks, w.candidates)
    ctx.debug_set_wait(64, True)
    ctx.select(d_p, 2, d_c, 1500, model, w.k)
    assert ctx.device_status() == ks.KS_ERR_TIMEOUT
    x = oracle.featurize(w.problems[:1], w.candidates, DESC)
    ctx.score(dev(ks, x), model)
    assert ctx.device_status() == ks.KS_ERR_TIMEOUT
    ctx.debug_set_wait(0, False)
    idx, sc = ctx.select(d_p, 2, d_c, 1500, model, w.k)
    assert ctx.device_status() == ks.KS_OK
    _, _, allsc = oracle.select(w.problems, w.candidates, DESC, w.k, mlp=w.mlp, want_scores=True)
    got_i, got_s = idx.cpu().numpy(), sc.cpu().numpy()
    for i in range(2):
        ref = allsc[i * 1500:(i + 1) * 1500]
        assert np.all(np.abs(got_s[i] - ref[got_i[i]]) <= 2e-2 * np.maximum(1, np.abs(ref[got_i[i]])))
    ctx.close()
