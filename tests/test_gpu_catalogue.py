"""Parity of the on-device search-space enumerator and validity filter (through the C ABI) with
the CPU oracle: records, positions and counts bit-exact; then the composition with the
selection path (filter -> select on the compacted catalogue -> positions mapped back)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import problem

pytestmark = pytest.mark.gpu

DESC = wl.gpu_desc()
DT = wl.CANDIDATE_DT
SIZE = 534600


@pytest.fixture(scope="module")
def ks():
    from paper_2609_35587_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(ks):
    c = ks.Context(DESC, 0)
    yield c
    c.close()


def records(t, n=None):
    a = t.cpu().numpy()
    a = a if n is None else a[:n]
    return np.ascontiguousarray(a).view(DT).reshape(-1)


def test_enumerate_whole_space_and_windows(ks, ctx):
    assert ks.KS_CATALOGUE_SIZE == oracle.catalogue_size() == SIZE
    got = records(ctx.enumerate(0, SIZE))
    assert got.tobytes() == oracle.enumerate_candidates(0, SIZE, DT).tobytes()
    for first, count in ((0, 1), (SIZE - 1, 1), (226262, 1), (12345, 1000), (SIZE - 777, 777), (5, 0)):
        got = records(ctx.enumerate(first, count))
        assert got.tobytes() == oracle.enumerate_candidates(first, count, DT).tobytes()
    for first, count in ((-1, 1), (0, SIZE + 1), (SIZE, 1), (1, -1)):
        with pytest.raises(ks.KsError) as ei:
            ctx.enumerate(first, count)
        assert ei.value.status == ks.KS_ERR_INVALID_ARG


@pytest.mark.parametrize("flags", [0, 1, 2, 3, 5, 7])
def test_valid_catalogue_of_the_search_space(ks, ctx, flags):
    cases = [problem(4096, 4096, 4096, lay, 1, 1) for lay in range(4)]
    cases += [problem(64, 64, 64, 0, 1, 1), problem(32, 128, 4096, 3, 1, 1),
              problem(4096, 4096, 4096, 2, 2, 1), problem(1000, 70, 512, 1, 3, 3), problem(1, 1, 1, 3, 0, 0)]
    for p in cases:
        out, idx, n = ctx.valid_catalogue(p, flags)
        rc, ri = oracle.valid_catalogue(p, DESC, flags, dtype=DT)
        assert n == len(rc), (p, n, len(rc))
        assert np.array_equal(idx.cpu().numpy()[:n], ri)
        assert records(out, n).tobytes() == rc.tobytes()


def test_valid_catalogue_counts_match_the_papers_layout_differences(ks, ctx):
    n = [ctx.valid_catalogue(problem(2048, 2048, 2048, lay, 1, 1), ks.KS_VALID_COUPLED,
                             want_records=False, want_index=False)[2] for lay in range(4)]
    assert n[0] - n[1] == 55 and n[1] == n[2] and n[0] - n[3] == 99
    assert all(abs(v - want) <= 0.01 * want for v, want in zip(n, (60795, 60740, 60740, 60696)))


def test_valid_catalogue_of_explicit_lists(ks, ctx):
    dev = torch.device("cuda", 0)
    _, cand, _, _ = wl.make_inputs(1)          # 60,000 records, includes a fourth kernel schedule
    space = oracle.enumerate_candidates(0, SIZE, DT)
    big = np.concatenate([space, space[::-1], cand, space[:150000]])   # > 1,024 blocks of 1,024
    p = problem(512, 8192, 1024, 3, 1, 1)
    for lst in (cand, cand[:1], cand[:1023], cand[:1025], cand[:0], big):
        d_c = ks.to_device(lst, dev) if len(lst) else torch.empty((0, 16), dtype=torch.uint8, device=dev)
        out, idx, n = ctx.valid_catalogue(p, 3, d_c)
        rc, ri = oracle.valid_catalogue(p, DESC, 3, candidates=lst)
        assert n == len(rc)
        assert np.array_equal(idx.cpu().numpy()[:n], ri)
        assert records(out, n).tobytes() == rc.tobytes()
    # asynchronous form: the count stays on the device
    d_c = ks.to_device(cand, dev)
    out, idx, d_n = ctx.valid_catalogue(p, 1, d_c, sync=False)
    torch.cuda.synchronize()
    rc, ri = oracle.valid_catalogue(p, DESC, 1, candidates=cand)
    assert int(d_n.item()) == len(rc) and np.array_equal(idx.cpu().numpy()[:len(rc)], ri)
    # twice in a row: same answer (scratch is rebuilt every call)
    out2, idx2, n2 = ctx.valid_catalogue(p, 1, d_c)
    assert n2 == len(rc) and torch.equal(idx2[:n2], idx[:n2])


def test_valid_catalogue_rejects_bad_arguments(ks, ctx):
    p = problem(64, 64, 64, 0, 1, 1)
    with pytest.raises(ks.KsError) as ei:
        ctx.valid_catalogue(p, 8)
    assert ei.value.status == ks.KS_ERR_INVALID_ARG
    with pytest.raises(ks.KsError):
        ctx.valid_catalogue(p, 1, None, C=SIZE + 1)
    with pytest.raises(ks.KsError):
        ctx.valid_catalogue(problem(64, 64, 64, 4, 1, 1), 1)
    buf = torch.zeros(16 * 9 + 8, dtype=torch.uint8, device="cuda")
    with pytest.raises(ks.KsError):
        ctx.valid_catalogue(p, 1, buf[8:8 + 16 * 8].view(8, 16))   # misaligned records


def test_filter_then_select_then_remap(ks, ctx):
    """The valid catalogue of one layout ranked for several problems of that layout: equal to
    the oracle ranking the same problems over the valid ids as segments."""
    dev = torch.device("cuda", 0)
    lay = 2
    prob = np.concatenate([problem(m, n, k, lay, 1, 1) for m, n, k in
                           ((4096, 4096, 4096), (32, 128, 4096), (12288, 128, 4096), (777, 3001, 129))])
    out, idx, n = ctx.valid_catalogue(prob[:1], ks.KS_VALID_COUPLED)
    space = oracle.enumerate_candidates(0, SIZE, DT)
    _, ri = oracle.valid_catalogue(prob[:1], DESC, 1, dtype=DT)
    so = np.arange(len(prob) + 1, dtype=np.int64) * len(ri)
    si = np.tile(ri, len(prob))
    k = 16
    # static sampling score: bit-exact scores, so the lists are simply equal
    model = ctx.model_create_static()
    tidx, tsc = ctx.select(ks.to_device(prob, dev), len(prob), out[:n], n, model, k)
    ctx.remap_indices(tidx, idx, n)
    torch.cuda.synchronize()
    ridx, rsc = oracle.select(prob, space, DESC, k, static=True, seg_off=so, seg_idx=si)
    assert np.array_equal(tidx.cpu().numpy(), ridx)
    assert np.array_equal(tsc.cpu().numpy().view(np.uint32), rsc.view(np.uint32))
    # tree ensemble on the same compacted catalogue
    w = wl.make_workload(1, P=1, C=16, trees=40)
    gm = ctx.model_create_gbdt(*w.gbdt)
    tidx, tsc = ctx.select(ks.to_device(prob, dev), len(prob), out[:n], n, gm, k)
    ctx.remap_indices(tidx, idx, n)
    torch.cuda.synchronize()
    ridx, rsc = oracle.select(prob, space, DESC, k, gbdt=w.gbdt, seg_off=so, seg_idx=si)
    tidx, tsc = tidx.cpu().numpy(), tsc.cpu().numpy()
    assert np.all(np.abs(tsc - rsc) <= 1e-5 * np.maximum(1, np.abs(rsc)))
    same = tidx == ridx
    # positions may differ only inside groups of (near-)equal scores
    assert np.all(same | (np.abs(tsc - rsc) <= 1e-5 * np.maximum(1, np.abs(rsc))))
    assert same.mean() > 0.9
    # remap leaves padding alone and rejects out-of-range positions
    t = torch.tensor([0, -1, 5, 10**6], dtype=torch.int32, device=dev)
    m = torch.arange(100, 110, dtype=torch.int32, device=dev)
    ctx.remap_indices(t, m)
    assert t.cpu().tolist() == [100, -1, 105, -1]
