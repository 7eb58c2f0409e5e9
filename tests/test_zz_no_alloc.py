"""ks_select_trees_static, the entry point for callers that may not allocate device memory
(their pool owns the whole GPU, or a synchronising cudaMalloc is off-limits where they run):
its results must match the CPU oracle and the regular ks_select on the same inputs, on calls in
a row that share the library's fixed scratch array; a call must leave the device's free memory
as it found it (measured with cudaMemGetInfo, which sees every allocation on the device, not
only torch's); and oversize requests must be refused up front.

The file name sorts last on purpose, so that a run that stops at the first failure has
already run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import topk_accept

pytestmark = pytest.mark.gpu

TOL = 1e-5


def device_nodes(ks, nodes):
    """The ensemble as 8-byte device records (what a caller without ks_model would upload)."""
    nd = np.zeros(len(nodes), ks.NODE_DEV_DT)
    nd["v"] = nodes["v"]
    nd["feat"] = nodes["feat"]
    nd["left"] = np.where(nodes["feat"] == 0xFFFF, 0, nodes["left"]).astype(np.uint16)
    return nd


def run_case(ks, ctx, w):
    dev = torch.device("cuda", 0)
    P, C, k = len(w.problems), len(w.candidates), w.k
    off, nodes, base = w.gbdt
    d_p, d_c = ks.to_device(w.problems, dev), ks.to_device(w.candidates, dev)
    model = ctx.model_create_gbdt(off, nodes, base)
    ref_idx, ref_sc = ctx.select(d_p, P, d_c, C, model, k)
    torch.cuda.synchronize()
    ref_idx, ref_sc = ref_idx.cpu().numpy(), ref_sc.cpu().numpy()

    d_nodes = ks.to_device(device_nodes(ks, nodes), dev)
    d_off = torch.from_numpy(off.astype(np.int32)).to(dev)
    out_idx = torch.full((P, k), -7, dtype=torch.int32, device=dev)
    out_sc = torch.zeros((P, k), dtype=torch.float32, device=dev)
    call = lambda: ks.ks_select_trees_static(w.desc, d_p, P, d_c, C, d_nodes, d_off, len(off) - 1, base, k,
                                             out_idx, out_sc)
    assert call() == ks.KS_OK       # warm call: module and array are on the device after it
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    out_idx.fill_(-7)
    assert call() == ks.KS_OK
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
    got_idx, got_sc = out_idx.cpu().numpy(), out_sc.cpu().numpy()
    # checker: the CPU oracle (every problem, full acceptance rule)
    for i in range(P):
        _, _, allsc = oracle.select(w.problems[i:i + 1], w.candidates, w.desc, k, gbdt=w.gbdt, want_scores=True)
        ok, msg = topk_accept(got_idx[i], got_sc[i], allsc, np.arange(C, dtype=np.int32), k, TOL)
        assert ok, f"problem {i}: {msg}"
    # and the regular entry point
    assert np.array_equal(got_idx, ref_idx)
    assert np.all(np.abs(got_sc - ref_sc) <= TOL * np.maximum(1, np.abs(ref_sc)))


def test_static_scratch_select_matches_select_twice_in_a_row():
    from paper_2609_35587_b200 import binding as ks
    ctx = ks.Context(wl.gpu_desc(), 0)
    # first call: a few blocks per problem; second call: other sizes, so stale keys of the
    # first call sit in the shared array when the second one runs
    run_case(ks, ctx, wl.make_workload(0, P=9, C=1500, trees=40, depth=6))
    run_case(ks, ctx, wl.make_workload(1, P=3, C=700, trees=25, depth=5))
    run_case(ks, ctx, wl.make_workload(0, P=9, C=1500, trees=40, depth=6))
    ctx.close()


def test_static_scratch_refuses_oversize_and_bad_arguments():
    from paper_2609_35587_b200 import binding as ks
    dev = torch.device("cuda", 0)
    w = wl.make_workload(0, P=2, C=64, trees=3, depth=2)
    off, nodes, base = w.gbdt
    d_p, d_c = ks.to_device(w.problems, dev), ks.to_device(w.candidates, dev)
    d_nodes = ks.to_device(device_nodes(ks, nodes), dev)
    d_off = torch.from_numpy(off.astype(np.int32)).to(dev)
    out_idx = torch.zeros((2, 32), dtype=torch.int32, device=dev)
    out_sc = torch.zeros((2, 32), dtype=torch.float32, device=dev)
    args = (d_nodes, d_off, len(off) - 1, base)
    # 4096 problems x 240 blocks x 32 entries would need far more than the fixed array holds:
    # refused before any launch (the pointers are never dereferenced)
    assert ks.ks_select_trees_static(w.desc, d_p, 4096, d_c, 61440, *args, 32, out_idx, out_sc) == ks.KS_ERR_UNSUPPORTED
    assert ks.ks_select_trees_static(w.desc, d_p, 2, d_c, 64, *args, 0, out_idx, out_sc) == ks.KS_ERR_INVALID_ARG
    assert ks.ks_select_trees_static(w.desc, d_p, 2, d_c, 64, *args, 33, out_idx, out_sc) == ks.KS_ERR_INVALID_ARG
    assert ks.ks_select_trees_static(w.desc, None, 2, d_c, 64, *args, 5, out_idx, out_sc) == ks.KS_ERR_INVALID_ARG
    assert ks.ks_select_trees_static(w.desc, d_p, 0, d_c, 64, *args, 5, out_idx, out_sc) == ks.KS_OK
    torch.cuda.synchronize()
