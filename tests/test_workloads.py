"""The seeded generators: shapes, domains, determinism, and checksums that catch drift."""
import zlib

import numpy as np

from paper_2609_35587_b200 import workloads as wl


def crc(a):
    return zlib.crc32(np.ascontiguousarray(a).tobytes())


def test_counter_based_generator_is_order_independent():
    a = wl.uniform(7, 3, np.arange(1000))
    b = np.concatenate([wl.uniform(7, 3, np.arange(500, 1000)), wl.uniform(7, 3, np.arange(500))])
    assert np.array_equal(a, np.concatenate([b[500:], b[:500]]))
    assert 0.45 < a.mean() < 0.55 and a.min() >= 0 and a.max() < 1
    n = wl.normal(7, 4, 5, np.arange(20000))
    assert abs(n.mean()) < 0.03 and 0.97 < n.std() < 1.03


def test_config0_inputs():
    prob, cand, so, si = wl.make_inputs(0)
    assert prob.shape == (64,) and cand.shape == (2048,) and so is None
    for d in ("m", "n", "k"):
        assert np.all(prob[d] % 16 == 0) and prob[d].min() >= 64 and prob[d].max() <= 8192
    assert set(np.unique(prob["layout"])) <= {0, 2}
    assert set(np.unique(cand["tile_m"])) == {64, 128, 256}
    assert set(np.unique(cand["stages"])) == set(range(2, 8))
    assert len(np.unique(cand.view("V16"))) == 2048
    assert len(wl.candidates_small_grid(1, None)) == 5184


def test_config1_catalogue_is_the_unfiltered_cross_product():
    full = wl.candidates_full_grid(wl.BASE_SEED + 1000, None)
    assert len(full) == 62208 and len(np.unique(full.view("V16"))) == 62208
    assert set(np.unique(full["tile_m"])) == {64, 128, 192, 256}
    assert set(np.unique(full["epi_sched"])) == {0, 1, 2}
    _, cand, _, _ = wl.make_inputs(1, P=4)
    assert len(cand) == 60000 and np.array_equal(cand, full[:60000])
    _, c3, _, _ = wl.make_inputs(3, P=4)
    _, c4, _, _ = wl.make_inputs(4, P=4)
    assert np.array_equal(c3, cand) and np.array_equal(c4, cand)


def test_config2_segments():
    prob, cand, so, si = wl.make_inputs(2, P=16, seg=1024)
    assert len(cand) == 62208 and so.tolist() == list(range(0, 16 * 1024 + 1, 1024))
    seg = si.reshape(16, 1024)
    assert np.all(np.diff(seg, axis=1) > 0) and seg.min() >= 0 and seg.max() < 62208
    assert len({tuple(r[:8]) for r in seg}) == 16
    assert set(np.unique(prob["dtype_ab"])) <= {0, 1, 2, 3}
    assert np.all(prob["dtype_d"][prob["dtype_ab"] == 2] == 1)
    assert np.all(prob["dtype_d"][prob["dtype_ab"] == 3] == 3)


def test_config3_stream():
    prob, _, _, _ = wl.make_inputs(3, P=4000, C=8)
    assert prob["m"].min() >= 1 and prob["n"].max() <= 16384
    assert 0.4 < np.mean(prob["m"] <= 64) < 0.75


def test_models():
    w = wl.make_workload(0, P=2, C=8)
    off, nodes, base = w.gbdt
    assert len(off) == 101 and len(nodes) == 100 * 127 and base == 0.0
    t = nodes[:127]
    assert np.all(t["feat"][:63] < 63) and np.all(t["feat"][63:] == 0xFFFF)
    assert np.array_equal(t["left"][:63], 2 * np.arange(63) + 1)
    leaves = nodes["v"][nodes["feat"] == 0xFFFF]
    assert 0.09 < leaves.std() < 0.11
    w3 = wl.make_workload(3, P=2, C=8)
    w1 = wl.make_workload(1, P=2, C=8)
    assert np.array_equal(w3.gbdt[1], w1.gbdt[1]) and len(w1.gbdt[0]) == 501
    m = wl.make_workload(4, P=2, C=8).mlp
    assert [x.shape for x in m["weights"]] == [(256, 64), (256, 256), (1, 256)]
    w1f = (m["weights"][0].astype(np.uint32) << 16).view(np.float32)
    a = np.sqrt(6.0 / (64 + 256))
    assert np.abs(w1f).max() <= a * 1.01 and np.abs(w1f).max() > 0.9 * a
    assert np.all(m["sigma"] != 0) and m["mu"][63] == 0 and m["sigma"][63] == 1


def test_threshold_laws():
    """Distinct thresholds per column under the three laws (config 1's ensemble): a quantile per
    node gives a continuous column well over a thousand, 256 bins at most 255, the slot table at
    most 128; every threshold lies strictly between two sample values of its column or beside
    its only one."""
    st = wl.feature_stats("cfg1")
    most = {}
    for law in wl.LAWS:
        nodes = wl.make_workload(1, P=1, C=8, law=law).gbdt[1]
        it = nodes[nodes["feat"] != 0xFFFF]
        assert len(it) == 500 * 255
        most[law] = max(len(np.unique(it["v"][it["feat"] == f])) for f in range(63))
        for f in (0, 16, 39, 44):
            d = st["dval"][st["doff"][f]:st["doff"][f + 1]]
            t = np.unique(it["v"][it["feat"] == f])
            assert not np.isin(t, d).any() and t.min() > d[0] and (t.max() < d[-1] or len(d) == 1)
    assert most["pernode"] > 1000 and 128 < most["hist256"] <= 255 and most["slots128"] <= 128
    # the quantile of a node: q = 0.5 of a column with values {1, 2, 3, 4} x 16 is the midpoint 2.5
    toy = {"dval": np.tile(np.array([1, 2, 3, 4], np.float32), 63), "doff": np.arange(64) * 4,
           "dcum": np.tile(np.array([16, 32, 48, 64], np.int32), 63)}
    got = wl.quantile_thresholds(toy, np.array([0, 5, 62, 7]), np.array([0.5, 0.05, 0.94, 0.99]))
    assert got.tolist() == [2.5, 1.5, 3.5, 3.5]


def test_checksums():
    """Drift guard: any change to the generators or the stats table shows up here."""
    prob, cand, _, _ = wl.make_inputs(0)
    w = wl.make_workload(0)
    got = dict(prob0=crc(prob), cand0=crc(cand), nodes0=crc(w.gbdt[1]),
               nodes0_hist256=crc(wl.make_workload(0, law="hist256").gbdt[1]),
               nodes0_slots128=crc(wl.make_workload(0, law="slots128").gbdt[1]),
               cand1=crc(wl.make_inputs(1, P=1)[1]), prob1=crc(wl.make_inputs(1)[0]))
    want = CHECKSUMS
    assert got == want, got


CHECKSUMS = {'prob0': 783310851, 'cand0': 485305090, 'nodes0': 3578089389, 'nodes0_hist256': 2769579378,
             'nodes0_slots128': 3560579726, 'cand1': 3090539893, 'prob1': 1331788314}
