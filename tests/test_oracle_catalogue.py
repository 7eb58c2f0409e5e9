"""Pins for the oracle's search-space enumerator (Table "Configuration knobs") and static validity
filter (Table "Static validity constraints"): the paper's 534,600 combinations per layout, the
knob value lists, a library enumeration of the same product, hand-decoded ids, hand-worked
capacity boundaries, and the paper's valid-catalogue counts per layout (Table "Held-out
evaluation shapes": 60,795 / 60,740 / 60,740 / 60,696 for TN / TT / NN / NT)."""
import itertools

import numpy as np

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import candidate, problem

DESC = wl.gpu_desc()
DT = wl.CANDIDATE_DT
TN_, TT_, NN_, NT_ = 0, 1, 2, 3
COUPLED = 1      # flag bit 0: epilogue <-> mainloop couplings
WASTEFUL = 2     # flag bit 1
PAPER_COUNTS = {TN_: 60795, TT_: 60740, NN_: 60740, NT_: 60696}


def whole_space():
    return oracle.enumerate_candidates(0, oracle.catalogue_size(), DT)


def bf16(layout=TN_, m=4096, n=4096, k=4096):
    return problem(m, n, k, layout, 1, 1)


def is_valid(p, c, flags=COUPLED):
    return len(oracle.valid_catalogue(p, DESC, flags, candidates=c)[0]) == len(c)


PRINTED = 4      # flag bit 2: the capacity rule exactly as the table prints it


def test_capacity_rule_as_printed_and_as_read():
    """bf16, tile 128 x 96 x 128, four stages: mainloop 4 * 128 * (128 + 96) * 2 = 229,376 B, TMA
    epilogue 2 * 64 * 32 * 2 = 8,192 B, reserve 2,048 B, capacity 232,448 B. A warp-specialised
    mainloop reuses its buffers for the epilogue (229,376 + 2,048 fits); the printed sum
    mainloop + epilogue + reserve = 239,616 does not. A cooperative mainloop holds both at once
    under either reading. Over the whole space the printed form keeps fewer candidates, and its
    between-layout differences are 50 / 50 / 90 instead of the paper's 55 / 55 / 99."""
    ws = candidate(128, 96, 128, 4, kernel_sched=0, epi_sched=1)
    assert is_valid(bf16(), ws, flags=COUPLED) and not is_valid(bf16(), ws, flags=COUPLED | PRINTED)
    coop = candidate(128, 96, 128, 4, kernel_sched=2, epi_sched=2)
    assert not is_valid(bf16(), coop, flags=COUPLED) and not is_valid(bf16(), coop, flags=COUPLED | PRINTED)
    small = candidate(128, 96, 128, 3, kernel_sched=0, epi_sched=1)
    assert is_valid(bf16(), small, flags=COUPLED | PRINTED)
    n_read = [len(oracle.valid_catalogue(bf16(lay), DESC, COUPLED, dtype=DT)[1]) for lay in range(4)]
    n_printed = [len(oracle.valid_catalogue(bf16(lay), DESC, COUPLED | PRINTED, dtype=DT)[1]) for lay in range(4)]
    assert all(a < b for a, b in zip(n_printed, n_read))
    assert (n_read[0] - n_read[1], n_read[0] - n_read[2], n_read[0] - n_read[3]) == (55, 55, 99)
    assert (n_printed[0] - n_printed[1], n_printed[0] - n_printed[2], n_printed[0] - n_printed[3]) == (50, 50, 90)


def test_size_is_the_papers_534600():
    assert oracle.catalogue_size() == 534600 == 4 * 9 * 5 * 11 * 15 * 3 * 3 * 2


def test_hand_decoded_ids():
    c = oracle.enumerate_candidates(0, 1, DT)
    assert c.tobytes() == candidate(64, 16, 32, 2, 1, 1, 0, 0, 0).tobytes()
    c = oracle.enumerate_candidates(534599, 1, DT)
    assert c.tobytes() == candidate(256, 256, 512, 12, 16, 1, 2, 2, 1).tobytes()
    # tile 128x128x64, 4 stages, cluster 1x1, WS, TMA epilogue, persistent: digits
    # (1, 6, 1, 2, 0, 0, 1, 0) -> ((((((1*9+6)*5+1)*11+2)*15+0)*3+0)*3+1)*2+0 = 226262
    c = oracle.enumerate_candidates(226262, 1, DT)
    assert c.tobytes() == candidate(128, 128, 64, 4, 1, 1, 0, 1, 0).tobytes()
    # the tile scheduler is the fastest digit, the cluster shape steps every 18 ids
    c = oracle.enumerate_candidates(17, 2, DT)
    assert (c["cluster_m"].tolist(), c["cluster_n"].tolist()) == ([1, 1], [1, 2])
    assert c["tile_sched"].tolist() == [1, 0] and c["epi_sched"].tolist() == [2, 0]


def test_space_is_the_knob_tables_product():
    c = whole_space()
    assert len(np.unique(c.view(np.dtype((np.void, 16))))) == 534600
    domains = {"tile_m": [64, 128, 192, 256], "tile_n": [16, 32, 48, 64, 80, 96, 128, 192, 256],
               "tile_k": [32, 64, 128, 256, 512], "stages": list(range(2, 13)),
               "kernel_sched": [0, 1, 2], "epi_sched": [0, 1, 2], "tile_sched": [0, 1]}
    for name, dom in domains.items():
        vals, counts = np.unique(c[name], return_counts=True)
        assert vals.tolist() == dom and np.all(counts == 534600 // len(dom)), name
    pairs = set(zip(c["cluster_m"].tolist(), c["cluster_n"].tolist()))
    assert pairs == {(a, b) for a in (1, 2, 4, 8, 16) for b in (1, 2, 4, 8, 16) if a * b <= 16}
    assert len(pairs) == 15
    assert np.all(c["instr_n"] == c["tile_n"]) and np.all(c["instr_m"] == 64) and np.all(c["instr_k"] == 16)
    # library enumeration of the same product, first knob slowest
    clusters = [(a, b) for a in (1, 2, 4, 8, 16) for b in (1, 2, 4, 8, 16) if a * b <= 16]
    g = np.array(list(itertools.product(domains["tile_m"], domains["tile_n"], domains["tile_k"],
                                        domains["stages"], range(15), range(3), range(3), range(2))))
    assert np.array_equal(g[:, 0], c["tile_m"]) and np.array_equal(g[:, 1], c["tile_n"])
    assert np.array_equal(g[:, 2], c["tile_k"]) and np.array_equal(g[:, 3], c["stages"])
    assert np.array_equal(np.array(clusters)[g[:, 4], 0], c["cluster_m"])
    assert np.array_equal(np.array(clusters)[g[:, 4], 1], c["cluster_n"])
    assert np.array_equal(g[:, 5], c["kernel_sched"]) and np.array_equal(g[:, 6], c["epi_sched"])
    assert np.array_equal(g[:, 7], c["tile_sched"])
    # a window in the middle equals the same slice of the whole
    w = oracle.enumerate_candidates(123457, 1000, DT)
    assert w.tobytes() == c[123457:124457].tobytes()


def test_each_rule_on_hand_built_candidates():
    p = bf16()
    ok = candidate(128, 128, 64, 4, 1, 1, 2, 2, 0)      # cooperative, TMA-cooperative epilogue
    assert is_valid(p, ok)
    # Stream-K needs the cooperative mainloop
    assert is_valid(p, candidate(128, 128, 64, 4, 1, 1, 2, 2, 1))
    assert not is_valid(p, candidate(128, 128, 64, 4, 1, 1, 0, 1, 1))
    assert not is_valid(p, candidate(128, 128, 64, 4, 1, 1, 1, 1, 1))
    # cooperative needs T_M = 0 mod 128
    for tm, good in ((64, False), (128, True), (192, False), (256, True)):
        assert is_valid(p, candidate(tm, 64, 32, 2, 1, 1, 2, 0, 0)) == good
        assert is_valid(p, candidate(tm, 64, 32, 2, 1, 1, 1, 0, 0))
    # capacity, bf16 128x128x64: one stage is 64*(128+128)*2 = 32,768 B; seven stages plus the
    # 2 KiB reserve are 231,424 <= 232,448, eight are not
    assert is_valid(p, candidate(128, 128, 64, 7, 1, 1, 1, 0, 0))
    assert not is_valid(p, candidate(128, 128, 64, 8, 1, 1, 1, 0, 0))
    # seven stages + a TMA epilogue (2*64*32*2 = 8,192 B): ping-pong holds both (239,616, too
    # much), the warp-specialised mainloop reuses its buffers (231,424, fits)
    assert not is_valid(p, candidate(128, 128, 64, 7, 1, 1, 1, 1, 0))
    assert is_valid(p, candidate(128, 128, 64, 7, 1, 1, 0, 1, 0))
    # fp8 operands halve the stage: 14 stages would fit, the knob range stops at 12
    assert is_valid(problem(4096, 4096, 4096, 0, 2, 1), candidate(128, 128, 64, 12, 1, 1, 1, 0, 0))
    # K-box limits: T_K = 512 needs C_N >= 2 when A is column-major (NN, NT) and C_M >= 2 when
    # B is row-major (TT, NT)
    k512 = lambda cm, cn: candidate(64, 16, 512, 2, cm, cn, 0, 0, 0)
    want = {TN_: (1, 1, 1, 1), TT_: (0, 0, 1, 1), NN_: (0, 1, 0, 1), NT_: (0, 0, 0, 1)}
    for lay, row in want.items():
        got = tuple(int(is_valid(bf16(lay), k512(cm, cn))) for cm, cn in ((1, 1), (1, 2), (2, 1), (2, 2)))
        assert got == row, (lay, got)
    assert all(is_valid(bf16(lay), candidate(64, 16, 256, 2, 1, 1, 0, 0, 0)) for lay in range(4))
    # the couplings are a flag: without it a TMA-cooperative epilogue may sit on any mainloop
    odd = candidate(128, 128, 64, 4, 1, 1, 0, 2, 0)
    assert is_valid(p, odd, flags=0) and not is_valid(p, odd, flags=COUPLED)
    odd = candidate(128, 128, 64, 4, 1, 1, 2, 1, 0)
    assert is_valid(p, odd, flags=0) and not is_valid(p, odd, flags=COUPLED)
    # the wasteful-tile rule as printed: T_N > 2M or T_N > 2N
    wide = candidate(64, 256, 32, 2, 1, 1, 0, 0, 0)
    assert is_valid(bf16(m=100, n=128), wide, flags=COUPLED | WASTEFUL) is False
    assert is_valid(bf16(m=128, n=100), wide, flags=COUPLED | WASTEFUL) is False
    assert is_valid(bf16(m=128, n=128), wide, flags=COUPLED | WASTEFUL)
    assert is_valid(bf16(m=100, n=100), wide, flags=COUPLED)


def test_tk512_family_listed_by_hand():
    """T_K = 512 in bf16: a stage is (T_M + T_N) KiB, so only two stages of T_M = 64 with
    T_N <= 48 fit under 225 KiB. T_N = 16, 32 leave room for an 8 KiB epilogue buffer on both
    non-cooperative mainloops (2 x 2 x 2 = 8 configurations); T_N = 48 leaves 1 KiB: no-smem
    epilogue on both, plus the TMA epilogue on the warp-specialised mainloop, which reuses the
    mainloop buffers (3). 11 per cluster shape."""
    c, _ = oracle.valid_catalogue(bf16(TN_), DESC, COUPLED, dtype=DT)
    f = c[(c["tile_k"] == 512) & (c["cluster_m"] == 1) & (c["cluster_n"] == 1)]
    got = sorted(zip(f["tile_m"].tolist(), f["tile_n"].tolist(), f["stages"].tolist(),
                     f["kernel_sched"].tolist(), f["epi_sched"].tolist(), f["tile_sched"].tolist()))
    want = sorted([(64, tn, 2, ks, es, 0) for tn in (16, 32) for ks in (0, 1) for es in (0, 1)] +
                  [(64, 48, 2, 0, 0, 0), (64, 48, 2, 1, 0, 0), (64, 48, 2, 0, 1, 0)])
    assert got == want
    assert (c["tile_k"] == 512).sum() == 11 * 15


def test_valid_counts_against_the_papers_table():
    n = {}
    for lay in range(4):
        c, idx = oracle.valid_catalogue(bf16(lay), DESC, COUPLED, dtype=DT)
        n[lay] = len(c)
        # stable: positions ascend and the kept records are those ids
        assert np.all(np.diff(idx) > 0)
        assert c[:500].tobytes() == np.concatenate(
            [oracle.enumerate_candidates(int(i), 1, DT) for i in idx[:500]]).tobytes()
    # between-layout differences, exact: the K-box rules only cut T_K = 512
    assert n[TN_] - n[TT_] == PAPER_COUNTS[TN_] - PAPER_COUNTS[TT_] == 55
    assert n[TT_] == n[NN_]
    assert n[TN_] - n[NT_] == PAPER_COUNTS[TN_] - PAPER_COUNTS[NT_] == 99
    # totals: within 1 % of the paper's (its epilogue-footprint estimator is not printed)
    for lay in range(4):
        assert abs(n[lay] - PAPER_COUNTS[lay]) <= 0.01 * PAPER_COUNTS[lay], (lay, n[lay])
    # the surviving share of the space is close to the paper's 11.36 %
    assert abs(sum(n.values()) / (4 * 534600) - 0.1136) < 0.002
    # the problem's dimensions do not enter without the wasteful-tile flag
    c2, idx2 = oracle.valid_catalogue(bf16(TN_, 64, 64, 64), DESC, COUPLED, dtype=DT)
    assert len(c2) == n[TN_]


def test_capacity_rule_agrees_with_the_footprint_column():
    """Rule 3 uses the same footprint as feature column 49 (smem_total)."""
    p = bf16(TN_)
    space = whole_space()[::7]
    x = oracle.featurize(p, space, DESC)
    fits = x[:, 49] <= np.float32(232448)
    structural = ~((space["tile_sched"] == 1) & (space["kernel_sched"] != 2)) & \
        ~((space["kernel_sched"] == 2) & (space["tile_m"] % 128 != 0))
    _, idx = oracle.valid_catalogue(p, DESC, 0, candidates=space)
    mask = np.zeros(len(space), bool)
    mask[idx] = True
    assert np.array_equal(mask, fits & structural)


def test_filter_of_an_explicit_list_equals_filter_by_id():
    p = bf16(NT_)
    sub_c, sub_i = oracle.valid_catalogue(p, DESC, COUPLED, count=50000, dtype=DT)
    lst = oracle.enumerate_candidates(0, 50000, DT)
    c2, i2 = oracle.valid_catalogue(p, DESC, COUPLED, candidates=lst)
    assert np.array_equal(sub_i, i2) and sub_c.tobytes() == c2.tobytes()
    # empty input
    c3, i3 = oracle.valid_catalogue(p, DESC, COUPLED, candidates=lst[:0])
    assert len(c3) == 0 and len(i3) == 0
