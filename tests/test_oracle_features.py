"""Pins for the oracle's feature map: hand-worked values, invariants the equations imply,
closed forms and special cases. None of these re-types a feature formula: every check is
either a literal expected value or a relation between the oracle's own outputs and inputs."""
import os

import numpy as np
import pytest

import oracle
from paper_2609_35587_b200 import workloads as wl
from tests.helpers import candidate, problem, read_worked_examples

DESC = wl.gpu_desc()
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.txt")

(LOG2_M, LOG2_N, LOG2_K) = (0, 1, 2)
(TILE_M, TILE_N, TILE_K, STAGES) = (10, 11, 12, 16)
(N_M, N_N, N_K, N_TILES, W_M, W_N, SUBSCR, WAVES, ETA, SK) = (23, 24, 25, 26, 27, 28, 29, 30, 31, 32)
(CL_WASTE, TPC_M, TPC_N, OVERSHOOT) = (33, 34, 35, 36)
(I_PROB, I_MAIN, R_STREAM, WS_L2, PANEL_A, PANEL_B, TRAFFIC, TRAFFIC_CL, TRAFFIC_EPI) = range(37, 46)
(B_STAGE, SMEM_MAIN, SMEM_EPI, SMEM_TOTAL, F_SMEM, FITS, R_PROXY, B_SMEM, B_REG, B_RES, OCC) = range(46, 57)
(T_PROD, T_CONS, R_PC, F_FILL, A_STAGE, S_X_FSMEM) = range(57, 63)


def feat(p, c, desc=DESC):
    return oracle.featurize(p, c, desc)


@pytest.mark.parametrize("ex", read_worked_examples(GOLDEN), ids=lambda e: e[0])
def test_worked_examples(ex):
    """Hand-worked values (tests/golden/worked_examples.txt): exact bits where a bit pattern is
    given, else the literal value."""
    name, p, c, pins = ex
    x = feat(p, c)[0]
    assert len(pins) > 30
    for col, val, bits in pins:
        if bits is not None:
            assert int(x[col].view(np.uint32)) == bits, (name, col, float(x[col]), val)
            assert float(x[col]) == pytest.approx(val, rel=2e-7, abs=1e-30)
        else:
            assert x[col] == np.float32(val), (name, col, float(x[col]), val)
    assert x[63] == 0.0


@pytest.fixture(scope="module")
def tiny():
    prob, cand, _, _ = wl.make_inputs(0, P=48, C=1500)
    x = oracle.featurize(prob, cand, DESC).reshape(len(prob), len(cand), 64).astype(np.float64)
    return prob, cand, x


def test_tile_counts_bracket_the_dimension(tiny):
    """n_M = ceil(M / T_M): n_M T_M >= M > (n_M - 1) T_M, likewise N and K."""
    prob, cand, x = tiny
    for dim, ncol, tcol in (("m", N_M, "tile_m"), ("n", N_N, "tile_n"), ("k", N_K, "tile_k")):
        D = prob[dim].astype(np.int64)[:, None]
        T = cand[tcol].astype(np.int64)[None, :]
        n = x[:, :, ncol].astype(np.int64)
        assert np.all(n * T >= D) and np.all((n - 1) * T < D)
    assert np.all(x[:, :, N_TILES] == x[:, :, N_M] * x[:, :, N_N])


def test_wave_quantisation_invariants(tiny):
    """q_SM = ceil(tiles / (S_SM b_res)): waves*SMs*b >= tiles > (waves-1)*SMs*b;
    eta_last in (0, 1], = 1 iff the tiles fill the last wave; Stream-K proxy = 1 - eta."""
    _, _, x = tiny
    tiles = x[:, :, N_TILES].astype(np.int64)
    waves = x[:, :, WAVES].astype(np.int64)
    b_eff = np.maximum(1, x[:, :, B_RES].astype(np.int64))
    resident = 148 * b_eff
    assert np.all(waves >= 1)
    assert np.all(waves * resident >= tiles) and np.all((waves - 1) * resident < tiles)
    eta = x[:, :, ETA]
    assert np.all(eta > 0) and np.all(eta <= 1)
    assert np.array_equal(eta == 1.0, tiles % resident == 0)
    np.testing.assert_allclose(eta, tiles / (waves * resident), rtol=1e-6)
    sk = x[:, :, SK]
    assert np.all(sk >= 0) and np.all(sk < 1)
    np.testing.assert_allclose(sk, 1 - eta, atol=1e-7)
    np.testing.assert_allclose(x[:, :, SUBSCR] * 148, tiles, rtol=1e-6)


def test_edge_waste(tiny):
    """w_M >= 0 with equality iff T_M divides M; w_M M = n_M T_M - M."""
    prob, cand, x = tiny
    for dim, wcol, ncol, tcol in (("m", W_M, N_M, "tile_m"), ("n", W_N, N_N, "tile_n")):
        D = prob[dim].astype(np.int64)[:, None]
        T = cand[tcol].astype(np.int64)[None, :]
        w = x[:, :, wcol]
        assert np.all(w >= 0)
        assert np.array_equal(w == 0, (D % T) == 0 + 0 * T)
        np.testing.assert_allclose(w * D, x[:, :, ncol] * T - D, rtol=1e-6, atol=1e-3)


def test_smem_footprint_and_residency(tiny):
    """S B_stage is linear in S; B_smem >= mainloop storage; b_res = min of its bounds;
    f_smem and b_smem are two views of the same ratio."""
    _, cand, x = tiny
    x0 = x[0]
    S = cand["stages"].astype(np.int64)
    assert np.all(x0[:, SMEM_MAIN] == S * x0[:, B_STAGE])
    assert np.all(x0[:, SMEM_TOTAL] >= x0[:, SMEM_MAIN] + 2048)
    assert np.all(x0[:, SMEM_TOTAL] <= x0[:, SMEM_MAIN] + x0[:, SMEM_EPI] + 2048)
    assert np.all(x0[:, SMEM_EPI][cand["epi_sched"] == 0] == 0)
    assert np.all(x0[:, SMEM_EPI][cand["epi_sched"] != 0] > 0)
    b_smem = x0[:, B_SMEM].astype(np.int64)
    tot = x0[:, SMEM_TOTAL].astype(np.int64)
    assert np.all(b_smem * tot <= 233472) and np.all((b_smem + 1) * tot > 233472)
    np.testing.assert_allclose(x0[:, F_SMEM] * 233472, tot, rtol=1e-6)
    assert np.all(x0[:, B_RES] <= x0[:, B_SMEM]) and np.all(x0[:, B_RES] <= x0[:, B_REG])
    assert np.all((x0[:, B_RES] == x0[:, B_SMEM]) | (x0[:, B_RES] == x0[:, B_REG]) |
                  (x0[:, B_RES] < np.minimum(x0[:, B_SMEM], x0[:, B_REG])))
    fits = x0[:, FITS]
    assert np.array_equal(fits == 1, x0[:, SMEM_MAIN] + x0[:, SMEM_EPI] + 2048 <= 232448)
    np.testing.assert_allclose(x0[:, S_X_FSMEM], S * x0[:, F_SMEM], rtol=1e-6)
    occ = x0[:, OCC]
    assert np.all(occ > 0) and np.all(occ <= 1)


def test_stage_monotonicity():
    """Raising the stage count tightens the shared-memory bound but not the register bound."""
    p = problem(2048, 2048, 2048)
    prev = None
    for s in range(2, 13):
        x = feat(p, candidate(128, 128, 64, s, kernel_sched=2, epi_sched=2))[0]
        cur = (x[SMEM_MAIN], x[SMEM_TOTAL], x[B_SMEM], x[B_REG], x[F_SMEM])
        if prev is not None:
            assert cur[0] > prev[0] and cur[1] > prev[1] and cur[4] > prev[4]
            assert cur[2] <= prev[2]
            assert cur[3] == prev[3]
        prev = cur
    assert prev[2] == 0  # twelve 32 KiB stages no longer fit one SM


def test_register_bound_non_increasing_in_tile_area():
    p = problem(2048, 2048, 2048)
    areas = [(64, 64), (64, 128), (128, 128), (128, 256), (256, 256)]
    for ks in range(4):
        b = [feat(p, candidate(tm, tn, 64, 3, kernel_sched=ks))[0][B_REG] for tm, tn in areas]
        assert all(b[i] >= b[i + 1] for i in range(len(b) - 1)), (ks, b)
        r = [feat(p, candidate(tm, tn, 64, 3, kernel_sched=ks))[0][R_PROXY] for tm, tn in areas]
        assert all(r[i] < r[i + 1] for i in range(len(r) - 1))


def test_tile_intensity_ignores_tile_k_and_is_symmetric():
    """I_mainloop: T_K cancels (the paper's tile-level ratio); swapping (T_M, T_N) leaves it
    unchanged when b_A = b_B."""
    p = problem(4096, 1024, 512, dtype_ab=2, dtype_d=1)
    vals = {feat(p, candidate(128, 64, tk, 3))[0][I_MAIN] for tk in (16, 32, 64, 128, 256, 512)}
    assert len(vals) == 1
    a = feat(p, candidate(128, 64, 64, 3))[0][I_MAIN]
    b = feat(p, candidate(64, 128, 64, 3))[0][I_MAIN]
    assert a == b
    # square tile, element size b: 2 T^2 / (2 T b) = T / b
    for dt, nbytes in ((0, 2), (2, 1), (3, 4)):
        x = feat(problem(512, 512, 512, dtype_ab=dt, dtype_d=1), candidate(128, 128, 32, 2))[0]
        assert x[I_MAIN] == 128 / nbytes


@pytest.mark.parametrize("s,dt,nbytes", [(4096, 1, 2), (1024, 0, 2), (768, 2, 1), (2048, 3, 4)])
def test_problem_intensity_square_closed_form(s, dt, nbytes):
    """Square GEMM with one element size b everywhere and no fusion: I_problem = 2s / (3b)."""
    dd = {1: 1, 0: 0, 2: 2, 3: 3}[dt]
    x = feat(problem(s, s, s, dtype_ab=dt, dtype_d=dd), candidate(128, 128, 64, 4))[0]
    assert float(x[I_PROB]) == pytest.approx(2 * s / (3 * nbytes), rel=2e-7)
    # bias adds epilogue bytes, so intensity drops; activations add none
    xb = feat(problem(s, s, s, dtype_ab=dt, dtype_d=dd, epi_flags=1), candidate(128, 128, 64, 4))[0]
    xr = feat(problem(s, s, s, dtype_ab=dt, dtype_d=dd, epi_flags=2), candidate(128, 128, 64, 4))[0]
    assert xb[I_PROB] < x[I_PROB] and xr[I_PROB] == x[I_PROB]
    assert xb[TRAFFIC_EPI] == x[TRAFFIC_EPI] + nbytes * s


def test_restreaming(tiny):
    """r_stream >= 1, = 1 iff a single tile covers the output, = (n_M + n_N)/2 when M = N."""
    prob, cand, x = tiny
    r = x[:, :, R_STREAM]
    assert np.all(r >= 1)
    one = (x[:, :, N_M] == 1) & (x[:, :, N_N] == 1)
    assert np.array_equal(r == 1, one)
    xs = feat(problem(1024, 1024, 512), candidate(128, 64, 32, 3))[0]
    assert xs[R_STREAM] == (xs[N_M] + xs[N_N]) / 2
    # numerator is the input-traffic column; denominator times L2 is the working-set column
    np.testing.assert_allclose(x[:, :, TRAFFIC] / r, x[:, :, WS_L2] * 132120576, rtol=1e-6)
    cl1 = (cand["cluster_m"] == 1) & (cand["cluster_n"] == 1)
    assert np.all(x[:, cl1, TRAFFIC_CL] == x[:, cl1, TRAFFIC])
    assert np.all(x[:, :, TRAFFIC_CL] <= x[:, :, TRAFFIC])


def test_pipeline_fill(tiny):
    """f_fill S = min(S, n_K); a_stage S = n_K; f_fill = 1 iff n_K >= S."""
    _, cand, x = tiny
    S = cand["stages"].astype(np.float64)[None, :]
    nk = x[:, :, N_K]
    np.testing.assert_allclose(x[:, :, F_FILL] * S, np.minimum(S, nk), rtol=1e-6)
    np.testing.assert_allclose(x[:, :, A_STAGE] * S, nk, rtol=1e-6)
    assert np.array_equal(x[:, :, F_FILL] == 1, nk >= S)
    np.testing.assert_allclose(x[:, :, R_PC] * x[:, :, T_PROD], x[:, :, T_CONS], rtol=1e-6)


def test_producer_consumer_scaling():
    """t_producer is proportional to B_stage; t_consumer halves with two consumer warpgroups
    and with a tensor rate twice as high."""
    p16 = problem(2048, 2048, 2048)
    a = feat(p16, candidate(128, 128, 64, 3, kernel_sched=0))[0]
    b = feat(p16, candidate(128, 128, 128, 3, kernel_sched=0))[0]
    assert b[B_STAGE] == 2 * a[B_STAGE] and b[T_PROD] == pytest.approx(2 * a[T_PROD], rel=1e-6)
    coop = feat(p16, candidate(128, 128, 64, 3, kernel_sched=2))[0]
    assert coop[T_CONS] == pytest.approx(a[T_CONS] / 2, rel=1e-6)
    p8 = problem(2048, 2048, 2048, dtype_ab=2, dtype_d=1)
    f8 = feat(p8, candidate(128, 128, 64, 3))[0]
    assert f8[T_CONS] == pytest.approx(a[T_CONS] / 2, rel=1e-6)


def test_cluster_fit():
    p = problem(64, 4096, 512)
    x = feat(p, candidate(64, 128, 64, 3, cluster_m=2, cluster_n=1))[0]
    assert (x[OVERSHOOT], x[TPC_M], x[TPC_N], x[CL_WASTE]) == (1, 0.5, 32, 1.0)
    x = feat(p, candidate(64, 128, 64, 3, cluster_m=1, cluster_n=2))[0]
    assert (x[OVERSHOOT], x[TPC_M], x[TPC_N], x[CL_WASTE]) == (0, 1, 16, 0.0)
    x = feat(p, candidate(64, 128, 64, 3))[0]
    assert (x[OVERSHOOT], x[CL_WASTE]) == (0, 0.0)


def test_log2_exact_for_powers_of_two_and_monotone():
    for e in range(0, 20):
        x = feat(problem(1 << e, 1 << e, 1 << e), candidate(64, 64, 32, 2))[0]
        assert x[LOG2_M] == e and x[LOG2_N] == e and x[LOG2_K] == e
    ms = np.arange(1, 3000)
    prob = np.zeros(len(ms), wl.PROBLEM_DT)
    prob["m"], prob["n"], prob["k"] = ms, 64, 64
    x = oracle.featurize(prob, candidate(64, 64, 32, 2), DESC)
    assert np.all(np.diff(x[:, LOG2_M]) > 0)
    np.testing.assert_allclose(x[:, LOG2_M], np.log2(ms), rtol=1e-7, atol=1e-7)


def test_structural_core_passthrough(tiny):
    prob, cand, x = tiny
    for col, name in ((10, "tile_m"), (11, "tile_n"), (12, "tile_k"), (13, "instr_m"),
                      (14, "instr_n"), (15, "instr_k"), (16, "stages"), (17, "kernel_sched"),
                      (18, "epi_sched"), (19, "tile_sched"), (20, "cluster_m"), (21, "cluster_n")):
        assert np.all(x[:, :, col] == cand[name][None, :].astype(np.float64)), name
    assert np.all(x[:, :, 22] == (cand["cluster_m"] * cand["cluster_n"])[None, :])
    assert np.all(x[:, :, 5] == prob["dtype_ab"][:, None])
    assert np.all(x[:, :, 3] == np.isin(prob["layout"], (2, 3))[:, None])
    assert np.all(x[:, :, 4] == np.isin(prob["layout"], (1, 3))[:, None])
    assert np.all(x[:, :, 63] == 0)
    assert np.all(np.isfinite(x))


def test_segment_form_matches_dense():
    prob, cand, so, si = wl.make_inputs(2, P=6, C=500, seg=40)
    dense = oracle.featurize(prob, cand, DESC).reshape(6, 500, 64)
    seg = oracle.featurize(prob, cand, DESC, so, si)
    assert seg.shape == (240, 64)
    for i in range(6):
        rows = si[so[i]:so[i + 1]]
        assert len(np.unique(rows)) == 40 and np.all(np.diff(rows) > 0)
        assert np.array_equal(seg[so[i]:so[i + 1]], dense[i, rows])
