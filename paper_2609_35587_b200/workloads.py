"""Seeded synthetic inputs for the selection path: problems, candidate pools, per-problem
segments, tree ensembles and MLP weights, shaped like the paper's workloads (a catalogue of
about 61k configurations per problem, dimensions log-uniform over a power-of-two box, the knob
domains of Table "Configuration knobs", ensembles of 10^2..10^3 trees of depth 6-8, the
dtypes and fusion flags of the transfer study).

This module is shared by the tests of the CPU oracle and of the CUDA library and therefore
holds NONE of the method's arithmetic: no feature formula, no model evaluation, no ranking.
Split thresholds and the MLP's standardisation constants are read from
``data/feature_stats.npz``, a table of per-column sample distributions / moments of each
workload's own feature distribution (written once by the committed script next to the
oracle that produced it).

Three threshold laws are offered for the synthetic ensembles (``LAWS``): "pernode", every
internal node draws its own quantile q ~ U(0.05, 0.95) of its column's sample (an ensemble
trained by exact greedy splitting: thousands of distinct thresholds per continuous column);
"hist256", q snapped to one of the 255 edges between 256 equal-mass bins (histogram-based
training); "slots128", one of 128 fixed quantile slots per column.

Random numbers come from a counter-based generator: a 64-bit mix of (seed, stream, index),
so every array is reproducible element by element and independent of generation order.
"""
from __future__ import annotations

import os
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20260935587
KS_F = 63
ROW = 64

PROBLEM_DT = np.dtype([("m", "<u4"), ("n", "<u4"), ("k", "<u4"), ("layout", "u1"),
                       ("dtype_ab", "u1"), ("dtype_d", "u1"), ("epi_flags", "u1")])
CANDIDATE_DT = np.dtype([("tile_m", "<u2"), ("tile_n", "<u2"), ("tile_k", "<u2"),
                         ("instr_n", "<u2"), ("stages", "u1"), ("cluster_m", "u1"),
                         ("cluster_n", "u1"), ("kernel_sched", "u1"), ("epi_sched", "u1"),
                         ("tile_sched", "u1"), ("instr_m", "u1"), ("instr_k", "u1")])
NODE_DT = np.dtype([("v", "<f4"), ("feat", "<u2"), ("kind", "<u2"), ("left", "<i4")])
GPU_DESC_DT = np.dtype([("num_sms", "<u4"), ("smem_per_sm", "<u4"), ("smem_per_cta_max", "<u4"),
                        ("smem_reserved", "<u4"), ("regs_per_sm", "<u4"),
                        ("max_threads_per_sm", "<u4"), ("max_ctas_per_sm", "<u4"),
                        ("reserved0", "<u4"), ("l2_bytes", "<u8"), ("tma_bytes_per_us", "<u8"),
                        ("tc_flops_per_us_per_sm", "<u8", (4,))])
assert PROBLEM_DT.itemsize == 16 and CANDIDATE_DT.itemsize == 16
assert NODE_DT.itemsize == 12 and GPU_DESC_DT.itemsize == 80

N_QUANTILE_SLOTS = 128
_STATS_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "data", "feature_stats.npz")

# stream ids (one per generated array)
_S_M, _S_N, _S_K, _S_LAYOUT, _S_DTYPE, _S_EPI, _S_DECODE = 1, 2, 3, 4, 5, 6, 7
_S_CAND_SHUFFLE, _S_SEG = 10, 11
_S_TREE_FEAT, _S_TREE_SLOT, _S_TREE_LEAF_A, _S_TREE_LEAF_B, _S_TREE_Q = 20, 21, 22, 23, 24
_S_MLP_W, _S_MLP_B = 30, 40
_S_SAMPLE = 50

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def mix64(seed: int, stream: int, index) -> np.ndarray:
    """64-bit counter-based hash of (seed, stream, index); index may be an array."""
    idx = np.asarray(index, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) ^ (np.uint64(stream) * np.uint64(0xD6E8FEB86659FD93))
        z = z + (idx + np.uint64(1)) * np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def uniform(seed: int, stream: int, index) -> np.ndarray:
    """Uniform doubles in [0, 1) from the top 53 bits of mix64."""
    return (mix64(seed, stream, index) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed: int, stream_a: int, stream_b: int, index) -> np.ndarray:
    """Standard normals by Box-Muller from two streams."""
    u1 = 1.0 - uniform(seed, stream_a, index)  # (0, 1]
    u2 = uniform(seed, stream_b, index)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def randint(seed: int, stream: int, index, n: int) -> np.ndarray:
    return np.minimum((uniform(seed, stream, index) * n).astype(np.int64), n - 1)


def permutation(seed: int, stream: int, n: int) -> np.ndarray:
    return np.argsort(mix64(seed, stream, np.arange(n)), kind="stable")


def gpu_desc() -> np.ndarray:
    """The target descriptor used by every workload ("B200-synthetic"): 148 SMs and 228 KiB
    of shared memory per SM; the remaining capacities and rates are plain descriptor data."""
    d = np.zeros((), dtype=GPU_DESC_DT)
    d["num_sms"] = 148
    d["smem_per_sm"] = 228 * 1024
    d["smem_per_cta_max"] = 227 * 1024
    d["smem_reserved"] = 2048
    d["regs_per_sm"] = 65536
    d["max_threads_per_sm"] = 2048
    d["max_ctas_per_sm"] = 32
    d["l2_bytes"] = 126 * 1024 * 1024
    d["tma_bytes_per_us"] = 8_000_000
    d["tc_flops_per_us_per_sm"] = (15_202_703, 15_202_703, 30_405_405, 7_601_351)
    return d


# ------------------------------------------------------------------------------------------
# problems
# ------------------------------------------------------------------------------------------

def _log_uniform_dim(seed, stream, idx, lo, hi, multiple):
    v = lo * (hi / lo) ** uniform(seed, stream, idx)
    if multiple > 1:
        v = multiple * np.floor(v / multiple + 0.5)
    else:
        v = np.floor(v)
    return np.clip(v, lo, hi).astype(np.uint32)


def problems_batch(seed: int, P: int, cross_precision: bool = False) -> np.ndarray:
    """M, N, K log-uniform in [64, 8192] rounded to multiples of 16. Plain: fp16 in/out, layout
    TN or NN. Cross-precision: dtype from {fp16, bf16, fp8_e4m3, tf32}, one of six fusion
    flag sets, all four layouts."""
    idx = np.arange(P)
    p = np.zeros(P, dtype=PROBLEM_DT)
    p["m"] = _log_uniform_dim(seed, _S_M, idx, 64, 8192, 16)
    p["n"] = _log_uniform_dim(seed, _S_N, idx, 64, 8192, 16)
    p["k"] = _log_uniform_dim(seed, _S_K, idx, 64, 8192, 16)
    if cross_precision:
        p["layout"] = randint(seed, _S_LAYOUT, idx, 4)
        dt = randint(seed, _S_DTYPE, idx, 4)
        p["dtype_ab"] = dt
        p["dtype_d"] = np.array([0, 1, 1, 3], dtype=np.uint8)[dt]
        p["epi_flags"] = np.array([0, 1, 2, 4, 3, 5], dtype=np.uint8)[randint(seed, _S_EPI, idx, 6)]
    else:
        p["layout"] = np.where(randint(seed, _S_LAYOUT, idx, 2) == 0, 0, 2)
    return p


def problems_stream(seed: int, n: int) -> np.ndarray:
    """Latency stream: N, K = floor(16384^u) in [1, 16384]; M likewise except that half of the
    problems are decode-like with M = floor(64^u) in [1, 64]. fp16, TN."""
    idx = np.arange(n)
    p = np.zeros(n, dtype=PROBLEM_DT)
    big = _log_uniform_dim(seed, _S_M, idx, 1, 16384, 1)
    small = _log_uniform_dim(seed, _S_M, idx, 1, 64, 1)
    p["m"] = np.where(uniform(seed, _S_DECODE, idx) < 0.5, small, big)
    p["n"] = _log_uniform_dim(seed, _S_N, idx, 1, 16384, 1)
    p["k"] = _log_uniform_dim(seed, _S_K, idx, 1, 16384, 1)
    return p


# ------------------------------------------------------------------------------------------
# candidates
# ------------------------------------------------------------------------------------------

def _grid(axes):
    mesh = np.meshgrid(*[np.asarray(a) for a in axes], indexing="ij")
    return [m.reshape(-1) for m in mesh]


def candidates_small_grid(seed: int, count: int | None = 2048) -> np.ndarray:
    """tile_m, tile_n in {64,128,256} x tile_k in {32,64,128} x stages 2..7 x 4 clusters x 4
    kernel schedules x 2 epilogue schedules = 5,184; seeded shuffle, first `count`."""
    clusters = [(1, 1), (2, 1), (1, 2), (2, 2)]
    tm, tn, tk, st, cl, ks, es = _grid([[64, 128, 256], [64, 128, 256], [32, 64, 128],
                                        range(2, 8), range(4), range(4), range(2)])
    c = np.zeros(len(tm), dtype=CANDIDATE_DT)
    c["tile_m"], c["tile_n"], c["tile_k"], c["stages"] = tm, tn, tk, st
    c["instr_n"] = tn
    c["instr_m"], c["instr_k"] = 64, 16
    cl_arr = np.array(clusters)
    c["cluster_m"], c["cluster_n"] = cl_arr[cl, 0], cl_arr[cl, 1]
    c["kernel_sched"], c["epi_sched"] = ks, es
    c = c[permutation(seed, _S_CAND_SHUFFLE, len(c))]
    return c if count is None else c[:count].copy()


def candidates_full_grid(seed: int, count: int | None = 60000) -> np.ndarray:
    """tile_m {64,128,192,256} x tile_n {64,128,256} x tile_k {32,64,128} x instr_n {tile_n,
    tile_n/2} x stages 2..7 x 6 clusters x 4 kernel schedules x 2 tile schedulers x 3 epilogue
    schedules = 62,208 (the unfiltered cross-product); seeded shuffle, first `count`."""
    clusters = [(1, 1), (2, 1), (1, 2), (2, 2), (4, 1), (1, 4)]
    tm, tn, tk, half, st, cl, ks, ts, es = _grid([[64, 128, 192, 256], [64, 128, 256],
                                                  [32, 64, 128], range(2), range(2, 8), range(6),
                                                  range(4), range(2), range(3)])
    c = np.zeros(len(tm), dtype=CANDIDATE_DT)
    c["tile_m"], c["tile_n"], c["tile_k"], c["stages"] = tm, tn, tk, st
    c["instr_n"] = np.where(half == 1, tn // 2, tn)
    c["instr_m"], c["instr_k"] = 64, 16
    cl_arr = np.array(clusters)
    c["cluster_m"], c["cluster_n"] = cl_arr[cl, 0], cl_arr[cl, 1]
    c["kernel_sched"], c["tile_sched"], c["epi_sched"] = ks, ts, es
    c = c[permutation(seed, _S_CAND_SHUFFLE, len(c))]
    return c if count is None else c[:count].copy()


def segments(seed: int, P: int, pool: int, per_problem: int):
    """Per-problem candidate sets: `per_problem` distinct pool indices each (seeded sample
    without replacement, ascending). Returns (seg_offsets int64 [P+1], seg_index int32)."""
    per_problem = min(per_problem, pool)
    seg_index = np.empty((P, per_problem), dtype=np.int32)
    cols = np.arange(pool, dtype=np.uint64)
    step = 128
    for lo in range(0, P, step):
        hi = min(P, lo + step)
        rows = np.arange(lo, hi, dtype=np.uint64)[:, None] * np.uint64(pool) + cols[None, :]
        keys = mix64(seed, _S_SEG, rows)
        part = np.argpartition(keys, per_problem - 1, axis=1)[:, :per_problem] if per_problem < pool \
            else np.broadcast_to(np.arange(pool), (hi - lo, pool))
        seg_index[lo:hi] = np.sort(part, axis=1)
    seg_offsets = np.arange(P + 1, dtype=np.int64) * per_problem
    return seg_offsets, seg_index.reshape(-1)


# ------------------------------------------------------------------------------------------
# models
# ------------------------------------------------------------------------------------------

# Feature columns that hold a categorical field's level code, with the number of levels: layout
# flags, operand type, bias flag, activation, kernel / epilogue schedule, tile scheduler.
CATEGORICAL_LEVELS = {3: 2, 4: 2, 5: 4, 8: 2, 9: 3, 17: 4, 18: 3, 19: 2}
_S_PARTITION = 0x70617274


def with_partition_splits(seed: int, nodes: np.ndarray) -> np.ndarray:
    """Copy of `nodes` in which every internal node on a categorical column becomes a partition
    split: kind = 1 and the bit pattern of v = a seeded, non-empty, proper subset of the field's
    levels (the members go to the right child)."""
    out = nodes.copy()
    for i in np.nonzero(np.isin(out["feat"], list(CATEGORICAL_LEVELS)))[0]:
        levels = CATEGORICAL_LEVELS[int(out["feat"][i])]
        full = (1 << levels) - 1
        mask = 1 + int(mix64(seed, _S_PARTITION, np.array([i], dtype=np.uint64))[0] % np.uint64(full - 1))
        out["v"][i] = np.array([mask], dtype=np.uint32).view(np.float32)[0]
        out["kind"][i] = 1
    return out


_stats_cache = None


def feature_stats(key: str) -> dict:
    """Per-column threshold slots [63, 128] and (mu, sigma) [64] of workload `key`."""
    global _stats_cache
    if _stats_cache is None:
        if not os.path.exists(_STATS_PATH):
            raise FileNotFoundError(f"{_STATS_PATH} is missing")
        with np.load(_STATS_PATH) as z:
            _stats_cache = {k: z[k] for k in z.files}
    return {"thr": _stats_cache[f"{key}_thr"], "mu": _stats_cache[f"{key}_mu"],
            "sigma": _stats_cache[f"{key}_sigma"], "dval": _stats_cache[f"{key}_dval"],
            "dcum": _stats_cache[f"{key}_dcum"], "doff": _stats_cache[f"{key}_doff"]}


LAWS = ("pernode", "hist256", "slots128")
DEFAULT_LAW = "pernode"


def quantile_thresholds(stats: dict, feat: np.ndarray, q: np.ndarray) -> np.ndarray:
    """Split threshold of every node: the q-quantile of the node's column over the stored sample,
    placed midway (in fp32) between the two adjacent distinct sample values around it; value +
    0.5 for a column that is constant in the sample."""
    feat = np.asarray(feat)
    q = np.asarray(q, dtype=np.float64)
    out = np.empty(feat.shape, dtype=np.float32)
    dval, dcum, doff = stats["dval"], stats["dcum"], stats["doff"]
    for f in range(KS_F):
        sel = feat == f
        if not sel.any():
            continue
        d = dval[doff[f]:doff[f + 1]]
        cum = dcum[doff[f]:doff[f + 1]]
        n = int(cum[-1])
        pos = np.floor(q[sel] * (n - 1)).astype(np.int64)
        i = np.searchsorted(cum, pos, side="right")  # the distinct value holding order statistic `pos`
        if len(d) == 1:
            out[sel] = np.float32(d[0] + np.float32(0.5))
            continue
        lo_i = np.where(i + 1 < len(d), i, i - 1)
        lo, hi = d[lo_i], d[lo_i + 1]
        t = ((lo.astype(np.float64) + hi.astype(np.float64)) / 2.0).astype(np.float32)
        out[sel] = np.where(t <= lo, hi, t)
    return out


def gbdt_complete(seed: int, n_trees: int, depth: int, stats: dict, leaf_sigma: float,
                  law: str = DEFAULT_LAW):
    """`n_trees` complete binary trees of `depth` in level order. Split feature uniform over the
    63 columns; threshold by `law` (see the module text); leaves ~ N(0, leaf_sigma).
    Returns (tree_offsets int64 [n_trees+1], nodes NODE_DT)."""
    n_int = (1 << depth) - 1
    n_leaf = 1 << depth
    per = n_int + n_leaf
    nodes = np.zeros(n_trees * per, dtype=NODE_DT).reshape(n_trees, per)
    iidx = (np.arange(n_trees)[:, None] * n_int + np.arange(n_int)[None, :])
    feat = randint(seed, _S_TREE_FEAT, iidx, KS_F)
    nodes["feat"][:, :n_int] = feat
    if law == "slots128":
        thr_slots = stats["thr"]
        slot = randint(seed, _S_TREE_SLOT, iidx, thr_slots.shape[1])
        nodes["v"][:, :n_int] = thr_slots[feat, slot]
    elif law in ("pernode", "hist256"):
        q = 0.05 + 0.9 * uniform(seed, _S_TREE_Q, iidx)
        if law == "hist256":
            q = (np.floor(q * 256.0) + 1.0) / 256.0
        nodes["v"][:, :n_int] = quantile_thresholds(stats, feat, q)
    else:
        raise ValueError(f"unknown threshold law {law!r}")
    nodes["left"][:, :n_int] = 2 * np.arange(n_int)[None, :] + 1
    lidx = (np.arange(n_trees)[:, None] * n_leaf + np.arange(n_leaf)[None, :])
    nodes["feat"][:, n_int:] = 0xFFFF
    nodes["v"][:, n_int:] = (leaf_sigma * normal(seed, _S_TREE_LEAF_A, _S_TREE_LEAF_B, lidx)).astype(np.float32)
    offsets = np.arange(n_trees + 1, dtype=np.int64) * per
    return offsets, nodes.reshape(-1)


def float_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (data preparation for weights)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def mlp_xavier(seed: int, widths, mu: np.ndarray, sigma: np.ndarray) -> dict:
    """Xavier-uniform bf16 weights U(-a, a), a = sqrt(6 / (fan_in + fan_out)); fp32 biases
    U(-0.05, 0.05); standardisation constants passed through."""
    widths = [int(w) for w in widths]
    weights, biases = [], []
    for l in range(len(widths) - 1):
        fin, fout = widths[l], widths[l + 1]
        a = np.sqrt(6.0 / (fin + fout))
        w = (2.0 * uniform(seed, _S_MLP_W + l, np.arange(fin * fout)) - 1.0) * a
        weights.append(float_to_bf16_bits(w.astype(np.float32)).reshape(fout, fin))
        biases.append(((2.0 * uniform(seed, _S_MLP_B + l, np.arange(fout)) - 1.0) * 0.05).astype(np.float32))
    return {"widths": np.array(widths, dtype=np.int32), "weights": weights, "biases": biases,
            "mu": np.ascontiguousarray(mu, dtype=np.float32),
            "sigma": np.ascontiguousarray(sigma, dtype=np.float32)}


ONEHOT_WIDTH = 80
ONEHOT_FIELDS = ((5, 4), (9, 3), (17, 4), (18, 3))   # (feature column, levels) expanded to indicators


def onehot_stats(mu: np.ndarray, sigma: np.ndarray):
    """Standardisation constants of the one-hot input layout from those of the 64-wide row: the
    59 kept columns keep theirs (ascending column order), the 14 indicators and the padding
    get mu = 0, sigma = 1."""
    keep = [j for j in range(63) if j not in (5, 9, 17, 18)]
    mu2, sg2 = np.zeros(ONEHOT_WIDTH, np.float32), np.ones(ONEHOT_WIDTH, np.float32)
    mu2[:59], sg2[:59] = np.asarray(mu, np.float32)[keep], np.asarray(sigma, np.float32)[keep]
    return mu2, sg2


# ------------------------------------------------------------------------------------------
# the five workloads
# ------------------------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    desc: np.ndarray
    problems: np.ndarray
    candidates: np.ndarray
    k: int
    seg_offsets: np.ndarray | None = None
    seg_index: np.ndarray | None = None
    gbdt: tuple | None = None      # (tree_offsets, nodes, base_score)
    mlp: dict | None = None
    meta: dict = field(default_factory=dict)

    @property
    def pairs(self) -> int:
        if self.seg_offsets is not None:
            return int(self.seg_offsets[-1])
        return len(self.problems) * len(self.candidates)


# (problems, pool, segment size, trees, depth, leaf sigma, k, stats key)
CONFIGS = {
    0: dict(name="tiny", P=64, C=2048, seg=None, trees=100, depth=6, leaf_sigma=0.1, k=5, stats="cfg0"),
    1: dict(name="full_space", P=1024, C=60000, seg=None, trees=500, depth=8, leaf_sigma=0.1, k=10, stats="cfg1"),
    2: dict(name="cross_precision", P=4096, C=62208, seg=16384, trees=1000, depth=8, leaf_sigma=0.05, k=10, stats="cfg2"),
    3: dict(name="dynamic", P=100000, C=60000, seg=None, trees=500, depth=8, leaf_sigma=0.1, k=10, stats="cfg1"),
    4: dict(name="neural_ranker", P=1024, C=60000, seg=None, trees=0, depth=0, leaf_sigma=0.0, k=10, stats="cfg1"),
}


def make_inputs(cfg: int, P: int | None = None, C: int | None = None, seg: int | None = None,
                seed: int = BASE_SEED):
    """Problems, pool and segments of config `cfg` (sizes may be overridden for tests)."""
    spec = CONFIGS[cfg]
    P = spec["P"] if P is None else P
    C = spec["C"] if C is None else C
    s = seed + 1000 * cfg
    if cfg == 3:
        prob = problems_stream(s, P)
    else:
        prob = problems_batch(s if cfg != 4 else seed + 1000, P, cross_precision=(cfg == 2))
    cs = seed + 1000 if cfg in (3, 4) else s  # configs 3 and 4 reuse config 1's catalogue
    cand = candidates_small_grid(cs, C) if cfg == 0 else candidates_full_grid(cs, C)
    so = si = None
    seg = spec["seg"] if seg is None else seg
    if spec["seg"] is not None:
        so, si = segments(s, P, len(cand), seg)
    return prob, cand, so, si


def make_workload(cfg: int, P: int | None = None, C: int | None = None, seg: int | None = None,
                  trees: int | None = None, depth: int | None = None,
                  seed: int = BASE_SEED, law: str = DEFAULT_LAW) -> Workload:
    spec = CONFIGS[cfg]
    prob, cand, so, si = make_inputs(cfg, P, C, seg, seed)
    st = feature_stats(spec["stats"])
    w = Workload(name=spec["name"], desc=gpu_desc(), problems=prob, candidates=cand, k=spec["k"],
                 seg_offsets=so, seg_index=si, meta=dict(cfg=cfg, seed=seed, law=law))
    if cfg == 4:
        w.mlp = mlp_xavier(seed + 4000, [64, 256, 256, 1], st["mu"], st["sigma"])
    else:
        ms = seed + 1000 if cfg == 3 else seed + 1000 * cfg  # config 3 uses config 1's ensemble
        T = spec["trees"] if trees is None else trees
        D = spec["depth"] if depth is None else depth
        off, nodes = gbdt_complete(ms, T, D, st, spec["leaf_sigma"], law)
        w.gbdt = (off, nodes, 0.0)
    return w
