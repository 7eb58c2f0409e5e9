"""ctypes binding of libks (the C ABI declared in include/ks.h).

Argument marshalling only: every step of the selection path runs inside the library's CUDA
kernels. torch supplies device memory (`tensor.data_ptr()`) and the current stream. There is
no CPU fallback: importing this module without the built library raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# KS_LIBRARY names another build of the same library (the checked build libks_debug.so)
LIB_PATH = os.environ.get("KS_LIBRARY") or os.path.join(_HERE, "libks.so")

KS_F, KS_F_PAD, KS_MAX_K, KS_MAX_DEPTH = 63, 64, 32, 15
KS_CATALOGUE_SIZE = 534600
KS_VALID_COUPLED, KS_VALID_WASTEFUL, KS_VALID_PRINTED_CAPACITY = 1, 2, 4
KS_OK, KS_ERR_INVALID_ARG, KS_ERR_UNSUPPORTED, KS_ERR_CUDA, KS_ERR_TIMEOUT, KS_ERR_OOM = range(6)

EXPORTS = ("ks_create", "ks_destroy", "ks_last_cuda_error", "ks_model_create_gbdt",
           "ks_model_create_mlp", "ks_model_create_static", "ks_model_destroy", "ks_featurize", "ks_score", "ks_select",
           "ks_select_one", "ks_select_host", "ks_status_string", "ks_feature_count",
           "ks_feature_name", "ks_launch_count", "ks_profile_enable", "ks_profile_last_ms", "ks_device_status", "ks_select_trees_static",
           "ks_enumerate", "ks_valid_catalogue", "ks_remap_indices", "ks_model_describe", "ks_merge_topk", "ks_catalogue_prepare", "ks_catalogue_destroy",
           "ks_select_one_prepared",
           "ks_debug_set_wait", "ks_debug_bounds_line", "ks_debug_bounds_clear", "ks_debug_walk_floor")


class KsError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = f"{where}: {_status_string(status)}"
        super().__init__(msg + (f" ({detail})" if detail else ""))


class _Problem(ctypes.Structure):
    _fields_ = [("m", ctypes.c_uint32), ("n", ctypes.c_uint32), ("k", ctypes.c_uint32),
                ("layout", ctypes.c_uint8), ("dtype_ab", ctypes.c_uint8),
                ("dtype_d", ctypes.c_uint8), ("epi_flags", ctypes.c_uint8)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is not built; run `python -c 'import __graft_entry__ as g; "
                          "g.build()'` (nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    lib.ks_create.argtypes = [ctypes.POINTER(vp), i32, vp]
    lib.ks_destroy.argtypes = [vp]
    lib.ks_last_cuda_error.argtypes = [vp]
    lib.ks_last_cuda_error.restype = ctypes.c_char_p
    lib.ks_model_create_gbdt.argtypes = [vp, i32, vp, vp, ctypes.c_float, ctypes.POINTER(vp)]
    lib.ks_model_create_mlp.argtypes = [vp, i32, vp, vp, vp, vp, vp, ctypes.POINTER(vp)]
    lib.ks_model_create_static.argtypes = [vp, ctypes.POINTER(vp)]
    lib.ks_model_destroy.argtypes = [vp]
    lib.ks_featurize.argtypes = [vp, vp, i32, vp, i32, vp, vp, i64, vp, vp]
    lib.ks_score.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    lib.ks_select.argtypes = [vp, vp, i32, vp, i32, vp, vp, i64, vp, i32, vp, vp, vp]
    lib.ks_select_one.argtypes = [vp, _Problem, vp, i32, vp, i32, vp, vp, vp]
    lib.ks_select_host.argtypes = [vp, vp, i32, vp, i32, vp, vp, i64, vp, i32, vp, vp, vp]
    lib.ks_status_string.argtypes = [i32]
    lib.ks_status_string.restype = ctypes.c_char_p
    lib.ks_feature_count.restype = i32
    lib.ks_feature_name.argtypes = [i32]
    lib.ks_feature_name.restype = ctypes.c_char_p
    lib.ks_launch_count.argtypes = [vp]
    lib.ks_launch_count.restype = i64
    lib.ks_profile_enable.argtypes = [vp, i32]
    lib.ks_device_status.argtypes = [vp]
    lib.ks_select_trees_static.argtypes = [i32, vp, vp, i32, vp, i32, vp, vp, i32, ctypes.c_float, i32, vp, vp, vp]
    lib.ks_profile_last_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.ks_enumerate.argtypes = [vp, i64, i64, vp, vp]
    lib.ks_valid_catalogue.argtypes = [vp, ctypes.POINTER(_Problem), ctypes.c_uint, vp, i32, vp, vp, vp,
                                       ctypes.POINTER(ctypes.c_int32), vp]
    lib.ks_remap_indices.argtypes = [vp, vp, i64, vp, i32, vp]
    lib.ks_model_describe.argtypes = [vp, ctypes.c_char_p, i32]
    lib.ks_merge_topk.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp]
    lib.ks_catalogue_prepare.argtypes = [vp, vp, i32, vp, ctypes.POINTER(vp), vp]
    lib.ks_catalogue_destroy.argtypes = [vp]
    lib.ks_select_one_prepared.argtypes = [vp, vp, _Problem, i32, vp, vp, vp]
    lib.ks_debug_set_wait.argtypes = [vp, i32, i32]
    lib.ks_debug_walk_floor.argtypes = [vp, vp, i64, vp, i32, vp, vp]
    lib.ks_debug_bounds_line.restype = i32
    lib.ks_debug_bounds_clear.restype = None
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int and name not in ("ks_feature_count",):
            fn.restype = ctypes.c_int
    return lib


_lib = _load()


def _status_string(s: int) -> str:
    return _lib.ks_status_string(int(s)).decode()


def ks_feature_count() -> int:
    return int(_lib.ks_feature_count())


def ks_feature_name(i: int):
    s = _lib.ks_feature_name(int(i))
    return None if s is None else s.decode()


def _dptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _hptr(a):
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous():
            raise ValueError("expected a contiguous host tensor")
        return ctypes.c_void_p(a.data_ptr())
    if not a.flags["C_CONTIGUOUS"]:
        raise ValueError("expected a C-contiguous array")
    return ctypes.c_void_p(a.ctypes.data)


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def problem_structs(problems: np.ndarray):
    """The problem records as an array of by-value arguments for `Context.select_one_caller`
    (the 16-byte record is the C struct: a byte copy)."""
    a = np.ascontiguousarray(problems).reshape(-1)
    if a.dtype.itemsize != ctypes.sizeof(_Problem):
        raise ValueError("expected ks_problem records")
    return (_Problem * len(a)).from_buffer_copy(a.tobytes())


def to_device(records: np.ndarray, device) -> torch.Tensor:
    """A numpy record / plain array as a device tensor of raw bytes (records) or values."""
    a = np.ascontiguousarray(records)
    if a.dtype.fields is not None:
        a = a.view(np.uint8).reshape(len(records), -1)
    return torch.from_numpy(a.copy()).to(device)


NODE_DEV_DT = np.dtype([("v", "<f4"), ("feat", "<u2"), ("left", "<u2")])


def ks_select_trees_static(desc: np.ndarray, d_p, P, d_c, C, d_nodes, d_tree_offsets, n_trees, base_score, k,
                           d_topk_idx, d_topk_score, device: int = 0) -> int:
    """Raw call of the allocation-free entry point: every buffer is the caller's (torch device
    tensors here), nothing is allocated on the way; returns the ks_status."""
    d = np.ascontiguousarray(desc).reshape(1)
    return int(_lib.ks_select_trees_static(device, _hptr(d), _dptr(d_p), P, _dptr(d_c), C, _dptr(d_nodes),
                                           _dptr(d_tree_offsets), n_trees, ctypes.c_float(base_score), k,
                                           _dptr(d_topk_idx), _dptr(d_topk_score), _stream()))


def debug_bounds_line() -> int:
    """Checked build: source line of the first out-of-range index the kernels met (0: none);
    -1 in a regular build."""
    return int(_lib.ks_debug_bounds_line())


def debug_bounds_clear() -> None:
    _lib.ks_debug_bounds_clear()


class Model:
    def __init__(self, ctx: "Context", handle: ctypes.c_void_p, kind: str, n_trees: int = 0):
        self.ctx, self._h, self.kind, self.n_trees = ctx, handle, kind, n_trees

    def describe(self) -> str:
        """The fused kernel ks_select runs for this model, with its tile geometry."""
        buf = ctypes.create_string_buffer(256)
        st = _lib.ks_model_describe(self._h, buf, 256)
        if st != KS_OK:
            raise KsError(st, "ks_model_describe")
        return buf.value.decode()

    def close(self):
        if self._h:
            _lib.ks_model_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Catalogue:
    """ks_catalogue: a candidate pool prepared for single-problem calls with one model."""

    def __init__(self, ctx: "Context", handle, d_c, C: int, model: Model):
        self.ctx, self._h, self.d_c, self.C, self.model = ctx, handle, d_c, C, model

    def close(self):
        if self._h:
            _lib.ks_catalogue_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Context:
    """ks_ctx plus thin methods named after the C entry points."""

    def __init__(self, desc: np.ndarray, device: int = 0):
        d = np.ascontiguousarray(desc)
        if d.nbytes != 80:
            raise ValueError("gpu descriptor must be 80 bytes")
        self.device = torch.device("cuda", device)
        h = ctypes.c_void_p()
        st = _lib.ks_create(ctypes.byref(h), device, _hptr(d.reshape(1)))
        if st != KS_OK:
            raise KsError(st, "ks_create")
        self._h = h

    def close(self):
        if self._h:
            _lib.ks_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, where: str):
        if st != KS_OK:
            raise KsError(st, where, _lib.ks_last_cuda_error(self._h).decode())

    def launch_count(self) -> int:
        return int(_lib.ks_launch_count(self._h))

    def device_status(self) -> int:
        return int(_lib.ks_device_status(self._h))

    def debug_set_wait(self, probe_limit: int = 0, starve: bool = False):
        """Test hook: probe budget of the kernels' bounded waits, and the starved-wait mode."""
        self._check(_lib.ks_debug_set_wait(self._h, int(probe_limit), int(starve)), "ks_debug_set_wait")

    def profile_enable(self, on: bool = True):
        self._check(_lib.ks_profile_enable(self._h, int(on)), "ks_profile_enable")

    def profile_last_ms(self) -> float:
        ms = ctypes.c_float()
        self._check(_lib.ks_profile_last_ms(self._h, ctypes.byref(ms)), "ks_profile_last_ms")
        return float(ms.value)

    # ---- models ---------------------------------------------------------------------------
    def model_create_gbdt(self, tree_offsets, nodes, base_score: float = 0.0) -> Model:
        off = np.ascontiguousarray(tree_offsets, dtype=np.int64)
        nd = np.ascontiguousarray(nodes)
        if nd.dtype.itemsize != 12:
            raise ValueError("nodes must be 12-byte records")
        h = ctypes.c_void_p()
        st = _lib.ks_model_create_gbdt(self._h, len(off) - 1, _hptr(off), _hptr(nd),
                                       ctypes.c_float(base_score), ctypes.byref(h))
        self._check(st, "ks_model_create_gbdt")
        return Model(self, h, "gbdt", len(off) - 1)

    def model_create_mlp(self, mlp: dict) -> Model:
        widths = np.ascontiguousarray(mlp["widths"], dtype=np.int32)
        L = len(widths) - 1
        ws = [np.ascontiguousarray(w, dtype=np.uint16) for w in mlp["weights"]]
        bs = [np.ascontiguousarray(b, dtype=np.float32) for b in mlp["biases"]]
        mu = np.ascontiguousarray(mlp["mu"], dtype=np.float32)
        sigma = np.ascontiguousarray(mlp["sigma"], dtype=np.float32)
        wp = (ctypes.c_void_p * L)(*[w.ctypes.data for w in ws])
        bp = (ctypes.c_void_p * L)(*[b.ctypes.data for b in bs])
        h = ctypes.c_void_p()
        st = _lib.ks_model_create_mlp(self._h, L, _hptr(widths), ctypes.cast(wp, ctypes.c_void_p),
                                      ctypes.cast(bp, ctypes.c_void_p), _hptr(mu), _hptr(sigma),
                                      ctypes.byref(h))
        self._check(st, "ks_model_create_mlp")
        return Model(self, h, "mlp")

    def model_create_static(self) -> Model:
        h = ctypes.c_void_p()
        self._check(_lib.ks_model_create_static(self._h, ctypes.byref(h)), "ks_model_create_static")
        return Model(self, h, "static")

    # ---- the path -------------------------------------------------------------------------
    @staticmethod
    def _pairs(P, C, seg_off_pairs):
        return P * C if seg_off_pairs is None else int(seg_off_pairs)

    def featurize(self, d_p, P, d_c, C, d_seg_off=None, d_seg_idx=None, pairs=None, out=None):
        pairs = P * C if pairs is None else pairs
        if out is None:
            out = torch.empty((pairs, KS_F_PAD), dtype=torch.float32, device=self.device)
        st = _lib.ks_featurize(self._h, _dptr(d_p), P, _dptr(d_c), C, _dptr(d_seg_off),
                               _dptr(d_seg_idx), pairs, _dptr(out), _stream())
        self._check(st, "ks_featurize")
        return out

    def score(self, d_features, model: Model, want_leaf_idx: bool = False):
        rows = d_features.shape[0]
        scores = torch.empty(rows, dtype=torch.float32, device=self.device)
        leaf = (torch.empty((rows, model.n_trees), dtype=torch.uint16, device=self.device)
                if want_leaf_idx else None)
        st = _lib.ks_score(self._h, _dptr(d_features), rows, model._h, _dptr(scores), _dptr(leaf),
                           _stream())
        self._check(st, "ks_score")
        return (scores, leaf) if want_leaf_idx else scores

    def debug_walk_floor(self, d_features, model: Model, repeat: int, out=None):
        """Measurement aid: the tree walk stripped to its gather stream (see ks_debug_walk_floor)."""
        rows = d_features.shape[0]
        if out is None:
            out = torch.empty(rows, dtype=torch.float32, device=self.device)
        st = _lib.ks_debug_walk_floor(self._h, _dptr(d_features), rows, model._h, int(repeat), _dptr(out), _stream())
        self._check(st, "ks_debug_walk_floor")
        return out

    def select(self, d_p, P, d_c, C, model: Model, k, d_seg_off=None, d_seg_idx=None, pairs=None,
               out_idx=None, out_score=None):
        pairs = P * C if pairs is None else pairs
        if out_idx is None:
            kk = max(int(k), 1)  # an invalid k is reported by the library, not by torch
            out_idx = torch.empty((P, kk), dtype=torch.int32, device=self.device)
            out_score = torch.empty((P, kk), dtype=torch.float32, device=self.device)
        st = _lib.ks_select(self._h, _dptr(d_p), P, _dptr(d_c), C, _dptr(d_seg_off), _dptr(d_seg_idx),
                            pairs, model._h, k, _dptr(out_idx), _dptr(out_score), _stream())
        self._check(st, "ks_select")
        return out_idx, out_score

    def merge_topk(self, d_idx, d_score, k, out_idx=None, out_score=None):
        """[P, n] gathered (index, score) entries -> the k best per problem, [P, k]."""
        P, n = d_idx.shape
        if out_idx is None:
            out_idx = torch.empty((P, k), dtype=torch.int32, device=self.device)
            out_score = torch.empty((P, k), dtype=torch.float32, device=self.device)
        st = _lib.ks_merge_topk(self._h, _dptr(d_idx), _dptr(d_score), P, n, k, _dptr(out_idx), _dptr(out_score),
                                _stream())
        self._check(st, "ks_merge_topk")
        return out_idx, out_score

    def catalogue_prepare(self, d_c, C, model: Model) -> Catalogue:
        h = ctypes.c_void_p()
        st = _lib.ks_catalogue_prepare(self._h, _dptr(d_c), C, model._h, ctypes.byref(h), _stream())
        self._check(st, "ks_catalogue_prepare")
        return Catalogue(self, h, d_c, C, model)

    def select_one_prepared(self, catalogue: Catalogue, problem: np.ndarray, k, h_idx=None, h_score=None):
        r = np.ascontiguousarray(problem).reshape(-1)[0]
        p = _Problem(int(r["m"]), int(r["n"]), int(r["k"]), int(r["layout"]), int(r["dtype_ab"]),
                     int(r["dtype_d"]), int(r["epi_flags"]))
        if h_idx is None:
            h_idx = torch.empty(k, dtype=torch.int32).pin_memory()
            h_score = torch.empty(k, dtype=torch.float32).pin_memory()
        st = _lib.ks_select_one_prepared(self._h, catalogue._h, p, k, _hptr(h_idx), _hptr(h_score), _stream())
        self._check(st, "ks_select_one_prepared")
        return h_idx, h_score

    def select_one_caller(self, d_c, C, model: Model, k, h_idx=None, h_score=None, catalogue: Catalogue = None):
        """For a stream of single problems: resolves the pointers, the model handle and the
        current stream once and returns f(p) -> (h_idx, h_score), where p is one element of
        `problem_structs(...)`. Per call only ks_select_one (ks_select_one_prepared when a prepared
        catalogue is given) itself runs; the result tensors are reused from call to call."""
        if h_idx is None:
            h_idx = torch.empty(k, dtype=torch.int32).pin_memory()
            h_score = torch.empty(k, dtype=torch.float32).pin_memory()
        check = self._check
        if catalogue is not None:
            fn = _lib.ks_select_one_prepared
            args = (k, _hptr(h_idx), _hptr(h_score), _stream())
            ctx_h, cat_h = self._h, catalogue._h
            keep = (catalogue, None, h_idx, h_score)

            def call_prepared(p):
                st = fn(ctx_h, cat_h, p, *args)
                if st != KS_OK:
                    check(st, "ks_select_one_prepared")
                return keep[2], keep[3]
            return call_prepared
        fn = _lib.ks_select_one
        args = (_dptr(d_c), C, model._h, k, _hptr(h_idx), _hptr(h_score), _stream())
        ctx_h = self._h
        keep = (d_c, model, h_idx, h_score)  # the closure keeps the buffers alive

        def call(p):
            st = fn(ctx_h, p, *args)
            if st != KS_OK:
                check(st, "ks_select_one")
            return keep[2], keep[3]
        return call

    def select_one(self, problem: np.ndarray, d_c, C, model: Model, k, h_idx=None, h_score=None):
        r = np.ascontiguousarray(problem).reshape(-1)[0]
        p = _Problem(int(r["m"]), int(r["n"]), int(r["k"]), int(r["layout"]), int(r["dtype_ab"]),
                     int(r["dtype_d"]), int(r["epi_flags"]))
        if h_idx is None:
            h_idx = torch.empty(k, dtype=torch.int32).pin_memory()
            h_score = torch.empty(k, dtype=torch.float32).pin_memory()
        st = _lib.ks_select_one(self._h, p, _dptr(d_c), C, model._h, k, _hptr(h_idx), _hptr(h_score),
                                _stream())
        self._check(st, "ks_select_one")
        return h_idx, h_score

    def select_host(self, h_p, P, h_c, C, model: Model, k, h_seg_off=None, h_seg_idx=None, pairs=None,
                    h_idx=None, h_score=None):
        pairs = P * C if pairs is None else pairs
        if h_idx is None:
            h_idx = torch.empty((P, k), dtype=torch.int32).pin_memory()
            h_score = torch.empty((P, k), dtype=torch.float32).pin_memory()
        st = _lib.ks_select_host(self._h, _hptr(h_p), P, _hptr(h_c), C, _hptr(h_seg_off),
                                 _hptr(h_seg_idx), pairs, model._h, k, _hptr(h_idx), _hptr(h_score),
                                 _stream())
        self._check(st, "ks_select_host")
        return h_idx, h_score

    # ---- search space and validity ----------------------------------------------------------
    def enumerate(self, first: int, count: int, out=None):
        """Candidates with search-space ids first .. first+count-1 as a [count, 16] uint8 tensor."""
        if out is None:
            out = torch.empty((max(int(count), 0), 16), dtype=torch.uint8, device=self.device)
        self._check(_lib.ks_enumerate(self._h, first, count, _dptr(out), _stream()), "ks_enumerate")
        return out

    def valid_catalogue(self, problem: np.ndarray, flags: int, d_c=None, C=None, want_records=True,
                        want_index=True, sync=True):
        """Validity filter + compaction. Returns (records [C,16] u8 or None, index [C] i32 or
        None, count); count is an int when sync, else a 1-element device tensor, and only the
        first `count` entries of the outputs are meaningful."""
        r = np.ascontiguousarray(problem).reshape(-1)[0]
        p = _Problem(int(r["m"]), int(r["n"]), int(r["k"]), int(r["layout"]), int(r["dtype_ab"]),
                     int(r["dtype_d"]), int(r["epi_flags"]))
        C = (KS_CATALOGUE_SIZE if d_c is None else d_c.shape[0]) if C is None else int(C)
        cap = max(C, 0)
        out = torch.empty((cap, 16), dtype=torch.uint8, device=self.device) if want_records else None
        idx = torch.empty(cap, dtype=torch.int32, device=self.device) if want_index else None
        d_count = torch.zeros(1, dtype=torch.int32, device=self.device)
        h_count = ctypes.c_int32(-1)
        st = _lib.ks_valid_catalogue(self._h, ctypes.byref(p), flags, _dptr(d_c), C, _dptr(out), _dptr(idx),
                                     _dptr(d_count), ctypes.byref(h_count) if sync else None, _stream())
        self._check(st, "ks_valid_catalogue")
        return out, idx, (int(h_count.value) if sync else d_count)

    def remap_indices(self, d_idx, d_map, map_len=None):
        n = d_idx.numel()
        map_len = d_map.numel() if map_len is None else int(map_len)
        self._check(_lib.ks_remap_indices(self._h, _dptr(d_idx), n, _dptr(d_map), map_len, _stream()),
                    "ks_remap_indices")
        return d_idx
