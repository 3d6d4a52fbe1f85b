"""ctypes binding of libqgbdt.so: the same calls as include/qgbdt.h, argument marshalling only.

Tensors are torch CUDA tensors (used as device memory); every step of the method runs in the
library's kernels.  Loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqgbdt.so")

OK, ERR_ARG, ERR_STATE, ERR_OVERFLOW, ERR_CUDA, ERR_ALLOC, ERR_VALUE = 0, -1, -2, -3, -4, -5, -6
OPT_COLUMN_COPY = 1
OPT_LEAF_VALUES = 2
INFO_COLUMN_COPY = 1

EXPORTS = [
    "qgbdt_create", "qgbdt_destroy", "qgbdt_last_error", "qgbdt_load_binned", "qgbdt_load_binned_host",
    "qgbdt_compute_gradients", "qgbdt_quantize_gradients", "qgbdt_build_histograms",
    "qgbdt_build_histograms_rows", "qgbdt_build_histograms_fp32", "qgbdt_subtract_histograms", "qgbdt_find_best_split", "qgbdt_split_leaf",
    "qgbdt_get_leaf_rows", "qgbdt_reset_leaves", "qgbdt_refit_leaves", "qgbdt_apply_leaf_values", "qgbdt_train", "qgbdt_train_host",
    "qgbdt_set_distributed", "qgbdt_set_option", "qgbdt_get_info", "qgbdt_get_counters", "qgbdt_profile_histograms", "qgbdt_get_histogram_profile", "qgbdt_get_timings",
    "qgbdt_build_histograms_noalloc", "qgbdt_noalloc_last_error",
]


class QgbdtError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("qgbdt error %d: %s" % (code, msg))
        self.code = code


class Params(C.Structure):
    _fields_ = [("bits", C.c_int32), ("objective", C.c_int32), ("num_leaves", C.c_int32),
                ("num_trees", C.c_int32), ("min_data_in_leaf", C.c_int32),
                ("learning_rate", C.c_double), ("lambda_l2", C.c_double),
                ("min_sum_hessian", C.c_double), ("min_gain", C.c_double), ("seed", C.c_uint64),
                ("hess_levels_mode", C.c_int32), ("rounding", C.c_int32)]


class Split(C.Structure):
    _fields_ = [("feature", C.c_int32), ("bin", C.c_int32), ("gain", C.c_double),
                ("gl", C.c_int64), ("hl", C.c_int64), ("gr", C.c_int64), ("hr", C.c_int64),
                ("nl_est", C.c_int64), ("nr_est", C.c_int64), ("valid", C.c_int32)]


class Model(C.Structure):
    _fields_ = [("num_leaves", C.POINTER(C.c_int32)), ("feature", C.POINTER(C.c_int32)),
                ("bin", C.POINTER(C.c_int32)), ("left", C.POINTER(C.c_int32)),
                ("right", C.POINTER(C.c_int32)), ("gain", C.POINTER(C.c_double)),
                ("leaf_value", C.POINTER(C.c_float)), ("leaf_count", C.POINTER(C.c_int64))]


_lib = None


def load_library() -> C.CDLL:
    """Loads libqgbdt.so; raises if it is missing (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libqgbdt.so is not built: run `python -m paper_2207_09682_b200.build` "
                              "(or __graft_entry__.build()); the CUDA library is the only implementation")
        lib = C.CDLL(LIB_PATH)
        lib.qgbdt_last_error.restype = C.c_char_p
        lib.qgbdt_last_error.argtypes = [C.c_void_p]
        _lib = lib
    return _lib


def make_params(bits=3, objective=0, num_leaves=31, num_trees=1, min_data_in_leaf=20, learning_rate=0.1,
                lambda_l2=0.0, min_sum_hessian=0.0, min_gain=0.0, seed=1, hess_levels_mode=0,
                rounding=0) -> Params:
    return Params(bits, objective, num_leaves, num_trees, min_data_in_leaf, learning_rate, lambda_l2,
                  min_sum_hessian, min_gain, seed, hess_levels_mode, rounding)


def _dptr(t):
    if t is None:
        return C.c_void_p(None)
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


class _DeviceView:
    """CUDA array interface over borrowed device memory holding n 32-bit words."""

    def __init__(self, ptr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<i4", "data": (ptr, False), "version": 2}


class HostModel:
    """Host arrays for the trees written by qgbdt_train."""

    def __init__(self, num_trees: int, num_leaves: int):
        L = num_leaves
        self.num_trees, self.L = num_trees, L
        self.num_leaves = np.zeros(num_trees, np.int32)
        n_nodes = max(num_trees * (L - 1), 1)
        self.feature = np.full(n_nodes, -1, np.int32)
        self.bin = np.full(n_nodes, -1, np.int32)
        self.left = np.zeros(n_nodes, np.int32)
        self.right = np.zeros(n_nodes, np.int32)
        self.gain = np.zeros(n_nodes, np.float64)
        self.leaf_value = np.zeros(num_trees * L, np.float32)
        self.leaf_count = np.zeros(num_trees * L, np.int64)

    def struct(self) -> Model:
        p = lambda a, t: a.ctypes.data_as(C.POINTER(t))
        return Model(p(self.num_leaves, C.c_int32), p(self.feature, C.c_int32), p(self.bin, C.c_int32),
                     p(self.left, C.c_int32), p(self.right, C.c_int32), p(self.gain, C.c_double),
                     p(self.leaf_value, C.c_float), p(self.leaf_count, C.c_int64))

    def tree(self, k: int) -> dict:
        L, nl = self.L, int(self.num_leaves[k])
        s = slice(k * (L - 1), k * (L - 1) + nl - 1)
        return dict(num_leaves=nl, feature=self.feature[s], bin=self.bin[s], left=self.left[s],
                    right=self.right[s], gain=self.gain[s], leaf_value=self.leaf_value[k * L:k * L + nl],
                    leaf_count=self.leaf_count[k * L:k * L + nl])


class Context:
    """One qgbdt_ctx; methods are the C calls of include/qgbdt.h with the prefix dropped."""

    def __init__(self, params: Params):
        self.lib = load_library()
        self.params = params
        self.h = C.c_void_p()
        rc = self.lib.qgbdt_create(C.byref(self.h), C.byref(params))
        if rc != OK:
            raise QgbdtError(rc, "qgbdt_create failed")
        self.n_rows = self.n_features = self.n_bins = 0

    def close(self):
        if self.h:
            self.lib.qgbdt_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != OK:
            raise QgbdtError(rc, self.lib.qgbdt_last_error(self.h).decode())

    def load_binned(self, bins: torch.Tensor, n_bins: int, layout: int = 0, stream=None):
        """bins: uint8 [N, F] (layout 0) or [F, N] (layout 1); CUDA tensor, or CPU tensor (host variant)."""
        assert bins.dtype == torch.uint8 and bins.dim() == 2 and bins.is_contiguous()
        n, f = (bins.shape if layout == 0 else (bins.shape[1], bins.shape[0]))
        ld = bins.shape[1]
        if bins.is_cuda:
            rc = self.lib.qgbdt_load_binned(self.h, _dptr(bins), C.c_int64(n), C.c_int32(f), C.c_int32(n_bins),
                                            C.c_int32(layout), C.c_int64(ld), _stream(stream))
        else:
            rc = self.lib.qgbdt_load_binned_host(self.h, C.c_void_p(bins.data_ptr()), C.c_int64(n), C.c_int32(f),
                                                 C.c_int32(n_bins), C.c_int32(layout), C.c_int64(ld),
                                                 _stream(stream))
        self._check(rc)
        self.n_rows, self.n_features, self.n_bins = n, f, n_bins

    def compute_gradients(self, scores, labels, g, h=None, stream=None):
        self._check(self.lib.qgbdt_compute_gradients(self.h, _dptr(scores), _dptr(labels), _dptr(g), _dptr(h),
                                                     _stream(stream)))

    def quantize_gradients(self, g, h=None, tree=0, gq=None, hq=None, stream=None) -> dict:
        gs, hs = C.c_double(), C.c_double()
        G, H = C.c_int64(), C.c_int64()
        self._check(self.lib.qgbdt_quantize_gradients(self.h, _dptr(g), _dptr(h), C.c_uint32(tree), _dptr(gq),
                                                      _dptr(hq), C.byref(gs), C.byref(hs), C.byref(G), C.byref(H),
                                                      _stream(stream)))
        return dict(g_scale=gs.value, h_scale=hs.value, G_total=G.value, H_total=H.value)

    def new_hist(self) -> torch.Tensor:
        """Device buffer for one histogram: int64 [F, n_bins], word = G * 2^32 + H."""
        return torch.empty((self.n_features, self.n_bins), dtype=torch.int64, device="cuda")

    def build_histograms(self, leaf: int, hist: torch.Tensor, stream=None):
        self._check(self.lib.qgbdt_build_histograms(self.h, C.c_int32(leaf), _dptr(hist), _stream(stream)))

    def build_histograms_rows(self, rows: torch.Tensor, hist: torch.Tensor, stream=None):
        assert rows.dtype in (torch.int32, torch.uint32)
        self._check(self.lib.qgbdt_build_histograms_rows(self.h, _dptr(rows), C.c_int64(rows.numel()), _dptr(hist),
                                                         _stream(stream)))

    def build_histograms_fp32(self, g, h=None, rows=None, stream=None) -> torch.Tensor:
        """Floating-point histogram of the original gradients: float32 [F, n_bins, 2] (gradient sum, hessian sum)."""
        assert g.dtype == torch.float32 and g.numel() == self.n_rows and (h is None or h.dtype == torch.float32)
        hist = torch.empty((self.n_features, self.n_bins, 2), dtype=torch.float32, device="cuda")
        n = self.n_rows if rows is None else rows.numel()
        self._check(self.lib.qgbdt_build_histograms_fp32(self.h, _dptr(g), _dptr(h), _dptr(rows), C.c_int64(n),
                                                         _dptr(hist), _stream(stream)))
        return hist

    def subtract_histograms(self, parent, small, large, stream=None):
        self._check(self.lib.qgbdt_subtract_histograms(self.h, _dptr(parent), _dptr(small), _dptr(large),
                                                       _stream(stream)))

    def find_best_split(self, hist, G: int, H: int, n_rows: int, stream=None) -> Split:
        out = Split()
        self._check(self.lib.qgbdt_find_best_split(self.h, _dptr(hist), C.c_int64(G), C.c_int64(H),
                                                   C.c_int64(n_rows), C.byref(out), _stream(stream)))
        return out

    def split_leaf(self, leaf: int, feature: int, bin_: int, stream=None) -> tuple[int, int, int]:
        r, nl, nr = C.c_int32(), C.c_int64(), C.c_int64()
        self._check(self.lib.qgbdt_split_leaf(self.h, C.c_int32(leaf), C.c_int32(feature), C.c_int32(bin_),
                                              C.byref(r), C.byref(nl), C.byref(nr), _stream(stream)))
        return r.value, nl.value, nr.value

    def get_leaf_rows(self, leaf: int) -> torch.Tensor:
        """Copy of the leaf's row list as an int64 CPU tensor (the device view is borrowed)."""
        p, n = C.c_void_p(), C.c_int64()
        self._check(self.lib.qgbdt_get_leaf_rows(self.h, C.c_int32(leaf), C.byref(p), C.byref(n)))
        torch.cuda.synchronize()
        if n.value == 0:
            return torch.zeros(0, dtype=torch.int64)
        view = torch.as_tensor(_DeviceView(p.value, n.value), device="cuda")   # int32 bits of uint32 rows
        return (view.cpu().to(torch.int64) & 0xFFFFFFFF)

    def reset_leaves(self, stream=None):
        self._check(self.lib.qgbdt_reset_leaves(self.h, _stream(stream)))

    def refit_leaves(self, g, h=None, n_leaves: int = None, stream=None) -> tuple[np.ndarray, np.ndarray]:
        L = self.params.num_leaves
        w = np.zeros(L, np.float64)
        v = np.zeros(L, np.float32)
        self._check(self.lib.qgbdt_refit_leaves(self.h, _dptr(g), _dptr(h), w.ctypes.data_as(C.c_void_p),
                                                v.ctypes.data_as(C.c_void_p), _stream(stream)))
        return (w, v) if n_leaves is None else (w[:n_leaves], v[:n_leaves])

    def apply_leaf_values(self, scores, stream=None):
        self._check(self.lib.qgbdt_apply_leaf_values(self.h, _dptr(scores), _stream(stream)))

    def train(self, labels, scores, first_tree: int, num_trees: int, stream=None) -> HostModel:
        """labels / scores: float32 [N]; CUDA tensors, or CPU tensors (host variant, scores updated in place)."""
        model = HostModel(num_trees, self.params.num_leaves)
        ms = model.struct()
        if labels.is_cuda:
            rc = self.lib.qgbdt_train(self.h, _dptr(labels), _dptr(scores), C.c_uint32(first_tree),
                                      C.c_int32(num_trees), C.byref(ms), _stream(stream))
        else:
            assert scores.is_contiguous() and labels.is_contiguous()
            rc = self.lib.qgbdt_train_host(self.h, C.c_void_p(labels.data_ptr()), C.c_void_p(scores.data_ptr()),
                                           C.c_uint32(first_tree), C.c_int32(num_trees), C.byref(ms),
                                           _stream(stream))
        self._check(rc)
        return model

    def set_distributed(self, rank: int, world: int, row_offset: int, total_rows: int, callback):
        """callback: a dist.ALLREDUCE_FN instance (kept alive by this object); None switches the mode off."""
        self._reduce_cb = callback
        self._check(self.lib.qgbdt_set_distributed(self.h, C.c_int32(rank), C.c_int32(world), C.c_int64(row_offset),
                                                   C.c_int64(total_rows), callback if callback is not None else None,
                                                   None))

    def set_option(self, option: int, value: int):
        self._check(self.lib.qgbdt_set_option(self.h, C.c_int32(option), C.c_int64(value)))

    def get_info(self, what: int) -> int:
        v = C.c_int64()
        self._check(self.lib.qgbdt_get_info(self.h, C.c_int32(what), C.byref(v)))
        return v.value

    def get_counters(self) -> dict:
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        self._check(self.lib.qgbdt_get_counters(self.h, C.byref(a), C.byref(b), C.byref(c)))
        return dict(kernel_launches=a.value, hist_builds=b.value, hist_row_features=c.value)


def _profile_histograms(self, enable: bool):
    self._check(self.lib.qgbdt_profile_histograms(self.h, C.c_int32(1 if enable else 0)))


def _get_histogram_profile(self) -> dict:
    ms, nbytes, builds = C.c_double(), C.c_int64(), C.c_int64()
    self._check(self.lib.qgbdt_get_histogram_profile(self.h, C.byref(ms), C.byref(nbytes), C.byref(builds)))
    return dict(total_ms=ms.value, total_bytes=nbytes.value, builds=builds.value)


PHASES = ("gradients", "quantize", "root_histogram", "partition", "child_histograms", "finish", "commit",
          "leaf_values", "score_update")


def _get_timings(self) -> dict:
    ms = (C.c_double * len(PHASES))()
    cnt = (C.c_int64 * len(PHASES))()
    self._check(self.lib.qgbdt_get_timings(self.h, ms, cnt))
    return {name: dict(ms=ms[i], intervals=cnt[i]) for i, name in enumerate(PHASES)}


Context.get_timings = _get_timings
Context.profile_histograms = _profile_histograms
Context.get_histogram_profile = _get_histogram_profile


def build_histograms_noalloc(bins: torch.Tensor, n_bins: int, gq: torch.Tensor, hq: torch.Tensor,
                             hist: torch.Tensor, rows: torch.Tensor = None, status: torch.Tensor = None, stream=None):
    """The context-free, allocation-free histogram call: bins uint8 [N, F] row-major, gq int8 [N],
    hq uint8 [N], hist int64 [F, n_bins] (overwritten), rows optional int32 list.  Marshalling only."""
    lib = load_library()
    lib.qgbdt_noalloc_last_error.restype = C.c_char_p
    # the C call takes raw pointers: a wrong dtype, a host tensor or a transposed view would be read as garbage
    assert bins.is_cuda and bins.dtype == torch.uint8 and bins.dim() == 2 and bins.stride(1) == 1
    assert gq.is_cuda and gq.dtype == torch.int8 and gq.is_contiguous() and gq.numel() == bins.shape[0]
    assert hq.is_cuda and hq.dtype == torch.uint8 and hq.is_contiguous() and hq.numel() == bins.shape[0]
    assert hist.is_cuda and hist.dtype == torch.int64 and hist.is_contiguous() and hist.numel() == bins.shape[1] * n_bins
    assert rows is None or (rows.is_cuda and rows.dtype in (torch.int32, torch.uint32) and rows.is_contiguous())
    assert status is None or (status.is_cuda and status.dtype == torch.int32)
    n_rows, f = bins.shape
    n = n_rows if rows is None else rows.numel()
    rc = lib.qgbdt_build_histograms_noalloc(C.c_void_p(bins.data_ptr()), C.c_int64(n_rows), C.c_int32(f), C.c_int32(n_bins),
                                            C.c_int64(bins.stride(0)), _dptr(gq), _dptr(hq), _dptr(rows), C.c_int64(n),
                                            _dptr(hist), _dptr(status), _stream(stream))
    if rc != OK:
        raise QgbdtError(rc, lib.qgbdt_noalloc_last_error().decode())


def unpack_hist(hist: torch.Tensor) -> tuple[np.ndarray, np.ndarray]:
    """Splits packed histogram words into (G, H) int64 arrays on the host."""
    w = hist.detach().cpu().numpy().astype(np.int64)
    return w >> 32, w & 0xFFFFFFFF
