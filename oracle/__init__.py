"""CPU oracle for quantized GBDT training -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrappers (numpy in, numpy out) around ``qgbdt_oracle.c``, the plain C
statement of the method.  Only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA product path never does, and
this package never imports the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qgbdt_oracle.c")
_LIB = os.path.join(_HERE, "libqgbdt_oracle.so")

OK = 0
ERR_ARG = -1
ERR_VALUE = -6


def build(force: bool = False) -> str:
    """Compile the oracle with contraction and fast-math off; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
             _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


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


def make_params(bits=3, objective=0, num_leaves=31, num_trees=1, min_data_in_leaf=20,
                learning_rate=0.1, lambda_l2=0.0, min_sum_hessian=0.0, min_gain=0.0, seed=1,
                hess_levels_mode=0, rounding=0) -> Params:
    return Params(bits, objective, num_leaves, num_trees, min_data_in_leaf, learning_rate, lambda_l2,
                  min_sum_hessian, min_gain, seed, hess_levels_mode, rounding)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.qo_gain.restype = C.c_double
        _lib.qo_gain.argtypes = [C.c_int64] * 4 + [C.c_double] * 3
        _lib.qo_sigmoid.restype = C.c_float
        _lib.qo_sigmoid.argtypes = [C.c_float]
        _lib.qo_partition.restype = C.c_int64
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def levels(bits: int, hess_levels_mode: int = 0) -> tuple[int, int]:
    return lib().qo_levels_g(bits), lib().qo_levels_h(bits, hess_levels_mode)


def sr_uniforms(seed: int, tree: int, row0: int, n: int) -> tuple[np.ndarray, np.ndarray]:
    """24-bit uniforms (u_g, u_h) of rows row0 .. row0+n-1."""
    ug = np.empty(n, np.uint32)
    uh = np.empty(n, np.uint32)
    lib().qo_sr_uniforms_range(C.c_uint64(seed), C.c_uint32(tree), C.c_uint32(row0), C.c_int64(n),
                               _p(ug, C.c_uint32), _p(uh, C.c_uint32))
    return ug, uh


@dataclass
class Quantized:
    gq: np.ndarray  # int8 [n]
    hq: np.ndarray  # uint8 [n]
    gmax: float
    hmax: float


def quantize(g, h, bits, seed=1, tree=0, hess_levels_mode=0, rounding=0) -> Quantized:
    g = _c(g, np.float32)
    h = None if h is None else _c(h, np.float32)
    n = g.shape[0]
    gq = np.empty(n, np.int8)
    hq = np.empty(n, np.uint8)
    gm, hm = C.c_float(), C.c_float()
    rc = lib().qo_quantize(_p(g, C.c_float), _p(h, C.c_float), C.c_int64(n), bits, hess_levels_mode,
                           rounding, C.c_uint64(seed), C.c_uint32(tree), _p(gq, C.c_int8),
                           _p(hq, C.c_uint8), C.byref(gm), C.byref(hm))
    if rc != OK:
        raise ValueError("qo_quantize failed: %d" % rc)
    return Quantized(gq, hq, gm.value, hm.value)


def histogram(data, n_bins, gq, hq, idx=None) -> tuple[np.ndarray, np.ndarray]:
    data = _c(data, np.uint8)
    n, J = data.shape
    gq = _c(gq, np.int8)
    hq = _c(hq, np.uint8)
    if idx is not None:
        idx = _c(idx, np.uint32)
    n_s = n if idx is None else idx.shape[0]
    hg = np.empty((J, n_bins), np.int64)
    hh = np.empty((J, n_bins), np.int64)
    rc = lib().qo_histogram(_p(data, C.c_uint8), C.c_int64(n), J, n_bins, _p(gq, C.c_int8),
                            _p(hq, C.c_uint8), _p(idx, C.c_uint32), C.c_int64(n_s),
                            _p(hg, C.c_int64), _p(hh, C.c_int64))
    if rc != OK:
        raise ValueError("qo_histogram failed: %d" % rc)
    return hg, hh


def histogram_fp(data, n_bins, g, h=None, idx=None) -> tuple[np.ndarray, np.ndarray]:
    """Algorithm 1 with the original gradients, float64 sums: (hist_g, hist_h), each [J, n_bins]."""
    data = _c(data, np.uint8)
    n, J = data.shape
    g = _c(g, np.float32)
    h = None if h is None else _c(h, np.float32)
    if idx is not None:
        idx = _c(idx, np.uint32)
    n_s = n if idx is None else idx.shape[0]
    hg = np.empty((J, n_bins), np.float64)
    hh = np.empty((J, n_bins), np.float64)
    rc = lib().qo_histogram_fp(_p(data, C.c_uint8), C.c_int64(n), J, n_bins, _p(g, C.c_float), _p(h, C.c_float),
                               _p(idx, C.c_uint32), C.c_int64(n_s), _p(hg, C.c_double), _p(hh, C.c_double))
    if rc != OK:
        raise ValueError("qo_histogram_fp failed: %d" % rc)
    return hg, hh


def gain(gl, hl, gr, hr, dg, dh, lambda_l2=0.0) -> float:
    return lib().qo_gain(gl, hl, gr, hr, dg, dh, lambda_l2)


def find_split(hist_g, hist_h, G, H, n_s, gmax, hmax, const_hessian, params: Params) -> Split:
    hist_g = _c(hist_g, np.int64)
    hist_h = _c(hist_h, np.int64)
    J, nb = hist_g.shape
    out = Split()
    rc = lib().qo_find_split(_p(hist_g, C.c_int64), _p(hist_h, C.c_int64), J, nb, C.c_int64(int(G)),
                             C.c_int64(int(H)), C.c_int64(int(n_s)), C.c_float(gmax), C.c_float(hmax),
                             int(bool(const_hessian)), C.byref(params), C.byref(out))
    if rc != OK:
        raise ValueError("qo_find_split failed: %d" % rc)
    return out


def partition(data, idx, feature, bin_) -> tuple[np.ndarray, int]:
    data = _c(data, np.uint8)
    idx = _c(idx, np.uint32)
    out = np.empty_like(idx)
    nl = lib().qo_partition(_p(data, C.c_uint8), data.shape[1], _p(idx, C.c_uint32),
                            C.c_int64(idx.shape[0]), feature, bin_, _p(out, C.c_uint32))
    return out, int(nl)


def refit(g, h, idx, lambda_l2=0.0, learning_rate=1.0) -> tuple[float, float]:
    g = _c(g, np.float32)
    h = None if h is None else _c(h, np.float32)
    idx = _c(idx, np.uint32)
    w, v = C.c_double(), C.c_float()
    lib().qo_refit(_p(g, C.c_float), _p(h, C.c_float), _p(idx, C.c_uint32), C.c_int64(idx.shape[0]),
                   C.c_double(lambda_l2), C.c_double(learning_rate), C.byref(w), C.byref(v))
    return w.value, v.value


def leaf_value_quantized(G, H, gmax, hmax, bits, hess_levels_mode=0, const_hessian=False, lambda_l2=0.0,
                         learning_rate=1.0) -> tuple[float, float]:
    w, v = C.c_double(), C.c_float()
    lib().qo_leaf_value_quantized(C.c_int64(int(G)), C.c_int64(int(H)), C.c_float(gmax), C.c_float(hmax), bits,
                                  hess_levels_mode, int(bool(const_hessian)), C.c_double(lambda_l2),
                                  C.c_double(learning_rate), C.byref(w), C.byref(v))
    return w.value, v.value


def sigmoid(s: float) -> float:
    return lib().qo_sigmoid(C.c_float(s))


def gradients(objective, scores, labels) -> tuple[np.ndarray, np.ndarray | None]:
    scores = _c(scores, np.float32)
    labels = _c(labels, np.float32)
    n = scores.shape[0]
    g = np.empty(n, np.float32)
    h = np.empty(n, np.float32) if objective == 0 else None
    lib().qo_gradients(objective, _p(scores, C.c_float), _p(labels, C.c_float), C.c_int64(n),
                       _p(g, C.c_float), _p(h, C.c_float))
    return g, h


@dataclass
class Tree:
    num_leaves: int
    feature: np.ndarray
    bin: np.ndarray
    left: np.ndarray
    right: np.ndarray
    gain: np.ndarray
    leaf_value: np.ndarray
    leaf_count: np.ndarray


def train_tree(data, n_bins, labels, scores, params: Params, tree: int, want_row_leaf=False, refit=True):
    """One boosting iteration; ``scores`` (float32) is updated in place.  refit=False: leaf values from
    the quantized sums (Sec. 4.2) instead of the original gradients."""
    data = _c(data, np.uint8)
    labels = _c(labels, np.float32)
    assert scores.dtype == np.float32 and scores.flags.c_contiguous
    n, J = data.shape
    L = params.num_leaves
    nf = np.full(max(L - 1, 1), -1, np.int32)
    nbn = np.full(max(L - 1, 1), -1, np.int32)
    nl = np.zeros(max(L - 1, 1), np.int32)
    nr = np.zeros(max(L - 1, 1), np.int32)
    ng = np.zeros(max(L - 1, 1), np.float64)
    lv = np.zeros(L, np.float32)
    lc = np.zeros(L, np.int64)
    rl = np.empty(n, np.int32) if want_row_leaf else None
    rc = lib().qo_train_tree_opt(_p(data, C.c_uint8), C.c_int64(n), J, n_bins, _p(labels, C.c_float),
                             _p(scores, C.c_float), C.byref(params), C.c_uint32(tree), 0 if refit else 1,
                             _p(nf, C.c_int32), _p(nbn, C.c_int32), _p(nl, C.c_int32),
                             _p(nr, C.c_int32), _p(ng, C.c_double), _p(lv, C.c_float),
                             _p(lc, C.c_int64), _p(rl, C.c_int32))
    if rc < 0:
        raise ValueError("qo_train_tree failed: %d" % rc)
    t = Tree(rc, nf[:rc - 1], nbn[:rc - 1], nl[:rc - 1], nr[:rc - 1], ng[:rc - 1], lv[:rc], lc[:rc])
    return (t, rl) if want_row_leaf else t


def train(data, n_bins, labels, scores, params: Params) -> list[Tree]:
    return [train_tree(data, n_bins, labels, scores, params, k) for k in range(params.num_trees)]


def predict_leaf(data, tree: Tree) -> np.ndarray:
    data = _c(data, np.uint8)
    out = np.empty(data.shape[0], np.int32)
    f = lib().qo_predict_leaf
    nf, nbn, nl, nr = (_c(a, np.int32) for a in (tree.feature, tree.bin, tree.left, tree.right))
    for i in range(data.shape[0]):
        out[i] = f(_p(data[i], C.c_uint8), tree.num_leaves, _p(nf, C.c_int32), _p(nbn, C.c_int32),
                   _p(nl, C.c_int32), _p(nr, C.c_int32))
    return out
