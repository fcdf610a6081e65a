"""ctypes front-end of the CPU checker (oracle/ocs_oracle.c).

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by the bench's
CPU-baseline leg; never by the CUDA library or its Python binding.  All arithmetic lives in
the C file; this module only builds it, marshals numpy arrays and allocates outputs.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ocs_oracle.c")
_LIB = os.path.join(_HERE, "libocs_oracle.so")
_lib = None

_f32p = C.POINTER(C.c_float)
_i32p = C.POINTER(C.c_int32)
_i8p = C.POINTER(C.c_int8)
_u64p = C.POINTER(C.c_uint64)
_f64p = C.POINTER(C.c_double)


def build(force: bool = False) -> str:
    """Compile the checker with gcc (no fast-math, no FMA contraction)."""
    hdr = os.path.join(_HERE, "ocs_oracle.h")
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= max(os.path.getmtime(_SRC), os.path.getmtime(hdr))):
        return _LIB
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
           "-fPIC", "-o", _LIB + ".tmp", _SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ocs_oracle_maxabs.restype = C.c_float
        _lib.ocs_oracle_sigmoid.restype = C.c_float
        _lib.ocs_oracle_tanh.restype = C.c_float
        _lib.ocs_oracle_sigmoid.argtypes = [C.c_float]
        _lib.ocs_oracle_tanh.argtypes = [C.c_float]
        _lib.ocs_oracle_num_splits.argtypes = [C.c_int, C.c_double]
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(t)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def threads() -> int:
    """Threads the OpenMP-parallel contractions use."""
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


def num_splits(Cn: int, ratio: float) -> int:
    return int(lib().ocs_oracle_num_splits(int(Cn), float(ratio)))


def split(W, S: int, qa_step: float = 0.0, literal: bool = False):
    """W [O, C] or [O, C, kh, kw] -> (W' [O, C+S, ...], idx_map, split_order, (max|W|, max|W'|))."""
    W = _f32(W)
    O, Cn = W.shape[0], W.shape[1]
    R = int(np.prod(W.shape[2:])) if W.ndim > 2 else 1
    out = np.empty((O, Cn + S) + tuple(W.shape[2:]), dtype=np.float32)
    idx = np.empty(Cn + S, dtype=np.int32)
    order = np.empty(max(S, 1), dtype=np.int32)
    mx = np.zeros(2, dtype=np.float32)
    fn = lib().ocs_oracle_split_literal if literal else lib().ocs_oracle_split_cached
    rc = fn(_p(W, _f32p), O, Cn, R, int(S), C.c_float(qa_step), _p(out, _f32p), _p(idx, _i32p),
            _p(order, _i32p), _p(mx, _f32p))
    _check(rc, "split")
    return out, idx, order[:S], (float(mx[0]), float(mx[1]))


def maxabs(T) -> float:
    T = _f32(T)
    return float(lib().ocs_oracle_maxabs(_p(T, _f32p), C.c_int64(T.size)))


def quantize(T, bits: int, is_signed: bool, alpha: float):
    """-> (codes int8/uint8 with T's shape, scale)."""
    T = _f32(T)
    codes = np.empty(T.shape, dtype=np.int8)
    scale = C.c_float(0)
    rc = lib().ocs_oracle_quantize(_p(T, _f32p), C.c_int64(T.size), int(bits), int(bool(is_signed)),
                                   C.c_float(alpha), _p(codes, _i8p), C.byref(scale))
    _check(rc, "quantize")
    return (codes if is_signed else codes.view(np.uint8)), float(scale.value)


def clip_mse(T, bits: int, is_signed: bool = True, n_bins: int = 2048, n_candidates: int = 128):
    """-> dict(alpha, max_abs, hist uint64 [n_bins], scores float64 [n_candidates])."""
    T = _f32(T)
    hist = np.zeros(n_bins, dtype=np.uint64)
    scores = np.zeros(n_candidates, dtype=np.float64)
    alpha, mx = C.c_float(0), C.c_float(0)
    rc = lib().ocs_oracle_clip_mse(_p(T, _f32p), C.c_int64(T.size), int(bits), int(bool(is_signed)),
                                   int(n_bins), int(n_candidates), C.byref(alpha), C.byref(mx),
                                   _p(hist, _u64p), _p(scores, _f64p))
    _check(rc, "clip_mse")
    return dict(alpha=float(alpha.value), max_abs=float(mx.value), hist=hist, scores=scores)


def clip_mse_exact(T, bits: int, is_signed: bool = True, n_candidates: int = 128):
    T = _f32(T)
    scores = np.zeros(n_candidates, dtype=np.float64)
    alpha = C.c_float(0)
    rc = lib().ocs_oracle_clip_mse_exact(_p(T, _f32p), C.c_int64(T.size), int(bits),
                                         int(bool(is_signed)), int(n_candidates), C.byref(alpha),
                                         _p(scores, _f64p))
    _check(rc, "clip_mse_exact")
    return dict(alpha=float(alpha.value), scores=scores)


def split_qa(W, S: int, qa_bits: int):
    """Split with the two-pass grid-step rule -> (W', idx_map, split_order, (max|W|, max|W'|), qa_step)."""
    W = _f32(W)
    O, Cn = W.shape[0], W.shape[1]
    R = int(np.prod(W.shape[2:])) if W.ndim > 2 else 1
    out = np.empty((O, Cn + S) + tuple(W.shape[2:]), dtype=np.float32)
    idx = np.empty(Cn + S, dtype=np.int32)
    order = np.empty(max(S, 1), dtype=np.int32)
    mx = np.zeros(3, dtype=np.float32)
    rc = lib().ocs_oracle_split_qa(_p(W, _f32p), O, Cn, R, int(S), int(qa_bits), _p(out, _f32p), _p(idx, _i32p),
                                   _p(order, _i32p), _p(mx, _f32p))
    _check(rc, "split_qa")
    return out, idx, order[:S], (float(mx[0]), float(mx[1])), float(mx[2])


def clip_kl(T, bits: int, is_signed: bool = True, n_bins: int = 2048, n_candidates: int = 128):
    """-> dict(alpha, max_abs, hist, scores) of the KL-divergence search (Section 4.3)."""
    T = _f32(T)
    hist = np.zeros(n_bins, dtype=np.uint64)
    scores = np.zeros(n_candidates, dtype=np.float64)
    alpha, mx = C.c_float(0), C.c_float(0)
    rc = lib().ocs_oracle_clip_kl(_p(T, _f32p), C.c_int64(T.size), int(bits), int(bool(is_signed)), int(n_bins),
                                  int(n_candidates), C.byref(alpha), C.byref(mx), _p(hist, _u64p), _p(scores, _f64p))
    _check(rc, "clip_kl")
    return dict(alpha=float(alpha.value), max_abs=float(mx.value), hist=hist, scores=scores)


def aciq_multiplier(n_intervals: float, laplace: bool) -> float:
    fn = lib().ocs_oracle_aciq_multiplier
    fn.restype = C.c_double
    fn.argtypes = [C.c_double, C.c_int]
    return float(fn(float(n_intervals), int(bool(laplace))))


def clip_aciq(T, bits: int, is_signed: bool = True, n_bins: int = 2048):
    """-> dict(alpha, max_abs, hist, b, sigma, laplace, multiplier) of the ACIQ threshold (Section 4.2)."""
    T = _f32(T)
    hist = np.zeros(n_bins, dtype=np.uint64)
    stats = np.zeros(4, dtype=np.float64)
    alpha, mx = C.c_float(0), C.c_float(0)
    rc = lib().ocs_oracle_clip_aciq(_p(T, _f32p), C.c_int64(T.size), int(bits), int(bool(is_signed)), int(n_bins),
                                    C.byref(alpha), C.byref(mx), _p(hist, _u64p), _p(stats, _f64p))
    _check(rc, "clip_aciq")
    return dict(alpha=float(alpha.value), max_abs=float(mx.value), hist=hist, b=float(stats[0]), sigma=float(stats[1]),
                laplace=bool(stats[2]), multiplier=float(stats[3]))


def range_curve(W, S_max: int):
    """max|W'| after s = 0..S_max greedy plain-halving splits -> float32 [S_max + 1]."""
    W = _f32(W)
    O, Cn = W.shape[0], W.shape[1]
    R = int(np.prod(W.shape[2:])) if W.ndim > 2 else 1
    curve = np.empty(S_max + 1, dtype=np.float32)
    _check(lib().ocs_oracle_range_curve(_p(W, _f32p), O, Cn, R, int(S_max), _p(curve, _f32p)), "range_curve")
    return curve


def knapsack(curves, unit_cost, budget: int):
    """curves: list of float32 arrays (one per layer, curve[s] for s = 0..s_max); unit_cost: elements one more
    channel adds to each layer (O * R) -> (S per layer int32, total reward)."""
    n = len(curves)
    s_max = np.array([len(c) - 1 for c in curves], dtype=np.int32)
    off = np.zeros(n, dtype=np.int64)
    off[1:] = np.cumsum([len(c) for c in curves])[:-1]
    flat = np.ascontiguousarray(np.concatenate([_f32(c) for c in curves]))
    cost = np.ascontiguousarray(unit_cost, dtype=np.int64)
    out = np.zeros(n, dtype=np.int32)
    tot = C.c_double(0)
    i64p = C.POINTER(C.c_int64)
    rc = lib().ocs_oracle_knapsack(n, _p(flat, _f32p), off.ctypes.data_as(i64p), _p(s_max, _i32p),
                                   cost.ctypes.data_as(i64p), C.c_int64(int(budget)), _p(out, _i32p), C.byref(tot))
    _check(rc, "knapsack")
    return out, float(tot.value)


def act_ocs(A, S: int):
    """Activation side of OCS (Eq. 4) with the channels chosen on the batch at hand (the
    per-batch "Oracle OCS" of Section 5.3).  A [rows, C] holds one batch, one row per sample
    (FC layer) or per pixel (conv layer, NHWC flattened): S times, the channel holding the largest
    |a| of the batch is duplicated and BOTH copies are halved, which is the greedy rule of
    Section 3.4 with the plain w/2 split.  -> (A' [rows, C+S], idx_map, split_order, (max|A|, max|A'|)).
    A composition: the arithmetic is the checker's own split() on the matrix whose channel axis is
    the activation's."""
    A = _f32(A)
    assert A.ndim == 2
    return split(A, S, 0.0)


def dup_weight_columns(Wc, idx_map):
    """Weight side of Eq. 4: a duplicated activation channel meets an unchanged copy of its weights.
    Wc [N, C] codes -> [N, C+S] with column j a copy of column idx_map[j]."""
    Wc = np.asarray(Wc)
    out = np.empty((Wc.shape[0], len(idx_map)), dtype=Wc.dtype)
    for j, src in enumerate(idx_map):
        out[:, j] = Wc[:, int(src)]
    return out


def act_ocs_linear(A, S: int, a_bits: int, a_signed: bool, Wc, w_scale, bias=None):
    """One layer with per-batch activation OCS: split the batch (Eq. 4), quantize the expanded
    activations on the grid of their own max |a'| (Section 3.1), duplicate the weight columns and
    evaluate the integer layer.  -> (Y fp32 [rows, N], acc, A' codes, a_scale, idx_map)."""
    Ap, idx, _, _ = act_ocs(A, S)
    ac, a_scale = quantize(Ap, a_bits, a_signed, maxabs(Ap))
    Wd = dup_weight_columns(Wc, idx)
    Y, acc = qlinear(ac, a_signed, a_scale, Wd, w_scale, np.arange(len(idx), dtype=np.int32), bias)
    return Y, acc, ac, a_scale, idx


def fold_duplicates(Wc, idx_map, Cn: int):
    """Wc int8 [N, C+S] or [N, C+S, kh, kw] -> (Wf int8 [N, C, ...], number of saturated sums)."""
    Wc = np.ascontiguousarray(Wc, dtype=np.int8)
    idx_map = np.ascontiguousarray(idx_map, dtype=np.int32)
    N, K = Wc.shape[0], Wc.shape[1]
    R = int(np.prod(Wc.shape[2:])) if Wc.ndim > 2 else 1
    out = np.empty((N, Cn) + tuple(Wc.shape[2:]), dtype=np.int8)
    lib().ocs_oracle_fold_duplicates.restype = C.c_int64
    rc = lib().ocs_oracle_fold_duplicates(_p(Wc, _i8p), N, int(Cn), R, K - int(Cn), _p(idx_map, _i32p), _p(out, _i8p))
    if rc < 0:
        raise RuntimeError("fold_duplicates: bad argument")
    return out, int(rc)


def act_select(P, S: int, quantile: float = 0.99):
    """Static channel choice of Section 5.3 on sampled activations P [rows, C]
    -> (sel int32 [S], counts int64 [C], threshold)."""
    P = _f32(P)
    assert P.ndim == 2
    rows, Cn = P.shape
    sel = np.empty(max(S, 1), dtype=np.int32)
    counts = np.zeros(Cn, dtype=np.int64)
    thr = C.c_float(0)
    rc = lib().ocs_oracle_act_select(_p(P, _f32p), C.c_int64(rows), Cn, int(S), C.c_double(quantile),
                                     _p(sel, _i32p), counts.ctypes.data_as(C.POINTER(C.c_int64)), C.byref(thr))
    _check(rc, "act_select")
    return sel[:S], counts, float(thr.value)


def act_split_static(A, sel):
    """Eq. 4 for a fixed channel list -> (A' [rows, C+S], idx_map)."""
    A = _f32(A)
    assert A.ndim == 2
    rows, Cn = A.shape
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    S = sel.size
    out = np.empty((rows, Cn + S), dtype=np.float32)
    idx = np.empty(Cn + S, dtype=np.int32)
    rc = lib().ocs_oracle_act_split_static(_p(A, _f32p), C.c_int64(rows), Cn, S, _p(sel, _i32p), _p(out, _f32p),
                                           _p(idx, _i32p))
    _check(rc, "act_split_static")
    return out, idx


def _codes(a, signed):
    return np.ascontiguousarray(a, dtype=np.int8 if signed else np.uint8)


def qlinear(A, a_signed, a_scale, Wc, w_scale, idx_map, bias=None):
    """A [M, C] codes, Wc [N, C+S] int8 -> (Y fp32 [M, N], acc int32 [M, N])."""
    A = _codes(A, a_signed)
    Wc = np.ascontiguousarray(Wc, dtype=np.int8)
    idx_map = np.ascontiguousarray(idx_map, dtype=np.int32)
    M, Cn = A.shape
    N, K = Wc.shape
    S = K - Cn
    assert idx_map.size == K
    Y = np.empty((M, N), dtype=np.float32)
    acc = np.empty((M, N), dtype=np.int32)
    b = None if bias is None else _f32(bias)
    rc = lib().ocs_oracle_qlinear(A.ctypes.data_as(C.c_void_p), int(bool(a_signed)),
                                  C.c_float(a_scale), M, Cn, _p(Wc, _i8p), C.c_float(w_scale), N,
                                  S, _p(idx_map, _i32p), _p(b, _f32p), _p(Y, _f32p),
                                  _p(acc, _i32p))
    _check(rc, "qlinear")
    return Y, acc


def qlinear_samples(A, a_signed, a_scale, Wc, w_scale, idx_map, ms, ns, bias=None):
    A = _codes(A, a_signed)
    Wc = np.ascontiguousarray(Wc, dtype=np.int8)
    idx_map = np.ascontiguousarray(idx_map, dtype=np.int32)
    ms = np.ascontiguousarray(ms, dtype=np.int32)
    ns = np.ascontiguousarray(ns, dtype=np.int32)
    M, Cn = A.shape
    N, K = Wc.shape
    Y = np.empty(ms.size, dtype=np.float32)
    acc = np.empty(ms.size, dtype=np.int32)
    b = None if bias is None else _f32(bias)
    rc = lib().ocs_oracle_qlinear_samples(A.ctypes.data_as(C.c_void_p), int(bool(a_signed)),
                                          C.c_float(a_scale), M, Cn, _p(Wc, _i8p),
                                          C.c_float(w_scale), N, K - Cn, _p(idx_map, _i32p),
                                          _p(b, _f32p), _p(ms, _i32p), _p(ns, _i32p), int(ms.size),
                                          _p(Y, _f32p), _p(acc, _i32p))
    _check(rc, "qlinear_samples")
    return Y, acc


def qconv(X, a_signed, a_scale, Wc, w_scale, idx_map, stride, pad, bias=None):
    """X NHWC codes [Nb, H, W, C]; Wc [O, C+S, kh, kw] int8 -> (Y NHWC fp32, acc NHWC int32)."""
    X = _codes(X, a_signed)
    Wc = np.ascontiguousarray(Wc, dtype=np.int8)
    idx_map = np.ascontiguousarray(idx_map, dtype=np.int32)
    Nb, H, Wd, Cn = X.shape
    O, K, kh, kw = Wc.shape
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (Wd + 2 * pad - kw) // stride + 1
    Y = np.empty((Nb, Ho, Wo, O), dtype=np.float32)
    acc = np.empty((Nb, Ho, Wo, O), dtype=np.int32)
    b = None if bias is None else _f32(bias)
    rc = lib().ocs_oracle_qconv(X.ctypes.data_as(C.c_void_p), int(bool(a_signed)),
                                C.c_float(a_scale), Nb, H, Wd, Cn, _p(Wc, _i8p),
                                C.c_float(w_scale), O, K - Cn, kh, kw, int(stride), int(pad),
                                _p(idx_map, _i32p), _p(b, _f32p), _p(Y, _f32p), _p(acc, _i32p))
    _check(rc, "qconv")
    return Y, acc


def relu(x):
    x = _f32(x)
    y = np.empty_like(x)
    lib().ocs_oracle_relu(_p(x, _f32p), C.c_int64(x.size), _p(y, _f32p))
    return y


def add_relu(a, b, do_relu=True):
    a, b = _f32(a), _f32(b)
    y = np.empty_like(a)
    lib().ocs_oracle_add_relu(_p(a, _f32p), _p(b, _f32p), C.c_int64(a.size), int(bool(do_relu)),
                              _p(y, _f32p))
    return y


def maxpool3x3s2(x):
    x = _f32(x)
    Nb, H, Wd, Cn = x.shape
    y = np.empty((Nb, (H - 1) // 2 + 1, (Wd - 1) // 2 + 1, Cn), dtype=np.float32)
    lib().ocs_oracle_maxpool3x3s2(_p(x, _f32p), Nb, H, Wd, Cn, _p(y, _f32p))
    return y


def global_avgpool(x):
    x = _f32(x)
    Nb, H, Wd, Cn = x.shape
    y = np.empty((Nb, Cn), dtype=np.float32)
    lib().ocs_oracle_global_avgpool(_p(x, _f32p), Nb, H, Wd, Cn, _p(y, _f32p))
    return y


def nchw_to_nhwc(x):
    x = _f32(x)
    Nb, Cn, H, Wd = x.shape
    y = np.empty((Nb, H, Wd, Cn), dtype=np.float32)
    lib().ocs_oracle_nchw_to_nhwc(_p(x, _f32p), Nb, Cn, H, Wd, _p(y, _f32p))
    return y


def sigmoid(x: float) -> float:
    return float(lib().ocs_oracle_sigmoid(C.c_float(x)))


def tanh(x: float) -> float:
    return float(lib().ocs_oracle_tanh(C.c_float(x)))


def lstm_cell(g_ih, g_hh, c, h=None):
    """Gates [batch, 4*hidden] (i, f, g, o); returns new (c, h) without touching the inputs."""
    g_ih, g_hh = _f32(g_ih), _f32(g_hh)
    c = _f32(c).copy()
    batch, hidden = c.shape
    hn = np.empty_like(c)
    lib().ocs_oracle_lstm_cell(_p(g_ih, _f32p), _p(g_hh, _f32p), batch, hidden, _p(c, _f32p),
                               _p(hn, _f32p))
    return c, hn
