"""Thin Python binding of the C ABI in include/ocs.h.

Argument marshalling only: every function takes torch CUDA tensors (used purely as device
buffers), allocates the outputs and the scratch workspace through torch, passes raw device
pointers and the current CUDA stream to the library and returns the output tensors.  All
arithmetic runs in the library's kernels.  There is no fallback: if the shared library is
missing or the device is not sm_100 the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libocs_b200.so")

OCS_OK = 0
STATUS_NAMES = {0: "OCS_OK", 1: "OCS_ERR_INVALID_ARG", 2: "OCS_ERR_SHAPE", 3: "OCS_ERR_WORKSPACE",
                4: "OCS_ERR_UNSUPPORTED", 5: "OCS_ERR_CUDA"}
DEV_NONFINITE, DEV_BAD_INDEX, DEV_TIMEOUT, DEV_DEPTH, DEV_OVERFLOW = 1, 2, 4, 8, 16
CLIP_NONE, CLIP_MSE, CLIP_MSE_EXACT, CLIP_KL, CLIP_ACIQ = 0, 1, 2, 3, 4

EXPORTS = [
    "ocs_num_splits", "ocs_poll_status", "ocs_version",
    "ocs_kernel_launches", "ocs_trace_start", "ocs_trace_stop",
    "ocs_split_workspace_bytes", "ocs_split", "ocs_selftest_wait_expiry",
    "ocs_range_curve_workspace_bytes", "ocs_range_curve", "ocs_knapsack_workspace_bytes", "ocs_knapsack_allocate",
    "ocs_split_quantize_workspace_bytes", "ocs_split_quantize", "ocs_dup_weight_columns",
    "ocs_split_quantize_batch_workspace_bytes", "ocs_split_quantize_batch",
    "ocs_fold_workspace_bytes", "ocs_fold_duplicates",
    "ocs_act_select_workspace_bytes", "ocs_act_select_channels", "ocs_act_split_quantize_static",
    "ocs_quantize_workspace_bytes", "ocs_quantize", "ocs_quantize_workspace_views", "ocs_quantize_noalloc",
    "ocs_qlinear_workspace_bytes", "ocs_qlinear", "ocs_transpose_codes", "ocs_selftest_force_gemm_plan",
    "ocs_conv_packed_k", "ocs_pack_conv_weights", "ocs_pack_conv_weights_batch", "ocs_qconv_workspace_bytes", "ocs_qconv",
    "ocs_add_relu", "ocs_maxpool3x3s2", "ocs_global_avgpool", "ocs_nchw_to_nhwc", "ocs_embedding", "ocs_lstm_cell",
]

_lib = None


class OcsError(RuntimeError):
    def __init__(self, what: str, status: int):
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}")
        self.status = status


def lib():
    """Loads the in-tree shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OcsError(f"{LIB_PATH} not built (run python -m paper_1901_09504_b200.build)", 5)
        L = C.CDLL(LIB_PATH)
        L.ocs_num_splits.argtypes = [C.c_int, C.c_double]
        L.ocs_version.restype = C.c_char_p
        for name in ("ocs_split_quantize_batch_workspace_bytes", "ocs_range_curve_workspace_bytes", "ocs_knapsack_workspace_bytes", "ocs_fold_workspace_bytes", "ocs_act_select_workspace_bytes", "ocs_split_quantize_workspace_bytes", "ocs_split_workspace_bytes", "ocs_quantize_workspace_bytes", "ocs_qlinear_workspace_bytes",
                     "ocs_qconv_workspace_bytes"):
            getattr(L, name).restype = C.c_size_t
        L.ocs_quantize_workspace_views.restype = None
        L.ocs_kernel_launches.restype = C.c_longlong
        L.ocs_conv_packed_k.restype = C.c_int64
        _lib = L
    return _lib


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ws(nbytes: int, device):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _check(status: int, what: str):
    if status != OCS_OK:
        raise OcsError(what, status)


def new_status(device="cuda"):
    """A zeroed device status word."""
    return torch.zeros(1, dtype=torch.int32, device=device)


def ocs_num_splits(channels: int, ratio: float) -> int:
    return int(lib().ocs_num_splits(int(channels), float(ratio)))


def ocs_poll_status(dev_status) -> int:
    out = C.c_int(0)
    _check(lib().ocs_poll_status(_ptr(dev_status), _stream(), C.byref(out)), "ocs_poll_status")
    return int(out.value)


class _TraceRow(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_longlong), ("total_ms", C.c_double)]


def ocs_kernel_launches() -> int:
    return int(lib().ocs_kernel_launches())


def ocs_trace_start(max_records: int = 65536) -> None:
    _check(lib().ocs_trace_start(int(max_records)), "ocs_trace_start")


def ocs_trace_stop(capacity: int = 64) -> dict:
    """-> {kernel name: (launches, total device ms)} of the launches since ocs_trace_start."""
    rows = (_TraceRow * capacity)()
    n = lib().ocs_trace_stop(rows, capacity)
    if n < 0:
        raise OcsError("ocs_trace_stop", 5)
    return {rows[i].name.decode(): (int(rows[i].launches), float(rows[i].total_ms)) for i in range(n)}


def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def ocs_split(W, S: int, qa_step: float = 0.0, qa_bits: int = 0, ld_out: int | None = None, dev_status=None,
              want_order: bool = True, out=None, ws=None):
    """W fp32 [O, C] or [O, C, kh, kw] (contiguous).  Returns (W_out [O, ld_out] fp32 whose first
    (C+S)*R columns are W', idx_map int32 [C+S], split_order int32 [S], max_abs fp32 [3]).
    `out` = (W_out, idx_map, order, max_abs) and `ws` reuse caller-held buffers instead of allocating."""
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
    O, Cn = W.shape[0], W.shape[1]
    R = 1
    for d in W.shape[2:]:
        R *= d
    cols_out = (Cn + S) * R
    if ld_out is None:
        ld_out = round_up(cols_out, 4)
    if out is not None:
        W_out, idx_map, order, max_abs = out
        ld_out = W_out.stride(0)
        assert W_out.shape[0] == O and ld_out >= cols_out and idx_map.numel() >= Cn + S and max_abs.numel() >= 3
        want_order = order is not None
    else:
        W_out = torch.empty((O, ld_out), dtype=torch.float32, device=W.device)
        idx_map = torch.empty(Cn + S, dtype=torch.int32, device=W.device)
        order = torch.empty(max(S, 1), dtype=torch.int32, device=W.device) if want_order else None
        max_abs = torch.empty(3, dtype=torch.float32, device=W.device)
    nws = lib().ocs_split_workspace_bytes(O, Cn, R, int(S))
    if ws is None:
        ws = _ws(nws, W.device)
    st = lib().ocs_split(_ptr(W), O, Cn, R, C.c_int64(Cn * R), int(S), C.c_float(qa_step), int(qa_bits),
                         _ptr(W_out), C.c_int64(ld_out), _ptr(idx_map), _ptr(order), _ptr(max_abs), _ptr(ws),
                         C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_split")
    return W_out, idx_map, (order[:S] if want_order else None), max_abs


def ocs_quantize(T, bits: int, is_signed: bool = True, mode: int = CLIP_NONE, n_candidates: int = 128,
                 n_bins: int = 2048, cols: int | None = None, ld_codes: int | None = None, max_abs_in=None,
                 dev_status=None, return_search: bool = False, out=None, ws=None):
    """T fp32 2-D [rows, ld_in] (row stride = T.stride(0)); `cols` valid columns per row (default all).
    Returns (codes int8/uint8 [rows, ld_codes], scale fp32 [1], alpha fp32 [1]) and, with
    return_search, also (hist uint64 [n_bins] as int64, scores float64 [n_candidates])."""
    assert T.is_cuda and T.dtype == torch.float32 and T.dim() == 2 and T.stride(1) == 1
    rows, ld_in = T.shape[0], T.stride(0)
    if cols is None:
        cols = T.shape[1]
    if ld_codes is None:
        ld_codes = round_up(cols, 16)
    if out is not None:
        codes, scale, alpha = out
        ld_codes = codes.stride(0)
        assert codes.shape[0] == rows and ld_codes >= cols
    else:
        codes = torch.empty((rows, ld_codes), dtype=torch.int8 if is_signed else torch.uint8, device=T.device)
        scale = torch.empty(1, dtype=torch.float32, device=T.device)
        alpha = torch.empty(1, dtype=torch.float32, device=T.device)
    if mode == CLIP_MSE_EXACT:
        n_bins = 0
    if mode == CLIP_ACIQ:
        n_candidates = 1
    nws = lib().ocs_quantize_workspace_bytes(int(n_bins), int(n_candidates))
    if ws is None:
        ws = _ws(nws, T.device)
    st = lib().ocs_quantize(_ptr(T), C.c_int64(rows), C.c_int64(cols), C.c_int64(ld_in), int(bits),
                            int(bool(is_signed)), int(mode), int(n_candidates), int(n_bins), _ptr(max_abs_in),
                            _ptr(codes), C.c_int64(ld_codes), _ptr(scale), _ptr(alpha), _ptr(ws),
                            C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_quantize")
    if not return_search:
        return codes, scale, alpha
    hp, sp = C.c_void_p(0), C.c_void_p(0)
    lib().ocs_quantize_workspace_views(_ptr(ws), int(n_bins), int(n_candidates), C.byref(hp), C.byref(sp))
    base = ws.data_ptr()
    hist = ws[hp.value - base: hp.value - base + 8 * max(n_bins, 1)].view(torch.int64).clone()
    scores = ws[sp.value - base: sp.value - base + 8 * n_candidates].view(torch.float64).clone()
    return codes, scale, alpha, hist, scores


def ocs_transpose_codes(codes, cols: int | None = None, out=None):
    """codes uint8/int8 [rows, ld >= cols] -> channel-major copy [cols, round_up(rows, 16)]."""
    assert codes.is_cuda and codes.dim() == 2 and codes.stride(1) == 1 and codes.element_size() == 1
    rows = codes.shape[0]
    if cols is None:
        cols = codes.shape[1]
    T = out if out is not None else torch.empty((cols, round_up(rows, 16)), dtype=codes.dtype, device=codes.device)
    _check(lib().ocs_transpose_codes(_ptr(codes), C.c_int64(rows), C.c_int64(cols), C.c_int64(codes.stride(0)), _ptr(T),
                                     C.c_int64(T.stride(0)), _stream()), "ocs_transpose_codes")
    return T


def ocs_qlinear(A_codes, a_scale, W_codes, w_scale, idx_map, C_in: int, S: int, bias=None, want_acc: bool = False,
                dev_status=None, out=None, ws=None, relu: bool = False, max_out=None, residual=None, A_codes_T=None):
    """A_codes uint8/int8 [M, lda>=C]; W_codes int8 [N, ldw>=C+S]; A_codes_T (optional) the channel-major copy
    [C, ld>=M] from ocs_transpose_codes.  Returns Y fp32 [M, N] (and acc int32)."""
    assert A_codes.is_cuda and A_codes.dim() == 2 and A_codes.stride(1) == 1
    assert W_codes.dtype == torch.int8 and W_codes.dim() == 2 and W_codes.stride(1) == 1
    M, N = A_codes.shape[0], W_codes.shape[0]
    a_signed = 1 if A_codes.dtype == torch.int8 else 0
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float32, device=A_codes.device)
    assert Y.stride(0) == N and Y.stride(1) == 1
    acc = torch.empty((M, N), dtype=torch.int32, device=A_codes.device) if want_acc else None
    nws = lib().ocs_qlinear_workspace_bytes(M, N, int(C_in), int(S))
    if ws is None:
        ws = _ws(nws, A_codes.device)
    st = lib().ocs_qlinear(_ptr(A_codes), _ptr(A_codes_T), C.c_int64(0 if A_codes_T is None else A_codes_T.stride(0)),
                           a_signed, _ptr(a_scale), M, int(C_in), C.c_int64(A_codes.stride(0)),
                           _ptr(W_codes), _ptr(w_scale), N, int(S), C.c_int64(W_codes.stride(0)), _ptr(idx_map),
                           _ptr(bias), _ptr(Y), C.c_int64(N), _ptr(acc), _ptr(residual), int(bool(relu)), _ptr(max_out), _ptr(ws),
                           C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_qlinear")
    return (Y, acc) if want_acc else Y


def ocs_conv_packed_k(C_in: int, S: int, kh: int, kw: int) -> int:
    """Contraction length of the packed conv weights (taps may be padded to the K-block)."""
    return int(lib().ocs_conv_packed_k(int(C_in), int(S), int(kh), int(kw)))


def ocs_pack_conv_weights(codes, O: int, C_in: int, S: int, kh: int, kw: int, ld_dst: int | None = None, out=None):
    """codes int8 [O, ld_src] in [C+S][kh*kw] order per row -> packed int8 [O, ld_dst]."""
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.dim() == 2 and codes.stride(1) == 1
    Kt = ocs_conv_packed_k(C_in, S, kh, kw)
    if ld_dst is None:
        ld_dst = round_up(Kt, 16)
    if out is not None:
        ld_dst = out.stride(0)
    packed = out if out is not None else torch.empty((O, ld_dst), dtype=torch.int8, device=codes.device)
    st = lib().ocs_pack_conv_weights(_ptr(codes), O, int(C_in), int(S), int(kh), int(kw),
                                     C.c_int64(codes.stride(0)), _ptr(packed), C.c_int64(ld_dst), _stream())
    _check(st, "ocs_pack_conv_weights")
    return packed


def ocs_qconv(X_codes, a_scale, W_packed, w_scale, idx_map, S: int, kh: int, kw: int, stride: int, pad: int,
              bias=None, want_acc: bool = False, dev_status=None, out=None, ws=None, relu: bool = False, max_out=None,
              residual=None):
    """X_codes uint8/int8 NHWC [Nb, H, W, C] contiguous; W_packed from ocs_pack_conv_weights.
    Returns Y fp32 NHWC [Nb, Ho, Wo, O] (and acc int32)."""
    assert X_codes.is_cuda and X_codes.dim() == 4 and X_codes.is_contiguous()
    Nb, H, Wd, Cn = X_codes.shape
    O = W_packed.shape[0]
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (Wd + 2 * pad - kw) // stride + 1
    a_signed = 1 if X_codes.dtype == torch.int8 else 0
    Y = out if out is not None else torch.empty((Nb, Ho, Wo, O), dtype=torch.float32, device=X_codes.device)
    acc = torch.empty((Nb, Ho, Wo, O), dtype=torch.int32, device=X_codes.device) if want_acc else None
    nws = lib().ocs_qconv_workspace_bytes(Nb, H, Wd, Cn, O, int(S), kh, kw, stride, pad)
    if ws is None:
        ws = _ws(nws, X_codes.device)
    st = lib().ocs_qconv(_ptr(X_codes), a_signed, _ptr(a_scale), Nb, H, Wd, Cn, _ptr(W_packed), _ptr(w_scale), O,
                         int(S), kh, kw, stride, pad, C.c_int64(W_packed.stride(0)), _ptr(idx_map), _ptr(bias),
                         _ptr(Y), _ptr(acc), _ptr(residual), int(bool(relu)), _ptr(max_out), _ptr(ws), C.c_size_t(ws.numel()),
                         _ptr(dev_status), _stream())
    _check(st, "ocs_qconv")
    return (Y, acc) if want_acc else Y


def ocs_add_relu(a, b=None, relu: bool = True, out=None, max_out=None):
    """y = a (+ b), then ReLU when relu; fp32 tensors of equal shape.  max_out (fp32 [1]) receives max |y|."""
    assert a.is_cuda and a.dtype == torch.float32 and a.is_contiguous()
    assert b is None or (b.shape == a.shape and b.dtype == torch.float32 and b.is_contiguous())
    y = out if out is not None else torch.empty_like(a)
    _check(lib().ocs_add_relu(_ptr(a), _ptr(b), C.c_int64(a.numel()), int(bool(relu)), _ptr(y), _ptr(max_out),
                              _stream()), "ocs_add_relu")
    return y


def ocs_maxpool3x3s2(x):
    """x fp32 NHWC -> 3x3 stride-2 pad-1 max pooling."""
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 4 and x.is_contiguous()
    Nb, H, Wd, Cn = x.shape
    y = torch.empty((Nb, (H - 1) // 2 + 1, (Wd - 1) // 2 + 1, Cn), dtype=torch.float32, device=x.device)
    _check(lib().ocs_maxpool3x3s2(_ptr(x), Nb, H, Wd, Cn, _ptr(y), _stream()), "ocs_maxpool3x3s2")
    return y


def ocs_global_avgpool(x):
    """x fp32 NHWC -> [Nb, C]."""
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 4 and x.is_contiguous()
    Nb, H, Wd, Cn = x.shape
    y = torch.empty((Nb, Cn), dtype=torch.float32, device=x.device)
    _check(lib().ocs_global_avgpool(_ptr(x), Nb, H, Wd, Cn, _ptr(y), _stream()), "ocs_global_avgpool")
    return y


def ocs_nchw_to_nhwc(x):
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 4 and x.is_contiguous()
    Nb, Cn, H, Wd = x.shape
    y = torch.empty((Nb, H, Wd, Cn), dtype=torch.float32, device=x.device)
    _check(lib().ocs_nchw_to_nhwc(_ptr(x), Nb, Cn, H, Wd, _ptr(y), _stream()), "ocs_nchw_to_nhwc")
    return y


def ocs_embedding(table, ids, dev_status=None):
    """table fp32 [V, E], ids int32 [...] -> fp32 [..., E]."""
    assert table.is_cuda and table.dtype == torch.float32 and table.dim() == 2 and table.is_contiguous()
    assert ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()
    out = torch.empty(tuple(ids.shape) + (table.shape[1],), dtype=torch.float32, device=table.device)
    _check(lib().ocs_embedding(_ptr(table), _ptr(ids), C.c_int64(ids.numel()), table.shape[0], table.shape[1],
                               _ptr(out), _ptr(dev_status), _stream()), "ocs_embedding")
    return out


def ocs_lstm_cell(g_ih, g_hh, c, h=None):
    """Gates fp32 [batch, 4*hidden] (i, f, g, o); c [batch, hidden] is updated IN PLACE; returns (c, h)."""
    assert g_ih.is_cuda and g_ih.dtype == torch.float32 and g_ih.is_contiguous() and g_hh.is_contiguous()
    batch, hidden = c.shape
    assert g_ih.shape == (batch, 4 * hidden) and g_hh.shape == g_ih.shape and c.is_contiguous()
    if h is None:
        h = torch.empty_like(c)
    _check(lib().ocs_lstm_cell(_ptr(g_ih), _ptr(g_hh), batch, hidden, _ptr(c), _ptr(h), _stream()), "ocs_lstm_cell")
    return c, h


def ocs_quantize_noalloc(T, bits: int, is_signed: bool = True, mode: int = CLIP_NONE, n_candidates: int = 128,
                         n_bins: int = 2048, cols: int | None = None, ld_codes: int | None = None, max_abs_in=None,
                         dev_status=None, out=None):
    """ocs_quantize without a workspace: for callers that must not allocate device memory where they
    quantize (the library's built-in 48 KB scratch is used instead).  The outputs are still the
    caller's: pass `out` = (codes, scale, alpha) to reuse buffers, otherwise this wrapper creates them
    with torch for convenience -- the library call itself allocates nothing either way.
    Returns (codes, scale, alpha)."""
    assert T.is_cuda and T.dtype == torch.float32 and T.dim() == 2 and T.stride(1) == 1
    rows, ld_in = T.shape[0], T.stride(0)
    if cols is None:
        cols = T.shape[1]
    if out is not None:
        codes, scale, alpha = out
        ld_codes = codes.stride(0)
    else:
        if ld_codes is None:
            ld_codes = round_up(cols, 16)
        codes = torch.empty((rows, ld_codes), dtype=torch.int8 if is_signed else torch.uint8, device=T.device)
        scale = torch.empty(1, dtype=torch.float32, device=T.device)
        alpha = torch.empty(1, dtype=torch.float32, device=T.device)
    st = lib().ocs_quantize_noalloc(_ptr(T), C.c_int64(rows), C.c_int64(cols), C.c_int64(ld_in), int(bits),
                                    int(bool(is_signed)), int(mode), int(n_candidates), int(n_bins),
                                    _ptr(max_abs_in), _ptr(codes), C.c_int64(ld_codes), _ptr(scale), _ptr(alpha),
                                    _ptr(dev_status), _stream())
    _check(st, "ocs_quantize_noalloc")
    return codes, scale, alpha


def ocs_split_quantize(W, S: int, bits: int, mode: int = CLIP_NONE, is_signed: bool = True, qa_step: float = 0.0,
                       qa_bits: int = 0,
                       n_candidates: int = 128, n_bins: int = 2048, ld_codes: int | None = None, dev_status=None,
                       want_order: bool = True, out=None, ws=None):
    """Split + clip search + quantization without the fp32 W'.  W fp32 [O, C] or [O, C, kh, kw].
    Returns (codes int8 [O, ld_codes] in the split's layout, scale [1], alpha [1], idx_map int32 [C+S],
    split_order int32 [S] or None, max_abs fp32 [3]).  `out` = (codes, scale, alpha, idx_map, order, max_abs)."""
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
    O, Cn = W.shape[0], W.shape[1]
    R = 1
    for d in W.shape[2:]:
        R *= d
    cols_out = (Cn + S) * R
    if out is not None:
        codes, scale, alpha, idx_map, order, max_abs = out
        ld_codes = codes.stride(0)
    else:
        if ld_codes is None:
            ld_codes = round_up(cols_out, 16)
        codes = torch.empty((O, ld_codes), dtype=torch.int8 if is_signed else torch.uint8, device=W.device)
        scale = torch.empty(1, dtype=torch.float32, device=W.device)
        alpha = torch.empty(1, dtype=torch.float32, device=W.device)
        idx_map = torch.empty(Cn + S, dtype=torch.int32, device=W.device)
        order = torch.empty(max(S, 1), dtype=torch.int32, device=W.device) if want_order else None
        max_abs = torch.empty(3, dtype=torch.float32, device=W.device)
    nws = lib().ocs_split_quantize_workspace_bytes(O, Cn, R, int(S), int(n_bins), int(n_candidates))
    if ws is None:
        ws = _ws(nws, W.device)
    st = lib().ocs_split_quantize(_ptr(W), O, Cn, R, C.c_int64(Cn * R), int(S), C.c_float(qa_step), int(qa_bits),
                                  int(bits), int(bool(is_signed)), int(mode), int(n_candidates), int(n_bins), _ptr(codes),
                                  C.c_int64(ld_codes), _ptr(idx_map), _ptr(order), _ptr(max_abs), _ptr(scale),
                                  _ptr(alpha), _ptr(ws), C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_split_quantize")
    return codes, scale, alpha, idx_map, (order[:S] if order is not None else None), max_abs


def ocs_dup_weight_columns(W_codes, C_in: int, S: int, idx_map, R: int = 1, dev_status=None):
    """W_codes int8 [N, ldw >= (C+S)*R]: fills channels C..C+S-1 in place with copies of their sources."""
    assert W_codes.is_cuda and W_codes.dtype == torch.int8 and W_codes.dim() == 2 and W_codes.stride(1) == 1
    _check(lib().ocs_dup_weight_columns(_ptr(W_codes), W_codes.shape[0], int(C_in), int(R), int(S),
                                        C.c_int64(W_codes.stride(0)), _ptr(idx_map), _ptr(dev_status), _stream()),
           "ocs_dup_weight_columns")
    return W_codes


def ocs_act_select_channels(P, S: int, quantile: float = 0.99, dev_status=None):
    """P fp32 [rows, C] sampled activations -> (sel int32 [S], counts int64 [C], threshold fp32 [1])."""
    assert P.is_cuda and P.dtype == torch.float32 and P.dim() == 2 and P.stride(1) == 1
    rows, Cn = P.shape
    sel = torch.empty(max(int(S), 1), dtype=torch.int32, device=P.device)
    counts = torch.empty(Cn, dtype=torch.int64, device=P.device)
    thr = torch.empty(1, dtype=torch.float32, device=P.device)
    ws = _ws(lib().ocs_act_select_workspace_bytes(Cn), P.device)
    st = lib().ocs_act_select_channels(_ptr(P), C.c_int64(rows), Cn, C.c_int64(P.stride(0)), int(S), C.c_double(quantile),
                                       _ptr(sel), _ptr(counts), _ptr(thr), _ptr(ws), C.c_size_t(ws.numel()),
                                       _ptr(dev_status), _stream())
    _check(st, "ocs_act_select_channels")
    return sel[:int(S)], counts, thr


def ocs_act_split_quantize_static(A, sel, bits: int, is_signed: bool, alpha_in=None, ld_codes: int | None = None,
                                  dev_status=None, out=None, ws=None):
    """A fp32 [rows, C], sel int32 [S] -> (expanded codes [rows, ld_codes], scale fp32 [1], idx_map int32 [C+S]).
    `out` = (codes, scale, idx_map)."""
    assert A.is_cuda and A.dtype == torch.float32 and A.dim() == 2 and A.stride(1) == 1
    rows, Cn = A.shape
    S = int(sel.numel())
    if out is not None:
        codes, scale, idx_map = out
        ld_codes = codes.stride(0)
    else:
        if ld_codes is None:
            ld_codes = round_up(Cn + S, 16)
        codes = torch.empty((rows, ld_codes), dtype=torch.int8 if is_signed else torch.uint8, device=A.device)
        scale = torch.empty(1, dtype=torch.float32, device=A.device)
        idx_map = torch.empty(Cn + S, dtype=torch.int32, device=A.device)
    nws = lib().ocs_split_quantize_workspace_bytes(rows, Cn, 1, S, 1, 1)
    if ws is None:
        ws = _ws(nws, A.device)
    st = lib().ocs_act_split_quantize_static(_ptr(A), rows, Cn, C.c_int64(A.stride(0)), S, _ptr(sel if S else None),
                                             int(bits), int(bool(is_signed)), _ptr(alpha_in), _ptr(codes),
                                             C.c_int64(ld_codes), _ptr(idx_map), _ptr(scale), _ptr(ws),
                                             C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_act_split_quantize_static")
    return codes, scale, idx_map


def ocs_fold_duplicates(W_codes, C_in: int, S: int, idx_map, R: int = 1, ld_out: int | None = None, dev_status=None):
    """W_codes int8 [N, ldw >= (C+S)*R] -> folded int8 [N, ld_out >= C*R] (copies summed into their sources)."""
    assert W_codes.is_cuda and W_codes.dtype == torch.int8 and W_codes.dim() == 2 and W_codes.stride(1) == 1
    N = W_codes.shape[0]
    if ld_out is None:
        ld_out = round_up(int(C_in) * int(R), 16)
    out = torch.zeros((N, ld_out), dtype=torch.int8, device=W_codes.device)
    ws = _ws(lib().ocs_fold_workspace_bytes(int(C_in), int(S)), W_codes.device)
    st = lib().ocs_fold_duplicates(_ptr(W_codes), N, int(C_in), int(R), int(S), C.c_int64(W_codes.stride(0)), _ptr(idx_map),
                                   _ptr(out), C.c_int64(ld_out), _ptr(ws), C.c_size_t(ws.numel()), _ptr(dev_status),
                                   _stream())
    _check(st, "ocs_fold_duplicates")
    return out


def ocs_range_curve(W, S_max: int, out=None, dev_status=None):
    """W fp32 [O, C] or [O, C, kh, kw] -> curve fp32 [S_max + 1]: max|W'| after s = 0..S_max greedy plain-halving splits."""
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
    O, Cn = W.shape[0], W.shape[1]
    R = 1
    for d in W.shape[2:]:
        R *= d
    curve = out if out is not None else torch.empty(int(S_max) + 1, dtype=torch.float32, device=W.device)
    ws = _ws(lib().ocs_range_curve_workspace_bytes(Cn, R, int(S_max)), W.device)
    st = lib().ocs_range_curve(_ptr(W), O, Cn, R, C.c_int64(Cn * R), int(S_max), _ptr(curve), _ptr(ws),
                               C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_range_curve")
    return curve


def ocs_knapsack_allocate(curves, unit_cost, budget: int):
    """curves: list of fp32 device tensors (one per layer, s_max + 1 entries each); unit_cost: list of ints (O * R per
    layer); budget in weight elements -> (S int32 [n_layers] on the device, total reward float64 [1])."""
    n = len(curves)
    flat = torch.cat([c.reshape(-1) for c in curves]).contiguous()
    sizes = [int(c.numel()) for c in curves]
    off = (C.c_int64 * n)(*[sum(sizes[:i]) for i in range(n)])
    smax = (C.c_int32 * n)(*[sz - 1 for sz in sizes])
    cost = (C.c_int64 * n)(*[int(c) for c in unit_cost])
    S = torch.empty(n, dtype=torch.int32, device=flat.device)
    total = torch.empty(1, dtype=torch.float64, device=flat.device)
    nws = lib().ocs_knapsack_workspace_bytes(n, cost, C.c_int64(int(budget)))
    if nws == 0:
        raise OcsError("ocs_knapsack_workspace_bytes", 4)
    ws = _ws(nws, flat.device)
    st = lib().ocs_knapsack_allocate(n, _ptr(flat), off, smax, cost, C.c_int64(int(budget)), _ptr(S), _ptr(total),
                                     _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(st, "ocs_knapsack_allocate")
    return S, total


def ocs_selftest_wait_expiry(W, dev_status):
    """Runs the row-staged copy with each CTA's last row group never requested: sets DEV_TIMEOUT in dev_status
    and returns the (partly unwritten) output."""
    assert W.is_cuda and W.dtype == torch.float32 and W.dim() == 2 and W.is_contiguous()
    O, Cn = W.shape
    out = torch.zeros_like(W)
    ws = _ws(lib().ocs_split_workspace_bytes(O, Cn, 1, 0) + round_up(4 * Cn, 256) + 256, W.device)
    st = lib().ocs_selftest_wait_expiry(_ptr(W), O, Cn, C.c_int64(Cn), _ptr(out), C.c_int64(Cn), _ptr(ws),
                                        C.c_size_t(ws.numel()), _ptr(dev_status), _stream())
    _check(st, "ocs_selftest_wait_expiry")
    return out


def ocs_selftest_force_gemm_plan(bn: int = 0, split_k: int = 0):
    """Fixes tile width / K split of the following ocs_qlinear / ocs_qconv calls (bn = 0: planner)."""
    _check(lib().ocs_selftest_force_gemm_plan(int(bn), int(split_k)), "ocs_selftest_force_gemm_plan")


class _LayerDesc(C.Structure):
    _fields_ = [("W", C.c_void_p), ("O", C.c_int), ("C", C.c_int), ("R", C.c_int), ("S", C.c_int),
                ("codes", C.c_void_p), ("ld_codes", C.c_int64), ("idx_map", C.c_void_p), ("scale", C.c_void_p),
                ("max_abs3", C.c_void_p)]


def ocs_split_quantize_batch(Ws, Ss, bits: int, is_signed: bool = True, dev_status=None, ws=None):
    """ocs_split_quantize (plain halving, no clip search) for a list of weight tensors in five launches.
    Ws: fp32 [O, C] or [O, C, kh, kw] device tensors; Ss: split counts.  Returns per layer (codes int8
    [O, ld_codes], scale fp32 [1], idx_map int32 [C+S])."""
    n = len(Ws)
    descs = (_LayerDesc * n)()
    outs = []
    for i, (W, S) in enumerate(zip(Ws, Ss)):
        assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
        O, Cn = W.shape[0], W.shape[1]
        R = 1
        for d in W.shape[2:]:
            R *= d
        ld = round_up((Cn + int(S)) * R, 16)
        codes = torch.empty((O, ld), dtype=torch.int8 if is_signed else torch.uint8, device=W.device)
        scale = torch.empty(1, dtype=torch.float32, device=W.device)
        idx_map = torch.empty(Cn + int(S), dtype=torch.int32, device=W.device)
        descs[i] = _LayerDesc(W.data_ptr(), O, Cn, R, int(S), codes.data_ptr(), ld, idx_map.data_ptr(), scale.data_ptr(), None)
        outs.append((codes, scale, idx_map))
    nws = lib().ocs_split_quantize_batch_workspace_bytes(descs, n)
    if nws == 0:
        raise OcsError("ocs_split_quantize_batch_workspace_bytes", 4)
    if ws is None:
        ws = _ws(nws, Ws[0].device)
    st = lib().ocs_split_quantize_batch(descs, n, int(bits), int(bool(is_signed)), _ptr(ws), C.c_size_t(ws.numel()),
                                        _ptr(dev_status), _stream())
    _check(st, "ocs_split_quantize_batch")
    return outs


class _PackDesc(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("O", C.c_int), ("C", C.c_int), ("S", C.c_int), ("kh", C.c_int), ("kw", C.c_int),
                ("ld_src", C.c_int64), ("packed", C.c_void_p), ("ld_dst", C.c_int64)]


def ocs_pack_conv_weights_batch(jobs):
    """jobs: list of (codes int8 [O, ld_src], O, C, S, kh, kw) -> list of packed int8 [O, ld_dst], one launch."""
    n = len(jobs)
    descs = (_PackDesc * n)()
    outs = []
    for i, (codes, O, Cn, S, kh, kw) in enumerate(jobs):
        assert codes.is_cuda and codes.dtype == torch.int8 and codes.dim() == 2 and codes.stride(1) == 1
        ld = round_up(ocs_conv_packed_k(Cn, S, kh, kw), 16)
        packed = torch.empty((O, ld), dtype=torch.int8, device=codes.device)
        descs[i] = _PackDesc(codes.data_ptr(), int(O), int(Cn), int(S), int(kh), int(kw), codes.stride(0), packed.data_ptr(), ld)
        outs.append(packed)
    _check(lib().ocs_pack_conv_weights_batch(descs, n, _stream()), "ocs_pack_conv_weights_batch")
    return outs
