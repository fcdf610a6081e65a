"""Chains of C-ABI calls for whole networks: the ResNet-50 convolution stack (Section 5's CNN
workloads) and the two-layer LSTM language model (Section 6).

Only call sequencing lives here: which tensor feeds which layer.  Every arithmetic step -- split,
clip search, quantization, the integer convolutions and GEMMs, ReLU, residual adds, pooling, the
LSTM cell -- is one of the library's kernels, reached through the binding.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import binding as B


@dataclass
class QLayer:
    """One layer after the offline steps of Section 3.5: split, quantized and (for a convolution)
    reordered weights, plus what the run-time layer needs to gather the duplicated channels."""
    codes: torch.Tensor        # int8: conv [O, ld] packed for ocs_qconv; linear [O, ld]
    w_scale: torch.Tensor      # fp32 [1]
    idx_map: torch.Tensor      # int32 [C + S]
    bias: torch.Tensor | None  # fp32 [O]
    C: int
    O: int
    S: int
    k: int = 1
    stride: int = 1
    pad: int = 0


def prepare_layer(W, bias, ratio: float, bits: int, clip_mode: int = B.CLIP_NONE, qa_bits: int = 0, conv: bool = False,
                  stride: int = 1, pad: int = 0, n_candidates: int = 128, n_bins: int = 2048, dev_status=None,
                  fold: bool = False) -> QLayer:
    """W fp32 [O, C] or [O, C, k, k] on the device -> QLayer (ocs_split_quantize, or ocs_split + ocs_quantize where
    the fused call cannot stage the rows; ocs_pack_conv_weights)."""
    O, Cn = W.shape[0], W.shape[1]
    k = W.shape[2] if W.dim() == 4 else 1
    R = k * k
    S = B.ocs_num_splits(Cn, ratio)
    try:
        # one call, no fp32 W' (rows that cannot be staged in shared memory are reported as unsupported)
        if clip_mode not in (B.CLIP_NONE, B.CLIP_MSE, B.CLIP_KL, B.CLIP_ACIQ):
            raise B.OcsError("ocs_split_quantize", 4)
        codes, scale, _, idx_map, _, _ = B.ocs_split_quantize(W.contiguous(), S, bits, clip_mode, qa_bits=qa_bits,
                                                              n_candidates=n_candidates, n_bins=n_bins,
                                                              dev_status=dev_status, want_order=False)
    except B.OcsError as e:
        if e.status != 4:
            raise
        W_out, idx_map, _, mx = B.ocs_split(W.contiguous(), S, qa_bits=qa_bits, dev_status=dev_status, want_order=False)
        codes, scale, _ = B.ocs_quantize(W_out, bits, True, clip_mode, n_candidates, n_bins, cols=(Cn + S) * R,
                                         max_abs_in=mx[1:2], dev_status=dev_status)
    if fold and S > 0:
        # k <= 7-bit codes: the copies are summed back into their source channel (ocs_fold_duplicates); the
        # layer then runs on C plain channels with the same accumulators.  (A sum that leaves int8 sets
        # OCS_DEV_OVERFLOW in dev_status.)
        codes = B.ocs_fold_duplicates(codes, Cn, S, idx_map, R=R, dev_status=dev_status)
        idx_map = idx_map[:Cn].contiguous()
        S = 0
    if conv:
        codes = B.ocs_pack_conv_weights(codes, O, Cn, S, k, k)
    return QLayer(codes, scale, idx_map, bias, Cn, O, S, k, stride, pad)


def quantize_activations(x, signed: bool, bits: int = 8, dev_status=None, max_abs=None):
    """Dynamic per-tensor grid (max |x| of the tensor handed to the layer): returns dense codes shaped
    like x and the fp32 [1] scale.  max_abs (fp32 [1] on the device): max |x| when the producer of x
    already took it."""
    flat = x.reshape(1, -1)
    codes, scale, _ = B.ocs_quantize(flat, bits, signed, B.CLIP_NONE, max_abs_in=max_abs, dev_status=dev_status)
    return codes[0, :flat.shape[1]].view(x.shape), scale


def conv_forward(L: QLayer, x, a_signed: bool, a_bits: int = 8, dev_status=None, max_abs=None, relu: bool = False,
                 max_out=None, residual=None, xq=None):
    """x fp32 NHWC -> fp32 NHWC (activation quantization + ocs_qconv; the shortcut addition, ReLU and max |y|
    in the layer's epilogue on request).  xq: (codes, scale) of x when another layer has quantized it already."""
    xc, xs = xq if xq is not None else quantize_activations(x, a_signed, a_bits, dev_status, max_abs)
    return B.ocs_qconv(xc, xs, L.codes, L.w_scale, L.idx_map, L.S, L.k, L.k, L.stride, L.pad, bias=L.bias,
                       dev_status=dev_status, relu=relu, max_out=max_out, residual=residual)


def linear_forward(L: QLayer, x, a_signed: bool, a_bits: int = 8, dev_status=None):
    """x fp32 [M, C] -> fp32 [M, O] (activation quantization + ocs_qlinear)."""
    M, Cn = x.shape
    ld = B.round_up(Cn, 16)
    codes, scale, _ = B.ocs_quantize(x.contiguous(), a_bits, a_signed, B.CLIP_NONE, ld_codes=ld, dev_status=dev_status)
    # with many rows and duplicated channels the layer gathers whole channels from a channel-major copy of the
    # codes; a handful of rows (a recurrent net's time step) is not worth the extra launch
    codes_T = B.ocs_transpose_codes(codes, cols=Cn) if (L.S > 0 and M >= 64) else None
    return B.ocs_qlinear(codes, scale, L.codes, L.w_scale, L.idx_map, Cn, L.S, bias=L.bias, dev_status=dev_status,
                         A_codes_T=codes_T)


# ------------------------------------------------------------------------------------------ ResNet-50
def batchable(W) -> bool:
    """True when ocs_split_quantize_batch can take this layer (the fused path's staging limits)."""
    R = 1
    for d in W.shape[2:]:
        R *= d
    Cn = W.shape[1]
    return (Cn * R) % 4 == 0 and 2 * 4 * (Cn + Cn // 8 + 8) * R <= 226 * 1024 and W.data_ptr() % 16 == 0


def prepare_layers_batch(Ws, biases, ratio: float, bits: int, conv_flags, strides, pads, dev_status=None):
    """All layers that fit the batched call are split and quantized together (ocs_split_quantize_batch: no clip
    search, plain halving); the convolution weights are then reordered in one more launch.  -> list of QLayer."""
    Ss = [B.ocs_num_splits(W.shape[1], ratio) for W in Ws]
    outs = B.ocs_split_quantize_batch([W.contiguous() for W in Ws], Ss, bits, dev_status=dev_status)
    jobs, where = [], []
    for i, (W, S, (codes, _, _), conv) in enumerate(zip(Ws, Ss, outs, conv_flags)):
        if conv:
            jobs.append((codes, W.shape[0], W.shape[1], S, W.shape[2], W.shape[3]))
            where.append(i)
    packed = dict(zip(where, B.ocs_pack_conv_weights_batch(jobs))) if jobs else {}
    layers = []
    for i, (W, b, S, (codes, scale, idx_map), stride, pad) in enumerate(zip(Ws, biases, Ss, outs, strides, pads)):
        O, Cn = W.shape[0], W.shape[1]
        k = W.shape[2] if W.dim() == 4 else 1
        layers.append(QLayer(packed.get(i, codes), scale, idx_map, b, Cn, O, S, k, stride, pad))
    return layers


def prepare_resnet50(cfg, device, dev_status=None, batched: bool = True, weights=None):
    """cfg from ocs_inputs.configs.config4 -> {layer name: QLayer}.  weights: {name: (W, bias)} already on the device
    (else they are uploaded from cfg).  With `batched` (and no clip search) every layer the batched call can take is
    prepared by ocs_split_quantize_batch; the rest (the first layer: 3 x 49 weights per filter) go one by one."""
    mode = B.CLIP_MSE if cfg["clip"] == "mse" else B.CLIP_NONE
    out = {}
    specs = cfg["layers"] + [cfg["fc"]]
    dev_w = {}
    for spec in specs:
        if weights is not None:
            dev_w[spec.name] = weights[spec.name]
        else:
            W, bias = cfg["params"][spec.name]
            dev_w[spec.name] = (torch.from_numpy(W).to(device), torch.from_numpy(bias).to(device))
    group = []
    for spec in specs:
        Wd, bd = dev_w[spec.name]
        if spec.name == "fc":
            Wd = Wd.reshape(spec.O, spec.C)
        if batched and mode == B.CLIP_NONE and batchable(Wd):
            group.append((spec, Wd, bd))
        elif spec.name == "fc":
            out["fc"] = prepare_layer(Wd, bd, cfg["ratio"], cfg["w_bits"], mode, dev_status=dev_status)
        else:
            out[spec.name] = prepare_layer(Wd, bd, cfg["ratio"], cfg["w_bits"], mode, conv=True, stride=spec.stride,
                                           pad=spec.pad, dev_status=dev_status)
    if group:
        ql = prepare_layers_batch([g[1] for g in group], [g[2] for g in group], cfg["ratio"], cfg["w_bits"],
                                  [g[0].name != "fc" for g in group], [g[0].stride for g in group],
                                  [g[0].pad for g in group], dev_status=dev_status)
        for (spec, _, _), L in zip(group, ql):
            out[spec.name] = L
    return out


def resnet50_forward(cfg, layers, X_nchw, a_bits: int = 8, keep: bool = False, dev_status=None):
    """X fp32 NCHW on the device -> logits fp32 [Nb, 1000]; with keep, also every named tensor."""
    t = {}
    mx = {}     # max |tensor| of the tensors whose producing layer took it in its epilogue
    xq = {}     # codes and scale of a tensor that two layers read (a block's first convolution and its projection)
    readers = {}
    for spec in cfg["layers"]:
        readers[spec.input_from] = readers.get(spec.input_from, 0) + 1
    x = B.ocs_nchw_to_nhwc(X_nchw.contiguous())
    first = True
    for spec in cfg["layers"]:
        src = t[spec.input_from] if spec.input_from else x
        m = torch.empty(1, dtype=torch.float32, device=x.device)
        # The ReLU after the layer is taken in its epilogue, with the maximum of the result, and so is the shortcut
        # addition of a bottleneck block's last convolution (one more rounded addition per output, before the
        # ReLU): the block's output is written once instead of written, read back with the shortcut and rewritten.
        take_max = spec.relu or bool(spec.residual_from)
        q = xq.get(id(src))
        if q is None and spec.input_from and readers[spec.input_from] > 1:
            q = xq[id(src)] = quantize_activations(src, first, a_bits, dev_status, mx.get(id(src)))
        y = conv_forward(layers[spec.name], src, a_signed=first, a_bits=a_bits, dev_status=dev_status,
                         max_abs=mx.get(id(src)), relu=spec.relu, max_out=m if take_max else None,
                         residual=t[spec.residual_from] if spec.residual_from else None, xq=q)
        if spec.residual_from:
            t[spec.name.rsplit(".", 1)[0] + ".out"] = y
        if take_max:
            mx[id(y)] = m
        t[spec.name] = y
        x = y
        if first:
            x = B.ocs_maxpool3x3s2(y)
            t["pool"] = x
            if spec.relu:
                mx[id(x)] = m   # the windows cover every value of y and none is negative: max |pool| = max |y|
            first = False
    feat = B.ocs_global_avgpool(x)
    t["avgpool"] = feat
    logits = linear_forward(layers["fc"], feat, a_signed=False, a_bits=a_bits, dev_status=dev_status)
    t["fc"] = logits
    return (logits, t) if keep else logits


# ------------------------------------------------------------------------------------------ LSTM
_SIDE_STREAMS = {}


def _side_stream(device, which: int = 0):
    """Helper streams per device, created on first use."""
    idx = torch.device(device).index if torch.device(device).index is not None else torch.cuda.current_device()
    key = (idx, which)
    if key not in _SIDE_STREAMS:
        _SIDE_STREAMS[key] = torch.cuda.Stream(device=idx)
    return _SIDE_STREAMS[key]


def prepare_lstm(cfg, device, dev_status=None, fold: bool = False):
    """cfg from ocs_inputs.configs.config5 -> dict of QLayers and the embedding table."""
    p = cfg["params"]
    mode = B.CLIP_MSE if cfg["clip"] == "mse" else B.CLIP_NONE
    out = {"emb": torch.from_numpy(p["emb"]).to(device)}
    for layer in range(2):
        for nm, bn in (("W_ih", "b_ih"), ("W_hh", "b_hh")):
            out[f"{nm}{layer}"] = prepare_layer(torch.from_numpy(p[f"{nm}{layer}"]).to(device),
                                                torch.from_numpy(p[f"{bn}{layer}"]).to(device), cfg["ratio"],
                                                cfg["w_bits"], mode, dev_status=dev_status, fold=fold)
    out["W_dec"] = prepare_layer(torch.from_numpy(p["W_dec"]).to(device), torch.from_numpy(p["b_dec"]).to(device),
                                 cfg["ratio"], cfg["w_bits"], mode, dev_status=dev_status, fold=fold)
    return out


def lstm_forward(cfg, layers, tokens, a_bits: int = 8, keep: bool = False, dev_status=None, before_decoder=None):
    """tokens int32 [seq, batch] on the device -> logits fp32 [seq * batch, vocab] (h0 = c0 = 0).
    before_decoder: called right before the decoder layer (a caller that prepares the decoder's weights on
    another stream while the time steps run makes its stream wait there)."""
    seq, batch = tokens.shape
    hidden = cfg["hidden"]
    dev = tokens.device
    emb = B.ocs_embedding(layers["emb"], tokens.contiguous(), dev_status=dev_status)
    zero_h = torch.zeros((batch, hidden), dtype=torch.float32, device=dev)
    c = [torch.zeros((batch, hidden), dtype=torch.float32, device=dev) for _ in range(2)]
    # hidden states of every step, preallocated (no buffer is recycled while another stream may still read it)
    hs = [torch.empty((seq, batch, hidden), dtype=torch.float32, device=dev) for _ in range(2)]
    tops = hs[1]
    # Two kinds of concurrency, both plain stream forks and joins.  (1) The two gate GEMMs of a cell are
    # independent: the hidden-to-hidden one runs on a helper stream beside the input-to-hidden one (each a
    # latency-bound chain of quantize + GEMM), and the cell waits for both.  (2) Layer 1 of step t only needs
    # layer 0's output of step t, so it runs on its own stream while layer 0 goes on with step t + 1.
    main = torch.cuda.current_stream()
    lay = [main, _side_stream(dev, 0)]
    helper = [_side_stream(dev, 1), _side_stream(dev, 2)]
    ev_start = torch.cuda.Event()
    ev_start.record(main)
    for st in (lay[1], helper[0], helper[1]):
        st.wait_event(ev_start)                      # emb, the zero states and the layers' weights are complete
    ev_in = [torch.cuda.Event(), torch.cuda.Event()]
    ev_hh = [torch.cuda.Event(), torch.cuda.Event()]
    ev_h0 = [torch.cuda.Event() for _ in range(seq)]
    for t in range(seq):
        for l in range(2):
            with torch.cuda.stream(lay[l]):
                if l == 1:
                    lay[1].wait_event(ev_h0[t])      # layer 0's output of this step
                x = emb[t] if l == 0 else hs[0][t]
                h_prev = zero_h if t == 0 else hs[l][t - 1]
                ev_in[l].record(lay[l])              # h_prev is complete on this layer's stream
                with torch.cuda.stream(helper[l]):
                    helper[l].wait_event(ev_in[l])
                    g_hh = linear_forward(layers[f"W_hh{l}"], h_prev, True, a_bits, dev_status)
                    ev_hh[l].record(helper[l])
                g_ih = linear_forward(layers[f"W_ih{l}"], x, True, a_bits, dev_status)
                lay[l].wait_event(ev_hh[l])
                B.ocs_lstm_cell(g_ih, g_hh, c[l], hs[l][t])
                if l == 0:
                    ev_h0[t].record(lay[0])
    ev_end = torch.cuda.Event()
    ev_end.record(lay[1])
    main.wait_event(ev_end)
    if before_decoder is not None:
        before_decoder()
    logits = linear_forward(layers["W_dec"], tops.view(seq * batch, hidden), True, a_bits, dev_status)
    return (logits, dict(emb=emb, tops=tops, c=c)) if keep else logits


# ------------------------------------------------------------------------------ activation OCS
def act_ocs_linear_forward(W_codes, w_scale, bias, x, S: int, a_bits: int, a_signed: bool, dev_status=None):
    """Per-batch activation OCS (Eq. 4, Section 5.3) for a linear layer: x fp32 [M, C], W_codes int8
    [N, ld >= C] unsplit weight codes.  The batch's S outlier channels are duplicated and halved while
    being quantized (ocs_split_quantize on x), the weight columns are duplicated (ocs_dup_weight_columns)
    and the integer layer runs on C+S plain channels.  -> (Y fp32 [M, N], idx_map)."""
    M, Cn = x.shape
    N = W_codes.shape[0]
    ld = B.round_up(Cn + S, 16)
    xc, xs, _, idx_map, _, _ = B.ocs_split_quantize(x.contiguous(), S, a_bits, B.CLIP_NONE, is_signed=a_signed,
                                                    ld_codes=ld, dev_status=dev_status, want_order=False)
    Wd = torch.zeros((N, ld), dtype=torch.int8, device=x.device)
    Wd[:, :Cn] = W_codes[:, :Cn]
    B.ocs_dup_weight_columns(Wd, Cn, S, idx_map, dev_status=dev_status)
    ident = torch.arange(Cn + S, dtype=torch.int32, device=x.device)
    return B.ocs_qlinear(xc, xs, Wd, w_scale, ident, Cn + S, 0, bias=bias, dev_status=dev_status), idx_map


def act_ocs_conv_forward(W_codes, w_scale, bias, x, S: int, k: int, stride: int, pad: int, a_bits: int,
                         a_signed: bool, dev_status=None):
    """The same for a convolution: x fp32 NHWC, W_codes int8 [O, ld >= C*k*k] unsplit codes in
    [channel][tap] order.  The batch's pixels are the rows of the activation matrix."""
    Nb, H, Wd_, Cn = x.shape
    O, R = W_codes.shape[0], k * k
    xc, xs, _, idx_map, _, _ = B.ocs_split_quantize(x.reshape(Nb * H * Wd_, Cn), S, a_bits, B.CLIP_NONE,
                                                    is_signed=a_signed, ld_codes=Cn + S, dev_status=dev_status,
                                                    want_order=False)
    Wdup = torch.zeros((O, B.round_up((Cn + S) * R, 16)), dtype=torch.int8, device=x.device)
    Wdup[:, :Cn * R] = W_codes[:, :Cn * R]
    B.ocs_dup_weight_columns(Wdup, Cn, S, idx_map, R=R, dev_status=dev_status)
    packed = B.ocs_pack_conv_weights(Wdup, O, Cn + S, 0, k, k)
    ident = torch.arange(Cn + S, dtype=torch.int32, device=x.device)
    y = B.ocs_qconv(xc.view(Nb, H, Wd_, Cn + S), xs, packed, w_scale, ident, 0, k, k, stride, pad, bias=bias,
                    dev_status=dev_status)
    return y, idx_map
