"""GPU parity at the full sizes of the five workloads, in the launch configurations the bench
times.  Where the CPU checker can produce the whole result in seconds it is compared in full;
the fc6 GEMM (at every sweep point kind) and every batch-128 ResNet-50 layer are compared on sampled
outputs that the checker computes one by one from the GPU path's own inputs to that layer."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs
from oracle import oracle as orc
from paper_1901_09504_b200 import nets

from oracle import net_oracle
from gpu_util import clear_winner, dev, host

pytestmark = pytest.mark.gpu


_C3 = {}


def _config3():
    """The fc6-shaped tensors, generated once per test process."""
    if "c" not in _C3:
        _C3["c"] = configs.config3()
        A = _C3["c"]["A"]
        _C3["ac"], _C3["ascale"] = orc.quantize(A, 8, False, orc.maxabs(A))
    return _C3["c"], _C3["ac"], _C3["ascale"]


# Table 2's sweep structure: every expand ratio at one bit width (r = 0: no split, the last partial K-block
# arrives by TMA; r = 0.1: 2509 splits, every one a tie-break), the other bit widths at one ratio, and one point
# under the quantization-aware split.  Each point runs at W [4096, 25088], activations [128, 25088]: the launch
# configuration the bench times.
_C3_POINTS = [(0.0, 4, 0), (0.01, 4, 0), (0.02, 4, 0), (0.05, 4, 0), (0.1, 4, 0), (0.1, 5, 0), (0.1, 6, 0), (0.1, 8, 0),
              (0.05, 6, 6)]


@pytest.mark.parametrize("ratio,bits,qa_bits", _C3_POINTS)
def test_config3_fc6_full_size_points(ratio, bits, qa_bits):
    """Split and codes compared in full, 4000 sampled GEMM outputs, and the fused call's codes."""
    c, ac, ascale = _config3()
    W, A = c["W"], c["A"]
    Cn = W.shape[1]
    S = ocs.ocs_num_splits(Cn, ratio)
    assert S == orc.num_splits(Cn, ratio)
    if qa_bits:
        Wp, idx, order, mx, step = orc.split_qa(W, S, qa_bits)
    else:
        Wp, idx, order, mx = orc.split(W, S, 0.0)
        step = 0.0
    srch = orc.clip_mse(Wp, bits, True, 2048, 128)
    assert clear_winner(srch["scores"])
    wc, wscale = orc.quantize(Wp, bits, True, srch["alpha"])
    st = ocs.new_status()
    Wd = dev(W)
    Wout, idx_d, order_d, mx_d = ocs.ocs_split(Wd, S, qa_bits=qa_bits, ld_out=ocs.round_up(Cn + S, 16), dev_status=st)
    np.testing.assert_array_equal(host(idx_d), idx)
    np.testing.assert_array_equal(host(order_d), order)
    assert host(mx_d)[0] == np.float32(mx[0]) and host(mx_d)[1] == np.float32(mx[1]) and host(mx_d)[2] == np.float32(step)
    np.testing.assert_array_equal(host(Wout)[:, :Cn + S].view(np.uint32), Wp.view(np.uint32))
    codes, scale, alpha, hist, _ = ocs.ocs_quantize(Wout, bits, True, ocs.CLIP_MSE, 128, 2048, cols=Cn + S,
                                                     max_abs_in=mx_d[1:2], dev_status=st, return_search=True)
    np.testing.assert_array_equal(host(hist).astype(np.uint64), srch["hist"])
    assert np.float32(host(alpha)[0]) == np.float32(srch["alpha"])
    assert abs(float(host(alpha)[0]) - srch["alpha"]) <= 1e-5 * srch["alpha"]
    assert float(host(scale)[0]) == np.float32(wscale)
    np.testing.assert_array_equal(host(codes)[:, :Cn + S], wc)
    del Wout
    a_codes, a_scale, _ = ocs.ocs_quantize(dev(A), 8, False, ocs.CLIP_NONE, dev_status=st)
    np.testing.assert_array_equal(host(a_codes)[:, :Cn], ac)
    # the launch configuration the bench times: with duplicated channels, gathered from the channel-major copy
    a_T = ocs.ocs_transpose_codes(a_codes, cols=Cn) if S > 0 else None
    Y, acc = ocs.ocs_qlinear(a_codes, a_scale, codes, scale, idx_d, Cn, S, want_acc=True, dev_status=st, A_codes_T=a_T)
    assert ocs.ocs_poll_status(st) == 0
    if S > 0:        # and the byte gather from the row-major codes gives the same accumulators
        acc_b = ocs.ocs_qlinear(a_codes, a_scale, codes, scale, idx_d, Cn, S, want_acc=True, dev_status=st)[1]
        assert torch.equal(acc, acc_b)
    rng = np.random.default_rng(3)
    ms = np.concatenate([rng.integers(0, A.shape[0], 3996), [0, 0, 127, 127]]).astype(np.int32)
    ns = np.concatenate([rng.integers(0, W.shape[0], 3996), [0, 4095, 0, 4095]]).astype(np.int32)
    Ys, accs = orc.qlinear_samples(ac, False, ascale, wc, wscale, idx, ms, ns)
    np.testing.assert_array_equal(host(acc)[ms, ns], accs)                      # int32 accumulators: bit-exact
    np.testing.assert_allclose(host(Y)[ms, ns], Ys, rtol=1e-5, atol=0)
    np.testing.assert_array_equal(host(Y)[ms, ns], Ys)
    # the fused call (no fp32 W') gives the same codes, scale and index map
    fc, fs, fa, fidx, _, _ = ocs.ocs_split_quantize(Wd, S, bits, ocs.CLIP_MSE, qa_bits=qa_bits, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(fidx), idx)
    assert host(fs)[0] == host(scale)[0] and host(fa)[0] == host(alpha)[0]
    np.testing.assert_array_equal(host(fc)[:, :Cn + S], wc)


def test_config2_conv_full_batch():
    """The 3x3 convolution at its full batch of 32: every stage compared in full."""
    c = configs.config2()
    W, X = c["W"], c["X"]
    S = ocs.ocs_num_splits(256, c["ratio"])
    Wp, idx, _, _ = orc.split(W, S)
    alpha = orc.clip_mse(Wp, 6, True, 2048, 128)["alpha"]
    wc, wscale = orc.quantize(Wp, 6, True, alpha)
    Xh = orc.nchw_to_nhwc(X)
    xc, xscale = orc.quantize(Xh, 8, False, orc.maxabs(Xh))
    Yo, acco = orc.qconv(xc, False, xscale, wc, wscale, idx, 1, 1)
    st = ocs.new_status()
    L = nets.prepare_layer(dev(W), None, c["ratio"], 6, ocs.CLIP_MSE, conv=True, stride=1, pad=1, dev_status=st)
    np.testing.assert_array_equal(host(L.idx_map), idx)
    assert float(host(L.w_scale)[0]) == np.float32(wscale)
    xd = ocs.ocs_nchw_to_nhwc(dev(X))
    np.testing.assert_array_equal(host(xd), Xh)
    xcodes, xs = nets.quantize_activations(xd, False, dev_status=st)
    np.testing.assert_array_equal(host(xcodes), xc)
    Y, acc = ocs.ocs_qconv(xcodes, xs, L.codes, L.w_scale, L.idx_map, S, 3, 3, 1, 1, want_acc=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(acc), acco)
    np.testing.assert_allclose(host(Y), Yo, rtol=1e-5, atol=0)
    np.testing.assert_array_equal(host(Y), Yo)


def _conv_samples(x_codes, a_signed, wc, idx, spec, positions):
    """int64 accumulators of a convolution at (n, oh, ow, o) positions, written out directly."""
    Nb, H, Wd, Cn = x_codes.shape
    xs = x_codes.astype(np.int64)
    out = []
    for n, oh, ow, o in positions:
        a = 0
        for dy in range(spec.k):
            for dx in range(spec.k):
                ih, iw = oh * spec.stride + dy - spec.pad, ow * spec.stride + dx - spec.pad
                if 0 <= ih < H and 0 <= iw < Wd:
                    a += int(np.dot(xs[n, ih, iw, idx], wc[o, :, dy, dx].astype(np.int64)))
        out.append(a)
    return np.array(out, dtype=np.int64)


def test_config4_resnet50_batch128_every_layer():
    """The ResNet-50 stack at batch 128 and 224x224 (the bench's launch configuration): the forward pass
    runs in full on the GPU; every one of the 53 convolutions and the fully-connected layer is checked on
    about 150 sampled outputs plus the image corners, which the checker recomputes from the GPU path's own
    input to that layer (so one early mismatch cannot hide later layers, and every tile plan the library
    picks at this size meets the checker)."""
    cfg = configs.config4()
    st = ocs.new_status()
    layers = nets.prepare_resnet50(cfg, torch.device("cuda"), dev_status=st)
    logits, t = nets.resnet50_forward(cfg, layers, dev(cfg["X"]), keep=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    assert torch.isfinite(logits).all()
    rng = np.random.default_rng(4)
    prev = None                       # name of the tensor the next layer reads when its spec names none
    for li, spec in enumerate(cfg["layers"]):
        name = spec.name
        first = li == 0
        W, bias = cfg["params"][name]
        S = orc.num_splits(spec.C, cfg["ratio"])
        Wp, idx, _, _ = orc.split(W, S)
        wc, wscale = orc.quantize(Wp, 8, True, orc.maxabs(Wp))
        np.testing.assert_array_equal(host(layers[name].idx_map), idx, err_msg=name)
        assert float(host(layers[name].w_scale)[0]) == np.float32(wscale), name
        src = spec.input_from if spec.input_from else prev
        x_in = orc.nchw_to_nhwc(cfg["X"]) if first else host(t[src])
        xc, xscale = orc.quantize(x_in, 8, first, orc.maxabs(x_in))
        del x_in
        Ho = spec.H_out
        pos = [(int(rng.integers(0, 128)), int(rng.integers(0, Ho)), int(rng.integers(0, Ho)), int(rng.integers(0, spec.O)))
               for _ in range(150)]
        pos += [(0, 0, 0, 0), (127, Ho - 1, Ho - 1, spec.O - 1), (5, 0, Ho - 1, 1)]          # image corners: padding taps
        acc = _conv_samples(xc, first, wc, idx, spec, pos)
        s_prod = np.float32(xscale) * np.float32(wscale)
        y = np.array([np.float32(np.float64(np.float32(a)) * np.float64(s_prod) + np.float64(bias[o]))
                      for a, (_, _, _, o) in zip(acc, pos)], dtype=np.float32)           # fmaf: one rounding
        got = host(t[name])
        got_s = np.array([got[p[0], p[1], p[2], p[3]] for p in pos])
        if spec.residual_from:
            res = host(t[spec.residual_from])
            y = np.array([np.float32(v + res[p[0], p[1], p[2], p[3]]) for v, p in zip(y, pos)], dtype=np.float32)
        if spec.relu:
            y = np.maximum(y, np.float32(0))
        np.testing.assert_allclose(got_s, y, rtol=1e-5, atol=0, err_msg=name)
        np.testing.assert_array_equal(got_s, y, err_msg=name)
        prev = "pool" if first else name
    # the classifier on the GPU path's own pooled features, in full
    fc = cfg["fc"]
    W, bias = cfg["params"]["fc"]
    W2 = W.reshape(fc.O, fc.C)
    S = orc.num_splits(fc.C, cfg["ratio"])
    Wp, idx, _, _ = orc.split(W2, S)
    wc, wscale = orc.quantize(Wp, 8, True, orc.maxabs(Wp))
    feat = host(t["avgpool"])
    fcodes, fscale = orc.quantize(feat, 8, False, orc.maxabs(feat))
    Yo, _ = orc.qlinear(fcodes, False, fscale, wc, wscale, idx, bias)
    np.testing.assert_array_equal(host(logits), Yo)


def test_config5_lstm_full_size():
    """The full language model: vocabulary 33278, batch 20, 35 time steps, compared in full."""
    cfg = configs.config5()
    ref_logits, ref = net_oracle.lstm(cfg)
    st = ocs.new_status()
    layers = nets.prepare_lstm(cfg, torch.device("cuda"), dev_status=st)
    logits, t = nets.lstm_forward(cfg, layers, dev(cfg["tokens"]), keep=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(t["tops"]), ref["tops"])
    np.testing.assert_allclose(host(logits), ref_logits, rtol=1e-5, atol=0)
    np.testing.assert_array_equal(host(logits), ref_logits)
