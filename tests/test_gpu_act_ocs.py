"""Per-batch activation OCS (Eq. 4, Section 5.3) on the GPU against the CPU checker: the expanded
activation codes, the duplicated weight columns and the layer outputs."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from paper_1901_09504_b200 import nets
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import dev, host

pytestmark = pytest.mark.gpu


def _weights(O, Cn, R, seed):
    W = prng.laplace(seed, 3, (O, Cn * R), 0.02)
    return orc.quantize(W, 8, True, orc.maxabs(W))


def _check_codes(A, S, bits, signed):
    """Expanded activation codes, scale and index map of the fused call, bit for bit."""
    Ap, idx, order, mx = orc.act_ocs(A, S)
    o_codes, o_scale = orc.quantize(Ap, bits, signed, orc.maxabs(Ap))
    st = ocs.new_status()
    codes, scale, alpha, idx_d, order_d, mx_d = ocs.ocs_split_quantize(dev(A), S, bits, ocs.CLIP_NONE, is_signed=signed,
                                                                       dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    assert codes.dtype == (torch.int8 if signed else torch.uint8)
    np.testing.assert_array_equal(host(idx_d), idx)
    np.testing.assert_array_equal(host(order_d), order)
    assert float(host(scale)[0]) == np.float32(o_scale)
    assert host(mx_d)[1] == np.float32(mx[1])
    np.testing.assert_array_equal(host(codes)[:, :Ap.shape[1]], o_codes)


def test_expanded_activation_codes_match_checker():
    c1 = configs.config1()
    A = c1["A"]                                            # non-negative, [64, 512]
    for bits, S in ((8, 11), (6, 26), (4, 3), (6, 0)):
        _check_codes(A, S, bits, False)
    As = prng.laplace(41, 0, (200, 260), 1.0)              # signed, ragged widths
    As[17, 33] = 40.0
    As[100, 33] = -55.0
    _check_codes(As, 13, 6, True)
    _check_codes(As, 13, 6, False)                         # negatives saturate at code 0
    _check_codes(As[:1], 5, 8, True)                       # batch of one (Table 4's finest granularity)
    _check_codes(As[:, :4], 9, 5, True)                    # more splits than channels: re-splits
    _check_codes(np.zeros((8, 16), np.float32), 4, 6, False)


def test_dup_weight_columns_match_checker_and_flag_bad_indices():
    for (N, Cn, R, S) in ((33, 20, 1, 7), (16, 12, 9, 5), (5, 8, 1, 0), (300, 64, 49, 3)):
        Wc, _ = _weights(N, Cn, R, 5)
        rng = np.random.default_rng(N)
        idx = np.concatenate([np.arange(Cn), rng.integers(0, Cn, S)]).astype(np.int32)
        ref = orc.dup_weight_columns(Wc.reshape(N, Cn, R).transpose(0, 2, 1).reshape(N * R, Cn), idx)
        ref = ref.reshape(N, R, Cn + S).transpose(0, 2, 1).reshape(N, (Cn + S) * R)
        ld = ocs.round_up((Cn + S) * R, 16)
        Wd = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
        Wd[:, :Cn * R] = dev(Wc)
        st = ocs.new_status()
        ocs.ocs_dup_weight_columns(Wd, Cn, S, dev(idx), R=R, dev_status=st)
        assert ocs.ocs_poll_status(st) == 0
        np.testing.assert_array_equal(host(Wd)[:, :(Cn + S) * R], ref)
        assert not host(Wd)[:, (Cn + S) * R:].any()
    bad = np.array([0, 1, 2, 3, 7], dtype=np.int32)        # source 7 outside [0, 4)
    Wd = torch.ones((2, 16), dtype=torch.int8, device="cuda")
    st = ocs.new_status()
    ocs.ocs_dup_weight_columns(Wd, 4, 1, dev(bad), dev_status=st)
    assert ocs.ocs_poll_status(st) & 2
    with pytest.raises(ocs.OcsError):
        ocs.ocs_dup_weight_columns(torch.zeros((2, 4), dtype=torch.int8, device="cuda"), 4, 1, dev(bad))


@pytest.mark.parametrize("M,Cn,N,S,bits,signed", [(64, 512, 256, 11, 6, False), (32, 1024, 384, 21, 6, True),
                                                   (1, 256, 128, 6, 8, False), (130, 260, 72, 9, 4, True)])
def test_act_ocs_linear_layer(M, Cn, N, S, bits, signed):
    A = prng.laplace(51, M, (M, Cn), 1.0)
    if not signed:
        A = np.abs(A)
    A[M // 2, Cn // 3] = 60.0
    Wc, ws = _weights(N, Cn, 1, 9)
    bias = prng.laplace(52, 0, (N,), 0.1)
    Y_o, acc_o, ac_o, as_o, idx_o = orc.act_ocs_linear(A, S, bits, signed, Wc, ws, bias)
    st = ocs.new_status()
    Y, idx = nets.act_ocs_linear_forward(dev(Wc), dev(np.array([ws], np.float32)), dev(bias), dev(A), S, bits, signed,
                                         dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(idx), idx_o)
    np.testing.assert_allclose(host(Y), Y_o, rtol=1e-5, atol=1e-5 * np.abs(Y_o).max())
    # the integer accumulators themselves, through the plain layer call
    ld = ocs.round_up(Cn + S, 16)
    xc, xs, _, idx_d, _, _ = ocs.ocs_split_quantize(dev(A), S, bits, ocs.CLIP_NONE, is_signed=signed, ld_codes=ld)
    Wd = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
    Wd[:, :Cn] = dev(Wc)
    ocs.ocs_dup_weight_columns(Wd, Cn, S, idx_d)
    ident = torch.arange(Cn + S, dtype=torch.int32, device="cuda")
    _, acc = ocs.ocs_qlinear(xc, xs, Wd, dev(np.array([ws], np.float32)), ident, Cn + S, 0, want_acc=True)
    np.testing.assert_array_equal(host(acc), acc_o)


@pytest.mark.parametrize("Nb,H,Cn,O,k,stride,pad,S", [(2, 14, 64, 32, 3, 1, 1, 2), (4, 8, 128, 64, 1, 1, 0, 3),
                                                       (1, 9, 20, 16, 3, 2, 1, 4)])
def test_act_ocs_conv_layer(Nb, H, Cn, O, k, stride, pad, S):
    """Conv layer: the batch's pixels are the rows; checker = expanded NHWC codes through its conv."""
    R = k * k
    X = np.abs(prng.laplace(61, Nb, (Nb, H, H, Cn), 1.0))
    X[0, 3, 4, Cn // 2] = 45.0
    Wc, ws = _weights(O, Cn, R, 13)
    bias = prng.laplace(62, 0, (O,), 0.1)
    Ap, idx_o, _, _ = orc.act_ocs(X.reshape(-1, Cn), S)
    ac, a_scale = orc.quantize(Ap, 6, False, orc.maxabs(Ap))
    Wd = orc.dup_weight_columns(Wc.reshape(O, Cn, R).transpose(0, 2, 1).reshape(O * R, Cn), idx_o)
    Wd = np.ascontiguousarray(Wd.reshape(O, R, Cn + S).transpose(0, 2, 1)).reshape(O, Cn + S, k, k)
    Y_o, _ = orc.qconv(ac.reshape(Nb, H, H, Cn + S), False, a_scale, Wd, ws, np.arange(Cn + S, dtype=np.int32), stride,
                       pad, bias)
    st = ocs.new_status()
    Y, idx = nets.act_ocs_conv_forward(dev(Wc), dev(np.array([ws], np.float32)), dev(bias), dev(X), S, k, stride, pad, 6,
                                       False, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(idx), idx_o)
    np.testing.assert_allclose(host(Y), Y_o, rtol=1e-5, atol=1e-5 * np.abs(Y_o).max())


# ------------------------------------------------------------------------------ static variant (Section 5.3)
@pytest.mark.parametrize("rows,Cn,S,q,seed", [(64, 512, 11, 0.99, 0), (3000, 260, 6, 0.99, 1), (1, 8, 8, 0.5, 2),
                                               (40000, 64, 2, 0.999, 3), (17, 1030, 0, 0.9, 4), (500, 96, 5, 1.0, 5)])
def test_static_channel_choice_matches_checker(rows, Cn, S, q, seed):
    P = prng.laplace(70 + seed, 0, (rows, Cn), 1.0)
    P[:, Cn // 3] *= 2.5                                    # heavier tails in two channels
    P[:, Cn - 1] *= 2.0
    P[rows // 2, 0] = 0.0
    P[0, Cn // 2] = -0.0
    sel_o, counts_o, thr_o = orc.act_select(P, S, q)
    st = ocs.new_status()
    sel, counts, thr = ocs.ocs_act_select_channels(dev(P), S, q, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    assert host(thr)[0] == np.float32(thr_o)
    np.testing.assert_array_equal(host(counts), counts_o)
    np.testing.assert_array_equal(host(sel), sel_o)


def test_static_channel_choice_with_padded_rows_and_ties():
    base = np.zeros((32, 24), np.float32)                   # everything ties: the first S channels win
    Pd = torch.full((32, 40), 7.0, dtype=torch.float32, device="cuda")
    Pd[:, :24] = dev(base)
    sel, counts, thr = ocs.ocs_act_select_channels(Pd[:, :24], 5, 0.99)
    assert host(sel).tolist() == [0, 1, 2, 3, 4] and host(thr)[0] == 0.0 and not host(counts).any()
    st = ocs.new_status()
    bad = dev(np.array([[1.0, np.inf, 2.0, 3.0]], np.float32))
    ocs.ocs_act_select_channels(bad, 1, 0.5, dev_status=st)
    assert ocs.ocs_poll_status(st) & 1


def _check_static_codes(A, sel, bits, signed, alpha=None):
    Ap, idx_o = orc.act_split_static(A, sel)
    a = float(np.float32(alpha)) if alpha is not None else orc.maxabs(Ap)
    o_codes, o_scale = orc.quantize(Ap, bits, signed, a)
    st = ocs.new_status()
    alpha_d = None if alpha is None else dev(np.array([alpha], np.float32))
    codes, scale, idx = ocs.ocs_act_split_quantize_static(dev(A), dev(np.asarray(sel, np.int32)), bits, signed,
                                                          alpha_in=alpha_d, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(idx), idx_o)
    assert float(host(scale)[0]) == np.float32(o_scale)
    np.testing.assert_array_equal(host(codes)[:, :Ap.shape[1]], o_codes)


def test_static_activation_codes_match_checker():
    A = np.abs(prng.laplace(81, 0, (300, 260), 1.0))
    A[5, 100] = 33.0
    _check_static_codes(A, [100, 7, 259, 0], 6, False)               # dynamic grid
    _check_static_codes(A, [100, 7, 259, 0], 6, False, alpha=9.5)    # profiled threshold: the outlier's halves saturate
    _check_static_codes(A, [], 8, False)
    As = prng.laplace(82, 0, (70, 512), 1.0)
    _check_static_codes(As, list(range(0, 512, 37)), 5, True)
    _check_static_codes(As[:1], [3], 8, True, alpha=2.0)
    _check_static_codes(np.zeros((8, 16), np.float32), [1, 2], 6, False)
    _check_static_codes(As[:, :8], list(range(8)), 4, True)          # every channel split
    # a channel listed twice or out of range is flagged
    for bad in ([3, 3], [600]):
        st = ocs.new_status()
        ocs.ocs_act_split_quantize_static(dev(As), dev(np.array(bad, np.int32)), 6, True, dev_status=st)
        assert ocs.ocs_poll_status(st) & 2
    with pytest.raises(ocs.OcsError):
        ocs.ocs_act_split_quantize_static(dev(As[:, :4]), dev(np.arange(5, dtype=np.int32) % 4), 6, True)   # S > C


def test_static_act_ocs_layer_end_to_end():
    """Profile on one batch, split another: selection -> expanded codes -> duplicated weights -> layer."""
    Cn, N, S = 256, 96, 6
    P = np.abs(prng.laplace(91, 0, (4096, Cn), 1.0))
    P[:, 40] *= 3.0
    A = np.abs(prng.laplace(92, 0, (128, Cn), 1.0))
    A[:, 40] *= 3.0
    Wc, ws = _weights(N, Cn, 1, 17)
    sel_o, _, _ = orc.act_select(P, S, 0.99)
    Ap, idx_o = orc.act_split_static(A, sel_o)
    ac, a_scale = orc.quantize(Ap, 6, False, orc.maxabs(Ap))
    Y_o, acc_o = orc.qlinear(ac, False, a_scale, orc.dup_weight_columns(Wc, idx_o), ws,
                             np.arange(Cn + S, dtype=np.int32))
    sel, _, _ = ocs.ocs_act_select_channels(dev(P), S, 0.99)
    ld = ocs.round_up(Cn + S, 16)
    codes, scale, idx = ocs.ocs_act_split_quantize_static(dev(A), sel, 6, False, ld_codes=ld)
    Wd = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
    Wd[:, :Cn] = dev(Wc)
    ocs.ocs_dup_weight_columns(Wd, Cn, S, idx)
    ident = torch.arange(Cn + S, dtype=torch.int32, device="cuda")
    Y, acc = ocs.ocs_qlinear(codes, scale, Wd, dev(np.array([ws], np.float32)), ident, Cn + S, 0, want_acc=True)
    assert 40 in host(sel).tolist()
    np.testing.assert_array_equal(host(acc), acc_o)
    np.testing.assert_allclose(host(Y), Y_o, rtol=1e-5, atol=1e-5 * np.abs(Y_o).max())
