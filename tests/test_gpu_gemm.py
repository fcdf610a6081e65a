"""GPU parity: ocs_qlinear / ocs_qconv against the CPU checker, through the C ABI.
Bars: int32 accumulators bit-exact; Y <= 1e-5 relative (it is one fmaf of exact inputs on both
sides, so equality is asserted too)."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import dev, host

pytestmark = pytest.mark.gpu


def _rand_idx(seed, Cn, S):
    return np.concatenate([np.arange(Cn), configs.random_codes(seed, 7, (S,), 0, Cn - 1, np.int32)]).astype(np.int32) \
        if S else np.arange(Cn, dtype=np.int32)


def _check_linear(seed, M, Cn, N, S, a_signed=False, lda=None, bias=True, a_scale=0.013, w_scale=0.0007):
    A = configs.random_codes(seed, 0, (M, Cn), -127 if a_signed else 0, 127 if a_signed else 255,
                             np.int8 if a_signed else np.uint8)
    Wc = configs.random_codes(seed, 1, (N, Cn + S), -127, 127, np.int8)
    idx = _rand_idx(seed, Cn, S)
    b = prng.normal(seed, 9, (N,)) if bias else None
    Yo, acco = orc.qlinear(A, a_signed, a_scale, Wc, w_scale, idx, b)
    lda = lda or Cn
    Ad = torch.zeros((M, lda), dtype=torch.int8 if a_signed else torch.uint8, device="cuda")
    Ad[:, :Cn] = dev(A)
    ldw = ocs.round_up(Cn + S, 16)
    Wd = torch.zeros((N, ldw), dtype=torch.int8, device="cuda")
    Wd[:, :Cn + S] = dev(Wc)
    st = ocs.new_status()
    Y, acc = ocs.ocs_qlinear(Ad, dev(np.array([a_scale], np.float32)), Wd, dev(np.array([w_scale], np.float32)),
                             dev(idx), Cn, S, bias=None if b is None else dev(b), want_acc=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(acc), acco)
    np.testing.assert_allclose(host(Y), Yo, rtol=1e-5, atol=0)
    np.testing.assert_array_equal(host(Y), Yo)
    # the same layer with the channel-major copy of the activations: the duplicated channels arrive as whole rows
    # of that copy (no byte gather); identical accumulators
    AT = ocs.ocs_transpose_codes(Ad, cols=Cn)
    np.testing.assert_array_equal(host(AT)[:, :M], A.T)
    Yt, acct = ocs.ocs_qlinear(Ad, dev(np.array([a_scale], np.float32)), Wd, dev(np.array([w_scale], np.float32)),
                               dev(idx), Cn, S, bias=None if b is None else dev(b), want_acc=True, dev_status=st,
                               A_codes_T=AT)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(acct), acco)
    np.testing.assert_array_equal(host(Yt), Yo)
    # ReLU and max |Y| taken in the layer's epilogue: the checker's relu and maxabs of its own output
    m = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    Yr = ocs.ocs_qlinear(Ad, dev(np.array([a_scale], np.float32)), Wd, dev(np.array([w_scale], np.float32)),
                         dev(idx), Cn, S, bias=None if b is None else dev(b), relu=True, max_out=m, dev_status=st)
    np.testing.assert_array_equal(host(Yr), orc.relu(Yo))
    assert host(m)[0] == np.float32(orc.maxabs(orc.relu(Yo)))
    ocs.ocs_qlinear(Ad, dev(np.array([a_scale], np.float32)), Wd, dev(np.array([w_scale], np.float32)),
                    dev(idx), Cn, S, bias=None if b is None else dev(b), max_out=m, dev_status=st)
    assert host(m)[0] == np.float32(orc.maxabs(Yo)) and ocs.ocs_poll_status(st) == 0
    # a shortcut tensor added in the epilogue: the checker's add_relu on its own output
    res = prng.normal(seed, 11, (M, N))
    Ys = ocs.ocs_qlinear(Ad, dev(np.array([a_scale], np.float32)), Wd, dev(np.array([w_scale], np.float32)),
                         dev(idx), Cn, S, bias=None if b is None else dev(b), residual=dev(res), relu=True, max_out=m,
                         dev_status=st)
    ref = orc.add_relu(Yo, res, True)
    np.testing.assert_array_equal(host(Ys), ref)
    assert host(m)[0] == np.float32(orc.maxabs(ref)) and ocs.ocs_poll_status(st) == 0


@pytest.mark.parametrize("M,Cn,N,S", [(64, 512, 256, 26), (128, 256, 128, 0), (1, 16, 8, 0), (5, 130, 70, 3),
                                      (200, 384, 300, 140), (20, 650, 2600, 13), (128, 1000, 64, 17)])
def test_qlinear_tma_path(M, Cn, N, S):
    _check_linear(M + Cn, M, Cn, N, S, lda=ocs.round_up(Cn, 16))


@pytest.mark.parametrize("M,Cn,N,S", [(64, 515, 256, 26), (3, 7, 5, 2), (130, 129, 33, 1)])
def test_qlinear_gather_path(M, Cn, N, S):
    _check_linear(M + Cn + 1, M, Cn, N, S, lda=Cn + 1)       # unaligned rows: every block is assembled by threads


def test_qlinear_signed_nobias_and_splitk():
    _check_linear(11, 20, 650, 2600, 13, a_signed=True, lda=656)
    _check_linear(12, 128, 6272, 512, 314, bias=False, lda=6272)    # few tiles, long K: split-K
    _check_linear(13, 100, 4099, 200, 77, lda=4112)


def test_qlinear_config1_end_to_end():
    """split -> quantize -> activation quantize -> qlinear, every stage compared."""
    c = configs.config1()
    W, A = c["W"], c["A"]
    S = 26
    Wp, idx, _, _ = orc.split(W, S)
    wc, ws_ = orc.quantize(Wp, 8, True, orc.maxabs(Wp))
    ac, as_ = orc.quantize(A, 8, False, orc.maxabs(A))
    Yo, acco = orc.qlinear(ac, False, as_, wc, ws_, idx)
    Wout, idx_d, _, mx = ocs.ocs_split(dev(W), S)
    codes, scale, _ = ocs.ocs_quantize(Wout, 8, True, ocs.CLIP_NONE, cols=512 + S, max_abs_in=mx[1:2])
    acodes, ascale, _ = ocs.ocs_quantize(dev(A), 8, False, ocs.CLIP_NONE)
    Y, acc = ocs.ocs_qlinear(acodes, ascale, codes, scale, idx_d, 512, S, want_acc=True)
    np.testing.assert_array_equal(host(codes)[:, :512 + S], wc)
    np.testing.assert_array_equal(host(acc), acco)
    np.testing.assert_array_equal(host(Y), Yo)
    # the quantized split layer tracks the float layer (Eq. 3 = Eq. 2 up to quantization error)
    ref = A.astype(np.float64) @ W.astype(np.float64).T
    assert np.abs(host(Y) - ref).max() < 0.02 * np.abs(ref).max()


def test_qlinear_bad_index_flag_and_args():
    A = torch.zeros((8, 32), dtype=torch.uint8, device="cuda")
    Wd = torch.zeros((8, 48), dtype=torch.int8, device="cuda")
    idx = np.arange(34, dtype=np.int32)
    idx[33] = 99
    one = dev(np.ones(1, np.float32))
    st = ocs.new_status()
    ocs.ocs_qlinear(A, one, Wd, one, dev(idx), 32, 2, dev_status=st)
    assert ocs.ocs_poll_status(st) & ocs.DEV_BAD_INDEX
    with pytest.raises(ocs.OcsError):
        ocs.ocs_qlinear(A, one, Wd[:, :40], one, dev(idx), 32, 20)       # ldw too small


def _check_conv(seed, Nb, H, Wd_, Cn, O, S, k, stride, pad, a_signed=False):
    X = configs.random_codes(seed, 0, (Nb, H, Wd_, Cn), -127 if a_signed else 0, 127 if a_signed else 255,
                             np.int8 if a_signed else np.uint8)
    Wc = configs.random_codes(seed, 1, (O, Cn + S, k, k), -127, 127, np.int8)
    idx = _rand_idx(seed, Cn, S)
    b = prng.normal(seed, 9, (O,))
    Yo, acco = orc.qconv(X, a_signed, 0.02, Wc, 0.003, idx, stride, pad, b)
    packed = ocs.ocs_pack_conv_weights(dev(Wc.reshape(O, -1)), O, Cn, S, k, k)
    # the packing is a pure permutation: check it against numpy
    Cp = ocs.ocs_conv_packed_k(Cn, 0, 1, 1)          # per-tap stride: C, or C padded to the K-block
    orig = np.zeros((O, k, k, Cp), np.int8)
    orig[..., :Cn] = Wc[:, :Cn].transpose(0, 2, 3, 1)
    ref_pack = np.concatenate([orig.reshape(O, -1), Wc[:, Cn:].transpose(0, 2, 3, 1).reshape(O, -1)], axis=1)
    assert ref_pack.shape[1] == ocs.ocs_conv_packed_k(Cn, S, k, k)
    np.testing.assert_array_equal(host(packed)[:, :ref_pack.shape[1]], ref_pack)
    assert not host(packed)[:, ref_pack.shape[1]:].any()
    st = ocs.new_status()
    Y, acc = ocs.ocs_qconv(dev(X), dev(np.array([0.02], np.float32)), packed, dev(np.array([0.003], np.float32)),
                           dev(idx), S, k, k, stride, pad, bias=dev(b), want_acc=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(acc), acco)
    np.testing.assert_array_equal(host(Y), Yo)
    m = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    Yr = ocs.ocs_qconv(dev(X), dev(np.array([0.02], np.float32)), packed, dev(np.array([0.003], np.float32)),
                       dev(idx), S, k, k, stride, pad, bias=dev(b), relu=True, max_out=m, dev_status=st)
    np.testing.assert_array_equal(host(Yr), orc.relu(Yo))
    assert host(m)[0] == np.float32(orc.maxabs(orc.relu(Yo))) and ocs.ocs_poll_status(st) == 0
    res = prng.normal(seed, 11, Yo.shape)
    Ys = ocs.ocs_qconv(dev(X), dev(np.array([0.02], np.float32)), packed, dev(np.array([0.003], np.float32)),
                       dev(idx), S, k, k, stride, pad, bias=dev(b), residual=dev(res), relu=False, max_out=m, dev_status=st)
    ref = orc.add_relu(Yo, res, False)
    np.testing.assert_array_equal(host(Ys), ref)
    assert host(m)[0] == np.float32(orc.maxabs(ref)) and ocs.ocs_poll_status(st) == 0


@pytest.mark.parametrize("Nb,H,W,Cn,O,S,k,stride,pad", [
    (2, 7, 8, 5, 4, 3, 3, 1, 1),        # tiny, odd channels
    (2, 11, 11, 3, 16, 1, 7, 2, 3),     # first-layer shape: 3 channels, 7x7 stride 2
    (3, 14, 14, 128, 64, 2, 3, 1, 1),   # C = 128: original channels by TMA, duplicates by threads
    (2, 9, 9, 256, 40, 3, 1, 1, 0),     # 1x1
    (2, 14, 14, 64, 32, 1, 3, 1, 1),    # C = 64: blocks straddle taps
    (2, 16, 16, 128, 24, 2, 3, 2, 1),   # stride 2
    (2, 8, 8, 256, 24, 3, 1, 2, 0),     # 1x1 stride 2 (downsample)
    (1, 5, 6, 32, 8, 0, 3, 1, 1),       # no splits
])
def test_qconv_shapes(Nb, H, W, Cn, O, S, k, stride, pad):
    _check_conv(Nb * 100 + Cn, Nb, H, W, Cn, O, S, k, stride, pad)


def test_qconv_signed_input():
    _check_conv(5, 2, 9, 9, 3, 8, 1, 7, 2, 3, a_signed=True)


def test_qconv_config2_reduced_batch():
    """Config 2's layer (256 -> 256, 3x3, 14x14, r = 0.02, 6-bit MSE-clipped weights) on 4 images."""
    c = configs.config2(batch=4)
    W, X = c["W"], c["X"]
    S = 6
    Wp, idx, _, _ = orc.split(W, S)
    alpha = orc.clip_mse(Wp, 6, True, 2048, 128)["alpha"]
    wc, wscale = orc.quantize(Wp, 6, True, alpha)
    Xh = orc.nchw_to_nhwc(X)
    xc, xscale = orc.quantize(Xh, 8, False, orc.maxabs(Xh))
    Yo, acco = orc.qconv(xc, False, xscale, wc, wscale, idx, 1, 1)
    Wout, idx_d, _, mx = ocs.ocs_split(dev(W), S)
    codes, scale, al = ocs.ocs_quantize(Wout, 6, True, ocs.CLIP_MSE, cols=(256 + S) * 9, max_abs_in=mx[1:2])
    assert np.float32(host(al)[0]) == np.float32(alpha)
    packed = ocs.ocs_pack_conv_weights(codes, 256, 256, S, 3, 3)
    xcodes, xs, _ = ocs.ocs_quantize(dev(Xh).reshape(-1, 256), 8, False, ocs.CLIP_NONE)
    Y, acc = ocs.ocs_qconv(xcodes.reshape(4, 14, 14, 256), xs, packed, scale, idx_d, S, 3, 3, 1, 1, want_acc=True)
    np.testing.assert_array_equal(host(acc), acco)
    np.testing.assert_array_equal(host(Y), Yo)


def test_qconv_first_layer_with_and_without_room_for_the_patch_matrix():
    """A 3-channel 7x7 stride-2 layer runs over its patch matrix when the workspace has room for it and through
    the in-kernel gather when it has not: the same accumulators either way."""
    Nb, H, Cn, O, S, k, stride, pad = 3, 20, 3, 16, 1, 7, 2, 3
    X = configs.random_codes(77, 0, (Nb, H, H, Cn), 0, 255, np.uint8)
    Wc = configs.random_codes(77, 1, (O, Cn + S, k, k), -127, 127, np.int8)
    idx = np.array([0, 1, 2, 1], np.int32)
    Yo, acco = orc.qconv(X, False, 0.02, Wc, 0.003, idx, stride, pad, None)
    packed = ocs.ocs_pack_conv_weights(dev(Wc.reshape(O, -1)), O, Cn, S, k, k)
    full = ocs.lib().ocs_qconv_workspace_bytes(Nb, H, H, Cn, O, S, k, k, stride, pad)
    Ho = (H + 2 * pad - k) // stride + 1
    assert full >= Nb * Ho * Ho * 196                      # includes the patch matrix
    for nbytes in (full, 1024):
        ws = torch.empty(int(nbytes), dtype=torch.uint8, device="cuda")
        st = ocs.new_status()
        Y, acc = ocs.ocs_qconv(dev(X), dev(np.array([0.02], np.float32)), packed, dev(np.array([0.003], np.float32)),
                               dev(idx), S, k, k, stride, pad, want_acc=True, dev_status=st, ws=ws)
        assert ocs.ocs_poll_status(st) == 0
        np.testing.assert_array_equal(host(acc), acco)
        np.testing.assert_array_equal(host(Y), Yo)


def test_accumulators_do_not_depend_on_the_tile_plan():
    """One problem under several forced (tile width, K split) plans: the int32 accumulators and
    the outputs are identical, and equal the checker's (integer sums do not depend on their order)."""
    M, Cn, N, S = 200, 2100, 384, 150
    A = configs.random_codes(31, 0, (M, Cn), 0, 255, np.uint8)
    Wc = configs.random_codes(31, 1, (N, Cn + S), -127, 127, np.int8)
    idx = np.concatenate([np.arange(Cn), configs.random_codes(31, 2, (S,), 0, Cn - 1, np.int32)]).astype(np.int32)
    bias = prng.normal(31, 3, (N,))
    Yo, acco = orc.qlinear(A, False, 0.013, Wc, 0.0007, idx, bias)
    ld = ocs.round_up(Cn + S, 16)
    Wd = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
    Wd[:, :Cn + S] = dev(Wc)
    Ad = torch.zeros((M, ocs.round_up(Cn, 16)), dtype=torch.uint8, device="cuda")
    Ad[:, :Cn] = dev(A)
    sa, sw = dev(np.array([0.013], np.float32)), dev(np.array([0.0007], np.float32))
    AT = ocs.ocs_transpose_codes(Ad, cols=Cn)
    try:
        for bn, sk in ((0, 0), (64, 1), (128, 1), (256, 1), (128, 2), (128, 4), (64, 2), (64, 4), (64, 8), (256, 2),
                       (256, 4), (256, 8), (128, 8), (192, 1), (192, 2), (192, 4)):
            ocs.ocs_selftest_force_gemm_plan(bn, sk)
            st = ocs.new_status()
            for _ in range(2):
                for at in (None, AT):
                    Y, acc = ocs.ocs_qlinear(Ad, sa, Wd, sw, dev(idx), Cn, S, bias=dev(bias), want_acc=True, dev_status=st,
                                             A_codes_T=at)
                    assert ocs.ocs_poll_status(st) == 0
                    np.testing.assert_array_equal(host(acc), acco, err_msg=f"plan {(bn, sk)}")
                    np.testing.assert_array_equal(host(Y), Yo, err_msg=f"plan {(bn, sk)}")
    finally:
        ocs.ocs_selftest_force_gemm_plan(0, 0)


@pytest.mark.parametrize("split", [False, True])
def test_shortcut_tensor_that_is_not_16_byte_aligned(split):
    """A shortcut tensor that starts 4 bytes into its buffer (a view): the epilogue reads it with scalar loads
    and the result is the checker's."""
    M, Cn, N, S = 96, 640, 256, 13
    if split:
        Cn = 4096                                                   # few tiles, long K: the planner slices K
    A = configs.random_codes(41, 0, (M, Cn), 0, 255, np.uint8)
    Wc = configs.random_codes(41, 1, (N, Cn + S), -127, 127, np.int8)
    idx = _rand_idx(41, Cn, S)
    Yo, _ = orc.qlinear(A, False, 0.02, Wc, 0.001, idx, None)
    res = prng.normal(41, 5, (M, N))
    buf = torch.zeros(M * N + 1, dtype=torch.float32, device="cuda")
    view = buf[1:].view(M, N)
    view.copy_(dev(res))
    assert view.data_ptr() % 16 == 4
    Wd = torch.zeros((N, ocs.round_up(Cn + S, 16)), dtype=torch.int8, device="cuda")
    Wd[:, :Cn + S] = dev(Wc)
    st = ocs.new_status()
    Y = ocs.ocs_qlinear(dev(A), dev(np.array([0.02], np.float32)), Wd, dev(np.array([0.001], np.float32)), dev(idx), Cn, S,
                        residual=view, relu=True, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(Y), orc.add_relu(Yo, res, True))


@pytest.mark.parametrize("rows,cols,ld,ld_t", [(128, 25088, 25088, 128), (20, 650, 656, 32), (7, 5, 5, 7), (300, 1031, 1040, 304),
                                                (129, 130, 131, 133), (4, 4, 4, 4)])
def test_transpose_codes(rows, cols, ld, ld_t):
    A = configs.random_codes(51, 0, (rows, cols), 0, 255, np.uint8)
    Ad = torch.zeros((rows, ld), dtype=torch.uint8, device="cuda")
    Ad[:, :cols] = dev(A)
    T = torch.full((cols, ld_t), 7, dtype=torch.uint8, device="cuda")
    ocs.ocs_transpose_codes(Ad, cols=cols, out=T)
    got = host(T)
    np.testing.assert_array_equal(got[:, :rows], A.T)
    assert (got[:, rows:] == 7).all()                      # padding beyond the rows is left alone
