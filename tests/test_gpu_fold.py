"""ocs_fold_duplicates on the GPU against the CPU checker, and the folded layer against the gathered one."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import dev, host

pytestmark = pytest.mark.gpu


def _fold(Wc2d, Cn, S, R, idx, ld=None):
    st = ocs.new_status()
    ldw = ld or ocs.round_up((Cn + S) * R, 16)
    Wd = torch.zeros((Wc2d.shape[0], ldw), dtype=torch.int8, device="cuda")
    Wd[:, :(Cn + S) * R] = dev(Wc2d)
    out = ocs.ocs_fold_duplicates(Wd, Cn, S, dev(idx), R=R, dev_status=st)
    return out, ocs.ocs_poll_status(st), Wd


@pytest.mark.parametrize("N,Cn,S,R,seed", [(13, 37, 6, 1, 0), (64, 512, 26, 1, 1), (16, 12, 5, 9, 2), (5, 8, 0, 1, 3),
                                            (300, 260, 40, 1, 4), (7, 64, 9, 49, 5)])
def test_fold_matches_checker(N, Cn, S, R, seed):
    Wc = configs.random_codes(seed, 1, (N, Cn + S, R), -20, 20, np.int8)
    rng = np.random.default_rng(seed)
    extra = rng.integers(0, Cn, S)
    if S >= 3:
        extra[:3] = extra[0]                                   # one channel with four copies
    idx = np.concatenate([np.arange(Cn), extra]).astype(np.int32)
    ref, over = orc.fold_duplicates(Wc.reshape(N, Cn + S, R, 1), idx, Cn)
    assert over == 0
    out, flags, _ = _fold(Wc.reshape(N, -1), Cn, S, R, idx)
    assert flags == 0
    np.testing.assert_array_equal(host(out)[:, :Cn * R], ref.reshape(N, Cn * R))
    assert not host(out)[:, Cn * R:].any()


def test_fold_saturates_and_flags():
    Wc = np.full((2, 5), 100, np.int8)
    Wc[1] = -100
    idx = np.array([0, 1, 2, 1, 1], np.int32)
    ref, over = orc.fold_duplicates(Wc, idx, 3)
    out, flags, _ = _fold(Wc, 3, 2, 1, idx)
    assert over == 2 and flags & ocs.DEV_OVERFLOW
    np.testing.assert_array_equal(host(out)[:, :3], ref)
    _, flags, _ = _fold(Wc, 3, 2, 1, np.array([0, 1, 2, 9, 1], np.int32))
    assert flags & ocs.DEV_BAD_INDEX


def test_folded_layers_equal_gathered_layers():
    """config 1 at 6 bits: split -> quantize -> fold; the plain layer on the folded codes gives the gathered
    layer's accumulators (and the checker's); the same for a 3x3 convolution."""
    c1 = configs.config1()
    S = ocs.ocs_num_splits(512, 0.05)
    Wp, idx_o, _, _ = orc.split(c1["W"], S)
    wc_o, ws_o = orc.quantize(Wp, 6, True, orc.maxabs(Wp))
    ac_o, as_o = orc.quantize(c1["A"], 8, False, orc.maxabs(c1["A"]))
    _, acc_o = orc.qlinear(ac_o, False, as_o, wc_o, ws_o, idx_o)
    codes, scale, _, idx, _, _ = ocs.ocs_split_quantize(dev(c1["W"]), S, 6, ocs.CLIP_NONE)
    st = ocs.new_status()
    folded = ocs.ocs_fold_duplicates(codes, 512, S, idx, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    ref_f, over = orc.fold_duplicates(wc_o, idx_o, 512)
    assert over == 0
    np.testing.assert_array_equal(host(folded)[:, :512], ref_f)
    a_codes, a_scale, _ = ocs.ocs_quantize(dev(c1["A"]), 8, False, ocs.CLIP_NONE, ld_codes=512)
    ident = torch.arange(512, dtype=torch.int32, device="cuda")
    Yf, accf = ocs.ocs_qlinear(a_codes, a_scale, folded, scale, ident, 512, 0, want_acc=True)
    Yg, accg = ocs.ocs_qlinear(a_codes, a_scale, codes, scale, idx, 512, S, want_acc=True)
    np.testing.assert_array_equal(host(accf), acc_o)
    np.testing.assert_array_equal(host(accg), acc_o)
    np.testing.assert_array_equal(host(Yf), host(Yg))

    c2 = configs.config2(batch=2)
    S2 = 6
    codes2, scale2, _, idx2, _, _ = ocs.ocs_split_quantize(dev(c2["W"]), S2, 6, ocs.CLIP_MSE)
    folded2 = ocs.ocs_fold_duplicates(codes2, 256, S2, idx2, R=9, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    x = ocs.ocs_nchw_to_nhwc(dev(c2["X"]))
    xc, xs, _ = ocs.ocs_quantize(x.reshape(1, -1), 8, False, ocs.CLIP_NONE)
    xc = xc[0, :x.numel()].view(x.shape)
    pg = ocs.ocs_pack_conv_weights(codes2, 256, 256, S2, 3, 3)
    pf = ocs.ocs_pack_conv_weights(folded2, 256, 256, 0, 3, 3)
    Yg, accg = ocs.ocs_qconv(xc, xs, pg, scale2, idx2, S2, 3, 3, 1, 1, want_acc=True)
    Yf, accf = ocs.ocs_qconv(xc, xs, pf, scale2, ident[:256].contiguous(), 0, 3, 3, 1, 1, want_acc=True)
    np.testing.assert_array_equal(host(accf), host(accg))
    np.testing.assert_array_equal(host(Yf), host(Yg))
