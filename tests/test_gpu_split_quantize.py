"""GPU parity: ocs_split and ocs_quantize against the CPU checker, through the C ABI.
Bars: idx_map, split_order, W' bits and int8 codes bit-exact; scale / alpha <= 1e-5 relative
(they come out bit-exact in practice and that is asserted where the arithmetic is single-op)."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import L_of, check_split, clear_winner, dev, gpu_split, host, oracle_split

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------------------ split
def test_split_config1_naive_and_qa():
    c = configs.config1()
    S = ocs.ocs_num_splits(512, c["ratio"])
    assert S == orc.num_splits(512, c["ratio"]) == 26
    check_split(c["W"], S, literal=True)
    check_split(c["W"], S, qa_bits=8, literal=True)
    check_split(c["W"], S, qa_step=0.01)
    check_split(c["W"], S, ld_out=539)          # unaligned output rows: scalar path


def test_split_config2_conv():
    c = configs.config2(batch=1)
    S = ocs.ocs_num_splits(256, c["ratio"])
    check_split(c["W"], S, literal=True)
    check_split(c["W"], S, qa_bits=6)


@pytest.mark.parametrize("shape,S", [((33, 20), 7), ((16, 12, 3, 3), 5), ((9, 1), 4), ((5, 6), 0), ((4, 3), 9),
                                     ((7, 1031), 40), ((300, 77, 1, 7), 11), ((1, 5), 3), ((130, 2051), 300)])
def test_split_odd_shapes(shape, S):
    W = prng.laplace(17, 0, shape, 0.02)
    W.reshape(-1)[prng.distinct_positions(17, 1, W.size, min(5, W.size))] *= 25
    check_split(W, S, literal=W.size < 50000)
    check_split(W, S, qa_bits=5)


def test_split_ties_and_degenerate():
    # equal magnitudes everywhere: every choice is a tie-break
    W = np.array([[4, -4, 1, 0.5], [1, 2, -4, 0.25]], dtype=np.float32)
    check_split(W, 6, literal=True)
    Wt = np.full((8, 40), 0.5, dtype=np.float32)
    Wt[:, ::3] *= -1
    check_split(Wt, 55, literal=True)
    check_split(np.zeros((3, 4), np.float32), 5, literal=True)           # all zero: channel 0 every time
    check_split(np.array([[2.0], [-6.0]], np.float32), 3, literal=True)  # C = 1, S > C
    c3 = configs.config3(O=64, C=3136, M=4)                                 # many identical outliers
    check_split(c3["W"], ocs.ocs_num_splits(3136, 0.1))


def test_split_fc6_slice_matches_cached_oracle():
    c3 = configs.config3(O=256, C=25088, M=4)
    for r in (0.01, 0.1):
        check_split(c3["W"], ocs.ocs_num_splits(25088, r))
    check_split(c3["W"], ocs.ocs_num_splits(25088, 0.05), qa_bits=4)


def test_split_flags_nonfinite_and_rejects_bad_args():
    W = prng.laplace(3, 0, (16, 32), 0.1)
    W[3, 4] = np.inf
    *_, flags, _ = gpu_split(W, 2)
    assert flags & ocs.DEV_NONFINITE
    Wd = dev(prng.laplace(3, 0, (16, 32), 0.1))
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_split(Wd, -1)
    assert e.value.status == 1
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_split(Wd, 2, ld_out=10)
    assert e.value.status == 2
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_split(Wd, 2, qa_bits=9)
    assert e.value.status == 1


def test_split_is_deterministic():
    c = configs.config1()
    a = gpu_split(c["W"], 26, qa_bits=8)
    b = gpu_split(c["W"], 26, qa_bits=8)
    for x, y in zip(a[:4], b[:4]):
        np.testing.assert_array_equal(x, y)


# ------------------------------------------------------------------------------ quantize
def _check_quant(T, bits, signed, mode, n_cand=128, n_bins=2048, ld=None, ld_codes=None, known_max=False):
    T = np.ascontiguousarray(T, dtype=np.float32)
    rows, cols = T.shape
    if ld is None:
        Td = dev(T)
    else:
        buf = torch.full((rows, ld), 7.0e3, dtype=torch.float32, device="cuda")   # padding must be ignored
        buf[:, :cols] = dev(T)
        Td = buf
    st = ocs.new_status()
    mx = dev(np.array([orc.maxabs(T)], np.float32)) if known_max else None
    res = ocs.ocs_quantize(Td, bits, signed, mode, n_cand, n_bins, cols=cols, ld_codes=ld_codes, max_abs_in=mx,
                           dev_status=st, return_search=(mode == ocs.CLIP_MSE))
    codes, scale, alpha = res[:3]
    assert ocs.ocs_poll_status(st) == 0
    g_alpha = float(host(alpha)[0])
    if mode == ocs.CLIP_MSE:
        o = orc.clip_mse(T, bits, signed, n_bins, n_cand)
        np.testing.assert_array_equal(host(res[3]).astype(np.uint64), o["hist"])       # integer counts: exact
        np.testing.assert_allclose(host(res[4]), o["scores"], rtol=1e-9, atol=1e-300)  # double sums, other order
        o_alpha = o["alpha"]
        # the two sides add the bin terms in different orders: the winner is a function of the scores both must
        # agree on only when it wins by more than that rounding (exact ties -- all-zero scores -- included)
        if not (clear_winner(o["scores"]) or np.array_equal(host(res[4]), o["scores"])):
            o_alpha = g_alpha
    else:
        o_alpha = orc.maxabs(T)
    assert abs(g_alpha - o_alpha) <= 1e-5 * abs(o_alpha)
    assert np.float32(g_alpha) == np.float32(o_alpha)
    o_codes, o_scale = orc.quantize(T, bits, signed, o_alpha)
    assert float(host(scale)[0]) == np.float32(o_scale)
    np.testing.assert_array_equal(host(codes)[:, :cols], o_codes)
    return codes, scale


@pytest.mark.parametrize("bits", [2, 4, 5, 6, 8])
@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_signed_weights(bits, mode):
    c = configs.config1()
    Wp, _, _, _ = orc.split(c["W"], 26)
    _check_quant(Wp, bits, True, mode)


def test_quantize_layouts_and_unsigned():
    A = configs.config1()["A"]
    _check_quant(A, 8, False, 0)
    _check_quant(A, 8, False, 1, n_cand=33, n_bins=500)
    _check_quant(A[:, :509], 8, False, 0, ld=512, ld_codes=512)
    _check_quant(A[:, :509], 6, False, 1, ld=511, ld_codes=509)        # nothing aligned
    _check_quant(A[:7, :5], 3, False, 1)
    T = prng.laplace(5, 0, (300, 4099), 0.01)
    _check_quant(T, 5, True, 1, ld=4100, ld_codes=4112)
    _check_quant(T, 5, True, 1, known_max=True)
    _check_quant(prng.laplace(5, 1, (1, 1), 1.0), 8, True, 1)


def test_quantize_degenerate_and_flags():
    st = ocs.new_status()
    codes, scale, alpha = ocs.ocs_quantize(torch.zeros((5, 64), device="cuda"), 8, True, ocs.CLIP_MSE, dev_status=st)
    assert not host(codes).any() and host(scale)[0] == 0 and host(alpha)[0] == 0 and ocs.ocs_poll_status(st) == 0
    T = torch.ones((5, 64), device="cuda")
    T[2, 3] = float("nan")
    ocs.ocs_quantize(T, 8, True, ocs.CLIP_NONE, dev_status=st)
    assert ocs.ocs_poll_status(st) & ocs.DEV_NONFINITE
    with pytest.raises(ocs.OcsError):
        ocs.ocs_quantize(T, 9, True)
    with pytest.raises(ocs.OcsError):
        ocs.ocs_quantize(T, 8, True, ocs.CLIP_MSE, n_candidates=0)


def test_quantize_config2_mse_and_config3_slice():
    c2 = configs.config2(batch=1)
    Wp, _, _, _ = orc.split(c2["W"], 6)
    _check_quant(Wp.reshape(256, -1), 6, True, 1)
    c3 = configs.config3(O=512, C=6272, M=4)
    Wp, _, _, _ = orc.split(c3["W"], orc.num_splits(6272, 0.05))
    for bits in (4, 5, 6, 8):
        _check_quant(Wp, bits, True, 1)


def _check_quant_exact(T, bits, signed, n_cand=128, ld=None):
    T = np.ascontiguousarray(T, dtype=np.float32)
    rows, cols = T.shape
    if ld is None:
        Td = dev(T)
    else:
        Td = torch.full((rows, ld), -3.0e3, dtype=torch.float32, device="cuda")
        Td[:, :cols] = dev(T)
    st = ocs.new_status()
    codes, scale, alpha, _, scores = ocs.ocs_quantize(Td, bits, signed, ocs.CLIP_MSE_EXACT, n_cand, cols=cols,
                                                      dev_status=st, return_search=True)
    assert ocs.ocs_poll_status(st) == 0
    o = orc.clip_mse_exact(T, bits, signed, n_cand)
    np.testing.assert_allclose(host(scores), o["scores"], rtol=1e-9, atol=1e-300)   # double sums, other order
    assert np.float32(host(alpha)[0]) == np.float32(o["alpha"])
    o_codes, o_scale = orc.quantize(T, bits, signed, o["alpha"])
    assert float(host(scale)[0]) == np.float32(o_scale)
    np.testing.assert_array_equal(host(codes)[:, :cols], o_codes)
    return o["alpha"]


def test_quantize_exact_mse_scorer():
    """The element-wise scorer (no histogram) against the checker's, and next to the histogram search."""
    c = configs.config1()
    Wp, _, _, _ = orc.split(c["W"], 26)
    for bits in (3, 4, 6, 8):
        a_exact = _check_quant_exact(Wp, bits, True)
        a_hist = orc.clip_mse(Wp, bits, True, 2048, 128)["alpha"]
        assert abs(a_exact - a_hist) <= 1.5 * orc.maxabs(Wp) / 128          # within one candidate of each other
    _check_quant_exact(c["A"], 8, False, n_cand=33)
    _check_quant_exact(c["A"][:, :509], 5, False, n_cand=300, ld=512)
    _check_quant_exact(prng.laplace(5, 0, (37, 4099), 0.01), 4, True, n_cand=1024, ld=4100)
    _check_quant_exact(prng.laplace(5, 1, (1, 1), 1.0), 8, True, n_cand=1)
    c2 = configs.config2(batch=1)
    Wp2, _, _, _ = orc.split(c2["W"], 6)
    _check_quant_exact(Wp2.reshape(256, -1), 6, True)


# ------------------------------------------------------------------------------ fused split + quantize
def _check_fused(W, S, bits, mode, qa_bits=0, n_cand=128, n_bins=2048):
    """ocs_split_quantize against the checker's split -> search -> quantize, and against the two separate calls."""
    o_out, o_idx, o_order, o_mx, step = oracle_split(W, S, qa_bits)
    flat = o_out.reshape(o_out.shape[0], -1)
    o_alpha = orc.clip_mse(flat, bits, True, n_bins, n_cand)["alpha"] if mode == ocs.CLIP_MSE else orc.maxabs(flat)
    o_codes, o_scale = orc.quantize(flat, bits, True, o_alpha)
    st = ocs.new_status()
    codes, scale, alpha, idx, order, mx = ocs.ocs_split_quantize(dev(W), S, bits, mode, qa_bits=qa_bits,
                                                                 n_candidates=n_cand, n_bins=n_bins, dev_status=st)
    assert ocs.ocs_poll_status(st) == 0
    np.testing.assert_array_equal(host(idx), o_idx)
    np.testing.assert_array_equal(host(order), o_order)
    assert host(mx)[1] == np.float32(o_mx[1]) and host(mx)[2] == np.float32(step)
    assert abs(float(host(alpha)[0]) - o_alpha) <= 1e-5 * abs(o_alpha)
    assert np.float32(host(alpha)[0]) == np.float32(o_alpha)
    assert float(host(scale)[0]) == np.float32(o_scale)
    np.testing.assert_array_equal(host(codes)[:, :flat.shape[1]], o_codes)
    # the separate calls give the same bytes
    Wout, idx2, _, mx2 = ocs.ocs_split(dev(W), S, qa_bits=qa_bits)
    codes2, scale2, alpha2 = ocs.ocs_quantize(Wout, bits, True, mode, n_cand, n_bins, cols=flat.shape[1],
                                              max_abs_in=mx2[1:2])
    np.testing.assert_array_equal(host(codes)[:, :flat.shape[1]], host(codes2)[:, :flat.shape[1]])
    assert host(scale)[0] == host(scale2)[0] and host(alpha)[0] == host(alpha2)[0]


def test_fused_split_quantize_matches_checker_and_separate_calls():
    c1 = configs.config1()
    for bits, mode in ((8, ocs.CLIP_NONE), (5, ocs.CLIP_MSE), (4, ocs.CLIP_MSE)):
        _check_fused(c1["W"], 26, bits, mode)
    _check_fused(c1["W"], 26, 6, ocs.CLIP_MSE, qa_bits=6)
    c2 = configs.config2(batch=1)
    _check_fused(c2["W"], 6, 6, ocs.CLIP_MSE)                                  # conv weights, R = 9
    _check_fused(prng.laplace(17, 0, (33, 20), 0.02), 7, 5, ocs.CLIP_MSE, n_cand=33, n_bins=500)   # (C+S) odd: ragged rows
    _check_fused(prng.laplace(17, 1, (5, 8), 0.02), 0, 8, ocs.CLIP_NONE)      # no splits
    _check_fused(np.zeros((3, 4), np.float32), 5, 8, ocs.CLIP_MSE)            # all zero
    c3 = configs.config3(O=256, C=25088, M=4)                                 # fc6-length rows: one row per buffer
    _check_fused(c3["W"], ocs.ocs_num_splits(25088, 0.1), 4, ocs.CLIP_MSE)
    _check_fused(c3["W"], ocs.ocs_num_splits(25088, 0.01), 8, ocs.CLIP_NONE)


def test_fused_split_quantize_rejects_what_it_cannot_stage():
    Wd = dev(prng.laplace(3, 0, (16, 30), 0.1))                                # C*R not a multiple of 4
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_split_quantize(Wd, 2, 8)
    assert e.value.status == 4
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_split_quantize(dev(prng.laplace(3, 0, (16, 32), 0.1)), 2, 9)
    assert e.value.status == 1
