"""GPU parity of the KL (Section 4.3) and ACIQ (Section 4.2) clip thresholds against the CPU checker:
histogram counts exact, candidate scores to 1e-9 relative (double sums in another order, another log
routine), chosen threshold within 1e-5 relative (expected equal), codes bit-exact for that threshold."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import clear_winner, dev, host

pytestmark = pytest.mark.gpu


def _check_mode(T, bits, signed, mode, n_cand=128, n_bins=2048, ld=None, noalloc=False):
    T = np.ascontiguousarray(T, dtype=np.float32)
    rows, cols = T.shape
    if ld is None:
        Td = dev(T)
    else:
        Td = torch.full((rows, ld), 7.0e3, dtype=torch.float32, device="cuda")
        Td[:, :cols] = dev(T)
    st = ocs.new_status()
    if noalloc:
        codes, scale, alpha = ocs.ocs_quantize_noalloc(Td, bits, signed, mode, n_cand, n_bins, cols=cols, dev_status=st)
        hist = scores = None
    else:
        codes, scale, alpha, hist, scores = ocs.ocs_quantize(Td, bits, signed, mode, n_cand, n_bins, cols=cols,
                                                             dev_status=st, return_search=True)
    assert ocs.ocs_poll_status(st) == 0
    if mode == ocs.CLIP_KL:
        o = orc.clip_kl(T, bits, signed, n_bins, n_cand)
        if scores is not None:
            fin = np.isfinite(o["scores"])
            np.testing.assert_array_equal(np.isfinite(host(scores)), fin)
            np.testing.assert_allclose(host(scores)[fin], o["scores"][fin], rtol=1e-9, atol=1e-13)
        winner_is_clear = clear_winner(o["scores"], rel=1e-8)
    else:
        o = orc.clip_aciq(T, bits, signed, n_bins)
        winner_is_clear = True
    if hist is not None:
        np.testing.assert_array_equal(host(hist).astype(np.uint64), o["hist"])
    g_alpha = float(host(alpha)[0])
    if winner_is_clear:
        assert abs(g_alpha - o["alpha"]) <= 1e-5 * abs(o["alpha"])
        assert np.float32(g_alpha) == np.float32(o["alpha"])
    o_codes, o_scale = orc.quantize(T, bits, signed, g_alpha)       # codes are a function of the threshold
    assert float(host(scale)[0]) == np.float32(o_scale)
    np.testing.assert_array_equal(host(codes)[:, :cols], o_codes)
    return g_alpha


@pytest.mark.parametrize("mode", [ocs.CLIP_KL, ocs.CLIP_ACIQ])
@pytest.mark.parametrize("bits", [2, 4, 5, 6, 8])
def test_clip_modes_signed_weights(mode, bits):
    c = configs.config1()
    Wp, _, _, _ = orc.split(c["W"], 26)
    _check_mode(Wp, bits, True, mode)


@pytest.mark.parametrize("mode", [ocs.CLIP_KL, ocs.CLIP_ACIQ])
def test_clip_modes_layouts_unsigned_and_degenerate(mode):
    A = configs.config1()["A"]
    _check_mode(A, 8, False, mode)
    _check_mode(A, 6, False, mode, n_cand=33, n_bins=500)
    _check_mode(A[:, :509], 4, False, mode, ld=511)
    T = prng.laplace(5, 0, (300, 4099), 0.01)
    _check_mode(T, 5, True, mode, ld=4100)
    _check_mode(prng.normal(5, 3, (64, 1000), 0.3), 4, True, mode)            # Gauss-shaped data: the other branch of ACIQ
    _check_mode(prng.laplace(5, 1, (1, 1), 1.0), 8, True, mode)
    _check_mode(T, 4, True, mode, n_cand=1024, n_bins=4096)
    _check_mode(T, 3, True, mode, noalloc=True)
    st = ocs.new_status()
    codes, scale, alpha = ocs.ocs_quantize(torch.zeros((5, 64), device="cuda"), 8, True, mode, dev_status=st)
    assert not host(codes).any() and host(scale)[0] == 0 and host(alpha)[0] == 0 and ocs.ocs_poll_status(st) == 0


def test_clip_modes_pick_the_branch_the_data_calls_for():
    lap = prng.laplace(6, 0, (256, 2048), 0.02)
    gau = prng.normal(6, 1, (256, 2048), 0.05)
    assert orc.clip_aciq(lap, 4)["laplace"] and not orc.clip_aciq(gau, 4)["laplace"]
    a_l = _check_mode(lap, 4, True, ocs.CLIP_ACIQ)
    a_g = _check_mode(gau, 4, True, ocs.CLIP_ACIQ)
    assert a_l < orc.maxabs(lap) and a_g < orc.maxabs(gau)                    # both clip


@pytest.mark.parametrize("mode", [ocs.CLIP_KL, ocs.CLIP_ACIQ])
def test_clip_modes_fused_split_quantize(mode):
    """ocs_split_quantize with the two modes: the checker's split -> search -> quantize, and the two separate calls."""
    for W, S, bits in ((configs.config1()["W"], 26, 5), (configs.config2(batch=1)["W"], 6, 6),
                       (configs.config3(O=256, C=6272, M=4)["W"], 63, 4)):
        Wp, o_idx, _, _ = orc.split(W, S, 0.0)
        flat = Wp.reshape(Wp.shape[0], -1)
        o = orc.clip_kl(flat, bits, True, 2048, 128) if mode == ocs.CLIP_KL else orc.clip_aciq(flat, bits, True, 2048)
        st = ocs.new_status()
        codes, scale, alpha, idx, _, mx = ocs.ocs_split_quantize(dev(W), S, bits, mode, dev_status=st)
        assert ocs.ocs_poll_status(st) == 0
        np.testing.assert_array_equal(host(idx), o_idx)
        g_alpha = float(host(alpha)[0])
        if mode == ocs.CLIP_ACIQ or clear_winner(o["scores"], rel=1e-8):
            assert np.float32(g_alpha) == np.float32(o["alpha"])
        o_codes, o_scale = orc.quantize(flat, bits, True, g_alpha)
        assert float(host(scale)[0]) == np.float32(o_scale)
        np.testing.assert_array_equal(host(codes)[:, :flat.shape[1]], o_codes)
        Wout, _, _, mx2 = ocs.ocs_split(dev(W), S)
        codes2, scale2, alpha2 = ocs.ocs_quantize(Wout, bits, True, mode, cols=flat.shape[1], max_abs_in=mx2[1:2])
        assert host(alpha2)[0] == host(alpha)[0] and host(scale2)[0] == host(scale)[0]
        np.testing.assert_array_equal(host(codes2)[:, :flat.shape[1]], host(codes)[:, :flat.shape[1]])
