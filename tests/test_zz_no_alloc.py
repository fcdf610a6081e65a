"""ocs_quantize_noalloc -- the entry point for callers that cannot allocate device memory where they
quantize (it keeps its scratch in an array built into the library) -- must give exactly what
ocs_quantize gives.  Two calls in a row share that array, so the second one also shows that stale
contents of the first do not leak into it.  Collected last on purpose: a failure here leaves every
other test already run."""
import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import prng

pytestmark = pytest.mark.gpu


def _both(T, bits, signed, mode, **kw):
    st = ocs.new_status()
    ref = ocs.ocs_quantize(T, bits, signed, mode, dev_status=st, **kw)[:3]
    got = ocs.ocs_quantize_noalloc(T, bits, signed, mode, dev_status=st, **kw)
    assert ocs.ocs_poll_status(st) == 0
    cols = kw.get("cols") or T.shape[1]
    for r, g, name in zip(ref, got, ("codes", "scale", "alpha")):
        r, g = r.cpu().numpy(), g.cpu().numpy()
        if name == "codes":
            r, g = r[:, :cols], g[:, :cols]
            np.testing.assert_array_equal(g, r, err_msg=name)                    # integer codes: bit-exact
        else:
            np.testing.assert_allclose(g, r, rtol=1e-5, atol=0, err_msg=name)     # the float bar of the other tests
            np.testing.assert_array_equal(g, r, err_msg=name)                    # same kernels: equal in fact


def test_noalloc_matches_workspace_entry_point_on_two_calls_in_a_row():
    big = torch.from_numpy(prng.laplace(31, 0, (300, 4099), 0.01)).cuda()        # several tiles and a ragged tail
    small = torch.from_numpy(prng.normal(31, 1, (64, 512), absolute=True)).cuda()
    # first call: MSE search leaves a full histogram and 128 scores in the built-in scratch
    _both(big, 5, True, ocs.CLIP_MSE)
    # second call right after it, other tensor, other grid: must not see the first call's leftovers
    _both(small, 8, False, ocs.CLIP_MSE, n_candidates=33, n_bins=500)
    _both(small, 6, False, ocs.CLIP_NONE)
    _both(big, 4, True, ocs.CLIP_MSE, cols=4000)


def test_noalloc_rejects_what_does_not_fit_its_scratch():
    T = torch.ones((4, 64), device="cuda")
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_quantize_noalloc(T, 8, True, ocs.CLIP_MSE_EXACT)
    assert e.value.status == 4                                                   # OCS_ERR_UNSUPPORTED
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_quantize_noalloc(T, 8, True, ocs.CLIP_MSE, n_bins=8192)
    assert e.value.status == 4
    with pytest.raises(ocs.OcsError) as e:
        ocs.ocs_quantize_noalloc(T, 8, True, ocs.CLIP_MSE, n_candidates=2048)
    assert e.value.status == 4
