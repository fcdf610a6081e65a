"""Helpers shared by the GPU parity tests: run one step on the CUDA library and on the CPU
checker with the same numpy inputs."""
import numpy as np
import torch

import paper_1901_09504_b200 as ocs
from oracle import oracle as orc


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


def L_of(bits, signed=True):
    return 2 ** (bits - 1) - 1 if signed else 2 ** bits - 1


def oracle_split(W, S, qa_bits=0, qa_step=0.0, literal=False):
    """The checker's split; with qa_bits the grid step comes from the checker's two-pass rule (split_qa)."""
    if qa_bits:
        out, idx, order, mx, qa_step = orc.split_qa(W, S, qa_bits)
        if not literal:
            return out, idx, order, mx, qa_step
    out, idx, order, mx = orc.split(W, S, qa_step, literal=literal)
    return out, idx, order, mx, qa_step


def gpu_split(W, S, qa_bits=0, qa_step=0.0, ld_out=None):
    st = ocs.new_status()
    Wd = dev(W)
    out, idx, order, mx = ocs.ocs_split(Wd, S, qa_step=qa_step, qa_bits=qa_bits, ld_out=ld_out, dev_status=st)
    O, Cn = W.shape[0], W.shape[1]
    R = int(np.prod(W.shape[2:])) if W.ndim > 2 else 1
    cols = (Cn + S) * R
    flags = ocs.ocs_poll_status(st)
    return host(out)[:, :cols].reshape((O, Cn + S) + tuple(W.shape[2:])), host(idx), host(order), host(mx), flags, out


def check_split(W, S, qa_bits=0, qa_step=0.0, ld_out=None, literal=False):
    o_out, o_idx, o_order, o_mx, step = oracle_split(W, S, qa_bits, qa_step, literal)
    g_out, g_idx, g_order, g_mx, flags, raw = gpu_split(W, S, qa_bits, qa_step, ld_out)
    assert flags == 0
    np.testing.assert_array_equal(g_idx, o_idx)
    np.testing.assert_array_equal(g_order, o_order)
    np.testing.assert_array_equal(g_out.view(np.uint32), o_out.view(np.uint32))   # bit-exact W'
    assert g_mx[0] == np.float32(o_mx[0]) and g_mx[1] == np.float32(o_mx[1])
    assert g_mx[2] == np.float32(step)
    return o_out, o_idx, raw


def clear_winner(scores, rel=1e-9):
    """True when the smallest candidate score beats the runner-up by more than the rounding the two sides'
    different summation orders can cause.  Only then is the chosen threshold a function of the scores that
    both sides must agree on; a near-tie may legitimately flip and is compared through its scores alone."""
    s = np.sort(np.asarray(scores, dtype=np.float64)[np.isfinite(scores)])
    if s.size < 2:
        return True
    return (s[1] - s[0]) > rel * max(abs(s[1]), 1e-300)
