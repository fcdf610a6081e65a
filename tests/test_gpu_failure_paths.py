"""Failure detection without a fault: a bounded device wait is made to run out (a copy that is never
requested), the kernel reports OCS_DEV_TIMEOUT through the status word and returns, and the same stream
goes on to pass parity.  Also the tracer's bookkeeping when its capacity is smaller than the launches."""
import time

import numpy as np
import pytest
import torch

import paper_1901_09504_b200 as ocs
from ocs_inputs import configs, prng
from oracle import oracle as orc

from gpu_util import check_split, dev, host

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_and_the_context_stays_usable():
    W = prng.laplace(23, 0, (600, 1024), 0.02)
    st = ocs.new_status()
    t0 = time.perf_counter()
    out = ocs.ocs_selftest_wait_expiry(dev(W), st)
    flags = ocs.ocs_poll_status(st)                      # synchronises: the kernel returned on its own
    assert time.perf_counter() - t0 < 5.0
    assert flags & ocs.DEV_TIMEOUT
    got = host(out)
    # rows whose copies were requested arrived intact; the dropped groups were left as they were (zeros)
    same = (got == W).all(axis=1)
    untouched = (got == 0).all(axis=1)
    assert (same | untouched).all() and same.any() and untouched.any()
    # the stream and the context go on working: an ordinary split afterwards is bit-exact
    c = configs.config1()
    check_split(c["W"], 26)
    st2 = ocs.new_status()
    ocs.ocs_split(dev(c["W"]), 26, dev_status=st2)
    assert ocs.ocs_poll_status(st2) == 0


def test_trace_with_less_capacity_than_launches():
    """A trace that fills up records nothing further and does not stretch its last record."""
    W = dev(configs.config1()["W"])
    ocs.ocs_split(W, 26)                                  # warm-up (attributes, module load)
    torch.cuda.synchronize()
    ocs.ocs_trace_start(1)
    n0 = ocs.ocs_kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        ocs.ocs_split(W, 26)
    e1.record()
    torch.cuda.synchronize()
    rows = ocs.ocs_trace_stop()
    assert ocs.ocs_kernel_launches() - n0 == 60           # extrema, plan, scatter per call
    assert list(rows) == ["col_minmax_kernel"] and rows["col_minmax_kernel"][0] == 1
    assert rows["col_minmax_kernel"][1] < 0.5 * e0.elapsed_time(e1)   # one launch, not the whole run
    ocs.ocs_trace_start(1000)
    ocs.ocs_split(W, 26)
    rows = ocs.ocs_trace_stop()
    assert {k: v[0] for k, v in rows.items()} == {"col_minmax_kernel": 1, "split_plan_kernel": 1, "split_rows_kernel": 1}
