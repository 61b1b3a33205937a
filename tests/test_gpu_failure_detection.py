"""Failure detection on the device without any fault: a bounded wait that runs out.

Every wait inside the kernels (on an mbarrier or a counter) polls under a time limit; when the limit passes the
waiting thread records DSN_ERR_TIMEOUT in the status word, the CTA leaves its loops and the kernel returns.  The
test shortens the limit to a millisecond, runs the library's self-test kernel (one CTA waiting on a barrier that
nothing arrives at: it always ends by itself), reads the status, and checks that ordinary work still runs on the
same context afterwards."""
import time

import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import DEV, check_status, down, route_on_gpu, up_bf16

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_the_context_stays_usable(dsn):
    ctx = dsn.Context(0)
    ctx.set_wait_limit(1000)                              # 1 ms instead of the 2 s default
    t0 = time.perf_counter()
    ctx.selftest_bounded_wait()
    code, detail = ctx.get_status()                       # waits for the stream
    waited = time.perf_counter() - t0
    assert code == dsn.ERR_TIMEOUT and detail == 9001
    assert waited < 1.0                                   # the short limit was used, not the 2 s default
    assert ctx.get_status() == (0, 0)                     # reading the status cleared it; the limit setting stays
    # an ordinary call on the same context afterwards: sliced linear against the oracle
    g = np.random.default_rng(5)
    B, R, C, T = 12, 40, 128, 3
    k_in, k_out = [64, 96, 128], [128, 64, 96]
    idx = g.integers(0, T, size=B).astype(np.int32)
    x, W = wl.normal(g, (B, R, C)), wl.normal(g, (C, C), std=C ** -0.5)
    r = route_on_gpu(dsn, ctx, idx, T)
    y = torch.zeros((B, R, C), dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, C, C, k_in, k_out, up_bf16(W)), r, up_bf16(x), y)
    check_status(ctx, dsn)
    ref = O.round_bf16(O.sliced_linear(x, W, idx, k_in, k_out, fill=0.0))
    got = down(y)
    for i in range(B):
        ko = k_out[idx[i]]
        assert np.max(np.abs(got[i, :, :ko] - ref[i, :, :ko])) <= 5e-3 * np.max(np.abs(ref[i, :, :ko]))
    # a second time-out is reported again, and the default limit can be restored
    ctx.selftest_bounded_wait()
    assert ctx.get_status()[0] == dsn.ERR_TIMEOUT
    ctx.set_wait_limit(0)
    assert ctx.get_status() == (0, 0)
