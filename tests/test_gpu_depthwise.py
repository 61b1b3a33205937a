"""GPU parity of the slice-able depthwise convolution (MobileNet DSConv shapes) against the CPU oracle."""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import DEV, SENTINEL, check_status, down, group_errors, route_on_gpu, up_bf16, up_f32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(dsn):
    return dsn.Context(0)


@pytest.mark.parametrize("hw,C,K,stride,orders", [(14, 640, 3, 1, (0, 0)), (14, 640, 7, 2, (1, 1)), (7, 1152, 7, 1, (0, 1)),
                                                  (28, 96, 5, 2, (1, 0)), (9, 44, 3, 1, (0, 0))])
def test_depthwise_mobilenet_shapes(dsn, ctx, hw, C, K, stride, orders):
    g = np.random.default_rng(hw * 100 + C + K)
    T = 6
    widths = sorted({max(4, int(C * r) // 4 * 4) for r in (0.35, 0.5, 0.65, 0.8, 0.9, 1.0)})
    if C == 44:
        widths = [10, 22, 26, 38, 42, 44]          # widths that are no multiple of 8
    T = len(widths)
    ksizes = [[3, 5, 7][t % 3] if K == 7 else (K if t % 2 else min(K, 3)) for t in range(T)]
    B = 10
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = wl.normal(g, (B, hw, hw, C), relu=True)
    W = wl.normal(g, (C, K, K), std=1.0 / K)
    bias = (0.1 * g.standard_normal(C)).astype(np.float32)
    r = route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2]
    Ho = (hw - 1) // stride + 1
    y = torch.full((B, Ho, Ho, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    d = dsn.make_depthwise_desc(hw, hw, K, stride, C, widths, ksizes, up_bf16(np.ascontiguousarray(np.transpose(W, (1, 2, 0)))),
                                bias=up_f32(bias), act=dsn.ACT_RELU, in_order=orders[0], out_order=orders[1])
    dsn.dsn_sliced_depthwise(ctx, d, r, up_bf16(x[perm] if orders[0] else x), y)
    check_status(ctx, dsn)
    got = down(y)
    if orders[1]:
        tmp = np.empty_like(got)
        tmp[perm] = got
        got = tmp
    ref = O.round_bf16(O.sliced_depthwise(x, W, idx, widths, ksizes, stride=stride, bias=bias, act=O.ACT_RELU))
    errs = group_errors(got, ref, idx, widths, T)
    assert max(errs.values()) <= 5e-3, errs
    for i in range(B):
        assert np.all(got[i][..., widths[idx[i]]:] == SENTINEL)
