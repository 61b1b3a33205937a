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


@pytest.fixture(scope="module")
def ctx_fused(dsn):
    """A context that runs the separable block as one kernel (the switch is read when the context is created)."""
    import os
    old = os.environ.get("DSN_DWPW")
    os.environ["DSN_DWPW"] = "fused"
    try:
        c = dsn.Context(0)
    finally:
        if old is None:
            del os.environ["DSN_DWPW"]
        else:
            os.environ["DSN_DWPW"] = old
    return c


@pytest.mark.parametrize("fused", [True, False], ids=["one-kernel", "two-launches"])
@pytest.mark.parametrize("hw,C,K,stride,B,gate,mult8", [(14, 640, 3, 1, 40, False, True), (14, 256, 7, 2, 23, True, True),
                                                        (7, 1152, 5, 1, 30, False, True), (28, 64, 3, 2, 9, False, True),
                                                        (9, 88, 3, 1, 12, False, False)])
def test_separable_block_through_layer_forward(dsn, ctx, ctx_fused, fused, hw, C, K, stride, B, gate, mult8, parity_report):
    """The DS-MBNet separable block as one dsn_layer_forward call: [gate ->] route -> depthwise k x k (c_t channels,
    bias, ReLU) -> pointwise 1x1 c_t -> c_t' (ReLU) -> input order.  With widths that are multiples of 8 the two
    layers can run as ONE kernel (the depthwise result never reaches global memory; context created under
    DSN_DWPW=fused); by default, and for other widths, they run one after the other.
    Either way the result must be the oracle's chain, which rounds the depthwise output to bf16 where a device
    that stored it would."""
    if fused:
        ctx = ctx_fused
    g = np.random.default_rng(hw * 1000 + C + K + B)
    widths = sorted({max(8, int(C * r) // 8 * 8) for r in (0.35, 0.5, 0.65, 0.8, 0.9, 1.0)}) if mult8 else [20, 44, 52, 76, 84, 88]
    T = len(widths)
    k_out = [min(C, w + 8 * (t % 3)) for t, w in enumerate(widths)] if mult8 else widths
    ksizes = [[3, 5, 7][t % 3] if K == 7 else (K if t % 2 else min(K, 3)) for t in range(T)]
    x = wl.normal(g, (B, hw, hw, C), relu=True)
    Wdw = wl.normal(g, (C, K, K), std=1.0 / K)
    Wpw = wl.normal(g, (C, C, 1, 1), std=C ** -0.5)
    bias = (0.1 * g.standard_normal(C)).astype(np.float32)
    gW1 = wl.normal(g, (32, C), std=C ** -0.5, bf16=False)
    gW2 = wl.normal(g, (T, 32), std=32 ** -0.5, bf16=False)
    Ho = (hw - 1) // stride + 1
    dw = dsn.make_depthwise_desc(hw, hw, K, stride, C, widths, ksizes, up_bf16(np.ascontiguousarray(np.transpose(Wdw, (1, 2, 0)))),
                                 bias=up_f32(bias), act=dsn.ACT_RELU)
    pw = dsn.make_conv_desc(dsn.BF16, Ho, Ho, 1, 0, C, C, widths, k_out, up_bf16(Wpw.reshape(C, C)), act=dsn.ACT_RELU)
    gd = None
    if gate:
        gw1, gw2 = up_f32(gW1), up_f32(gW2)
        gd = dsn.make_gate_desc(dsn.BF16, B, hw * hw, C, 32, T, gw1, gw2)
    L = dsn.make_layer_desc(B, T, [dw, pw], gd)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, Ho, Ho, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    idx_out = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    idx_given = g.integers(0, T, size=B).astype(np.int32)
    dsn.dsn_layer_forward(ctx, L, up_bf16(x), None if gate else torch.from_numpy(idx_given).to(DEV), y, ws, idx_out=idx_out)
    check_status(ctx, dsn)
    idx = idx_out.cpu().numpy()
    if gate:
        idx_ref, _, margin = O.gate(x.reshape(B, hw * hw, C), gW1, gW2)
        safe = margin >= 1e-4
        np.testing.assert_array_equal(idx[safe], idx_ref[safe])
    else:
        np.testing.assert_array_equal(idx, idx_given)
    d_ref = O.round_bf16(O.sliced_depthwise(x, Wdw, idx, widths, ksizes, stride=stride, bias=bias, act=O.ACT_RELU, fill=0.0))
    ref = O.sliced_conv(d_ref, Wpw, idx, widths, k_out, 0, act=O.ACT_RELU)       # unrounded: half an ulp + a rare flip upstream
    got = down(y)
    errs = group_errors(got, ref, idx, k_out, T)
    assert max(errs.values()) <= 1e-2, errs
    parity_report.append(f"separable block {hw}x{hw} C={C} k<={K} stride {stride} ({'one kernel' if (mult8 and fused) else 'two launches'}): "
                         f"worst {max(errs.values()):.2e} (bound 1e-02 for two stored bf16 layers)")
    for i in range(B):
        assert np.all(got[i][..., k_out[idx[i]]:] == SENTINEL)
