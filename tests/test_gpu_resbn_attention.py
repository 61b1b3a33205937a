"""GPU parity of the widened rows: Re-SBN in the layer epilogue and the attention head of the gate."""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import (DEV, SENTINEL, assert_tail_untouched, check_status, down, group_errors, route_on_gpu, up_bf16,
                      up_f32)

pytestmark = pytest.mark.gpu
TOL_BF16 = 5e-3


@pytest.fixture(scope="module")
def ctx(dsn):
    return dsn.Context(0)


def fold_on_gpu(dsn, ctx, gamma, beta, mu, sigma):
    T, C = mu.shape
    sc = torch.zeros(T, C, dtype=torch.float32, device=DEV)
    sh = torch.zeros(T, C, dtype=torch.float32, device=DEV)
    dsn.dsn_resbn_fold(ctx, T, C, up_f32(gamma), up_f32(beta), up_f32(mu), up_f32(sigma), sc, sh)
    return sc, sh


def test_resbn_fold_values(dsn, ctx):
    g = np.random.default_rng(0)
    T, C = 5, 37
    gamma, beta = g.standard_normal(C).astype(np.float32), g.standard_normal(C).astype(np.float32)
    mu = g.standard_normal((T, C)).astype(np.float32)
    sigma = (np.abs(g.standard_normal((T, C))) + 0.5).astype(np.float32)
    sc, sh = fold_on_gpu(dsn, ctx, gamma, beta, mu, sigma)
    check_status(ctx, dsn)
    a = gamma.astype(np.float64) / sigma
    np.testing.assert_allclose(sc.cpu().numpy(), a, rtol=1e-6)
    np.testing.assert_allclose(sh.cpu().numpy(), beta - a * mu, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("K,orders", [(3, (0, 0)), (1, (1, 1)), (3, (1, 0))])
def test_conv_with_resbn_and_relu(dsn, ctx, K, orders):
    g = np.random.default_rng(5 + K)
    B, hw, C = 18, 14, 256
    widths = wl.WIDTHS_14[C]
    T = len(widths)
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = wl.normal(g, (B, hw, hw, C), relu=True)
    W = wl.normal(g, (C, C, K, K), std=(K * K * C) ** -0.5)
    gamma = (1.0 + 0.2 * g.standard_normal(C)).astype(np.float32)
    beta = (0.3 * g.standard_normal(C)).astype(np.float32)
    mu = (0.2 * g.standard_normal((T, C))).astype(np.float32)
    sigma = (0.6 + np.abs(g.standard_normal((T, C))) * 0.5).astype(np.float32)
    sc, sh = fold_on_gpu(dsn, ctx, gamma, beta, mu, sigma)
    r = route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2]
    xs = x[perm] if orders[0] else x
    y = torch.full((B, hw, hw, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    d = dsn.make_conv_desc(dsn.BF16, hw, hw, K, K // 2, C, C, widths, widths,
                           up_bf16(np.ascontiguousarray(np.transpose(W, (0, 2, 3, 1)))), act=dsn.ACT_RELU,
                           in_order=orders[0], out_order=orders[1], bn_scale=sc, bn_shift=sh)
    dsn.dsn_sliced_conv(ctx, d, r, up_bf16(xs), y)
    check_status(ctx, dsn)
    got = down(y)
    if orders[1]:
        tmp = np.empty_like(got)
        tmp[perm] = got
        got = tmp
    ref = O.round_bf16(O.sliced_conv(x, W, idx, widths, widths, K // 2, act=O.ACT_RELU, bn=(gamma, beta, mu, sigma)))
    errs = group_errors(got, ref, idx, widths, T)
    assert max(errs.values()) <= TOL_BF16, errs
    assert_tail_untouched(got, idx, widths)
    # the statistics of the sample's own route are the ones applied: another route's would be far off
    wrong = O.sliced_conv(x[:1], W, [(idx[0] + 1) % T], widths, widths, K // 2, act=O.ACT_RELU, bn=(gamma, beta, mu, sigma))
    k = min(widths[idx[0]], widths[(idx[0] + 1) % T])
    assert np.max(np.abs(wrong[0, ..., :k] - ref[0, ..., :k])) > 0.05


def test_fp32_linear_with_resbn(dsn, ctx):
    cfg = wl.config1()
    g = np.random.default_rng(9)
    C, T = 256, 4
    gamma, beta = g.standard_normal(C).astype(np.float32), g.standard_normal(C).astype(np.float32)
    mu = g.standard_normal((T, C)).astype(np.float32)
    sigma = (np.abs(g.standard_normal((T, C))) + 0.5).astype(np.float32)
    sc, sh = fold_on_gpu(dsn, ctx, gamma, beta, mu, sigma)
    r = route_on_gpu(dsn, ctx, cfg["idx"], T)
    y = torch.full((64, 1, C), SENTINEL, dtype=torch.float32, device=DEV)
    d = dsn.make_linear_desc(dsn.F32, 1, C, C, cfg["k_in"], cfg["k_out"], up_f32(cfg["W"]), bn_scale=sc, bn_shift=sh,
                             act=dsn.ACT_RELU)
    dsn.dsn_sliced_linear(ctx, d, r, up_f32(cfg["x"]), y)
    check_status(ctx, dsn)
    ref = O.sliced_linear(cfg["x"], cfg["W"], cfg["idx"], cfg["k_in"], cfg["k_out"], act=O.ACT_RELU,
                          bn=(gamma, beta, mu, sigma))
    errs = group_errors(down(y), ref, cfg["idx"], cfg["k_out"], T)
    assert max(errs.values()) <= 2e-5, errs


@pytest.mark.parametrize("B,R,C,M,T,cv", [(128, 196, 1024, 128, 14, None), (40, 197, 384, 128, 48, None),
                                          (7, 9, 40, 10, 3, 24), (5, 50, 64, 32, 4, None)])
def test_gate_attention_head_and_scaling(dsn, ctx, B, R, C, M, T, cv):
    g = np.random.default_rng(B + C)
    x = wl.normal(g, (B, R, C))
    W1 = (g.standard_normal((M, C)) / np.sqrt(C)).astype(np.float32)
    W2 = (g.standard_normal((T, M)) / np.sqrt(M)).astype(np.float32)
    W3 = (g.standard_normal((C, M)) / np.sqrt(M)).astype(np.float32)
    b3 = (0.1 * g.standard_normal(C)).astype(np.float32)
    c_valid = C if cv is None else cv
    dx = up_bf16(x)
    desc = dsn.make_gate_desc(dsn.BF16, B, R, C, M, T, up_f32(W1), up_f32(W2), c_valid=c_valid)
    ws = torch.empty(dsn.dsn_gate_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
    idx = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    idx_plain = torch.full((B,), -2, dtype=torch.int32, device=DEV)
    scale = torch.zeros(B, c_valid, dtype=torch.float32, device=DEV)
    dsn.dsn_gate_attention(ctx, desc, up_f32(W3), up_f32(b3), dx, idx, scale, workspace=ws)
    dsn.dsn_gate(ctx, desc, dx, idx_plain, None, ws)
    check_status(ctx, dsn)
    assert torch.equal(idx, idx_plain)                               # the routing head is unchanged
    s_ref, xh_ref = O.gate_attention(x, W1, W3, b3=b3, c_valid=c_valid)
    s_gpu = scale.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(s_gpu - s_ref)) <= 2e-5
    # apply it: in place in input order, and fused with the gather into grouped order
    idx_np = idx.cpu().numpy()
    r = route_on_gpu(dsn, ctx, idx_np, T)
    perm = O.route(idx_np, T)[2]
    y = torch.full((B, R, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_scale_channels(ctx, None, False, dsn.BF16, B, R, c_valid, dx, C, scale, y, C)
    yg = torch.full((B, R, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_scale_channels(ctx, r, True, dsn.BF16, B, R, c_valid, dx, C, scale, yg, C)
    check_status(ctx, dsn)
    got, gotg = down(y), down(yg)
    ref = O.round_bf16(xh_ref)
    tol = TOL_BF16 * np.max(np.abs(ref))
    assert np.max(np.abs(got[..., :c_valid] - ref)) <= tol
    assert np.max(np.abs(gotg[..., :c_valid] - ref[perm])) <= tol
    assert np.all(got[..., c_valid:] == SENTINEL) and np.all(gotg[..., c_valid:] == SENTINEL)
    # almost every element is the correctly rounded product (a different fp32 scale can flip a rounding)
    assert np.mean(got[..., :c_valid] != ref) < 0.02


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_residual_block_tail_with_sliced_shortcut(dsn, ctx, dtype):
    """DS-ResNet first block of a stage: every width of the block follows the path, including the projection
    shortcut; out = ReLU(Re-SBN(conv3(h)) + shortcut(x)) with shortcut = sliced 1x1 convolution."""
    g = np.random.default_rng(21)
    if dtype == "bf16":
        B, hw, Cin, Cmid, Cout = 12, 14, 256, 128, 512
    else:
        B, hw, Cin, Cmid, Cout = 9, 1, 64, 32, 48          # the fp32 kernel is linear only (one row per sample)
    ratios = [0.25, 0.5, 0.75, 1.0]
    T = 4
    k_in = [int(Cin * r) for r in ratios]
    k_mid = [int(Cmid * r) for r in ratios]
    k_out = [int(Cout * r) for r in ratios]
    idx = g.integers(0, T, size=B).astype(np.int32)
    mk = (lambda a: wl.to_bf16_values(a)) if dtype == "bf16" else (lambda a: a.astype(np.float32))
    x = mk(np.maximum(g.standard_normal((B, hw, hw, Cin)), 0).astype(np.float32))
    h = mk(np.maximum(g.standard_normal((B, hw, hw, Cmid)), 0).astype(np.float32))
    Ws = mk((g.standard_normal((Cout, Cin, 1, 1)) * Cin ** -0.5).astype(np.float32))
    W3 = mk((g.standard_normal((Cout, Cmid, 1, 1)) * Cmid ** -0.5).astype(np.float32))
    gamma = (1.0 + 0.2 * g.standard_normal(Cout)).astype(np.float32)
    beta = (0.3 * g.standard_normal(Cout)).astype(np.float32)
    mu = (0.2 * g.standard_normal((T, Cout))).astype(np.float32)
    sigma = (0.6 + np.abs(g.standard_normal((T, Cout))) * 0.5).astype(np.float32)
    sc, sh = fold_on_gpu(dsn, ctx, gamma, beta, mu, sigma)
    r = route_on_gpu(dsn, ctx, idx, T)
    if dtype == "bf16":
        up, tdt, code = up_bf16, torch.bfloat16, dsn.BF16
        short = torch.full((B, hw, hw, Cout), SENTINEL, dtype=tdt, device=DEV)
        y = torch.full((B, hw, hw, Cout), SENTINEL, dtype=tdt, device=DEV)
        dsn.dsn_sliced_conv(ctx, dsn.make_conv_desc(code, hw, hw, 1, 0, Cin, Cout, k_in, k_out, up(Ws.reshape(Cout, Cin))), r, up(x), short)
        dsn.dsn_sliced_conv(ctx, dsn.make_conv_desc(code, hw, hw, 1, 0, Cmid, Cout, k_mid, k_out, up(W3.reshape(Cout, Cmid)),
                                                    act=dsn.ACT_RELU, bn_scale=sc, bn_shift=sh, residual=short), r, up(h), y)
    else:
        up, tdt, code = up_f32, torch.float32, dsn.F32
        short = torch.full((B, 1, Cout), SENTINEL, dtype=tdt, device=DEV)
        y = torch.full((B, 1, Cout), SENTINEL, dtype=tdt, device=DEV)
        dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(code, 1, Cin, Cout, k_in, k_out, up(Ws.reshape(Cout, Cin))), r,
                              up(x.reshape(B, 1, Cin)), short)
        dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(code, 1, Cmid, Cout, k_mid, k_out, up(W3.reshape(Cout, Cmid)),
                                                        act=dsn.ACT_RELU, bn_scale=sc, bn_shift=sh, residual=short), r,
                              up(h.reshape(B, 1, Cmid)), y)
    check_status(ctx, dsn)
    s_ref = O.sliced_conv(x, Ws, idx, k_in, k_out, 0, fill=0.0)
    if dtype == "bf16":
        s_ref = O.round_bf16(s_ref)
    ref = O.sliced_conv(h, W3, idx, k_mid, k_out, 0, act=O.ACT_RELU, bn=(gamma, beta, mu, sigma), residual=s_ref)
    got = down(y).reshape(B, hw, hw, Cout)
    if dtype == "bf16":
        ref = O.round_bf16(ref)
    errs = group_errors(got, ref, idx, k_out, T)
    assert max(errs.values()) <= (1e-2 if dtype == "bf16" else 2e-5), errs     # bf16: two chained stages
    assert_tail_untouched(got, idx, k_out)
