"""GPU parity: routing (bit-exact) and gate (exact outside a 1e-4 score margin) against the oracle."""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import DEV, alloc_routing, check_status, route_on_gpu, routing_arrays, up_bf16, up_f32, up_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(dsn):
    return dsn.Context(0)


@pytest.mark.parametrize("B,T", [(1, 1), (5, 1), (1, 7), (64, 4), (128, 14), (256, 48), (1024, 8), (1025, 64),
                                 (5000, 14), (33, 64)])
def test_route_bit_exact(dsn, ctx, B, T):
    idx = np.random.default_rng(B * 131 + T).integers(0, T, size=B).astype(np.int32)
    r = route_on_gpu(dsn, ctx, idx, T)
    check_status(ctx, dsn)
    got = routing_arrays(r)
    ref = O.route(idx, T)
    for g, e in zip(got, ref):
        np.testing.assert_array_equal(g, e)


def test_route_stress_distributions(dsn, ctx):
    B, T = 1024, 8
    cases = [wl.idx_all_one(B, 7), wl.idx_all_one(B, 0), wl.idx_quota_uniform(wl.rng(5, 9), B, T),
             wl.idx_zipf(wl.rng(5, 9), B, T), (np.arange(B) % T).astype(np.int32),
             wl.idx_skewed_bands(wl.rng(41, 6), 256, 14)]
    for idx in cases:
        T_ = 14 if len(idx) == 256 else T
        r = route_on_gpu(dsn, ctx, idx, T_)
        for g, e in zip(routing_arrays(r), O.route(idx, T_)):
            np.testing.assert_array_equal(g, e)
    check_status(ctx, dsn)


def test_route_empty_batch_and_determinism(dsn, ctx):
    r = alloc_routing(dsn, 0, 3)
    dsn.dsn_route(ctx, up_i32(np.zeros(1, np.int32)), 0, 3, r)
    counts, offsets, _, _ = routing_arrays(r)
    assert counts.tolist() == [0, 0, 0] and offsets.tolist() == [0, 0, 0, 0]
    idx = np.random.default_rng(1).integers(0, 14, size=3000).astype(np.int32)
    a = routing_arrays(route_on_gpu(dsn, ctx, idx, 14))
    b = routing_arrays(route_on_gpu(dsn, ctx, idx, 14))
    for u, v in zip(a, b):
        np.testing.assert_array_equal(u, v)
    check_status(ctx, dsn)


def test_route_bad_index_is_reported_not_used(dsn, ctx):
    idx = np.array([0, 2, 9, 1, -3, 2], dtype=np.int32)
    r = route_on_gpu(dsn, ctx, idx, 3)
    code, detail = ctx.get_status()
    assert code == dsn.ERR_BAD_INDEX and detail == 2
    counts, offsets, perm, inv = routing_arrays(r)
    assert counts.tolist() == [1, 1, 2] and offsets.tolist() == [0, 1, 2, 4]
    assert perm.tolist() == [0, 3, 1, 5, -1, -1] and inv.tolist() == [0, 2, -1, 1, -1, 3]
    assert ctx.get_status() == (0, 0)           # reading clears it


def _run_gate(dsn, ctx, x_np, W1, W2, b1=None, b2=None, c_valid=None, dtype="bf16"):
    B, R, C = x_np.shape
    T, M = W2.shape
    x = up_bf16(x_np) if dtype == "bf16" else up_f32(x_np)
    dW1, dW2 = up_f32(W1), up_f32(W2)
    db1 = None if b1 is None else up_f32(b1)
    db2 = None if b2 is None else up_f32(b2)
    g = dsn.make_gate_desc(dsn.BF16 if dtype == "bf16" else dsn.F32, B, R, C, M, T, dW1, dW2, db1, db2, c_valid=c_valid)
    ws = torch.empty(dsn.dsn_gate_workspace_bytes(g), dtype=torch.uint8, device=DEV)
    idx = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    logits = torch.zeros(B, T, dtype=torch.float32, device=DEV)
    dsn.dsn_gate(ctx, g, x, idx, logits, ws)
    check_status(ctx, dsn)
    return idx.cpu().numpy(), logits.cpu().numpy().astype(np.float64)


def _compare_gate(idx_gpu, logits_gpu, ref):
    idx_ref, s_ref, margin = ref
    scale = max(1.0, np.max(np.abs(s_ref)))
    assert np.max(np.abs(logits_gpu - s_ref)) <= 2e-5 * scale
    safe = margin >= 1e-4
    np.testing.assert_array_equal(idx_gpu[safe], idx_ref[safe])
    # inside the margin the device may pick either of the two leaders
    for i in np.nonzero(~safe)[0]:
        assert s_ref[i, idx_gpu[i]] >= s_ref[i].max() - 1e-4
    return int((~safe).sum())


def test_gate_resnet_shape(dsn, ctx):
    cfg = wl.config2(B=128)
    B, R, C = cfg["B"], cfg["H"] * cfg["W"], cfg["C_outer"]
    x = cfg["x"].reshape(B, R, C)
    idx, logits = _run_gate(dsn, ctx, x, cfg["gate_W1"], cfg["gate_W2"])
    _compare_gate(idx, logits, O.gate(x, cfg["gate_W1"], cfg["gate_W2"]))
    assert len(np.unique(idx)) > 1


def test_gate_vit_shape_48_paths(dsn, ctx):
    cfg = wl.config3(B=64)
    idx, logits = _run_gate(dsn, ctx, cfg["x"], cfg["gate_W1"], cfg["gate_W2"])
    _compare_gate(idx, logits, O.gate(cfg["x"], cfg["gate_W1"], cfg["gate_W2"]))


@pytest.mark.parametrize("B,R,C,M,T,dtype", [(3, 1, 8, 4, 2, "bf16"), (5, 7, 20, 9, 3, "bf16"), (9, 49, 2048, 128, 14, "bf16"),
                                             (6, 13, 50, 16, 5, "f32"), (2, 300, 64, 32, 64, "f32"), (130, 16, 40, 8, 1, "bf16")])
def test_gate_odd_shapes_bias_and_elastic_input(dsn, ctx, B, R, C, M, T, dtype):
    g = np.random.default_rng(B + R + C)
    x = g.standard_normal((B, R, C)).astype(np.float32)
    if dtype == "bf16":
        x = wl.to_bf16_values(x)
    W1 = (g.standard_normal((M, C)) / np.sqrt(C)).astype(np.float32)
    W2 = (g.standard_normal((T, M)) / np.sqrt(M)).astype(np.float32)
    b1 = g.standard_normal(M).astype(np.float32) * 0.1
    b2 = g.standard_normal(T).astype(np.float32) * 0.1
    cv = C - 8 if (C % 8 == 0 and C > 8) else C
    idx, logits = _run_gate(dsn, ctx, x, W1, W2, b1, b2, c_valid=cv, dtype=dtype)
    _compare_gate(idx, logits, O.gate(x, W1, W2, b1, b2, c_valid=cv))


def test_gate_ties_take_lowest_index_and_nonfinite_is_reported(dsn, ctx):
    B, R, C, M, T = 4, 3, 8, 8, 4
    x = np.full((B, R, C), 2.0, dtype=np.float32)
    W1 = np.eye(M, C, dtype=np.float32)
    W2 = np.zeros((T, M), dtype=np.float32)
    W2[1, 0] = 1.0
    W2[3, 0] = 1.0
    idx, _ = _run_gate(dsn, ctx, x, W1, W2)
    assert idx.tolist() == [1, 1, 1, 1]
    xb = x.copy()
    xb[2, 0, 0] = np.inf
    B_, R_, C_ = xb.shape
    dx, dW1, dW2 = up_bf16(xb), up_f32(W1), up_f32(W2)
    g = dsn.make_gate_desc(dsn.BF16, B_, R_, C_, M, T, dW1, dW2)
    ws = torch.empty(dsn.dsn_gate_workspace_bytes(g), dtype=torch.uint8, device=DEV)
    out = torch.zeros(B_, dtype=torch.int32, device=DEV)
    dsn.dsn_gate(ctx, g, dx, out, None, ws)
    code, detail = ctx.get_status()
    assert code == dsn.ERR_NONFINITE and detail == 2
    assert all(0 <= v < T for v in out.cpu().tolist())
