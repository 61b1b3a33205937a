"""GPU parity of dsn_sliced_linear / dsn_permute_rows against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import (DEV, SENTINEL, alloc_routing, assert_tail_untouched, check_status, down, group_errors,
                      route_on_gpu, up_bf16, up_f32, up_i32)

pytestmark = pytest.mark.gpu
TOL_BF16 = 5e-3   # max|err| / max|ref| per group, bf16 operands with fp32 accumulation
TOL_F32 = 1e-5


@pytest.fixture(scope="module")
def ctx(dsn):
    return dsn.Context(0)


def test_config1_fp32_linear(dsn, ctx):
    cfg = wl.config1()
    B, C, T = cfg["B"], cfg["C_in"], cfg["T"]
    r = route_on_gpu(dsn, ctx, cfg["idx"], T)
    x, W = up_f32(cfg["x"]), up_f32(cfg["W"])
    y = torch.full((B, 1, C), SENTINEL, dtype=torch.float32, device=DEV)
    d = dsn.make_linear_desc(dsn.F32, 1, C, C, cfg["k_in"], cfg["k_out"], W)
    dsn.dsn_sliced_linear(ctx, d, r, x, y)
    check_status(ctx, dsn)
    ref = O.sliced_linear(cfg["x"], cfg["W"], cfg["idx"], cfg["k_in"], cfg["k_out"])
    got = down(y)
    errs = group_errors(got, ref, cfg["idx"], cfg["k_out"], T)
    assert len(errs) == T and max(errs.values()) <= TOL_F32, errs
    assert_tail_untouched(got, cfg["idx"], cfg["k_out"])


@pytest.mark.parametrize("R,act,orders", [(1, 0, (0, 0)), (5, 1, (0, 1)), (70, 2, (1, 0)), (3, 0, (1, 1))])
def test_fp32_linear_orders_bias_act_ragged(dsn, ctx, R, act, orders):
    g = np.random.default_rng(R)
    B, Ci, Co, T = 37, 50, 70, 3
    k_in, k_out = [7, 33, 50], [70, 5, 41]
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = g.standard_normal((B, R, Ci)).astype(np.float32)
    W = (g.standard_normal((Co, Ci)) / 7).astype(np.float32)
    b = g.standard_normal(Co).astype(np.float32)
    r = route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2]
    x_dev = up_f32(x[perm] if orders[0] else x)
    y = torch.full((B, R, Co), SENTINEL, dtype=torch.float32, device=DEV)
    d = dsn.make_linear_desc(dsn.F32, R, Ci, Co, k_in, k_out, up_f32(W), bias=up_f32(b), act=act,
                             in_order=orders[0], out_order=orders[1])
    dsn.dsn_sliced_linear(ctx, d, r, x_dev, y)
    check_status(ctx, dsn)
    ref = O.sliced_linear(x, W, idx, k_in, k_out, bias=b, act=act)
    got = down(y)
    if orders[1]:
        tmp = np.empty_like(got)
        tmp[perm] = got
        got = tmp
    errs = group_errors(got, ref, idx, k_out, T)
    assert max(errs.values()) <= TOL_F32, errs
    assert_tail_untouched(got, idx, k_out)


def _run_bf16_linear(dsn, ctx, x, W, idx, k_in, k_out, R, in_order=0, out_order=0, bias=None, act=0, tail=0,
                     routing=None, ldx=None, ldy=None):
    B, _, Ci = x.shape
    Co = W.shape[0]
    T = len(k_in)
    r = routing if routing is not None else route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2] if routing is None else routing._perm_np
    xs = x[perm] if in_order else x
    ldx = ldx or Ci
    ldy = ldy or Co
    xbuf = torch.full((B, R, ldx), 3.0e38, dtype=torch.bfloat16, device=DEV)   # padding columns hold junk
    xbuf[..., :Ci] = up_bf16(xs)
    y = torch.full((B, R, ldy), SENTINEL, dtype=torch.bfloat16, device=DEV)
    d = dsn.make_linear_desc(dsn.BF16, R, Ci, Co, k_in, k_out, up_bf16(W), bias=None if bias is None else up_f32(bias),
                             act=act, in_order=in_order, out_order=out_order, tail=tail, ldx=ldx, ldy=ldy)
    dsn.dsn_sliced_linear(ctx, d, r, xbuf, y)
    check_status(ctx, dsn)
    got = down(y)
    if out_order:
        tmp = np.empty_like(got)
        tmp[perm] = got
        got = tmp
    return got


@pytest.mark.parametrize("in_order,out_order", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_bf16_linear_vit_small_all_orders(dsn, ctx, in_order, out_order):
    """ViT fc1 shape with GELU and bias: 48 paths, 197 tokens (two row tiles with a ragged tail)."""
    cfg = wl.config3(B=96, routing="iid")
    k_in, k_out = wl.vit_layer_slices(cfg["paths"], 64, "fc1")
    bias = np.random.default_rng(3).standard_normal(cfg["D_mlp"]).astype(np.float32) * 0.5
    got = _run_bf16_linear(dsn, ctx, cfg["x"], cfg["Wfc1"], cfg["idx"], k_in, k_out, cfg["R"], in_order, out_order,
                           bias=bias, act=dsn.ACT_GELU)
    ref = O.round_bf16(O.sliced_linear(cfg["x"], cfg["Wfc1"], cfg["idx"], k_in, k_out, bias=bias, act=O.ACT_GELU))
    errs = group_errors(got, ref, cfg["idx"], k_out, cfg["T"])
    assert max(errs.values()) <= TOL_BF16, errs
    assert_tail_untouched(got, cfg["idx"], k_out)


def test_bf16_linear_qkv_head_major_layout(dsn, ctx):
    """Fused QKV weight stored [H][3][D_h][D_e]: h heads are one leading block of 3*h*D_h rows."""
    cfg = wl.config3(B=48, routing="iid")
    Dh, paths, T = cfg["D_h"], cfg["paths"], cfg["T"]
    k_in, k_out = wl.vit_layer_slices(paths, Dh, "qkv")
    Wf = wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh)
    got = _run_bf16_linear(dsn, ctx, cfg["x"], Wf, cfg["idx"], k_in, k_out, cfg["R"])
    q, k, v = O.vit_qkv(cfg["x"], cfg["Wq"], cfg["Wk"], cfg["Wv"], cfg["idx"], paths, Dh)
    B, R = cfg["B"], cfg["R"]
    H = cfg["H"]
    ref = np.stack([q.reshape(B, R, H, Dh), k.reshape(B, R, H, Dh), v.reshape(B, R, H, Dh)], axis=3)  # [B][R][H][3][Dh]
    ref = O.round_bf16(ref.reshape(B, R, 3 * H * Dh))
    errs = group_errors(got, ref, cfg["idx"], k_out, T)
    assert max(errs.values()) <= TOL_BF16, errs
    assert_tail_untouched(got, cfg["idx"], k_out)


@pytest.mark.parametrize("R", [1, 49, 130])
def test_bf16_linear_ragged_widths_strided_and_zero_tail(dsn, ctx, R):
    """Slice widths that are no multiple of 16 (22, 26, 38 ...), leading dimensions larger than the
    tensors, padding columns full of huge values, empty groups, zero-filled tail."""
    g = np.random.default_rng(R)
    B, Ci, Co, T = 29, 72, 136, 6
    k_in, k_out = [22, 26, 38, 64, 72, 8], [136, 22, 54, 8, 100, 129]
    idx = g.choice([0, 1, 2, 4, 5], size=B).astype(np.int32)      # path 3 stays empty
    x = wl.normal(g, (B, R, Ci))
    W = wl.normal(g, (Co, Ci), std=Ci ** -0.5)
    got = _run_bf16_linear(dsn, ctx, x, W, idx, k_in, k_out, R, in_order=1, out_order=0, tail=1, ldx=80, ldy=144)
    ref = O.round_bf16(O.sliced_linear(x, W, idx, k_in, k_out))
    errs = group_errors(got, ref, idx, k_out, T)
    assert max(errs.values()) <= TOL_BF16, errs
    for i, t in enumerate(idx):
        assert np.all(got[i][:, k_out[t]:Co] == 0.0)               # zero-filled up to C_out
        assert np.all(got[i][:, Co:] == SENTINEL)                  # padding beyond C_out untouched


@pytest.mark.parametrize("in_order,out_order", [(1, 1), (0, 0)])
def test_bf16_linear_wide_slices_split_into_even_n_tiles(dsn, ctx, in_order, out_order):
    """Slices wider than one 256-column tile are dealt out over their n-tiles in 64-column units (320 = 192 + 128,
    576 = 3 x 192, 840 = 256 + 3 x 192 + a ragged end, 1344 = 6 x 224 rounded to units): every column of every tile
    boundary must come out right, with bias and ReLU, and the columns beyond a slice stay untouched."""
    g = np.random.default_rng(320)
    B, R, Ci, Co, T = 23, 70, 96, 1344, 6
    k_in, k_out = [96, 64, 96, 40, 96, 96], [320, 576, 840, 331, 1344, 264]
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = wl.normal(g, (B, R, Ci))
    W = wl.normal(g, (Co, Ci), std=Ci ** -0.5)
    bias = g.standard_normal(Co).astype(np.float32) * 0.5
    got = _run_bf16_linear(dsn, ctx, x, W, idx, k_in, k_out, R, in_order, out_order, bias=bias, act=dsn.ACT_RELU)
    ref = O.round_bf16(O.sliced_linear(x, W, idx, k_in, k_out, bias=bias, act=O.ACT_RELU))
    errs = group_errors(got, ref, idx, k_out, T)
    assert max(errs.values()) <= TOL_BF16, errs
    assert_tail_untouched(got, idx, k_out)


def test_bf16_linear_vit_base_shape_sampled(dsn, ctx):
    """ViT-B width (768 -> 3072, 8 diagonal paths), Zipf routing; the oracle checks whole samples."""
    cfg = wl.config5(B=64, routing="zipf")
    k_in, k_out = wl.vit_layer_slices(cfg["paths"], 64, "fc1")
    got = _run_bf16_linear(dsn, ctx, cfg["x"], cfg["Wfc1"], cfg["idx"], k_in, k_out, cfg["R"], act=dsn.ACT_GELU)
    counts, offsets, perm, _ = O.route(cfg["idx"], cfg["T"])
    samples = sorted({int(perm[offsets[t]]) for t in range(cfg["T"]) if counts[t]} |
                     {int(perm[offsets[t + 1] - 1]) for t in range(cfg["T"]) if counts[t]})
    ref = O.round_bf16(O.sliced_linear(cfg["x"], cfg["Wfc1"], cfg["idx"], k_in, k_out, act=O.ACT_GELU, samples=samples))
    for i in samples:
        t = cfg["idx"][i]
        e = np.max(np.abs(got[i, :, :k_out[t]] - ref[i, :, :k_out[t]])) / np.max(np.abs(ref[i, :, :k_out[t]]))
        assert e <= TOL_BF16, (i, t, e)
    assert_tail_untouched(got, cfg["idx"], k_out)


def test_bf16_linear_singleton_groups(dsn, ctx):
    """Caller-built group list: one group per sample, slice g mod T (several groups share a slice)."""
    cfg = wl.config5(B=40, routing="singleton")
    B, T, R = cfg["B"], cfg["T"], cfg["R"]
    k_in, k_out = wl.vit_layer_slices(cfg["paths"], 64, "qkv")
    Wf = wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], 64)
    order = np.random.default_rng(0).permutation(B).astype(np.int32)   # group g holds sample order[g]
    slices = cfg["idx"][order]
    inv = np.empty(B, np.int32)
    inv[order] = np.arange(B, dtype=np.int32)
    bufs = [up_i32(np.ones(B)), up_i32(np.arange(B + 1)), up_i32(order), up_i32(inv), up_i32(slices)]
    r = dsn.make_routing(B, B, *bufs)
    r._perm_np = order
    got = _run_bf16_linear(dsn, ctx, cfg["x"], Wf, cfg["idx"], k_in, k_out, R, routing=r)
    q, k, v = O.vit_qkv(cfg["x"], cfg["Wq"], cfg["Wk"], cfg["Wv"], cfg["idx"], cfg["paths"], 64)
    H, Dh = cfg["H"], 64
    ref = np.stack([q.reshape(B, R, H, Dh), k.reshape(B, R, H, Dh), v.reshape(B, R, H, Dh)], axis=3)
    ref = O.round_bf16(ref.reshape(B, R, 3 * H * Dh))
    errs = group_errors(got, ref, cfg["idx"], k_out, T)
    assert max(errs.values()) <= TOL_BF16, errs


def test_bf16_linear_runs_are_bitwise_reproducible(dsn, ctx):
    cfg = wl.config3(B=32, routing="iid")
    k_in, k_out = wl.vit_layer_slices(cfg["paths"], 64, "fc2")
    x = wl.normal(np.random.default_rng(5), (32, cfg["R"], cfg["D_mlp"]))
    a = _run_bf16_linear(dsn, ctx, x, cfg["Wfc2"], cfg["idx"], k_in, k_out, cfg["R"])
    b = _run_bf16_linear(dsn, ctx, x, cfg["Wfc2"], cfg["idx"], k_in, k_out, cfg["R"])
    np.testing.assert_array_equal(a, b)
    ref = O.round_bf16(O.sliced_linear(x, cfg["Wfc2"], cfg["idx"], k_in, k_out))
    assert max(group_errors(a, ref, cfg["idx"], k_out, cfg["T"]).values()) <= TOL_BF16


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_permute_rows_roundtrip(dsn, ctx, dtype):
    g = np.random.default_rng(11)
    B, R, C, T = 23, 6, 40, 4
    k = [8, 13, 40, 24]
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = wl.normal(g, (B, R, C))
    r = route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2]
    up, tdt, code = (up_bf16, torch.bfloat16, dsn.BF16) if dtype == "bf16" else (up_f32, torch.float32, dsn.F32)
    src = up(x)
    grouped = torch.full((B, R, C), SENTINEL, dtype=tdt, device=DEV)
    back = torch.full((B, R, C), SENTINEL, dtype=tdt, device=DEV)
    dsn.dsn_permute_rows(ctx, r, code, R, k, src, C, grouped, C, True)
    dsn.dsn_permute_rows(ctx, r, code, R, k, grouped, C, back, C, False)
    check_status(ctx, dsn)
    gq, bk = down(grouped), down(back)
    for p in range(B):
        i = perm[p]
        kk = k[idx[i]]
        np.testing.assert_array_equal(gq[p][:, :kk], x[i][:, :kk])
        assert np.all(gq[p][:, kk:] == SENTINEL)
        np.testing.assert_array_equal(bk[i][:, :kk], x[i][:, :kk])
        assert np.all(bk[i][:, kk:] == SENTINEL)


def test_host_side_argument_errors_launch_nothing(dsn, ctx):
    B, R, C, T = 4, 2, 16, 2
    r = route_on_gpu(dsn, ctx, np.zeros(B, np.int32), T)
    x = torch.zeros(B, R, C, dtype=torch.bfloat16, device=DEV)
    W = torch.zeros(C, C, dtype=torch.bfloat16, device=DEV)
    y = torch.full((B, R, C), SENTINEL, dtype=torch.bfloat16, device=DEV)

    def code_of(**kw):
        args = dict(dtype=dsn.BF16, R=R, C_in=C, C_out=C, k_in=[8, 16], k_out=[8, 16], W=W)
        args.update(kw)
        xx = args.pop("x", x)
        d = dsn.make_linear_desc(**args)
        try:
            dsn.dsn_sliced_linear(ctx, d, r, xx, y)
        except dsn.DsnError as e:
            return e.code
        return 0

    assert code_of(k_in=[8, 17]) == dsn.ERR_INVALID_ARG          # k > C
    assert code_of(k_out=[0, 16]) == dsn.ERR_INVALID_ARG
    assert code_of(ldx=C + 4) == dsn.ERR_ALIGNMENT               # bf16 leading dimension not a multiple of 8
    assert code_of(x=x.view(-1)[1:]) == dsn.ERR_ALIGNMENT        # misaligned pointer
    assert code_of(act=9) == dsn.ERR_INVALID_ARG
    assert code_of(W=None) == dsn.ERR_INVALID_ARG
    assert code_of(k_in=[8] * 65, k_out=[8] * 65) == dsn.ERR_INVALID_ARG   # T too large
    assert np.all(down(y) == SENTINEL)
    check_status(ctx, dsn)


def test_tensor_maps_are_encoded_once_per_buffer_and_slice(dsn):
    """Repeated calls on the same buffers reuse the context's cached tensor maps (no misses after the first call) and
    give the same bytes; another output buffer misses only for the maps that name it."""
    import os
    saved = os.environ.pop("DSN_MAP_CACHE", None)          # the switch is read when the context is created
    try:
        c = dsn.Context(0)
    finally:
        if saved is not None:
            os.environ["DSN_MAP_CACHE"] = saved
    g = np.random.default_rng(9)
    B, R, C, T = 20, 50, 192, 4
    k_in, k_out = [64, 128, 192, 192], [192, 64, 128, 192]
    idx = g.integers(0, T, size=B).astype(np.int32)
    r = route_on_gpu(dsn, c, idx, T)
    x, W = up_bf16(wl.normal(g, (B, R, C))), up_bf16(wl.normal(g, (C, C), std=C ** -0.5))
    d = dsn.make_linear_desc(dsn.BF16, R, C, C, k_in, k_out, W)
    y1 = torch.zeros((B, R, C), dtype=torch.bfloat16, device=DEV)
    y2 = torch.zeros((B, R, C), dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(c, d, r, x, y1)
    h0, m0 = c.map_cache_stats()
    assert m0 > 0
    dsn.dsn_sliced_linear(c, d, r, x, y1)
    h1, m1 = c.map_cache_stats()
    assert m1 == m0 and h1 - h0 == m0 + h0                 # every map of the second call came from the cache
    dsn.dsn_sliced_linear(c, d, r, x, y2)
    h2, m2 = c.map_cache_stats()
    assert 0 < m2 - m1 < m0                                # only the output maps are new
    check_status(c, dsn)
    assert torch.equal(y1, y2)
    st = c.stats()                                          # the library's own launch counters
    assert st["calls"] == 3 and st["launches_route"] == 1 and st["launches_gemm_pair"] + st["launches_gemm_one_cta"] == 3
    assert st["launches"] == 4 and st["map_hits"] == h2 and st["map_misses"] == m2


def test_layer_forward_rejects_a_layer_that_reads_more_than_was_written(dsn, ctx):
    """All layers of a block inherit one decision: a path may not read more columns of an intermediate than
    the layer before wrote for it (those columns hold stale workspace bytes).  Refused on the host."""
    B, R, C, T = 4, 8, 64, 2
    W = torch.zeros(C, C, dtype=torch.bfloat16, device=DEV)
    x = torch.zeros(B, R, C, dtype=torch.bfloat16, device=DEV)
    y = torch.full((B, R, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    idx = torch.zeros(B, dtype=torch.int32, device=DEV)

    def code_of(k_out0, k_in1, heads=None):
        layers = [dsn.make_linear_desc(dsn.BF16, R, C, 3 * C if heads else C, [C, C], k_out0, torch.zeros(3 * C if heads else C, C, dtype=torch.bfloat16, device=DEV))]
        if heads:
            layers.append(dsn.make_attention_desc(R, 1, 64, heads))
        layers.append(dsn.make_linear_desc(dsn.BF16, R, C, C, k_in1, [C, C], W))
        L = dsn.make_layer_desc(B, T, layers, None)
        ws = torch.empty(max(1024, dsn.dsn_layer_workspace_bytes(L) + 4096), dtype=torch.uint8, device=DEV)
        try:
            dsn.dsn_layer_forward(ctx, L, x, idx, y, ws)
        except dsn.DsnError as e:
            return e.code
        return 0

    assert code_of([32, 64], [32, 64]) == 0
    assert code_of([32, 64], [40, 64]) == dsn.ERR_INVALID_ARG           # path 0 reads 40 columns, 32 were written
    assert code_of([192, 128], [64, 64], heads=[1, 1]) == dsn.ERR_INVALID_ARG   # QKV of path 1 too narrow for its head
    assert code_of([192, 192], [64, 64], heads=[1, 2]) == dsn.ERR_INVALID_ARG   # more heads than the layer has
    assert code_of([192, 192], [64, 64], heads=[1, 1]) == 0
    check_status(ctx, dsn)


@pytest.mark.parametrize("T,in_order,out_order", [(40, 0, 0), (64, 1, 1)])
def test_bf16_linear_more_slices_than_one_launch_holds(dsn, ctx, T, in_order, out_order):
    """A launch carries tensor maps for 16 distinct slices; a layer with more (here 40, and the maximum of
    64 paths, all distinct) runs as several launches over disjoint sets of groups.  Every group must come out
    right and nothing outside a group's own columns may be touched."""
    g = np.random.default_rng(1000 + T)
    B, R, Ci, Co = 3 * T + 5, 33, 264, 328
    k_in = [8 * (1 + (5 * t) % 33) for t in range(T)]            # 8 .. 264, all multiples of 8
    k_out = [8 * (1 + (7 * t + 3) % 41) for t in range(T)]       # 8 .. 328
    assert len({(a, b) for a, b in zip(k_in, k_out)}) == T
    idx = g.integers(0, T, size=B).astype(np.int32)
    x = wl.normal(g, (B, R, Ci))
    W = wl.normal(g, (Co, Ci), std=Ci ** -0.5)
    got = _run_bf16_linear(dsn, ctx, x, W, idx, k_in, k_out, R, in_order, out_order, act=dsn.ACT_RELU)
    ref = O.round_bf16(O.sliced_linear(x, W, idx, k_in, k_out, act=O.ACT_RELU))
    errs = group_errors(got, ref, idx, k_out, T)
    assert max(errs.values()) <= TOL_BF16, errs
    assert_tail_untouched(got, idx, k_out)
