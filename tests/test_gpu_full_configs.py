"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times.  The oracle evaluates whole samples (every sample for the small configs, the first
and last sample of every group for the large ones: samples are independent, so that is exact)."""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import DEV, SENTINEL, check_status, down, up_bf16, up_f32, up_i32

pytestmark = pytest.mark.gpu
TOL_BF16 = 5e-3
TOL_CHAIN_MAX = 1e-2     # chained bf16 layers: one output ulp, see test_gpu_conv_layer.py
TOL_CHAIN_MEAN = 2e-4


@pytest.fixture(scope="module")
def ctx(dsn):
    return dsn.Context(0)


def ohwi(W):
    return np.ascontiguousarray(np.transpose(W, (0, 2, 3, 1)))


def group_samples(idx, T):
    """First and last sample of every non-empty group."""
    counts, offsets, perm, _ = O.route(idx, T)
    s = set()
    for t in range(T):
        if counts[t]:
            s.add(int(perm[offsets[t]]))
            s.add(int(perm[offsets[t + 1] - 1]))
    return sorted(s)


def check_samples(got, ref, idx, k_out, samples, tol_max, tol_mean=None, report=None, what=""):
    worst, worst_mean = 0.0, 0.0
    for i in samples:
        ko = k_out[idx[i]]
        g, r = got[i][..., :ko], ref[i][..., :ko]
        assert np.all(np.isfinite(r))
        scale = np.max(np.abs(r))
        err = np.max(np.abs(g - r)) / scale
        worst = max(worst, err)
        assert err <= tol_max, (i, int(idx[i]), err)
        worst_mean = max(worst_mean, np.mean(np.abs(g - r)) / scale)
        if tol_mean is not None:
            assert np.mean(np.abs(g - r)) / scale <= tol_mean, (i, int(idx[i]))
        assert np.all(got[i][..., ko:] == SENTINEL), f"sample {i}: columns >= k_out were written"
    if report is not None:
        report.append(f"{what}: worst max {worst:.2e}, worst mean {worst_mean:.2e} over {len(list(samples))} samples "
                      f"(bounds {tol_max:.0e}" + (f" / {tol_mean:.0e})" if tol_mean is not None else ")"))
    return worst


def bottleneck_forward(dsn, ctx, cfg, with_gate):
    B, H, Wd, C, Ci, T, widths = cfg["B"], cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"], cfg["widths"]
    full = [C] * T
    W1, W2, W3 = up_bf16(cfg["W1"].reshape(Ci, C)), up_bf16(ohwi(cfg["W2"])), up_bf16(cfg["W3"].reshape(C, Ci))
    layers = [dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, Ci, full, widths, W1, act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 3, 1, Ci, Ci, widths, widths, W2, act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, Ci, C, widths, full, W3)]
    gate = None
    if with_gate:
        gW1, gW2 = up_f32(cfg["gate_W1"]), up_f32(cfg["gate_W2"])
        gate = dsn.make_gate_desc(dsn.BF16, B, H * Wd, C, gW1.shape[0], T, gW1, gW2)
    L = dsn.make_layer_desc(B, T, layers, gate)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, H, Wd, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    idx_out = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    r_out = dsn.Routing()
    dsn.dsn_layer_forward(ctx, L, up_bf16(cfg["x"]), None if with_gate else up_i32(cfg["idx"]), y, ws, r_out=r_out,
                          idx_out=idx_out)
    check_status(ctx, dsn)
    base = ws.data_ptr()
    def view(ptr, n):
        return ws[ptr - base:ptr - base + 4 * n].view(torch.int32).cpu().numpy()
    routing = (view(r_out.counts, T), view(r_out.offsets, T + 1), view(r_out.perm, B), view(r_out.inv_perm, B))
    return down(y), idx_out.cpu().numpy(), routing


def test_config2_full_batch_gate_driven(dsn, ctx, parity_report):
    """The benchmark's default workload: B = 128, 14x14, 1024 -> w -> w -> 1024, gate-driven routing."""
    cfg = wl.config2(B=128)
    B, R, C, T = cfg["B"], cfg["H"] * cfg["W"], cfg["C_outer"], cfg["T"]
    got, idx_gpu, routing = bottleneck_forward(dsn, ctx, cfg, with_gate=True)
    idx_ref, _, margin = O.gate(cfg["x"].reshape(B, R, C), cfg["gate_W1"], cfg["gate_W2"])
    safe = margin >= 1e-4
    np.testing.assert_array_equal(idx_gpu[safe], idx_ref[safe])
    idx_used = np.where(safe, idx_ref, idx_gpu)
    for g_arr, o_arr in zip(routing, O.route(idx_gpu, T)):
        np.testing.assert_array_equal(g_arr, o_arr)          # bit-exact routing of the gate's choice
    assert routing[0].sum() == B                              # histogram sums to the batch size
    _, _, ref = O.bottleneck(cfg["x"], cfg["W1"], cfg["W2"], cfg["W3"], idx_used, cfg["widths"], mirror_bf16=True)
    check_samples(got, ref, idx_used, [C] * T, range(B), TOL_CHAIN_MAX, TOL_CHAIN_MEAN, parity_report,
                  "cfg2 bottleneck chain (3 bf16 layers, one chained launch), B=128 gate-driven")


@pytest.mark.parametrize("stage,routing", [(1, "skewed"), (2, "uniform"), (3, "skewed"), (3, "uniform"), (4, "skewed")])
def test_config4_resnet_stages_full_batch(dsn, ctx, stage, routing, parity_report):
    cfg = wl.config4(stage, B=256, routing=routing)
    T, C = cfg["T"], cfg["C_outer"]
    got, idx_gpu, routing_arrays = bottleneck_forward(dsn, ctx, cfg, with_gate=False)
    np.testing.assert_array_equal(idx_gpu, cfg["idx"])
    for g_arr, o_arr in zip(routing_arrays, O.route(cfg["idx"], T)):
        np.testing.assert_array_equal(g_arr, o_arr)
    samples = group_samples(cfg["idx"], T)
    _, _, ref = O.bottleneck(cfg["x"], cfg["W1"], cfg["W2"], cfg["W3"], cfg["idx"], cfg["widths"], mirror_bf16=True,
                             samples=samples)
    check_samples(got, ref, cfg["idx"], [C] * T, samples, TOL_CHAIN_MAX, TOL_CHAIN_MEAN, parity_report,
                  f"cfg4 stage {stage} bottleneck chain (3 bf16 layers), B=256 {routing}")


def bottleneck_case(name):
    if name == "cfg2":
        return wl.config2(B=128, routing="uniform")
    stage, routing = name
    return wl.config4(stage, B=256, routing=routing)


@pytest.mark.parametrize("case", ["cfg2", (1, "skewed"), (1, "uniform"), (2, "uniform"), (3, "skewed"), (4, "skewed")],
                         ids=lambda c: c if isinstance(c, str) else f"cfg4-stage{c[0]}-{c[1]}")
def test_bottleneck_layers_teacher_forced_full_batch(dsn, ctx, case, parity_report):
    """Every layer of the bottleneck on its own at the full batch, in the launch configuration of the per-layer
    path (grouped intermediates): conv2 and conv3 read the ORACLE's bf16-mirrored intermediate for the checked
    samples, so each layer is held to the single-layer bound with no error carried over from the layer before.
    The device's bf16 output is compared with the oracle's UNROUNDED value of that layer (its input is the rounded
    intermediate): a correct result is then within half a bf16 ulp (2^-8 of the value) plus the fp32 accumulation
    error, always inside 5e-3, whereas two rounded values can differ by a whole ulp (up to 7.8e-3 of the value)
    wherever the two accumulations fall on different sides of a rounding boundary."""
    from gpu_util import route_on_gpu
    cfg = bottleneck_case(case)
    B, H, Wd, C, Ci, T, widths, idx = (cfg["B"], cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"],
                                       cfg["widths"], cfg["idx"])
    full = [C] * T
    samples = group_samples(idx, T)
    y1u = O.sliced_conv(cfg["x"], cfg["W1"], idx, full, widths, 0, act=O.ACT_RELU, fill=0.0, samples=samples)
    y1 = O.round_bf16(y1u)
    y2u = O.sliced_conv(y1, cfg["W2"], idx, widths, widths, 1, act=O.ACT_RELU, fill=0.0, samples=samples)
    y2 = O.round_bf16(y2u)
    y3u = O.sliced_conv(y2, cfg["W3"], idx, widths, full, 0, fill=0.0, samples=samples)
    r = route_on_gpu(dsn, ctx, idx, T)
    inv = O.route(idx, T)[3]
    pos = torch.from_numpy(inv[samples].astype(np.int64)).to(DEV)
    W1, W2, W3 = up_bf16(cfg["W1"].reshape(Ci, C)), up_bf16(ohwi(cfg["W2"])), up_bf16(cfg["W3"].reshape(C, Ci))
    mk = dsn.make_conv_desc
    t1 = torch.full((B, H, Wd, Ci), SENTINEL, dtype=torch.bfloat16, device=DEV)
    t2 = torch.full((B, H, Wd, Ci), SENTINEL, dtype=torch.bfloat16, device=DEV)
    y = torch.full((B, H, Wd, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_conv(ctx, mk(dsn.BF16, H, Wd, 1, 0, C, Ci, full, widths, W1, act=dsn.ACT_RELU, in_order=0, out_order=1),
                        r, up_bf16(cfg["x"]), t1)
    check_status(ctx, dsn)
    got1 = down(t1[pos])
    tag = "cfg2 B=128 uniform" if case == "cfg2" else f"cfg4 stage {case[0]} B=256 {case[1]}"
    check_samples(got1, y1u[samples], idx[samples], widths, range(len(samples)), TOL_BF16, None, parity_report,
                  f"{tag} conv1 1x1 alone")
    t1[pos] = up_bf16(y1[samples])                       # teacher forcing: the oracle's intermediate for the checked samples
    dsn.dsn_sliced_conv(ctx, mk(dsn.BF16, H, Wd, 3, 1, Ci, Ci, widths, widths, W2, act=dsn.ACT_RELU, in_order=1, out_order=1),
                        r, t1, t2)
    check_status(ctx, dsn)
    check_samples(down(t2[pos]), y2u[samples], idx[samples], widths, range(len(samples)), TOL_BF16, None, parity_report,
                  f"{tag} conv2 3x3 alone (oracle input)")
    t2[pos] = up_bf16(y2[samples])
    dsn.dsn_sliced_conv(ctx, mk(dsn.BF16, H, Wd, 1, 0, Ci, C, widths, full, W3, in_order=1, out_order=0), r, t2, y)
    check_status(ctx, dsn)
    sel = torch.from_numpy(np.asarray(samples, dtype=np.int64)).to(DEV)
    check_samples(down(y[sel]), y3u[samples], idx[samples], full, range(len(samples)), TOL_BF16, None, parity_report,
                  f"{tag} conv3 1x1 alone (oracle input)")


def test_config3_vit_small_full_batch(dsn, ctx):
    """B = 256 x 197 tokens, 48 paths: fused QKV, proj on its own input, gate + fc1(GELU) + fc2 chain."""
    cfg = wl.config3(B=256, routing="uniform")
    B, R, De, Dm, T, paths, Dh, H = (cfg["B"], cfg["R"], cfg["D_e"], cfg["D_mlp"], cfg["T"], cfg["paths"], cfg["D_h"],
                                     cfg["H"])
    x = up_bf16(cfg["x"])
    # gate + MLP chain
    ki1, ko1 = wl.vit_layer_slices(paths, Dh, "fc1")
    ki2, ko2 = wl.vit_layer_slices(paths, Dh, "fc2")
    layers = [dsn.make_linear_desc(dsn.BF16, R, De, Dm, ki1, ko1, up_bf16(cfg["Wfc1"]), act=dsn.ACT_GELU),
              dsn.make_linear_desc(dsn.BF16, R, Dm, De, ki2, ko2, up_bf16(cfg["Wfc2"]))]
    gW1, gW2 = up_f32(cfg["gate_W1"]), up_f32(cfg["gate_W2"])
    gate = dsn.make_gate_desc(dsn.BF16, B, R, De, gW1.shape[0], T, gW1, gW2)
    L = dsn.make_layer_desc(B, T, layers, gate)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    idx_out = torch.zeros(B, dtype=torch.int32, device=DEV)
    r_out = dsn.Routing()
    dsn.dsn_layer_forward(ctx, L, x, None, y, ws, r_out=r_out, idx_out=idx_out)
    check_status(ctx, dsn)
    idx_gpu = idx_out.cpu().numpy()
    idx_ref, _, margin = O.gate(cfg["x"], cfg["gate_W1"], cfg["gate_W2"])
    safe = margin >= 1e-4
    np.testing.assert_array_equal(idx_gpu[safe], idx_ref[safe])
    idx_used = np.where(safe, idx_ref, idx_gpu)
    samples = group_samples(idx_used, T)
    _, ref = O.vit_mlp(cfg["x"], cfg["Wfc1"], cfg["Wfc2"], idx_used, paths, mirror_bf16=True, samples=samples)
    check_samples(down(y), ref, idx_used, ko2, samples, TOL_CHAIN_MAX, TOL_CHAIN_MEAN)

    # QKV and proj with the block's routing (arrays left in the workspace by the forward call)
    kq, koq = wl.vit_layer_slices(paths, Dh, "qkv")
    Wf = up_bf16(wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh))
    yq = torch.full((B, R, 3 * H * Dh), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, De, 3 * H * Dh, kq, koq, Wf), r_out, x, yq)
    check_status(ctx, dsn)
    q, k, v = O.vit_qkv(cfg["x"], cfg["Wq"], cfg["Wk"], cfg["Wv"], idx_gpu, paths, Dh, samples=samples)
    ref = np.stack([q.reshape(B, R, H, Dh), k.reshape(B, R, H, Dh), v.reshape(B, R, H, Dh)], axis=3)
    check_samples(down(yq), O.round_bf16(ref.reshape(B, R, 3 * H * Dh)), idx_gpu, koq, samples, TOL_BF16)
    kp, kop = wl.vit_layer_slices(paths, Dh, "proj")
    a = wl.normal(wl.rng(3, 20), (B, R, H * Dh))
    yp = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, H * Dh, De, kp, kop, up_bf16(cfg["Wproj"])), r_out,
                          up_bf16(a), yp)
    check_status(ctx, dsn)
    ref = O.round_bf16(O.sliced_linear(a, cfg["Wproj"], idx_gpu, kp, kop, samples=samples))
    check_samples(down(yp), ref, idx_gpu, kop, samples, TOL_BF16)


@pytest.fixture(scope="module")
def vit_base():
    cfg = wl.config5(B=1024, routing="uniform")
    return cfg, up_bf16(cfg["x"])


@pytest.mark.parametrize("case", ["one7", "one0", "uniform", "zipf", "singleton"])
def test_config5_vit_base_routing_stress(dsn, ctx, vit_base, case):
    """B = 1024 x 197 tokens, ViT-B width, 8 diagonal paths: QKV and the fc1(GELU) -> fc2 chain."""
    cfg, x = vit_base
    B, R, De, Dm, T, paths, Dh, H = (cfg["B"], cfg["R"], cfg["D_e"], cfg["D_mlp"], cfg["T"], cfg["paths"], cfg["D_h"],
                                     cfg["H"])
    g = wl.rng(5, 9)
    if case == "one7":
        idx = wl.idx_all_one(B, 7)
    elif case == "one0":
        idx = wl.idx_all_one(B, 0)
    elif case == "uniform":
        idx = wl.idx_quota_uniform(g, B, T)
    elif case == "zipf":
        idx = wl.idx_zipf(g, B, T)
    else:
        idx = (np.arange(B) % T).astype(np.int32)
    ints = lambda n: torch.zeros(n, dtype=torch.int32, device=DEV)
    if case == "singleton":     # 1024 caller-built groups of one sample each, slice g mod 8
        order = np.random.default_rng(1).permutation(B).astype(np.int32)
        inv = np.empty(B, np.int32)
        inv[order] = np.arange(B, dtype=np.int32)
        bufs = [up_i32(np.ones(B)), up_i32(np.arange(B + 1)), up_i32(order), up_i32(inv), up_i32(idx[order])]
        r = dsn.make_routing(B, B, *bufs)
        samples = [0, 1, 7, 500, 1023]
    else:
        r = dsn.make_routing(B, T, ints(T), ints(T + 1), ints(B), ints(B))
        dsn.dsn_route(ctx, up_i32(idx), B, T, r)
        samples = group_samples(idx, T)[:6]
    kq, koq = wl.vit_layer_slices(paths, Dh, "qkv")
    Wf = up_bf16(wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh))
    yq = torch.full((B, R, 3 * H * Dh), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, De, 3 * H * Dh, kq, koq, Wf), r, x, yq)
    check_status(ctx, dsn)
    got = down(yq[samples])
    q, k, v = O.vit_qkv(cfg["x"][samples], cfg["Wq"], cfg["Wk"], cfg["Wv"], idx[samples], paths, Dh)
    n = len(samples)
    ref = np.stack([q.reshape(n, R, H, Dh), k.reshape(n, R, H, Dh), v.reshape(n, R, H, Dh)], axis=3)
    check_samples(got, O.round_bf16(ref.reshape(n, R, 3 * H * Dh)), idx[samples], koq, range(n), TOL_BF16)
    del yq

    # fc1 (input order -> grouped, GELU) then fc2 (grouped -> input order), as dsn_layer_forward chains them
    ki1, ko1 = wl.vit_layer_slices(paths, Dh, "fc1")
    ki2, ko2 = wl.vit_layer_slices(paths, Dh, "fc2")
    hid = torch.empty((B, R, Dm), dtype=torch.bfloat16, device=DEV)
    y = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, De, Dm, ki1, ko1, up_bf16(cfg["Wfc1"]), act=dsn.ACT_GELU,
                                                    in_order=dsn.INPUT_ORDER, out_order=dsn.GROUPED), r, x, hid)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, Dm, De, ki2, ko2, up_bf16(cfg["Wfc2"]),
                                                    in_order=dsn.GROUPED, out_order=dsn.INPUT_ORDER), r, hid, y)
    check_status(ctx, dsn)
    got = down(y[samples])
    _, ref = O.vit_mlp(cfg["x"][samples], cfg["Wfc1"], cfg["Wfc2"], idx[samples], paths, mirror_bf16=True)
    check_samples(got, ref, idx[samples], ko2, range(n), TOL_CHAIN_MAX, TOL_CHAIN_MEAN)


@pytest.mark.parametrize("name,routing", [("cfg5", "uniform"), ("cfg3", "gate")])
def test_vit_block_one_call_full_batch(dsn, ctx, vit_base, name, routing, parity_report):
    """The benchmark's step at its full size: gate, then ONE dsn_layer_forward call whose five elements (QKV,
    attention core, proj, fc1-GELU, fc2) inherit one routing.  cfg5: 1024 x 197 tokens on the given quota-uniform
    routing; cfg3: 256 x 197 tokens routed by the gate inside the call.  The oracle runs the same chain, rounding
    to bf16 where the device stores bf16, on the first and last sample of every group."""
    if name == "cfg5":
        cfg, x = vit_base
    else:
        cfg = wl.config3(B=256, routing="uniform")
        x = up_bf16(cfg["x"])
    B, R, De, Dm, T, paths, Dh, H = (cfg["B"], cfg["R"], cfg["D_e"], cfg["D_mlp"], cfg["T"], cfg["paths"], cfg["D_h"],
                                     cfg["H"])
    heads = [p[1] for p in paths]
    sl = {n: wl.vit_layer_slices(paths, Dh, n) for n in ("qkv", "proj", "fc1", "fc2")}
    Wf = up_bf16(wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh))
    layers = [dsn.make_linear_desc(dsn.BF16, R, De, 3 * H * Dh, *sl["qkv"], Wf),
              dsn.make_attention_desc(R, H, Dh, heads),
              dsn.make_linear_desc(dsn.BF16, R, H * Dh, De, *sl["proj"], up_bf16(cfg["Wproj"])),
              dsn.make_linear_desc(dsn.BF16, R, De, Dm, *sl["fc1"], up_bf16(cfg["Wfc1"]), act=dsn.ACT_GELU),
              dsn.make_linear_desc(dsn.BF16, R, Dm, De, *sl["fc2"], up_bf16(cfg["Wfc2"]))]
    gate = None
    if routing == "gate":
        gW1, gW2 = up_f32(cfg["gate_W1"]), up_f32(cfg["gate_W2"])
        gate = dsn.make_gate_desc(dsn.BF16, B, R, De, gW1.shape[0], T, gW1, gW2)
    L = dsn.make_layer_desc(B, T, layers, gate)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    idx_out = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    dsn.dsn_layer_forward(ctx, L, x, None if gate is not None else up_i32(cfg["idx"]), y, ws,
                          idx_out=idx_out if gate is not None else None)
    check_status(ctx, dsn)
    if gate is not None:
        idx_gpu = idx_out.cpu().numpy()
        idx_ref, _, margin = O.gate(cfg["x"], cfg["gate_W1"], cfg["gate_W2"])
        safe = margin >= 1e-4
        np.testing.assert_array_equal(idx_gpu[safe], idx_ref[safe])
        idx = np.where(safe, idx_ref, idx_gpu).astype(np.int32)
    else:
        idx = np.asarray(cfg["idx"], np.int32)
    samples = group_samples(idx, T)[:8]
    xs, ids = cfg["x"][samples], idx[samples]
    h = O.vit_attention_half(xs, cfg["Wq"], cfg["Wk"], cfg["Wv"], cfg["Wproj"], ids, paths, Dh, mirror_bf16=True)[4]
    _, ref = O.vit_mlp(np.nan_to_num(h), cfg["Wfc1"], cfg["Wfc2"], ids, paths, mirror_bf16=True)
    sel = torch.from_numpy(np.asarray(samples, dtype=np.int64)).to(DEV)
    # Five stored bf16 tensors between input and output, and the device rounds the attention probabilities to
    # bf16 before the second product (the oracle does not): the attention core alone is held to 5e-3, and the
    # three linear layers after it carry that deviation on.  Bounds: 1.5e-2 on the largest, 1.5e-3 on the mean.
    check_samples(down(y[sel]), ref, ids, sl["fc2"][1], range(len(samples)), 1.5e-2, 1.5e-3, parity_report,
                  f"{name} ViT block chain (5 elements, 5 stored bf16 tensors), B={B} {routing}")
