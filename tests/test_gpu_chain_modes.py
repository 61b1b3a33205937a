"""dsn_layer_forward runs a small-batch chain of sliced layers as one launch (every CTA pair owns
whole samples and walks the layers itself); larger batches, and every batch with DSN_CHAIN=0 (read
when a context is created), run one launch per layer.  The parity tests of the chained layers in
this process use the default; here they run once more in a child process with chaining off, and the
two modes are compared with each other on one bottleneck."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_layer_forward_parity_with_one_launch_per_layer():
    env = dict(os.environ, DSN_CHAIN="0")
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_conv_layer.py"), "-k", "layer_forward"]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout


_CHILD = r"""
import sys, numpy as np, torch
sys.path.insert(0, {root!r})
import paper_2109_10060_b200 as dsn
import dsn_workloads as wl
dev = torch.device("cuda:0")
cfg = wl.config2(B=40)
B, H, Wd, C, Ci, T, widths = cfg["B"], cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"], cfg["widths"]
up = lambda a: torch.from_numpy(wl.bf16_bits(np.ascontiguousarray(a)).view(np.int16)).to(dev).view(torch.bfloat16)
x = up(cfg["x"]); W1 = up(cfg["W1"].reshape(Ci, C)); W2 = up(np.transpose(cfg["W2"], (0, 2, 3, 1))); W3 = up(cfg["W3"].reshape(C, Ci))
ctx = dsn.Context(0)
full = [C] * T
layers = [dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, Ci, full, widths, W1, act=dsn.ACT_RELU),
          dsn.make_conv_desc(dsn.BF16, H, Wd, 3, 1, Ci, Ci, widths, widths, W2, act=dsn.ACT_RELU),
          dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, Ci, C, widths, full, W3)]
L = dsn.make_layer_desc(B, T, layers, None)
ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=dev)
y = torch.zeros(B, H, Wd, C, dtype=torch.bfloat16, device=dev)
idx = torch.from_numpy(cfg["idx"]).to(dev)
dsn.dsn_layer_forward(ctx, L, x, idx, y, ws)
code, detail = ctx.get_status()
assert code == 0, (code, detail)
np.save(sys.argv[1], y.view(torch.int16).cpu().numpy())
"""


def test_chained_and_unchained_outputs_agree(tmp_path):
    """The 1x1 layers run the same arithmetic in both modes.  The 3x3 layer does not sum in the same
    order (the chained launch walks taps then channel chunks, the single-layer launch stages a chunk
    with its halo and walks the taps inside it), so fp32 sums differ in the last bits and a few bf16
    results land on the other side of a rounding boundary: the outputs must agree like two correct
    evaluations of a three-layer chain do (one output ulp at most, rarely)."""
    outs = []
    for mode in ("1", "0"):
        path = str(tmp_path / f"y_{mode}.npy")
        env = dict(os.environ, DSN_CHAIN=mode)
        res = subprocess.run([sys.executable, "-c", _CHILD.format(root=ROOT), path], cwd=ROOT, env=env,
                             capture_output=True, text=True, timeout=600)
        assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-3000:]
        bits = np.load(path).astype(np.uint16).astype(np.uint32) << 16
        outs.append(bits.view(np.float32).astype(np.float64))
    a, b = outs
    scale = np.max(np.abs(a))
    assert np.max(np.abs(a - b)) <= 1e-2 * scale
    assert np.mean(np.abs(a - b)) <= 2e-4 * scale
    assert np.mean(a != b) <= 0.05


# ------------------------------------------------------------------------------------------------
# Edge cases of the chained launch against the oracle: batch sizes around the limits of the sample
# hand-out (one sample, an odd count, exactly two per CTA pair, one more than that, which runs one
# launch per layer), slice widths that are no multiple of 8, every sample on one path, and samples
# whose index is out of range (they belong to no group; their output rows stay untouched).
import torch  # noqa: E402

import dsn_workloads as wl  # noqa: E402
from oracle import dsn_oracle as O  # noqa: E402
from gpu_util import DEV, SENTINEL, down, group_errors, up_bf16, up_i32  # noqa: E402


def _small_bottleneck(dsn, ctx, B, idx, seed=77):
    cfg = wl.bottleneck(seed, B, 14, 14, 256, 64, routing="uniform", with_gate=False)   # inner widths 22 .. 64
    H, Wd, C, Ci, T, widths = cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"], cfg["widths"]
    full = [C] * T
    W2 = np.ascontiguousarray(np.transpose(cfg["W2"], (0, 2, 3, 1)))
    layers = [dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, Ci, full, widths, up_bf16(cfg["W1"].reshape(Ci, C)), act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 3, 1, Ci, Ci, widths, widths, up_bf16(W2), act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, Ci, C, widths, full, up_bf16(cfg["W3"].reshape(C, Ci)))]
    L = dsn.make_layer_desc(B, T, layers, None)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, H, Wd, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_layer_forward(ctx, L, up_bf16(cfg["x"]), up_i32(idx), y, ws)
    return cfg, down(y)


@pytest.mark.parametrize("B,routing", [(1, "uniform"), (2, "uniform"), (75, "uniform"), (148, "uniform"), (149, "uniform"),
                                       (37, "one_path"), (60, "some_invalid"), (9, "all_invalid")])
def test_chained_bottleneck_edge_batches(dsn, B, routing):
    ctx = dsn.Context(0)
    T = 14
    if routing == "one_path":
        idx = np.full(B, 5, dtype=np.int32)
    else:
        idx = wl.idx_quota_uniform(wl.rng(77, 6), B, T)
    if routing == "some_invalid":
        idx = idx.copy()
        idx[::7] = -1
        idx[3::11] = T
    if routing == "all_invalid":
        idx = np.full(B, T + 3, dtype=np.int32)
    cfg, got = _small_bottleneck(dsn, ctx, B, idx)
    code, detail = ctx.get_status()
    valid = (idx >= 0) & (idx < T)
    if routing in ("some_invalid", "all_invalid"):
        assert code == dsn.ERR_BAD_INDEX and detail == int(np.sum(~valid))   # reported, not fatal
        assert np.all(got[~valid] == SENTINEL)                                # rows of unrouted samples untouched
    else:
        assert code == 0, (code, detail)
    sel = np.nonzero(valid)[0]
    if len(sel) == 0:
        return
    _, _, ref = O.bottleneck(cfg["x"][sel], cfg["W1"], cfg["W2"], cfg["W3"], idx[sel], cfg["widths"], mirror_bf16=True)
    errs = group_errors(got[sel], ref, idx[sel], [cfg["C_outer"]] * T, T)
    assert max(errs.values()) <= 1e-2, errs


def _context_with(dsn, **switches):
    """A context created while the given environment switches hold (they are read at creation only)."""
    saved = {k: os.environ.get(k) for k in switches}
    os.environ.update(switches)
    try:
        return dsn.Context(0)
    finally:
        for k, v in saved.items():
            if v is None:
                del os.environ[k]
            else:
                os.environ[k] = v


@pytest.mark.parametrize("B,with_skip,C_outer,C_inner", [(37, False, 256, 64), (37, True, 256, 64), (148, False, 256, 64),
                                                         (3, True, 256, 64), (21, False, 1024, 256)],
                         ids=["plain", "skip-features", "two-per-pair", "tiny", "wide"])
def test_bottleneck_last_layer_fed_from_tensor_memory(dsn, B, with_skip, C_outer, C_inner, parity_report):
    """DSN_CHAIN_FUSE=1: in the chained launch the 3x3 layer's output tile is converted in place in tensor memory and the
    last 1x1 layer takes it from there as its A operand (nothing of it is stored or loaded).  Same bottleneck, same
    oracle chain and same bound as the default form; the launch counter shows that the form ran."""
    ctx = _context_with(dsn, DSN_CHAIN="1", DSN_CHAIN_FUSE="1")
    cfg = wl.bottleneck(79, B, 14, 14, C_outer, C_inner, routing="uniform", with_gate=False)
    H, Wd, C, Ci, T, widths, idx = cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"], cfg["widths"], cfg["idx"]
    full = [C] * T
    x = up_bf16(cfg["x"])
    W2 = np.ascontiguousarray(np.transpose(cfg["W2"], (0, 2, 3, 1)))
    layers = [dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, Ci, full, widths, up_bf16(cfg["W1"].reshape(Ci, C)), act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 3, 1, Ci, Ci, widths, widths, up_bf16(W2), act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, Ci, C, widths, full, up_bf16(cfg["W3"].reshape(C, Ci)),
                                 act=dsn.ACT_RELU if with_skip else dsn.ACT_NONE, residual=x if with_skip else None)]
    L = dsn.make_layer_desc(B, T, layers, None)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, H, Wd, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    before = ctx.stats()
    dsn.dsn_layer_forward(ctx, L, x, up_i32(idx), y, ws)
    code, detail = ctx.get_status()
    assert code == 0, (code, detail)
    after = ctx.stats()
    assert after["launches_gemm_chain_tmem"] - before["launches_gemm_chain_tmem"] == 1
    y1 = O.round_bf16(O.sliced_conv(cfg["x"], cfg["W1"], idx, full, widths, 0, act=O.ACT_RELU, fill=0.0))
    y2 = O.round_bf16(O.sliced_conv(y1, cfg["W2"], idx, widths, widths, 1, act=O.ACT_RELU, fill=0.0))
    ref = O.sliced_conv(y2, cfg["W3"], idx, widths, full, 0, act=O.ACT_RELU if with_skip else O.ACT_NONE,
                        residual=cfg["x"] if with_skip else None)
    errs = group_errors(down(y), ref, idx, full, T)
    assert max(errs.values()) <= 1e-2, errs
    parity_report.append(f"bottleneck, last layer fed from tensor memory, B={B}{' with skip features' if with_skip else ''}: "
                         f"worst {max(errs.values()):.2e} (chain bound 1e-02)")


@pytest.mark.parametrize("B,chained", [(37, True), (37, False), (160, True)], ids=["chained", "per-layer", "large-batch"])
def test_bottleneck_with_identity_shortcut(dsn, B, chained, parity_report):
    """The residual tail of a DS-ResNet block (Sec. 5) inside dsn_layer_forward: out = ReLU(conv3(h) + x) with the block
    input itself as skip features.  Small batches run the three layers as one chained launch, which adds the skip
    features in its last layer's epilogue; with DSN_CHAIN=0, and for batches beyond two samples per CTA pair, one
    launch per layer.  All three against the oracle's chain (each stored tensor rounded to bf16)."""
    saved = os.environ.get("DSN_CHAIN")
    os.environ["DSN_CHAIN"] = "1" if chained else "0"       # read when the context is created
    try:
        ctx = dsn.Context(0)
    finally:
        if saved is None:
            del os.environ["DSN_CHAIN"]
        else:
            os.environ["DSN_CHAIN"] = saved
    cfg = wl.bottleneck(78, B, 14, 14, 256, 64, routing="uniform", with_gate=False)
    H, Wd, C, Ci, T, widths, idx = cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"], cfg["widths"], cfg["idx"]
    full = [C] * T
    x = up_bf16(cfg["x"])
    W2 = np.ascontiguousarray(np.transpose(cfg["W2"], (0, 2, 3, 1)))
    layers = [dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, Ci, full, widths, up_bf16(cfg["W1"].reshape(Ci, C)), act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 3, 1, Ci, Ci, widths, widths, up_bf16(W2), act=dsn.ACT_RELU),
              dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, Ci, C, widths, full, up_bf16(cfg["W3"].reshape(C, Ci)), act=dsn.ACT_RELU,
                                 residual=x)]
    L = dsn.make_layer_desc(B, T, layers, None)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, H, Wd, C), SENTINEL, dtype=torch.bfloat16, device=DEV)
    before = ctx.stats()
    dsn.dsn_layer_forward(ctx, L, x, up_i32(idx), y, ws)
    code, detail = ctx.get_status()
    assert code == 0, (code, detail)
    after = ctx.stats()
    if chained and B <= 148:
        assert after["launches_gemm_chain"] - before["launches_gemm_chain"] == 1     # the block ran as one launch
    else:
        assert after["launches_gemm_chain"] == before["launches_gemm_chain"]
    y1 = O.round_bf16(O.sliced_conv(cfg["x"], cfg["W1"], idx, full, widths, 0, act=O.ACT_RELU, fill=0.0))
    y2 = O.round_bf16(O.sliced_conv(y1, cfg["W2"], idx, widths, widths, 1, act=O.ACT_RELU, fill=0.0))
    ref = O.sliced_conv(y2, cfg["W3"], idx, widths, full, 0, act=O.ACT_RELU, residual=cfg["x"])
    errs = group_errors(down(y), ref, idx, full, T)
    assert max(errs.values()) <= 1e-2, errs
    parity_report.append(f"bottleneck with identity shortcut, B={B} ({'chained launch' if chained and B <= 148 else 'one launch per layer'}): "
                         f"worst {max(errs.values()):.2e} (chain bound 1e-02)")
