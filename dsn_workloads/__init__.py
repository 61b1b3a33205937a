"""Seeded synthetic workloads for the dynamic-weight-slicing hot path.

This module only *draws inputs*: tensor shapes, slice-width tables, routing
draws and random values rounded once to the storage dtype.  It contains none
of the method's arithmetic (no gate, no grouping, no contraction), so both the
CPU oracle's tests and the CUDA path's tests may use it without sharing code.

Shapes follow the paper's models: ResNet-50 bottlenecks (routing-space table
of DS-ResNet), MobileNetV1 pointwise layers (routing-space table of DS-MBNet)
and ViT blocks (routing-space table of DS-ViT++).  Values are N(0,1) tokens or
ReLU(N(0,1)) feature maps and N(0, 1/fan_in) weights; they stand in for
ImageNet activations and trained weights, which are not available.

Seeds: ``SEED_BASE + 1000*config + ordinal`` with ordinals assigned in the
order x, layer weights, gate W1, gate W2, routing draw.
"""
from __future__ import annotations

import numpy as np
import torch

SEED_BASE = 210910060

# Literal width lists for the 14 ratios 0.35 .. 1.00 (step 0.05) at the inner
# widths of the four ResNet-50 stages, and the DS-MBNet lists from the paper's
# routing-space table.
RATIOS_14 = [0.35 + 0.05 * i for i in range(14)]
WIDTHS_14 = {
    64: [22, 26, 28, 32, 36, 38, 42, 44, 48, 52, 54, 58, 60, 64],
    128: [44, 52, 56, 64, 72, 76, 84, 88, 96, 104, 108, 116, 120, 128],
    256: [88, 104, 112, 128, 144, 152, 168, 176, 192, 208, 216, 232, 240, 256],
    512: [176, 208, 232, 256, 280, 304, 336, 360, 384, 408, 432, 464, 488, 512],
    640: list(range(224, 641, 32)),
    1152: list(range(736, 1153, 32)),
}


def rng(config: int, ordinal: int) -> np.random.Generator:
    return np.random.default_rng(SEED_BASE + 1000 * config + ordinal)


def to_bf16_values(a: np.ndarray) -> np.ndarray:
    """Round fp32 values once to bf16-representable fp32 values (library cast)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-representable fp32 values (exact, no rounding)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """fp32 values of bf16 bit patterns."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def normal(g: np.random.Generator, shape, std=1.0, relu=False, bf16=True) -> np.ndarray:
    a = (g.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)
    if relu:
        a = np.maximum(a, np.float32(0))
    return to_bf16_values(a) if bf16 else a


# ----------------------------------------------------------------------------
# routing draws (per-sample slice index); none of these is the method's gate
# ----------------------------------------------------------------------------
def idx_iid_uniform(g, B, T):
    return g.integers(0, T, size=B, dtype=np.int64).astype(np.int32)


def _quota_to_idx(g, quotas):
    idx = np.concatenate([np.full(q, t, dtype=np.int32) for t, q in enumerate(quotas)])
    g.shuffle(idx)
    return idx


def largest_remainder(total, weights):
    w = np.asarray(weights, dtype=np.float64)
    raw = total * w / w.sum()
    q = np.floor(raw).astype(np.int64)
    rem = total - int(q.sum())
    order = np.argsort(-(raw - q), kind="stable")
    for j in range(rem):
        q[order[j]] += 1
    return q.tolist()


def idx_quota_uniform(g, B, T):
    return _quota_to_idx(g, largest_remainder(B, [1.0] * T))


def idx_skewed_bands(g, B, T=14):
    """40/30/20/10 % of the batch over bands of 3,4,4,3 paths, widest band first,
    spread evenly inside a band (round-robin from the widest path)."""
    assert T == 14
    band_sizes = [3, 4, 4, 3]
    band_quota = largest_remainder(B, [0.4, 0.3, 0.2, 0.1])
    quotas = [0] * T
    path = T - 1
    for bs, bq in zip(band_sizes, band_quota):
        paths = list(range(path, path - bs, -1))
        for j in range(bq):
            quotas[paths[j % bs]] += 1
        path -= bs
    return _quota_to_idx(g, quotas)


def idx_zipf(g, B, T, s=1.2):
    """Zipf(s) quotas with rank 1 = path 0."""
    return _quota_to_idx(g, largest_remainder(B, [1.0 / (r + 1) ** s for r in range(T)]))


def idx_all_one(B, t):
    return np.full(B, t, dtype=np.int32)


# ----------------------------------------------------------------------------
# path tables
# ----------------------------------------------------------------------------
def vit_small_paths():
    """48 paths = embed {192..384} x heads {3..6} x mlp {768,1152,1536}, lexicographic."""
    paths = []
    for de in (192, 256, 320, 384):
        for h in (3, 4, 5, 6):
            for dm in (768, 1152, 1536):
                paths.append((de, h, dm))
    return paths


def vit_base_paths():
    """8 diagonal paths: t-th value of each dimension."""
    return [(320 + 64 * t, 5 + t, 1280 + 256 * t) for t in range(8)]


# ----------------------------------------------------------------------------
# configs
# ----------------------------------------------------------------------------
def config1(B=64, C=256):
    """Single dynamic sliced linear layer, fp32, gate bypassed."""
    c = 1
    widths = [C // 4, C // 2, 3 * C // 4, C]
    return dict(
        name="cfg1_linear_fp32", dtype="f32", B=B, R=1, C_in=C, C_out=C, T=4,
        k_in=widths, k_out=widths,
        x=normal(rng(c, 0), (B, 1, C), bf16=False),
        W=normal(rng(c, 1), (C, C), std=C ** -0.5, bf16=False),
        idx=idx_iid_uniform(rng(c, 4), B, 4),
    )


def bottleneck(config, B, H, Wd, C_outer, C_inner, routing="uniform", with_gate=True, C_mlp=128):
    """ResNet-50-style dynamic bottleneck: 1x1 C_outer->w, 3x3 w->w (pad 1), 1x1 w->C_outer.
    Weights use the paper's [C_O][C_I][K][K] indexing."""
    widths = WIDTHS_14[C_inner]
    T = len(widths)
    d = dict(
        name=f"bottleneck_{H}x{Wd}_{C_inner}_{C_outer}", dtype="bf16", B=B, H=H, W=Wd,
        C_outer=C_outer, C_inner=C_inner, T=T, widths=widths,
        x=normal(rng(config, 0), (B, H, Wd, C_outer), relu=True),
        W1=normal(rng(config, 1), (C_inner, C_outer, 1, 1), std=C_outer ** -0.5),
        W2=normal(rng(config, 2), (C_inner, C_inner, 3, 3), std=(9 * C_inner) ** -0.5),
        W3=normal(rng(config, 3), (C_outer, C_inner, 1, 1), std=C_inner ** -0.5),
    )
    if with_gate:
        d["gate_W1"] = normal(rng(config, 4), (C_mlp, C_outer), std=C_outer ** -0.5, bf16=False)
        d["gate_W2"] = normal(rng(config, 5), (T, C_mlp), std=C_mlp ** -0.5, bf16=False)
    g = rng(config, 6)
    if routing == "uniform":
        d["idx"] = idx_quota_uniform(g, B, T)
    elif routing == "skewed":
        d["idx"] = idx_skewed_bands(g, B, T)
    elif routing == "iid":
        d["idx"] = idx_iid_uniform(g, B, T)
    else:
        raise ValueError(routing)
    d["routing"] = routing
    return d


def config2(B=128, routing="uniform"):
    return bottleneck(2, B, 14, 14, 1024, 256, routing)


RESNET_STAGES = {1: (56, 256, 64), 2: (28, 512, 128), 3: (14, 1024, 256), 4: (7, 2048, 512)}


def config4(stage, B=256, routing="skewed"):
    hw, outer, inner = RESNET_STAGES[stage]
    return bottleneck(4 * 10 + stage, B, hw, hw, outer, inner, routing)


def vit_block(config, B, N_tok, D_e, H, D_h, D_mlp, paths, routing="uniform", C_mlp=128, zipf_s=1.2,
              one_path=0):
    """ViT block weights in [out][in] storage; Wq/Wk/Wv kept separate (the paper's form)."""
    T = len(paths)
    HD = H * D_h
    d = dict(
        name=f"vit_{D_e}_{H}h_{D_mlp}", dtype="bf16", B=B, R=N_tok, D_e=D_e, H=H, D_h=D_h, D_mlp=D_mlp,
        T=T, paths=paths,
        x=normal(rng(config, 0), (B, N_tok, D_e)),
        Wq=normal(rng(config, 1), (HD, D_e), std=D_e ** -0.5),
        Wk=normal(rng(config, 2), (HD, D_e), std=D_e ** -0.5),
        Wv=normal(rng(config, 3), (HD, D_e), std=D_e ** -0.5),
        Wproj=normal(rng(config, 4), (D_e, HD), std=HD ** -0.5),
        Wfc1=normal(rng(config, 5), (D_mlp, D_e), std=D_e ** -0.5),
        Wfc2=normal(rng(config, 6), (D_e, D_mlp), std=D_mlp ** -0.5),
        gate_W1=normal(rng(config, 7), (C_mlp, D_e), std=D_e ** -0.5, bf16=False),
        gate_W2=normal(rng(config, 8), (T, C_mlp), std=C_mlp ** -0.5, bf16=False),
    )
    g = rng(config, 9)
    if routing == "uniform":
        d["idx"] = idx_quota_uniform(g, B, T)
    elif routing == "zipf":
        d["idx"] = idx_zipf(g, B, T, zipf_s)
    elif routing == "one":
        d["idx"] = idx_all_one(B, one_path)
    elif routing == "iid":
        d["idx"] = idx_iid_uniform(g, B, T)
    elif routing == "singleton":
        d["idx"] = (np.arange(B) % T).astype(np.int32)  # group g = sample g, slice g mod T
    else:
        raise ValueError(routing)
    d["routing"] = routing
    return d


def config3(B=256, routing="uniform"):
    return vit_block(3, B, 197, 384, 6, 64, 1536, vit_small_paths(), routing)


def config5(B=1024, routing="uniform", one_path=7):
    return vit_block(5, B, 197, 768, 12, 64, 3072, vit_base_paths(), routing, one_path=one_path)


def pack_qkv_head_major(Wq, Wk, Wv, D_h):
    """Rearrange separate [H*D_h][D_e] projections into one [H][3][D_h][D_e] matrix so that
    the first h heads of q, k and v together form one leading block of 3*h*D_h rows."""
    HD, D_e = Wq.shape
    H = HD // D_h
    stack = np.stack([Wq.reshape(H, D_h, D_e), Wk.reshape(H, D_h, D_e), Wv.reshape(H, D_h, D_e)], axis=1)
    return np.ascontiguousarray(stack.reshape(3 * HD, D_e))


def vit_layer_slices(paths, D_h, layer):
    """(k_in[T], k_out[T]) of one ViT layer for a path table of (d_e, h, d_mlp) tuples."""
    if layer == "qkv":
        return [p[0] for p in paths], [3 * p[1] * D_h for p in paths]
    if layer == "proj":
        return [p[1] * D_h for p in paths], [p[0] for p in paths]
    if layer == "fc1":
        return [p[0] for p in paths], [p[2] for p in paths]
    if layer == "fc2":
        return [p[2] for p in paths], [p[0] for p in paths]
    raise ValueError(layer)


def mobilenet_pointwise(B=256, hw=14, C=640):
    """DS-MBNet pointwise 1x1 conv c_t -> c_t (supplementary workload)."""
    config = 6
    widths = WIDTHS_14[C]
    return dict(
        name=f"mbnet_pw_{hw}x{hw}_{C}", dtype="bf16", B=B, H=hw, W=hw, C=C, T=len(widths), widths=widths,
        x=normal(rng(config, 0 if C == 640 else 10), (B, hw, hw, C), relu=True),
        Wpw=normal(rng(config, 1 if C == 640 else 11), (C, C, 1, 1), std=C ** -0.5),
        idx=idx_quota_uniform(rng(config, 6), B, len(widths)),
    )


def mobilenet_block(B=256, hw=14, C=640, K=3, C_mlp=128):
    """DS-MBNet separable block (routing-space table of DS-MBNet): depthwise KxK on the c_t leading channels,
    ReLU, then pointwise 1x1 c_t -> c_t, ReLU.  Depthwise filter in the oracle's [C][K][K] indexing."""
    config = 6
    widths = WIDTHS_14[C]
    T = len(widths)
    return dict(
        name=f"mbnet_dwpw_{hw}x{hw}_{C}", dtype="bf16", B=B, H=hw, W=hw, C=C, K=K, T=T, widths=widths,
        x=normal(rng(config, 20), (B, hw, hw, C), relu=True),
        Wdw=normal(rng(config, 21), (C, K, K), std=1.0 / K),
        Wpw=normal(rng(config, 22), (C, C, 1, 1), std=C ** -0.5),
        gate_W1=normal(rng(config, 24), (C_mlp, C), std=C ** -0.5, bf16=False),
        gate_W2=normal(rng(config, 25), (T, C_mlp), std=C_mlp ** -0.5, bf16=False),
        idx=idx_quota_uniform(rng(config, 26), B, T), routing="uniform",
    )
