"""GPU parity of the slimmable self-attention core against the CPU oracle."""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O
from gpu_util import DEV, SENTINEL, check_status, down, route_on_gpu, up_bf16

pytestmark = pytest.mark.gpu
TOL = 5e-3   # max|err| / max|ref| per sample; probabilities are rounded to bf16 before the second product


@pytest.fixture(scope="module")
def ctx(dsn):
    return dsn.Context(0)


def head_major(q, k, v, H, Dh):
    """[B][N][H*Dh] x3 -> [B][N][H][3][Dh] flattened: the fused QKV layer's output layout."""
    B, N, _ = q.shape
    st = np.stack([q.reshape(B, N, H, Dh), k.reshape(B, N, H, Dh), v.reshape(B, N, H, Dh)], axis=3)
    return np.ascontiguousarray(st.reshape(B, N, 3 * H * Dh))


@pytest.mark.parametrize("B,N,H,heads,order", [(24, 197, 6, [3, 4, 5, 6], 0), (24, 197, 6, [3, 4, 5, 6], 1),
                                               (10, 197, 12, [5, 6, 7, 8, 9, 10, 11, 12], 1), (6, 64, 4, [1, 4], 0),
                                               (5, 256, 2, [2, 1], 1), (7, 130, 3, [3], 0), (4, 16, 2, [2, 1], 0),
                                               # more (sample, head, half) items than resident CTAs: several per CTA
                                               (96, 197, 6, [3, 4, 5, 6], 0), (96, 197, 6, [3, 4, 5, 6], 1),
                                               (200, 100, 3, [1, 2, 3], 1)])
def test_attention_matches_oracle(dsn, ctx, B, N, H, heads, order):
    g = np.random.default_rng(B * 1000 + N + H)
    Dh, T = 64, len(heads)
    idx = g.integers(0, T, size=B).astype(np.int32)
    q, k, v = (wl.normal(g, (B, N, H * Dh)) for _ in range(3))
    q = wl.to_bf16_values(q * 1.5)                      # sharper softmax than unit-variance scores
    qkv = head_major(q, k, v, H, Dh)
    r = route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2]
    src = qkv[perm] if order else qkv
    out = torch.full((B, N, H * Dh), SENTINEL, dtype=torch.bfloat16, device=DEV)
    d = dsn.make_attention_desc(N, H, Dh, heads, order=order)
    dsn.dsn_sliced_attention(ctx, d, r, up_bf16(src), out)
    check_status(ctx, dsn)
    got = down(out)
    if order:
        tmp = np.empty_like(got)
        tmp[perm] = got
        got = tmp
    ref = O.attention(q, k, v, idx, heads, Dh)
    for i in range(B):
        w = heads[idx[i]] * Dh
        err = np.max(np.abs(got[i, :, :w] - ref[i, :, :w])) / np.max(np.abs(ref[i, :, :w]))
        assert err <= TOL, (i, int(idx[i]), err)
        assert np.all(got[i, :, w:] == SENTINEL)          # heads the path does not have stay untouched


def test_attention_more_groups_than_the_item_table_holds(dsn, ctx):
    """Caller-built list of 70 one-sample groups (slice g mod T): the one-CTA-per-item form of the kernel."""
    B, N, H, Dh, heads = 70, 197, 4, 64, [2, 4, 3]
    g = np.random.default_rng(11)
    T = len(heads)
    order = g.permutation(B).astype(np.int32)             # group j holds sample order[j]
    idx = (np.arange(B) % T).astype(np.int32)
    slices = idx[order]
    inv = np.empty(B, np.int32)
    inv[order] = np.arange(B, dtype=np.int32)
    q, k, v = (wl.normal(g, (B, N, H * Dh)) for _ in range(3))
    bufs = [torch.from_numpy(a.astype(np.int32)).to(DEV) for a in (np.ones(B), np.arange(B + 1), order, inv, slices)]
    r = dsn.make_routing(B, B, *bufs)
    out = torch.full((B, N, H * Dh), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_attention(ctx, dsn.make_attention_desc(N, H, Dh, heads, order=0), r,
                             up_bf16(head_major(q, k, v, H, Dh)), out)
    check_status(ctx, dsn)
    got = down(out)
    ref = O.attention(q, k, v, idx, heads, Dh)
    for i in range(B):
        w = heads[idx[i]] * Dh
        err = np.max(np.abs(got[i, :, :w] - ref[i, :, :w])) / np.max(np.abs(ref[i, :, :w]))
        assert err <= TOL, (i, int(idx[i]), err)
        assert np.all(got[i, :, w:] == SENTINEL)


def test_attention_full_size_vit_small_sampled(dsn, ctx):
    """The ViT-S style configuration at its full size (256 samples, 48 paths, grouped order, as the per-layer
    benchmark launches it): every CTA works several items.  The oracle is evaluated on a spread of samples."""
    B, N, H, Dh = 256, 197, 6, 64
    heads = [p_[1] for p_ in wl.vit_small_paths()]
    T = len(heads)
    idx = np.asarray(wl.idx_quota_uniform(wl.rng(3, 9), B, T), np.int32)
    g = np.random.default_rng(77)
    q, k, v = (wl.to_bf16_values(wl.normal(g, (B, N, H * Dh))) for _ in range(3))
    r = route_on_gpu(dsn, ctx, idx, T)
    perm = O.route(idx, T)[2]
    out = torch.full((B, N, H * Dh), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_attention(ctx, dsn.make_attention_desc(N, H, Dh, heads, order=dsn.GROUPED), r,
                             up_bf16(head_major(q, k, v, H, Dh)[perm]), out)
    check_status(ctx, dsn)
    got = np.empty((B, N, H * Dh), np.float32)
    got[perm] = down(out)
    sel = np.unique(np.concatenate([[0, 1, B // 2, B - 2, B - 1], g.integers(0, B, size=11)]))
    ref = O.attention(q[sel], k[sel], v[sel], idx[sel], heads, Dh)
    for j, i in enumerate(sel):
        w = heads[idx[i]] * Dh
        err = np.max(np.abs(got[i, :, :w] - ref[j, :, :w])) / np.max(np.abs(ref[j, :, :w]))
        assert err <= TOL, (int(i), int(idx[i]), err)
    for i in range(B):                                    # every sample: written where it has heads, untouched beyond
        w = heads[idx[i]] * Dh
        assert np.all(got[i, :, w:] == SENTINEL)
        assert np.all(got[i, :, :w] != SENTINEL)


def test_attention_full_size_vit_base_sampled(dsn, ctx, parity_report):
    """The serving-scale configuration at its full size: 1024 samples x 197 tokens, 12 heads of which a path uses
    5..12, quota-uniform routing over the 8 paths, grouped order, row pitch 2304 (what the QKV layer of the
    benchmark step hands over).  The batch tiles a block of 64 seeded samples; the oracle evaluates the first and
    last sample of every group."""
    B, N, H, Dh, blk = 1024, 197, 12, 64, 64
    heads = [p_[1] for p_ in wl.vit_base_paths()]
    T = len(heads)
    idx = np.asarray(wl.idx_quota_uniform(wl.rng(5, 9), B, T), np.int32)
    g = np.random.default_rng(55)
    q, k, v = (wl.to_bf16_values(wl.normal(g, (blk, N, H * Dh))) for _ in range(3))
    block = up_bf16(head_major(q, k, v, H, Dh))                 # [64][N][3*H*Dh]
    counts, offsets, perm, inv = O.route(idx, T)
    r = route_on_gpu(dsn, ctx, idx, T)
    src = block[torch.from_numpy((perm % blk).astype(np.int64)).to(DEV)]      # grouped: position p holds sample perm[p]
    out = torch.full((B, N, H * Dh), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_attention(ctx, dsn.make_attention_desc(N, H, Dh, heads, order=dsn.GROUPED), r, src, out)
    check_status(ctx, dsn)
    sel = sorted({int(perm[offsets[t]]) for t in range(T) if counts[t]} | {int(perm[offsets[t + 1] - 1]) for t in range(T) if counts[t]})
    src_of = [i % blk for i in sel]
    ref = O.attention(q[src_of], k[src_of], v[src_of], idx[sel], heads, Dh)
    got = down(out[torch.from_numpy(inv[sel].astype(np.int64)).to(DEV)])
    worst = 0.0
    for j, i in enumerate(sel):
        w = heads[idx[i]] * Dh
        err = np.max(np.abs(got[j, :, :w] - ref[j, :, :w])) / np.max(np.abs(ref[j, :, :w]))
        worst = max(worst, err)
        assert err <= TOL, (int(i), int(idx[i]), err)
        assert np.all(got[j, :, w:] == SENTINEL)
    parity_report.append(f"cfg5 attention core alone, B=1024, 5..12 heads: worst {worst:.2e} over {len(sel)} samples (bound {TOL:.0e})")
    written = (out[:, 0, ::Dh] != SENTINEL).sum(dim=1).cpu().numpy()          # heads written per grouped position
    np.testing.assert_array_equal(written, np.asarray(heads)[idx[perm]])


def test_attention_closed_forms_on_device(dsn, ctx):
    """Zero queries -> every output row is the mean of the values; a dominant key copies its value."""
    B, N, H, Dh = 2, 197, 2, 64
    g = np.random.default_rng(3)
    v = wl.normal(g, (B, N, H * Dh))
    k = wl.normal(g, (B, N, H * Dh))
    q = np.zeros((B, N, H * Dh), np.float32)
    k[1] = 0.0
    k[1, 100] = 8.0                                       # with q = 8: score 64*64/8 = 512 above all others
    q[1] = 8.0
    r = route_on_gpu(dsn, ctx, np.zeros(B, np.int32), 1)
    out = torch.zeros((B, N, H * Dh), dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_attention(ctx, dsn.make_attention_desc(N, H, Dh, [H]), r, up_bf16(head_major(q, k, v, H, Dh)), out)
    check_status(ctx, dsn)
    got = down(out)
    mean = v[0].astype(np.float64).mean(axis=0)
    assert np.max(np.abs(got[0] - mean)) <= 5e-3
    np.testing.assert_array_equal(got[1], np.broadcast_to(v[1, 100].astype(np.float64), (N, H * Dh)))


def test_vit_block_qkv_attention_proj_chain(dsn, ctx):
    """QKV layer -> attention -> projection in grouped order with one routing: the path through a ViT
    block's attention half, against the oracle evaluated on the device's own QKV output."""
    cfg = wl.config3(B=32, routing="iid")
    B, R, De, H, Dh, T, paths = cfg["B"], cfg["R"], cfg["D_e"], cfg["H"], cfg["D_h"], cfg["T"], cfg["paths"]
    heads = [p[1] for p in paths]
    r = route_on_gpu(dsn, ctx, cfg["idx"], T)
    kq, koq = wl.vit_layer_slices(paths, Dh, "qkv")
    kp, kop = wl.vit_layer_slices(paths, Dh, "proj")
    Wf = up_bf16(wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh))
    qkv = torch.zeros((B, R, 3 * H * Dh), dtype=torch.bfloat16, device=DEV)
    att = torch.zeros((B, R, H * Dh), dtype=torch.bfloat16, device=DEV)
    y = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, De, 3 * H * Dh, kq, koq, Wf, out_order=dsn.GROUPED), r,
                          up_bf16(cfg["x"]), qkv)
    dsn.dsn_sliced_attention(ctx, dsn.make_attention_desc(R, H, Dh, heads, order=dsn.GROUPED), r, qkv, att)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, H * Dh, De, kp, kop, up_bf16(cfg["Wproj"]),
                                                    in_order=dsn.GROUPED), r, att, y)
    check_status(ctx, dsn)
    perm = O.route(cfg["idx"], T)[2]
    qkv_in = np.empty((B, R, 3 * H * Dh))
    qkv_in[perm] = down(qkv)                                    # device QKV, back in input order
    five = qkv_in.reshape(B, R, H, 3, Dh)
    q, k, v = (np.nan_to_num(five[:, :, :, w].reshape(B, R, H * Dh)) for w in range(3))
    a_ref = O.round_bf16(O.attention(q, k, v, cfg["idx"], heads, Dh, fill=0.0))
    ref = O.round_bf16(O.sliced_linear(a_ref, cfg["Wproj"], cfg["idx"], kp, kop))
    got = down(y)
    for i in range(B):
        w = kop[cfg["idx"][i]]
        err = np.max(np.abs(got[i, :, :w] - ref[i, :, :w])) / np.max(np.abs(ref[i, :, :w]))
        assert err <= 1e-2, (i, err)                            # two chained bf16 stages after the QKV layer
        assert np.all(got[i, :, w:] == SENTINEL)


def test_layer_forward_gate_qkv_attention_proj(dsn, ctx):
    """The attention half of a ViT block as one dsn_layer_forward call: gate -> route -> QKV -> attention ->
    proj -> input order, against the same chain made of separate calls."""
    from gpu_util import up_f32
    cfg = wl.config3(B=40, routing="iid")
    B, R, De, H, Dh, T, paths = cfg["B"], cfg["R"], cfg["D_e"], cfg["H"], cfg["D_h"], cfg["T"], cfg["paths"]
    heads = [p[1] for p in paths]
    kq, koq = wl.vit_layer_slices(paths, Dh, "qkv")
    kp, kop = wl.vit_layer_slices(paths, Dh, "proj")
    Wf = up_bf16(wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh))
    Wp = up_bf16(cfg["Wproj"])
    x = up_bf16(cfg["x"])
    gW1, gW2 = up_f32(cfg["gate_W1"]), up_f32(cfg["gate_W2"])
    gate = dsn.make_gate_desc(dsn.BF16, B, R, De, gW1.shape[0], T, gW1, gW2)
    layers = [dsn.make_linear_desc(dsn.BF16, R, De, 3 * H * Dh, kq, koq, Wf),
              dsn.make_attention_desc(R, H, Dh, heads),
              dsn.make_linear_desc(dsn.BF16, R, H * Dh, De, kp, kop, Wp)]
    L = dsn.make_layer_desc(B, T, layers, gate)
    ws = torch.empty(dsn.dsn_layer_workspace_bytes(L), dtype=torch.uint8, device=DEV)
    y = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    idx_out = torch.zeros(B, dtype=torch.int32, device=DEV)
    dsn.dsn_layer_forward(ctx, L, x, None, y, ws, idx_out=idx_out)
    check_status(ctx, dsn)
    idx = idx_out.cpu().numpy()
    # separate calls with the same routing
    r = route_on_gpu(dsn, ctx, idx, T)
    qkv = torch.zeros((B, R, 3 * H * Dh), dtype=torch.bfloat16, device=DEV)
    att = torch.zeros((B, R, H * Dh), dtype=torch.bfloat16, device=DEV)
    y2 = torch.full((B, R, De), SENTINEL, dtype=torch.bfloat16, device=DEV)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, De, 3 * H * Dh, kq, koq, Wf, out_order=dsn.GROUPED), r, x, qkv)
    dsn.dsn_sliced_attention(ctx, dsn.make_attention_desc(R, H, Dh, heads, order=dsn.GROUPED), r, qkv, att)
    dsn.dsn_sliced_linear(ctx, dsn.make_linear_desc(dsn.BF16, R, H * Dh, De, kp, kop, Wp, in_order=dsn.GROUPED), r, att, y2)
    check_status(ctx, dsn)
    assert torch.equal(y, y2)
    # and against the oracle end to end (three bf16 stages: chain tolerance)
    q, k, v = O.vit_qkv(cfg["x"], cfg["Wq"], cfg["Wk"], cfg["Wv"], idx, paths, Dh)
    q, k, v = (O.round_bf16(np.nan_to_num(a)) for a in (q, k, v))
    a_ref = O.round_bf16(O.attention(q, k, v, idx, heads, Dh, fill=0.0))
    ref = O.round_bf16(O.sliced_linear(a_ref, cfg["Wproj"], idx, kp, kop))
    got = down(y)
    for i in range(B):
        w = kop[idx[i]]
        err = np.max(np.abs(got[i, :, :w] - ref[i, :, :w])) / np.max(np.abs(ref[i, :, :w]))
        assert err <= 1e-2, (i, err)
