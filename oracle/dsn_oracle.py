"""CPU fp64 oracle for the dynamic-weight-slicing inference path (TEST INFRASTRUCTURE).

This file is the checker, not the product: only the tests, the smoke check and
the benchmark's CPU-baseline leg may import it.  It shares no code with the
CUDA library and never imports it.

Every function evaluates the paper's per-sample definition directly, sample by
sample in input order, in float64, with no grouping, permutation of data,
tiling or fusion.  A numpy matmul serves as the contraction step.

Passages followed (DS-Net++, "Dynamic Weight Slicing"):
  * dynamic network = route picked per input .......... Eq. (dyn_net), Sec. 3.1
  * weight slicing  psi(x) = W[:k] x ................... Eq. (weight_slicing), Sec. 3.2
  * slice-able convolution W[:c_O, :c_I] * X ........... Sec. 3.3, "Filter number"
  * slice-able depthwise conv, kernel-size slicing ..... Sec. 3.3, "Group number ...", "Kernel size"
  * ViT QKV / proj / MLP slicing, self-attention ....... Sec. 3.4, Eq. (slimmableMLP)
  * gate: average-pool encoder, two-layer MLP, one-hot . Sec. 3.5
  * gate attention head X * (1 + tanh(W3 ReLU(W1 X_E))) . Sec. 3.5, "double-headed dynamic gate"
  * split batch norm with re-calibration (Re-SBN) ...... Sec. 3.3
  * on-the-fly multiply-add count ...................... Sec. 4.3 "Complexity penalty"

Readings where the paper is silent (each is listed in the design notes):
  gate hidden activation = ReLU; inference routing = argmax of the scores
  (softmax is monotone), lowest index wins ties; convolution = cross-correlation
  with zero padding, stride 1; weights stored [out][in]; batch grouping = stable
  ordering by path index.

Parity status: `widths_from_ratios` is a convention ("parity unpinned" beyond the
paper's own DS-MBNet list); all other functions are pinned by tests/test_oracle_*.py.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

F64 = np.float64

ACT_NONE, ACT_RELU, ACT_GELU = 0, 1, 2


# --------------------------------------------------------------------------- helpers
def round_bf16(a):
    """Round float64 values to the nearest bfloat16 value (ties to even), returned as float64.

    bfloat16 keeps the sign, the 8 exponent bits and the top 7 mantissa bits of binary32.
    The value is first rounded to binary32, then to bfloat16, which is the order in which a
    device that accumulates in binary32 and stores bfloat16 rounds.
    """
    f = np.asarray(a, dtype=F64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    out = r.astype(np.uint32).view(np.float32).astype(F64)
    nan = np.isnan(f)
    if np.any(nan):
        out = np.where(nan, np.nan, out)
    return out.reshape(np.shape(a))


def activation(z, act):
    if act == ACT_NONE:
        return z
    if act == ACT_RELU:
        return np.maximum(z, 0.0)
    if act == ACT_GELU:  # exact erf form
        return 0.5 * z * (1.0 + _erf(z / np.sqrt(2.0)))
    raise ValueError(f"unknown activation {act}")


def widths_from_ratios(C, ratios, granule=0):
    """Ratio -> channel count: k = g * floor(r*C/g + 1/2) clamped to [g, C], g = min(8, C/32)
    unless given.  Reproduces the paper's DS-MBNet list 224..640 step 32 at C = 640."""
    g = granule if granule > 0 else max(1, min(8, C // 32))
    out = []
    for r in ratios:
        k = g * int(np.floor(r * C / g + 0.5 + 1e-9))
        out.append(int(min(max(k, g), C)))
    return out


# --------------------------------------------------------------------------- gate (Sec. 3.5)
def gate(x, W1, W2, b1=None, b2=None, c_valid=None):
    """Routing head of the gate.

    x  [B][R][C]   feature map flattened over its R = H*W positions (or tokens)
    W1 [C_mlp][C]  W2 [T][C_mlp]; optional biases.
    Returns idx[B] (int32, first index attaining the maximum score), scores[B][T], margin[B]
    (top-1 minus top-2 score; +inf when T == 1).
    """
    x = np.asarray(x, dtype=F64)
    W1 = np.asarray(W1, dtype=F64)
    W2 = np.asarray(W2, dtype=F64)
    B, R, C = x.shape
    cv = C if c_valid is None else int(c_valid)
    T = W2.shape[0]
    idx = np.zeros(B, dtype=np.int32)
    scores = np.zeros((B, T), dtype=F64)
    margin = np.zeros(B, dtype=F64)
    for i in range(B):
        pooled = x[i, :, :cv].sum(axis=0) / R              # average over positions
        hid = W1[:, :cv] @ pooled
        if b1 is not None:
            hid = hid + np.asarray(b1, dtype=F64)
        hid = np.maximum(hid, 0.0)
        s = W2 @ hid
        if b2 is not None:
            s = s + np.asarray(b2, dtype=F64)
        best = 0
        for t in range(1, T):                              # ascending scan, strict >
            if s[t] > s[best]:
                best = t
        idx[i] = best
        scores[i] = s
        if T > 1:
            others = np.delete(s, best)
            margin[i] = s[best] - others.max()
        else:
            margin[i] = np.inf
    return idx, scores, margin


def gate_attention(x, W1, W3, b1=None, b3=None, c_valid=None):
    """Channel-attention head of the double-headed gate (Sec. 3.5): it shares W1 with the routing head.

    scale[i][c] = 1 + tanh(b3[c] + sum_j W3[c][j] * ReLU(b1[j] + sum_c' W1[j][c'] * pooled[i][c']))
    x_hat[i][r][c] = x[i][r][c] * scale[i][c]          for c < c_valid
    x [B][R][C], W1 [C_mlp][C], W3 [C][C_mlp].  Returns (scale [B][c_valid], x_hat [B][R][c_valid]).
    """
    x = np.asarray(x, dtype=F64)
    W1 = np.asarray(W1, dtype=F64)
    W3 = np.asarray(W3, dtype=F64)
    B, R, C = x.shape
    cv = C if c_valid is None else int(c_valid)
    scale = np.zeros((B, cv), dtype=F64)
    for i in range(B):
        pooled = x[i, :, :cv].sum(axis=0) / R
        hid = W1[:, :cv] @ pooled
        if b1 is not None:
            hid = hid + np.asarray(b1, dtype=F64)
        hid = np.maximum(hid, 0.0)
        a = W3[:cv] @ hid
        if b3 is not None:
            a = a + np.asarray(b3, dtype=F64)[:cv]
        scale[i] = 1.0 + np.tanh(a)
    return scale, x[:, :, :cv] * scale[:, None, :]


# --------------------------------------------------------------------------- routing
def route(idx, T):
    """Group samples by path index, defined by enumeration.

    counts[t]  = number of samples with idx == t
    offsets    = exclusive prefix sum of counts (length T+1)
    perm       = for t = 0..T-1 in turn, the ascending list of samples with idx == t;
                 perm[p] = i means grouped position p holds sample i
    inv_perm[perm[p]] = p
    """
    idx = np.asarray(idx)
    B = idx.shape[0]
    if B and (idx.min() < 0 or idx.max() >= T):
        raise ValueError("routing index outside [0, T)")
    counts = np.zeros(T, dtype=np.int32)
    offsets = np.zeros(T + 1, dtype=np.int32)
    perm_list = []
    for t in range(T):
        members = [i for i in range(B) if idx[i] == t]
        counts[t] = len(members)
        offsets[t + 1] = offsets[t] + counts[t]
        perm_list.extend(members)
    perm = np.asarray(perm_list, dtype=np.int32).reshape(B)
    inv_perm = np.zeros(B, dtype=np.int32)
    for p in range(B):
        inv_perm[perm[p]] = p
    return counts, offsets, perm, inv_perm


# --------------------------------------------------------------------------- sliced layers
def split_bn(z, t, gamma, beta, mu, sigma):
    """Re-SBN for an input of route t with c = z.shape[-1] channels (Sec. 3.3):
    gamma[:c] * (z - mu_t[:c]) / sigma_t[:c] + beta[:c]; mu, sigma are [T][C] per-route statistics."""
    c = z.shape[-1]
    g, b = np.asarray(gamma, dtype=F64)[:c], np.asarray(beta, dtype=F64)[:c]
    m, s = np.asarray(mu, dtype=F64)[t, :c], np.asarray(sigma, dtype=F64)[t, :c]
    return g * ((z - m) / s) + b


def sliced_linear(x, W, idx, k_in, k_out, bias=None, act=ACT_NONE, fill=np.nan, samples=None, bn=None, residual=None):
    """y[i][r][o] = act(b[o] + sum_{c<k_in[t]} x[i][r][c] W[o][c]),  o < k_out[t],  t = idx[i].

    bn = (gamma[C_out], beta[C_out], mu[T][C_out], sigma[T][C_out]) inserts Re-SBN between the
    contraction (+ bias) and the activation; residual [B][R][C_out] (the skip features of a residual block,
    Sec. 5 "DS-ResNet": shortcut and residual output have the same sliced width) is added just before the
    activation.
    x [B][R][C_in], W [C_out][C_in] (stored [out][in]).  Entries with o >= k_out[t] are not part
    of the result and hold `fill`.  `samples` restricts evaluation to a subset of samples (others
    hold `fill`); the per-sample definition makes that exact.
    """
    x = np.asarray(x, dtype=F64)
    W = np.asarray(W, dtype=F64)
    B, R, _ = x.shape
    C_out = W.shape[0]
    y = np.full((B, R, C_out), fill, dtype=F64)
    todo = range(B) if samples is None else samples
    for i in todo:
        t = int(idx[i])
        ki, ko = int(k_in[t]), int(k_out[t])
        z = x[i, :, :ki] @ W[:ko, :ki].T
        if bias is not None:
            z = z + np.asarray(bias, dtype=F64)[:ko]
        if bn is not None:                          # layer -> Re-SBN -> (+ shortcut) -> activation
            z = split_bn(z, t, *bn)
        if residual is not None:                    # residual block: the skip features are added before the activation
            z = z + np.asarray(residual, dtype=F64)[i, :, :ko]
        y[i, :, :ko] = activation(z, act)
    return y


def sliced_conv(x, W, idx, k_in, k_out, pad, bias=None, act=ACT_NONE, fill=np.nan, samples=None, bn=None, residual=None):
    """Slice-able convolution, stride 1, zero padding, no kernel flip.

    x [B][H][W][C_in] (channels last), W [C_O][C_I][K][K] (the paper's indexing).
    y[i][yy][xx][o] = act(b[o] + sum_{r,s} sum_{c<k_in[t]} xpad[i][yy+r-pad][xx+s-pad][c] W[o][c][r][s])
    for o < k_out[t]; the output keeps the input's H x W (requires K == 2*pad + 1).
    """
    x = np.asarray(x, dtype=F64)
    W = np.asarray(W, dtype=F64)
    B, H, Wd, _ = x.shape
    C_out, _, K, K2 = W.shape
    assert K == K2 and K == 2 * pad + 1
    y = np.full((B, H, Wd, C_out), fill, dtype=F64)
    todo = range(B) if samples is None else samples
    for i in todo:
        t = int(idx[i])
        ki, ko = int(k_in[t]), int(k_out[t])
        xp = np.zeros((H + 2 * pad, Wd + 2 * pad, ki), dtype=F64)
        xp[pad:pad + H, pad:pad + Wd, :] = x[i, :, :, :ki]
        z = np.zeros((H, Wd, ko), dtype=F64)
        for r in range(K):
            for s in range(K):
                z += xp[r:r + H, s:s + Wd, :] @ W[:ko, :ki, r, s].T
        if bias is not None:
            z = z + np.asarray(bias, dtype=F64)[:ko]
        if bn is not None:
            z = split_bn(z, t, *bn)
        if residual is not None:
            z = z + np.asarray(residual, dtype=F64)[i, :, :, :ko]
        y[i, :, :, :ko] = activation(z, act)
    return y


def sliced_depthwise(x, W, idx, c, ksize, stride=1, bias=None, act=ACT_NONE, fill=np.nan, samples=None, bn=None):
    """Slice-able depthwise convolution: group convolution with one filter per group (Sec. 3.3, "Group number
    and filter number per group", first scheme: the output width follows the input width c), with kernel-size
    slicing (the centred k x k part of the K x K filter) and the matching padding (k - 1) / 2, so that every
    kernel size yields the same output size ("Kernel size", "Padding").

    x [B][H][W][C] channels last, W [C][K][K].  For a sample of path t: channels < c[t], kernel ksize[t].
    y[i][yy][xx][ch] = act(b[ch] + sum_{r,s<k} xpad[i][yy*stride + r - p][xx*stride + s - p][ch] * W[ch][k0+r][k0+s]),
    k0 = (K - k) / 2, p = (k - 1) / 2, zero outside the image.  Output [B][Ho][Wo][C], Ho = (H - 1) // stride + 1.
    """
    x = np.asarray(x, dtype=F64)
    W = np.asarray(W, dtype=F64)
    B, H, Wd, C = x.shape
    K = W.shape[1]
    Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
    y = np.full((B, Ho, Wo, C), fill, dtype=F64)
    todo = range(B) if samples is None else samples
    for i in todo:
        t = int(idx[i])
        ct, k = int(c[t]), int(ksize[t])
        assert k % 2 == 1 and k <= K
        k0, p = (K - k) // 2, (k - 1) // 2
        xp = np.zeros((H + 2 * p, Wd + 2 * p, ct), dtype=F64)
        xp[p:p + H, p:p + Wd, :] = x[i, :, :, :ct]
        z = np.zeros((Ho, Wo, ct), dtype=F64)
        for r in range(k):
            for s in range(k):
                win = xp[r:r + (Ho - 1) * stride + 1:stride, s:s + (Wo - 1) * stride + 1:stride, :]
                z += win * W[:ct, k0 + r, k0 + s]
        if bias is not None:
            z = z + np.asarray(bias, dtype=F64)[:ct]
        if bn is not None:
            z = split_bn(z, t, *bn)
        y[i, :, :, :ct] = activation(z, act)
    return y


# --------------------------------------------------------------------------- chains
def _store(y, mirror_bf16):
    return round_bf16(y) if mirror_bf16 else y


def bottleneck(x, W1, W2, W3, idx, widths, mirror_bf16=True, samples=None):
    """1x1 (C -> w_t, ReLU) -> 3x3 pad 1 (w_t -> w_t, ReLU) -> 1x1 (w_t -> C); only the inner
    width is sliced.  With mirror_bf16 every layer output is rounded to bfloat16 where a device
    that stores bfloat16 activations would round.  Returns (y1, y2, y3)."""
    C = np.asarray(W1).shape[1]
    T = len(widths)
    full = [C] * T
    y1 = _store(sliced_conv(x, W1, idx, full, widths, 0, act=ACT_RELU, fill=0.0, samples=samples), mirror_bf16)
    y2 = _store(sliced_conv(y1, W2, idx, widths, widths, 1, act=ACT_RELU, fill=0.0, samples=samples), mirror_bf16)
    y3 = _store(sliced_conv(y2, W3, idx, widths, full, 0, act=ACT_NONE, fill=np.nan, samples=samples), mirror_bf16)
    return y1, y2, y3


def vit_qkv(x, Wq, Wk, Wv, idx, paths, D_h, samples=None):
    """Q, K, V = W_{q,k,v}[:h*D_h, :d_e] X for the path (d_e, h, d_mlp) of each sample."""
    k_in = [p[0] for p in paths]
    k_out = [p[1] * D_h for p in paths]
    return tuple(sliced_linear(x, Wm, idx, k_in, k_out, samples=samples) for Wm in (Wq, Wk, Wv))


def attention(q, k, v, idx, heads, D_h, samples=None, fill=np.nan):
    """Slimmable self-attention (Sec. 3.4): for every sample with h = heads[idx] heads,
    A_a = Softmax(Q_a K_a^T / sqrt(D_h)) V_a for a < h, output = Concat(A_0 .. A_{h-1}).

    q, k, v [B][N][H*D_h] (head a occupies columns a*D_h .. (a+1)*D_h - 1).  Returns [B][N][H*D_h] with
    the columns of heads >= h holding `fill`.
    """
    q, k, v = (np.asarray(a, dtype=F64) for a in (q, k, v))
    B, N, HD = q.shape
    out = np.full((B, N, HD), fill, dtype=F64)
    todo = range(B) if samples is None else samples
    for i in todo:
        h = int(heads[int(idx[i])])
        for a in range(h):
            sl = slice(a * D_h, (a + 1) * D_h)
            s = q[i, :, sl] @ k[i, :, sl].T / np.sqrt(D_h)
            s = s - s.max(axis=1, keepdims=True)          # softmax over the keys, row by row
            p = np.exp(s)
            p = p / p.sum(axis=1, keepdims=True)
            out[i, :, sl] = p @ v[i, :, sl]
    return out


def vit_attention_half(x, Wq, Wk, Wv, Wproj, idx, paths, D_h, mirror_bf16=True, samples=None):
    """Attention half of a slimmable ViT block (Sec. 3.4): Q, K, V from the sliced projections, the h heads of
    the sample's path through Softmax(Q K^T / sqrt(D_h)) V, concatenated, then W_proj[:d_e, :h*D_h].
    With mirror_bf16 the three stored tensors (QKV, attention output, projection output) are rounded to
    bfloat16 where a device that stores bfloat16 activations would round.  Returns (q, k, v, a, out);
    out holds NaN beyond the sample's d_e columns, a holds zeros beyond its heads."""
    heads = [p[1] for p in paths]
    q, k, v = vit_qkv(x, Wq, Wk, Wv, idx, paths, D_h, samples=samples)
    q, k, v = (_store(np.nan_to_num(t), mirror_bf16) for t in (q, k, v))
    a = _store(attention(q, k, v, idx, heads, D_h, samples=samples, fill=0.0), mirror_bf16)
    k_in = [p[1] * D_h for p in paths]
    k_out = [p[0] for p in paths]
    out = _store(sliced_linear(a, Wproj, idx, k_in, k_out, samples=samples), mirror_bf16)
    return q, k, v, a, out


def vit_mlp(x, Wfc1, Wfc2, idx, paths, mirror_bf16=True, samples=None):
    """W2[:d_e, :d_mlp] GELU(W1[:d_mlp, :d_e] X) (Eq. slimmableMLP).  Returns (hidden, out)."""
    de = [p[0] for p in paths]
    dm = [p[2] for p in paths]
    h = _store(sliced_linear(x, Wfc1, idx, de, dm, act=ACT_GELU, fill=0.0, samples=samples), mirror_bf16)
    o = _store(sliced_linear(h, Wfc2, idx, dm, de, samples=samples), mirror_bf16)
    return h, o


# --------------------------------------------------------------------------- counters
def executed_macs(idx, R, k_in, k_out, K=1):
    """Multiply-adds actually executed: sum_i R * k_in[t_i] * k_out[t_i] * K*K."""
    return int(sum(R * int(k_in[int(t)]) * int(k_out[int(t)]) * K * K for t in idx))
