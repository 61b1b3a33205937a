"""Pins for the CPU oracle: brute force on tiny inputs, closed forms, identities the paper's
equations imply, and library special cases (torch CPU fp64).  No GPU, no CUDA library."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import dsn_oracle as O

RNG = np.random.default_rng(7)


def rand(*shape):
    return RNG.standard_normal(shape)


# ------------------------------------------------------------------ brute-force definitions
def brute_linear(x, W, idx, k_in, k_out, bias=None, act=0):
    B, R, _ = x.shape
    y = np.full((B, R, W.shape[0]), np.nan)
    for i in range(B):
        t = idx[i]
        for r in range(R):
            for o in range(k_out[t]):
                acc = 0.0 if bias is None else float(bias[o])
                for c in range(k_in[t]):
                    acc += float(x[i, r, c]) * float(W[o, c])
                if act == 1:
                    acc = max(acc, 0.0)
                elif act == 2:
                    acc = 0.5 * acc * (1.0 + math.erf(acc / math.sqrt(2.0)))
                y[i, r, o] = acc
    return y


def brute_conv(x, W, idx, k_in, k_out, pad):
    B, H, Wd, _ = x.shape
    CO, _, K, _ = W.shape
    y = np.full((B, H, Wd, CO), np.nan)
    for i in range(B):
        t = idx[i]
        for yy in range(H):
            for xx in range(Wd):
                for o in range(k_out[t]):
                    acc = 0.0
                    for r in range(K):
                        for s in range(K):
                            iy, ix = yy + r - pad, xx + s - pad
                            if 0 <= iy < H and 0 <= ix < Wd:
                                for c in range(k_in[t]):
                                    acc += float(x[i, iy, ix, c]) * float(W[o, c, r, s])
                    y[i, yy, xx, o] = acc
    return y


# ------------------------------------------------------------------ sliced linear
def test_linear_brute_force():
    B, R, Ci, Co = 5, 3, 12, 10
    x, W, b = rand(B, R, Ci), rand(Co, Ci), rand(Co)
    idx = np.array([2, 0, 1, 2, 0])
    k_in, k_out = [4, 7, 12], [3, 10, 6]
    for act in (0, 1, 2):
        got = O.sliced_linear(x, W, idx, k_in, k_out, bias=b, act=act)
        ref = brute_linear(x, W, idx, k_in, k_out, bias=b, act=act)
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12, equal_nan=True)


def test_linear_mask_equals_slice():
    """Weight nesting (mask form) and weight slicing give the same result."""
    B, R, C = 4, 2, 16
    x, W = rand(B, R, C), rand(C, C)
    idx = np.array([0, 1, 2, 1])
    k_in, k_out = [5, 9, 16], [7, 16, 11]
    got = O.sliced_linear(x, W, idx, k_in, k_out)
    for i in range(B):
        t = idx[i]
        m = np.zeros((C, C))
        m[:k_out[t], :k_in[t]] = 1.0
        full = x[i] @ (m * W).T
        np.testing.assert_allclose(got[i, :, :k_out[t]], full[:, :k_out[t]], rtol=1e-12, atol=1e-12)
        assert np.all(full[:, k_out[t]:] == 0.0)
        assert np.all(np.isnan(got[i, :, k_out[t]:]))


def test_linear_full_width_is_dense_and_library_case():
    B, R, C = 3, 4, 8
    x, W, b = rand(B, R, C), rand(6, C), rand(6)
    got = O.sliced_linear(x, W, np.zeros(B, int), [C], [6], bias=b)
    ref = torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(W), torch.from_numpy(b)).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)
    # hand-sliced library call
    got = O.sliced_linear(x, W, np.zeros(B, int), [5], [4])
    ref = torch.nn.functional.linear(torch.from_numpy(x[..., :5].copy()), torch.from_numpy(W[:4, :5].copy())).numpy()
    np.testing.assert_allclose(got[..., :4], ref, rtol=1e-12, atol=1e-12)


def test_linear_out_prefix_and_in_additivity():
    B, R, C = 2, 3, 20
    x, W = rand(B, R, C), rand(C, C)
    z = np.zeros(B, int)
    ya = O.sliced_linear(x, W, z, [12], [6])
    yb = O.sliced_linear(x, W, z, [12], [15])
    np.testing.assert_allclose(ya[..., :6], yb[..., :6], rtol=0, atol=0)        # output prefix
    y1 = O.sliced_linear(x, W, z, [8], [C])
    y2 = O.sliced_linear(x, W, z, [14], [C])
    resid = x[..., 8:14] @ W[:, 8:14].T                                         # psi_2 = psi_1 + W[k1:k2] x
    np.testing.assert_allclose(y2, y1 + resid, rtol=1e-12, atol=1e-12)


def test_linear_closed_forms():
    B, R, C = 3, 2, 9
    idx = np.array([0, 1, 2])
    k = [2, 5, 9]
    y = O.sliced_linear(np.ones((B, R, C)), np.ones((C, C)), idx, k, k)
    for i in range(B):
        assert np.all(y[i, :, :k[i]] == k[i])
    x = rand(B, R, C)
    y = O.sliced_linear(x, np.eye(C), idx, k, k)
    for i in range(B):
        np.testing.assert_array_equal(y[i, :, :k[i]], x[i, :, :k[i]])
    # transposed-operand check: W = e_o e_c^T picks x[c] into y[o]
    W = np.zeros((C, C)); W[1, 0] = 1.0
    y = O.sliced_linear(x, W, np.full(B, 2), k, k)
    np.testing.assert_array_equal(y[..., 1], x[..., 0])
    np.testing.assert_array_equal(y[..., 0], 0 * x[..., 0])


def test_linear_subset_of_samples_matches_full():
    B, R, C = 6, 2, 8
    x, W = rand(B, R, C), rand(C, C)
    idx = np.array([0, 1, 1, 0, 1, 0])
    full = O.sliced_linear(x, W, idx, [3, 8], [8, 5])
    part = O.sliced_linear(x, W, idx, [3, 8], [8, 5], samples=[1, 4])
    np.testing.assert_array_equal(part[[1, 4]], full[[1, 4]])
    assert np.all(np.isnan(part[[0, 2, 3, 5]]))


# ------------------------------------------------------------------ sliced conv
def test_conv_brute_force():
    B, H, Wd, Ci, Co = 3, 4, 5, 6, 7
    x, W = rand(B, H, Wd, Ci), rand(Co, Ci, 3, 3)
    idx = np.array([1, 0, 2])
    k_in, k_out = [2, 4, 6], [7, 3, 5]
    got = O.sliced_conv(x, W, idx, k_in, k_out, 1)
    ref = brute_conv(x, W, idx, k_in, k_out, 1)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12, equal_nan=True)


def test_conv_library_case():
    B, H, Wd, Ci, Co = 2, 6, 5, 8, 9
    x, W, b = rand(B, H, Wd, Ci), rand(Co, Ci, 3, 3), rand(Co)
    ki, ko = 5, 7
    got = O.sliced_conv(x, W, np.zeros(B, int), [ki], [ko], 1, bias=b, act=1)
    xt = torch.from_numpy(x[..., :ki].copy()).permute(0, 3, 1, 2)
    ref = torch.relu(torch.nn.functional.conv2d(xt, torch.from_numpy(W[:ko, :ki].copy()),
                                                 torch.from_numpy(b[:ko].copy()), padding=1))
    np.testing.assert_allclose(got[..., :ko], ref.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)


def test_conv_1x1_is_linear_and_centre_tap():
    B, H, Wd, C = 2, 3, 4, 6
    x, W = rand(B, H, Wd, C), rand(C, C)
    idx = np.array([0, 1]); k_in, k_out = [3, 6], [5, 2]
    lin = O.sliced_linear(x.reshape(B, H * Wd, C), W, idx, k_in, k_out).reshape(B, H, Wd, C)
    c1 = O.sliced_conv(x, W[:, :, None, None], idx, k_in, k_out, 0)
    np.testing.assert_allclose(c1, lin, rtol=1e-12, atol=1e-12, equal_nan=True)
    W3 = np.zeros((C, C, 3, 3)); W3[:, :, 1, 1] = W
    c3 = O.sliced_conv(x, W3, idx, k_in, k_out, 1)
    np.testing.assert_allclose(c3, lin, rtol=1e-12, atol=1e-12, equal_nan=True)


def test_conv_delta_image_returns_unflipped_kernel():
    """Cross-correlation: a unit impulse at (2,2) reads out W[o, c, r, s] at output (3-r, 3-s)... i.e.
    y[yy, xx] = W[r = 2 - yy + 1, s = 2 - xx + 1]; an asymmetric kernel pins the orientation."""
    H = Wd = 5
    x = np.zeros((1, H, Wd, 1)); x[0, 2, 2, 0] = 1.0
    W = np.arange(9, dtype=float).reshape(1, 1, 3, 3)
    y = O.sliced_conv(x, W, [0], [1], [1], 1)[0, :, :, 0]
    # y[yy, xx] = sum_{r,s} x[yy+r-1, xx+s-1] W[r, s]  => nonzero where yy+r-1 == 2, xx+s-1 == 2
    for yy in range(H):
        for xx in range(Wd):
            r, s = 3 - yy, 3 - xx
            want = W[0, 0, r, s] if 0 <= r < 3 and 0 <= s < 3 else 0.0
            assert y[yy, xx] == want
    assert y[1, 1] == 8.0 and y[3, 3] == 0.0 and y[1, 3] == 6.0    # spelled out: no flip


def test_conv_zero_padding_counts():
    H, Wd, C = 4, 6, 5
    idx = np.array([0, 1]); k = [3, 5]
    y = O.sliced_conv(np.ones((2, H, Wd, C)), np.ones((2, C, 3, 3)), idx, k, [2, 2], 1)
    for i in range(2):
        assert y[i, 1, 1, 0] == 9 * k[i]
        assert y[i, 0, 2, 0] == 6 * k[i] and y[i, 2, 0, 1] == 6 * k[i]
        assert y[i, 0, 0, 0] == 4 * k[i] and y[i, H - 1, Wd - 1, 1] == 4 * k[i]


def test_depthwise_library_brute_force_and_kernel_slicing():
    B, H, Wd, C, K = 3, 7, 6, 5, 7
    x, W, b = rand(B, H, Wd, C), rand(C, K, K), rand(C)
    idx = np.array([2, 0, 1]); c = [2, 5, 4]; ks = [3, 7, 5]
    for stride in (1, 2):
        got = O.sliced_depthwise(x, W, idx, c, ks, stride=stride, bias=b, act=O.ACT_RELU)
        Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
        assert got.shape == (B, Ho, Wo, C)
        for i in range(B):
            ct, k = c[idx[i]], ks[idx[i]]
            k0 = (K - k) // 2
            xt = torch.from_numpy(x[i:i + 1, :, :, :ct].copy()).permute(0, 3, 1, 2)
            wt = torch.from_numpy(W[:ct, k0:k0 + k, k0:k0 + k].copy()).unsqueeze(1)
            ref = torch.relu(torch.nn.functional.conv2d(xt, wt, torch.from_numpy(b[:ct].copy()), stride=stride,
                                                         padding=(k - 1) // 2, groups=ct))
            np.testing.assert_allclose(got[i, :, :, :ct], ref[0].permute(1, 2, 0).numpy(), rtol=1e-12, atol=1e-12)
            assert np.all(np.isnan(got[i, :, :, ct:]))
    # brute force, one output element (stride 2, 5x5 slice of the 7x7 filter)
    got = O.sliced_depthwise(x, W, idx, c, ks, stride=2)
    i, yy, xx, ch = 0, 1, 2, 3
    acc = 0.0
    for r in range(5):
        for s_ in range(5):
            iy, ix = yy * 2 + r - 2, xx * 2 + s_ - 2
            if 0 <= iy < H and 0 <= ix < Wd:
                acc += x[i, iy, ix, ch] * W[ch, 1 + r, 1 + s_]
    assert abs(got[i, yy, xx, ch] - acc) < 1e-12
    # a filter that is zero outside its centre 3x3 gives the same result for every kernel size
    Wc = np.zeros((C, K, K)); Wc[:, 2:5, 2:5] = rand(C, 3, 3)
    a3 = O.sliced_depthwise(x, Wc, np.zeros(B, int), [C], [3])
    a7 = O.sliced_depthwise(x, Wc, np.zeros(B, int), [C], [7])
    np.testing.assert_allclose(a3, a7, rtol=1e-12, atol=1e-12)
    # channels are independent: channel ch of the output depends on channel ch of the input only
    x2 = x.copy(); x2[..., 1] += 1.0
    d = O.sliced_depthwise(x2, W, np.ones(B, int), c, ks) - O.sliced_depthwise(x, W, np.ones(B, int), c, ks)
    assert np.all(d[..., [0, 2, 3, 4]] == 0) and np.any(d[..., 1] != 0)


# ------------------------------------------------------------------ gate
def brute_gate(x, W1, W2):
    B, R, C = x.shape
    out = []
    for i in range(B):
        pooled = [sum(float(x[i, r, c]) for r in range(R)) / R for c in range(C)]
        hid = [max(0.0, sum(float(W1[j, c]) * pooled[c] for c in range(C))) for j in range(W1.shape[0])]
        s = [sum(float(W2[t, j]) * hid[j] for j in range(W1.shape[0])) for t in range(W2.shape[0])]
        out.append(s)
    return np.array(out)


def test_gate_brute_force_and_library():
    B, R, C, M, T = 6, 5, 7, 4, 5
    x, W1, W2 = rand(B, R, C), rand(M, C), rand(T, M)
    idx, s, margin = O.gate(x, W1, W2)
    ref = brute_gate(x, W1, W2)
    np.testing.assert_allclose(s, ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(idx, ref.argmax(axis=1))
    xt = torch.from_numpy(x)
    lib = torch.relu(xt.mean(dim=1) @ torch.from_numpy(W1).T) @ torch.from_numpy(W2).T
    np.testing.assert_allclose(s, lib.numpy(), rtol=1e-12, atol=1e-12)
    srt = np.sort(ref, axis=1)
    np.testing.assert_allclose(margin, srt[:, -1] - srt[:, -2], rtol=1e-12, atol=1e-14)
    # softmax is monotone: argmax of probabilities equals argmax of scores
    np.testing.assert_array_equal(idx, torch.softmax(lib, dim=1).argmax(dim=1).numpy())


def test_gate_known_winner_permutation_ties_bias_cvalid():
    B, R, C, M, T = 4, 3, 5, 5, 4
    x = np.full((B, R, C), 2.0)                    # constant map => pooled = 2
    W1 = np.eye(M, C)                              # hid = pooled
    W2 = np.zeros((T, M)); W2[2, 0] = 1.0; W2[1, 0] = 0.5
    idx, s, margin = O.gate(x, W1, W2)
    assert np.all(idx == 2) and np.allclose(s[:, 2], 2.0) and np.allclose(margin, 1.0)
    p = [3, 0, 2, 1]
    idx_p, _, _ = O.gate(x, W1, W2[p])
    assert np.all(idx_p == p.index(2))             # permuting rows of W2 permutes the choice
    W2t = np.zeros((T, M)); W2t[1, 0] = 1.0; W2t[3, 0] = 1.0
    idx_t, _, m_t = O.gate(x, W1, W2t)
    assert np.all(idx_t == 1) and np.all(m_t == 0)  # tie -> lowest index
    # ReLU really clips: negative pooled value gives zero hidden, all scores 0 -> index 0
    idx_n, s_n, _ = O.gate(-x, W1, W2)
    assert np.all(idx_n == 0) and np.all(s_n == 0)
    # biases
    idx_b, s_b, _ = O.gate(x, W1, W2, b1=np.ones(M), b2=np.array([0, 0, 0, 10.0]))
    assert np.all(idx_b == 3) and np.allclose(s_b[:, 2], 3.0)
    # elastic input: only the first c_valid channels are read
    xr = rand(B, R, C)
    xr2 = xr.copy(); xr2[..., 3:] = 1e9
    W1r = rand(M, C)
    i1, s1, _ = O.gate(xr, W1r, W2, c_valid=3)
    i2, s2, _ = O.gate(xr2, W1r, W2, c_valid=3)
    np.testing.assert_array_equal(s1, s2)


def test_gate_attention_head_brute_force_library_and_identity():
    B, R, C, M = 4, 5, 6, 3
    x, W1, W3, b1, b3 = rand(B, R, C), rand(M, C), rand(C, M), rand(M), rand(C)
    scale, xh = O.gate_attention(x, W1, W3, b1, b3)
    for i in range(B):
        pooled = [sum(float(x[i, r, c]) for r in range(R)) / R for c in range(C)]
        hid = [max(0.0, float(b1[j]) + sum(float(W1[j, c]) * pooled[c] for c in range(C))) for j in range(M)]
        for c in range(C):
            a = float(b3[c]) + sum(float(W3[c, j]) * hid[j] for j in range(M))
            assert abs(scale[i, c] - (1.0 + math.tanh(a))) < 1e-12
            for r in range(R):
                assert abs(xh[i, r, c] - x[i, r, c] * (1.0 + math.tanh(a))) < 1e-12
    xt = torch.from_numpy(x)
    h = torch.relu(torch.nn.functional.linear(xt.mean(dim=1), torch.from_numpy(W1), torch.from_numpy(b1)))
    lib = 1 + torch.tanh(torch.nn.functional.linear(h, torch.from_numpy(W3), torch.from_numpy(b3)))
    np.testing.assert_allclose(scale, lib.numpy(), rtol=1e-12, atol=1e-12)
    s0, x0 = O.gate_attention(x, W1, np.zeros((C, M)))             # delta(0) = 1: the head is the identity
    assert np.all(s0 == 1.0) and np.array_equal(x0, x)
    assert np.all(scale > 0.0) and np.all(scale < 2.0)              # 1 + tanh lies in (0, 2)
    s_cv, x_cv = O.gate_attention(x, W1, W3, c_valid=4)             # elastic input
    assert s_cv.shape == (B, 4) and x_cv.shape == (B, R, 4)
    x2 = x.copy(); x2[..., 4:] = 1e9
    np.testing.assert_array_equal(O.gate_attention(x2, W1, W3, c_valid=4)[0], s_cv)


def test_split_bn_library_brute_force_and_identity():
    B, H, Wd, Ci, Co, T = 3, 4, 3, 5, 6, 2
    x, W = rand(B, H, Wd, Ci), rand(Co, Ci, 3, 3)
    gamma, beta = rand(Co), rand(Co)
    mu, sigma = rand(T, Co), np.abs(rand(T, Co)) + 0.5
    idx = np.array([1, 0, 1]); k_in, k_out = [3, 5], [4, 6]
    got = O.sliced_conv(x, W, idx, k_in, k_out, 1, bn=(gamma, beta, mu, sigma), act=O.ACT_RELU)
    plain = O.sliced_conv(x, W, idx, k_in, k_out, 1)
    for i in range(B):
        t, ko = idx[i], k_out[idx[i]]
        z = torch.from_numpy(plain[i:i + 1, :, :, :ko].copy()).permute(0, 3, 1, 2)
        ref = torch.nn.functional.batch_norm(z, torch.from_numpy(mu[t, :ko].copy()), torch.from_numpy(sigma[t, :ko] ** 2),
                                             torch.from_numpy(gamma[:ko].copy()), torch.from_numpy(beta[:ko].copy()),
                                             training=False, eps=1e-30)
        np.testing.assert_allclose(got[i, :, :, :ko], torch.relu(ref)[0].permute(1, 2, 0).numpy(), rtol=1e-11, atol=1e-12)
        # brute force on one element: per-route statistics, shared gamma / beta sliced to the width
        o = ko - 1
        want = max(0.0, gamma[o] * (plain[i, 1, 1, o] - mu[t, o]) / sigma[t, o] + beta[o])
        assert abs(got[i, 1, 1, o] - want) < 1e-12
    ident = O.sliced_linear(rand(2, 3, 4), rand(5, 4), [0, 0], [4], [5],
                            bn=(np.ones(5), np.zeros(5), np.zeros((1, 5)), np.ones((1, 5))))
    # identity statistics leave the layer unchanged; wrong-route statistics change it
    xx, WW = rand(2, 3, 4), rand(5, 4)
    a = O.sliced_linear(xx, WW, [0, 1], [4, 4], [5, 5])
    b = O.sliced_linear(xx, WW, [0, 1], [4, 4], [5, 5], bn=(np.ones(5), np.zeros(5), np.zeros((2, 5)), np.ones((2, 5))))
    np.testing.assert_array_equal(a, b)
    mu2 = np.zeros((2, 5)); mu2[1] = 1.0
    c = O.sliced_linear(xx, WW, [0, 1], [4, 4], [5, 5], bn=(np.ones(5), np.zeros(5), mu2, np.ones((2, 5))))
    np.testing.assert_array_equal(c[0], a[0])
    np.testing.assert_allclose(c[1], a[1] - 1.0, rtol=0, atol=1e-15)
    assert ident.shape == (2, 3, 5)


def test_residual_add_before_activation():
    B, H, Wd, C = 2, 3, 3, 6
    x, W, res = rand(B, H, Wd, C), rand(C, C, 1, 1), rand(B, H, Wd, C)
    idx = np.array([0, 1]); k = [4, 6]
    plain = O.sliced_conv(x, W, idx, k, k, 0)
    got = O.sliced_conv(x, W, idx, k, k, 0, act=O.ACT_RELU, residual=res)
    for i in range(B):
        w = k[idx[i]]
        np.testing.assert_allclose(got[i, ..., :w], np.maximum(plain[i, ..., :w] + res[i, ..., :w], 0.0), rtol=0, atol=1e-15)
        assert np.all(np.isnan(got[i, ..., w:]))
    # library form of a residual block tail: relu(conv(x) + shortcut)
    xt = torch.from_numpy(x[:1, ..., :4].copy()).permute(0, 3, 1, 2)
    ref = torch.relu(torch.nn.functional.conv2d(xt, torch.from_numpy(W[:4, :4].copy())) +
                     torch.from_numpy(res[:1, ..., :4].copy()).permute(0, 3, 1, 2))
    np.testing.assert_allclose(got[0, ..., :4], ref[0].permute(1, 2, 0).numpy(), rtol=1e-12, atol=1e-12)
    lin = O.sliced_linear(x.reshape(B, 9, C), W[:, :, 0, 0], idx, k, k, residual=res.reshape(B, 9, C))
    np.testing.assert_allclose(lin[0, :, :4], (plain[0] + res[0]).reshape(9, C)[:, :4], rtol=0, atol=1e-15)


# ------------------------------------------------------------------ routing
@pytest.mark.parametrize("B,T", [(1, 1), (7, 1), (1, 5), (33, 4), (100, 14), (64, 48)])
def test_route_invariants(B, T):
    idx = RNG.integers(0, T, size=B)
    counts, offsets, perm, inv = O.route(idx, T)
    assert counts.sum() == B and offsets[0] == 0 and offsets[-1] == B
    np.testing.assert_array_equal(np.diff(offsets), counts)
    np.testing.assert_array_equal(np.sort(perm), np.arange(B))
    np.testing.assert_array_equal(inv[perm], np.arange(B))
    np.testing.assert_array_equal(perm[inv], np.arange(B))
    for t in range(T):
        seg = perm[offsets[t]:offsets[t + 1]]
        assert np.all(idx[seg] == t) and np.all(np.diff(seg) > 0)
    # a stable sort is the same ordering
    np.testing.assert_array_equal(perm, np.argsort(idx, kind="stable"))
    np.testing.assert_array_equal(counts, np.bincount(idx, minlength=T))


def test_route_edge_cases():
    c, o, p, inv = O.route(np.array([3, 3, 3]), 5)
    assert c.tolist() == [0, 0, 0, 3, 0] and o.tolist() == [0, 0, 0, 0, 3, 3] and p.tolist() == [0, 1, 2]
    c, o, p, inv = O.route(np.zeros(0, int), 3)
    assert c.tolist() == [0, 0, 0] and p.shape == (0,)
    c, o, p, inv = O.route(np.array([1, 0, 1, 0]), 2)
    assert p.tolist() == [1, 3, 0, 2] and inv.tolist() == [2, 0, 3, 1]
    with pytest.raises(ValueError):
        O.route(np.array([0, 4]), 4)


# ------------------------------------------------------------------ rounding, chains, counters
def test_round_bf16_matches_library_and_is_idempotent():
    a = np.concatenate([rand(4096) * 10.0 ** RNG.integers(-6, 6, 4096), [0.0, -0.0, 1.0, 1.00390625, 1.01171875]])
    got = O.round_bf16(a)
    lib = torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(got, lib)
    np.testing.assert_array_equal(O.round_bf16(got), got)
    assert O.round_bf16(1.00390625) == 1.0          # tie -> even mantissa
    assert O.round_bf16(1.01171875) == 1.015625     # tie -> even mantissa (up)
    assert np.max(np.abs(got - a) / np.maximum(np.abs(a), 1e-30)) <= 2.0 ** -8


def test_gelu_closed_points():
    z = np.array([0.0, 1.0, -1.0, 3.0])
    g = O.activation(z, O.ACT_GELU)
    np.testing.assert_allclose(g, [0.0, 0.8413447460685429, -0.15865525393145707, 2.9959503059051097], rtol=1e-12)
    ref = torch.nn.functional.gelu(torch.from_numpy(z)).numpy()
    np.testing.assert_allclose(g, ref, rtol=1e-12, atol=1e-15)


def test_bottleneck_chain_composition_and_mirror():
    B, H, Wd, C = 3, 4, 4, 16
    widths = [4, 8]
    x = np.maximum(rand(B, H, Wd, C), 0)
    W1, W2, W3 = rand(8, C, 1, 1) / 4, rand(8, 8, 3, 3) / 8, rand(C, 8, 1, 1) / 3
    idx = np.array([1, 0, 1])
    y1, y2, y3 = O.bottleneck(x, W1, W2, W3, idx, widths, mirror_bf16=False)
    # library chain per sample on hand-sliced tensors
    for i in range(B):
        w = widths[idx[i]]
        xt = torch.from_numpy(x[i:i + 1]).permute(0, 3, 1, 2)
        a = torch.relu(torch.nn.functional.conv2d(xt, torch.from_numpy(W1[:w].copy())))
        b = torch.relu(torch.nn.functional.conv2d(a, torch.from_numpy(W2[:w, :w].copy()), padding=1))
        c = torch.nn.functional.conv2d(b, torch.from_numpy(W3[:, :w].copy()))
        np.testing.assert_allclose(y3[i], c[0].permute(1, 2, 0).numpy(), rtol=1e-11, atol=1e-12)
    m1, m2, m3 = O.bottleneck(x, W1, W2, W3, idx, widths, mirror_bf16=True)
    np.testing.assert_array_equal(O.round_bf16(m3), m3)
    assert np.max(np.abs(m3 - y3)) / np.max(np.abs(y3)) < 3 * 2.0 ** -8
    assert np.max(np.abs(m3 - y3)) > 0


def test_vit_pieces_against_library():
    B, N, De, H, Dh, Dm = 3, 5, 16, 4, 4, 32
    paths = [(8, 2, 16), (16, 4, 32), (12, 3, 24)]
    x = rand(B, N, De)
    Wq, Wk, Wv = rand(H * Dh, De), rand(H * Dh, De), rand(H * Dh, De)
    Wfc1, Wfc2 = rand(Dm, De) / 4, rand(De, Dm) / 5
    idx = np.array([2, 0, 1])
    q, k, v = O.vit_qkv(x, Wq, Wk, Wv, idx, paths, Dh)
    hid, out = O.vit_mlp(x, Wfc1, Wfc2, idx, paths, mirror_bf16=False)
    for i in range(B):
        de, h, dm = paths[idx[i]]
        xi = torch.from_numpy(x[i, :, :de].copy())
        for got, Wm in ((q, Wq), (k, Wk), (v, Wv)):
            ref = xi @ torch.from_numpy(Wm[:h * Dh, :de].copy()).T
            np.testing.assert_allclose(got[i, :, :h * Dh], ref.numpy(), rtol=1e-12, atol=1e-12)
            assert np.all(np.isnan(got[i, :, h * Dh:]))
        hr = torch.nn.functional.gelu(xi @ torch.from_numpy(Wfc1[:dm, :de].copy()).T)
        orf = hr @ torch.from_numpy(Wfc2[:de, :dm].copy()).T
        np.testing.assert_allclose(out[i, :, :de], orf.numpy(), rtol=1e-11, atol=1e-12)


def test_vit_attention_half_against_library_composition():
    """Sliced QKV -> h heads of softmax attention -> sliced projection, against torch's own
    scaled_dot_product_attention and matmul on hand-sliced tensors (unrounded), and the mirrored form
    within bf16 error of it."""
    B, N, De, H, Dh = 3, 6, 16, 4, 4
    paths = [(8, 2, 16), (16, 4, 32), (12, 3, 24)]
    x = rand(B, N, De)
    Wq, Wk, Wv, Wp = rand(H * Dh, De) / 3, rand(H * Dh, De) / 3, rand(H * Dh, De) / 3, rand(De, H * Dh) / 3
    idx = np.array([1, 2, 0])
    q, k, v, a, out = O.vit_attention_half(x, Wq, Wk, Wv, Wp, idx, paths, Dh, mirror_bf16=False)
    for i in range(B):
        de, h, _ = paths[idx[i]]
        xi = torch.from_numpy(x[i, :, :de].copy())
        qt, kt, vt = ((xi @ torch.from_numpy(Wm[:h * Dh, :de].copy()).T).reshape(N, h, Dh).permute(1, 0, 2)
                      for Wm in (Wq, Wk, Wv))
        at = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt).permute(1, 0, 2).reshape(N, h * Dh)
        ref = at @ torch.from_numpy(Wp[:de, :h * Dh].copy()).T
        np.testing.assert_allclose(a[i, :, :h * Dh], at.numpy(), rtol=1e-10, atol=1e-12)
        assert np.all(a[i, :, h * Dh:] == 0)
        np.testing.assert_allclose(out[i, :, :de], ref.numpy(), rtol=1e-10, atol=1e-12)
        assert np.all(np.isnan(out[i, :, de:]))
    m = O.vit_attention_half(x, Wq, Wk, Wv, Wp, idx, paths, Dh, mirror_bf16=True)[4]
    ok = ~np.isnan(out)
    np.testing.assert_array_equal(O.round_bf16(m[ok]), m[ok])
    assert np.max(np.abs(m[ok] - out[ok])) / np.max(np.abs(out[ok])) < 4 * 2.0 ** -8


def test_attention_library_brute_force_and_closed_forms():
    B, N, H, Dh = 3, 7, 4, 5
    q, k, v = rand(B, N, H * Dh), rand(B, N, H * Dh), rand(B, N, H * Dh)
    heads, idx = [2, 4, 1], np.array([1, 0, 2])
    out = O.attention(q, k, v, idx, heads, Dh)
    for i in range(B):
        h = heads[idx[i]]
        qt, kt, vt = (torch.from_numpy(a[i].reshape(N, H, Dh)[:, :h].transpose(1, 0, 2).copy()) for a in (q, k, v))
        ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt)       # [h][N][Dh], scale 1/sqrt(Dh)
        np.testing.assert_allclose(out[i, :, :h * Dh], ref.permute(1, 0, 2).reshape(N, h * Dh).numpy(), rtol=1e-11, atol=1e-12)
        assert np.all(np.isnan(out[i, :, h * Dh:]))
    # brute force for one (sample, head, query)
    i, a, n = 0, 3, 2
    s = [sum(q[i, n, a * Dh + d] * k[i, m, a * Dh + d] for d in range(Dh)) / math.sqrt(Dh) for m in range(N)]
    e = [math.exp(x - max(s)) for x in s]
    for d in range(Dh):
        want = sum(e[m] / sum(e) * v[i, m, a * Dh + d] for m in range(N))
        assert abs(out[i, n, a * Dh + d] - want) < 1e-12
    # zero queries give uniform attention: the mean of the values; one dominant key copies its value
    o0 = O.attention(np.zeros_like(q), k, v, np.zeros(B, int), [H], Dh)
    np.testing.assert_allclose(o0, np.broadcast_to(v.mean(axis=1, keepdims=True), v.shape), rtol=1e-12, atol=1e-12)
    kk = np.zeros((1, N, Dh)); kk[0, 3] = 50.0
    o1 = O.attention(np.ones((1, N, Dh)), kk, v[:1, :, :Dh], [0], [1], Dh)
    np.testing.assert_allclose(o1[0], np.broadcast_to(v[0, 3, :Dh], (N, Dh)), rtol=1e-9, atol=1e-9)


def test_executed_macs_closed_form():
    idx = np.array([0, 2, 2, 1, 0, 2])
    k_in, k_out, R = [4, 8, 16], [3, 6, 9], 7
    counts = np.bincount(idx, minlength=3)
    want = sum(int(counts[t]) * R * k_in[t] * k_out[t] * 9 for t in range(3))
    assert O.executed_macs(idx, R, k_in, k_out, K=3) == want
    # a 0.25x-wide inner 3x3 conv executes 1/16 of the full-width multiply-adds
    full = O.executed_macs([1], 196, [64, 256], [64, 256], K=3)
    quarter = O.executed_macs([0], 196, [64, 256], [64, 256], K=3)
    assert full == 16 * quarter == 196 * 256 * 256 * 9


def test_widths_rule_reproduces_paper_list():
    path = os.path.join(os.path.dirname(__file__), "golden", "dsmbnet_widths.txt")
    rows = [l for l in open(path).read().splitlines() if l and not l.startswith("#")]
    paper = [int(v) for v in rows[0].split()]
    ratios = [0.35 + 0.05 * i for i in range(14)]
    assert O.widths_from_ratios(640, ratios) == paper
    from dsn_workloads import WIDTHS_14
    for C in (64, 128, 256, 512, 640):
        assert O.widths_from_ratios(C, ratios) == WIDTHS_14[C]
    assert O.widths_from_ratios(256, [0.25, 0.5, 0.75, 1.0]) == [64, 128, 192, 256]


# ------------------------------------------------------------------ planted mistakes are caught
def test_pins_catch_planted_mistakes():
    """Each plausible slip, planted into a copy of the oracle's contraction, must break a pin."""
    x, W = rand(2, 3, 10), rand(10, 10)
    z = np.zeros(2, int)
    good = O.sliced_linear(x, W, z, [6], [4])
    transposed = x[:, :, :6] @ W[:6, :4]             # W indexed [in][out]
    off_by_one = x[:, :, :5] @ W[:4, :5].T           # dropped last input channel
    ref = brute_linear(x, W, z, [6], [4])[..., :4]
    assert np.allclose(good[..., :4], ref)
    assert not np.allclose(transposed, ref) and not np.allclose(off_by_one, ref)
