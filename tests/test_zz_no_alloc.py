"""The allocation-free gate entry point against the ordinary one.

dsn_gate_static serves callers that are not allowed to allocate device memory (for example a
serving loop that must never enter the CUDA allocator, or a plug-in that only gets its input and
output buffers): its scratch is a fixed array inside the library instead of a caller workspace.
It must give exactly what dsn_gate gives, also when called twice in a row on the shared scratch,
and must refuse problems that do not fit the fixed array.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import dsn_workloads as wl
from oracle import dsn_oracle as O

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _upload(cfg, B, R, C):
    x = torch.from_numpy(wl.bf16_bits(cfg["x"].reshape(B, R, C)).view(np.int16)).to(DEV).view(torch.bfloat16)
    W1 = torch.from_numpy(cfg["gate_W1"]).to(DEV)
    W2 = torch.from_numpy(cfg["gate_W2"]).to(DEV)
    return x, W1, W2


def _both(dsn, ctx, cfg, B, R, C):
    T = cfg["T"]
    x, W1, W2 = _upload(cfg, B, R, C)
    g = dsn.make_gate_desc(dsn.BF16, B, R, C, W1.shape[0], T, W1, W2)
    ws = torch.empty(dsn.dsn_gate_workspace_bytes(g), dtype=torch.uint8, device=DEV)
    idx_ref = torch.full((B,), -1, dtype=torch.int32, device=DEV)
    log_ref = torch.zeros(B, T, dtype=torch.float32, device=DEV)
    dsn.dsn_gate(ctx, g, x, idx_ref, log_ref, ws)
    idx_new = torch.full((B,), -2, dtype=torch.int32, device=DEV)
    log_new = torch.full((B, T), 7.0, dtype=torch.float32, device=DEV)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()            # the driver's own count of free device memory
    dsn.dsn_gate_static(ctx, g, x, idx_new, log_new)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                      # the call took no device memory from anyone
    assert ctx.get_status() == (0, 0)
    scale = max(1.0, float(log_ref.abs().max()))
    assert float((log_new - log_ref).abs().max()) <= 2e-5 * scale      # the gate tests' score tolerance
    assert torch.equal(idx_new, idx_ref)
    assert int(idx_ref.min()) >= 0 and int(idx_ref.max()) < T
    # and directly against the CPU oracle: scores within the gate tolerance, choices equal outside the 1e-4 margin
    idx_o, scores_o, margin = O.gate(cfg["x"].reshape(B, R, C), cfg["gate_W1"], cfg["gate_W2"])
    got = log_new.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got - scores_o)) <= 2e-5 * max(1.0, float(np.max(np.abs(scores_o))))
    safe = margin >= 1e-4
    np.testing.assert_array_equal(idx_new.cpu().numpy()[safe], idx_o[safe])


def test_static_gate_matches_workspace_gate_on_two_calls_in_a_row(dsn):
    ctx = dsn.Context(0)
    cnn = wl.config2(B=128)                     # ResNet-shaped gate: 128 x 196 x 1024 -> 14 paths
    _both(dsn, ctx, cnn, 128, 196, 1024)
    vit = wl.config3(B=40)                      # a different shape reuses (and overwrites) the same scratch
    _both(dsn, ctx, vit, 40, 197, 384)
    _both(dsn, ctx, cnn, 128, 196, 1024)


def test_static_gate_rejects_what_does_not_fit(dsn):
    ctx = dsn.Context(0)
    B, R, C, M, T = 1024, 512, 2048, 8, 2       # B * splits * C is beyond 1,048,576 floats for any split count
    x = torch.zeros(1, dtype=torch.bfloat16, device=DEV)            # never read: the call must refuse first
    W1 = torch.zeros(M, C, dtype=torch.float32, device=DEV)
    W2 = torch.zeros(T, M, dtype=torch.float32, device=DEV)
    g = dsn.make_gate_desc(dsn.BF16, B, R, C, M, T, W1, W2)
    idx = torch.full((B,), -5, dtype=torch.int32, device=DEV)
    with pytest.raises(dsn.DsnError) as err:
        dsn.dsn_gate_static(ctx, g, x, idx)
    assert err.value.code == dsn.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert int(idx.max()) == -5 and ctx.get_status() == (0, 0)
