"""Helpers shared by the GPU parity tests (upload, routing buffers, comparisons)."""
import numpy as np
import torch

import dsn_workloads as wl

DEV = "cuda:0"
SENTINEL = 776.0   # bf16-representable marker for "must stay untouched"


def up_bf16(a):
    """Upload bf16-representable fp32 values as a bf16 device tensor (exact)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return torch.from_numpy(wl.bf16_bits(a).view(np.int16)).to(DEV).view(torch.bfloat16).reshape(a.shape)


def up_f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)


def up_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def down(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def alloc_routing(dsn, B, G):
    counts = torch.zeros(max(G, 1), dtype=torch.int32, device=DEV)
    offsets = torch.zeros(G + 1, dtype=torch.int32, device=DEV)
    perm = torch.zeros(max(B, 1), dtype=torch.int32, device=DEV)
    inv = torch.zeros(max(B, 1), dtype=torch.int32, device=DEV)
    return dsn.make_routing(B, G, counts, offsets, perm, inv)


def route_on_gpu(dsn, ctx, idx_np, T):
    B = len(idx_np)
    r = alloc_routing(dsn, B, T)
    idx = up_i32(idx_np)
    dsn.dsn_route(ctx, idx, B, T, r)
    r._keep = r._keep + (idx,)
    return r


def routing_arrays(r):
    counts, offsets, perm, inv = r._keep[:4]
    return (counts.cpu().numpy(), offsets.cpu().numpy(), perm.cpu().numpy()[:r.B], inv.cpu().numpy()[:r.B])


def group_errors(got, ref, idx, k_out, T):
    """max|err| / max|ref| per group over the valid columns; got/ref [B][...][C]."""
    out = {}
    for t in range(T):
        sel = np.nonzero(np.asarray(idx) == t)[0]
        if len(sel) == 0:
            continue
        g = got[sel][..., :k_out[t]]
        r = ref[sel][..., :k_out[t]]
        assert np.all(np.isfinite(r)), "oracle produced non-finite values inside the slice"
        denom = np.max(np.abs(r))
        out[t] = float(np.max(np.abs(g - r)) / (denom if denom > 0 else 1.0))
    return out


def assert_tail_untouched(got, idx, k_out, sentinel=SENTINEL):
    for i, t in enumerate(idx):
        tail = got[i][..., k_out[t]:]
        assert np.all(tail == sentinel), f"sample {i}: columns >= k_out were written"


def check_status(ctx, dsn):
    code, detail = ctx.get_status()
    assert code == 0, f"device status {code} ({dsn.dsn_strerror(code)}), detail {detail}"
