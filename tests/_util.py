"""Helpers shared by the GPU parity tests: run the CUDA path through the binding,
run the oracle on the same bytes, compare under the stated tolerances."""
import numpy as np

import oracle
from paper_2609_37626_b200 import workloads as W

# tolerances of the parity bar: bf16 KV -> |dO| <= 1e-2, row-normwise relative error
# <= 2e-2 (max_d |dO| / max_d |O_ref| per (request, head) row), |dLSE| <= 1e-3;
# e4m3 KV -> |dO| <= 5e-2 (LSE reported, bounded loosely).
TOL = {0: dict(abs_o=1e-2, rel_o=2e-2, lse=1e-3), 1: dict(abs_o=5e-2, rel_o=None, lse=2e-2)}


def oracle_run(w, **kw):
    args = dict(softmax_scale=w.softmax_scale, kv_scales=w.kv_scales, head_begin=w.head_begin,
                head_end=w.head_end, kv_begin=w.kv_begin, kv_end=w.kv_end)
    args.update(kw)
    return oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, **args)


def gpu_run(w, dw=None, sentinel=None, **kw):
    """Returns (out, lse) as numpy float32 arrays [B][H][512], [B][H]."""
    import torch
    from paper_2609_37626_b200 import binding
    if dw is None:
        dw = binding.DeviceWorkload(w)
    out = lse = None
    if sentinel is not None:
        out = torch.full((w.B, w.H, W.D_V), float(sentinel), dtype=torch.float32, device="cuda")
        lse = torch.full((w.B, w.H), float(sentinel), dtype=torch.float32, device="cuda")
    out, lse = dw.decode(out=out, lse=lse, **kw)
    torch.cuda.synchronize()
    ws = binding.decode_workspace(out.device)
    if ws is not None and w.B > 0 and (kw.get("head_end", w.head_end) - kw.get("head_begin", w.head_begin)) > 0:
        rc, detail = binding.splash_workspace_status(ws)
        assert rc == 0, f"device status {rc} detail {detail}"
    return out.cpu().numpy(), lse.cpu().numpy()


def compare(out, lse, ref_out, ref_lse, kv_dtype, rows=None, what=""):
    """rows: iterable of (request, head) to compare (default: all finite-or-inf ref rows)."""
    tol = TOL[kv_dtype]
    if rows is None:
        B, H = ref_lse.shape
        rows = [(i, g) for i in range(B) for g in range(H) if not np.isnan(ref_lse[i, g])]
    worst = dict(abs_o=0.0, rel_o=0.0, lse=0.0)
    for i, g in rows:
        o, r = out[i, g].astype(np.float64), ref_out[i, g]
        assert np.isfinite(o).all(), f"{what} non-finite output at {(i, g)}"
        if np.isneginf(ref_lse[i, g]):
            assert np.all(o == 0.0) and np.isneginf(lse[i, g]), f"{what} empty range at {(i, g)}"
            continue
        d = np.abs(o - r).max()
        worst["abs_o"] = max(worst["abs_o"], d)
        worst["rel_o"] = max(worst["rel_o"], d / np.abs(r).max())
        worst["lse"] = max(worst["lse"], abs(float(lse[i, g]) - ref_lse[i, g]))
    assert worst["abs_o"] <= tol["abs_o"], f"{what} |dO| {worst}"
    if tol["rel_o"] is not None:
        assert worst["rel_o"] <= tol["rel_o"], f"{what} rel {worst}"
    assert worst["lse"] <= tol["lse"], f"{what} LSE {worst}"
    return worst
