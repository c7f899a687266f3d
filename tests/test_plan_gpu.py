"""The split-KV plan the device writes.

The plan is an integer step with many valid answers (any cut of the tile sequence into contiguous runs gives
correct attention), so what PINS it are the partition properties checked at the end: effective ranges as
defined, boundaries that start at 0, end at the tile total and never decrease, and every non-empty request's
first / last worker containing its first / last tile -- i.e. every (request, tile) is covered exactly once, in
order.  The equality with ``python_plan`` below is a regression check only: that function restates the
kernel's own balancing rule and is no independent source of truth."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def python_plan(lo, hi, W, overhead=4):
    n = np.where(hi > lo, (hi + 63) // 64 - lo // 64, 0)
    ts = np.concatenate([[0], np.cumsum(n)])
    cost = np.where(n > 0, n + overhead, 0)
    cs = np.concatenate([[0], np.cumsum(cost)])
    total = int(cs[-1])
    wb = []
    for w in range(W + 1):
        if w == W or total == 0:
            wb.append(int(ts[-1])); continue
        target = total * w // W
        i = int(np.searchsorted(cs, target, side="right") - 1)
        off = max(0, target - int(cs[i]) - overhead)
        wb.append(int(ts[i]) + off)
    return ts, np.array(wb)


# the last case has more requests than the plan kernel stages in shared memory (4,096): its prefix arrays and
# bisections then live in global memory
@pytest.mark.parametrize("seed,B,div", [(1, 1, 8), (2, 7, 8), (3, 64, 8), (4, 512, 8), (5, 2100, 8), (6, 5000, 64)])
def test_plan_matches_python_and_partitions_tiles(seed, B, div):
    import ctypes
    import torch
    from paper_2609_37626_b200 import binding, workloads as W
    rng = np.random.default_rng(seed)
    lens = W.rollout_lengths(seed, B) // div
    lens[rng.integers(0, B, size=max(1, B // 10))] = 0
    kb = rng.integers(-3, 50, size=B).astype(np.int32)
    ke = (lens + rng.integers(-40, 5, size=B)).astype(np.int32)
    w = W.make_workload("plan", seed, lens, H=16, poison=False)
    dw = binding.DeviceWorkload(w)
    dw.decode(kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda(), flags=1)
    torch.cuda.synchronize()
    ws = binding.decode_workspace(torch.device("cuda", 0)).cpu().numpy()
    sm = torch.cuda.get_device_properties(0).multi_processor_count
    Wn = (2 * sm) // 2         # SIMT path: 16 heads = 2 groups of 8 -> 2*SMs/2 workers
    ints = ws.view(np.int32)
    off = 16
    ts = ints[off:off + B + 1]; off += B + 1
    lo = ints[off:off + B]; off += B
    hi = ints[off:off + B]; off += B
    wf = ints[off:off + B]; off += B
    wl = ints[off:off + B]; off += B
    cs = ints[off:off + B + 1]; off += B + 1
    wb = ints[off:off + Wn + 1]
    elo = np.maximum(kb, 0); ehi = np.maximum(np.minimum(ke, lens), elo)
    assert np.array_equal(lo, elo) and np.array_equal(hi, ehi)
    # the per-request overhead the library chose for this kernel: read back from its own cost prefix
    n_tiles = np.where(ehi > elo, (ehi + 63) // 64 - elo // 64, 0)
    nz = np.flatnonzero(n_tiles > 0)
    overhead = int(cs[nz[0] + 1] - cs[nz[0]] - n_tiles[nz[0]]) if len(nz) else 4
    assert 1 <= overhead <= 16
    pts, pwb = python_plan(elo.astype(np.int64), ehi.astype(np.int64), Wn, overhead)
    assert np.array_equal(ts, pts) and np.array_equal(wb, pwb)
    assert wb[0] == 0 and wb[-1] == ts[-1] and np.all(np.diff(wb) >= 0)
    for i in range(B):
        if ts[i + 1] == ts[i]:
            assert wf[i] == -1
        else:
            assert wb[wf[i]] <= ts[i] < wb[wf[i] + 1] and wb[wl[i]] <= ts[i + 1] - 1 < wb[wl[i] + 1]
