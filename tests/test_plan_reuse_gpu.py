"""SPLASH_FLAG_REUSE_PLAN: a decode step runs the same batch through every layer, so the work partition of the first
layer's call serves the others (the partition depends on the lengths, the ranges and the shape only).  Each case plans
once on "layer 0" and decodes further layers -- other queries, another cache and block table, the same lengths -- with
the plan kernel left out; every layer is compared with the oracle."""
import numpy as np
import pytest

from paper_2609_37626_b200 import workloads as W
from _util import oracle_run, compare

pytestmark = pytest.mark.gpu


def layers(seed, lens, n, **kw):
    return [W.make_workload("layer%d" % k, seed + 17 * k, lens, **kw) for k in range(n)]


@pytest.mark.parametrize("kv_dtype,H,hb,he,flags", [(0, 16, 0, 16, 0), (0, 128, 0, 128, 0), (1, 128, 0, 128, 0),
                                                     (1, 128, 32, 48, 0), (0, 64, 0, 64, 0), (1, 128, 0, 128, 2)])
def test_layers_share_one_plan(kv_dtype, H, hb, he, flags):
    import torch
    from paper_2609_37626_b200 import binding
    rng = np.random.default_rng(900 + H + kv_dtype)
    lens = np.concatenate([rng.integers(1, 3000, size=40), [0, 9000, 64, 65]]).astype(np.int32)
    ws = layers(5100 + H + kv_dtype, lens, 3, H=H, head_begin=hb, head_end=he, kv_dtype=kv_dtype)
    dws = [binding.DeviceWorkload(w) for w in ws]
    launches = []
    for k, (w, dw) in enumerate(zip(ws, dws)):
        out, lse = dw.decode(flags=flags | (binding.SPLASH_FLAG_REUSE_PLAN if k > 0 else 0))
        launches.append(binding.splash_last_launch_count())
        torch.cuda.synchronize()
        rc, detail = binding.splash_workspace_status(binding.decode_workspace(out.device))
        assert rc == 0, f"device status {rc} detail {detail}"
        ref = oracle_run(w)
        compare(out.cpu().numpy(), lse.cpu().numpy(), *ref, kv_dtype=kv_dtype,
                rows=[(i, g) for i in range(len(lens)) for g in range(hb, he)], what=f"layer {k}")
    assert launches[1] == launches[0] - 1 and launches[2] == launches[1]      # the plan kernel is the one left out


def test_ranges_and_rows_share_the_plan_too():
    import torch
    from paper_2609_37626_b200 import binding
    lens = np.array([700, 64, 3000, 129], np.int32)
    kb = np.array([10, 0, 1000, 64], np.int32); ke = np.array([650, 64, 2900, 129], np.int32)
    ws = layers(5300, lens, 2, H=32)
    for k, w in enumerate(ws):
        dw = binding.DeviceWorkload(w)
        out, lse = dw.decode(kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda(),
                             flags=binding.SPLASH_FLAG_REUSE_PLAN if k > 0 else 0)
        torch.cuda.synchronize()
        ref = oracle_run(w, kv_begin=kb, kv_end=ke)
        compare(out.cpu().numpy(), lse.cpu().numpy(), *ref, kv_dtype=0, what=f"ranges, layer {k}")
