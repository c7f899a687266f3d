"""Validation mode (SPLASH_FLAG_VALIDATE): a block-table entry that names no page of the pool is reported through
the workspace status word as SPLASH_BAD_PAGE_ID with (request, page index, id); with or without the flag such an id
is never dereferenced (the page reads as zeros), so nothing here faults, and the other requests are unaffected."""
import numpy as np
import pytest

from paper_2609_37626_b200 import workloads as W
from _util import compare, oracle_run

pytestmark = pytest.mark.gpu


def run(w, flags):
    import torch
    from paper_2609_37626_b200 import binding
    dw = binding.DeviceWorkload(w)
    out, lse = dw.decode(flags=flags)
    torch.cuda.synchronize()
    rc, detail = binding.splash_workspace_status(binding.decode_workspace(out.device))
    return out.cpu().numpy(), lse.cpu().numpy(), rc, detail


# (heads, cache format, implementation flag): every kernel family, the SIMT path included
@pytest.mark.parametrize("H,kv_dtype,impl", [(16, 0, 0), (64, 0, 0), (128, 0, 0), (128, 0, 2), (16, 0, 1),
                                             (64, 1, 0), (128, 1, 0), (16, 1, 1)])
@pytest.mark.parametrize("bad_id", [-3, 10 ** 6])
def test_bad_page_id_is_reported_and_never_dereferenced(H, kv_dtype, impl, bad_id):
    from paper_2609_37626_b200 import binding
    lens = [300, 700, 64, 1000]
    w = W.make_workload("validate", 9100 + H + kv_dtype, lens, H=H, kv_dtype=kv_dtype)
    ref = oracle_run(w)
    good = [(i, g) for i in (0, 2, 3) for g in range(H)]
    w.block_table[1, 4] = bad_id if bad_id < 0 else w.num_pool_pages + 5     # request 1, its fifth page
    want_id = int(w.block_table[1, 4])
    out, lse, rc, detail = run(w, impl | binding.SPLASH_FLAG_VALIDATE)
    assert rc == binding.SPLASH_BAD_PAGE_ID and detail == [1, 4, want_id]
    compare(out, lse, *ref, kv_dtype=kv_dtype, rows=good, what="other requests, validation on")
    assert np.isfinite(out[1]).all()
    # without the flag: same results, nothing reported
    out2, lse2, rc2, _ = run(w, impl)
    assert rc2 == 0
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_a_clean_table_reports_ok_and_entries_outside_the_range_are_not_checked():
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("validate_ok", 9200, [500, 130], H=16)
    out, lse, rc, _ = run(w, binding.SPLASH_FLAG_VALIDATE)
    assert rc == 0
    compare(out, lse, *oracle_run(w), kv_dtype=0, what="clean table")
    # a bad entry on a page the KV range does not touch is not an error
    w.block_table[0, 0] = -7
    dw = binding.DeviceWorkload(w)
    kb = torch.tensor([64, 0], dtype=torch.int32, device="cuda"); ke = torch.tensor([500, 130], dtype=torch.int32, device="cuda")
    o, l = dw.decode(flags=binding.SPLASH_FLAG_VALIDATE, kv_begin=kb, kv_end=ke)
    torch.cuda.synchronize()
    rc, _ = binding.splash_workspace_status(binding.decode_workspace(o.device))
    assert rc == 0
    ref = oracle_run(w, kv_begin=np.array([64, 0], np.int32), kv_end=np.array([500, 130], np.int32))
    compare(o.cpu().numpy(), l.cpu().numpy(), *ref, kv_dtype=0, what="range skips the bad entry")
