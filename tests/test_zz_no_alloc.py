"""The allocation-free page-migration entry point against the regular one.

Some callers of this library cannot allocate device memory at the point where they
move pages (the pool already owns the HBM budget, or a host framework owns the
allocator), so ``splash_kv_page_migrate_static`` keeps its remap table in a fixed
device array inside the library.  This test drives it through the C ABI twice in a
row -- the table keeps the first call's contents, so the second call shows that stale
entries are cleared -- and requires byte-identical pools and tables to what
``splash_kv_page_migrate`` produces with a caller-provided workspace.  It lives in a
file that pytest collects last, so that a run stopping at the first failure has
already run everything else.
"""
import ctypes

import numpy as np
import pytest

from paper_2609_37626_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_both(w, src_ids, dst_ids, n_src, dw_a, dw_b):
    """Migrate on two device copies: regular entry point on a, static one on b."""
    import torch
    from paper_2609_37626_b200 import binding
    lib = binding.load()
    s, d = torch.from_numpy(src_ids).cuda(), torch.from_numpy(dst_ids).cuda()
    binding.splash_kv_page_migrate(dw_a.kv_pool[:n_src], dw_a.kv_pool[n_src:], s, d, dw_a.block_table,
                                   src_scales=None if dw_a.kv_scales is None else dw_a.kv_scales[:n_src],
                                   dst_scales=None if dw_a.kv_scales is None else dw_a.kv_scales[n_src:],
                                   src_id_base=0, dst_id_base=n_src, max_page_id=w.num_pool_pages)
    # the new entry point, straight through ctypes: no workspace argument at all
    vp = ctypes.c_void_p
    page_bytes = 64 * 576 * dw_b.kv_pool.element_size()
    src_sc = None if dw_b.kv_scales is None else vp(dw_b.kv_scales[:n_src].data_ptr())
    dst_sc = None if dw_b.kv_scales is None else vp(dw_b.kv_scales[n_src:].data_ptr())
    rc = lib.splash_kv_page_migrate_static(
        vp(dw_b.kv_pool[:n_src].data_ptr()), src_sc, vp(dw_b.kv_pool[n_src:].data_ptr()), dst_sc, page_bytes,
        vp(s.data_ptr()), vp(d.data_ptr()), len(src_ids), 0, n_src, w.num_pool_pages,
        vp(dw_b.block_table.data_ptr()), dw_b.block_table.numel(), vp(torch.cuda.current_stream().cuda_stream))
    assert rc == 0, lib.splash_last_error()
    torch.cuda.synchronize()
    assert torch.equal(dw_a.kv_pool.view(torch.uint8), dw_b.kv_pool.view(torch.uint8))
    assert torch.equal(dw_a.block_table, dw_b.block_table)
    if dw_a.kv_scales is not None:
        assert torch.equal(dw_a.kv_scales.view(torch.int32), dw_b.kv_scales.view(torch.int32))


@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_static_migrate_matches_workspace_migrate_twice(kv_dtype):
    from paper_2609_37626_b200 import binding
    lens = [10, 64, 3000, 129, 700]
    n_used = sum((s + 63) // 64 for s in lens)
    w = W.make_workload("static_mig", 990 + kv_dtype, lens, H=16, kv_dtype=kv_dtype, extra_pool_pages=n_used)
    n_src = w.num_pool_pages - n_used
    used = np.unique(w.block_table[w.block_table >= 0])
    dw_a, dw_b = binding.DeviceWorkload(w), binding.DeviceWorkload(w)
    # first call: 30% of the pages
    src1, dst1 = W.migration_plan(1, used, n_used, 0.3)
    run_both(w, src1, dst1, n_src, dw_a, dw_b)
    # second call right after: other pages; stale entries of the first call must not leak
    rest = np.setdiff1d(used, src1)
    free_dst = np.setdiff1d(np.arange(n_used, dtype=np.int32), dst1)
    src2 = rest[: len(rest) // 2].astype(np.int32)
    dst2 = free_dst[: len(src2)].astype(np.int32)
    run_both(w, src2, dst2, n_src, dw_a, dw_b)
    # and the table really moved: no entry names a migrated source page any more
    table = dw_b.block_table.cpu().numpy()
    assert not np.isin(table, np.concatenate([src1, src2])).any()


def test_static_migrate_rejects_oversized_tables():
    from paper_2609_37626_b200 import binding
    lib = binding.load()
    p = ctypes.c_void_p(0x1000)
    rc = lib.splash_kv_page_migrate_static(p, None, p, None, 73728, p, p, 1, 0, 0, (1 << 18) + 1, p, 8, None)
    assert rc == binding.SPLASH_INVALID_ARG and b"exceeds" in lib.splash_last_error()
    assert lib.splash_last_launch_count() == 0
