"""The decode call under CUDA graph capture: the library allocates nothing, never synchronises
the host and plans on the device, so a captured call replays correctly -- also after its
inputs (lengths, queries) changed in place."""
import numpy as np
import pytest

from paper_2609_37626_b200 import workloads as W

pytestmark = pytest.mark.gpu

CASES = {
    "bf16_16_heads": dict(lens=[3000, 40, 900, 64, 2000], H=16, kv_dtype=0),
    "bf16_128_heads": dict(lens=[3000, 40, 900, 64, 2000], H=128, kv_dtype=0),
    "e4m3_128_heads": dict(lens=[3000, 40, 900, 64, 2000], H=128, kv_dtype=1),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_decode_replays_from_a_cuda_graph(case):
    import torch
    from paper_2609_37626_b200 import binding
    c = CASES[case]
    w = W.make_workload("graph", 4100, c["lens"], H=c["H"], kv_dtype=c["kv_dtype"])
    dw = binding.DeviceWorkload(w)
    out = torch.empty((w.B, w.H, W.D_V), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.B, w.H), dtype=torch.float32, device="cuda")
    dw.decode(out=out, lse=lse)                      # eager: the reference, and first-use set-up outside the capture
    torch.cuda.synchronize()
    ref_out, ref_lse = out.clone(), lse.clone()

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dw.decode(out=out, lse=lse)
    for _ in range(2):
        out.fill_(float("nan")); lse.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)

    # new lengths (within the pages each request owns) and queries in the same buffers: the replay plans again on
    # the device
    new_lens = torch.tensor([100, 40, 500, 1, 777], dtype=torch.int32, device="cuda")
    dw.seq_lens.copy_(new_lens)
    dw.q.copy_(torch.flip(dw.q, dims=[0]))
    graph.replay()
    torch.cuda.synchronize()
    got_out, got_lse = out.clone(), lse.clone()
    dw.decode(out=out, lse=lse)
    torch.cuda.synchronize()
    assert torch.equal(got_out, out) and torch.equal(got_lse, lse)
    rc, detail = binding.splash_workspace_status(binding.decode_workspace(out.device))
    assert rc == 0, (rc, detail)
    assert np.isfinite(got_out.cpu().numpy()).all()


@pytest.mark.parametrize("flags", [0, 4])
def test_sparse_decode_replays_from_a_cuda_graph(flags):
    """Both sparse paths (gather + dense kernels; the fused kernel): captured once, replayed with new token lists."""
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("graphsp", 4200, [3000, 40, 900, 64, 2000], H=128, kv_dtype=2)
    dw = binding.DeviceWorkload(w)
    sel, cnt = W.select_tokens(4201, w.seq_lens, 256)
    sel_d, cnt_d = torch.from_numpy(sel).cuda(), torch.from_numpy(cnt).cuda()
    out = torch.empty((w.B, w.H, W.D_V), dtype=torch.float32, device="cuda")
    lse = torch.empty((w.B, w.H), dtype=torch.float32, device="cuda")
    call = lambda: binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, sel_d, cnt_d,
                                                    softmax_scale=w.softmax_scale, out=out, lse=lse, flags=flags)
    call()
    torch.cuda.synchronize()
    ref_out, ref_lse = out.clone(), lse.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    out.fill_(float("nan")); lse.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)
    # another draw of the lists in the same buffers
    sel2, cnt2 = W.select_tokens(4202, w.seq_lens, 256)
    sel_d.copy_(torch.from_numpy(sel2)); cnt_d.copy_(torch.from_numpy(cnt2))
    graph.replay()
    torch.cuda.synchronize()
    got_out, got_lse = out.clone(), lse.clone()
    call()
    torch.cuda.synchronize()
    assert torch.equal(got_out, out) and torch.equal(got_lse, lse)
    assert not torch.equal(got_out, ref_out)
    assert np.isfinite(got_out.cpu().numpy()).all()


def test_lse_merge_replays_from_a_cuda_graph():
    import torch
    from paper_2609_37626_b200 import binding
    g = torch.Generator(device="cuda").manual_seed(5)
    po = torch.randn((3, 40, 512), device="cuda", generator=g)
    pl = torch.randn((3, 40), device="cuda", generator=g)
    out, lse = binding.splash_lse_merge(po, pl)
    torch.cuda.synchronize()
    ref_out, ref_lse = out.clone(), lse.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.splash_lse_merge(po, pl, out=out, lse=lse)
    out.zero_(); lse.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)


def test_page_migrate_replays_from_a_cuda_graph():
    """A captured migration, replayed on a fresh copy of the pool and table, moves the same pages and rewrites the
    same table entries as the oracle."""
    import torch
    import oracle
    from paper_2609_37626_b200 import binding
    lens = [10, 64, 3000, 129, 700]
    n_used = sum((s + 63) // 64 for s in lens)
    w = W.make_workload("miggraph", 4300, lens, H=16, kv_dtype=1, extra_pool_pages=n_used)
    n_src = w.num_pool_pages - n_used
    src_ids, dst_ids = W.migration_plan(78, np.unique(w.block_table[w.block_table >= 0]), n_used, 0.3)
    ref_pool, ref_table, ref_sc = w.kv_pool.copy(), w.block_table.copy(), w.kv_scales.copy()
    oracle.kv_page_migrate(ref_pool[:n_src], ref_pool[n_src:], src_ids, dst_ids, ref_table, src_scales=ref_sc[:n_src],
                           dst_scales=ref_sc[n_src:], dst_id_base=n_src)
    dw = binding.DeviceWorkload(w)
    pool0, table0, sc0 = dw.kv_pool.clone(), dw.block_table.clone(), dw.kv_scales.clone()
    src_d, dst_d = torch.from_numpy(src_ids).cuda(), torch.from_numpy(dst_ids).cuda()
    call = lambda: binding.splash_kv_page_migrate(
        dw.kv_pool[:n_src], dw.kv_pool[n_src:], src_d, dst_d, dw.block_table, src_scales=dw.kv_scales[:n_src],
        dst_scales=dw.kv_scales[n_src:], src_id_base=0, dst_id_base=n_src, max_page_id=w.num_pool_pages)
    call()                                           # eager once: workspace allocation and first-use set-up
    torch.cuda.synchronize()
    dw.kv_pool.copy_(pool0); dw.block_table.copy_(table0); dw.kv_scales.copy_(sc0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    dw.kv_pool.copy_(pool0); dw.block_table.copy_(table0); dw.kv_scales.copy_(sc0)
    graph.replay()
    torch.cuda.synchronize()
    assert np.array_equal(dw.kv_pool.view(torch.uint8).cpu().numpy().reshape(-1), ref_pool.view(np.uint8).reshape(-1))
    assert np.array_equal(dw.block_table.cpu().numpy(), ref_table)
    assert np.array_equal(dw.kv_scales.cpu().numpy().view(np.uint32), ref_sc.view(np.uint32))
