"""The five workload configurations at their full sizes, in the launch configuration
bench.py times, against the oracle on sampled (request, head) outputs (the oracle
computes any output on its own), plus the properties that hold at any size: head
slices concatenate, KV ranges merge to the unsplit result, decode after a page
migration is bit-identical."""
import numpy as np
import pytest

from paper_2609_37626_b200 import workloads as W
from _util import compare, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


def sample_pairs(w, n, seed, must=()):
    rng = np.random.default_rng(seed)
    heads = np.arange(w.head_begin, w.head_end)
    pairs = {(int(i), int(g)) for i, g in must}
    while len(pairs) < n:
        pairs.add((int(rng.integers(0, w.B)), int(rng.choice(heads))))
    return sorted(pairs)


def check_sampled(w, out, lse, pairs, what, **kw):
    ref_o, ref_l = oracle_run(w, pairs=np.array(pairs, np.int32), **kw)
    return compare(out, lse, ref_o, ref_l, w.kv_dtype, rows=pairs, what=what)


def test_c2_dp_attention_full_size():
    w = W.config(2)
    assert w.B == 64 and w.H == 128 and w.seq_lens.min() >= 1024 and w.seq_lens.max() <= 8192
    out, lse = gpu_run(w)
    longest, shortest = int(np.argmax(w.seq_lens)), int(np.argmin(w.seq_lens))
    pairs = sample_pairs(w, 96, 2, must=[(longest, 0), (longest, 127), (shortest, 64), (0, 0), (63, 127)])
    check_sampled(w, out, lse, pairs, "c2")
    assert np.isfinite(out).all() and np.isfinite(lse).all()


def test_c3_head_slice_full_size_and_all_slices_concatenate():
    import torch
    from paper_2609_37626_b200 import binding
    w = W.config(3)
    assert w.B == 16 and list(w.seq_lens) == [32768] * 16 and (w.head_begin, w.head_end) == (32, 48)
    dw = binding.DeviceWorkload(w)
    out, lse = gpu_run(w, dw=dw, sentinel=5.0)
    pairs = sample_pairs(w, 24, 3, must=[(0, 32), (15, 47)])
    check_sampled(w, out, lse, pairs, "c3 slice")
    assert np.all(out[:, :32] == 5.0) and np.all(out[:, 48:] == 5.0)
    # all 8 slices into one buffer reproduce the unsplit 128-head call (each vs the oracle,
    # and the two CUDA results against each other at twice the tolerance)
    cat_o = torch.zeros((16, 128, 512), dtype=torch.float32, device="cuda")
    cat_l = torch.zeros((16, 128), dtype=torch.float32, device="cuda")
    for hb in range(0, 128, 16):
        dw.decode(out=cat_o, lse=cat_l, head_begin=hb, head_end=hb + 16)
    full_o, full_l = dw.decode(head_begin=0, head_end=128)
    torch.cuda.synchronize()
    w_all = W.Workload(**{**w.__dict__, "head_begin": 0, "head_end": 128})
    pairs = sample_pairs(w_all, 24, 33, must=[(3, 0), (3, 127), (9, 63)])
    check_sampled(w_all, cat_o.cpu().numpy(), cat_l.cpu().numpy(), pairs, "c3 8 slices", head_begin=0, head_end=128)
    check_sampled(w_all, full_o.cpu().numpy(), full_l.cpu().numpy(), pairs, "c3 unsplit", head_begin=0, head_end=128)
    assert (cat_o - full_o).abs().max().item() <= 2e-2 and (cat_l - full_l).abs().max().item() <= 2e-3


def test_c4_cp_ranges_merge_full_size():
    import torch
    from paper_2609_37626_b200 import binding
    w = W.config(4)
    assert w.B == 1 and int(w.seq_lens[0]) == 262144
    dw = binding.DeviceWorkload(w)
    out, lse = gpu_run(w, dw=dw)
    pairs = [(0, g) for g in (0, 1, 31, 64, 100, 127)]
    check_sampled(w, out, lse, pairs, "c4 unsplit")
    po = torch.empty((8, 128, 512), dtype=torch.float32, device="cuda")
    pl = torch.empty((8, 128), dtype=torch.float32, device="cuda")
    for j, (a, b) in enumerate(W.cp_ranges(w.seq_lens, 8)):
        dw.decode(out=po[j:j + 1], lse=pl[j:j + 1], kv_begin=torch.from_numpy(a).cuda(), kv_end=torch.from_numpy(b).cuda())
        if j in (0, 5):   # a chunk on its own against the oracle
            torch.cuda.synchronize()
            check_sampled(w, po[j:j + 1].cpu().numpy(), pl[j:j + 1].cpu().numpy(), [(0, 7), (0, 90)], f"c4 chunk {j}",
                          kv_begin=a, kv_end=b)
    mo, ml = binding.splash_lse_merge(po, pl)
    torch.cuda.synchronize()
    mo, ml = mo.cpu().numpy()[None], ml.cpu().numpy()[None]
    check_sampled(w, mo, ml, pairs, "c4 merged")
    assert np.abs(mo - out).max() <= 2e-2 and np.abs(ml - lse).max() <= 2e-3
    # rope columns carry sigma = 2: the logits use all 576 columns, V only the first 512
    qf = W.bf16_bits_to_f32(w.q[0, 0]).astype(np.float64)
    sig2 = np.ones(576); sig2[512:] = 4.0
    limit = np.log(262144) + 0.5 * w.softmax_scale ** 2 * float((sig2 * qf ** 2).sum())
    assert abs(lse[0, 0] - limit) < 0.1


def test_c5_rollout_fp8_and_page_migration_full_size():
    import torch
    from paper_2609_37626_b200 import binding
    w = W.config(5, extra_pool_factor=0.3)
    assert w.B == 512 and w.kv_dtype == 1 and w.seq_lens.min() >= 16 and w.seq_lens.max() <= 131072
    n_extra = int(np.ceil(len(w.used_pages) * 0.3))
    n_src = w.num_pool_pages - n_extra
    dw = binding.DeviceWorkload(w)
    out, lse = gpu_run(w, dw=dw)
    # one head of EVERY request (a fault tied to particular worker boundaries of the long-tailed draw cannot hide
    # between samples) plus all 128 heads of the 8 longest and the 8 shortest requests
    rng = np.random.default_rng(5)
    order = np.argsort(w.seq_lens, kind="stable")
    pairs = {(i, int(rng.integers(0, 128))) for i in range(w.B)}
    pairs |= {(int(i), g) for i in list(order[:8]) + list(order[-8:]) for g in range(128)}
    pairs = sorted(pairs)
    check_sampled(w, out, lse, pairs, "c5")
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    # migrate a seeded 30% of the in-use pages to the second pool, poison the vacated pages
    src, dst = W.migration_plan(W.BASE_SEED + 55, w.used_pages, n_extra, 0.3)
    table0 = w.block_table.copy()
    binding.splash_kv_page_migrate(dw.kv_pool[:n_src], dw.kv_pool[n_src:], torch.from_numpy(src).cuda(),
                                   torch.from_numpy(dst).cuda(), dw.block_table, src_scales=dw.kv_scales[:n_src],
                                   dst_scales=dw.kv_scales[n_src:], src_id_base=0, dst_id_base=n_src,
                                   max_page_id=w.num_pool_pages)
    torch.cuda.synchronize()
    remap = np.arange(w.num_pool_pages, dtype=np.int32)
    remap[src] = n_src + dst
    expect = np.where(table0 >= 0, remap[np.maximum(table0, 0)], table0)
    assert np.array_equal(dw.block_table.cpu().numpy(), expect)
    moved = dw.kv_pool[n_src:][torch.from_numpy(dst).long().cuda()].cpu().numpy()
    assert np.array_equal(moved, w.kv_pool[src])
    assert np.array_equal(dw.kv_scales[n_src:][torch.from_numpy(dst).long().cuda()].cpu().numpy().view(np.uint32),
                          w.kv_scales[src].view(np.uint32))
    dw.kv_pool[torch.from_numpy(src).long().cuda()] = 0x7F
    dw.kv_scales[torch.from_numpy(src).long().cuda()] = float("nan")
    out2, lse2 = gpu_run(w, dw=dw)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_c5_tp8_share_full_size():
    """A TP-8 rank's 16 heads of the rollout workload, as bench.py times it (heads [32, 48) of the same cache and
    requests): one head of every request and all 16 heads of the 8 longest and 8 shortest against the oracle; nothing
    written outside the slice; the eight shares side by side equal the 128-head call within twice the tolerance."""
    import torch
    from paper_2609_37626_b200 import binding
    w = W.config(5)
    dw = binding.DeviceWorkload(w)
    out, lse = gpu_run(w, dw=dw, sentinel=3.0, head_begin=32, head_end=48)
    rng = np.random.default_rng(58)
    order = np.argsort(w.seq_lens, kind="stable")
    pairs = {(i, int(rng.integers(32, 48))) for i in range(w.B)}
    pairs |= {(int(i), g) for i in list(order[:8]) + list(order[-8:]) for g in range(32, 48)}
    check_sampled(w, out, lse, sorted(pairs), "c5 heads [32, 48)", head_begin=32, head_end=48)
    assert np.all(out[:, :32] == 3.0) and np.all(out[:, 48:] == 3.0) and np.all(lse[:, :32] == 3.0) and np.all(lse[:, 48:] == 3.0)
    assert np.isfinite(out[:, 32:48]).all() and np.isfinite(lse[:, 32:48]).all()
    cat_o = torch.zeros((w.B, 128, 512), dtype=torch.float32, device="cuda")
    cat_l = torch.zeros((w.B, 128), dtype=torch.float32, device="cuda")
    for hb in range(0, 128, 16):
        dw.decode(out=cat_o, lse=cat_l, head_begin=hb, head_end=hb + 16)
    full_o, full_l = dw.decode()
    torch.cuda.synchronize()
    assert (cat_o - full_o).abs().max().item() <= 1e-1 and (cat_l - full_l).abs().max().item() <= 1e-2
    assert np.array_equal(cat_o[:, 32:48].cpu().numpy(), out[:, 32:48])       # the same launch twice: the same bits
