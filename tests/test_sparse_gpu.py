"""GPU parity of sparse decode (a token list per request over 656-byte cache rows) through the C ABI
against the sparse oracle on the same seeded bytes and lists."""
import numpy as np
import pytest

import oracle
from paper_2609_37626_b200 import workloads as W
from _util import TOL

pytestmark = pytest.mark.gpu

# The rows are e4m3 with block scales: the fp8 bar.  The path rounds the dequantised rows (code x fp32 scale) to bf16
# before the contraction, a relative 2^-9 per key element, which moves a logit of magnitude ~6 by a few 1e-3.
TOL_O = TOL[1]["abs_o"]
TOL_LSE = TOL[1]["lse"]


# 0: the gather kernel followed by the dense kernels; 4: the fused kernel (gather + dequantise + attention on CTA pairs)
PATHS = {"two_stage": 0, "fused": 4}


@pytest.fixture(params=list(PATHS))
def flags(request):
    return PATHS[request.param]


def gpu_sparse(w, sel, cnt, sentinel=None, **kw):
    import torch
    from paper_2609_37626_b200 import binding
    dw = binding.DeviceWorkload(w)
    out = lse = None
    if sentinel is not None:
        out = torch.full((w.B, w.H, W.D_V), float(sentinel), dtype=torch.float32, device="cuda")
        lse = torch.full((w.B, w.H), float(sentinel), dtype=torch.float32, device="cuda")
    args = dict(softmax_scale=w.softmax_scale, head_begin=w.head_begin, head_end=w.head_end, out=out, lse=lse)
    args.update(kw)
    out, lse = binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, torch.from_numpy(sel).cuda(),
                                                torch.from_numpy(cnt).cuda(), **args)
    torch.cuda.synchronize()
    ws = binding.decode_workspace(out.device)
    if w.B > 0 and args["head_end"] > args["head_begin"]:
        rc, detail = binding.splash_workspace_status(ws)
        assert rc == 0, f"device status {rc} detail {detail}"
    return out.cpu().numpy(), lse.cpu().numpy()


def compare_sparse(out, lse, ref_out, ref_lse, hb, he, what):
    o, r = out[:, hb:he].astype(np.float64), ref_out[:, hb:he]
    L, rl = lse[:, hb:he].astype(np.float64), ref_lse[:, hb:he]
    assert np.isfinite(o).all(), f"{what}: non-finite output"
    empty = np.isneginf(rl)
    assert np.array_equal(np.isneginf(L), empty), f"{what}: empty lists differ"
    assert np.all(o[empty] == 0.0)
    assert np.abs(o - r).max() <= TOL_O, f"{what}: |dO| {np.abs(o - r).max()}"
    dl = np.abs(L[~empty] - rl[~empty])
    assert dl.size == 0 or dl.max() <= TOL_LSE, f"{what}: LSE {dl.max()}"


@pytest.mark.parametrize("H,lens,topk", [
    (16, [1, 63, 64, 65, 200, 5000], 128),          # lists shorter and longer than the context, ragged last page
    (128, [3000, 70, 2048, 9000], 2048),            # the indexer's k of the sparse backend, all heads (CTA pair)
    (64, [700, 0, 129, 4000, 1], 300),              # an empty request, a list that ends inside a page
    (8, [100000], 1000),                            # one long context, a sparse pick
])
def test_sparse_matches_the_oracle(flags, H, lens, topk):
    w = W.make_workload("sparse", 900 + H, lens, H=H, kv_dtype=2)
    sel, cnt = W.select_tokens(900 + H, w.seq_lens, topk)
    ref = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=w.softmax_scale)
    out, lse = gpu_sparse(w, sel, cnt, flags=flags)
    compare_sparse(out, lse, *ref, 0, H, f"H={H} topk={topk}")


def test_sparse_head_slice_leaves_the_rest_untouched_and_is_reproducible(flags):
    H, hb, he = 32, 8, 24
    w = W.make_workload("sparseslice", 910, [900, 70, 3000, 129, 6], H=H, kv_dtype=2, head_begin=hb, head_end=he)
    sel, cnt = W.select_tokens(910, w.seq_lens, 256)
    cnt[1] = 0                                                # an empty list for a non-empty request
    ref = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=w.softmax_scale,
                                   head_begin=hb, head_end=he)
    a = gpu_sparse(w, sel, cnt, sentinel=7.0, flags=flags)
    compare_sparse(*a, *ref, hb, he, "slice")
    assert np.all(a[0][:, :hb] == 7.0) and np.all(a[0][:, he:] == 7.0) and np.all(a[1][:, :hb] == 7.0) and np.all(a[1][:, he:] == 7.0)
    b = gpu_sparse(w, sel, cnt, sentinel=7.0, flags=flags)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_sparse_duplicates_and_wide_list_stride(flags):
    w = W.make_workload("sparsedup", 920, [500, 64], H=16, kv_dtype=2)
    rng = np.random.Generator(np.random.PCG64(920))
    sel = np.full((2, 200), -1, dtype=np.int32)               # a stride wider than max_selected
    sel[0, :90] = rng.integers(0, 500, size=90); sel[1, :70] = rng.integers(0, 64, size=70)     # with repeats
    cnt = np.array([90, 70], dtype=np.int32)
    ref = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=w.softmax_scale)
    out, lse = gpu_sparse(w, sel, cnt, max_selected=96, flags=flags)
    compare_sparse(out, lse, *ref, 0, 16, "duplicates")


def test_sparse_bad_entries_give_nan_for_that_request_only(flags):
    w = W.make_workload("sparsebad", 930, [300, 300, 300], H=16, kv_dtype=2)
    sel, cnt = W.select_tokens(930, w.seq_lens, 64)
    good = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=w.softmax_scale)
    bad = sel.copy(); bad[1, 17] = 300                        # one position past the end of request 1
    out, lse = gpu_sparse(w, bad, cnt, flags=flags)
    assert np.isnan(out[1]).all() and np.isnan(lse[1]).all()
    assert np.abs(out[[0, 2]] - good[0][[0, 2]]).max() <= TOL_O
    cnt2 = cnt.copy(); cnt2[2] = 65                           # a count above max_selected
    out, lse = gpu_sparse(w, sel, cnt2, max_selected=64, flags=flags)
    assert np.isnan(out[2]).all() and np.isfinite(out[:2]).all()


def test_sparse_argument_checks():
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("sparseargs", 940, [100], H=16, kv_dtype=2)
    dw = binding.DeviceWorkload(w)
    sel = torch.zeros((1, 8), dtype=torch.int32, device="cuda"); cnt = torch.ones(1, dtype=torch.int32, device="cuda")
    with pytest.raises(Exception):                            # the dense entry point does not read 656-byte rows
        binding.splash_mla_decode(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, softmax_scale=0.1)
    with pytest.raises(Exception):                            # a workspace that is too small
        binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, sel, cnt, softmax_scale=0.1,
                                         workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    out, lse = binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, sel, cnt, softmax_scale=0.1)
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()


def test_sparse_at_the_size_the_benchmark_times(flags):
    # c2's 64 context lengths, 2,048 listed tokens per request, all 128 heads: every output against the oracle
    c2 = W.config(2)
    w = W.make_workload("sparse_top2048", W.BASE_SEED + 60, c2.seq_lens, H=128, kv_dtype=2)
    del c2
    sel, cnt = W.select_tokens(W.BASE_SEED + 60, w.seq_lens, 2048)
    assert cnt.max() == 2048 and cnt.sum() > 100000
    ref = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=w.softmax_scale)
    out, lse = gpu_sparse(w, sel, cnt, flags=flags)
    compare_sparse(out, lse, *ref, 0, 128, "bench size")


def test_sparse_all_lists_empty_and_zero_capacity(flags):
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("sparseempty", 950, [100, 7], H=16, kv_dtype=2)
    dw = binding.DeviceWorkload(w)
    cnt = torch.zeros(2, dtype=torch.int32, device="cuda")
    for sel in (torch.zeros((2, 0), dtype=torch.int32, device="cuda"), torch.full((2, 5), -1, dtype=torch.int32, device="cuda")):
        out, lse = binding.splash_mla_decode_sparse(dw.q, dw.kv_pool, dw.block_table, dw.seq_lens, sel, cnt,
                                                    softmax_scale=w.softmax_scale, flags=flags)
        torch.cuda.synchronize()
        assert torch.all(out == 0) and torch.all(torch.isneginf(lse))


@pytest.mark.parametrize("seed", range(8))
def test_sparse_random_shapes_and_slices(flags, seed):
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 24))
    H = int(rng.choice([1, 3, 8, 16, 24, 40, 64, 72, 128]))
    lens = rng.integers(0, 2500, size=B)
    topk = int(rng.choice([1, 7, 64, 65, 200, 513]))
    hb = int(rng.integers(0, H)); he = int(rng.integers(hb + 1, H + 1))
    w = W.make_workload("sparserand", 1000 + seed, lens, H=H, kv_dtype=2, head_begin=hb, head_end=he)
    sel, cnt = W.select_tokens(1000 + seed, w.seq_lens, topk)
    cnt[rng.integers(0, B)] = 0                                   # one request with an empty list
    ref = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=w.softmax_scale,
                                   head_begin=hb, head_end=he)
    out, lse = gpu_sparse(w, sel, cnt, sentinel=3.0, flags=flags)
    compare_sparse(out, lse, *ref, hb, he, f"seed {seed}: B={B} H={H} slice [{hb},{he}) topk={topk}")
    assert np.all(out[:, :hb] == 3.0) and np.all(out[:, he:] == 3.0)
