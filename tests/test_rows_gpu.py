"""GPU parity for several causal query rows per request (q_rows = R > 1): the CUDA path
through the C ABI against the multi-row oracle on the same seeded bytes."""
import numpy as np
import pytest

import oracle
from paper_2609_37626_b200 import workloads as W
from _util import TOL

pytestmark = pytest.mark.gpu

# 0: the CTA-pair tcgen05 kernels (the only tensor-core path for R > 1); 1: the fp32 SIMT kernel
IMPLS = {"umma": 0, "simt": 1}


@pytest.fixture(params=list(IMPLS))
def flags(request):
    return IMPLS[request.param]


def gpu_rows(w, q4, flags=0, sentinel=None, **kw):
    import torch
    from paper_2609_37626_b200 import binding
    dw = binding.DeviceWorkload(w)
    q = torch.from_numpy(q4.view(np.int16)).cuda().view(torch.bfloat16)
    B, H, R, _ = q4.shape
    out = lse = None
    if sentinel is not None:
        out = torch.full((B, H, R, W.D_V), float(sentinel), dtype=torch.float32, device="cuda")
        lse = torch.full((B, H, R), float(sentinel), dtype=torch.float32, device="cuda")
    args = dict(softmax_scale=w.softmax_scale, kv_scales=dw.kv_scales, head_begin=w.head_begin, head_end=w.head_end,
                out=out, lse=lse, flags=flags)
    args.update(kw)
    out, lse = binding.splash_mla_decode(q, dw.kv_pool, dw.block_table, dw.seq_lens, **args)
    torch.cuda.synchronize()
    rc, detail = binding.splash_workspace_status(binding.decode_workspace(out.device))
    assert rc == 0, f"device status {rc} detail {detail}"
    return out.cpu().numpy(), lse.cpu().numpy()


def oracle_rows(w, q4, **kw):
    args = dict(softmax_scale=w.softmax_scale, kv_scales=w.kv_scales, head_begin=w.head_begin, head_end=w.head_end)
    args.update(kw)
    return oracle.mla_decode_rows(q4, w.kv_pool, w.block_table, w.seq_lens, **args)


def compare_rows(out, lse, ref_out, ref_lse, kv_dtype, hb, he, what):
    tol = TOL[kv_dtype]
    o, r = out[:, hb:he].astype(np.float64), ref_out[:, hb:he]
    L, rl = lse[:, hb:he].astype(np.float64), ref_lse[:, hb:he]
    assert np.isfinite(o).all(), f"{what}: non-finite output"
    empty = np.isneginf(rl)
    assert np.array_equal(np.isneginf(L), empty), f"{what}: empty rows differ"
    assert np.all(o[empty] == 0.0), f"{what}: an empty row is not zero"
    d = np.abs(o - r).max(axis=-1)
    assert d.max() <= tol["abs_o"], f"{what}: |dO| {d.max()}"
    if tol["rel_o"] is not None:
        scale = np.abs(r).max(axis=-1)
        rel = np.where(empty, 0.0, d / np.where(scale > 0, scale, 1.0))
        assert rel.max() <= tol["rel_o"], f"{what}: rel {rel.max()}"
    dl = np.abs(L[~empty] - rl[~empty])
    assert dl.size == 0 or dl.max() <= tol["lse"], f"{what}: LSE {dl.max()}"


# lengths around page and tile edges (the causal cut falls into the last page, or crosses into the one before),
# a request with exactly R tokens and one with fewer tokens than rows
@pytest.mark.parametrize("kv_dtype", [0, 1])
@pytest.mark.parametrize("R,H,lens", [
    (2, 16, [2, 63, 64, 65, 128, 129, 1000]), (4, 16, [3, 4, 64, 66, 67, 300, 4097]), (8, 16, [5, 8, 65, 70, 200]),
    (2, 64, [1, 64, 65, 777]), (3, 40, [130, 64, 2, 5000]), (2, 128, [66, 1500, 64]), (4, 128, [131, 12345]),
    # more than 128 (head, row) pairs: several CTA pairs per KV worker in one launch (8 x 128 = 1,024 pairs in 8 groups;
    # 3 x 100 = 300 pairs in 3 groups, the last one partly filled)
    (8, 128, [300, 70, 2000]), (3, 100, [129, 3000, 7]),
])
def test_rows_match_the_oracle(flags, kv_dtype, R, H, lens):
    w = W.make_workload("rows", 800 + R + H, lens, H=H, kv_dtype=kv_dtype)
    q4 = W.make_query_rows(800 + R + H, w.B, H, R)
    ref = oracle_rows(w, q4)
    out, lse = gpu_rows(w, q4, flags=flags)
    compare_rows(out, lse, *ref, kv_dtype, 0, H, f"R={R} H={H}")


@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_rows_head_slice_ranges_and_untouched_rest(flags, kv_dtype):
    R, H, hb, he = 4, 32, 8, 24
    w = W.make_workload("rowsslice", 830 + kv_dtype, [900, 70, 3000, 129, 6], H=H, kv_dtype=kv_dtype, head_begin=hb, head_end=he)
    q4 = W.make_query_rows(830, w.B, H, R)
    import torch
    # ranges: a cut in the middle, one that ends inside the causal window, one that starts at the last token,
    # one past the end, an empty one
    kb = np.array([100, 0, 2999, 64, 3], dtype=np.int32); ke = np.array([800, 68, 3000, 500, 3], dtype=np.int32)
    ref = oracle_rows(w, q4, kv_begin=kb, kv_end=ke)
    out, lse = gpu_rows(w, q4, flags=flags, sentinel=9.0, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    compare_rows(out, lse, *ref, kv_dtype, hb, he, "slice + ranges")
    assert np.all(out[:, :hb] == 9.0) and np.all(out[:, he:] == 9.0) and np.all(lse[:, :hb] == 9.0) and np.all(lse[:, he:] == 9.0)


def test_rows_many_requests_split_over_workers_and_determinism():
    R, H = 2, 64
    rng = np.random.Generator(np.random.PCG64(845))
    lens = [int(x) for x in rng.integers(2, 3000, size=96)]
    w = W.make_workload("rowsmany", 845, lens, H=H)
    q4 = W.make_query_rows(845, w.B, H, R)
    ref = oracle_rows(w, q4)
    a = gpu_rows(w, q4)
    compare_rows(*a, *ref, 0, 0, H, "many requests")
    b = gpu_rows(w, q4)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_rows_last_row_equals_plain_decode_on_the_gpu():
    # the newest row has no causal cut: it must agree with the one-row call of the same query (both against the
    # oracle's tolerance of each other: different kernels may tile differently)
    import torch
    from paper_2609_37626_b200 import binding
    R, H = 4, 32
    w = W.make_workload("rowslast", 850, [500, 64, 4000], H=H)
    q4 = W.make_query_rows(850, w.B, H, R)
    out4, lse4 = gpu_rows(w, q4)
    dw = binding.DeviceWorkload(w)
    q1 = torch.from_numpy(np.ascontiguousarray(q4[:, :, R - 1]).view(np.int16)).cuda().view(torch.bfloat16)
    o1, l1 = binding.splash_mla_decode(q1, dw.kv_pool, dw.block_table, dw.seq_lens, softmax_scale=w.softmax_scale)
    torch.cuda.synchronize()
    assert np.abs(out4[:, :, R - 1] - o1.cpu().numpy()).max() <= 2 * TOL[0]["abs_o"]
    assert np.abs(lse4[:, :, R - 1] - l1.cpu().numpy()).max() <= 2 * TOL[0]["lse"]


def test_rows_argument_checks():
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("rowsargs", 860, [100], H=16)
    dw = binding.DeviceWorkload(w)
    q = torch.zeros((1, 16, 9, 576), dtype=torch.bfloat16, device="cuda")     # 9 rows: more than the library builds
    with pytest.raises(Exception):
        binding.splash_mla_decode(q, dw.kv_pool, dw.block_table, dw.seq_lens, softmax_scale=0.1)
    q = torch.zeros((1, 16, 2, 576), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Exception):                                              # pairs switched off: not with rows
        binding.splash_mla_decode(q, dw.kv_pool, dw.block_table, dw.seq_lens, softmax_scale=0.1, flags=2)
