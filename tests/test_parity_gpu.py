"""GPU parity: the CUDA path, called through the C ABI binding, against the CPU
oracle on the same seeded bytes -- element by element at sizes the oracle finishes
in seconds (several tiles, ragged tails), plus the edge cases of the method."""
import math

import numpy as np
import pytest

from paper_2609_37626_b200 import workloads as W
from _util import compare, gpu_run, oracle_run

pytestmark = pytest.mark.gpu

# 0: the tcgen05 kernels (CTA pairs for slices of more than 64 heads); 2: the same with pairs switched
# off (two independent 64-head CTAs); 1: the fp32 SIMT kernel
IMPLS = {"umma": 0, "umma_single": 2, "simt": 1}


@pytest.fixture(params=list(IMPLS))
def flags(request):
    return IMPLS[request.param]


def test_config1_tiny_full_shard(flags):
    w = W.config(1)
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags)
    compare(out, lse, *ref, kv_dtype=0, what="c1")


@pytest.mark.parametrize("lens", [[1], [63], [64], [65], [127, 128, 129], [4095, 4097], [1, 17, 64, 200, 1000]])
def test_page_and_tile_edges(flags, lens):
    w = W.make_workload("edges", 101 + len(lens) + lens[0], lens, H=16)
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags)
    compare(out, lse, *ref, kv_dtype=0, what=f"lens {lens}")


@pytest.mark.parametrize("H,hb,he", [(16, 0, 16), (32, 0, 32), (64, 0, 64), (128, 0, 128), (128, 32, 48),
                                     (128, 0, 16), (128, 112, 128), (128, 64, 128), (128, 32, 64), (24, 3, 11)])
def test_head_slices_touch_only_their_slice(flags, H, hb, he):
    w = W.make_workload("heads", 200 + H + hb, [300, 70, 1500], H=H, head_begin=hb, head_end=he)
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags, sentinel=7.0)
    compare(out, lse, *ref, kv_dtype=0, rows=[(i, g) for i in range(3) for g in range(hb, he)], what="slice")
    mask = np.ones(H, bool); mask[hb:he] = False
    assert np.all(out[:, mask] == 7.0) and np.all(lse[:, mask] == 7.0)


def test_head_slices_concatenate(flags):
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("concat", 230, [500, 2100], H=128)
    dw = binding.DeviceWorkload(w)
    out = torch.zeros((2, 128, 512), dtype=torch.float32, device="cuda")
    lse = torch.zeros((2, 128), dtype=torch.float32, device="cuda")
    for hb in range(0, 128, 16):
        dw.decode(out=out, lse=lse, head_begin=hb, head_end=hb + 16, flags=flags)
    full_o, full_l = dw.decode(flags=flags)
    torch.cuda.synchronize()
    ref = oracle_run(w)
    compare(out.cpu().numpy(), lse.cpu().numpy(), *ref, kv_dtype=0, what="8 slices")
    compare(full_o.cpu().numpy(), full_l.cpu().numpy(), *ref, kv_dtype=0, what="unsplit")
    assert (out - full_o).abs().max().item() <= 2e-2


@pytest.mark.parametrize("B", [1, 4, 64])
def test_request_counts_and_skewed_lengths(flags, B):
    rng = np.random.default_rng(B)
    lens = rng.integers(1, 700, size=B)
    if B == 64:
        lens[5] = 9000     # one long request among many short ones: exercises the split-KV plan
    w = W.make_workload("reqs", 300 + B, lens, H=16)
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags)
    compare(out, lse, *ref, kv_dtype=0, what=f"B={B}")


# Every KV worker gets several requests of dozens of tiles each: the pipelines reach their steady state (all stages, both
# S and P buffers in flight, the softmax warps as far ahead of the P.V issuers as the barriers allow) and cross request
# boundaries in it.  One case per kernel family; sampled outputs against the oracle, the device status word clean.
@pytest.mark.parametrize("kv_dtype,H,flags", [(1, 16, 0), (1, 32, 0), (1, 64, 0), (1, 128, 0), (1, 128, 2),
                                              (0, 16, 0), (0, 32, 0), (0, 64, 0), (0, 128, 0), (0, 128, 2)])
def test_long_segments_several_per_worker(kv_dtype, H, flags):
    rng = np.random.default_rng(4000 + H + kv_dtype)
    lens = rng.integers(2500, 4500, size=150)
    w = W.make_workload("steady", 380 + H + kv_dtype, lens, H=H, kv_dtype=kv_dtype)
    out, lse = gpu_run(w, flags=flags)
    pairs = np.array(sorted({(int(rng.integers(0, len(lens))), int(rng.integers(0, H))) for _ in range(120)}), np.int32)
    ref_o, ref_l = oracle_run(w, pairs=pairs)
    compare(out, lse, ref_o, ref_l, kv_dtype=kv_dtype, rows=[tuple(p) for p in pairs], what=f"steady H={H} dtype={kv_dtype}")
    assert np.isfinite(out).all() and np.isfinite(lse).all()


def test_more_requests_than_the_plan_stages_in_shared_memory():
    # 4,500 short requests (the plan kernel keeps its prefix arrays in shared memory up to 4,096): sampled outputs
    # against the oracle, every output finite, empty requests zero
    B = 4500
    rng = np.random.default_rng(77)
    lens = rng.integers(0, 200, size=B)
    w = W.make_workload("manyreq", 377, lens, H=16)
    out, lse = gpu_run(w)
    pairs = np.array(sorted({(int(rng.integers(0, B)), int(rng.integers(0, 16))) for _ in range(300)}), np.int32)
    ref_o, ref_l = oracle_run(w, pairs=pairs)
    compare(out, lse, ref_o, ref_l, kv_dtype=0, rows=[tuple(p) for p in pairs], what="B=4500")
    assert np.isfinite(out).all()
    empty = lens == 0
    assert np.all(out[empty] == 0) and np.all(np.isneginf(lse[empty])) and np.isfinite(lse[~empty]).all()


def test_empty_batch_and_empty_slice_are_no_ops(flags):
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("idle", 310, [100], H=16)
    dw = binding.DeviceWorkload(w)
    out = torch.full((1, 16, 512), 3.0, device="cuda"); lse = torch.full((1, 16), 3.0, device="cuda")
    dw.decode(out=out, lse=lse, head_begin=8, head_end=8, flags=flags)
    assert binding.splash_last_launch_count() == 0
    torch.cuda.synchronize()
    assert torch.all(out == 3.0) and torch.all(lse == 3.0)
    q0 = dw.q[:0]
    o, l = binding.splash_mla_decode(q0, dw.kv_pool, dw.block_table[:0], dw.seq_lens[:0], softmax_scale=0.1, flags=flags)
    assert o.shape == (0, 16, 512)


@pytest.mark.parametrize("cuts", [[0, 1000, 2000, 3000, 4000, 5000, 6000, 7000, 8000], [0, 1, 130, 5000, 8000],
                                  [0, 63, 64, 65, 8000]])
def test_kv_ranges_and_lse_merge(flags, cuts):
    import torch
    from paper_2609_37626_b200 import binding
    w = W.make_workload("cp", 400, [8000, 3000], H=16, rope_scale=2.0)
    dw = binding.DeviceWorkload(w)
    ref = oracle_run(w)
    parts_o, parts_l = [], []
    for a, b in zip(cuts[:-1], cuts[1:]):
        kb = np.array([a, a], np.int32); ke = np.array([b, b], np.int32)
        o, l = gpu_run(w, dw=dw, flags=flags, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
        ro, rl = oracle_run(w, kv_begin=kb, kv_end=ke)
        compare(o, l, ro, rl, kv_dtype=0, what=f"range [{a},{b})")
        parts_o.append(torch.from_numpy(o).cuda().reshape(-1, 512)); parts_l.append(torch.from_numpy(l).cuda().reshape(-1))
    mo, ml = binding.splash_lse_merge(torch.stack(parts_o), torch.stack(parts_l))
    torch.cuda.synchronize()
    compare(mo.cpu().numpy().reshape(2, 16, 512), ml.cpu().numpy().reshape(2, 16), *ref, kv_dtype=0, what="merged")


def test_ranges_clipped_empty_and_beyond(flags):
    import torch
    w = W.make_workload("clip", 410, [100, 300, 0, 64], H=16)
    kb = np.array([-5, 290, 0, 64], np.int32); ke = np.array([1000, 290, 10, 200], np.int32)
    ref = oracle_run(w, kv_begin=kb, kv_end=ke)
    out, lse = gpu_run(w, flags=flags, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    compare(out, lse, *ref, kv_dtype=0, what="clipped")
    assert np.all(out[1] == 0) and np.all(np.isneginf(lse[1])) and np.all(np.isneginf(lse[2:]))


@pytest.mark.parametrize("placement,factor", [("identity", 1.0), ("permute", 1.25), ("reversed", 2.0)])
def test_paging_layouts_and_shared_pages(flags, placement, factor):
    w = W.make_workload("paging", 500, [130, 700, 64], H=16, placement=placement, pool_factor=factor, table_stride=20)
    w.block_table[2, 0] = w.block_table[1, 3]      # a full page shared by two requests
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags)
    compare(out, lse, *ref, kv_dtype=0, what=placement)


def test_closed_forms_on_gpu(flags):
    # n = 1 -> V row exactly; identical V rows -> that row; q = 0 -> mean of V, ln n
    w = W.make_workload("one", 600, [1, 1], H=16)
    out, lse = gpu_run(w, flags=flags)
    for i in range(2):
        row = W.bf16_bits_to_f32(w.kv_pool[w.block_table[i, 0], 0])
        assert np.abs(out[i] - row[None, :512]).max() <= 1e-6
    w = W.make_workload("q0", 601, [333], H=16)
    w.q[...] = 0
    out, lse = gpu_run(w, flags=flags)
    ref = oracle_run(w)
    assert np.abs(lse - math.log(333)).max() < 1e-5
    compare(out, lse, *ref, kv_dtype=0, what="q=0")


@pytest.mark.parametrize("lens", [[1, 17, 64, 200], [1000, 3, 4097]])
def test_fp8_kv(flags, lens):
    w = W.make_workload("fp8", 700 + lens[0], lens, H=16, kv_dtype=1)
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags)
    compare(out, lse, *ref, kv_dtype=1, what="fp8")


# Narrow e4m3 slices run with the tokens on the MMA's M: 16 or 32 heads per CTA.  Widths that fill a group, widths
# that leave it ragged, a slice in the middle of a wider layer, a request that many workers split, many short ones.
@pytest.mark.parametrize("H,hb,he,lens", [
    (32, 0, 32, [1, 17, 64, 200]), (24, 0, 24, [1000, 3, 4097]), (128, 48, 80, [333, 64, 129, 2000]),
    (128, 100, 109, [65, 5000]), (32, 0, 32, [30000]), (16, 0, 16, [130] * 300), (20, 3, 20, list(range(1, 300, 5))),
])
def test_fp8_narrow_head_slices(H, hb, he, lens):
    w = W.make_workload("fp8n", 740 + H + he + len(lens), lens, H=H, head_begin=hb, head_end=he, kv_dtype=1)
    ref = oracle_run(w)
    out, lse = gpu_run(w)
    compare(out, lse, *ref, kv_dtype=1, rows=[(i, g) for i in range(len(lens)) for g in range(hb, he)], what="fp8 narrow")


def test_fp8_extreme_rows(flags):
    w = W.make_workload("fp8x", 710, [200], H=16, kv_dtype=1)
    p = w.block_table[0, 0]
    w.kv_pool[p, 3] = 0; w.kv_scales[p, 3] = 1.0                  # all-zero row, scale 1
    w.kv_pool[p, 4, :] = 0x7E; w.kv_scales[p, 4] = 2.0 ** -12     # every code at +448, tiny scale
    w.kv_pool[p, 5, ::2] = 0xFE                                    # -448 on even columns
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=flags)
    compare(out, lse, *ref, kv_dtype=1, what="fp8 extremes")


# Slices of more than 64 heads over an e4m3 cache run on CTA pairs (one page per CTA, two pages per
# step); flag 2 selects two independent 64-head CTAs instead.  Lengths cover a lone ragged page, odd
# and even page counts, requests that several workers split, and many short requests per worker.
@pytest.mark.parametrize("no_pair", [0, 2], ids=["pair", "single"])
@pytest.mark.parametrize("H,lens", [
    (128, [1]), (128, [63, 64, 65, 128, 129]), (128, [200, 5000, 1, 777, 12345]), (80, [333, 64, 4097]),
    (72, [130] * 40), (128, list(range(1, 400, 7))), (128, [40000]),
])
def test_fp8_wide_head_slices(no_pair, H, lens):
    w = W.make_workload("fp8w", 720 + H + len(lens), lens, H=H, kv_dtype=1)
    ref = oracle_run(w)
    out, lse = gpu_run(w, flags=no_pair)
    compare(out, lse, *ref, kv_dtype=1, what="fp8 wide")


@pytest.mark.parametrize("no_pair", [0, 2], ids=["pair", "single"])
def test_fp8_wide_slice_of_a_wider_layer_and_kv_ranges(no_pair):
    import torch
    kb = np.array([100, 0, 64, 128], dtype=np.int32); ke = np.array([899, 70, 2500, 129], dtype=np.int32)
    w = W.make_workload("fp8ws", 731, [900, 70, 3000, 129], H=128, kv_dtype=1, head_begin=16, head_end=112)
    ref = oracle_run(w, kv_begin=kb, kv_end=ke)
    out, lse = gpu_run(w, flags=no_pair, sentinel=5.0,
                       kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    assert (out[:, :16] == 5.0).all() and (out[:, 112:] == 5.0).all()
    compare(out, lse, *ref, kv_dtype=1, rows=[(i, g) for i in range(4) for g in range(16, 112)], what="fp8 wide slice")


def test_many_empty_requests_among_live_ones(flags):
    """Idle shards inside a batch: every other request has an empty range (or no tokens);
    they get O = 0, LSE = -inf from the decode CTAs, the live ones are unaffected."""
    import torch
    rng = np.random.default_rng(77)
    B = 200
    lens = rng.integers(0, 400, size=B).astype(np.int32)
    lens[::7] = 0
    w = W.make_workload("empties", 820, lens, H=32)
    kb = np.zeros(B, np.int32); ke = lens.copy()
    kb[1::2] = lens[1::2]            # empty range for every other request
    ref = oracle_run(w, kv_begin=kb, kv_end=ke)
    out, lse = gpu_run(w, flags=flags, sentinel=3.0, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    compare(out, lse, *ref, kv_dtype=0, what="empties")
    assert np.all(out[1::2] == 0) and np.all(np.isneginf(lse[1::2]))


@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_wide_slices_are_deterministic_too(kv_dtype):
    w = W.make_workload("det128", 830 + kv_dtype, [3000, 40, 900, 64, 2000], H=128, kv_dtype=kv_dtype)
    a = gpu_run(w)
    b = gpu_run(w)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    compare(a[0], a[1], *oracle_run(w), kv_dtype=kv_dtype, what="det128")


def test_run_to_run_determinism(flags):
    import torch
    w = W.make_workload("det", 800, [5000, 100, 2500], H=16)
    a = gpu_run(w, flags=flags)
    junk = torch.empty(1 << 22, device="cuda").normal_()
    b = gpu_run(w, flags=flags)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    del junk


# ---------------------------------------------------------------- merge / migrate
def test_lse_merge_laws():
    import torch
    import oracle
    from paper_2609_37626_b200 import binding
    rng = np.random.default_rng(9)
    o = rng.standard_normal((5, 37, 512)).astype(np.float32); l = rng.standard_normal((5, 37)).astype(np.float32)
    l[2] = -np.inf; o[2] = np.nan
    l[:, 5] = -np.inf
    mo, ml = binding.splash_lse_merge(torch.from_numpy(o).cuda(), torch.from_numpy(l).cuda())
    ro, rl = oracle.lse_merge(o[[0, 1, 3, 4]].astype(np.float64), l[[0, 1, 3, 4]].astype(np.float64))
    mo, ml = mo.cpu().numpy(), ml.cpu().numpy()
    assert np.all(mo[5] == 0) and np.isneginf(ml[5])
    keep = np.arange(37) != 5
    assert np.abs(mo[keep] - ro[keep]).max() < 1e-5 and np.abs(ml[keep] - rl[keep]).max() < 1e-5
    one_o, one_l = binding.splash_lse_merge(torch.from_numpy(o[:1]).cuda(), torch.from_numpy(l[:1]).cuda())
    assert np.array_equal(one_o.cpu().numpy()[keep], o[0][keep])


@pytest.mark.parametrize("kv_dtype,fraction", [(0, 0.3), (1, 0.3), (0, 1.0), (1, 0.02)])
def test_page_migrate_bit_exact_and_decode_identical(flags, kv_dtype, fraction):
    import torch
    import oracle
    from paper_2609_37626_b200 import binding
    lens = [10, 64, 3000, 129, 700]
    n_used = sum((s + 63) // 64 for s in lens)
    w = W.make_workload("mig", 900 + kv_dtype, lens, H=16, kv_dtype=kv_dtype, extra_pool_pages=n_used)
    n_src = w.num_pool_pages - n_used
    w.block_table[0, 0] = w.block_table[1, 0]
    src_ids, dst_ids = W.migration_plan(77, np.unique(w.block_table[w.block_table >= 0]), n_used, fraction)
    dw = binding.DeviceWorkload(w)
    before = gpu_run(w, dw=dw, flags=flags)
    # oracle side, on numpy copies
    ref_pool, ref_table = w.kv_pool.copy(), w.block_table.copy()
    ref_sc = None if w.kv_scales is None else w.kv_scales.copy()
    oracle.kv_page_migrate(ref_pool[:n_src], ref_pool[n_src:], src_ids, dst_ids, ref_table,
                           src_scales=None if ref_sc is None else ref_sc[:n_src],
                           dst_scales=None if ref_sc is None else ref_sc[n_src:], dst_id_base=n_src)
    # CUDA side
    binding.splash_kv_page_migrate(
        dw.kv_pool[:n_src], dw.kv_pool[n_src:], torch.from_numpy(src_ids).cuda(), torch.from_numpy(dst_ids).cuda(),
        dw.block_table, src_scales=None if dw.kv_scales is None else dw.kv_scales[:n_src],
        dst_scales=None if dw.kv_scales is None else dw.kv_scales[n_src:], src_id_base=0, dst_id_base=n_src,
        max_page_id=w.num_pool_pages)
    torch.cuda.synchronize()
    got_pool = dw.kv_pool.view(torch.uint8).cpu().numpy()
    assert np.array_equal(got_pool.reshape(-1), ref_pool.view(np.uint8).reshape(-1))
    assert np.array_equal(dw.block_table.cpu().numpy(), ref_table)
    if ref_sc is not None:
        assert np.array_equal(dw.kv_scales.cpu().numpy().view(np.uint32), ref_sc.view(np.uint32))
    # vacated pages poisoned, decode again: bit-identical
    dw.kv_pool.view(torch.uint8)[torch.from_numpy(src_ids).long().cuda()] = 0x7F
    after = gpu_run(w, dw=dw, flags=flags)
    assert np.array_equal(before[0], after[0]) and np.array_equal(before[1], after[1])


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_ranges_and_slices(seed):
    """Seeded random small problems: batch size, lengths, head count and slice, KV ranges,
    placement and KV format all drawn at random; both CUDA paths against the oracle."""
    import torch
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 7))
    lens = rng.integers(0, 700, size=B).astype(np.int32)
    if rng.random() < 0.3:
        lens[rng.integers(0, B)] = int(rng.integers(2000, 6000))
    H = int(rng.choice([16, 32, 64, 128, 24]))
    hb = int(rng.integers(0, H))
    he = int(rng.integers(hb + 1, H + 1))
    kv_dtype = int(rng.integers(0, 2))
    w = W.make_workload("rand", 5000 + seed, lens, H=H, head_begin=hb, head_end=he, kv_dtype=kv_dtype,
                        placement=str(rng.choice(["permute", "identity", "reversed"])), pool_factor=float(rng.choice([1.0, 1.5])))
    kb = ke = None
    if rng.random() < 0.6:
        kb = np.array([int(rng.integers(-10, max(1, s))) for s in lens], np.int32)
        ke = np.array([int(rng.integers(0, s + 20)) for s in lens], np.int32)
        if seed >= 12:      # the later seeds: whatever lies outside a request's range is NaN / Inf (only its own tokens are its own)
            W.poison_outside_ranges(w, kb, ke)
    ref = oracle_run(w, kv_begin=kb, kv_end=ke)
    kw = {} if kb is None else dict(kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    rows = [(i, g) for i in range(B) for g in range(hb, he)]
    for flags in (0, 1) + ((2,) if he - hb > 64 else ()):
        out, lse = gpu_run(w, flags=flags, sentinel=9.0, **kw)
        compare(out, lse, *ref, kv_dtype=kv_dtype, rows=rows, what=f"seed {seed} flags {flags}")
        mask = np.ones(H, bool); mask[hb:he] = False
        assert np.all(out[:, mask] == 9.0) and np.all(lse[:, mask] == 9.0)


@pytest.mark.parametrize("shift", [17, -20])
@pytest.mark.parametrize("H", [128, 80])
def test_split_requests_with_large_and_tiny_cache_values(H, shift):
    """Requests cut into several pieces on the CTA-pair kernel, whose partial outputs travel as f16 rows: cache
    values of magnitude 2^17 (beyond f16's largest number) and 2^-20 (inside its subnormal range), the queries
    scaled the other way so that the logits stay those of N(0,1) data.  Every piece is stored relative to a
    per-row power of two, so neither overflows nor loses bits."""
    w = W.make_workload("magnitude", 930 + H, [6000, 300, 9000, 64], H=H)
    f = np.float32(2.0 ** shift)
    kv = W.bf16_bits_to_f32(w.kv_pool)
    fin = np.isfinite(kv)
    w.kv_pool[fin] = W.f32_to_bf16_bits(kv[fin] * f)                 # a power of two: exact in bf16; poison stays poison
    w.q[...] = W.f32_to_bf16_bits(W.bf16_bits_to_f32(w.q) / f)
    ref_o, ref_l = oracle_run(w)
    out, lse = gpu_run(w)
    assert np.isfinite(out).all()
    compare(out / f, lse, ref_o / float(f), ref_l, kv_dtype=0, what=f"values x 2^{shift}")
