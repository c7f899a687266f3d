"""GPU parity when the cache rows NEXT to a request's KV range hold NaN / Inf.

A position-sharded rank owns only its tokens of a boundary page (App. E); the other slots of
that page, although below seq_lens[i], hold whatever was there.  The definition ignores every
byte outside the range, so must the CUDA path: a masked token's weight is 0, and 0 x NaN inside
the P.V contraction would still be NaN.  Every kernel path is driven over ranges that lie
strictly inside one page, touch one page edge, straddle page edges with both ends unaligned,
and hold a single token, with every in-seq_len slot outside the range poisoned."""
import numpy as np
import pytest

import oracle
from paper_2609_37626_b200 import workloads as W
from _util import compare, gpu_run, oracle_run
from test_rows_gpu import compare_rows, gpu_rows

pytestmark = pytest.mark.gpu

# (context length, kv_begin, kv_end): inside the first page; inside a middle page; inside the last, ragged page;
# one token; ending at a page edge; starting at one; across one edge; across several; the whole context;
# ending inside the ragged tail page; a range that reaches beyond the context
CASES = [(64, 3, 40), (200, 70, 100), (200, 193, 199), (500, 130, 131), (300, 70, 128), (300, 128, 170),
         (300, 50, 90), (1000, 10, 700), (150, 0, 150), (150, 129, 149), (90, 65, 4000), (70, 1, 63)]


def make(H, kv_dtype, seed, head_begin=0, head_end=None):
    lens = [c[0] for c in CASES]
    w = W.make_workload("neighbours", seed, lens, H=H, kv_dtype=kv_dtype, head_begin=head_begin, head_end=head_end)
    kb = np.array([c[1] for c in CASES], np.int32)
    ke = np.array([c[2] for c in CASES], np.int32)
    W.poison_outside_ranges(w, kb, ke)
    return w, kb, ke


# bf16: 16 / 32 / 64 heads per CTA, the CTA-pair kernel (128), two independent 64-head CTAs (flag 2), SIMT (flag 1)
@pytest.mark.parametrize("H,flags", [(16, 0), (32, 0), (64, 0), (128, 0), (128, 2), (16, 1), (80, 0)])
def test_bf16_ranges_with_poisoned_neighbours(H, flags):
    import torch
    w, kb, ke = make(H, 0, 4100 + H + flags)
    ref = oracle_run(w, kv_begin=kb, kv_end=ke)
    out, lse = gpu_run(w, flags=flags, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    compare(out, lse, *ref, kv_dtype=0, what=f"bf16 H={H} flags={flags}")


# e4m3: 16 / 32 / 64 heads per CTA (24 and 40 pad their group), the CTA-pair kernel, two independent CTAs, SIMT
@pytest.mark.parametrize("H,flags", [(16, 0), (24, 0), (32, 0), (40, 0), (64, 0), (128, 0), (128, 2), (16, 1), (96, 0)])
def test_e4m3_ranges_with_poisoned_neighbours(H, flags):
    import torch
    w, kb, ke = make(H, 1, 4200 + H + flags)
    ref = oracle_run(w, kv_begin=kb, kv_end=ke)
    out, lse = gpu_run(w, flags=flags, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    compare(out, lse, *ref, kv_dtype=1, what=f"e4m3 H={H} flags={flags}")


# several causal query rows per request (the CTA-pair kernels whatever the width, or SIMT)
@pytest.mark.parametrize("kv_dtype", [0, 1])
@pytest.mark.parametrize("R,H,flags", [(2, 16, 0), (4, 32, 0), (2, 64, 0), (3, 16, 1)])
def test_rows_ranges_with_poisoned_neighbours(kv_dtype, R, H, flags):
    import torch
    w, kb, ke = make(H, kv_dtype, 4300 + H + R)
    q4 = W.make_query_rows(4300 + H + R, w.B, H, R)
    ref = oracle.mla_decode_rows(q4, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                                 kv_scales=w.kv_scales, kv_begin=kb, kv_end=ke)
    out, lse = gpu_rows(w, q4, flags=flags, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
    compare_rows(out, lse, *ref, kv_dtype, 0, H, f"rows R={R} H={H} dtype={kv_dtype}")


def test_slice_of_a_wider_layer_with_poisoned_neighbours():
    import torch
    for kv_dtype in (0, 1):
        w, kb, ke = make(128, kv_dtype, 4400 + kv_dtype, head_begin=24, head_end=120)
        ref = oracle_run(w, kv_begin=kb, kv_end=ke)
        out, lse = gpu_run(w, sentinel=4.0, kv_begin=torch.from_numpy(kb).cuda(), kv_end=torch.from_numpy(ke).cuda())
        compare(out, lse, *ref, kv_dtype=kv_dtype, rows=[(i, g) for i in range(w.B) for g in range(24, 120)], what="slice")
        assert np.all(out[:, :24] == 4.0) and np.all(out[:, 120:] == 4.0)
