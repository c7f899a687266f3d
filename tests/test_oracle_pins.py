"""Pins for the CPU oracle: closed forms, invariants, a dense library attention,
brute force in high precision, the e4m3 code table, merge and migrate laws.

None of these call the CUDA path.  Each is chosen so that a plausible slip in the
oracle (dropped rope columns, V taken from the wrong columns, a wrong scale or
sign, a transposed operand, a paging or range off-by-one) fails at least one.
"""
import math

import mpmath
import numpy as np
import pytest
import torch

import oracle
from paper_2609_37626_b200 import workloads as W

SCALE = W.SOFTMAX_SCALE


def f32(bits):
    return W.bf16_bits_to_f32(bits).astype(np.float64)


def dense_rows(w, i):
    """Gather request i's cache rows into a dense fp64 [s][576] matrix."""
    s = int(w.seq_lens[i])
    rows = np.empty((s, W.D_QK), dtype=np.float64)
    for t in range(s):
        page = w.block_table[i, t // 64]
        if w.kv_dtype == 0:
            rows[t] = f32(w.kv_pool[page, t % 64])
        else:
            codes = torch.from_numpy(w.kv_pool[page, t % 64].copy()).view(torch.float8_e4m3fn)
            rows[t] = codes.to(torch.float64).numpy() * float(w.kv_scales[page, t % 64])
    return rows


def run(w, **kw):
    args = dict(softmax_scale=w.softmax_scale, kv_scales=w.kv_scales, head_begin=w.head_begin,
                head_end=w.head_end, kv_begin=w.kv_begin, kv_end=w.kv_end)
    args.update(kw)
    return oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, **args)


# ---------------------------------------------------------------- e4m3 table
def test_e4m3_table_matches_library_decode():
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for c in range(256):
        v = oracle.e4m3_to_double(c)
        if c in (0x7F, 0xFF):
            assert math.isnan(v) and math.isnan(lib[c])
        else:
            assert v == lib[c], c
    assert oracle.e4m3_to_double(0x7E) == 448.0
    assert oracle.e4m3_to_double(0x01) == 2.0 ** -9
    assert oracle.e4m3_to_double(0x08) == 2.0 ** -6
    assert oracle.e4m3_to_double(0x80 | 0x38) == -1.0


def test_e4m3_encode_decode_identity_on_finite_codes():
    finite = np.array([c for c in range(256) if c not in (0x7F, 0xFF)], dtype=np.uint8)
    vals = np.array([oracle.e4m3_to_double(int(c)) for c in finite], dtype=np.float32)
    back = torch.from_numpy(vals).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    # +0 and -0 keep their own codes
    assert np.array_equal(back, finite)


# ---------------------------------------------------------------- closed forms
def test_context_of_one_returns_v0():
    w = W.make_workload("one", 11, [1, 1, 1], H=4)
    out, lse = run(w)
    for i in range(3):
        row = dense_rows(w, i)[0]
        for g in range(4):
            assert np.array_equal(out[i, g], row[:512])
            ref = SCALE * math.fsum(f32(w.q[i, g]) * row)
            assert abs(lse[i, g] - ref) <= 1e-12 * max(1.0, abs(ref))


def test_two_tokens_sigmoid_form():
    w = W.make_workload("two", 12, [2], H=8)
    out, lse = run(w)
    rows = dense_rows(w, 0)
    for g in range(8):
        qv = f32(w.q[0, g])
        l0 = SCALE * math.fsum(qv * rows[0])
        l1 = SCALE * math.fsum(qv * rows[1])
        s0 = 1.0 / (1.0 + math.exp(l1 - l0))
        ref = s0 * rows[0, :512] + (1.0 - s0) * rows[1, :512]
        assert np.allclose(out[0, g], ref, rtol=0, atol=1e-13)
        assert abs(lse[0, g] - (max(l0, l1) + math.log1p(math.exp(-abs(l0 - l1))))) < 1e-12


def test_zero_query_gives_mean_of_v_and_log_n():
    w = W.make_workload("q0", 13, [37, 130], H=3)
    w.q[...] = 0
    out, lse = run(w)
    for i, n in enumerate([37, 130]):
        rows = dense_rows(w, i)
        for g in range(3):
            assert np.allclose(out[i, g], rows[:, :512].mean(axis=0), rtol=0, atol=1e-13)
            assert abs(lse[i, g] - math.log(n)) < 1e-13


def test_zero_scale_gives_mean_and_log_n():
    w = W.make_workload("s0", 14, [70], H=2)
    out, lse = run(w, softmax_scale=0.0)
    rows = dense_rows(w, 0)
    assert np.allclose(out[0, 0], rows[:, :512].mean(axis=0), rtol=0, atol=1e-13)
    assert abs(lse[0, 1] - math.log(70)) < 1e-13


def test_identical_v_rows_return_that_row():
    w = W.make_workload("same", 15, [100], H=4)
    # same latent part in every token, different rope part: weights differ, O does not
    first = w.kv_pool[w.block_table[0, 0], 0, :512].copy()
    for t in range(100):
        w.kv_pool[w.block_table[0, t // 64], t % 64, :512] = first
    out, _ = run(w)
    for g in range(4):
        assert np.allclose(out[0, g], f32(first), rtol=0, atol=1e-14)


def test_dominant_key_selects_its_row():
    w = W.make_workload("dom", 16, [90], H=2)
    # token 41's row := 8 * q of head 0 (exact in bf16: a power-of-two multiple)
    qv = W.bf16_bits_to_f32(w.q[0, 0])
    w.kv_pool[w.block_table[0, 0], 41] = W.f32_to_bf16_bits(qv * np.float32(8.0))
    out, lse = run(w)
    # logit of token 41 ~ 8*|q|^2/sqrt(192) ~ 330, the rest are O(10)
    assert np.allclose(out[0, 0], 8.0 * qv[:512].astype(np.float64), rtol=0, atol=1e-12)
    assert abs(lse[0, 0] - SCALE * 8.0 * math.fsum(qv.astype(np.float64) ** 2)) < 1e-9


# ---------------------------------------------------------------- several causal query rows per request
def run_rows(w, q4, **kw):
    args = dict(softmax_scale=w.softmax_scale, kv_scales=w.kv_scales, head_begin=w.head_begin,
                head_end=w.head_end, kv_begin=w.kv_begin, kv_end=w.kv_end)
    args.update(kw)
    return oracle.mla_decode_rows(q4, w.kv_pool, w.block_table, w.seq_lens, **args)


@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_rows_one_row_is_plain_decode(kv_dtype):
    w = W.make_workload("rows1", 61 + kv_dtype, [1, 64, 130], H=5, kv_dtype=kv_dtype)
    out, lse = run(w)
    out4, lse4 = run_rows(w, np.ascontiguousarray(w.q[:, :, None, :]))
    assert np.array_equal(out4[:, :, 0], out) and np.array_equal(lse4[:, :, 0], lse)


@pytest.mark.parametrize("R", [2, 3, 8])
def test_rows_each_row_is_plain_decode_over_its_causal_prefix(R):
    # row r of an R-row call = the one-row decode of the same query over the first s - (R-1-r) tokens:
    # reduces every row to the single-row oracle pinned above (bit for bit, same loops)
    lens = [R, R + 1, 64, 65, 200]
    w = W.make_workload("rowsR", 63 + R, lens, H=3)
    q4 = W.make_query_rows(63 + R, w.B, w.H, R)
    out4, lse4 = run_rows(w, q4)
    for r in range(R):
        shorter = (w.seq_lens - (R - 1 - r)).astype(np.int32)
        o, l = oracle.mla_decode(np.ascontiguousarray(q4[:, :, r]), w.kv_pool, w.block_table, shorter,
                                 softmax_scale=w.softmax_scale)
        assert np.array_equal(out4[:, :, r], o) and np.array_equal(lse4[:, :, r], l)


def test_rows_match_dense_causal_library_attention():
    R = 4
    w = W.make_workload("rowslib", 67, [4, 70, 131], H=4)
    q4 = W.make_query_rows(67, w.B, w.H, R)
    out4, lse4 = run_rows(w, q4)
    for i in range(w.B):
        rows = torch.from_numpy(dense_rows(w, i)); s = rows.shape[0]
        q = torch.from_numpy(f32(q4[i]))                              # [H][R][576]
        mask = torch.arange(s)[None, :] <= (s - R + torch.arange(R))[:, None]      # row r sees tokens <= its position
        ref = torch.nn.functional.scaled_dot_product_attention(
            q[None], rows[None, None].expand(1, w.H, -1, -1),
            torch.nn.functional.pad(rows[:, :512], (0, 64))[None, None].expand(1, w.H, -1, -1),
            attn_mask=mask, scale=SCALE)[0, :, :, :512].numpy()
        assert np.allclose(out4[i], ref, rtol=0, atol=1e-12)
        logits = SCALE * torch.einsum("hrd,td->hrt", q, rows).masked_fill(~mask[None], -math.inf)
        assert np.allclose(lse4[i], torch.logsumexp(logits, dim=2).numpy(), rtol=0, atol=1e-12)


def test_rows_first_row_of_a_fresh_request_sees_one_token_and_ranges_can_empty_a_row():
    R = 3
    w = W.make_workload("rowsedge", 69, [3, 100], H=2)
    q4 = W.make_query_rows(69, w.B, w.H, R)
    out4, lse4 = run_rows(w, q4)
    # request 0 has exactly R tokens: row 0 attends token 0 only -> O = that row's latent part, LSE = scale q.k
    k0 = f32(w.kv_pool[w.block_table[0, 0], 0])
    for g in range(w.H):
        assert np.array_equal(out4[0, g, 0], k0[:512])
        assert abs(lse4[0, g, 0] - SCALE * float(f32(q4[0, g, 0]) @ k0)) < 1e-12
    # a range that starts at the last token: only the last row has anything to attend
    kb = (w.seq_lens - 1).astype(np.int32)
    out4, lse4 = run_rows(w, q4, kv_begin=kb)
    assert np.all(np.isneginf(lse4[:, :, : R - 1])) and np.all(out4[:, :, : R - 1] == 0.0)
    assert np.all(np.isfinite(lse4[:, :, R - 1]))
    # fewer tokens than rows: the oldest rows have an empty range
    w1 = W.make_workload("rowsshort", 70, [2], H=2)
    o, l = run_rows(w1, W.make_query_rows(70, 1, 2, 4))
    assert np.all(np.isneginf(l[0, :, :2])) and np.all(np.isfinite(l[0, :, 2:]))


# ---------------------------------------------------------------- library and brute force
@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_matches_dense_library_attention(kv_dtype):
    w = W.make_workload("lib", 21 + kv_dtype, [1, 63, 64, 65, 129, 300], H=6, kv_dtype=kv_dtype)
    out, lse = run(w)
    for i in range(w.B):
        rows = torch.from_numpy(dense_rows(w, i))
        q = torch.from_numpy(f32(w.q[i]))                       # [H][576]
        ref = torch.nn.functional.scaled_dot_product_attention(
            q[None, :, None, :], rows[None, None, :, :].expand(1, w.H, -1, -1),
            torch.nn.functional.pad(rows[:, :512], (0, 64))[None, None].expand(1, w.H, -1, -1),
            scale=SCALE)[0, :, 0, :512].numpy()
        assert np.allclose(out[i], ref, rtol=0, atol=1e-12)
        ref_lse = torch.logsumexp(SCALE * (q @ rows.T), dim=1).numpy()
        assert np.allclose(lse[i], ref_lse, rtol=0, atol=1e-12)


def test_config1_brute_force_high_precision():
    """Config 1 as specified (4 requests, lengths 1/17/64/200, 16 heads, 16-page
    pool), every output against 40-digit arithmetic written with plain loops."""
    w = W.config(1)
    assert list(w.seq_lens) == [1, 17, 64, 200] and w.kv_pool.shape[0] == 16
    out, lse = run(w)
    mpmath.mp.dps = 40
    sc = mpmath.mpf(1) / mpmath.sqrt(192)
    worst_o, worst_l = 0.0, 0.0
    for i in range(4):
        rows = dense_rows(w, i)
        for g in (0, 7, 15):
            qv = f32(w.q[i, g])
            logits = []
            for t in range(rows.shape[0]):
                acc = mpmath.mpf(0)
                for d in range(576):
                    acc += mpmath.mpf(float(qv[d])) * mpmath.mpf(float(rows[t, d]))
                logits.append(sc * acc)
            Z = sum(mpmath.exp(l) for l in logits)
            worst_l = max(worst_l, abs(float(mpmath.log(Z) - mpmath.mpf(float(lse[i, g])))))
            for d in (0, 1, 255, 511):
                o = sum(mpmath.exp(l) * mpmath.mpf(float(rows[t, d])) for t, l in enumerate(logits)) / Z
                worst_o = max(worst_o, abs(float(o - mpmath.mpf(float(out[i, g, d])))))
    # fp64 accumulation of <= 576 products and <= 200 weights; the softmax scale the
    # oracle receives is the fp64 value of 1/sqrt(192)
    assert worst_o < 1e-13 and worst_l < 1e-12


def test_softmax_weights_sum_to_one():
    # V columns all equal to 1 -> O must be exactly the sum of the weights
    w = W.make_workload("ones", 23, [250], H=5)
    one = W.f32_to_bf16_bits(np.ones(512, dtype=np.float32))
    for t in range(250):
        w.kv_pool[w.block_table[0, t // 64], t % 64, :512] = one
    out, _ = run(w)
    assert np.allclose(out[0], 1.0, rtol=0, atol=1e-14)


# ---------------------------------------------------------------- invariants
def test_key_shift_leaves_o_and_shifts_lse():
    w = W.make_workload("shift", 31, [77], H=3)
    out0, lse0 = run(w)
    # add c to the rope columns of every key (rope columns are not part of V)
    c = np.zeros(576, dtype=np.float32)
    c[512:] = np.arange(64, dtype=np.float32) / 8.0 - 4.0      # exactly representable
    w2 = W.make_workload("shift", 31, [77], H=3)
    for t in range(77):
        p, s = w2.block_table[0, t // 64], t % 64
        # keep the sum exact in bf16: use rope values rounded to multiples of 1/8 first
        base = np.round(W.bf16_bits_to_f32(w2.kv_pool[p, s]) * 8.0) / 8.0
        w.kv_pool[p, s, 512:] = W.f32_to_bf16_bits(base)[512:]
        w2.kv_pool[p, s, 512:] = W.f32_to_bf16_bits(base + c)[512:]
    out0, lse0 = run(w)
    out1, lse1 = run(w2)
    assert np.allclose(out0, out1, rtol=0, atol=1e-12)
    for g in range(3):
        shift = SCALE * math.fsum(f32(w.q[0, g]) * c.astype(np.float64))
        assert abs((lse1[0, g] - lse0[0, g]) - shift) < 1e-11


def test_rope_columns_enter_logits_but_not_v():
    w = W.make_workload("rope", 32, [150], H=4, rope_scale=2.0)
    out, lse = run(w)
    rows = dense_rows(w, 0)
    # reference with all 576 columns in the logits and the first 512 as V
    for g in range(4):
        l = SCALE * rows @ f32(w.q[0, g])
        p = np.exp(l - l.max())
        p /= p.sum()
        assert np.allclose(out[0, g], p @ rows[:, :512], rtol=0, atol=1e-13)
        # and dropping the rope columns from the logits changes the answer
        l2 = SCALE * rows[:, :512] @ f32(w.q[0, g, :512])
        p2 = np.exp(l2 - l2.max()); p2 /= p2.sum()
        assert np.abs(out[0, g] - p2 @ rows[:, :512]).max() > 1e-3
    # zero rope part of q -> result independent of the cache's rope columns
    w.q[:, :, 512:] = 0
    a, la = run(w)
    w.kv_pool[:, :, 512:] = W.f32_to_bf16_bits(np.float32(3.0) * np.ones(1, np.float32))[0]
    b, lb = run(w)
    assert np.array_equal(a, b) and np.array_equal(la, lb)


def test_token_permutation_invariance():
    w = W.make_workload("perm", 33, [128], H=3, placement="identity", pool_pages=2, poison=False)
    out0, lse0 = run(w)
    flat = w.kv_pool.reshape(128, 576)
    perm = np.random.default_rng(5).permutation(128)
    w.kv_pool = flat[perm].reshape(2, 64, 576).copy()
    out1, lse1 = run(w)
    assert np.allclose(out0, out1, rtol=0, atol=1e-13) and np.allclose(lse0, lse1, rtol=0, atol=1e-13)


def test_page_placement_and_pool_size_do_not_matter():
    lens = [5, 64, 191, 260]
    a = W.make_workload("place", 34, lens, H=4, placement="identity", pool_factor=1.0)
    b = W.make_workload("place", 34, lens, H=4, placement="permute", pool_factor=1.25)
    c = W.make_workload("place", 34, lens, H=4, placement="reversed", pool_factor=2.0)
    ra, rb, rc = run(a), run(b), run(c)
    for x, y in zip(ra, rb):
        assert np.array_equal(x, y)
    for x, y in zip(ra, rc):
        assert np.array_equal(x, y)
    # and the table really is what maps tokens to rows: breaking it changes the result
    b.block_table[3, [0, 1]] = b.block_table[3, [1, 0]]
    out_swapped, _ = run(b)
    assert np.allclose(out_swapped[3], ra[0][3], atol=1e-12)      # swapping whole pages = permuting tokens
    b.block_table[3, 0] = b.block_table[1, 0]                      # pointing at another request's (full) page is not
    assert np.abs(run(b)[0][3] - ra[0][3]).max() > 1e-3


def test_head_and_request_slices_concatenate_bit_identically():
    w = W.make_workload("slices", 35, [30, 100, 200], H=16)
    full_o, full_l = run(w)
    o = np.full_like(full_o, np.nan); l = np.full_like(full_l, np.nan)
    for hb in range(0, 16, 4):
        run(w, head_begin=hb, head_end=hb + 4, out=o, lse=l)
    assert np.array_equal(o, full_o) and np.array_equal(l, full_l)
    # a slice call leaves everything outside the slice untouched
    o2 = np.full_like(full_o, 7.0); l2 = np.full_like(full_l, 7.0)
    run(w, head_begin=4, head_end=8, out=o2, lse=l2)
    assert np.all(o2[:, :4] == 7.0) and np.all(o2[:, 8:] == 7.0) and np.all(l2[:, 8:] == 7.0)
    # request slices: each request alone
    for i in range(3):
        oi, li = oracle.mla_decode(w.q[i:i + 1], w.kv_pool, w.block_table[i:i + 1], w.seq_lens[i:i + 1],
                                   softmax_scale=SCALE)
        assert np.array_equal(oi[0], full_o[i]) and np.array_equal(li[0], full_l[i])
    # explicit (request, head) pair lists agree too
    op, lp = run(w, pairs=[[2, 5], [0, 15]])
    assert np.array_equal(op[2, 5], full_o[2, 5]) and np.array_equal(lp[0, 15], full_l[0, 15])
    assert np.isnan(op[1]).all()


@pytest.mark.parametrize("cuts", [[0, 25, 50, 75, 100, 125, 150, 175, 200], [0, 1, 63, 200], [0, 64, 65, 200]])
def test_kv_ranges_merge_to_unsplit(cuts):
    w = W.make_workload("cp", 36, [200, 90], H=4)
    full_o, full_l = run(w)
    po, pl = [], []
    for a, b in zip(cuts[:-1], cuts[1:]):
        o, l = run(w, kv_begin=np.array([a, a], np.int32), kv_end=np.array([b, b], np.int32))
        po.append(o.reshape(-1, 512)); pl.append(l.reshape(-1))
    mo, ml = oracle.lse_merge(np.stack(po), np.stack(pl))
    assert np.allclose(mo, full_o.reshape(-1, 512), rtol=0, atol=1e-12)
    assert np.allclose(ml, full_l.reshape(-1), rtol=0, atol=1e-12)


def test_ranges_are_clipped_and_empty_ranges_are_neutral():
    w = W.make_workload("clip", 37, [100], H=2)
    full = run(w)
    clipped = run(w, kv_begin=np.array([-5], np.int32), kv_end=np.array([1000], np.int32))
    assert np.array_equal(full[0], clipped[0]) and np.array_equal(full[1], clipped[1])
    for a, b in ([50, 50], [70, 30], [100, 200]):
        o, l = run(w, kv_begin=np.array([a], np.int32), kv_end=np.array([b], np.int32))
        assert np.all(o == 0.0) and np.all(np.isneginf(l))
    w0 = W.make_workload("zero", 38, [0, 3], H=2)
    o, l = run(w0)
    assert np.all(o[0] == 0.0) and np.all(np.isneginf(l[0])) and np.all(np.isfinite(l[1]))
    # a range of one token is that token's V row
    o, l = run(w, kv_begin=np.array([64], np.int32), kv_end=np.array([65], np.int32))
    assert np.array_equal(o[0, 0], dense_rows(w, 0)[64, :512])


def test_poison_is_never_read():
    a = W.make_workload("poison", 39, [1, 70, 129], H=3, poison=True)
    b = W.make_workload("poison", 39, [1, 70, 129], H=3, poison=False)
    ra, rb = run(a), run(b)
    assert np.isfinite(ra[0]).all() and np.array_equal(ra[0], rb[0]) and np.array_equal(ra[1], rb[1])
    f = W.make_workload("poison8", 40, [3, 100], H=2, kv_dtype=1, poison=True)
    assert np.isfinite(run(f)[0]).all()


def test_gaussian_limit_sanity():
    """Loose statistical check at a size where brute force is slow: for i.i.d.
    N(0, sigma_d^2) key columns, LSE -> ln n + scale^2/2 * sum sigma_d^2 q_d^2 and
    O -> scale * q[:512] (sigma = 1 on the latent columns)."""
    w = W.make_workload("limit", 41, [32768], H=2, rope_scale=2.0)
    out, lse = run(w)
    for g in range(2):
        qv = f32(w.q[0, g])
        sig2 = np.ones(576); sig2[512:] = 4.0
        lim = math.log(32768) + 0.5 * SCALE ** 2 * float((sig2 * qv ** 2).sum())
        assert abs(lse[0, g] - lim) < 0.3
        assert np.sqrt(np.mean((out[0, g] - SCALE * qv[:512]) ** 2)) < 0.1


# ---------------------------------------------------------------- merge laws
def test_merge_laws():
    rng = np.random.default_rng(3)
    o = rng.standard_normal((3, 5, 512)); l = rng.standard_normal((3, 5))
    # one part: identity
    a, b = oracle.lse_merge(o[:1], l[:1])
    assert np.allclose(a, o[0], atol=1e-15) and np.allclose(b, l[0], atol=1e-15)
    # two equal parts: (O, L + ln 2)
    a, b = oracle.lse_merge(np.stack([o[0], o[0]]), np.stack([l[0], l[0]]))
    assert np.allclose(a, o[0], atol=1e-15) and np.allclose(b, l[0] + math.log(2), atol=1e-14)
    # -inf part ignored, all -inf gives (0, -inf) without NaN
    linf = l.copy(); linf[1] = -np.inf
    oinf = o.copy(); oinf[1] = np.nan
    a, b = oracle.lse_merge(oinf, linf)
    a2, b2 = oracle.lse_merge(o[[0, 2]], l[[0, 2]])
    assert np.array_equal(a, a2) and np.array_equal(b, b2)
    a, b = oracle.lse_merge(oinf[1:2], linf[1:2])
    assert np.all(a == 0.0) and np.all(np.isneginf(b))
    # associativity: merge(merge(0,1),2) == merge(0,1,2)
    m01 = oracle.lse_merge(o[:2], l[:2])
    left = oracle.lse_merge(np.stack([m01[0], o[2]]), np.stack([m01[1], l[2]]))
    allp = oracle.lse_merge(o, l)
    assert np.allclose(left[0], allp[0], atol=1e-14) and np.allclose(left[1], allp[1], atol=1e-14)
    # explicit formula on one row
    w = np.exp(l[:, 0]); ref = (w[:, None] * o[:, 0]).sum(0) / w.sum()
    assert np.allclose(allp[0][0], ref, atol=1e-14) and abs(allp[1][0] - math.log(w.sum())) < 1e-14


# ---------------------------------------------------------------- migrate
@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_migrate_bytes_table_and_decode(kv_dtype):
    w = W.make_workload("mig", 51 + kv_dtype, [10, 64, 300, 129], H=4, kv_dtype=kv_dtype, extra_pool_pages=8)
    n_src = w.num_pool_pages - 8
    # a page shared by two requests (prefix sharing): both entries must be rewritten
    w.block_table[0, 0] = w.block_table[1, 0]
    before = run(w)
    src_ids, dst_ids = W.migration_plan(99, np.unique(w.block_table[w.block_table >= 0]), 8, fraction=0.5)
    pool0 = w.kv_pool.copy(); table0 = w.block_table.copy()
    sc0 = None if w.kv_scales is None else w.kv_scales.copy()
    src_pool, dst_pool = w.kv_pool[:n_src], w.kv_pool[n_src:]
    src_sc = None if sc0 is None else w.kv_scales[:n_src]
    dst_sc = None if sc0 is None else w.kv_scales[n_src:]
    oracle.kv_page_migrate(src_pool, dst_pool, src_ids, dst_ids, w.block_table,
                           src_scales=src_sc, dst_scales=dst_sc, src_id_base=0, dst_id_base=n_src)
    # bytes: moved pages equal their sources, every other byte untouched
    moved = np.zeros(w.num_pool_pages, bool)
    for s, d in zip(src_ids, dst_ids):
        assert np.array_equal(w.kv_pool[n_src + d], pool0[s])
        if sc0 is not None:
            assert np.array_equal(w.kv_scales[n_src + d].view(np.uint32), sc0[s].view(np.uint32))
        moved[n_src + d] = True
    assert np.array_equal(w.kv_pool[~moved].view(np.uint8), pool0[~moved].view(np.uint8))
    if sc0 is not None:
        assert np.array_equal(w.kv_scales[~moved].view(np.uint32), sc0[~moved].view(np.uint32))
    # table: plain-python remap
    remap = {int(s): int(n_src + d) for s, d in zip(src_ids, dst_ids)}
    expect = np.array([[remap.get(int(e), int(e)) for e in row] for row in table0], dtype=np.int32)
    assert np.array_equal(w.block_table, expect)
    assert w.block_table[0, 0] == w.block_table[1, 0]
    # histories preserved: poison the vacated pages, decode again, bit-identical
    w.kv_pool[src_ids] = W.BF16_NAN if kv_dtype == 0 else W.E4M3_NAN
    after = run(w)
    assert np.array_equal(before[0], after[0]) and np.array_equal(before[1], after[1])


def test_migrate_nothing_is_a_no_op():
    w = W.make_workload("mig0", 53, [100], H=2, extra_pool_pages=2)
    pool0, table0 = w.kv_pool.copy(), w.block_table.copy()
    oracle.kv_page_migrate(w.kv_pool[:-2], w.kv_pool[-2:], np.zeros(0, np.int32), np.zeros(0, np.int32),
                           w.block_table, dst_id_base=w.num_pool_pages - 2)
    assert np.array_equal(pool0.view(np.uint8), w.kv_pool.view(np.uint8)) and np.array_equal(table0, w.block_table)
