"""Pins of the sparse-decode oracle (656-byte rows, a token list per request) against things other
than itself: the dense oracle (already pinned) on a gathered cache whose values the packed rows hit
exactly, closed forms, scale linearity, and the bytes of the row format against the cast of a library."""
import numpy as np
import pytest

import oracle
from paper_2609_37626_b200 import workloads as W

ROW = 656


def exact_rows(rng, n):
    """n packed rows whose dequantised values are exactly representable in bf16: random finite e4m3
    codes, power-of-two block scales (a different one per block), rope = small multiples of a power of two.
    Returns (rows [n][656] uint8, values [n][576] float64)."""
    import torch
    codes = rng.integers(0, 256, size=(n, 512), dtype=np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x3C                      # no NaN codes
    exps = rng.integers(-9, -3, size=(n, 4))
    scales = np.ldexp(np.float32(1.0), exps).astype(np.float32)
    lat = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()      # library decode
    vals = np.empty((n, 576), dtype=np.float64)
    vals[:, :512] = lat * np.repeat(scales.astype(np.float64), 128, axis=1)
    rope = rng.integers(-64, 65, size=(n, 64)).astype(np.float64) / 32.0
    vals[:, 512:] = rope
    rows = np.empty((n, ROW), dtype=np.uint8)
    rows[:, :512] = codes
    rows[:, 512:528] = scales.view(np.uint8).reshape(n, 16)
    rows[:, 528:] = W.f32_to_bf16_bits(rope.astype(np.float32)).view(np.uint8).reshape(n, 128)
    return rows, vals


def paged(rng, rows_per_request, fill=0xFF):
    """Scatter each request's rows over a shuffled pool of 64-row pages."""
    lens = np.array([r.shape[0] for r in rows_per_request], dtype=np.int32)
    ppr = (lens + 63) // 64
    P = int(ppr.sum()) + 3
    order = rng.permutation(P)
    width = rows_per_request[0].shape[1]
    pool = np.full((P, 64, width), fill, dtype=rows_per_request[0].dtype)
    table = np.full((len(lens), max(1, int(ppr.max()))), -1, dtype=np.int32)
    cur = 0
    for i, r in enumerate(rows_per_request):
        for pg in range(int(ppr[i])):
            page = int(order[cur]); cur += 1
            table[i, pg] = page
            chunk = r[64 * pg:64 * pg + 64]
            pool[page, :chunk.shape[0]] = chunk
    return pool, table, lens


def small_q(rng, B, H):
    return W.f32_to_bf16_bits((rng.integers(-8, 9, size=(B, H, 576)) / 4.0).astype(np.float32))


def test_any_selection_equals_the_dense_oracle_on_the_gathered_rows():
    # the listed rows, gathered by hand in list order into a dense bf16 cache that holds the same values
    # exactly: the dense oracle over that cache is the definition of the result
    rng = np.random.Generator(np.random.PCG64(31))
    lens = [1, 64, 65, 300, 130]
    packed, vals = zip(*[exact_rows(rng, n) for n in lens])
    pool, table, seq = paged(rng, list(packed))
    B, H, K = len(lens), 3, 96
    q = small_q(rng, B, H)
    sel = np.full((B, K), -1, dtype=np.int32)
    cnt = np.zeros(B, dtype=np.int32)
    dense_rows = []
    for i, n in enumerate(lens):
        k = min(K, n) if i != 3 else 77
        pick = rng.permutation(n)[:k]
        sel[i, :k] = pick; cnt[i] = k
        dense_rows.append(W.f32_to_bf16_bits(vals[i][pick].astype(np.float32)))
        assert np.array_equal(W.bf16_bits_to_f32(dense_rows[-1]).astype(np.float64), vals[i][pick])     # exact in bf16
    dpool, dtable, dlens = paged(rng, dense_rows, fill=0x7FC0)
    ref_o, ref_l = oracle.mla_decode(q, dpool, dtable, dlens, softmax_scale=0.07)
    o, l = oracle.mla_decode_sparse(q, pool, table, seq, sel, cnt, softmax_scale=0.07)
    assert np.abs(o - ref_o).max() < 1e-12 and np.abs(l - ref_l).max() < 1e-12


def test_one_token_closed_form_and_row_offsets():
    # one listed token: O is that token's latent, LSE its logit; values decoded here from the bytes with
    # numpy / torch views at the offsets of the format
    import torch
    rng = np.random.Generator(np.random.PCG64(32))
    w = W.make_workload("one", 32, [200, 70], H=2, kv_dtype=2)
    sel = np.array([[137], [5]], dtype=np.int32); cnt = np.array([1, 1], dtype=np.int32)
    o, l = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=0.05)
    for i, t in enumerate([137, 5]):
        row = w.kv_pool[w.block_table[i, t // 64], t % 64]
        lat = torch.from_numpy(row[:512].copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
        sc = row[512:528].copy().view(np.float32).astype(np.float64)
        rope = W.bf16_bits_to_f32(row[528:].copy().view(np.uint16)).astype(np.float64)
        k = np.concatenate([lat * np.repeat(sc, 128), rope])
        qf = W.bf16_bits_to_f32(w.q[i]).astype(np.float64)
        assert np.allclose(o[i], np.broadcast_to(k[:512], (2, 512)), rtol=0, atol=1e-13)
        assert np.allclose(l[i], 0.05 * qf @ k, rtol=1e-13, atol=1e-12)


def test_the_scale_of_block_b_multiplies_dims_128b_to_128b_plus_127():
    # tripling the scale of one block: the logits change as if q's block were tripled, O's block triples
    rng = np.random.Generator(np.random.PCG64(33))
    rows, _ = exact_rows(rng, 90)
    pool, table, seq = paged(rng, [rows])
    q = small_q(rng, 1, 2)
    sel = rng.permutation(90)[:40].astype(np.int32)[None]; cnt = np.array([40], dtype=np.int32)
    for b in range(4):
        pool3 = pool.copy()
        sc = pool3[:, :, 512 + 4 * b:516 + 4 * b].copy().view(np.float32)
        pool3[:, :, 512 + 4 * b:516 + 4 * b] = (sc * np.float32(3.0)).view(np.uint8)
        q3 = W.bf16_bits_to_f32(q).copy(); q3[:, :, 128 * b:128 * b + 128] *= 3.0
        o_a, l_a = oracle.mla_decode_sparse(q, pool3, table, seq, sel, cnt, softmax_scale=0.03)
        o_b, l_b = oracle.mla_decode_sparse(W.f32_to_bf16_bits(q3), pool, table, seq, sel, cnt, softmax_scale=0.03)
        o_b[:, :, 128 * b:128 * b + 128] *= 3.0
        assert np.abs(l_a - l_b).max() < 1e-12 and np.abs(o_a - o_b).max() < 1e-12


def test_empty_list_duplicates_order_and_full_list():
    w = W.make_workload("misc", 34, [150, 40, 64], H=2, kv_dtype=2)
    B = 3
    # empty list
    sel = np.zeros((B, 4), dtype=np.int32); cnt = np.array([0, 2, 0], dtype=np.int32)
    o, l = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=0.04)
    assert np.all(o[0] == 0) and np.all(np.isneginf(l[0])) and np.all(o[2] == 0) and np.all(np.isneginf(l[2]))
    # the same token twice: same O, LSE + ln 2
    s1 = np.array([[7], [7], [7]], dtype=np.int32); s2 = np.array([[7, 7]] * 3, dtype=np.int32)
    o1, l1 = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, s1, np.ones(B, np.int32), softmax_scale=0.04)
    o2, l2 = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, s2, np.full(B, 2, np.int32), softmax_scale=0.04)
    assert np.abs(o1 - o2).max() < 1e-13 and np.abs(l2 - l1 - np.log(2.0)).max() < 1e-13
    # order of the list does not matter
    sel, cnt = W.select_tokens(34, w.seq_lens, 32)
    a = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, sel, cnt, softmax_scale=0.04)
    srt = sel.copy()
    for i in range(B):
        srt[i, :cnt[i]] = np.sort(sel[i, :cnt[i]])
    b = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, srt, cnt, softmax_scale=0.04)
    assert np.abs(a[0] - b[0]).max() < 1e-12 and np.abs(a[1] - b[1]).max() < 1e-12
    # entries beyond the count are never read
    junk = sel.copy(); junk[junk < 0] = 10 ** 6
    c = oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, junk, cnt, softmax_scale=0.04)
    assert np.array_equal(a[0], c[0])


def test_an_index_outside_the_request_is_rejected():
    w = W.make_workload("bad", 35, [50], H=1, kv_dtype=2)
    for t in (-1, 50):
        with pytest.raises(ValueError):
            oracle.mla_decode_sparse(w.q, w.kv_pool, w.block_table, w.seq_lens, np.array([[t]], np.int32), np.array([1], np.int32),
                                     softmax_scale=0.1)


def test_generator_rows_decode_close_to_what_was_packed_and_selection_is_a_subset():
    rng = np.random.Generator(np.random.PCG64(36))
    x = rng.standard_normal((50, 576), dtype=np.float32)
    x[7, 128:256] = 0.0                                       # an all-zero block: scale 1
    rows = W.pack_sparse_rows(x)
    assert rows.shape == (50, ROW)
    import torch
    lat = torch.from_numpy(rows[:, :512].copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    sc = rows[:, 512:528].copy().view(np.float32)
    assert sc[7, 1] == 1.0 and np.all(sc > 0)
    deq = lat * np.repeat(sc, 128, axis=1)
    assert np.abs(deq - x[:, :512]).max() <= np.abs(x).max() / 16 + 1e-6      # e4m3: 3 mantissa bits
    assert np.abs(lat).max() <= 448.0
    rope = W.bf16_bits_to_f32(rows[:, 528:].copy().view(np.uint16))
    assert np.abs(rope - x[:, 512:]).max() <= np.abs(x).max() / 256
    sel, cnt = W.select_tokens(36, [10, 5000, 0, 2048], 2048)
    assert list(cnt) == [10, 2048, 0, 2048]
    for i, s in enumerate([10, 5000, 0, 2048]):
        v = sel[i, :cnt[i]]
        assert len(set(v.tolist())) == cnt[i] and (cnt[i] == 0 or (v.min() >= 0 and v.max() < s))
        assert np.all(sel[i, cnt[i]:] == -1)
