"""Pins of the DOP layout-change oracle (no GPU): a simulated exchange among T ranks must turn
head slices of all rows into all heads of the owned rows and back (App. E: packing preserves row
identity, head order and positions; ranks that own no rows still take part)."""
import numpy as np
import pytest

import oracle


def owners_and_order(rng, N, T, empty_owner=None):
    owner = rng.integers(0, T, size=N)
    if empty_owner is not None:
        owner[owner == empty_owner] = (empty_owner + 1) % T
    send_row = np.argsort(owner, kind="stable").astype(np.int32)      # rows grouped by owner, original order inside
    counts = np.bincount(owner, minlength=T)
    return owner, send_row, counts


@pytest.mark.parametrize("N,T,h,empty", [(13, 4, 3, None), (40, 8, 2, 5), (1, 2, 4, None), (0, 4, 2, None)])
def test_exchange_round_trip(N, T, h, empty):
    rng = np.random.Generator(np.random.PCG64(900 + N + T))
    H = T * h
    full_nope = rng.integers(0, 2 ** 16, size=(N, H, 8), dtype=np.uint16)     # stands for [N][H][512]
    full_rope = rng.integers(0, 2 ** 16, size=(N, H, 3), dtype=np.uint16)     # stands for [N][H][64]
    owner, send_row, counts = owners_and_order(rng, N, T, empty)
    offs = np.concatenate(([0], np.cumsum(counts)))
    # every rank packs its head slice of ALL rows, grouped by owner
    send = [oracle.dop_pack_rows(full_nope[:, s * h:(s + 1) * h], full_rope[:, s * h:(s + 1) * h], send_row) for s in range(T)]
    for o in range(T):
        n = counts[o]
        # the all-to-all: owner o receives from every source s the rows it owns
        recv = np.stack([send[s][offs[o]:offs[o + 1]] for s in range(T)]) if n else np.zeros((T, 0, h, 11), np.uint16)
        q_owner = oracle.dop_swap_outer(recv).reshape(n, H, 11)
        rows = send_row[offs[o]:offs[o + 1]]
        assert np.array_equal(q_owner[:, :, :8], full_nope[rows]) and np.array_equal(q_owner[:, :, 8:], full_rope[rows])
        assert np.array_equal(owner[rows], np.full(n, o)) and np.all(np.diff(rows) > 0)       # identity and order
    # reverse exchange of an all-head result of the owners back to global-row, local-head order
    full_out = rng.integers(0, 2 ** 16, size=(N, H, 5), dtype=np.uint16)
    back = [np.zeros((N, h, 5), np.uint16) for _ in range(T)]
    recv_rows = [[] for _ in range(T)]
    for o in range(T):
        rows = send_row[offs[o]:offs[o + 1]]
        per_source = oracle.dop_swap_outer(full_out[rows].reshape(counts[o], T, h, 5))        # [T][n][h][5]
        for s in range(T):
            recv_rows[s].append(per_source[s])
    for s in range(T):
        recv = np.concatenate(recv_rows[s]) if N else np.zeros((0, h, 5), np.uint16)
        back[s] = oracle.dop_unpack_rows(recv, send_row, N)
        assert np.array_equal(back[s], full_out[:, s * h:(s + 1) * h])


def test_pack_is_the_indexing_expression_and_unpack_its_inverse():
    rng = np.random.Generator(np.random.PCG64(911))
    a = rng.integers(0, 255, size=(9, 2, 6), dtype=np.uint8); b = rng.integers(0, 255, size=(9, 2, 2), dtype=np.uint8)
    perm = rng.permutation(9).astype(np.int32)
    packed = oracle.dop_pack_rows(a, b, perm)
    assert np.array_equal(packed, np.concatenate((a[perm], b[perm]), axis=-1))
    assert np.array_equal(oracle.dop_unpack_rows(packed, perm, 9), np.concatenate((a, b), axis=-1))
    sub = perm[:4]                                           # a subset of the rows: the others stay untouched
    keep = np.full((9, 2, 8), 7, np.uint8)
    got = oracle.dop_unpack_rows(packed[:4], sub, 9, out=keep.copy())
    mask = np.zeros(9, bool); mask[sub] = True
    assert np.array_equal(got[mask], np.concatenate((a, b), axis=-1)[mask]) and np.all(got[~mask] == 7)
    x = rng.integers(0, 255, size=(3, 5, 2, 4), dtype=np.uint8)
    assert np.array_equal(oracle.dop_swap_outer(x), x.transpose(1, 0, 2, 3))
    assert np.array_equal(oracle.dop_swap_outer(oracle.dop_swap_outer(x)), x)
