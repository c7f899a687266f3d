"""GPU parity (bit-exact) of the DOP layout-change kernels against the numpy oracle, on both the
16-byte vector path and the 2-byte scalar fallback, including a simulated exchange among T ranks."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


def dev(x):
    import torch
    return torch.from_numpy(x).cuda()


@pytest.mark.parametrize("N,h,da,db", [(37, 16, 512, 64), (5, 3, 24, 8), (64, 128, 512, 64), (9, 2, 7, 3), (0, 4, 512, 64)])
@pytest.mark.parametrize("strided", [False, True])
def test_pack_rows(N, h, da, db, strided):
    from paper_2609_37626_b200 import binding
    rng = np.random.Generator(np.random.PCG64(1000 + N + da))
    # uint16 stands for bf16 bits; strided: a and b are views into a wider [N][h][da+db+pad] tensor
    if strided:
        wide = rng.integers(0, 2 ** 16, size=(max(N, 1), h, da + db + 8), dtype=np.uint16)[:N]
        a_h, b_h = wide[:, :, :da], wide[:, :, da:da + db]
        w_d = dev(np.ascontiguousarray(wide))
        a_d, b_d = w_d[:, :, :da], w_d[:, :, da:da + db]
    else:
        a_h = rng.integers(0, 2 ** 16, size=(N, h, da), dtype=np.uint16); b_h = rng.integers(0, 2 ** 16, size=(N, h, db), dtype=np.uint16)
        a_d, b_d = dev(a_h), dev(b_h)
    n = N - N // 4                                                   # not every row is sent
    send_row = rng.permutation(N)[:n].astype(np.int32)
    ref = oracle.dop_pack_rows(a_h, b_h, send_row)
    got = binding.splash_dop_pack_rows(a_d, b_d, dev(send_row)).cpu().numpy()
    assert np.array_equal(got, ref)
    ref = oracle.dop_pack_rows(a_h, None, send_row)
    got = binding.splash_dop_pack_rows(a_d, None, dev(send_row)).cpu().numpy()
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("A,B,inner", [(8, 33, (16, 576)), (3, 5, (2, 7)), (2, 1, (128, 512)), (4, 0, (2, 8))])
def test_swap_outer(A, B, inner):
    from paper_2609_37626_b200 import binding
    rng = np.random.Generator(np.random.PCG64(1100 + A + B))
    x = rng.integers(0, 2 ** 16, size=(A, B) + inner, dtype=np.uint16)
    got = binding.splash_dop_swap_outer(dev(x)).cpu().numpy()
    assert np.array_equal(got, oracle.dop_swap_outer(x))


@pytest.mark.parametrize("N,shape", [(41, (16, 512)), (7, (3, 5)), (3, (128, 512))])
def test_unpack_rows_leaves_unlisted_rows_untouched(N, shape):
    import torch
    from paper_2609_37626_b200 import binding
    rng = np.random.Generator(np.random.PCG64(1200 + N))
    n = N - 2
    send_row = rng.permutation(N)[:n].astype(np.int32)
    recv = rng.standard_normal((n,) + shape).astype(np.float32)          # fp32 rows: the attention output
    keep = np.full((N,) + shape, 3.5, np.float32)
    ref = oracle.dop_unpack_rows(recv, send_row, N, out=keep.copy())
    got = binding.splash_dop_unpack_rows(dev(recv), dev(send_row), dev(keep.copy())).cpu().numpy()
    assert np.array_equal(got, ref)


def test_simulated_exchange_round_trip_on_the_gpu():
    """T ranks' packs, the all-to-all done by slicing, swap to all-head order: every owner ends up with all
    heads of exactly its rows; the reverse path restores every rank's head slice of all rows."""
    import torch
    from paper_2609_37626_b200 import binding
    rng = np.random.Generator(np.random.PCG64(1300))
    N, T, h = 50, 4, 32
    H = T * h
    nope = rng.integers(0, 2 ** 16, size=(N, H, 512), dtype=np.uint16); rope = rng.integers(0, 2 ** 16, size=(N, H, 64), dtype=np.uint16)
    owner = rng.integers(0, T, size=N); owner[owner == 2] = 3                        # rank 2 owns nothing
    send_row = np.argsort(owner, kind="stable").astype(np.int32)
    counts = np.bincount(owner, minlength=T); offs = np.concatenate(([0], np.cumsum(counts)))
    nope_d, rope_d, sr_d = dev(nope), dev(rope), dev(send_row)
    send = [binding.splash_dop_pack_rows(nope_d[:, s * h:(s + 1) * h], rope_d[:, s * h:(s + 1) * h], sr_d) for s in range(T)]
    full = np.concatenate((nope, rope), axis=-1)
    outs = []
    for o in range(T):
        recv = torch.stack([send[s][offs[o]:offs[o + 1]] for s in range(T)]).contiguous()      # [T][n][h][576]
        q_owner = binding.splash_dop_swap_outer(recv).reshape(counts[o], H, 576)
        assert np.array_equal(q_owner.cpu().numpy(), full[send_row[offs[o]:offs[o + 1]]])
        outs.append(q_owner[:, :, :512].contiguous())                                             # stands for the result rows
    for s in range(T):
        parts = [binding.splash_dop_swap_outer(outs[o].reshape(counts[o], T, h, 512))[s] for o in range(T)]
        recv = torch.cat(parts).contiguous()
        back = binding.splash_dop_unpack_rows(recv, sr_d, torch.zeros((N, h, 512), dtype=recv.dtype, device="cuda"))
        assert np.array_equal(back.cpu().numpy(), nope[:, s * h:(s + 1) * h])
