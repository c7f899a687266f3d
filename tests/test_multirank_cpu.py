"""World-size-2 checks of the multi-rank host logic on CPU (gloo): the shard index
helpers cover every unit exactly once, shard results gathered over the process group
reproduce the unsplit result (the oracle stands in for each rank's device call), and
the timing reduction takes the maximum over ranks."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_37626_b200 import sharding, workloads as W

    w = W.make_workload("ranks", 4321, [70, 129, 300, 5], H=8)
    full_o, full_l = oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale)

    # TP / DOP: head slices, gathered along the head axis
    hb, he = sharding.head_slice(rank, world, w.H)
    o, l = oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                             head_begin=hb, head_end=he)
    mine = torch.from_numpy(np.ascontiguousarray(o[:, hb:he]))
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    assert np.array_equal(torch.cat(parts, dim=1).numpy(), full_o)

    # DP-attention: request slices, every request owned exactly once
    own = sharding.request_slice(rank, world, w.B)
    counts = torch.zeros(w.B, dtype=torch.int64)
    counts[torch.from_numpy(own)] = 1
    dist.all_reduce(counts)
    assert torch.all(counts == 1)
    o, l = oracle.mla_decode(w.q[own], w.kv_pool, w.block_table[own], w.seq_lens[own], softmax_scale=w.softmax_scale)
    assert np.array_equal(o, full_o[own]) and np.array_equal(l, full_l[own])

    # CP: contiguous token ranges, partials all-gathered, merged on every rank
    kb, ke = sharding.kv_range(rank, world, w.seq_lens)
    po, pl = oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                               kv_begin=kb, kv_end=ke)
    po_t, pl_t = torch.from_numpy(po), torch.from_numpy(pl)
    go = [torch.empty_like(po_t) for _ in range(world)]
    gl = [torch.empty_like(pl_t) for _ in range(world)]
    dist.all_gather(go, po_t); dist.all_gather(gl, pl_t)
    mo, ml = oracle.lse_merge(torch.stack(go).numpy().reshape(world, -1, 512), torch.stack(gl).numpy().reshape(world, -1))
    assert np.allclose(mo.reshape(full_o.shape), full_o, atol=1e-12) and np.allclose(ml.reshape(full_l.shape), full_l, atol=1e-12)
    ends = torch.from_numpy(ke.astype(np.int64)); begins = torch.from_numpy(kb.astype(np.int64))
    covered = ends - begins
    dist.all_reduce(covered)
    assert np.array_equal(covered.numpy(), w.seq_lens.astype(np.int64))

    # timing: the slowest rank decides
    ms, e2e = sharding.max_over_ranks([1.0 + rank, 5.0 - rank])
    assert ms == float(world) and e2e == 5.0
    assert sharding.weak_scaling_value(64, world, 2.0) == world * 64 / 2e-3
    open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))


def test_shard_helpers_single_process():
    sys.path.insert(0, ROOT)
    from paper_2609_37626_b200 import sharding
    assert [sharding.head_slice(r, 8, 128) for r in (0, 3, 7)] == [(0, 16), (48, 64), (112, 128)]
    assert sorted(np.concatenate([sharding.request_slice(r, 4, 10) for r in range(4)]).tolist()) == list(range(10))
    lens = np.array([1, 7, 64, 1000])
    edges = [sharding.kv_range(r, 8, lens) for r in range(8)]
    for r in range(7):
        assert np.array_equal(edges[r][1], edges[r + 1][0])
    assert np.array_equal(edges[0][0], 0 * lens) and np.array_equal(edges[7][1], lens)
    assert sharding.max_over_ranks([3.5]) == [3.5]
