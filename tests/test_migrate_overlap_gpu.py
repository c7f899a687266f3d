"""Layer-pipelined migration under decode (Sec. 4.1 "Overlapped transfer" / "Handoff"): layer l + 1's pages move
while layer l decodes, and every layer's decode must then read the MOVED pages through the REWRITTEN table.

The migration of layer l + 1 rides in the decode call of layer l (splash_mla_decode_migrating: on the CTA-pair kernels
the copy runs in otherwise idle warps of the decode kernel; elsewhere as a kernel behind it).  After a layer's pages
have moved, the vacated pages are poisoned, so a decode that still read the old location could not pass.  Checked per
layer: pools, scales and table byte-for-byte against the migrate oracle, the decode against the attention oracle and
bit-for-bit against the same decode made before anything moved."""
import numpy as np
import pytest

import oracle
from paper_2609_37626_b200 import workloads as W
from _util import compare, oracle_run

pytestmark = pytest.mark.gpu

LENS = [10, 64, 3000, 129, 700, 2, 5000]


def make_layers(n_layers, H, kv_dtype, head_begin=0, head_end=None):
    n_used = sum((s + 63) // 64 for s in LENS)
    layers = []
    for l in range(n_layers):
        w = W.make_workload("layer%d" % l, 7000 + 10 * l + kv_dtype, LENS, H=H, kv_dtype=kv_dtype, head_begin=head_begin,
                            head_end=head_end, extra_pool_pages=n_used)
        n_src = w.num_pool_pages - n_used
        src, dst = W.migration_plan(70 + l, w.used_pages, n_used, 0.5)
        layers.append((w, n_src, src, dst))
    return layers


def migrate_oracle(w, n_src, src, dst):
    pool, table = w.kv_pool.copy(), w.block_table.copy()
    sc = None if w.kv_scales is None else w.kv_scales.copy()
    oracle.kv_page_migrate(pool[:n_src], pool[n_src:], src, dst, table, src_scales=None if sc is None else sc[:n_src],
                           dst_scales=None if sc is None else sc[n_src:], dst_id_base=n_src)
    return pool, sc, table


def job_for(binding, torch, dw, w, n_src, src, dst):
    return binding.make_migrate_job(
        dw.kv_pool[:n_src], dw.kv_pool[n_src:], torch.from_numpy(src).cuda(), torch.from_numpy(dst).cuda(), dw.block_table,
        src_scales=None if dw.kv_scales is None else dw.kv_scales[:n_src],
        dst_scales=None if dw.kv_scales is None else dw.kv_scales[n_src:], src_id_base=0, dst_id_base=n_src,
        max_page_id=w.num_pool_pages)


def poison_vacated(torch, dw, src):
    idx = torch.from_numpy(src).long().cuda()
    dw.kv_pool.view(torch.uint8)[idx] = 0x7F
    if dw.kv_scales is not None:
        dw.kv_scales[idx] = float("nan")


# 128 and 80 heads: the CTA-pair kernels carry the copy; 16 heads: the copy runs as a kernel behind the decode
@pytest.mark.parametrize("H,kv_dtype,hb,he", [(128, 1, 0, 128), (128, 0, 0, 128), (80, 1, 0, 80), (16, 0, 0, 16), (128, 1, 32, 48)])
def test_each_layer_decodes_its_moved_pages(H, kv_dtype, hb, he):
    import torch
    from paper_2609_37626_b200 import binding
    layers = make_layers(3, H, kv_dtype, hb, he)
    dws = [binding.DeviceWorkload(w) for w, *_ in layers]
    before = []
    for dw in dws:                                   # every layer's decode before anything moves
        o, l = dw.decode()
        before.append((o.clone(), l.clone()))
    jobs = [job_for(binding, torch, dw, *layer) for dw, layer in zip(dws, layers)]
    # layer 0's pages move on their own (the exposed first layer); then layer l decodes while layer l + 1 moves
    w0, n_src0, src0, dst0 = layers[0]
    binding.splash_kv_page_migrate(dws[0].kv_pool[:n_src0], dws[0].kv_pool[n_src0:], torch.from_numpy(src0).cuda(),
                                   torch.from_numpy(dst0).cuda(), dws[0].block_table,
                                   src_scales=None if dws[0].kv_scales is None else dws[0].kv_scales[:n_src0],
                                   dst_scales=None if dws[0].kv_scales is None else dws[0].kv_scales[n_src0:],
                                   src_id_base=0, dst_id_base=n_src0, max_page_id=w0.num_pool_pages)
    poison_vacated(torch, dws[0], src0)
    after = []
    for l, dw in enumerate(dws):
        nxt = jobs[l + 1] if l + 1 < len(dws) else None
        o, ls = dw.decode(migrate_job=nxt)
        after.append((o, ls))
        if nxt is not None:
            poison_vacated(torch, dws[l + 1], layers[l + 1][2])
    torch.cuda.synchronize()
    rc, detail = binding.splash_workspace_status(binding.decode_workspace(after[0][0].device))
    assert rc == 0, (rc, detail)
    rows = [(i, g) for i in range(len(LENS)) for g in range(hb, he)]
    for l, ((w, n_src, src, dst), dw) in enumerate(zip(layers, dws)):
        ref_pool, ref_sc, ref_table = migrate_oracle(w, n_src, src, dst)
        assert np.array_equal(dw.block_table.cpu().numpy(), ref_table), f"layer {l}: table"
        got = dw.kv_pool.view(torch.uint8).cpu().numpy().reshape(ref_pool.shape[0], -1)
        moved = n_src + dst
        assert np.array_equal(got[moved], ref_pool.view(np.uint8).reshape(ref_pool.shape[0], -1)[moved]), f"layer {l}: moved pages"
        keep = np.setdiff1d(np.arange(w.num_pool_pages), src)      # every page that was not vacated (and poisoned) is as the oracle has it
        assert np.array_equal(got[keep], ref_pool.view(np.uint8).reshape(ref_pool.shape[0], -1)[keep]), f"layer {l}: other pages"
        if ref_sc is not None:
            assert np.array_equal(dw.kv_scales.cpu().numpy().view(np.uint32)[keep], ref_sc.view(np.uint32)[keep])
        o, ls = after[l][0].cpu().numpy(), after[l][1].cpu().numpy()
        compare(o, ls, *oracle_run(w), kv_dtype=kv_dtype, rows=rows, what=f"layer {l} after its pages moved")
        assert np.array_equal(o[:, hb:he], before[l][0].cpu().numpy()[:, hb:he]) and \
            np.array_equal(ls[:, hb:he], before[l][1].cpu().numpy()[:, hb:he]), f"layer {l}: not bit-identical"


def test_decode_behind_a_migration_on_another_stream():
    """The two-stream form with the plain entry points: layer l's migration on a side stream, layer l's decode ordered
    behind it by an event."""
    import torch
    from paper_2609_37626_b200 import binding
    layers = make_layers(2, 128, 1)
    dws = [binding.DeviceWorkload(w) for w, *_ in layers]
    before = [tuple(t.clone() for t in dw.decode()) for dw in dws]
    side = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    side.wait_stream(main)
    outs = []
    ws = [torch.empty(1 << 20, dtype=torch.uint8, device="cuda") for _ in dws]
    for l, ((w, n_src, src, dst), dw) in enumerate(zip(layers, dws)):
        with torch.cuda.stream(side):
            binding.splash_kv_page_migrate(dw.kv_pool[:n_src], dw.kv_pool[n_src:], torch.from_numpy(src).cuda(),
                                           torch.from_numpy(dst).cuda(), dw.block_table, src_scales=dw.kv_scales[:n_src],
                                           dst_scales=dw.kv_scales[n_src:], src_id_base=0, dst_id_base=n_src,
                                           max_page_id=w.num_pool_pages, workspace=ws[l], stream=side)
            poison_vacated(torch, dw, src)
            moved = torch.cuda.Event(); moved.record(side)
        main.wait_event(moved)
        outs.append(dw.decode())
    torch.cuda.synchronize()
    for l, (w, *_ ) in enumerate(layers):
        o, ls = outs[l][0].cpu().numpy(), outs[l][1].cpu().numpy()
        compare(o, ls, *oracle_run(w), kv_dtype=1, what=f"layer {l}")
        assert np.array_equal(o, before[l][0].cpu().numpy()) and np.array_equal(ls, before[l][1].cpu().numpy())


def test_job_argument_checks_and_empty_job():
    import torch
    from paper_2609_37626_b200 import binding
    (w, n_src, src, dst), = make_layers(1, 128, 1)
    dw = binding.DeviceWorkload(w)
    ref = dw.decode()
    job, keep = job_for(binding, torch, dw, w, n_src, src[:0], dst[:0])          # n = 0: exactly the plain call
    o, l = dw.decode(migrate_job=(job, keep))
    torch.cuda.synchronize()
    assert torch.equal(o, ref[0]) and torch.equal(l, ref[1])
    job, keep = job_for(binding, torch, dw, w, n_src, src, dst)
    job.page_bytes = 100                                                          # not a multiple of 16
    with pytest.raises(binding.SplashError):
        dw.decode(migrate_job=(job, keep))
    assert binding.splash_last_launch_count() == 0
