"""Property tests for the CPU oracle: over small drawn shapes, KV ranges, page placements,
head slices and both cache formats it must agree with a dense numpy computation of
softmax(scale q K^T) V on the gathered rows (written here from the definition, sharing
nothing with the oracle), and its laws (slice concatenation, range merge) must hold.

None of these call the CUDA path.
"""
import numpy as np
import torch
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
from paper_2609_37626_b200 import workloads as W


def gathered_rows(w, i):
    """Request i's cache rows as fp64 [s][576], decoded from the pool bytes."""
    s = int(w.seq_lens[i])
    rows = np.empty((s, W.D_QK), dtype=np.float64)
    for t in range(s):
        page = w.block_table[i, t // 64]
        if w.kv_dtype == 0:
            rows[t] = W.bf16_bits_to_f32(w.kv_pool[page, t % 64]).astype(np.float64)
        else:
            codes = torch.from_numpy(w.kv_pool[page, t % 64].copy()).view(torch.float8_e4m3fn)
            rows[t] = codes.to(torch.float64).numpy() * float(w.kv_scales[page, t % 64])
    return rows


def dense_reference(w, i, g, lo, hi):
    """(O[512], LSE) of request i, head g over tokens [lo, hi) from the definition."""
    if hi <= lo:
        return np.zeros(512), -np.inf
    rows = gathered_rows(w, i)[lo:hi]
    q = W.bf16_bits_to_f32(w.q[i, g]).astype(np.float64)
    logits = w.softmax_scale * (rows @ q)
    m = logits.max()
    e = np.exp(logits - m)
    z = e.sum()
    return (e @ rows[:, :512]) / z, m + np.log(z)


cases = st.fixed_dictionaries({
    "seed": st.integers(0, 2**16),
    "lens": st.lists(st.sampled_from([0, 1, 2, 17, 63, 64, 65, 127, 128, 129, 200]), min_size=1, max_size=4),
    "H": st.sampled_from([1, 3, 8]),
    "kv_dtype": st.sampled_from([0, 1]),
    "placement": st.sampled_from(["identity", "permute", "reversed"]),
    "pool_factor": st.sampled_from([1.0, 1.5]),
    "cut": st.tuples(st.floats(0, 1), st.floats(0, 1)),
    "use_ranges": st.booleans(),
    "slice": st.tuples(st.floats(0, 1), st.floats(0, 1)),
})


@settings(max_examples=40, deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(cases)
def test_oracle_equals_the_definition_on_drawn_cases(c):
    w = W.make_workload("prop", c["seed"], c["lens"], H=c["H"], kv_dtype=c["kv_dtype"], placement=c["placement"],
                        pool_factor=c["pool_factor"])
    hb, he = sorted(int(round(x * w.H)) for x in c["slice"])
    kvb = kve = None
    if c["use_ranges"]:
        a, b = sorted(c["cut"])
        kvb = np.array([int(a * s) - 1 for s in w.seq_lens], np.int32)       # may start below 0
        kve = np.array([int(b * s) + 2 for s in w.seq_lens], np.int32)       # may end past the context
    out, lse = oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                                 kv_scales=w.kv_scales, head_begin=hb, head_end=he, kv_begin=kvb, kv_end=kve)
    assert out.shape == (w.B, w.H, 512) and lse.shape == (w.B, w.H)
    for i in range(w.B):
        s = int(w.seq_lens[i])
        lo = max(0, int(kvb[i])) if kvb is not None else 0
        hi = min(s, int(kve[i])) if kve is not None else s
        for g in range(hb, he):
            ref_o, ref_l = dense_reference(w, i, g, lo, hi)
            assert np.allclose(out[i, g], ref_o, rtol=0, atol=1e-12)
            if np.isneginf(ref_l):
                assert np.isneginf(lse[i, g])
            else:
                assert abs(lse[i, g] - ref_l) <= 1e-12


@settings(max_examples=20, deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(st.integers(0, 2**16), st.lists(st.integers(1, 199), min_size=1, max_size=4, unique=True), st.sampled_from([0, 1]))
def test_ranges_merge_to_the_unsplit_result_on_drawn_cuts(seed, cuts, kv_dtype):
    w = W.make_workload("propcp", seed, [200, 77], H=2, kv_dtype=kv_dtype)
    full_o, full_l = oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                                       kv_scales=w.kv_scales)
    edges = [0] + sorted(cuts) + [200]
    po, pl = [], []
    for a, b in zip(edges[:-1], edges[1:]):
        o, l = oracle.mla_decode(w.q, w.kv_pool, w.block_table, w.seq_lens, softmax_scale=w.softmax_scale,
                                 kv_scales=w.kv_scales, kv_begin=np.array([a, a], np.int32), kv_end=np.array([b, b], np.int32))
        po.append(o.reshape(-1, 512)); pl.append(l.reshape(-1))
    mo, ml = oracle.lse_merge(np.stack(po), np.stack(pl))
    assert np.allclose(mo, full_o.reshape(-1, 512), rtol=0, atol=1e-12)
    assert np.allclose(ml, full_l.reshape(-1), rtol=0, atol=1e-12)
