// Building blocks of the CTA-pair (tcgen05 cta_group::2) decode kernels: cluster addressing,
// barrier arrivals and waits across the pair, TMA loads that complete on the leader's barrier.
#pragma once

#include "splash_umma.cuh"

namespace splash {
namespace umma {

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
// Arrival on a barrier of the other CTA that carries no data with it: a release at cluster scope
// stalls the arriving thread for ~300 cycles and takes ~500 to land, the relaxed form ~20 and
// ~200.  It is used where what the arrival announces is already in place on this SM when it is
// sent -- shared-memory writes followed by fence.proxy.async, tensor-memory reads followed by
// tcgen05.wait::ld -- and is consumed on this SM, by MMAs that the pair's leader issues only
// after it has seen the arrival.
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// cluster-scope acquire for barriers the peer CTA arrives on
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
static __device__ __noinline__ bool mbar_wait_cluster(const Ctx &ctx, uint32_t bar, uint32_t parity, int bar_id) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*ctx.abort_flag) return false;
    const unsigned long long start = global_timer_ns();
    for (;;) {
        for (int k = 0; k < 256; ++k)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*ctx.abort_flag) return false;
        if (global_timer_ns() - start > kWaitLimitNs) {
            *ctx.abort_flag = 1;
            if (atomicCAS(ctx.status, 0, (int)SPLASH_DEVICE_TIMEOUT) == 0) {
                ctx.status[1] = (int)blockIdx.x; ctx.status[2] = 200 + bar_id; ctx.status[3] = (int)threadIdx.x;
            }
            return false;
        }
    }
}
// Reports `bytes` as delivered on a barrier given by its cluster address (this CTA's or the leader's): what a TMA load
// does on completion, for a tile that a warp wrote by hand.  The cluster-scope fence orders the warp's writes (made
// visible to the tensor core by fence.proxy.async, gathered by __syncwarp) before the report.
__device__ __forceinline__ void mbar_complete_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("fence.acq_rel.cluster;" ::: "memory");
    asm volatile("mbarrier.complete_tx.relaxed.cluster.shared::cluster.b64 [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// TMA load whose completion bytes go to a barrier of the pair's leader CTA
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int c0, int c1,
                                                 int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// pull a contiguous range into L2 ahead of the loads that will need it (one request to the copy engine; the
// tensor form below costs the engine as much as the load itself: one 128-byte request per row and chunk)
__device__ __forceinline__ void bulk_prefetch_l2(const void *gptr, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gptr), "r"(bytes) : "memory");
}
// pull a box into L2 ahead of the load that will need it
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap *map, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global [%0, {%1, %2, %3, %4}];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// commit: arrive on the barrier at this offset in BOTH CTAs once all MMAs issued so far have retired
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
// 32 consecutive fp32 columns of this warp's 32 lanes
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    tmem_ld16(taddr, *reinterpret_cast<float(*)[16]>(&v[0]));
    tmem_ld16(taddr + 16, *reinterpret_cast<float(*)[16]>(&v[16]));
}

// The page-copy job of a decode call (a layer's pages moving while another layer decodes), as carried by one warp:
// copy warp cw of ncw takes pages cw, cw + ncw, ...  A page is copied in pieces of 4 KB (eight 16-byte loads per
// lane); the loads of the next piece are issued before the stores of the current one, across page boundaries, so
// that a warp always has 4 KB of loads in flight.  Streaming loads and stores: the bytes are not needed again soon.
// (Pulling each page into L2 ahead of its loads made the copy slower and the decode beside it too.)  Byte-exact.  A
// page that is not a multiple of 4 KB has its remainder copied 512 bytes at a time; scale pages ride along.
__device__ __forceinline__ void copy_pages_in_idle_warp(const DecodeParams &p, int cw, int ncw, int lane) {
    constexpr int kInFlight = 8, kPiece = kInFlight * 32;        // 16-byte vectors per piece
    const int64_t vecs = p.mig_page_vecs;
    const int pieces_per_page = (int)(vecs / kPiece);
    const int my_pages = p.mig_n > cw ? (p.mig_n - cw + ncw - 1) / ncw : 0;
    if (my_pages == 0) return;
    auto page_src = [&](int k) { return p.mig_src + (int64_t)p.mig_src_ids[cw + (int64_t)k * ncw] * vecs; };
    auto page_dst = [&](int k) { return p.mig_dst + (int64_t)p.mig_dst_ids[cw + (int64_t)k * ncw] * vecs; };
    // what does not fit the 4 KB pieces: the tail of every page and the scale pages
    for (int k = 0; k < my_pages; ++k) {
        const int64_t j = cw + (int64_t)k * ncw;
        for (int64_t c = (int64_t)pieces_per_page * kPiece + lane; c < vecs; c += 32) __stcs(page_dst(k) + c, __ldcs(page_src(k) + c));
        if (p.mig_src_scales != nullptr && lane < kPage * 4 / 16)
            __stcs(p.mig_dst_scales + (int64_t)p.mig_dst_ids[j] * (kPage * 4 / 16) + lane,
                   __ldcs(p.mig_src_scales + (int64_t)p.mig_src_ids[j] * (kPage * 4 / 16) + lane));
    }
    if (pieces_per_page == 0) return;
    const int64_t total = (int64_t)my_pages * pieces_per_page;
    const uint4 *src = nullptr;
    uint4 *dst_page = nullptr;
    // loads piece `it` into v and returns where it goes
    auto load_piece = [&](uint4 (&v)[kInFlight], int64_t it) -> uint4 * {
        const int piece = (int)(it % pieces_per_page);
        if (piece == 0) {
            const int k = (int)(it / pieces_per_page);
            src = page_src(k); dst_page = page_dst(k);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) v[u] = __ldcs(src + (int64_t)piece * kPiece + u * 32 + lane);
        return dst_page + (int64_t)piece * kPiece + lane;
    };
    auto store_piece = [&](const uint4 (&v)[kInFlight], uint4 *to) {
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) __stcs(to + u * 32, v[u]);
    };
    uint4 va[kInFlight], vb[kInFlight];
    uint4 *ta = load_piece(va, 0), *tb = nullptr;
    for (int64_t it = 0; it < total; it += 2) {
        if (it + 1 < total) tb = load_piece(vb, it + 1);
        store_piece(va, ta);
        if (it + 1 >= total) break;
        if (it + 2 < total) ta = load_piece(va, it + 2);
        store_piece(vb, tb);
    }
}

// Page tiles of the two CTAs of a pair for one step, after the token shift.
struct PairGeom { TileGeom a, b; bool has_b; };

}  // namespace umma
}  // namespace splash
