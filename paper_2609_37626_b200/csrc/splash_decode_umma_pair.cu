// bf16 decode kernel for slices of 65..128 heads: a CLUSTER OF TWO CTAs per KV worker that
// issues its MMAs with tcgen05 cta_group::2.
//
// Two independent 64-head CTAs each pull every page (72 KB) through their own shared memory
// and their own tensor core.  A CTA pair splits the page instead: CTA r loads tokens
// [32 r, 32 r + 32) of the 64-token page (all 9 chunks of 64 columns, 36 KB), and
//
//   S [128 heads x 64 tokens] = Q K^T      M = 128 (64 heads per CTA), N = 64: each CTA supplies
//                                           its 32 tokens as its half of the B operand
//   O [128 heads x 256 dv]   += P V        M = 128, N = 256 (x 2 halves of dv): each CTA supplies
//                                           its 64 heads of P and 128 of the 256 dv columns
//
// For P.V CTA r supplies dv columns [256 n + 128 r, + 128) of BOTH half-pages, at the same
// shared-memory offsets in both CTAs (the two CTAs of an MMA share one descriptor).  Its own
// half-page has them in chunk slots 4 n + 2 r, 4 n + 2 r + 1 of the stage; the other four
// latent chunk slots hold columns only the peer multiplies, so once QK^T of the stage has
// retired they are overwritten with the peer half-page's chunks 4 n + 2 r, 4 n + 2 r + 1.
// The MMAs over half-page g then start at slot 4 n + 2 g in both CTAs.  That second load
// (L2 hits: the peer has just read the page) hides behind the softmax of the tile.
// P of a tile is written in two [64 heads x 32 tokens] halves: the first into the stage's rope
// chunk slot, which nothing reads after QK^T (that is what makes room for a fourth stage), the
// second into a small buffer of its own.
// Accumulators: CTA r holds its 64 heads; a head's row is TMEM lane h (first half of N) and
// lane 64 + h (second half).
//
// Roles per CTA (512 threads): page + query producer, 4 QK^T issuers and 2 P.V issuers
// (leader CTA only), 8 softmax warps, 1 producer of the peer chunks.  Barriers that the
// issuers wait on live in the leader; the peer's warps arrive on them across the cluster
// (relaxed arrivals: what they announce is already in place on the peer's SM), and TMA loads
// of the peer complete on them too.
#include <cuda_fp16.h>

#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kQkWarps = 4, kPvWarps = 2, kSoftmaxWarps = 8;
constexpr int kWarpProducer = 0;
constexpr int kWarpQk = 1;
constexpr int kWarpPv = kWarpQk + kQkWarps;
constexpr int kWarpSoftmax = kWarpPv + kPvWarps;       // 7: TMEM quadrant = warp & 3
constexpr int kWarpVProducer = kWarpSoftmax + kSoftmaxWarps;
constexpr int kThreads = (kWarpVProducer + 1) * 32;    // 16 warps = 512 threads
constexpr int kN = 64;                              // heads per CTA
constexpr int kHalf = 32;                           // tokens per CTA and tile
constexpr uint32_t kSlab = kHalf * 128;             // one chunk of a half-page: 32 tokens x 128 B
constexpr uint32_t kStageBytes = 9 * kSlab;         // 36,864
constexpr uint32_t kPeerBytes = 4 * kSlab;          // the peer half-page's chunks this CTA multiplies: 16,384
constexpr uint32_t kQSlab = kN * 128;               // one chunk of the query rows: 64 heads x 128 B
constexpr uint32_t kQBytes = 9 * kQSlab;            // 73,728
constexpr uint32_t kPHalfBytes = kN * 64;           // P of one half-page: 64 heads x 32 tokens bf16
constexpr int kStages = 4;
constexpr int kPrefetchAhead = 1;                   // tiles between the L2 prefetch of a page and its use (4: 3 % slower; none: 4 %)
constexpr int kPrefetchAheadBusy = 4;               // the same while the call carries a page-copy job
constexpr float kTau = 8.0f;                        // O is rescaled only when a row maximum grows by more than 2^8

enum BarrierId {
    kBarKFull = 0,                        // [4] leader: both half-pages landed (tx bytes of both CTAs)
    kBarQkDone = kBarKFull + kStages,     // [4] QK^T of the stage retired (multicast commit): peer chunks may land
    kBarVFull = kBarQkDone + kStages,     // [4] leader: both CTAs' peer chunks landed
    kBarStageEmpty = kBarVFull + kStages, // [4] P.V of the stage retired (multicast commit): stage and P buffers
                                          //     are free, O is up to date
    kBarQFull = kBarStageEmpty + kStages, // leader: query rows of both CTAs landed
    kBarQEmpty,                           // last QK^T of the request retired (multicast commit)
    kBarSFull,                            // [2] S buffer written (multicast commit)
    kBarSEmpty = kBarSFull + 2,           // [2] S buffer read (leader: by both CTAs)
    kBarPFull = kBarSEmpty + 2,           // [2] P buffer written (leader: by both CTAs)
    kBarOFull = kBarPFull + 2,            // last P.V of the request retired (multicast commit)
    kBarOEmpty,                           // O drained (leader: by both CTAs)
    kNumBarriers
};

constexpr uint32_t kOffK = 0;                                   // [4 stages] 9 chunk slots of 32 tokens
constexpr uint32_t kOffQ = kOffK + kStages * kStageBytes;       // 9 chunks x 64 heads x 128 B
constexpr uint32_t kOffP1 = kOffQ + kQBytes;                    // [2 buffers] P of half-page 1: 64 heads x 64 B
constexpr uint32_t kOffAlpha = kOffP1 + 2 * kPHalfBytes;            // float [64]
constexpr uint32_t kOffL = kOffAlpha + kN * 4;                  // float [64]
constexpr uint32_t kOffXch = kOffL + kN * 4;                    // float [64][4]
constexpr uint32_t kOffBar = kOffXch + kN * 16;
constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;
constexpr uint32_t kSmemBytes = kOffMisc + 32;
static_assert(kSmemBytes <= 232448, "shared memory overflow");
static_assert(kOffQ % 1024 == 0 && kOffP1 % 1024 == 0 && kSlab % 1024 == 0, "swizzle atoms need 1024-byte alignment");
// tensor memory: O two halves of dv x 128 columns, then 2 S buffers x 4 partials x 32 columns
constexpr uint32_t kColO = 0, kColS = 256;

__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
decode_umma_pair_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_half,
                        const __grid_constant__ CUtensorMap tmap_peer, const __grid_constant__ CUtensorMap tmap_q) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();             // 0 = leader: issues the MMAs
    const int pair_id = blockIdx.x >> 1;                // CTA pair: (KV worker, group of 128 heads)
    const int worker = pair_id / p.pair_groups;
    const int head0 = p.head_begin + (pair_id % p.pair_groups) * (2 * kN) + (int)rank * kN;
    const int h = p.head_end - p.head_begin;

    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + kOffMisc);
    Ctx ctx{misc + 1, p.status};
    auto bar = [&](int id) -> uint32_t { return sbase + kOffBar + 8u * (uint32_t)id; };
    auto leader_bar = [&](int id) -> uint32_t { return map_to_cta(sbase + kOffBar + 8u * (uint32_t)id, 0); };
    // one arrival of a warp of either CTA on a barrier that lives in the leader
    auto arrive_on_leader = [&](int id) {
        if (rank == 0) mbar_arrive(bar(id));
        else mbar_arrive_cluster_relaxed(leader_bar(id));
    };

    if (tid == 0) {
        // barriers the leader's issuers wait on count the warps of both CTAs (the peer's copies are unused)
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1); mbar_init(bar(kBarQkDone + s), kQkWarps);
            mbar_init(bar(kBarVFull + s), 1); mbar_init(bar(kBarStageEmpty + s), kPvWarps);
        }
        mbar_init(bar(kBarQFull), 1); mbar_init(bar(kBarQEmpty), kQkWarps);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(kBarSFull + b), kQkWarps); mbar_init(bar(kBarSEmpty + b), 2 * kSoftmaxWarps);
            mbar_init(bar(kBarPFull + b), 2 * kSoftmaxWarps);
        }
        mbar_init(bar(kBarOFull), kPvWarps); mbar_init(bar(kBarOEmpty), 2 * kSoftmaxWarps);
        misc[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + kOffMisc), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                   // barriers of both CTAs exist before anyone signals them
    tcgen05_fence_after();
    const uint32_t tmem_base = misc[0];
    grid_dependency_wait();                               // the plan kernel's output is read from here on
    const long long t_start = clock64();
    const unsigned long long ns_start = global_timer_ns();

    SegmentIter it;
    it.init(p, worker);
    Segment seg;
    seg.lo = seg.hi = seg.tile_begin = seg.tile_end = 0;

    if (warp == kWarpProducer || warp == kWarpVProducer) {
        // ===================================================== TMA producers
        // warp 0: the query rows of this CTA's heads and its half of every page, up to three tiles
        // ahead; last warp: the peer half-page's chunks, into the dead slots of the stage once QK^T
        // has read it
        const bool is_v = warp == kWarpVProducer;
        uint32_t kv_it = 0, seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            if (!is_v && lane == 0) {
                ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
                if (ok) {
                    if (rank == 0) mbar_expect_tx(bar(kBarQFull), 2 * kQBytes);
                    tma_load_4d_pair(sbase + kOffQ, &tmap_q, leader_bar(kBarQFull), 0, head0, 0, seg.request);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            const int first_page = seg.lo / kPage;
            const int32_t *table = p.block_table + (int64_t)seg.request * p.table_stride;
            for (int tile = seg.tile_begin; ok && tile < seg.tile_end; ++tile, ++kv_it) {
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);
                const uint32_t stage = kv_it % kStages, ph = (kv_it / kStages) & 1;
                const uint32_t k0 = sbase + kOffK + stage * kStageBytes;
                int page = 0;
                if (lane == 0) {
                    page = table[first_page + tile];
                    if (!is_v) {
                        ok = mbar_wait(ctx, bar(kBarStageEmpty + stage), ph ^ 1, kBarStageEmpty + stage);
                        if (ok) {
                            // the leader's barrier expects the halves of both CTAs
                            if (rank == 0) mbar_expect_tx(bar(kBarKFull + stage), 2 * kStageBytes);
                            if (!g.both) tma_load_4d_pair(k0, &tmap_half, leader_bar(kBarKFull + stage), 0, g.tok0 + kHalf * (int)rank, 0, page);
                            // A stage is held from its load until P.V has read it, about three tiles, so the
                            // load of tile t + 3 starts only when the issuers are about to need it: have its
                            // half of the page in L2 by then.
                            // (further ahead while a page-copy job shares the memory system: the loads then take longer)
                            const int tf = tile + (p.mig_n > 0 ? kPrefetchAheadBusy : kPrefetchAhead);
                            if (tf < seg.tile_end) {
                                const int page_f = table[first_page + tf];
                                // this CTA's half of the page is 32 consecutive rows: one contiguous range
                                if (page_f >= 0 && page_f < p.num_pool_pages)
                                    bulk_prefetch_l2(static_cast<const uint8_t *>(p.kv_pool) + ((size_t)page_f * kPage + kHalf * rank) * (kDQK * 2),
                                                     kStageBytes);
                            }
                        }
                    } else {
                        ok = mbar_wait(ctx, bar(kBarQkDone + stage), ph, kBarQkDone + stage);
                        if (ok) {
                            if (rank == 0) mbar_expect_tx(bar(kBarVFull + stage), 2 * kPeerBytes);
                            // peer half-page chunks 4n + 2 rank, + 1 -> slots 4n + 2 (1 - rank), + 1
                            if (!g.both) {
#pragma unroll
                                for (int n = 0; n < 2; ++n)
                                    tma_load_4d_pair(k0 + (4 * n + 2 * (1 - (int)rank)) * kSlab, &tmap_peer, leader_bar(kBarVFull + stage), 0,
                                                     g.tok0 + kHalf * (1 - (int)rank), 4 * n + 2 * (int)rank, page);
                            }
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (ok && g.both) {
                    // a range cut at both ends inside this page: the warp writes what the box(es) would have
                    // delivered, zeros outside the range, and reports the bytes on the leader's barrier
                    page = __shfl_sync(0xffffffffu, page, 0);
                    const uint8_t *src = page >= 0 && page < p.num_pool_pages
                        ? static_cast<const uint8_t *>(p.kv_pool) + (size_t)page * (kPage * kDQK * 2) : nullptr;
                    uint8_t *slabs = smem + kOffK + stage * kStageBytes;
                    if (!is_v) {
                        fill_rows_by_hand<128>(slabs, kSlab, kHalf, src, g.tok0 + kHalf * (int)rank, g.a, g.b, 0, 0, 9, lane);
                    } else {
                        for (int n = 0; n < 2; ++n)
                            fill_rows_by_hand<128>(slabs, kSlab, kHalf, src, g.tok0 + kHalf * (1 - (int)rank), g.a, g.b,
                                                   4 * n + 2 * (int)rank, 4 * n + 2 * (1 - (int)rank), 2, lane);
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_complete_tx_cluster(leader_bar(is_v ? kBarVFull + stage : kBarKFull + stage), is_v ? kPeerBytes : kStageBytes);
                }
            }
            ++seg_it;
        }
    } else if (warp >= kWarpQk && warp < kWarpQk + kQkWarps && rank == 0) {
        // ===================================================== QK^T issuers (leader CTA)
        // One thread sustains one tcgen05.mma per ~65 cycles and a chain of MMAs into one accumulator
        // runs at the MMA latency, so the 36 K = 16 steps of a tile go to four issuers with a partial
        // accumulator each.
        if (lane == 0) {
            const int a = warp - kWarpQk;
            constexpr uint32_t kIdescQK = make_idesc(128, 64, 0, 0);
            uint32_t kv_it = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                ok = mbar_wait_cluster(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
                for (int tile = seg.tile_begin; ok && tile < seg.tile_end; ++tile, ++kv_it) {
                    const uint32_t stage = kv_it % kStages, b = kv_it & 1;
                    ok = mbar_wait_cluster(ctx, bar(kBarKFull + stage), (kv_it / kStages) & 1, kBarKFull + stage) &&
                         mbar_wait_cluster(ctx, bar(kBarSEmpty + b), ((kv_it >> 1) & 1) ^ 1, kBarSEmpty + b);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t k0 = sbase + kOffK + stage * kStageBytes;
                    const uint32_t d = tmem_base + kColS + (b * kQkWarps + a) * kHalf;
#pragma unroll
                    for (int t = 0; t < 36 / kQkWarps; ++t) {
                        const int idx = t * kQkWarps + a, c = idx >> 2, k = idx & 3;
                        uint64_t dq = make_desc(sbase + kOffQ + c * kQSlab + k * 32, 16, 1024);   // A: 2 x 64 heads x 16
                        uint64_t dk = make_desc(k0 + c * kSlab + k * 32, 16, 1024);             // B: 2 x 32 tokens x 16
                        umma_bf16_pair(d, dq, dk, kIdescQK, t != 0);
                    }
                    umma_commit_pair(bar(kBarSFull + b));
                    umma_commit_pair(bar(kBarQkDone + stage));
                }
                if (ok) umma_commit_pair(bar(kBarQEmpty));
                ++seg_it;
            }
        }
    } else if (warp >= kWarpPv && warp < kWarpPv + kPvWarps && rank == 0) {
        // ===================================================== P.V issuers (leader CTA)
        if (lane == 0) {
            const int n = warp - kWarpPv;                 // dv half: columns [256 n, 256 n + 256)
            constexpr uint32_t kIdescPV = make_idesc(128, 256, 0, 1);
            uint32_t kv_it = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                for (int tile = seg.tile_begin; ok && tile < seg.tile_end; ++tile, ++kv_it) {
                    const uint32_t stage = kv_it % kStages, pb = kv_it & 1;
                    ok = mbar_wait_cluster(ctx, bar(kBarVFull + stage), (kv_it / kStages) & 1, kBarVFull + stage) &&
                         mbar_wait_cluster(ctx, bar(kBarPFull + pb), (kv_it >> 1) & 1, kBarPFull + pb);
                    if (ok && tile == seg.tile_begin) ok = mbar_wait_cluster(ctx, bar(kBarOEmpty), (seg_it & 1) ^ 1, kBarOEmpty);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t k0 = sbase + kOffK + stage * kStageBytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // 16 tokens of half-page g.  A: P rows (heads), 32 bytes of the 64-byte row (g = 0: in the
                        // stage's rope slot, g = 1: in its own buffer);
                        // B: slots 4n + 2g, + 1 (two 64-wide dv chunks, LBO apart), 16 token rows, MN-major
                        const int g = j >> 1;
                        const uint32_t p0 = g == 0 ? k0 + 8 * kSlab : sbase + kOffP1 + pb * kPHalfBytes;
                        uint64_t da = make_desc_sw64(p0 + (j & 1) * 32, 16, 512);
                        uint64_t db = make_desc(k0 + (4 * n + 2 * g) * kSlab + (j & 1) * 2048, kSlab, 1024);
                        umma_bf16_pair(tmem_base + kColO + n * 128, da, db, kIdescPV, (tile != seg.tile_begin) || j != 0);
                    }
                    umma_commit_pair(bar(kBarStageEmpty + stage));
                    if (tile + 1 == seg.tile_end) umma_commit_pair(bar(kBarOFull));
                }
                ++seg_it;
            }
        }
    } else if (warp >= kWarpQk && warp < kWarpSoftmax) {
        // the issuer warps of the peer CTA have nothing to do for the attention itself: they carry the call's page-copy
        // job, if it has one (a layer's pages on the move while this layer decodes)
        if (p.mig_n > 0)
            copy_pages_in_idle_warp(p, pair_id * (kQkWarps + kPvWarps) + (warp - kWarpQk), p.num_workers * p.pair_groups * (kQkWarps + kPvWarps), lane);
    } else {
        // ===================================================== softmax + epilogue warps
        // S partial layout per CTA: TMEM lane L < 64 = head L, tokens of half-page 0 in 32 columns;
        // lane 64 + L = head L, tokens of half-page 1.  Two warps per quadrant take 16 columns each,
        // so a thread owns ONE head and 16 tokens of one half-page.
        const int sw = warp - kWarpSoftmax;             // 0..7
        const int q4 = warp & 3;                        // TMEM lane quadrant
        const int cf = sw >> 2;                         // column half: tokens [16 cf, 16 cf + 16) of the half-page
        const int g = q4 >> 1;                          // half-page
        const int hd = 32 * (q4 & 1) + lane;            // this thread's head (0..63 within the CTA)
        const int half_id = q4 & 1;                     // heads 0-31 or 32-63: the four warps that share them sync on bar 2 + half_id
        const int row0 = kHalf * g + 16 * cf;           // first of this thread's 16 rows of the 64-row tile
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        float *alpha_s = reinterpret_cast<float *>(smem + kOffAlpha);
        float *l_s = reinterpret_cast<float *>(smem + kOffL);
        float *xch = reinterpret_cast<float *>(smem + kOffXch);
        const float scale_log2 = p.softmax_scale * kLog2e;
        const int slot4 = g * 2 + cf;                   // this thread's slot among the 4 threads of its head
        uint32_t kv_it = 0, seg_it = 0;
        // A failed (timed-out) wait only clears `ok`; the role keeps walking its tiles so that every
        // thread still meets the named barriers -- once the CTA aborts, waits return at once.
        bool ok = true;
        while (it.next(p, seg)) {
            float m = -INFINITY, l = 0.f;               // running maximum in scaled log2 units
            const int first_page = seg.lo / kPage;
            // several query rows per request: this thread's (virtual) head is row (head mod R) and sees the
            // tokens below causal_end only
            const int causal_end = p.q_rows > 1 ? p.seq_lens[seg.request] - (p.q_rows - 1 - (head0 + hd) % p.q_rows) : 0x3fffffff;   // (far above any token index, and safe to subtract a negative offset from)
            for (int tile = seg.tile_begin; tile < seg.tile_end; ++tile, ++kv_it) {
                const TileGeom geo = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);
                const uint32_t b = kv_it & 1;
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (kv_it >> 1) & 1, kBarSFull + b);
                tcgen05_fence_after();
                float sv[16];
                {
                    float pa[16], pb[16], pc[16];
                    const uint32_t sb = tmem_base + lane_addr + kColS + (b * kQkWarps) * kHalf + 16 * cf;
                    tmem_ld16(sb, sv);
                    tmem_ld16(sb + kHalf, pa);
                    tmem_ld16(sb + 2 * kHalf, pb);
                    tmem_ld16(sb + 3 * kHalf, pc);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) sv[j] = ((sv[j] + pa[j]) + (pb[j] + pc[j])) * scale_log2;
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) arrive_on_leader(kBarSEmpty + b);
                // rows outside [r_lo, r_hi) are zero fill or tokens outside the request's range (or beyond this
                // head's causal end: row r of the tile holds token (first_page + tile) * 64 + tok0 + r)
                const int r_hi = min(geo.r_hi, causal_end - ((first_page + tile) * kPage + geo.tok0));
                if (row0 < geo.r_lo || row0 + 16 > r_hi) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (row0 + j < geo.r_lo || row0 + j >= r_hi) sv[j] = -INFINITY;
                }
                float mt = sv[0];
#pragma unroll
                for (int j = 1; j < 16; ++j) mt = fmaxf(mt, sv[j]);
                // row maximum over the 4 threads of this head (2 half-pages x 2 column halves, 4 different warps)
                xch[hd * 4 + slot4] = mt;
                named_bar_sync_dyn<128>(2 + half_id);
                {
                    const float4 x4 = *reinterpret_cast<const float4 *>(&xch[hd * 4]);
                    mt = fmaxf(fmaxf(x4.x, x4.y), fmaxf(x4.z, x4.w));
                }
                bool grew = false;
                float al = 1.f;
                if (mt > m + kTau) { al = (m == -INFINITY) ? 0.f : fast_exp2(m - mt); m = mt; l *= al; grew = true; }
                if (slot4 == 0) alpha_s[hd] = al;
                const float mref = m == -INFINITY ? 0.f : m;   // a head that has seen no token yet: all weights 0, not NaN
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 16; j += 2) {
                    const float u0 = fast_exp2(sv[j] - mref), u1 = fast_exp2(sv[j + 1] - mref);
                    l += u0 + u1;
                    pk[j >> 1] = pack_bf16x2(u0, u1);
                }
                const bool rescale = named_bar_or<1, kSoftmaxWarps * 32>(grew);
                // P.V of the tile that last used the P buffer of half-page 1 (two back) must be done; a rescale
                // of O also needs the previous tile's P.V
                if (kv_it > 1) ok &= mbar_wait(ctx, bar(kBarStageEmpty + (kv_it - 2) % kStages), ((kv_it - 2) / kStages) & 1, kBarStageEmpty);
                if (rescale && tile != seg.tile_begin) {
                    ok &= mbar_wait(ctx, bar(kBarStageEmpty + (kv_it - 1) % kStages), ((kv_it - 1) / kStages) & 1, kBarStageEmpty);
                    tcgen05_fence_after();
                    // O rows are TMEM lanes: this thread scales its lane's columns [128 cf, 128 cf + 128)
                    const float a_row = alpha_s[hd];
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        float o[32];
                        const uint32_t addr = tmem_base + lane_addr + kColO + 128 * cf + c * 32;
                        tmem_ld32(addr, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 32; ++k) o[k] *= a_row;
                        tmem_st16(addr, *reinterpret_cast<float(*)[16]>(&o[0]));
                        tmem_st16(addr + 16, *reinterpret_cast<float(*)[16]>(&o[16]));
                    }
                    tmem_wait_st();
                }
                {
                    // P of this half-page: K-major, 64-byte swizzle; row = head, bytes [32 cf, 32 cf + 32)
                    uint8_t *ph = g == 0 ? smem + kOffK + (kv_it % kStages) * kStageBytes + 8 * kSlab : smem + kOffP1 + b * kPHalfBytes;
                    *reinterpret_cast<uint4 *>(ph + sw64((uint32_t)hd, (uint32_t)(32 * cf))) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *reinterpret_cast<uint4 *>(ph + sw64((uint32_t)hd, (uint32_t)(32 * cf + 16))) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
                fence_proxy_async();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) arrive_on_leader(kBarPFull + b);
            }
            // ---- row sums of the 4 threads of a head
            xch[hd * 4 + slot4] = l;
            named_bar_sync<1, kSoftmaxWarps * 32>();
            if (slot4 == 0) {
                const float4 x4 = *reinterpret_cast<const float4 *>(&xch[hd * 4]);
                const float lt = (x4.x + x4.y) + (x4.z + x4.w);
                l_s[hd] = lt > 0.f ? 1.f / lt : 0.f;       // no token at all (an empty causal range): O = 0, LSE = -inf
                const int gh = head0 + hd;
                if (gh < p.head_end) {
                    float lse = lt > 0.f ? (m + log2f(lt)) * kLn2 : -INFINITY;
                    if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                    else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                }
            }
            named_bar_sync<1, kSoftmaxWarps * 32>();
            // ---- epilogue: lane L < 64 holds head L, dv [256 n, 256 n + 128) in columns n * 128 + j;
            // lane 64 + L holds head L, dv [256 n + 128, 256 n + 256).  The two warps of a quadrant
            // take one n each.  Read in the accumulator fragment layout (16 lanes at a time: thread T
            // gets rows T/4 and T/4 + 8, two columns of every eight), so that a store instruction
            // writes whole 32-byte sectors: 8 rows x 4 lanes x 8 bytes.
            ok &= mbar_wait(ctx, bar(kBarOFull), seg_it & 1, kBarOFull);
            tcgen05_fence_after();
            {
                float *obase;
                int64_t ostride;
                if (seg.slot < 0) {
                    obase = p.out + (int64_t)seg.request * p.out_stride_request + (int64_t)head0 * p.out_stride_head;
                    ostride = p.out_stride_head;
                } else {
                    obase = p.partial_out + ((int64_t)seg.slot * h + (head0 - p.head_begin)) * kDV;
                    ostride = kDV;
                }
                const int n = cf;
                const int dv0 = 256 * n + 128 * g + 2 * (lane & 3);
                const int nvalid = min(kN, p.head_end - head0);
                // A partial piece is stored as f16.  So that neither large nor tiny cache values leave f16's range, every
                // row is first multiplied by the power of two that puts its largest entry into [2^14, 2^15) -- exact --
                // and the inverse goes to partial_scale beside the row's LSE for the combine kernel.  The row maximum
                // takes one more pass over the accumulator: this thread's four rows over its 128 columns, the 4 lanes
                // that share a row, then the 4 warps that hold the row's other columns (through the exchange buffer).
                float up[2][2] = {{1.f, 1.f}, {1.f, 1.f}};        // 2^k of rows (half, A / B)
                if (seg.slot >= 0) {
                    float mx[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll 1
                    for (int hc = 0; hc < 4; ++hc) {
                        const int half = hc >> 1, c = hc & 1;
                        float o[32];
                        tmem_ld_16x256b_x8(tmem_base + ((uint32_t)(32 * q4 + 16 * half) << 16) + kColO + n * 128 + c * 64, o);
                        tmem_wait_ld();
                        float a = 0.f, b = 0.f;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            a = fmaxf(a, fmaxf(fabsf(o[4 * k]), fabsf(o[4 * k + 1])));
                            b = fmaxf(b, fmaxf(fabsf(o[4 * k + 2]), fabsf(o[4 * k + 3])));
                        }
                        if (half == 0) { mx[0][0] = fmaxf(mx[0][0], a); mx[0][1] = fmaxf(mx[0][1], b); }
                        else { mx[1][0] = fmaxf(mx[1][0], a); mx[1][1] = fmaxf(mx[1][1], b); }
                    }
#pragma unroll
                    for (int half = 0; half < 2; ++half)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int row = 32 * (q4 & 1) + 16 * half + 8 * e + (lane >> 2);
                            float v = mx[half][e] * l_s[row];
                            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
                            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
                            if ((lane & 3) == 0) xch[row * 4 + slot4] = v;
                        }
                    named_bar_sync_dyn<128>(2 + half_id);
#pragma unroll
                    for (int half = 0; half < 2; ++half)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int row = 32 * (q4 & 1) + 16 * half + 8 * e + (lane >> 2);
                            const float4 x4 = *reinterpret_cast<const float4 *>(&xch[row * 4]);
                            const float rmax = fmaxf(fmaxf(x4.x, x4.y), fmaxf(x4.z, x4.w));
                            const int ex = (int)((__float_as_uint(rmax) >> 23) & 0xffu);
                            int k = (ex == 0 || ex == 255) ? 0 : 14 - (ex - 127);      // zero / subnormal / non-finite rows stay as they are
                            k = max(-100, min(100, k));
                            up[half][e] = __uint_as_float((uint32_t)(127 + k) << 23);
                            if (slot4 == 0 && (lane & 3) == 0 && row < nvalid)
                                p.partial_scale[(int64_t)seg.slot * h + (head0 - p.head_begin) + row] = __uint_as_float((uint32_t)(127 - k) << 23);
                        }
                    named_bar_sync_dyn<128>(2 + half_id);            // the exchange buffer may be written again
                }
#pragma unroll 1
                for (int hc = 0; hc < 4; ++hc) {
                    const int half = hc >> 1, c = hc & 1;
                    const int hA = 32 * (q4 & 1) + 16 * half + (lane >> 2), hB = hA + 8;
                    float o[32];
                    tmem_ld_16x256b_x8(tmem_base + ((uint32_t)(32 * q4 + 16 * half) << 16) + kColO + n * 128 + c * 64, o);
                    const float iA = l_s[hA] * (half ? up[1][0] : up[0][0]), iB = l_s[hB] * (half ? up[1][1] : up[0][1]);
                    float *rowA = obase + (int64_t)hA * ostride + dv0 + c * 64, *rowB = obase + (int64_t)hB * ostride + dv0 + c * 64;
                    tmem_wait_ld();
                    if (seg.slot >= 0) {
                        // a partial piece: f16 rows of the slot (the combine kernel weighs and sums them in fp32)
                        __half *base16 = reinterpret_cast<__half *>(p.partial_out) + ((int64_t)seg.slot * h + (head0 - p.head_begin)) * kDV;
                        // A thread holds columns 8 k + 2 i, + 1 (i = lane & 3) of its two rows.  Neighbouring lanes swap one
                        // packed pair per two k, so that every lane owns four consecutive columns (8 bytes) and a store
                        // instruction writes whole 32-byte sectors: even lanes columns 16 k' + 2 i .. + 3, odd lanes
                        // 16 k' + 8 + 2 (i - 1) .. + 3.
                        const int i4 = lane & 3;
                        const int col = (i4 & 1) ? 8 + 2 * (i4 - 1) : 2 * i4;
                        uint2 *hrowA = reinterpret_cast<uint2 *>(base16 + (int64_t)hA * kDV + 256 * n + 128 * g + c * 64 + col);
                        uint2 *hrowB = reinterpret_cast<uint2 *>(base16 + (int64_t)hB * kDV + 256 * n + 128 * g + c * 64 + col);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            const uint32_t a0 = pack_f16x2(o[8 * kk] * iA, o[8 * kk + 1] * iA), a1 = pack_f16x2(o[8 * kk + 4] * iA, o[8 * kk + 5] * iA);
                            const uint32_t b0 = pack_f16x2(o[8 * kk + 2] * iB, o[8 * kk + 3] * iB), b1 = pack_f16x2(o[8 * kk + 6] * iB, o[8 * kk + 7] * iB);
                            // even lanes keep the first of their two pairs and get the partner's first; odd lanes the second
                            const uint32_t ra = __shfl_xor_sync(0xffffffffu, (i4 & 1) ? a0 : a1, 1);
                            const uint32_t rb = __shfl_xor_sync(0xffffffffu, (i4 & 1) ? b0 : b1, 1);
                            const uint2 va = (i4 & 1) ? make_uint2(ra, a1) : make_uint2(a0, ra);
                            const uint2 vb = (i4 & 1) ? make_uint2(rb, b1) : make_uint2(b0, rb);
                            if (hA < nvalid) hrowA[4 * kk] = va;          // 16 halves on
                            if (hB < nvalid) hrowB[4 * kk] = vb;
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            if (hA < nvalid) *reinterpret_cast<float2 *>(rowA + 8 * k) = make_float2(o[4 * k] * iA, o[4 * k + 1] * iA);
                            if (hB < nvalid) *reinterpret_cast<float2 *>(rowB + 8 * k) = make_float2(o[4 * k + 2] * iB, o[4 * k + 3] * iB);
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) arrive_on_leader(kBarOEmpty);
            ++seg_it;
        }
    }

    fill_empty_requests(p, worker, head0, kN, tid, kThreads);
    if (p.trace != nullptr && tid == 0) {   // per-CTA cycles and nanoseconds
        p.trace[512 + blockIdx.x] = clock64() - t_start;
        if (blockIdx.x < 256) p.trace[768 + blockIdx.x] = (long long)(global_timer_ns() - ns_start);
    }

    // ---- teardown: nobody leaves while its partner may still touch its shared memory or barriers
    if (*ctx.abort_flag) {
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { __nanosleep(1000); }
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace

cudaError_t launch_decode_umma_pair(const DecodeParams &p, cudaStream_t stream) {
    alignas(64) CUtensorMap mhalf, mpeer, mq;
    const uint64_t pages = (uint64_t)(p.num_pool_pages > 0 ? p.num_pool_pages : 1);
    if (!make_map_4d(&mhalf, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, p.kv_pool, kPage, pages,
                     (uint64_t)kDQK * 2, 128, (uint64_t)kPage * kDQK * 2, kHalf, 9))
        return cudaErrorInvalidValue;
    if (!make_map_4d(&mpeer, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, p.kv_pool, kPage, pages,
                     (uint64_t)kDQK * 2, 128, (uint64_t)kPage * kDQK * 2, kHalf, 2))
        return cudaErrorInvalidValue;
    if (!make_map_4d(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, p.q, (uint64_t)p.H,
                     (uint64_t)p.B, (uint64_t)p.q_stride_head * 2, 128,
                     (uint64_t)(p.B > 1 ? p.q_stride_request : p.q_stride_head * p.H) * 2, (uint32_t)kN, 9))
        return cudaErrorInvalidValue;
    static DeviceOnce once;
    cudaError_t e = once.run([&] { return cudaFuncSetAttribute(decode_umma_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes); });
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.num_workers * p.pair_groups * 2)); cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = stream;
    cudaLaunchAttribute attr[1];      // (the cluster shape is part of the kernel's declaration)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, decode_umma_pair_kernel, p, mhalf, mpeer, mq);
    count_launch();
    return e;
}

}  // namespace splash
