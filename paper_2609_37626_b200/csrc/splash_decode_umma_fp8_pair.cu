// e4m3 decode kernel for slices of 65..128 heads: a CLUSTER OF TWO CTAs per KV worker that
// issues its MMAs with tcgen05 cta_group::2.
//
// Why: with both operands in shared memory a small MMA costs what its operands cost to
// stream ((A + B bytes) / 128 B per cycle).  Two independent 64-head CTAs each stream every
// K row and every V row themselves.  A CTA pair shares them:
//
//   S [128 heads x 128 tokens] = Q K^T      M = 128 (64 heads per CTA), N = 128: each CTA supplies
//                                            ONE page (64 tokens) as its half of the B operand
//   O [128 heads x 256 dv]    += P V        M = 128, N = 256 (x 2 halves of dv): each CTA supplies
//                                            its 64 heads of P and 128 of the 256 dv columns
//
// so per 128 tokens and per CTA the tensor cores read 72 KB (QK^T) + 96 KB (P.V) instead of
// 288 + 192 KB.  A "supertile" is two consecutive page tiles of a segment: CTA r loads page r
// (all 9 chunks of 64 columns) into a stage for QK^T.  For P.V CTA r supplies dv columns
// [256 n + 128 r, + 128) of BOTH pages, at the same shared-memory offsets in both CTAs (the
// two CTAs of an MMA share one descriptor).  Its own page already has them in chunk slots
// 4 n + 2 r, 4 n + 2 r + 1 of the stage; the other four latent chunk slots of the stage hold
// columns only the peer needs, so once QK^T of the stage has retired they are overwritten
// with the peer page's chunks 4 n + 2 r, 4 n + 2 r + 1.  The MMAs over page g then start at
// slot 4 n + 2 g in both CTAs.  That second load hides behind the softmax of the supertile.
// Accumulators: CTA r holds its 64 heads; a head's row is TMEM lane h (tokens / dv of the
// first half of N) and lane 64 + h (second half).
//
// Roles per CTA (576 threads): K-page + scale producer, 2 QK^T issuers and 2 P.V issuers
// (leader CTA only), 8 softmax warps, 4 query converters, 1 producer of the peer chunks.
// Barriers that the issuers wait on live in the leader; the peer's warps arrive on them across
// the cluster (relaxed arrivals: what they announce is already in place on the peer's SM), and
// TMA loads of the peer complete on them too.
#include "splash_fp8.cuh"
#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kQkWarps = 2, kPvWarps = 2, kSoftmaxWarps = 8, kConvertWarps = 4;
constexpr int kWarpProducer = 0;
constexpr int kWarpQk = 1;
constexpr int kWarpPv = kWarpQk + kQkWarps;
constexpr int kWarpSoftmax = kWarpPv + kPvWarps;
constexpr int kWarpConvert = kWarpSoftmax + kSoftmaxWarps;
constexpr int kWarpVProducer = kWarpConvert + kConvertWarps;
constexpr int kThreads = (kWarpVProducer + 1) * 32;    // 18 warps = 576 threads
constexpr int kN = 64;                              // heads per CTA
constexpr uint32_t kSlab = 64 * 64;                 // 64 rows x 64 B
constexpr uint32_t kPageBytes = 9 * kSlab;          // 36,864
constexpr uint32_t kPeerBytes = 4 * kSlab;          // the peer page's chunks this CTA multiplies: 16,384
constexpr uint32_t kScaleBytes = 256;
constexpr int kStages = 3;
constexpr int kPrefetchAhead = 1;                    // supertiles between the L2 prefetch of a page and its use (4: 1.5 % slower; none: 5 %)
constexpr int kPrefetchAheadBusy = 4;                // the same while the call carries a page-copy job
constexpr float kTau = 7.0f;                          // (6 / 2.75: 0.3 % slower on the rollout workload, 4 / 4.75 more)
constexpr float kLift = 1.75f;

enum BarrierId {
    kBarKFull = 0,                        // [3] leader: both CTAs' pages landed (tx bytes of both)
    kBarQkDone = kBarKFull + kStages,     // [3] QK^T of the stage retired (multicast commit): peer chunks may land
    kBarVFull = kBarQkDone + kStages,     // [3] leader: both CTAs' peer chunks landed
    kBarStageEmpty = kBarVFull + kStages, // [3] P.V of the stage retired (multicast commit): stage, its scales and
                                          //     the P buffer are free, O is up to date
    kBarScFull = kBarStageEmpty + kStages,// [3] local: scale pages of the stage landed
    kBarQFull = kBarScFull + kStages,     // leader: query operands of both CTAs written
    kBarQLocal,                           // local: this CTA's query scales written
    kBarQEmpty,                           // last QK^T of the request retired (multicast commit)
    kBarQsRead,                           // local: the softmax warps have picked up the request's query scales
    kBarSFull,                            // [2] S buffer written (multicast commit)
    kBarSEmpty = kBarSFull + 2,           // [2] S buffer read (leader: by both CTAs)
    kBarPFull = kBarSEmpty + 2,           // [2] P buffer written (leader: by both CTAs)
    kBarOFull = kBarPFull + 2,            // last P.V of the request retired (multicast commit)
    kBarOEmpty,                           // O drained (leader: by both CTAs)
    kNumBarriers
};

constexpr uint32_t kOffK = 0;                                   // [3 stages] 9 chunk slots
constexpr uint32_t kOffQHi = kOffK + kStages * kPageBytes;
constexpr uint32_t kOffQLo = kOffQHi + kN * kDQK;
constexpr uint32_t kOffP = kOffQLo + kN * kDQK;                 // [2 buffers][hi, lo][2 page slabs] x 4096
constexpr uint32_t kOffScale = kOffP + 2 * 2 * 2 * kSlab;       // float [3 stages][2 pages][64]
constexpr uint32_t kOffQs = kOffScale + kStages * 2 * kScaleBytes;    // float [4][64]
constexpr uint32_t kOffAlpha = kOffQs + 4 * kN * 4;             // float [64]
constexpr uint32_t kOffL = kOffAlpha + kN * 4;                  // float [64]
constexpr uint32_t kOffXch = kOffL + kN * 4;                    // float [64][4]
constexpr uint32_t kTokBytes = 32 * 8 + 32 * 4;                 // per warp: (scale, log2 scale) x 32, 1 / scale x 32
constexpr uint32_t kOffTok = kOffXch + kN * 16;
constexpr uint32_t kOffBar = kOffTok + kSoftmaxWarps * kTokBytes;
constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;
constexpr uint32_t kSmemBytes = kOffMisc + 32;
static_assert(kSmemBytes <= 232448, "shared memory overflow");
static_assert(kOffQHi % 1024 == 0 && kOffP % 1024 == 0 && kOffTok % 16 == 0 && kTokBytes % 16 == 0, "alignment");
// tensor memory: O two halves of dv x 128 columns, then 2 S buffers x 2 partials x 64 columns
constexpr uint32_t kColO = 0, kColS = 256;

__device__ __forceinline__ void umma_e4m3_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
decode_umma_fp8_pair_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_page,
                            const __grid_constant__ CUtensorMap tmap_pair, const __grid_constant__ CUtensorMap tmap_out,
                            const __grid_constant__ CUtensorMap tmap_part) {
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
            mbar_init(bar(kBarScFull + s), 1);
        }
        mbar_init(bar(kBarQFull), 2 * kConvertWarps); mbar_init(bar(kBarQLocal), kConvertWarps); mbar_init(bar(kBarQEmpty), kQkWarps);
        mbar_init(bar(kBarQsRead), kSoftmaxWarps);
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
    // geometry of supertile s of the current segment: page tiles 2s (page A, CTA 0) and 2s + 1 (page B, CTA 1)
    auto pair_geom = [&](int s) -> PairGeom {
        PairGeom g;
        const int first_page = seg.lo / kPage;
        const int ta = seg.tile_begin + 2 * s, tb = ta + 1;
        g.a = tile_geom(seg.lo, seg.hi, (first_page + ta) * kPage);
        g.has_b = tb < seg.tile_end;
        if (g.has_b) g.b = tile_geom(seg.lo, seg.hi, (first_page + tb) * kPage);
        else { g.b.tok0 = 0; g.b.r_lo = 0; g.b.r_hi = 0; g.b.a = 0; g.b.b = 0; g.b.both = false; }
        return g;
    };

    if (warp == kWarpProducer || warp == kWarpVProducer) {
        // ===================================================== TMA producers
        // warp 0: this CTA's page and the scale pages of both pages, up to three supertiles ahead;
        // last warp: the peer page's chunks, into the dead half of the stage once QK^T has read it
        const bool is_v = warp == kWarpVProducer;
        uint32_t st_it = 0;                               // supertile counter
        bool ok = true;
        while (ok && it.next(p, seg)) {
            const int first_page = seg.lo / kPage;
            const int32_t *table = p.block_table + (int64_t)seg.request * p.table_stride;
            const int nsuper = (seg.tile_end - seg.tile_begin + 1) >> 1;
            for (int s = 0; ok && s < nsuper; ++s, ++st_it) {
                const PairGeom g = pair_geom(s);
                const int ta = seg.tile_begin + 2 * s;
                const uint32_t stage = st_it % kStages, ph = (st_it / kStages) & 1;
                const uint32_t k0 = sbase + kOffK + stage * kPageBytes;
                // the page this warp fetches: its CTA's own for QK^T, the other CTA's for the P.V chunks.  A tile cut at
                // both ends inside its page is written by hand instead (zeros outside the range); only a request whose
                // whole range lies inside one page has such a tile, and it is page A.
                const TileGeom &tg = (rank == 0) != is_v ? g.a : g.b;
                int page_a = 0, page_b = 0;
                if (lane == 0) {
                    page_a = table[first_page + ta];
                    page_b = g.has_b ? table[first_page + ta + 1] : p.num_pool_pages;   // a page past the pool reads as zeros
                    if (!is_v) {
                        ok = mbar_wait(ctx, bar(kBarStageEmpty + stage), ph ^ 1, kBarStageEmpty + stage);
                        if (ok) {
                            // the leader's barrier expects the pages of both CTAs
                            if (rank == 0) mbar_expect_tx(bar(kBarKFull + stage), 2 * kPageBytes);
                            if (!tg.both)
                                tma_load_4d_pair(k0, &tmap_page, leader_bar(kBarKFull + stage), 0, tg.tok0, 0, rank == 0 ? page_a : page_b);
                            // scale pages of both pages, for this CTA's softmax warps
                            const bool in_a = page_a >= 0 && page_a < p.num_pool_pages;
                            const bool in_b = g.has_b && page_b >= 0 && page_b < p.num_pool_pages;
                            if (!in_a || (g.has_b && !in_b)) {     // a page outside the pool reads as zeros; give its tokens the scale 1
                                float *sc1 = reinterpret_cast<float *>(smem + kOffScale + stage * 2 * kScaleBytes);
                                for (int t = 0; t < kPage; ++t) {
                                    if (!in_a) sc1[t] = 1.0f;
                                    if (g.has_b && !in_b) sc1[kPage + t] = 1.0f;
                                }
                            }
                            mbar_expect_tx(bar(kBarScFull + stage), (in_a ? kScaleBytes : 0u) + (in_b ? kScaleBytes : 0u));
                            const uint32_t sdst = sbase + kOffScale + stage * 2 * kScaleBytes;
                            if (in_a) bulk_load(sdst, p.kv_scales + (int64_t)page_a * kPage, kScaleBytes, bar(kBarScFull + stage));
                            if (in_b) bulk_load(sdst + kScaleBytes, p.kv_scales + (int64_t)page_b * kPage, kScaleBytes, bar(kBarScFull + stage));
                            // A stage is held from its load until P.V has read it, about three supertiles, so the
                            // load of supertile s + 3 starts only when the issuers are about to need it: have its
                            // page in L2 by then.
                            // (further ahead while a page-copy job shares the memory system: the loads then take longer)
                            const int tf = ta + 2 * (p.mig_n > 0 ? kPrefetchAheadBusy : kPrefetchAhead) + (int)rank;
                            if (tf < seg.tile_end) {
                                const int page_f = table[first_page + tf];
                                if (page_f >= 0 && page_f < p.num_pool_pages) tma_prefetch_4d(&tmap_page, 0, 0, 0, page_f);
                            }
                        }
                    } else {
                        ok = mbar_wait(ctx, bar(kBarQkDone + stage), ph, kBarQkDone + stage);
                        if (ok) {
                            if (rank == 0) mbar_expect_tx(bar(kBarVFull + stage), 2 * kPeerBytes);
                            // peer page chunks 4n + 2 rank, + 1 -> slots 4n + 2 (1 - rank), + 1
                            if (!tg.both) {
#pragma unroll
                                for (int n = 0; n < 2; ++n)
                                    tma_load_4d_pair(k0 + (4 * n + 2 * (1 - (int)rank)) * kSlab, &tmap_pair, leader_bar(kBarVFull + stage), 0,
                                                     tg.tok0, 4 * n + 2 * (int)rank, rank == 0 ? page_b : page_a);
                            }
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (ok && tg.both) {
                    const int page = __shfl_sync(0xffffffffu, (rank == 0) != is_v ? page_a : page_b, 0);
                    const uint8_t *src = page >= 0 && page < p.num_pool_pages
                        ? static_cast<const uint8_t *>(p.kv_pool) + (size_t)page * (kPage * kDQK) : nullptr;
                    uint8_t *slabs = smem + kOffK + stage * kPageBytes;
                    if (!is_v) {
                        fill_rows_by_hand<64>(slabs, kSlab, kPage, src, tg.tok0, tg.a, tg.b, 0, 0, 9, lane);
                    } else {
                        for (int n = 0; n < 2; ++n)
                            fill_rows_by_hand<64>(slabs, kSlab, kPage, src, tg.tok0, tg.a, tg.b, 4 * n + 2 * (int)rank,
                                                  4 * n + 2 * (1 - (int)rank), 2, lane);
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_complete_tx_cluster(leader_bar(is_v ? kBarVFull + stage : kBarKFull + stage), is_v ? kPeerBytes : kPageBytes);
                }
            }
        }
    } else if (warp >= kWarpQk && warp < kWarpQk + kQkWarps && rank == 0) {
        // ===================================================== QK^T issuers (leader CTA)
        if (lane == 0) {
            const int a = warp - kWarpQk;                 // partial accumulator a
            constexpr uint32_t kIdescQK = make_idesc_e4m3(128, 128, 0);
            uint32_t st_it = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                const int nsuper = (seg.tile_end - seg.tile_begin + 1) >> 1;
                ok = mbar_wait_cluster(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
                for (int s = 0; ok && s < nsuper; ++s, ++st_it) {
                    const uint32_t stage = st_it % kStages, b = st_it & 1;
                    ok = mbar_wait_cluster(ctx, bar(kBarKFull + stage), (st_it / kStages) & 1, kBarKFull + stage) &&
                         mbar_wait_cluster(ctx, bar(kBarSEmpty + b), ((st_it >> 1) & 1) ^ 1, kBarSEmpty + b);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t k0 = sbase + kOffK + stage * kPageBytes;
                    const uint32_t d = tmem_base + kColS + (b * kQkWarps + a) * kN;
                    // 18 K = 32 steps x (q hi, q lo) = 36 MMAs per supertile; this issuer takes every second
#pragma unroll
                    for (int t = 0; t < 36 / kQkWarps; ++t) {
                        const int idx = t * kQkWarps + a, hl = idx / 18, ks = idx % 18, c = ks >> 1, k = ks & 1;
                        const uint32_t q0 = sbase + (hl ? kOffQLo : kOffQHi);
                        uint64_t dq = make_desc_sw64(q0 + c * kSlab + k * 32, 16, 512);     // A: 2 x 64 heads x 32
                        uint64_t dk = make_desc_sw64(k0 + c * kSlab + k * 32, 16, 512);     // B: 2 x 64 tokens x 32
                        umma_e4m3_pair(d, dq, dk, kIdescQK, t != 0);
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
            constexpr uint32_t kIdescPV = make_idesc_e4m3(128, 256, 0, 0, 1, 0);
            constexpr uint32_t kIdescPVLo = make_idesc_e4m3(128, 256, 0, 0, 1, 1);   // P lo is e5m2 (A operand)
            uint32_t st_it = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                const int nsuper = (ntiles + 1) >> 1;
                for (int s = 0; ok && s < nsuper; ++s, ++st_it) {
                    const uint32_t stage = st_it % kStages, pb = st_it & 1;
                    ok = mbar_wait_cluster(ctx, bar(kBarVFull + stage), (st_it / kStages) & 1, kBarVFull + stage) &&
                         mbar_wait_cluster(ctx, bar(kBarPFull + pb), (st_it >> 1) & 1, kBarPFull + pb);
                    if (ok && s == 0) ok = mbar_wait_cluster(ctx, bar(kBarOEmpty), (seg_it & 1) ^ 1, kBarOEmpty);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t k0 = sbase + kOffK + stage * kPageBytes;
                    const bool has_b = 2 * s + 1 < ntiles;
                    const int ksteps = has_b ? 4 : 2;     // 32 tokens each; page B's are skipped when it does not exist
#pragma unroll
                    for (int hl = 0; hl < 2; ++hl) {
                        const uint32_t p0 = sbase + kOffP + (pb * 2 + hl) * 2 * kSlab;
                        for (int ks = 0; ks < ksteps; ++ks) {
                            // A: P rows, slab = page, 32 tokens; B: slots 4n + 2 page, + 1 (two 64-wide dv chunks, LBO), 32 tokens
                            const int pg = ks >> 1;
                            uint64_t da = make_desc_sw64(p0 + pg * kSlab + (ks & 1) * 32, 16, 512);
                            uint64_t db = make_desc_sw64(k0 + (4 * n + 2 * pg) * kSlab + (ks & 1) * 2048, kSlab, 512);
                            umma_e4m3_pair(tmem_base + kColO + n * 128, da, db, hl ? kIdescPVLo : kIdescPV, (s != 0) || (hl | ks) != 0);
                        }
                    }
                    umma_commit_pair(bar(kBarStageEmpty + stage));
                    if (s + 1 == nsuper) umma_commit_pair(bar(kBarOFull));
                }
                ++seg_it;
            }
        }
    } else if (warp >= kWarpQk && warp < kWarpSoftmax) {
        // the issuer warps of the peer CTA have nothing to do for the attention itself: they carry the call's page-copy
        // job, if it has one (a layer's pages on the move while this layer decodes)
        if (p.mig_n > 0)
            copy_pages_in_idle_warp(p, pair_id * (kQkWarps + kPvWarps) + (warp - kWarpQk), p.num_workers * p.pair_groups * (kQkWarps + kPvWarps), lane);
    } else if (warp >= kWarpConvert && warp < kWarpConvert + kConvertWarps) {
        // ===================================================== query converters (this CTA's 64 heads)
        const int ct = (warp - kWarpConvert) * 32 + lane;   // 0..127
        float *qs_s = reinterpret_cast<float *>(smem + kOffQs);
        uint32_t seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            {
                const int hd = ct >> 1, part = ct & 1;
                const int gh = head0 + hd;
                const bool live = gh < p.head_end;
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const __nv_bfloat16 *>(p.q) + (int64_t)seg.request * p.q_stride_request +
                    (int64_t)(live ? gh : p.head_begin) * p.q_stride_head + part * 288);
                // first pass (row maximum) while the previous request is still being multiplied
                float amax = 0.f;
                if (live) {
#pragma unroll 1
                    for (int v0 = 0; v0 < 36; v0 += 12) {
                        uint4 x[12];
#pragma unroll
                        for (int i = 0; i < 12; ++i) x[i] = __ldg(src + v0 + i);
#pragma unroll
                        for (int i = 0; i < 12; ++i) {
                            const uint32_t w[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                amax = fmaxf(amax, fabsf(__uint_as_float(w[k] << 16)));
                                amax = fmaxf(amax, fabsf(__uint_as_float(w[k] & 0xffff0000u)));
                            }
                        }
                    }
                }
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                const float qs = amax > 0.f ? amax * (1.0f / 448.0f) : 1.0f;
                const float inv = amax > 0.f ? 448.0f / amax : 1.0f;
                if (part == 0) qs_s[(seg_it & 3) * kN + hd] = qs;
                // second pass in four batches of nine 16-byte loads, a batch ahead: the first batch is in
                // flight while this warp waits for the operand buffers, which are free once the last
                // QK^T of the previous request has retired
                uint4 xa[9], xb[9];
                auto load_batch = [&](uint4 (&x)[9], int v0) {
#pragma unroll
                    for (int i = 0; i < 9; ++i) x[i] = live ? __ldg(src + v0 + i) : make_uint4(0u, 0u, 0u, 0u);
                };
                auto convert_batch = [&](const uint4 (&x)[9], int v0) {
#pragma unroll
                    for (int i = 0; i < 9; ++i) {
                        const uint32_t w[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
                        uint16_t hi[4], lo[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float e0 = __uint_as_float(w[k] << 16) * inv, e1 = __uint_as_float(w[k] & 0xffff0000u) * inv;
                            split_e4m3_e4m3_x2(e0, e1, hi[k], lo[k]);      // packed f16 arithmetic: half the instructions
                        }
                        const uint32_t d = (uint32_t)(part * 288 + (v0 + i) * 8);
                        const uint32_t off = (d >> 6) * kSlab + sw64((uint32_t)hd, d & 63);
                        *reinterpret_cast<uint2 *>(smem + kOffQHi + off) =
                            make_uint2((uint32_t)hi[0] | ((uint32_t)hi[1] << 16), (uint32_t)hi[2] | ((uint32_t)hi[3] << 16));
                        *reinterpret_cast<uint2 *>(smem + kOffQLo + off) =
                            make_uint2((uint32_t)lo[0] | ((uint32_t)lo[1] << 16), (uint32_t)lo[2] | ((uint32_t)lo[3] << 16));
                    }
                };
                load_batch(xa, 0);
                ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
                if (!ok) break;
                load_batch(xb, 9);  convert_batch(xa, 0);
                load_batch(xa, 18); convert_batch(xb, 9);
                load_batch(xb, 27); convert_batch(xa, 18);
                convert_batch(xb, 27);
                fence_proxy_async();
                __syncwarp();
                // The softmax warps wait on QLocal by phase parity, so it must never complete two phases
                // ahead of them: hold this request's arrival until they have entered the previous one.
                if (lane == 0) {
                    if (seg_it > 0) ok = mbar_wait(ctx, bar(kBarQsRead), (seg_it - 1) & 1, kBarQsRead);
                    mbar_arrive(bar(kBarQLocal)); arrive_on_leader(kBarQFull);
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            }
            ++seg_it;
        }
    } else {
        // ===================================================== softmax + epilogue warps
        // S partial layout per CTA: TMEM lane L < 64 = head L, tokens of page A in 64 columns;
        // lane 64 + L = head L, tokens of page B.  Two warps per quadrant take 32 columns each,
        // so a thread owns ONE head and 32 tokens of one page.
        const int sw = warp - kWarpSoftmax;             // 0..7
        const int q4 = warp & 3;                        // TMEM lane quadrant
        const int cf = sw >> 2;                         // column half: tokens [32 cf, 32 cf + 32) of the page
        const int pg = q4 >> 1;                         // 0: page A, 1: page B
        const int hd = 32 * (q4 & 1) + lane;            // this thread's head (0..63 within the CTA)
        const int half_id = q4 & 1;                     // heads 0-31 or 32-63: the four warps that share them sync on bar 2 + half_id
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        float *qs_s = reinterpret_cast<float *>(smem + kOffQs);
        float *alpha_s = reinterpret_cast<float *>(smem + kOffAlpha);
        float *l_s = reinterpret_cast<float *>(smem + kOffL);
        float *xch = reinterpret_cast<float *>(smem + kOffXch);
        // per-warp table of its 32 tokens, read back as 16-byte broadcasts:
        // tok_a[j / 2] = (scale_j, log2 scale_j, scale_j+1, log2 scale_j+1), tok_r[j / 4] = 1 / scale of four tokens
        float4 *tok_a = reinterpret_cast<float4 *>(smem + kOffTok + sw * kTokBytes);
        float4 *tok_r = tok_a + 16;
        const float *scale_s = reinterpret_cast<const float *>(smem + kOffScale);
        const float scale_log2 = p.softmax_scale * kLog2e;
        const int slot4 = pg * 2 + cf;                  // this thread's slot among the 4 threads of its head
        uint32_t st_it = 0, seg_it = 0;
        // A failed (timed-out) wait only clears `ok`; the role keeps walking its supertiles so that every
        // thread still meets the named barriers -- once the CTA aborts, waits return at once.
        bool ok = true;
        while (it.next(p, seg)) {
            ok &= mbar_wait(ctx, bar(kBarQLocal), seg_it & 1, kBarQLocal);
            const float cq = scale_log2 * qs_s[(seg_it & 3) * kN + hd];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQsRead));
            float m = -INFINITY, l = 0.f;
            const int nsuper = (seg.tile_end - seg.tile_begin + 1) >> 1;
            // several query rows per request: this thread's (virtual) head is row (head mod R) and sees the
            // tokens below causal_end only
            const int causal_end = p.q_rows > 1 ? p.seq_lens[seg.request] - (p.q_rows - 1 - (head0 + hd) % p.q_rows) : 0x3fffffff;   // (far above any token index, and safe to subtract a negative offset from)
            for (int s = 0; s < nsuper; ++s, ++st_it) {
                const PairGeom g = pair_geom(s);
                const TileGeom geo = pg ? g.b : g.a;
                const uint32_t stage = st_it % kStages, b = st_it & 1;
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (st_it >> 1) & 1, kBarSFull + b);
                ok &= mbar_wait(ctx, bar(kBarScFull + stage), (st_it / kStages) & 1, kBarScFull + stage);
                tcgen05_fence_after();
                float sv[32];
                {
                    float part[32];
                    const uint32_t sb = tmem_base + lane_addr + kColS + (b * kQkWarps) * kN + 32 * cf;
                    tmem_ld32(sb, sv);
                    tmem_ld32(sb + kN, part);
                    // meanwhile: lane j prepares token 32 cf + j.  A token outside the range gets scale 0 and
                    // log2 scale -inf; its row of K may hold anything, so its logit is also forced below.
                    const int r = 32 * cf + lane;
                    const bool v = r >= geo.r_lo && r < geo.r_hi;
                    const float ts = v ? scale_s[(stage * 2 + pg) * 64 + geo.tok0 + r] : 0.f;
                    reinterpret_cast<float2 *>(tok_a)[lane] = make_float2(ts, v ? fast_log2(ts) : -INFINITY);
                    reinterpret_cast<float *>(tok_r)[lane] = v ? fast_rcp(ts) : 0.f;
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) sv[j] += part[j];
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) arrive_on_leader(kBarSEmpty + b);
                uint32_t valid = __ballot_sync(0xffffffffu, 32 * cf + lane >= geo.r_lo && 32 * cf + lane < geo.r_hi);
                {
                    // how many of this thread's 32 tokens lie below its head's causal end: token j of the thread is
                    // token (page index) * 64 + tok0 + 32 cf + j of the request
                    const int lim = causal_end - ((seg.lo / kPage + seg.tile_begin + 2 * s + pg) * kPage + geo.tok0 + 32 * cf);
                    if (lim < 32) valid &= lim <= 0 ? 0u : (1u << lim) - 1u;
                }
                float mt = -INFINITY;
                if (__all_sync(0xffffffffu, valid == 0xffffffffu)) {
#pragma unroll
                    for (int j2 = 0; j2 < 16; ++j2) {
                        const float4 t = tok_a[j2];
                        sv[2 * j2] = fmaf(sv[2 * j2], cq * t.x, t.y);
                        sv[2 * j2 + 1] = fmaf(sv[2 * j2 + 1], cq * t.z, t.w);
                        mt = fmaxf(mt, fmaxf(sv[2 * j2], sv[2 * j2 + 1]));
                    }
                } else {
#pragma unroll
                    for (int j2 = 0; j2 < 16; ++j2) {
                        const float4 t = tok_a[j2];
                        sv[2 * j2] = (valid >> (2 * j2)) & 1u ? fmaf(sv[2 * j2], cq * t.x, t.y) : -INFINITY;
                        sv[2 * j2 + 1] = (valid >> (2 * j2 + 1)) & 1u ? fmaf(sv[2 * j2 + 1], cq * t.z, t.w) : -INFINITY;
                        mt = fmaxf(mt, fmaxf(sv[2 * j2], sv[2 * j2 + 1]));
                    }
                }
                // row maximum over the 4 threads of this head (2 pages x 2 column halves, 4 different warps)
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
                const float off = kLift - (m == -INFINITY ? 0.f : m);   // a head that has seen no token yet: all weights 0, not NaN
                uint32_t phi[8], plo[8];
#pragma unroll
                for (int j4 = 0; j4 < 8; ++j4) {
                    const float4 rt = tok_r[j4];
                    const float rts[4] = {rt.x, rt.y, rt.z, rt.w};
                    float u[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        u[e] = fast_exp2(sv[4 * j4 + e] + off);
                        l = fmaf(u[e], rts[e], l);
                    }
                    uint16_t h01, h23, r01, r23;
                    split_e4m3_e5m2_x2(u[0], u[1], h01, r01);
                    split_e4m3_e5m2_x2(u[2], u[3], h23, r23);
                    phi[j4] = (uint32_t)h01 | ((uint32_t)h23 << 16);
                    plo[j4] = (uint32_t)r01 | ((uint32_t)r23 << 16);
                }
                const bool rescale = named_bar_or<1, kSoftmaxWarps * 32>(grew);
                // P.V of the supertile that last used this P buffer (two back) must be done; a rescale
                // of O also needs the previous supertile's P.V
                if (st_it > 1) ok &= mbar_wait(ctx, bar(kBarStageEmpty + (st_it - 2) % kStages), ((st_it - 2) / kStages) & 1, kBarStageEmpty);
                if (rescale && s > 0) {
                    ok &= mbar_wait(ctx, bar(kBarStageEmpty + (st_it - 1) % kStages), ((st_it - 1) / kStages) & 1, kBarStageEmpty);
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
                    // P hi / lo: K-major, 64-byte swizzle; slab = page, row = head, bytes [32 cf, 32 cf + 32)
                    uint8_t *ph = smem + kOffP + ((b * 2 + 0) * 2 + pg) * kSlab;
                    uint8_t *pl = smem + kOffP + ((b * 2 + 1) * 2 + pg) * kSlab;
#pragma unroll
                    for (int u16 = 0; u16 < 2; ++u16) {
                        const uint32_t o = sw64((uint32_t)hd, (uint32_t)(32 * cf + 16 * u16));
                        *reinterpret_cast<uint4 *>(ph + o) = make_uint4(phi[4 * u16], phi[4 * u16 + 1], phi[4 * u16 + 2], phi[4 * u16 + 3]);
                        *reinterpret_cast<uint4 *>(pl + o) = make_uint4(plo[4 * u16], plo[4 * u16 + 1], plo[4 * u16 + 2], plo[4 * u16 + 3]);
                    }
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
                    float lse = lt > 0.f ? (m - kLift + log2f(lt)) * kLn2 : -INFINITY;
                    if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                    else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                }
            }
            named_bar_sync<1, kSoftmaxWarps * 32>();
            // ---- epilogue: lane L < 64 holds head L, dv [256 n, 256 n + 128) in columns n * 128 + j;
            // lane 64 + L holds head L, dv [256 n + 128, 256 n + 256).  The two warps of a quadrant
            // take one n each.
            ok &= mbar_wait(ctx, bar(kBarOFull), seg_it & 1, kBarOFull);
            tcgen05_fence_after();
            // Every warp drains its [32 heads x 128 dv] block in four rounds of 32 columns through a
            // 4 KB tile of the P buffers (idle now: the last P.V has retired): a thread writes its row
            // in the 128-byte swizzle (conflict-free), one TMA store moves the tile out in whole lines
            // and clips the rows past the head slice.
            {
                const int n = cf;
                const int dv0 = 256 * n + 128 * pg;
                const int row0 = 32 * (q4 & 1);
                uint8_t *stg = smem + kOffP + sw * 4096;
                const float inv_l = l_s[hd];
                const bool final_out = seg.slot < 0;
                const CUtensorMap *omap = final_out ? &tmap_out : &tmap_part;
                const int rowc = final_out ? head0 + row0 : head0 - p.head_begin + row0;
                const int outer = final_out ? seg.request : seg.slot;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    float o[32];
                    tmem_ld32(tmem_base + lane_addr + kColO + n * 128 + c * 32, o);
                    tmem_wait_ld();
                    if (c > 0) {                          // the previous round's store has read the tile
                        if (lane == 0) bulk_wait_group_read();
                        __syncwarp();
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<float4 *>(stg + lane * 128 + ((i ^ (lane & 7)) << 4)) =
                            make_float4(o[4 * i] * inv_l, o[4 * i + 1] * inv_l, o[4 * i + 2] * inv_l, o[4 * i + 3] * inv_l);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) { tma_store_3d(omap, smem_u32(stg), dv0 + 32 * c, rowc, outer); bulk_commit_group(); }
                }
                if (lane == 0) bulk_wait_group_read();    // the tile goes back to being a P buffer
                __syncwarp();
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

cudaError_t launch_decode_umma_fp8_pair(const DecodeParams &p, cudaStream_t stream) {
    alignas(64) CUtensorMap mpage, mpair;
    const uint64_t pages = (uint64_t)(p.num_pool_pages > 0 ? p.num_pool_pages : 1);
    if (!make_map_4d(&mpage, CU_TENSOR_MAP_DATA_TYPE_UINT8, CU_TENSOR_MAP_SWIZZLE_64B, p.kv_pool, kPage, pages,
                     (uint64_t)kDQK, 64, (uint64_t)kPage * kDQK, 64, 9))
        return cudaErrorInvalidValue;
    if (!make_map_4d(&mpair, CU_TENSOR_MAP_DATA_TYPE_UINT8, CU_TENSOR_MAP_SWIZZLE_64B, p.kv_pool, kPage, pages,
                     (uint64_t)kDQK, 64, (uint64_t)kPage * kDQK, 64, 2))
        return cudaErrorInvalidValue;
    // output maps: (512 dv, heads below head_end, requests) over `out`, (512, h, partial slots) over the workspace
    alignas(64) CUtensorMap mout, mpart;
    if (p.out_stride_head % 4 || p.out_stride_request % 4) return cudaErrorNotSupported;   // rows must start on 16-byte boundaries
    const uint64_t hbytes = (uint64_t)p.out_stride_head * 4;
    if (!make_store_map_3d(&mout, p.out, kDV, (uint64_t)p.head_end, (uint64_t)p.B, hbytes,
                           p.B > 1 ? (uint64_t)p.out_stride_request * 4 : hbytes * (uint64_t)p.head_end, 32))
        return cudaErrorNotSupported;
    const uint64_t h = (uint64_t)(p.head_end - p.head_begin);
    if (!make_store_map_3d(&mpart, p.partial_out, kDV, h, (uint64_t)2 * p.num_workers, (uint64_t)kDV * 4, h * kDV * 4, 32))
        return cudaErrorInvalidValue;
    static DeviceOnce once;
    cudaError_t e = once.run([&] { return cudaFuncSetAttribute(decode_umma_fp8_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes); });
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.num_workers * p.pair_groups * 2)); cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = stream;
    cudaLaunchAttribute attr[1];      // (the cluster shape is part of the kernel's declaration)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, decode_umma_fp8_pair_kernel, p, mpage, mpair, mout, mpart);
    count_launch();
    return e;
}

}  // namespace splash
