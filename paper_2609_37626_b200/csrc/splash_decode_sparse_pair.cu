// Sparse decode kernel: attention over a LIST of tokens per request, cache rows in the 656-byte
// format (512 e4m3 latent codes, four float scales -- one per 128 latent dims --, 64 bf16 rope
// values; Sec. 5 setup, App. B payload), on a CLUSTER OF TWO CTAs per KV worker issuing
// tcgen05 cta_group::2 MMAs.
//
// The contractions, the softmax, the accumulators and the epilogue are those of the bf16
// CTA-pair kernel: per tile of 64 listed tokens
//   S [128 heads x 64 tokens] = Q K^T      M = 128 (64 heads per CTA), N = 64: each CTA supplies 32 tokens
//   O [128 heads x 256 dv]   += P V        M = 128, N = 256 (x 2 halves of dv): each CTA supplies 128 dv columns
// over a bf16 tile in shared memory (9 chunk slabs of 32 tokens x 128 B, 128-byte swizzle; after
// QK^T the four latent slots this CTA does not multiply are overwritten with the peer's tokens'
// columns that it does).  What differs is where the tile comes from: no TMA can fetch scattered
// 656-byte rows into that layout, so
//   * an address warp walks the token list a few tiles ahead: list entry -> page id -> row
//     address, four tiles abreast so that the chain of dependent loads is paid once per four
//     tiles; it leaves the addresses in a ring in shared memory and pulls the rows into L2;
//   * the eight softmax warps copy the raw rows into a staging area (one bulk copy per row, no
//     registers held while the rows travel) and, between the softmax of one tile and the next,
//     dequantise from there (code x block scale, as f16 -- tile, query rows and P are f16 in
//     this kernel) into the swizzled tile: this CTA's 32 tokens in full for QK^T, and the peer's
//     32 tokens' 256 columns for P.V once QK^T has retired.  Each warp copies and converts its
//     own four rows only, so the staging area needs no barrier.
// Every listed row crosses HBM once (twice through L2: the peer reads it too).
//
// Roles per CTA (480 threads): address warp, 4 QK^T issuers and 2 P.V issuers (leader CTA only;
// the first issuer warp of either CTA also loads that CTA's query rows), 8 softmax warps that
// also copy and convert the rows.  Barriers that the issuers wait on live in the leader; the peer's warps
// arrive on them across the cluster (relaxed arrivals: what they announce is already in place on
// the peer's SM).
#include <cuda_bf16.h>

#include "splash_fp8.cuh"
#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kQkWarps = 4, kPvWarps = 2, kSoftmaxWarps = 8;
constexpr int kWarpAddr = 0;
constexpr int kWarpQk = 1;
constexpr int kWarpPv = kWarpQk + kQkWarps;
constexpr int kWarpSoftmax = kWarpPv + kPvWarps;       // 7: TMEM quadrant = warp & 3
constexpr int kThreads = (kWarpSoftmax + kSoftmaxWarps) * 32;   // 15 warps = 480 threads
constexpr int kRowsPerWarp = 4;                         // raw rows a softmax warp copies and converts per tile and duty
constexpr int kN = 64;                              // heads per CTA
constexpr int kHalf = 32;                           // tokens per CTA and tile
constexpr uint32_t kSlab = kHalf * 128;             // one chunk of a half-page: 32 tokens x 128 B
constexpr uint32_t kStageBytes = 9 * kSlab;         // 36,864
constexpr uint32_t kQSlab = kN * 128;               // one chunk of the query rows: 64 heads x 128 B
constexpr uint32_t kQBytes = 9 * kQSlab;            // 73,728
constexpr uint32_t kPHalfBytes = kN * 64;           // P of one half-page: 64 heads x 32 tokens bf16
constexpr int kStages = 2;
constexpr int kRing = 8;                            // tiles of row addresses the address warp may be ahead
constexpr int kAddrBatch = 4;                       // tiles whose addresses are resolved abreast
constexpr uint32_t kRowBytes = 656;                 // a cache row: 512 codes, 4 scales, 64 bf16 rope values
constexpr uint32_t kVRowBytes = 528;                // a peer row without its rope part: 512 codes, 4 scales (P.V reads half the codes)
constexpr float kTau = 8.0f;                        // O is rescaled only when a row maximum grows by more than 2^8

enum BarrierId {
    kBarKFull = 0,                        // [2] leader: both CTAs' 32 tokens converted (all converter warps of both)
    kBarQkDone = kBarKFull + kStages,     // [2] QK^T of the stage retired (multicast commit): peer columns may be written
    kBarVFull = kBarQkDone + kStages,     // [2] leader: both CTAs' peer columns converted
    kBarStageEmpty = kBarVFull + kStages, // [2] P.V of the stage retired (multicast commit): stage and P buffers
                                          //     are free, O is up to date
    kBarQFull = kBarStageEmpty + kStages, // leader: query rows of both CTAs converted to f16 (all softmax warps of both)
    kBarQLanded,                          // local: this CTA's query rows (bf16) landed
    kBarQEmpty,                           // last QK^T of the request retired (multicast commit)
    kBarSFull,                            // [2] S buffer written (multicast commit)
    kBarSEmpty = kBarSFull + 2,           // [2] S buffer read (leader: by both CTAs)
    kBarPFull = kBarSEmpty + 2,           // [2] P buffer written (leader: by both CTAs)
    kBarOFull = kBarPFull + 2,            // last P.V of the request retired (multicast commit)
    kBarOEmpty,                           // O drained (leader: by both CTAs)
    kBarAddrFull,                         // [8] local: row addresses of a tile written to the ring
    kBarAddrEmpty = kBarAddrFull + kRing, // [8] local: the converter warps are done with the ring slot
    kBarRaw = kBarAddrEmpty + kRing,      // [8 warps][own tokens, peer columns] local: a softmax warp's raw rows landed (tx bytes)
    kNumBarriers = kBarRaw + 2 * kSoftmaxWarps
};

constexpr uint32_t kOffK = 0;                                   // [2 stages] 9 chunk slots of 32 tokens
constexpr uint32_t kOffQ = kOffK + kStages * kStageBytes;       // 9 chunks x 64 heads x 128 B
constexpr uint32_t kOffP1 = kOffQ + kQBytes;                    // [2 buffers] P of half-page 1: 64 heads x 64 B
constexpr uint32_t kRawKBytes = kHalf * kRowBytes, kRawVBytes = kHalf * kVRowBytes;
constexpr uint32_t kOffRawK = kOffP1 + 2 * kPHalfBytes;         // raw rows of this CTA's 32 tokens: 32 x 656 B
constexpr uint32_t kOffRawV = kOffRawK + kRawKBytes;            // the peer's 32 tokens, codes and scales: 32 x 528 B
constexpr uint32_t kOffRing = kOffRawV + kRawVBytes;            // uint64 [8][64] row addresses (0: zero row, 1: poisoned row)
constexpr uint32_t kOffAlpha = kOffRing + kRing * 64 * 8;       // float [64]
constexpr uint32_t kOffL = kOffAlpha + kN * 4;                  // float [64]
constexpr uint32_t kOffXch = kOffL + kN * 4;                    // float [64][4]
constexpr uint32_t kOffBar = kOffXch + kN * 16;
constexpr uint32_t kOffMisc = (kOffBar + kNumBarriers * 8 + 15) / 16 * 16;
constexpr uint32_t kSmemBytes = kOffMisc + 32;
static_assert(kSmemBytes <= 232448, "shared memory overflow");
static_assert(kOffQ % 1024 == 0 && kOffP1 % 1024 == 0 && kSlab % 1024 == 0, "swizzle atoms need 1024-byte alignment");
static_assert(kOffRawK % 16 == 0 && kOffRawV % 16 == 0 && kOffRing % 8 == 0 && kOffBar % 8 == 0, "alignment");
// tensor memory: O two halves of dv x 128 columns, then 2 S buffers x 4 partials x 32 columns
constexpr uint32_t kColO = 0, kColS = 256;

// The tile, the query rows and P are F16 here, not BF16: an e4m3 code becomes f16 exactly in one instruction and
// the block scale is one packed multiply, where the way to bf16 leads through fp32 and costs three times the
// instructions -- and the converter warps are what bounds this kernel.  (f16 also keeps three more significant
// bits of code x scale.  Its range, 6e-5 .. 65504 for normal numbers, holds latent values and queries with room
// to spare; a block scale above 146 would overflow.)
constexpr uint32_t kF16Formats = ~((1u << 7) | (1u << 10));     // instruction descriptor: A and B formats F16 (0), not BF16 (1)
constexpr uint32_t kF16NanPair = 0x7E007E00u;

__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
    return pack_f16x2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint16_t v) {
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
    return r;
}
__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// 4 e4m3 codes (one 32-bit word) times a scale (the same in both halves of s2) -> 4 f16 (two words)
__device__ __forceinline__ uint2 dequant4(uint32_t w, uint32_t s2) {
    return make_uint2(hmul2(e4m3x2_to_f16x2((uint16_t)(w & 0xffffu)), s2), hmul2(e4m3x2_to_f16x2((uint16_t)(w >> 16)), s2));
}

__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
decode_sparse_pair_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_q) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();             // 0 = leader: issues the MMAs
    const int worker = blockIdx.x >> 1;
    const int head0 = p.head_begin + (int)rank * kN;
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
            mbar_init(bar(kBarKFull + s), 2 * kSoftmaxWarps); mbar_init(bar(kBarQkDone + s), kQkWarps);
            mbar_init(bar(kBarVFull + s), 2 * kSoftmaxWarps); mbar_init(bar(kBarStageEmpty + s), kPvWarps);
        }
        for (int s = 0; s < 2 * kSoftmaxWarps; ++s) mbar_init(bar(kBarRaw + s), 1);
        for (int s = 0; s < kRing; ++s) { mbar_init(bar(kBarAddrFull + s), 1); mbar_init(bar(kBarAddrEmpty + s), kSoftmaxWarps); }
        mbar_init(bar(kBarQFull), 2 * kSoftmaxWarps); mbar_init(bar(kBarQLanded), 1); mbar_init(bar(kBarQEmpty), kQkWarps);
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

    if (warp == kWarpAddr) {
        // ===================================================== address warp
        // Box row R of a tile holds list entry tile * 64 + tok0 + R (tile_geom with lo = 0: a short last tile is
        // aligned to the end of the box, the rows before it are zero).  Lane l resolves rows l and 32 + l of each
        // of four consecutive tiles at once, so the two dependent loads (list entry, page id) cost one round trip
        // each per four tiles.  Address 0 stands for a zero row, 1 for a poisoned one (a list entry outside the
        // request, a page id outside the pool, a count outside [0, len_cap]).
        unsigned long long *ring = reinterpret_cast<unsigned long long *>(smem + kOffRing);
        const uint8_t *pool = static_cast<const uint8_t *>(p.kv_pool);
        uint32_t kv_it = 0;
        bool ok = true, more = it.next(p, seg);
        int tile = more ? seg.tile_begin : 0;
        while (ok && more) {
            int n_tiles = 0;
            int tok[kAddrBatch][2], len[kAddrBatch];
            const int32_t *table[kAddrBatch];
            unsigned long long addr[kAddrBatch][2];
#pragma unroll
            for (int u = 0; u < kAddrBatch; ++u) {
                tok[u][0] = tok[u][1] = -1; len[u] = 0; table[u] = p.block_table; addr[u][0] = addr[u][1] = 0ull;
                if (!more) continue;
                n_tiles = u + 1;
                const int cnt = p.seq_lens[seg.request];
                const bool bad_count = cnt < 0 || cnt > p.len_cap;
                const TileGeom g = tile_geom(seg.lo, seg.hi, tile * kPage);
                const int32_t *list = p.sel + (int64_t)seg.request * p.sel_stride;
                len[u] = p.ctx_lens[seg.request];
                table[u] = p.block_table + (int64_t)seg.request * p.table_stride;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int R = 32 * e + lane;
                    if (R >= g.r_lo && R < g.r_hi) {
                        addr[u][e] = 1ull;                                           // poisoned unless resolved below
                        if (!bad_count) tok[u][e] = __ldg(list + tile * kPage + g.tok0 + R);
                    }
                }
                if (++tile == seg.tile_end) { more = it.next(p, seg); tile = more ? seg.tile_begin : 0; }
            }
            int page[kAddrBatch][2];
#pragma unroll
            for (int u = 0; u < kAddrBatch; ++u)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool live = addr[u][e] == 1ull && tok[u][e] >= 0 && tok[u][e] < len[u];
                    page[u][e] = live ? __ldg(table[u] + tok[u][e] / kPage) : -1;
                }
#pragma unroll
            for (int u = 0; u < kAddrBatch; ++u) {
                if (u >= n_tiles) continue;
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (page[u][e] >= 0 && page[u][e] < p.num_pool_pages)
                        addr[u][e] = reinterpret_cast<unsigned long long>(pool + ((int64_t)page[u][e] * kPage + tok[u][e] % kPage) * kRowBytes);
                const uint32_t slot = kv_it % kRing, ph = (kv_it / kRing) & 1;
                if (lane == 0) ok = mbar_wait(ctx, bar(kBarAddrEmpty + slot), ph ^ 1, kBarAddrEmpty + slot);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                ring[slot * 64 + lane] = addr[u][0];
                ring[slot * 64 + 32 + lane] = addr[u][1];
                // this CTA's own 32 tokens of the tile: into L2 ahead of the converter warps' copies
                const unsigned long long own = rank == 0 ? addr[u][0] : addr[u][1];
                if (own > 1ull) bulk_prefetch_l2(reinterpret_cast<const void *>(own), kRowBytes);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarAddrFull + slot));
                ++kv_it;
            }
        }
    } else if (warp >= kWarpQk && warp < kWarpQk + kQkWarps && rank == 0) {
        // ===================================================== QK^T issuers (leader CTA)
        // One thread sustains one tcgen05.mma per ~65 cycles and a chain of MMAs into one accumulator
        // runs at the MMA latency, so the 36 K = 16 steps of a tile go to four issuers with a partial
        // accumulator each.
        if (lane == 0) {
            const int a = warp - kWarpQk;
            constexpr uint32_t kIdescQK = make_idesc(128, 64, 0, 0) & kF16Formats;
            uint32_t kv_it = 0, seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                if (a == 0) {
                    // the query rows of the request, once the last QK^T of the previous one has retired
                    ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
                    if (!ok) break;
                    mbar_expect_tx(bar(kBarQLanded), kQBytes);
                    tma_load_4d(sbase + kOffQ, &tmap_q, bar(kBarQLanded), 0, head0, 0, seg.request);
                }
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
            constexpr uint32_t kIdescPV = make_idesc(128, 256, 0, 1) & kF16Formats;
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
    } else if (warp == kWarpQk) {
        // peer CTA: its first issuer warp only loads the query rows of this CTA's heads
        if (lane == 0) {
            uint32_t seg_it = 0;
            bool ok = true;
            while (ok && it.next(p, seg)) {
                ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
                if (ok) {
                    mbar_expect_tx(bar(kBarQLanded), kQBytes);
                    tma_load_4d(sbase + kOffQ, &tmap_q, bar(kBarQLanded), 0, head0, 0, seg.request);
                }
                ++seg_it;
            }
        }
    } else if (warp >= kWarpQk && warp < kWarpSoftmax) {
        // the other issuer warps of the peer CTA have nothing to do
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

        // ---- the same eight warps also build the tiles (separate converter warps ran an order of magnitude below
        // their instruction count: a dozen roles per SM wait on instruction fetch; eight warps that walk the same
        // loops do not).  Warp sw owns rows 4 sw .. 4 sw + 3 of this CTA's 32 tokens (all 576 columns) and of the
        // peer's 32 tokens (the 256 latent columns this CTA multiplies in P.V): it copies the raw rows (one bulk
        // copy per row, lane u < 4 issues row u; they complete on the warp's own barrier) and later converts the
        // rows it copied, so the staging area needs no barrier of its own.  Tile kv + 1 is built while P.V of tile
        // kv - 1 has long retired (after the softmax of tile kv); the peer columns of tile kv follow at once, QK^T
        // of tile kv having retired before its softmax could start.
        const unsigned long long *ring = reinterpret_cast<const unsigned long long *>(smem + kOffRing);
        uint32_t total = 0;         // tiles of this worker: the building duties do not care about request boundaries
        {
            SegmentIter it2 = it;
            Segment seg2;
            while (it2.next(p, seg2)) total += (uint32_t)(seg2.tile_end - seg2.tile_begin);
        }
        const int raw_bar_k = kBarRaw + 2 * sw, raw_bar_v = raw_bar_k + 1;
        // Ask for the raw rows of two tiles at once: this CTA's tokens of tile kv_own (lanes 0-3, one row each) and the
        // peer's tokens of tile kv_peer (lanes 4-7).  What becomes of each row -- copied, zero, poisoned -- is kept in
        // two 4-bit masks per duty, so that the builders need not read the ring again.
        uint32_t own_valid = 0, own_poison = 0, peer_valid = 0, peer_poison = 0;
        auto issue_rows = [&](uint32_t kv_own, uint32_t kv_peer) {
            const bool do_own = kv_own < total, do_peer = kv_peer < total;
            if (!do_own && !do_peer) return;
            if (do_own) ok &= mbar_wait(ctx, bar(kBarAddrFull + kv_own % kRing), (kv_own / kRing) & 1, kBarAddrFull);
            if (do_peer) ok &= mbar_wait(ctx, bar(kBarAddrFull + kv_peer % kRing), (kv_peer / kRing) & 1, kBarAddrFull);
            const int duty = lane >> 2, u = lane & 3;          // lanes 0-3: own rows, 4-7: peer rows
            const bool mine = ok && lane < 8 && (duty == 0 ? do_own : do_peer);
            const int t = kRowsPerWarp * sw + u;
            const uint32_t slot = (duty == 0 ? kv_own : kv_peer) % kRing;
            const int half_of_rows = duty == 0 ? (int)rank : 1 - (int)rank;
            const unsigned long long a = mine ? ring[slot * 64 + 32 * half_of_rows + t] : 0ull;
            const unsigned valid = __ballot_sync(0xffffffffu, a > 1ull), poison = __ballot_sync(0xffffffffu, a == 1ull);
            if (do_own) { own_valid = valid & 15u; own_poison = poison & 15u; }
            if (do_peer) { peer_valid = (valid >> 4) & 15u; peer_poison = (poison >> 4) & 15u; }
            fence_proxy_async();          // the rows' staging space was last read through the generic proxy
            __syncwarp();
            if (lane == 0) {
                if (do_own) mbar_expect_tx(bar(raw_bar_k), (uint32_t)__popc(valid & 15u) * kRowBytes);
                if (do_peer) mbar_expect_tx(bar(raw_bar_v), (uint32_t)__popc(valid & 0xf0u) * kVRowBytes);
            }
            __syncwarp();
            if (a > 1ull) {
                if (duty == 0) bulk_load(sbase + kOffRawK + t * kRowBytes, reinterpret_cast<const void *>(a), kRowBytes, bar(raw_bar_k));
                else bulk_load(sbase + kOffRawV + t * kVRowBytes, reinterpret_cast<const void *>(a), kVRowBytes, bar(raw_bar_v));
            }
        };
        // this CTA's tokens of tile kv: raw rows -> f16 rows of the stage (needs P.V of tile kv - kStages retired).
        // All loads of the four rows first, then the arithmetic and the stores.
        auto build_own = [&](uint32_t kv) {
            if (kv >= total) return;
            const uint32_t stage = kv % kStages, sph = (kv / kStages) & 1;
            ok &= mbar_wait(ctx, bar(raw_bar_k), kv & 1, raw_bar_k);
            ok &= mbar_wait(ctx, bar(kBarStageEmpty + stage), sph ^ 1, kBarStageEmpty + stage);
            uint8_t *k0 = smem + kOffK + stage * kStageBytes;
            // lane l: codes [16 l, 16 l + 16) = units 2 (l & 3), + 1 of chunk l >> 2; rope word l of the ninth chunk
            uint8_t *dst_lane = k0 + (lane >> 2) * kSlab;
            const uint32_t u0 = 2 * (lane & 3);
            const uint32_t valid = ok ? own_valid : 0u;
            uint4 lat[kRowsPerWarp];
            float scf[kRowsPerWarp];
            uint32_t rope[kRowsPerWarp];
#pragma unroll
            for (int u = 0; u < kRowsPerWarp; ++u) {
                const uint8_t *src = smem + kOffRawK + (kRowsPerWarp * sw + u) * kRowBytes;
                if ((valid >> u) & 1u) {
                    lat[u] = *reinterpret_cast<const uint4 *>(src + 16 * lane);
                    scf[u] = *reinterpret_cast<const float *>(src + 512 + 4 * (lane >> 3));
                    rope[u] = *reinterpret_cast<const uint32_t *>(src + 528 + 4 * lane);
                }
            }
#pragma unroll
            for (int u = 0; u < kRowsPerWarp; ++u) {
                const int t = kRowsPerWarp * sw + u;
                uint4 lo, hi;
                uint32_t rp;
                if ((valid >> u) & 1u) {
                    const uint32_t sc = pack_f16x2(scf[u], 0.f);
                    const uint32_t s2 = __byte_perm(sc, sc, 0x1010);          // the scale in both halves
                    const uint2 x0 = dequant4(lat[u].x, s2), x1 = dequant4(lat[u].y, s2), x2 = dequant4(lat[u].z, s2), x3 = dequant4(lat[u].w, s2);
                    lo = make_uint4(x0.x, x0.y, x1.x, x1.y); hi = make_uint4(x2.x, x2.y, x3.x, x3.y);
                    rp = bf16x2_to_f16x2(rope[u]);
                } else {
                    const uint32_t fill = ((own_poison >> u) & 1u) ? kF16NanPair : 0u;
                    lo = hi = make_uint4(fill, fill, fill, fill);
                    rp = fill;
                }
                uint8_t *dst = dst_lane + t * 128;
                *reinterpret_cast<uint4 *>(dst + ((u0 ^ (t & 7)) << 4)) = lo;
                *reinterpret_cast<uint4 *>(dst + (((u0 + 1) ^ (t & 7)) << 4)) = hi;
                *reinterpret_cast<uint32_t *>(k0 + 8 * kSlab + t * 128 + ((((lane >> 2) ^ (t & 7))) << 4) + 4 * (lane & 3)) = rp;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) arrive_on_leader(kBarKFull + stage);
        };
        // the peer's tokens of tile kv, the columns this CTA multiplies in P.V: into the slots QK^T of the tile has left
        auto build_peer = [&](uint32_t kv) {
            const uint32_t stage = kv % kStages, sph = (kv / kStages) & 1, slot = kv % kRing;
            ok &= mbar_wait(ctx, bar(raw_bar_v), kv & 1, raw_bar_v);
            ok &= mbar_wait(ctx, bar(kBarQkDone + stage), sph, kBarQkDone + stage);
            uint8_t *k0 = smem + kOffK + stage * kStageBytes;
            // lane l = 16 n + 8 e + w: codes [8 w, + 8) of chunk 4 n + 2 rank + e -> unit w of slot 4 n + 2 (1 - rank) + e
            const int n = lane >> 4, e = (lane >> 3) & 1, w = lane & 7;
            uint8_t *dst_slot = k0 + (4 * n + 2 * (1 - (int)rank) + e) * kSlab;
            const uint32_t code_off = (4 * n + 2 * (int)rank + e) * 64 + 8 * w, scale_off = 512 + 4 * (2 * n + (int)rank);
            const uint32_t valid = ok ? peer_valid : 0u;
            uint2 codes[kRowsPerWarp];
            float scf[kRowsPerWarp];
#pragma unroll
            for (int u = 0; u < kRowsPerWarp; ++u) {
                const uint8_t *src = smem + kOffRawV + (kRowsPerWarp * sw + u) * kVRowBytes;
                if ((valid >> u) & 1u) {
                    codes[u] = *reinterpret_cast<const uint2 *>(src + code_off);
                    scf[u] = *reinterpret_cast<const float *>(src + scale_off);
                }
            }
#pragma unroll
            for (int u = 0; u < kRowsPerWarp; ++u) {
                const int t = kRowsPerWarp * sw + u;
                uint4 v;
                if ((valid >> u) & 1u) {
                    const uint32_t sc = pack_f16x2(scf[u], 0.f);
                    const uint32_t s2 = __byte_perm(sc, sc, 0x1010);
                    const uint2 x0 = dequant4(codes[u].x, s2), x1 = dequant4(codes[u].y, s2);
                    v = make_uint4(x0.x, x0.y, x1.x, x1.y);
                } else {
                    const uint32_t fill = ((peer_poison >> u) & 1u) ? kF16NanPair : 0u;
                    v = make_uint4(fill, fill, fill, fill);
                }
                *reinterpret_cast<uint4 *>(dst_slot + t * 128 + ((w ^ (t & 7)) << 4)) = v;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) { arrive_on_leader(kBarVFull + stage); mbar_arrive(bar(kBarAddrEmpty + slot)); }
        };
        // diagnostic timeline of the first softmax warp of CTA 0: S landed, P written, own tokens of the next tile
        // built, peer columns built, next rows asked for
        long long *const trace = (blockIdx.x == 0 && sw == 0 && lane == 0) ? p.trace : nullptr;
        auto mark = [&](uint32_t tile, int ev) { if (trace != nullptr && tile < 64) trace[tile * 8 + ev] = clock64(); };
        issue_rows(0, 0);
        build_own(0);
        issue_rows(1, 0xffffffffu);       // (the masks now describe tile 1 / tile 0: the builders of the loop run before the next request)

        while (it.next(p, seg)) {
            float m = -INFINITY, l = 0.f;               // running maximum in scaled log2 units
            const int first_page = seg.lo / kPage;
            {
                // the query rows arrive as bf16; the tile is f16 (see the converter warps), so they are rewritten in
                // place, element for element (exact: eight significant bits fit f16's eleven), before QK^T may read them
                ok &= mbar_wait(ctx, bar(kBarQLanded), seg_it & 1, kBarQLanded);
                uint4 *qv = reinterpret_cast<uint4 *>(smem + kOffQ);
                for (int i = sw * 32 + lane; i < (int)(kQBytes / 16); i += kSoftmaxWarps * 32) {
                    uint4 x = qv[i];
                    x.x = bf16x2_to_f16x2(x.x); x.y = bf16x2_to_f16x2(x.y); x.z = bf16x2_to_f16x2(x.z); x.w = bf16x2_to_f16x2(x.w);
                    qv[i] = x;
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) arrive_on_leader(kBarQFull);
            }
            // several query rows per request: this thread's (virtual) head is row (head mod R) and sees the
            // tokens below causal_end only
            const int causal_end = p.q_rows > 1 ? p.seq_lens[seg.request] - (p.q_rows - 1 - (head0 + hd) % p.q_rows) : 0x3fffffff;   // (far above any token index, and safe to subtract a negative offset from)
            for (int tile = seg.tile_begin; tile < seg.tile_end; ++tile, ++kv_it) {
                const TileGeom geo = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);   // (lo = 0: list positions)
                const uint32_t b = kv_it & 1;
                mark(kv_it, 0);
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (kv_it >> 1) & 1, kBarSFull + b);
                mark(kv_it, 1);
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
                    pk[j >> 1] = pack_f16x2(u0, u1);
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
                // ---- the tiles ahead: this CTA's tokens of the next tile, then the peer's columns of this one
                mark(kv_it, 2);
                build_own(kv_it + 1);
                mark(kv_it, 3);
                build_peer(kv_it);
                mark(kv_it, 4);
                issue_rows(kv_it + 2, kv_it + 1);
                mark(kv_it, 5);
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
                    // (a poisoned row makes the sum NaN: it is passed on, so that the request's LSE is NaN like its output)
                    float lse = lt > 0.f ? (m + log2f(lt)) * kLn2 : (lt == 0.f ? -INFINITY : lt);
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
#pragma unroll 1
                for (int hc = 0; hc < 4; ++hc) {
                    const int half = hc >> 1, c = hc & 1;
                    const int hA = 32 * (q4 & 1) + 16 * half + (lane >> 2), hB = hA + 8;
                    float o[32];
                    tmem_ld_16x256b_x8(tmem_base + ((uint32_t)(32 * q4 + 16 * half) << 16) + kColO + n * 128 + c * 64, o);
                    const float iA = l_s[hA], iB = l_s[hB];
                    float *rowA = obase + (int64_t)hA * ostride + dv0 + c * 64, *rowB = obase + (int64_t)hB * ostride + dv0 + c * 64;
                    tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (hA < nvalid) *reinterpret_cast<float2 *>(rowA + 8 * k) = make_float2(o[4 * k] * iA, o[4 * k + 1] * iA);
                        if (hB < nvalid) *reinterpret_cast<float2 *>(rowB + 8 * k) = make_float2(o[4 * k + 2] * iB, o[4 * k + 3] * iB);
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

cudaError_t launch_decode_sparse_pair(const DecodeParams &p, cudaStream_t stream) {
    alignas(64) CUtensorMap mq;
    if (!make_map_4d(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, p.q, (uint64_t)p.H,
                     (uint64_t)p.B, (uint64_t)p.q_stride_head * 2, 128,
                     (uint64_t)(p.B > 1 ? p.q_stride_request : p.q_stride_head * p.H) * 2, (uint32_t)kN, 9))
        return cudaErrorInvalidValue;
    static DeviceOnce once;
    cudaError_t e = once.run([&] { return cudaFuncSetAttribute(decode_sparse_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes); });
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.num_workers * 2)); cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = stream;
    cudaLaunchAttribute attr[1];      // (the cluster shape is part of the kernel's declaration)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, decode_sparse_pair_kernel, p, mq);
    count_launch();
    return e;
}

}  // namespace splash
