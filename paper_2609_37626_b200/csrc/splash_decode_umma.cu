// tcgen05 / TMA decode kernel for sm_100a.
//
// One CTA per (KV worker, head group).  A head group is N = 16, 32 or 64 query heads
// of one request; the CTA streams the request's pages through shared memory and keeps
// the transposed problem in tensor memory ("tokens on M"):
//
//     S^T [64 tokens x N heads]  = K_tile [64 x 576]   * Q^T [576 x N]      (M = 64)
//     O^T [512 dv    x N heads] += V_tile^T [512 x 64] * P^T [64 x N]       (4 x M = 128)
//
// so a 16-head TP/DOP slice costs a 16-wide MMA instead of a padded 64/128-row one,
// and both contractions read the SAME shared-memory tile: V is the first 512 columns
// of the K rows (the latent), taken as an MN-major operand, so every KV byte crosses
// HBM once per head group.
//
// Warp roles (288 threads):
//   warp 0     TMA producer: block-table driven page gathers into a ring of stages
//              (nine 64x64-element boxes per page, 128-byte swizzle), and the query
//              rows of each segment.  Page tails and unaligned KV ranges are handled
//              by shifting the box in the token dimension so that out-of-range tokens
//              fall outside the page and are zero-filled by the TMA unit.
//   warps 1-4  MMA issuers (one thread each).  One thread sustains only one tcgen05.mma
//              per ~65 cycles whatever the shape, far below the pipe's rate for these
//              small-N MMAs, so the work is spread: every issuer owns one of the
//              independent S^T partial accumulators and one of the four dv blocks of
//              O^T, runs its own ready-driven loop over the barriers and commits its
//              own MMAs (the consumer barriers count one arrival per issuer).  QK^T of
//              tile i+1 is issued while the softmax warps handle tile i.
//   warps 5-8  online softmax over tokens (= TMEM lanes): per-head maxima by a
//              warp-shuffle reduce-scatter plus a small shared-memory exchange, lazy
//              rescaling of O^T (only when a maximum grows by more than 2^8), P written
//              to shared memory as the K-major B operand, epilogue.
//
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA records
// SPLASH_DEVICE_TIMEOUT in the workspace status block, raises a CTA-wide abort flag,
// lets copies in flight land, frees its tensor memory and returns.
#include "splash_pair.cuh"

namespace splash {

namespace {

using namespace umma;

constexpr int kThreads = 288;                      // 9 warps: producer, 4 MMA issuers, 4 softmax
constexpr int kMmaWarps = 4;
constexpr int kNumSoftmaxWarps = 4;                // barriers fed by the softmax role count one arrival per warp
constexpr int kChunks = 9;                         // 576 / 64-element (128 B) chunks
constexpr uint32_t kSlabBytes = 64 * 128;          // one chunk of one page: 64 tokens x 128 B
constexpr uint32_t kStageBytes = kChunks * kSlabBytes;   // 73,728
constexpr int kStages = 2;
constexpr int kPrefetchTiles = 1;                  // tiles between the L2 prefetch of a page and its load (2: 1.6 % slower, 4: 14 %)
constexpr float kRescaleThreshold = 8.0f;          // log2 units

enum BarrierId {
    kBarKvFull = 0,                    // [kStages]
    kBarKvEmpty = kBarKvFull + kStages,
    kBarQFull = kBarKvEmpty + kStages,
    kBarQEmpty,
    kBarSFull,                         // [2]
    kBarSEmpty = kBarSFull + 2,        // [2]
    kBarPFull = kBarSEmpty + 2,
    kBarOFull,
    kBarOEmpty,
    kNumBarriers
};

template <int N>
struct Layout {
    static constexpr uint32_t kQBytes = N * kDQK * 2;
    static constexpr uint32_t kPBytes = N * 128;             // N rows (heads) x 64 tokens bf16
    static constexpr uint32_t kOffKv = 0;
    static constexpr uint32_t kOffQ = kOffKv + kStages * kStageBytes;
    static constexpr uint32_t kOffP = kOffQ + kQBytes;
    // output staging for the narrow groups, [N heads][256 dv] floats: the finished tile leaves through the bulk-copy engine
    // (64-head groups have no shared memory left for it and store from registers)
    static constexpr uint32_t kOutBytes = N < 64 ? N * 1024 : 0;
    static constexpr uint32_t kOffOut = kOffP + kPBytes;
    static constexpr uint32_t kOffRed = kOffOut + kOutBytes; // float [N][4]
    static constexpr uint32_t kOffM = kOffRed + N * 16;      // float [N] running max, log2 domain
    static constexpr uint32_t kOffAlpha = kOffM + N * 4;     // float [N]
    static constexpr uint32_t kOffL = kOffAlpha + N * 4;     // float [N]
    static constexpr uint32_t kOffBar = kOffL + N * 4;       // uint64 [kNumBarriers]
    static constexpr uint32_t kOffMisc = kOffBar + kNumBarriers * 8;   // u32: tmem base, abort, rescale flag
    static constexpr uint32_t kBytes = kOffMisc + 16;
    // tensor memory columns
    static constexpr uint32_t kColO = 0;                     // 4 blocks x N columns
    // S^T is accumulated in kAcc independent partial sums (summed by the softmax warps): a
    // chain of 36 small MMAs into ONE accumulator runs at the MMA latency, not its rate.
    // 64-head groups compute S = Q K^T with the heads on the MMA's M (a softmax row lives in
    // one thread: no shuffles, no exchange); narrower groups compute S^T with the tokens on M
    // so that a 16- or 32-head slice is not padded to 64 rows.
    static constexpr bool kHeadsOnM = N == 64;
    static constexpr int kAcc = 4;                           // = number of issuers that take part in QK^T
    // two S buffers let QK^T run a tile ahead of the softmax; the 64-head kernel has tensor
    // memory for one only (O^T 256 columns + 4 partials x 64)
    static constexpr int kSBufs = N >= 64 ? 1 : 2;
    static constexpr uint32_t kColS = 4 * N;                 // kSBufs buffers x kAcc x N columns
    static_assert(kColS + kSBufs * kAcc * N <= 512, "tensor memory overflow");
    static_assert(kBytes <= 232448, "shared memory overflow");
    static_assert(kOffQ % 1024 == 0 && kOffP % 1024 == 0 && (N * 128) % 1024 == 0, "swizzle atoms need 1024-byte alignment");
};

// ---------------------------------------------------------------- the kernel
template <int N>
__global__ void __launch_bounds__(kThreads, 1)
decode_umma_kernel(const DecodeParams p, const __grid_constant__ CUtensorMap tmap_kv,
                   const __grid_constant__ CUtensorMap tmap_q) {
    using L = Layout<N>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int worker = blockIdx.x / p.num_groups;
    const int group = blockIdx.x % p.num_groups;
    const int head0 = p.head_begin + group * N;
    const int h = p.head_end - p.head_begin;

    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + L::kOffMisc);
    Ctx ctx{misc + 1, p.status};
    auto bar = [&](int id) -> uint32_t { return sbase + L::kOffBar + 8u * (uint32_t)id; };

    if ((sbase & 1023u) != 0) {      // swizzle atoms need a 1024-byte aligned window
        if (tid == 0 && atomicCAS(p.status, 0, (int)SPLASH_CUDA_ERROR) == 0) { p.status[1] = (int)blockIdx.x; p.status[2] = -100; }
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(kBarKvFull + s), 1); mbar_init(bar(kBarKvEmpty + s), kMmaWarps); }
        mbar_init(bar(kBarQFull), 1); mbar_init(bar(kBarQEmpty), L::kAcc);
        for (int b = 0; b < L::kSBufs; ++b) { mbar_init(bar(kBarSFull + b), L::kAcc); mbar_init(bar(kBarSEmpty + b), kNumSoftmaxWarps); }
        mbar_init(bar(kBarPFull), kNumSoftmaxWarps);
        mbar_init(bar(kBarOFull), kMmaWarps); mbar_init(bar(kBarOEmpty), kNumSoftmaxWarps);
        misc[1] = 0; misc[2] = 0; misc[3] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + L::kOffMisc), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = misc[0];
    grid_dependency_wait();       // the plan kernel's output is read from here on
    const long long t_start = clock64();

    SegmentIter it;
    it.init(p, worker);
    Segment seg;
    long long *const trace = blockIdx.x == 0 ? p.trace : nullptr;
    auto mark = [&](uint32_t tile, int ev) {
        if (trace != nullptr && tile < 64) trace[tile * 8 + ev] = clock64();
    };

    if (warp == 0) {
        // ===================================================== TMA producer
        uint32_t kv_it = 0, seg_it = 0;
        bool ok = true;
        while (ok && it.next(p, seg)) {
            if (lane == 0) {
                ok = mbar_wait(ctx, bar(kBarQEmpty), (seg_it & 1) ^ 1, kBarQEmpty);
                if (ok) {
                    mbar_expect_tx(bar(kBarQFull), L::kQBytes);
                    tma_load_4d(sbase + L::kOffQ, &tmap_q, bar(kBarQFull), 0, head0, 0, seg.request);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            const int first_page = seg.lo / kPage;
            const int32_t *table = p.block_table + (int64_t)seg.request * p.table_stride;
            int entry = 0;
            for (int tile = seg.tile_begin; ok && tile < seg.tile_end; ++tile) {
                const int rel = tile - seg.tile_begin;
                if ((rel & 31) == 0) {
                    int idx = tile + lane;
                    entry = idx < seg.tile_end ? table[first_page + idx] : 0;
                }
                const int page = __shfl_sync(0xffffffffu, entry, rel & 31);
                // the next page (when its table entry is among the 32 this warp holds): pulled into L2 now, so
                // that its TMA load, which can only start when a stage comes free, finds it there
                const int page_ahead = __shfl_sync(0xffffffffu, entry, (rel + kPrefetchTiles) & 31);
                const bool ahead_ok = (rel & 31) + kPrefetchTiles < 32 && tile + kPrefetchTiles < seg.tile_end;
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + tile) * kPage);
                const uint32_t stage = kv_it % kStages, ph = (kv_it / kStages) & 1;
                if (lane == 0) {
                    ok = mbar_wait(ctx, bar(kBarKvEmpty + stage), ph ^ 1, kBarKvEmpty + stage);
                    mark(kv_it, 0);
                    if (ok && !g.both) {
                        mbar_expect_tx(bar(kBarKvFull + stage), kStageBytes);
                        const uint32_t dst = sbase + L::kOffKv + stage * kStageBytes;
                        // one box = the whole page: (64 elements, 64 tokens, 9 chunks) -> [chunk][token][128 B]
                        tma_load_4d(dst, &tmap_kv, bar(kBarKvFull + stage), 0, g.tok0, 0, page);
                        if (ahead_ok && page_ahead >= 0 && page_ahead < p.num_pool_pages)
                            bulk_prefetch_l2(static_cast<const uint8_t *>(p.kv_pool) + (size_t)page_ahead * (kPage * kDQK * 2), kStageBytes);
                        mark(kv_it, 1);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (ok && g.both) {
                    // a range cut at both ends inside this page: the warp writes the box itself, zeros outside the range
                    const uint8_t *src = page >= 0 && page < p.num_pool_pages
                        ? static_cast<const uint8_t *>(p.kv_pool) + (size_t)page * (kPage * kDQK * 2) : nullptr;
                    fill_rows_by_hand<128>(smem + L::kOffKv + stage * kStageBytes, kSlabBytes, kPage, src, g.tok0, g.a, g.b, 0, 0, kChunks, lane);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarKvFull + stage));
                }
                ++kv_it;
            }
            ++seg_it;
        }
    } else if (warp <= kMmaWarps) {
        // ===================================================== MMA issuers
        if (lane == 0) {
            const int mw = warp - 1;                 // issuer index: S^T accumulator mw, dv block mw
            const bool does_qk = mw < L::kAcc;
            constexpr uint32_t kIdescQK = L::kHeadsOnM ? make_idesc(64, 64, 0, 0) : make_idesc(64, N, 0, 0);
            // P^T is K-major (swizzled) when the softmax has the heads on M, MN-major (plain) when it has the tokens on M
            constexpr uint32_t kIdescPV = make_idesc(128, N, 1, L::kHeadsOnM ? 0 : 1);
            uint32_t kv_it = 0, s_it = 0, p_it = 0, seg_it = 0;
            bool ok = true;
            // This issuer's share of S^T for the tile with global index kv: the K = 16 steps
            // idx = mw, mw + kAcc, ... of the 36, into partial accumulator mw.
            auto issue_qk = [&](uint32_t kv, uint32_t sidx) {
                const uint32_t stage = kv % kStages, b = sidx % L::kSBufs;
                if (mw == 0) mark(kv, 2);
                tcgen05_fence_after();
                const uint32_t a0 = sbase + L::kOffKv + stage * kStageBytes;
                const uint32_t b0 = sbase + L::kOffQ;
                const uint32_t d = tmem_base + L::kColS + (b * L::kAcc + mw) * N;
#pragma unroll
                for (int t = 0; t < 36 / L::kAcc; ++t) {
                    const int idx = t * L::kAcc + mw, c = idx >> 2, k = idx & 3;
                    uint64_t dk = make_desc(a0 + c * kSlabBytes + k * 32, 16, 1024);      // K tile rows = tokens
                    uint64_t dq = make_desc(b0 + c * (N * 128) + k * 32, 16, 1024);       // Q rows = heads
                    if constexpr (L::kHeadsOnM) umma_bf16(d, dq, dk, kIdescQK, t != 0);   // S  [heads x tokens]
                    else umma_bf16(d, dk, dq, kIdescQK, t != 0);                          // S^T [tokens x heads]
                }
                umma_commit(bar(kBarSFull + b));
                if (mw == 0) mark(kv, 3);
            };
            // O^T block mw += V^T block mw (128 dv x 64 tokens) * P^T, four K = 16 steps.
            auto issue_pv = [&](uint32_t stage, bool first_tile) {
                tcgen05_fence_after();
                const uint32_t v0 = sbase + L::kOffKv + stage * kStageBytes + (2 * mw) * kSlabBytes;
                const uint32_t p0 = sbase + L::kOffP;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // A: two 64-element chunks (LBO apart) x 16 tokens (SBO per 8 tokens), MN-major
                    uint64_t da = make_desc(v0 + k * 2048, kSlabBytes, 1024);
                    // B: 16 tokens x N heads.  K-major: 32 B into the swizzled rows; MN-major: two groups of eight tokens
                    // (128 B apart) x groups of eight heads (1,024 B apart)
                    uint64_t db = L::kHeadsOnM ? make_desc(p0 + k * 32, 16, 1024) : make_desc_mn_plain(p0 + k * 256, 128, 1024);
                    umma_bf16(tmem_base + L::kColO + mw * N, da, db, kIdescPV, (!first_tile) || k != 0);
                }
            };
            while (ok && it.next(p, seg)) {
                const int ntiles = seg.tile_end - seg.tile_begin;
                if (does_qk) {
                    ok = mbar_wait(ctx, bar(kBarQFull), seg_it & 1, kBarQFull);
                    if (!ok) break;
                }
                // Issue whatever is ready: P.V of tile pv_i (frees a stage) or QK^T of tile qk_i
                // (at most one tile ahead of the softmax: two S buffers).
                int qk_i = does_qk ? 0 : ntiles, pv_i = 0;
                unsigned long long idle_since = 0;
                uint32_t idle_polls = 0;          // the wall clock is read once per 256 idle polls: reading it costs hundreds of cycles
                while (pv_i < ntiles) {
                    bool progressed = false;
                    if ((qk_i > pv_i) && mbar_test_wait(bar(kBarPFull), (p_it + pv_i) & 1)) {
                        if (pv_i == 0 && !mbar_wait(ctx, bar(kBarOEmpty), (seg_it & 1) ^ 1, kBarOEmpty)) { ok = false; break; }
                        if (mw == 0) mark(kv_it + pv_i, 6);
                        const uint32_t stage = (kv_it + pv_i) % kStages;
                        issue_pv(stage, pv_i == 0);
                        umma_commit(bar(kBarKvEmpty + stage));   // P.V done: stage free, P buffer free, O^T updated
                        if (pv_i + 1 == ntiles) umma_commit(bar(kBarOFull));
                        if (mw == 0) mark(kv_it + pv_i, 7);
                        ++pv_i;
                        progressed = true;
                    }
                    if (does_qk && qk_i < ntiles && qk_i < pv_i + 2) {
                        const uint32_t kv = kv_it + qk_i, sidx = s_it + qk_i;
                        if (mbar_test_wait(bar(kBarKvFull + kv % kStages), (kv / kStages) & 1) &&
                            mbar_test_wait(bar(kBarSEmpty + sidx % L::kSBufs), ((sidx / L::kSBufs) & 1) ^ 1)) {
                            issue_qk(kv, sidx);
                            ++qk_i;
                            if (qk_i == ntiles) umma_commit(bar(kBarQEmpty));
                            progressed = true;
                        }
                    }
                    if (progressed) { idle_since = 0; idle_polls = 0; continue; }
                    if ((++idle_polls & 255u) != 0u) continue;
                    if (*ctx.abort_flag) { ok = false; break; }
                    const unsigned long long now = global_timer_ns();
                    if (idle_since == 0) idle_since = now;
                    else if (now - idle_since > kWaitLimitNs) {
                        *ctx.abort_flag = 1;
                        if (atomicCAS(ctx.status, 0, (int)SPLASH_DEVICE_TIMEOUT) == 0) {
                            ctx.status[1] = (int)blockIdx.x; ctx.status[2] = 100 + (qk_i > pv_i ? kBarPFull : kBarKvFull);
                            ctx.status[3] = pv_i;
                        }
                        ok = false; break;
                    }
                }
                kv_it += ntiles; s_it += ntiles; p_it += ntiles;
                ++seg_it;
            }
        }
    } else {
        // ===================================================== softmax + epilogue warps
        const int q4 = warp & 3;                       // TMEM lane quadrant of this warp
        const int sw = warp - 1 - kMmaWarps;           // softmax warp 0..3
        const int st = sw * 32 + lane;                 // 0..127
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        float *red = reinterpret_cast<float *>(smem + L::kOffRed);
        float *m_s = reinterpret_cast<float *>(smem + L::kOffM);
        float *alpha_s = reinterpret_cast<float *>(smem + L::kOffAlpha);
        float *l_s = reinterpret_cast<float *>(smem + L::kOffL);
        const float scale_log2 = p.softmax_scale * kLog2e;
        uint32_t s_it = 0, p_it = 0, seg_it = 0;
        // A failed (timed-out) wait only clears `ok`: the role keeps walking its tiles so that every thread still
        // meets the named barriers -- once the CTA aborts, waits return at once.
        bool ok = true;
        while (it.next(p, seg)) {
            if (st < N) m_s[st] = -INFINITY;
            // heads-on-M: this thread's two heads (reference maxima; partial row sums over its tokens)
            const int hA = 16 * q4 + (lane >> 2);
            float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
            // tokens on M: sums over this thread's two tokens, heads 8k + 2 tq + e at [2k + e]
            constexpr int kR = L::kHeadsOnM ? 1 : N / 8;
            float l_tk[2 * kR];
#pragma unroll
            for (int k = 0; k < 2 * kR; ++k) l_tk[k] = 0.f;
            softmax_bar_sync();
            const int first_page = seg.lo / kPage;
            const int ntiles = seg.tile_end - seg.tile_begin;
            for (int i = 0; i < ntiles; ++i) {
                const TileGeom g = tile_geom(seg.lo, seg.hi, (first_page + seg.tile_begin + i) * kPage);
                const uint32_t b = s_it % L::kSBufs;
                ok &= mbar_wait(ctx, bar(kBarSFull + b), (s_it / L::kSBufs) & 1, kBarSFull + b);
                if (st == 0) mark(s_it, 4);
                tcgen05_fence_after();
                if constexpr (L::kHeadsOnM) {
                // ---- heads on M.  S [64 heads x 64 tokens] sits in 16 lanes per TMEM quadrant; the
                // fragment load spreads those over all 32 threads: this thread holds heads
                // hA = 16 q4 + lane/4 and hB = hA + 8, tokens 8k + 2(lane%4) + {0,1}, k = 0..7.
                float s[32];
                {
                    const uint32_t sb = tmem_base + lane_addr + L::kColS + b * (L::kAcc * N);
                    tmem_ld_16x256b_x8(sb, s);
#pragma unroll
                    for (int a = 1; a < L::kAcc; ++a) {
                        float part[32];
                        tmem_ld_16x256b_x8(sb + a * N, part);
                        tmem_wait_ld();
#pragma unroll
                        for (int n = 0; n < 32; ++n) s[n] += part[n];
                    }
                }
                tmem_wait_ld();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSEmpty + b));
                const int tq = lane & 3;
                float mtA = -INFINITY, mtB = -INFINITY;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int t = 8 * k + 2 * tq + e;
                        const bool v = t >= g.r_lo && t < g.r_hi;
                        s[4 * k + e] = v ? s[4 * k + e] * scale_log2 : -INFINITY;
                        s[4 * k + 2 + e] = v ? s[4 * k + 2 + e] * scale_log2 : -INFINITY;
                        mtA = fmaxf(mtA, s[4 * k + e]);
                        mtB = fmaxf(mtB, s[4 * k + 2 + e]);
                    }
                }
                mtA = fmaxf(mtA, __shfl_xor_sync(0xffffffffu, mtA, 1)); mtB = fmaxf(mtB, __shfl_xor_sync(0xffffffffu, mtB, 1));
                mtA = fmaxf(mtA, __shfl_xor_sync(0xffffffffu, mtA, 2)); mtB = fmaxf(mtB, __shfl_xor_sync(0xffffffffu, mtB, 2));
                // the four threads of a head take the same decision from the same numbers
                bool grew = false;
                float alA = 1.f, alB = 1.f;
                if (mtA > mA + kRescaleThreshold) { alA = (mA == -INFINITY) ? 0.f : fast_exp2(mA - mtA); mA = mtA; lA *= alA; grew = true; }
                if (mtB > mB + kRescaleThreshold) { alB = (mB == -INFINITY) ? 0.f : fast_exp2(mB - mtB); mB = mtB; lB *= alB; grew = true; }
                if (tq == 0) { alpha_s[hA] = alA; alpha_s[hA + 8] = alB; }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        s[4 * k + e] = fast_exp2(s[4 * k + e] - mA); lA += s[4 * k + e];
                        s[4 * k + 2 + e] = fast_exp2(s[4 * k + 2 + e] - mB); lB += s[4 * k + 2 + e];
                    }
                }
                const bool rescale = softmax_bar_or(grew);
                // P.V of the previous tile must be done with the P buffer and with O^T
                if (s_it > 0) {
                    const uint32_t prev = s_it - 1;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                }
                tcgen05_fence_after();
                if (rescale && i > 0) {
#pragma unroll 1
                    for (int c = 0; c < 4 * N / 16; ++c) {
                        float o[16];
                        const uint32_t addr = tmem_base + lane_addr + L::kColO + c * 16;
                        tmem_ld16(addr, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) o[k] *= alpha_s[(c * 16 + k) % N];
                        tmem_st16(addr, o);
                    }
                    tmem_wait_st();
                }
                {
                    // P as the K-major, 128-byte-swizzled B operand of P.V: row = head, chunk k = tokens 8k..8k+7
                    uint8_t *pA = smem + L::kOffP + hA * 128 + tq * 4;
                    uint8_t *pB = pA + 8 * 128;                       // head hA + 8: same (h & 7)
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t off = (uint32_t)(k ^ (hA & 7)) << 4;
                        *reinterpret_cast<uint32_t *>(pA + off) = pack_bf16x2(s[4 * k + 0], s[4 * k + 1]);
                        *reinterpret_cast<uint32_t *>(pB + off) = pack_bf16x2(s[4 * k + 2], s[4 * k + 3]);
                    }
                }
                } else {
                // ---- tokens on M.  S^T [64 tokens x N heads] sits in 16 lanes per TMEM quadrant; the fragment load
                // spreads them over all 32 threads: this thread holds tokens rA = 16 q4 + lane/4 and rB = rA + 8 and,
                // of each group of eight heads, heads 2 tq and 2 tq + 1.
                const int rA = 16 * q4 + (lane >> 2), rB = rA + 8, tq = lane & 3;
                const bool vA = rA >= g.r_lo && rA < g.r_hi, vB = rB >= g.r_lo && rB < g.r_hi;
                float s[4 * kR];
                {
                    float t0[4 * kR], t1[4 * kR], t2[4 * kR];
                    const uint32_t sb = tmem_base + lane_addr + L::kColS + b * (L::kAcc * N);
                    tmem_ld_frag<N>(sb, s);
                    tmem_ld_frag<N>(sb + N, t0);
                    tmem_ld_frag<N>(sb + 2 * N, t1);
                    tmem_ld_frag<N>(sb + 3 * N, t2);
                    tmem_wait_ld();
#pragma unroll
                    for (int n = 0; n < 4 * kR; ++n) s[n] = (s[n] + t0[n]) + (t1[n] + t2[n]);
                    static_assert(L::kAcc == 4, "four partial accumulators are summed here");
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSEmpty + b));
                // One reference maximum per head, moved only when a logit exceeds it by more than the threshold: whether
                // any does is one barrier-wide OR; the common tile needs no reduction over tokens at all.
                bool exceeds = false;
#pragma unroll
                for (int k = 0; k < kR; ++k) {
                    const float2 m2 = *reinterpret_cast<const float2 *>(&m_s[8 * k + 2 * tq]);
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float lim = (e ? m2.y : m2.x) + kRescaleThreshold;
                        const float yA = vA ? s[4 * k + e] * scale_log2 : -INFINITY;
                        const float yB = vB ? s[4 * k + 2 + e] * scale_log2 : -INFINITY;
                        s[4 * k + e] = yA; s[4 * k + 2 + e] = yB;
                        exceeds |= (yA > lim) | (yB > lim);
                    }
                }
                const bool rescale = softmax_bar_or(exceeds);
                if (rescale) {
                    // the rare path (the first tile of a request, then a handful of times): per-head maxima over the
                    // tile's tokens, new references for the heads that grew, their rescale factors
#pragma unroll
                    for (int k = 0; k < kR; ++k) {
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            float mx = fmaxf(s[4 * k + e], s[4 * k + 2 + e]);
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                            if (lane < 4) red[(8 * k + 2 * tq + e) * 4 + sw] = mx;
                        }
                    }
                    softmax_bar_sync();
                    if (st < N) {
                        float4 r4 = *reinterpret_cast<const float4 *>(&red[st * 4]);
                        float mt = fmaxf(fmaxf(r4.x, r4.y), fmaxf(r4.z, r4.w));
                        float m_old = m_s[st];
                        float al = 1.f;
                        if (mt > m_old + kRescaleThreshold) {        // also taken when m_old = -inf
                            al = (m_old == -INFINITY) ? 0.f : fast_exp2(m_old - mt);
                            m_s[st] = mt;
                        }
                        alpha_s[st] = al;
                    }
                    softmax_bar_sync();
#pragma unroll
                    for (int k = 0; k < kR; ++k) {
                        const float2 a2 = *reinterpret_cast<const float2 *>(&alpha_s[8 * k + 2 * tq]);
                        l_tk[2 * k] *= a2.x; l_tk[2 * k + 1] *= a2.y;
                    }
                }
                uint32_t pA[kR], pB[kR];          // two adjacent heads per word
#pragma unroll
                for (int k = 0; k < kR; ++k) {
                    const float2 m2 = *reinterpret_cast<const float2 *>(&m_s[8 * k + 2 * tq]);
                    const float a0 = fast_exp2(s[4 * k + 0] - m2.x), a1 = fast_exp2(s[4 * k + 1] - m2.y);
                    const float b0 = fast_exp2(s[4 * k + 2] - m2.x), b1 = fast_exp2(s[4 * k + 3] - m2.y);
                    l_tk[2 * k] += a0 + b0; l_tk[2 * k + 1] += a1 + b1;
                    pA[k] = pack_bf16x2(a0, a1); pB[k] = pack_bf16x2(b0, b1);
                }
                // P.V of the previous tile must be done with the P buffer and with O^T
                if (s_it > 0) {
                    const uint32_t prev = s_it - 1;
                    ok &= mbar_wait(ctx, bar(kBarKvEmpty + prev % kStages), (prev / kStages) & 1, kBarKvEmpty + prev % kStages);
                }
                tcgen05_fence_after();
                if (rescale && i > 0) {
#pragma unroll 1
                    for (int c = 0; c < 4 * N / 16; ++c) {
                        float o[16];
                        const uint32_t addr = tmem_base + lane_addr + L::kColO + c * 16;
                        tmem_ld16(addr, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) o[k] *= alpha_s[(c * 16 + k) % N];
                        tmem_st16(addr, o);
                    }
                    tmem_wait_st();
                }
                {
                    // P^T as the MN-major B operand: eight heads of a token are 16 adjacent bytes, groups of eight heads
                    // 1,024 B apart
                    uint8_t *pa = smem + L::kOffP + rA * 16 + tq * 4;
#pragma unroll
                    for (int k = 0; k < kR; ++k) {
                        *reinterpret_cast<uint32_t *>(pa + k * 1024) = pA[k];
                        *reinterpret_cast<uint32_t *>(pa + k * 1024 + 8 * 16) = pB[k];
                    }
                }
                }
                fence_proxy_async();
                tcgen05_fence_before();
                if (st == 0) mark(s_it, 5);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull));
                ++s_it; ++p_it;
            }
            if constexpr (L::kHeadsOnM) {
                lA += __shfl_xor_sync(0xffffffffu, lA, 1); lB += __shfl_xor_sync(0xffffffffu, lB, 1);
                lA += __shfl_xor_sync(0xffffffffu, lA, 2); lB += __shfl_xor_sync(0xffffffffu, lB, 2);
                if ((lane & 3) == 0) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int hh = hA + 8 * e;
                        const float l = e ? lB : lA, m = e ? mB : mA;
                        l_s[hh] = 1.f / l;
                        const int gh = head0 + hh;
                        if (gh < p.head_end) {
                            float lse = (m + log2f(l)) * kLn2;
                            if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                            else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                        }
                    }
                }
            } else {
                // ---- row sums: over the 16 tokens of a warp (the eight threads with this tq), then over the four warps
                const int tq = lane & 3;
#pragma unroll
                for (int n = 0; n < 2 * kR; ++n) {
                    float v = l_tk[n];
                    v += __shfl_xor_sync(0xffffffffu, v, 4);
                    v += __shfl_xor_sync(0xffffffffu, v, 8);
                    v += __shfl_xor_sync(0xffffffffu, v, 16);
                    if (lane < 4) red[(8 * (n >> 1) + 2 * tq + (n & 1)) * 4 + sw] = v;
                }
                softmax_bar_sync();
                if (st < N) {
                    float4 r4 = *reinterpret_cast<const float4 *>(&red[st * 4]);
                    float l = (r4.x + r4.y) + (r4.z + r4.w);
                    l_s[st] = 1.f / l;
                    const int gh = head0 + st;
                    if (gh < p.head_end) {
                        float lse = (m_s[st] + log2f(l)) * kLn2;
                        if (seg.slot < 0) p.lse[(int64_t)seg.request * p.lse_stride_request + gh] = lse;
                        else p.partial_lse[(int64_t)seg.slot * h + (gh - p.head_begin)] = lse;
                    }
                }
            }
            softmax_bar_sync();
            // ---- epilogue: O^T block j holds dv = 128 j + TMEM lane, one column per head
            ok &= mbar_wait(ctx, bar(kBarOFull), seg_it & 1, kBarOFull);
            tcgen05_fence_after();
            float *obase;
            int64_t ostride;
            if (seg.slot < 0) {
                obase = p.out + (int64_t)seg.request * p.out_stride_request + (int64_t)head0 * p.out_stride_head;
                ostride = p.out_stride_head;
            } else {
                obase = p.partial_out + ((int64_t)seg.slot * h + (head0 - p.head_begin)) * kDV;
                ostride = kDV;
            }
            const int nvalid = min(N, p.head_end - head0);
            bool staged = false;
            if constexpr (N < 64) {
                if (((reinterpret_cast<uintptr_t>(obase) | (uintptr_t)(ostride * 4)) & 15) == 0) {
                    // Through shared memory and the bulk-copy engine: plain stores of this tile (one 128-byte line per
                    // warp instruction, 64 of them per thread) take ~6,000 cycles while the cache streams, 2.5 times this.
                    staged = true;
                    float *stg = reinterpret_cast<float *>(smem + L::kOffOut);
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            const int j = 2 * half + jj;
#pragma unroll
                            for (int c = 0; c < N / 16; ++c) {
                                float o[16];
                                tmem_ld16(tmem_base + lane_addr + L::kColO + j * N + c * 16, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int k = 0; k < 16; ++k) {
                                    const int n = c * 16 + k;
                                    stg[n * 256 + jj * 128 + 32 * q4 + lane] = o[k] * l_s[n];
                                }
                            }
                        }
                        fence_proxy_async();
                        softmax_bar_sync();
                        if (st < nvalid) {
                            bulk_store(obase + (int64_t)st * ostride + half * 256, smem_u32(stg + st * 256), 1024);
                            bulk_commit_group();
                            bulk_wait_group_read();          // the row has left shared memory
                        }
                        softmax_bar_sync();
                    }
                }
            }
            if (!staged) {
#pragma unroll 1
                for (int j = 0; j < 4; ++j) {
                    const int dv = 128 * j + 32 * q4 + lane;
#pragma unroll
                    for (int c = 0; c < N / 16; ++c) {
                        float o[16];
                        tmem_ld16(tmem_base + lane_addr + L::kColO + j * N + c * 16, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const int n = c * 16 + k;
                            if (n < nvalid) obase[(int64_t)n * ostride + dv] = o[k] * l_s[n];
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarOEmpty));
            ++seg_it;
        }
    }

    fill_empty_requests(p, worker, head0, N, tid, kThreads);
    if (p.trace != nullptr && tid == 0) p.trace[512 + blockIdx.x] = clock64() - t_start;   // per-CTA cycles

    // ---- teardown
    if (*ctx.abort_flag) {
        // let bulk copies that were already issued land before the CTA's shared memory goes away
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { __nanosleep(1000); }
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 0) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---------------------------------------------------------------- host side
template <int N>
cudaError_t launch_n(const DecodeParams &p, const CUtensorMap &mkv, const CUtensorMap &mq, cudaStream_t stream) {
    const int smem = (int)Layout<N>::kBytes;
    static DeviceOnce once;
    cudaError_t e = once.run([&] { return cudaFuncSetAttribute(decode_umma_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem); });
    if (e != cudaSuccess) return e;
    e = launch_dependent(decode_umma_kernel<N>, dim3((unsigned)(p.num_workers * p.num_groups)), dim3(kThreads), (size_t)smem,
                         stream, p, mkv, mq);
    count_launch();
    return e;
}

}  // namespace

void umma_tiling(int kv_dtype, int h, int sm_count, int *heads_per_group, int *num_groups, int *num_workers) {
    (void)kv_dtype;       // both cache formats have 16-, 32- and 64-head kernels
    const int n = h <= 16 ? 16 : (h <= 32 ? 32 : 64);
    *heads_per_group = n;
    *num_groups = (h + n - 1) / n;
    const int w = sm_count / *num_groups;
    *num_workers = w > 0 ? w : 1;
}

cudaError_t launch_decode_umma(const DecodeParams &p, const splash_mla_shape &shape, cudaStream_t stream) {
    if (shape.kv_dtype != SPLASH_KV_BF16) {
        // slices of more than 64 heads run on CTA pairs (cta_group::2) unless the caller opts out
        if (p.num_groups == 2 && !(shape.flags & SPLASH_FLAG_NO_PAIR)) {
            const cudaError_t e = launch_decode_umma_fp8_pair(p, stream);
            if (e != cudaErrorNotSupported) return e;      // output rows not 16-byte aligned: no TMA stores
        }
        return p.heads_per_group < 64 ? launch_decode_umma_fp8_narrow(p, stream) : launch_decode_umma_fp8(p, stream);
    }
    if (p.num_groups == 2 && p.heads_per_group == 64 && !(shape.flags & SPLASH_FLAG_NO_PAIR)) return launch_decode_umma_pair(p, stream);
    alignas(64) CUtensorMap mkv, mq;
    const int n = p.heads_per_group;
    if (!make_map_4d(&mkv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, p.kv_pool, kPage,
                     (uint64_t)(p.num_pool_pages > 0 ? p.num_pool_pages : 1), (uint64_t)kDQK * 2, 128,
                     (uint64_t)kPage * kDQK * 2, 64))
        return cudaErrorInvalidValue;
    if (!make_map_4d(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, p.q, (uint64_t)p.H,
                     (uint64_t)p.B, (uint64_t)p.q_stride_head * 2, 128,
                     (uint64_t)(p.B > 1 ? p.q_stride_request : p.q_stride_head * p.H) * 2, (uint32_t)n))
        return cudaErrorInvalidValue;
    switch (n) {
        case 16: return launch_n<16>(p, mkv, mq, stream);
        case 32: return launch_n<32>(p, mkv, mq, stream);
        case 64: return launch_n<64>(p, mkv, mq, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace splash
