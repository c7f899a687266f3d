// Plain SIMT decode kernel: fp32 CUDA-core arithmetic, no tensor cores, no TMA.
// It is the diagnostic path of the library (shape flag SPLASH_FLAG_SIMT): it walks
// the same work plan, writes the same partial slots and feeds the same combine
// kernel as the tcgen05 kernel, so paging, range masking, the split-KV plan and the
// epilogue can be checked independently of the tensor-core pipeline.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "splash_common.cuh"

namespace splash {

namespace {

constexpr int kSimtHeads = 8;          // heads per CTA
constexpr int kSimtThreads = 256;
constexpr int kRowStride = kDQK + 8;   // padded 16-bit elements per staged row

struct SimtSmem {
    float q[kSimtHeads][kDQK];
    float s[kSimtHeads][kPage];
    float tok_scale[kPage];
    float alpha[kSimtHeads];
    float m[kSimtHeads];
    float l[kSimtHeads];
    uint16_t rows[kPage][kRowStride];
};

template <int KV_DTYPE>
__device__ __forceinline__ float elem_to_float(uint16_t v) {
    if (KV_DTYPE == 0) return __uint_as_float(((uint32_t)v) << 16);
    return __half2float(__ushort_as_half(v));
}

template <int KV_DTYPE>
__global__ void __launch_bounds__(kSimtThreads)
decode_simt_kernel(const DecodeParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SimtSmem &sm = *reinterpret_cast<SimtSmem *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int worker = blockIdx.x / p.num_groups;
    const int group = blockIdx.x % p.num_groups;
    const int head0 = p.head_begin + group * kSimtHeads;       // first global head of this CTA
    const int h = p.head_end - p.head_begin;

    grid_dependency_wait();       // the plan kernel's output is read from here on
    SegmentIter it;
    it.init(p, worker);
    Segment seg;
    while (it.next(p, seg)) {
        // ---- query rows of this CTA's heads, as fp32 -------------------------------
        const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(p.q) + (int64_t)seg.request * p.q_stride_request;
        for (int idx = tid; idx < kSimtHeads * kDQK; idx += kSimtThreads) {
            int hd = idx / kDQK, d = idx % kDQK;
            int g = head0 + hd;
            sm.q[hd][d] = g < p.head_end ? __bfloat162float(qg[(int64_t)g * p.q_stride_head + d]) : 0.f;
        }
        if (tid < kSimtHeads) { sm.m[tid] = -INFINITY; sm.l[tid] = 0.f; }
        float acc[kSimtHeads][2];
#pragma unroll
        for (int hd = 0; hd < kSimtHeads; ++hd) acc[hd][0] = acc[hd][1] = 0.f;
        __syncthreads();

        const int first_page = seg.lo / kPage;
        // several query rows per request: (virtual) head g is row g mod R and sees the tokens below its causal end
        const int s_len = p.q_rows > 1 ? p.seq_lens[seg.request] : 0;
        auto causal_end = [&](int hd) { return p.q_rows > 1 ? s_len - (p.q_rows - 1 - (head0 + hd) % p.q_rows) : 0x3fffffff; };
        for (int tile = seg.tile_begin; tile < seg.tile_end; ++tile) {
            const int page_idx = first_page + tile;
            const int t0 = page_idx * kPage;
            const int a = max(seg.lo, t0) - t0;
            const int b = min(seg.hi, t0 + kPage) - t0;
            int64_t page = p.block_table[(int64_t)seg.request * p.table_stride + page_idx];
            // an id outside the pool is never dereferenced: the page reads as zeros, like a box outside a tensor map
            const bool in_pool = page >= 0 && page < p.num_pool_pages;
            if (!in_pool) page = 0;

            // ---- stage rows [a, b) of the page ------------------------------------
            if (KV_DTYPE == 0) {
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const uint16_t *>(p.kv_pool) + page * (int64_t)(kPage * kDQK));
                constexpr int kVecPerRow = kDQK / 8;   // 72
                for (int idx = a * kVecPerRow + tid; idx < b * kVecPerRow; idx += kSimtThreads) {
                    int r = idx / kVecPerRow, c = idx % kVecPerRow;
                    *reinterpret_cast<uint4 *>(&sm.rows[r][c * 8]) = in_pool ? src[idx] : make_uint4(0u, 0u, 0u, 0u);
                }
            } else {
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    static_cast<const uint8_t *>(p.kv_pool) + page * (int64_t)(kPage * kDQK));
                constexpr int kVecPerRow = kDQK / 16;  // 36
                for (int idx = a * kVecPerRow + tid; idx < b * kVecPerRow; idx += kSimtThreads) {
                    int r = idx / kVecPerRow, c = idx % kVecPerRow;
                    uint4 v = in_pool ? src[idx] : make_uint4(0u, 0u, 0u, 0u);
                    const __nv_fp8x2_storage_t *pairs = reinterpret_cast<const __nv_fp8x2_storage_t *>(&v);
                    uint32_t o[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        __half2_raw h2 = __nv_cvt_fp8x2_to_halfraw2(pairs[k], __NV_E4M3);
                        o[k] = (uint32_t)h2.x | ((uint32_t)h2.y << 16);
                    }
                    uint4 *dst = reinterpret_cast<uint4 *>(&sm.rows[r][c * 16]);
                    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                }
                if (tid >= a && tid < b) sm.tok_scale[tid] = in_pool ? p.kv_scales[page * kPage + tid] : 1.0f;
            }
            __syncthreads();

            // ---- logits ---------------------------------------------------------------
            for (int idx = tid; idx < kSimtHeads * kPage; idx += kSimtThreads) {
                int hd = idx / kPage, t = idx % kPage;
                float sv = -INFINITY;
                if (t >= a && t < min(b, causal_end(hd) - t0)) {
                    float dot = 0.f;
                    const uint4 *row = reinterpret_cast<const uint4 *>(&sm.rows[t][0]);
                    const float *qh = sm.q[hd];
#pragma unroll 4
                    for (int c = 0; c < kDQK / 8; ++c) {
                        uint4 v = row[c];
                        const uint16_t *e = reinterpret_cast<const uint16_t *>(&v);
#pragma unroll
                        for (int k = 0; k < 8; ++k) dot = fmaf(qh[c * 8 + k], elem_to_float<KV_DTYPE>(e[k]), dot);
                    }
                    sv = dot * p.softmax_scale;
                    if (KV_DTYPE == 1) sv *= sm.tok_scale[t];
                }
                sm.s[hd][t] = sv;
            }
            __syncthreads();

            // ---- online softmax: warp `wid` owns head `wid` --------------------------
            {
                const int hd = wid;
                const int bh = min(b, causal_end(hd) - t0);      // this head's end within the tile
                float s0 = sm.s[hd][lane], s1 = sm.s[hd][lane + 32];
                float mx = fmaxf(s0, s1);
                for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                float m_old = sm.m[hd];
                float m_new = fmaxf(m_old, mx);           // -inf only while the head has seen no token
                float p0 = (lane >= a && lane < bh) ? __expf(s0 - m_new) : 0.f;
                float p1 = (lane + 32 >= a && lane + 32 < bh) ? __expf(s1 - m_new) : 0.f;
                float sum = p0 + p1;
                for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                float al = (m_old == -INFINITY) ? 0.f : __expf(m_old - m_new);
                if (KV_DTYPE == 1) { p0 *= sm.tok_scale[lane < b ? lane : 0]; p1 *= sm.tok_scale[lane + 32 < b ? lane + 32 : 0]; }
                if (!(lane >= a && lane < bh)) p0 = 0.f;
                if (!(lane + 32 >= a && lane + 32 < bh)) p1 = 0.f;
                sm.s[hd][lane] = p0; sm.s[hd][lane + 32] = p1;
                if (lane == 0) { sm.alpha[hd] = al; sm.m[hd] = m_new; sm.l[hd] = sm.l[hd] * al + sum; }
            }
            __syncthreads();

            // ---- O += P V: thread owns value columns 2*tid, 2*tid+1 --------------------
#pragma unroll
            for (int hd = 0; hd < kSimtHeads; ++hd) { float al = sm.alpha[hd]; acc[hd][0] *= al; acc[hd][1] *= al; }
            for (int t = a; t < b; ++t) {
                uint32_t v2 = *reinterpret_cast<const uint32_t *>(&sm.rows[t][2 * tid]);
                float v0 = elem_to_float<KV_DTYPE>((uint16_t)(v2 & 0xffffu));
                float v1 = elem_to_float<KV_DTYPE>((uint16_t)(v2 >> 16));
#pragma unroll
                for (int hd = 0; hd < kSimtHeads; ++hd) {
                    float pw = sm.s[hd][t];
                    acc[hd][0] = fmaf(pw, v0, acc[hd][0]);
                    acc[hd][1] = fmaf(pw, v1, acc[hd][1]);
                }
            }
            __syncthreads();
        }

        // ---- epilogue -------------------------------------------------------------------
#pragma unroll
        for (int hd = 0; hd < kSimtHeads; ++hd) {
            int g = head0 + hd;
            if (g >= p.head_end) continue;
            float l = sm.l[hd];
            float inv = l > 0.f ? 1.f / l : 0.f;          // no token at all: O = 0, LSE = -inf
            float2 o = make_float2(acc[hd][0] * inv, acc[hd][1] * inv);
            float L = l > 0.f ? sm.m[hd] + logf(l) : -INFINITY;
            if (seg.slot < 0) {
                float *dst = p.out + (int64_t)seg.request * p.out_stride_request + (int64_t)g * p.out_stride_head;
                *reinterpret_cast<float2 *>(dst + 2 * tid) = o;
                if (tid == 0) p.lse[(int64_t)seg.request * p.lse_stride_request + g] = L;
            } else {
                int64_t row = (int64_t)seg.slot * h + (g - p.head_begin);
                *reinterpret_cast<float2 *>(p.partial_out + row * kDV + 2 * tid) = o;
                if (tid == 0) p.partial_lse[row] = L;
            }
        }
        __syncthreads();
    }
    fill_empty_requests(p, worker, head0, kSimtHeads, tid, kSimtThreads);
}

}  // namespace

cudaError_t launch_decode_simt(const DecodeParams &p, int kv_dtype, cudaStream_t stream) {
    const size_t smem = sizeof(SimtSmem);
    dim3 grid((unsigned)(p.num_workers * p.num_groups));
    cudaError_t e;
    if (kv_dtype == 0) {
        e = cudaFuncSetAttribute(decode_simt_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        e = launch_dependent(decode_simt_kernel<0>, grid, dim3(kSimtThreads), smem, stream, p);
    } else {
        e = cudaFuncSetAttribute(decode_simt_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        e = launch_dependent(decode_simt_kernel<1>, grid, dim3(kSimtThreads), smem, stream, p);
    }
    count_launch();
    return e;
}

int simt_heads_per_group() { return kSimtHeads; }

}  // namespace splash
