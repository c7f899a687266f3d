// Log-sum-exp merges: the public CP merge (splash_lse_merge) and the reduction of
// the decode kernels' split-KV partial slots.  Both compute, per row,
//     L = ln sum_j exp(L_j),   O = sum_j exp(L_j - L) O_j,
// parts with L_j = -inf contributing nothing.  Pure fp32, HBM-bound.
#include <cuda_fp16.h>

#include <type_traits>

#include "splash_common.cuh"

namespace splash {

namespace {

constexpr int kMergeThreads = 128;

// One CTA per row; each thread owns float4 columns tid, tid + 128, ...
__global__ void __launch_bounds__(kMergeThreads)
lse_merge_kernel(int num_parts, int64_t rows, int d_v, const float *__restrict__ part_out,
                 const float *__restrict__ part_lse, float *__restrict__ out, float *__restrict__ lse) {
    const int64_t r = blockIdx.x;
    float m = -INFINITY;
    for (int j = 0; j < num_parts; ++j) m = fmaxf(m, part_lse[(int64_t)j * rows + r]);
    float4 *o4 = reinterpret_cast<float4 *>(out + r * d_v);
    const int nvec = d_v / 4;
    if (m == -INFINITY) {
        for (int c = threadIdx.x; c < nvec; c += kMergeThreads) o4[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (threadIdx.x == 0) lse[r] = -INFINITY;
        return;
    }
    float Z = 0.f;
    for (int j = 0; j < num_parts; ++j) {
        float Lj = part_lse[(int64_t)j * rows + r];
        if (Lj != -INFINITY) Z += expf(Lj - m);
    }
    const float L = m + logf(Z);
    for (int c = threadIdx.x; c < nvec; c += kMergeThreads) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < num_parts; ++j) {
            float Lj = part_lse[(int64_t)j * rows + r];
            if (Lj == -INFINITY) continue;
            float w = expf(Lj - L);
            float4 v = reinterpret_cast<const float4 *>(part_out + ((int64_t)j * rows + r) * d_v)[c];
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
        o4[c] = acc;
    }
    if (threadIdx.x == 0) lse[r] = L;
}

// Grid W*h: block = (entry of the plan's list of split requests, head k of the slice).  A
// request computed in one piece and an empty one were written by the decode kernel itself; a
// split request is merged from the slots of its workers in worker order.  The weights are
// computed once per block (thread j takes worker wf + j), then every thread streams its
// float4 column over the parts with several loads in flight.
constexpr int kMaxParts = 512;     // >= number of workers of any launch (one per SM at most)

// kF16: the partial outputs are f16 (rows of 512 halves) or fp32.  kLean: a variant for launches whose requests are cut
// into few pieces each (many requests per worker): at most four part loads in flight, few enough registers for sixteen
// resident blocks per SM instead of eight -- its blocks are short chains of round trips to DRAM, and what bounds
// the kernel is how many of them an SM holds at a time.
template <bool kF16, bool kLean>
__global__ void __launch_bounds__(kMergeThreads, kLean ? 16 : 8)
split_combine_kernel(const DecodeParams p, const int4 *__restrict__ split_rec) {
    __shared__ float w_s[kMaxParts];
    __shared__ float sc_s[kF16 ? kMaxParts : 1];      // f16 pieces: the power of two each row was divided by
    __shared__ int slot_s[kMaxParts];
    __shared__ float red_s[kMergeThreads / 32];
    const int h = p.head_end - p.head_begin;
    const int k = blockIdx.x % h, entry = blockIdx.x / h;
    const int g = p.head_begin + k;
    grid_dependency_wait();       // the decode kernel's partial slots (and the plan) are read from here on
    // Three rounds of loads, each independent within itself (the plan's arrays have long left L2 by now, so every
    // dependent load is a trip to DRAM): the list length and this entry's record; then the worker boundaries and the
    // LSE of every candidate slot; then the partial outputs.
    const int n_entries = p.status[8];
    const int4 rec = split_rec[entry];             // (request, first worker, last worker, first tile); unused past the list's end
    if (entry >= n_entries) return;
    const int i = rec.x, wf = rec.y, wl = rec.z;
    float4 *o4 = reinterpret_cast<float4 *>(p.out + (int64_t)i * p.out_stride_request + (int64_t)g * p.out_stride_head);
    float *lse = p.lse + (int64_t)i * p.lse_stride_request + g;
    const int c = threadIdx.x;             // 128 threads x float4 = 512 columns
    // workers between the first and the last may own no tiles at all (their start snapped to
    // the same tile as their successor's): they wrote no slot and get weight 0
    const int rs = rec.w;
    const int nparts = wl - wf + 1;
    float m = -INFINITY;
    for (int j = c; j < nparts; j += kMergeThreads) {
        const int w = wf + j;
        // slot 2 w + 1 can only be the first worker's (the request starts inside its run); both candidates' LSEs are
        // fetched beside the boundaries that decide between them (a slot nobody wrote holds stale bytes: not used)
        const int wb0 = p.worker_begin[w], wb1 = p.worker_begin[w + 1];
        const float L0 = p.partial_lse[(int64_t)(2 * w) * h + k];
        const float L1 = j == 0 ? p.partial_lse[(int64_t)(2 * w + 1) * h + k] : 0.f;
        float S0 = 1.f, S1 = 1.f;
        if constexpr (kF16) {
            S0 = p.partial_scale[(int64_t)(2 * w) * h + k];
            if (j == 0) S1 = p.partial_scale[(int64_t)(2 * w + 1) * h + k];
        }
        const bool live = wb1 > wb0;
        const int slot = 2 * w + (rs <= wb0 ? 0 : 1);
        const float L = live ? ((slot & 1) ? L1 : L0) : -INFINITY;
        if constexpr (kF16) sc_s[j] = (slot & 1) ? S1 : S0;
        slot_s[j] = slot;
        w_s[j] = L;
        m = fmaxf(m, L);
    }
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((c & 31) == 0) red_s[c >> 5] = m;
    __syncthreads();
    m = fmaxf(fmaxf(red_s[0], red_s[1]), fmaxf(red_s[2], red_s[3]));
    if (m == -INFINITY) {                  // no piece saw a token (a query row whose causal range is empty)
        o4[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c == 0) *lse = -INFINITY;
        return;
    }
    for (int j = c; j < nparts; j += kMergeThreads) w_s[j] = expf(w_s[j] - m);     // 0 for dead workers
    __syncthreads();
    float Z = 0.f;
    for (int j = 0; j < nparts; ++j) Z += w_s[j];          // same order in every thread: one value of Z
    const float L = m + logf(Z);
    const float inv_z = 1.f / Z;
    // this thread's four columns of a slot's row as they lie in memory (loads first, conversions with the arithmetic:
    // a conversion next to its load would make every load wait for the one before it)
    using Raw = typename std::conditional<kF16, uint2, float4>::type;
    auto load_part = [&](int slot) -> Raw {
        const int64_t row = (int64_t)slot * h + k;
        if constexpr (kF16) return reinterpret_cast<const uint2 *>(reinterpret_cast<const __half *>(p.partial_out) + row * kDV)[c];
        else return reinterpret_cast<const float4 *>(p.partial_out + row * kDV)[c];
    };
    auto widen = [](const Raw &r) -> float4 {
        if constexpr (kF16) {
            const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&r.x)), b = __half22float2(*reinterpret_cast<const __half2 *>(&r.y));
            return make_float4(a.x, a.y, b.x, b.y);
        } else {
            return r;
        }
    };
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int j = 0;
    // sixteen, then (up to) four part loads in flight per thread: one long context cut into a piece per worker is merged by
    // one block per head, and the part loop is a chain of round trips to L2 / HBM
    for (; !kLean && j + 16 <= nparts; j += 16) {
        Raw raw[16];
#pragma unroll
        for (int u = 0; u < 16; ++u)
            raw[u] = load_part(slot_s[j + u]);
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            float wgt = w_s[j + u] * inv_z;
            if (wgt != 0.f) {          // a dead worker's slot holds stale bytes
                if constexpr (kF16) wgt *= sc_s[j + u];
                const float4 v = widen(raw[u]);
                acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y);
                acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
            }
        }
    }
    // the rest four at a time as well, loads first: taken one by one, each part's load would wait for the previous
    // part's arithmetic, and a request cut into two or three pieces (the usual case) would pay a round trip per piece
    for (; j < nparts; j += 4) {
        Raw raw[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (j + u < nparts) raw[u] = load_part(slot_s[j + u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float wgt = j + u < nparts ? w_s[j + u] * inv_z : 0.f;
            if (wgt != 0.f) {          // a dead worker's slot holds stale bytes
                if constexpr (kF16) wgt *= sc_s[j + u];
                const float4 v = widen(raw[u]);
                acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y);
                acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
            }
        }
    }
    o4[c] = acc;
    if (c == 0) *lse = L;
}

}  // namespace

cudaError_t launch_lse_merge(int num_parts, int64_t rows, int d_v, const float *part_out,
                             const float *part_lse, float *out, float *lse, cudaStream_t stream) {
    lse_merge_kernel<<<(unsigned)rows, kMergeThreads, 0, stream>>>(num_parts, rows, d_v, part_out, part_lse, out, lse);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_split_combine(const DecodeParams &p, const int4 *split_rec, cudaStream_t stream) {
    // at most one request straddles each boundary between consecutive workers
    const int max_split = p.num_workers < p.B ? p.num_workers : p.B;
    dim3 grid((unsigned)((int64_t)(p.head_end - p.head_begin) * max_split));
    static DeviceOnce once;
    once.run([&] {   // keep the decode kernel's shared-memory carve-out (a preference: a failure is not an error)
        cudaFuncSetAttribute(split_combine_kernel<false, false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        cudaFuncSetAttribute(split_combine_kernel<true, false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        cudaFuncSetAttribute(split_combine_kernel<false, true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        cudaFuncSetAttribute(split_combine_kernel<true, true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        return cudaSuccess;
    });
    // many requests per worker: every request is cut into a few pieces at most
    const bool lean = (int64_t)p.B * 4 >= p.num_workers;
    auto kernel = p.partial_f16 ? (lean ? split_combine_kernel<true, true> : split_combine_kernel<true, false>)
                                : (lean ? split_combine_kernel<false, true> : split_combine_kernel<false, false>);
    cudaError_t e = launch_dependent(kernel, grid, dim3(kMergeThreads), 0, stream, p, split_rec);
    count_launch();
    return e;
}

}  // namespace splash
