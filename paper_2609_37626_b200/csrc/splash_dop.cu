// DOP transfer layout changes (App. E): the regrouping kernels on either side of the two
// all-to-alls that turn a tensor in global-row, local-head order into owner-row, all-head
// order and back.  Whole rows of bytes are moved, nothing is computed: byte-exact.
//
//   pack_rows     send[p][j][0 .. da + db) = a[send_row[p]][j][0 .. da) ++ b[send_row[p]][j][0 .. db)
//                 (rows grouped by destination owner; the no-position and the rotary part of the query
//                 are fused into one row so that one collective moves both)
//   unpack_rows   out[send_row[p]][j][:] = recv[p][j][:]                  (the reverse exchange's last step)
//   swap_outer    out[r][s][:] = in[s][r][:]        ([T][n][h][d] <-> [n][T][h][d]: source-rank-major receive
//                 buffer to all-head order, head s * h + j from rank s, and its inverse)
//
// Each has a 16-byte vector path (all base pointers, row pitches and part lengths multiples of 16
// bytes) and a 2-byte scalar fallback.  HBM-bound: bytes read + bytes written.
#include "splash_common.cuh"

namespace splash {

namespace {

constexpr int kDopThreads = 256;

// One (position, head) row of out per loop trip of a warp-sized group; VEC = uint4 or uint16_t.
// grid.x walks positions, blockDim covers (heads x vectors).
template <typename VEC>
__global__ void __launch_bounds__(kDopThreads)
pack_rows_kernel(const VEC *__restrict__ a, const VEC *__restrict__ b, VEC *__restrict__ out,
                 const int32_t *__restrict__ send_row, int64_t n, int h, int va, int vb,
                 int64_t a_row_pitch, int64_t a_head_pitch, int64_t b_row_pitch, int64_t b_head_pitch) {
    const int vrow = va + vb;                      // vectors per (position, head)
    const int64_t per_pos = (int64_t)h * vrow;
    for (int64_t p = blockIdx.x; p < n; p += gridDim.x) {
        const int64_t src = send_row[p];
        for (int64_t i = threadIdx.x; i < per_pos; i += kDopThreads) {
            const int j = (int)(i / vrow), c = (int)(i % vrow);
            VEC v = c < va ? __ldg(a + src * a_row_pitch + (int64_t)j * a_head_pitch + c)
                           : __ldg(b + src * b_row_pitch + (int64_t)j * b_head_pitch + (c - va));
            out[p * per_pos + i] = v;
        }
    }
}

template <typename VEC>
__global__ void __launch_bounds__(kDopThreads)
unpack_rows_kernel(const VEC *__restrict__ recv, VEC *__restrict__ out, const int32_t *__restrict__ send_row,
                   int64_t n, int64_t per_pos, int64_t out_row_pitch) {
    for (int64_t p = blockIdx.x; p < n; p += gridDim.x) {
        const int64_t dst = send_row[p];
        for (int64_t i = threadIdx.x; i < per_pos; i += kDopThreads) out[dst * out_row_pitch + i] = __ldg(recv + p * per_pos + i);
    }
}

// block (s, r) of `inner` vectors moves from in[s][r] to out[r][s]
template <typename VEC>
__global__ void __launch_bounds__(kDopThreads)
swap_outer_kernel(const VEC *__restrict__ in, VEC *__restrict__ out, int64_t A, int64_t Bn, int64_t inner) {
    const int64_t blocks = A * Bn;
    for (int64_t blk = blockIdx.x; blk < blocks; blk += gridDim.x) {
        const int64_t s = blk / Bn, r = blk % Bn;
        const VEC *src = in + blk * inner;
        VEC *dst = out + (r * A + s) * inner;
        for (int64_t i = threadIdx.x; i < inner; i += kDopThreads) dst[i] = __ldg(src + i);
    }
}

inline bool mult16(int64_t x) { return (x & 15) == 0; }
inline bool ptr16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline unsigned grid_for(int64_t items, int sm_count) {
    const int64_t cap = (int64_t)(sm_count > 0 ? sm_count : 148) * 8;
    return (unsigned)(items < cap ? (items > 0 ? items : 1) : cap);
}

}  // namespace

cudaError_t launch_dop_pack_rows(const void *a, const void *b, void *out, const int32_t *send_row, int64_t n, int h,
                                 int64_t a_bytes, int64_t b_bytes, int64_t a_row_pitch, int64_t a_head_pitch,
                                 int64_t b_row_pitch, int64_t b_head_pitch, int sm_count, cudaStream_t stream) {
    const bool vec = ptr16(a) && ptr16(out) && (b == nullptr || ptr16(b)) && mult16(a_bytes) && mult16(b_bytes) &&
                     mult16(a_row_pitch) && mult16(a_head_pitch) && mult16(b_row_pitch) && mult16(b_head_pitch);
    const dim3 grid(grid_for(n, sm_count));
    if (vec)
        pack_rows_kernel<uint4><<<grid, kDopThreads, 0, stream>>>(
            static_cast<const uint4 *>(a), static_cast<const uint4 *>(b), static_cast<uint4 *>(out), send_row, n, h,
            (int)(a_bytes / 16), (int)(b_bytes / 16), a_row_pitch / 16, a_head_pitch / 16, b_row_pitch / 16, b_head_pitch / 16);
    else
        pack_rows_kernel<uint16_t><<<grid, kDopThreads, 0, stream>>>(
            static_cast<const uint16_t *>(a), static_cast<const uint16_t *>(b), static_cast<uint16_t *>(out), send_row, n, h,
            (int)(a_bytes / 2), (int)(b_bytes / 2), a_row_pitch / 2, a_head_pitch / 2, b_row_pitch / 2, b_head_pitch / 2);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dop_unpack_rows(const void *recv, void *out, const int32_t *send_row, int64_t n, int64_t row_bytes,
                                   int64_t out_row_pitch, int sm_count, cudaStream_t stream) {
    const bool vec = ptr16(recv) && ptr16(out) && mult16(row_bytes) && mult16(out_row_pitch);
    const dim3 grid(grid_for(n, sm_count));
    if (vec)
        unpack_rows_kernel<uint4><<<grid, kDopThreads, 0, stream>>>(static_cast<const uint4 *>(recv), static_cast<uint4 *>(out),
                                                                    send_row, n, row_bytes / 16, out_row_pitch / 16);
    else
        unpack_rows_kernel<uint16_t><<<grid, kDopThreads, 0, stream>>>(static_cast<const uint16_t *>(recv),
                                                                       static_cast<uint16_t *>(out), send_row, n,
                                                                       row_bytes / 2, out_row_pitch / 2);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dop_swap_outer(const void *in, void *out, int64_t A, int64_t Bn, int64_t inner_bytes, int sm_count,
                                  cudaStream_t stream) {
    const bool vec = ptr16(in) && ptr16(out) && mult16(inner_bytes);
    const dim3 grid(grid_for(A * Bn, sm_count));
    if (vec)
        swap_outer_kernel<uint4><<<grid, kDopThreads, 0, stream>>>(static_cast<const uint4 *>(in), static_cast<uint4 *>(out), A, Bn,
                                                                   inner_bytes / 16);
    else
        swap_outer_kernel<uint16_t><<<grid, kDopThreads, 0, stream>>>(static_cast<const uint16_t *>(in),
                                                                      static_cast<uint16_t *>(out), A, Bn, inner_bytes / 2);
    count_launch();
    return cudaGetLastError();
}

}  // namespace splash
