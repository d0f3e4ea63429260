// Compaction kernels (Section 2.1: the compressed memory is (K_S, V_S), rows unchanged).
//
//   gather           out of place: packed [G, cap, d] outputs, one 16-byte chunk per thread,
//                    K and V rows of a batch of output rows copied by the same CTA
//   gather_in_place  each head's retained rows move to the front of its own slab
#include "nkv_common.cuh"

namespace nkv {

namespace {

constexpr int kRowsPerBatch = 32;   // in-place kernel
constexpr int kGatherRows = 128;    // out-of-place kernel: rows per batch (64: 8 % slower at 9.7 GB of rows)
constexpr int kGatherInFlight = 8;  // 16-byte loads each thread issues before its first store

struct GatherArgs {
    const unsigned char* src[2];
    unsigned char* dst[2];
    int64_t stride_g[2], stride_h[2];  // bytes
    int row_bytes[2];
    int H, N;
    int64_t cap;
    int64_t total_rows;  // G * cap
};

__global__ void __launch_bounds__(256) gather_kernel(GatherArgs A, const int32_t* __restrict__ idx,
                                                     const int32_t* __restrict__ head_offsets) {
    __shared__ int64_t src_off[2][kGatherRows];
    const int64_t nbatch = (A.total_rows + kGatherRows - 1) / kGatherRows;
    const int cpr0 = A.row_bytes[0] >> 4, cpr1 = A.dst[1] ? (A.row_bytes[1] >> 4) : 0;   // 16-byte chunks per row
    const int total0 = A.dst[0] ? kGatherRows * cpr0 : 0, total = total0 + kGatherRows * cpr1;
    for (int64_t batch = blockIdx.x; batch < nbatch; batch += gridDim.x) {
        const int64_t row0 = batch * kGatherRows;
        __syncthreads();
        if (threadIdx.x < kGatherRows) {
            const int64_t J = row0 + threadIdx.x;
            int64_t o0 = -1, o1 = -1;
            if (J < A.total_rows) {
                const int64_t g = J / A.cap;
                const int j = (int)(J - g * A.cap);
                const int32_t* offs = head_offsets + g * (A.H + 1);
                if (j < offs[A.H]) {
                    int h = 0;
                    while (h + 1 < A.H && j >= offs[h + 1]) ++h;
                    const int r = idx[J];
                    if (r >= 0 && r < A.N) {
                        o0 = g * A.stride_g[0] + h * A.stride_h[0] + (int64_t)r * A.row_bytes[0];
                        o1 = g * A.stride_g[1] + h * A.stride_h[1] + (int64_t)r * A.row_bytes[1];
                    }
                }
            }
            src_off[0][threadIdx.x] = o0;
            src_off[1][threadIdx.x] = o1;
        }
        __syncthreads();
        // the chunks of the batch's K rows, then of its V rows, form one list; every thread keeps
        // kGatherInFlight loads in flight before it stores
        for (int c0 = threadIdx.x; c0 < total; c0 += 256 * kGatherInFlight) {
            uint4 q[kGatherInFlight];
            uint4* dst[kGatherInFlight];
#pragma unroll
            for (int e = 0; e < kGatherInFlight; ++e) {
                const int c = c0 + e * 256;
                dst[e] = nullptr;
                if (c < total) {
                    const int t = c >= total0 ? 1 : 0;
                    const int cc = t ? c - total0 : c;
                    const int cpr = t ? cpr1 : cpr0;
                    const int r = cc / cpr, k = cc - r * cpr;
                    const int64_t so = src_off[t][r];
                    if (so >= 0) {
                        q[e] = __ldcs(reinterpret_cast<const uint4*>(A.src[t] + so) + k);
                        dst[e] = reinterpret_cast<uint4*>(A.dst[t] + (row0 + r) * A.row_bytes[t]) + k;
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < kGatherInFlight; ++e)
                if (dst[e]) __stcs(dst[e], q[e]);
        }
    }
}

// One CTA per head.  Positions are ascending and idx[j] >= j, so processing the output rows in
// order, a batch at a time with all loads of a batch completed before its stores, never overwrites
// a row that is still needed.
__global__ void __launch_bounds__(256) gather_in_place_kernel(GatherArgs A, const int32_t* __restrict__ idx,
                                                              const int32_t* __restrict__ head_offsets) {
    const int u = blockIdx.x, g = u / A.H, h = u % A.H;
    const int32_t* offs = head_offsets + (int64_t)g * (A.H + 1);
    const int off = offs[h], B = offs[h + 1] - offs[h];
    const int32_t* my = idx + (int64_t)g * A.cap + off;
    for (int j0 = 0; j0 < B; j0 += kRowsPerBatch) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            if (A.src[t] == nullptr) continue;
            unsigned char* slab = const_cast<unsigned char*>(A.src[t]) + g * A.stride_g[t] + h * A.stride_h[t];
            const int cpr = A.row_bytes[t] >> 4;
            const int total = kRowsPerBatch * cpr;   // at most 32 * 32 = 1024 chunks: 4 per thread
            uint4 q[4];
            bool ok[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = threadIdx.x + e * 256;
                ok[e] = false;
                if (c < total) {
                    const int r = c / cpr;
                    if (j0 + r < B) {
                        const int s = my[j0 + r];
                        if (s >= 0 && s < A.N) {
                            ok[e] = true;
                            q[e] = *(reinterpret_cast<const uint4*>(slab + (int64_t)s * A.row_bytes[t]) + (c - r * cpr));
                        }
                    }
                }
            }
            __syncthreads();
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = threadIdx.x + e * 256;
                if (ok[e]) {
                    const int r = c / cpr;
                    *(reinterpret_cast<uint4*>(slab + (int64_t)(j0 + r) * A.row_bytes[t]) + (c - r * cpr)) = q[e];
                }
            }
            __syncthreads();
        }
    }
}

GatherArgs make_args(const TensorView& K, int kb, const TensorView& V, int vb, int G, int64_t cap, void* K_out,
                     void* V_out) {
    GatherArgs A;
    A.src[0] = reinterpret_cast<const unsigned char*>(K.ptr);
    A.src[1] = reinterpret_cast<const unsigned char*>(V.ptr);
    A.dst[0] = reinterpret_cast<unsigned char*>(K_out);
    A.dst[1] = reinterpret_cast<unsigned char*>(V_out);
    A.stride_g[0] = K.stride_g * kb;
    A.stride_h[0] = K.stride_h * kb;
    A.stride_g[1] = V.stride_g * vb;
    A.stride_h[1] = V.stride_h * vb;
    A.row_bytes[0] = K.d * kb;
    A.row_bytes[1] = V.d * vb;
    A.H = K.H;
    A.N = K.N;
    A.cap = cap;
    A.total_rows = (int64_t)G * cap;
    return A;
}

}  // namespace

cudaError_t launch_gather(const TensorView& K, int k_elem_bytes, const TensorView& V, int v_elem_bytes, int G,
                          const int32_t* idx, const int32_t* head_offsets, int64_t idx_capacity, void* K_out,
                          void* V_out, int sm_count, cudaStream_t stream, int64_t* launches) {
    GatherArgs A = make_args(K, k_elem_bytes, V, v_elem_bytes, G, idx_capacity, K_out, V_out);
    const int64_t nbatch = (A.total_rows + kGatherRows - 1) / kGatherRows;
    if (nbatch == 0) return cudaSuccess;
    int64_t grid = (int64_t)sm_count * 8;
    if (grid > nbatch) grid = nbatch;
    gather_kernel<<<(unsigned)grid, 256, 0, stream>>>(A, idx, head_offsets);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_gather_in_place(const TensorView& K, int k_elem_bytes, const TensorView& V, int v_elem_bytes, int G,
                                   const int32_t* idx, const int32_t* head_offsets, int64_t idx_capacity,
                                   cudaStream_t stream, int64_t* launches) {
    GatherArgs A = make_args(K, k_elem_bytes, V, v_elem_bytes, G, idx_capacity, nullptr, nullptr);
    gather_in_place_kernel<<<G * K.H, 256, 0, stream>>>(A, idx, head_offsets);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
