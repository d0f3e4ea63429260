// Shared device helpers and internal launch interfaces of the nkv library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "nkv.h"

namespace nkv {

constexpr float kEps = 1e-12f;       // floor for a norm used as a denominator
constexpr int kMaxWindow = 64;       // rows of halo the scoring tile carries
constexpr int kSeg = 8;              // rows per window segment (one 8-lane group walks one segment)

// Layout of the status words at the start of every workspace.
constexpr int kStatusWords = 64;     // 256 bytes
constexpr int kStatusCode = 0;       // 0, NKV_ERR_TIMEOUT or NKV_ERR_DEVICE_CHECK
constexpr int kStatusDetail = 1;     // where it happened
constexpr int kStatusFallbacks = 2;  // number of selections that took the radix fallback (informational)

// Internal description of a key/value tensor passed to kernels by value.
struct TensorView {
    const void* ptr;
    int64_t stride_g, stride_h;  // elements
    int H, N, d;
};

// Host-side resolved parameters handed to kernels.
struct ScoreParams {
    int window, n_sink, block, nblocks, gate_mode, top_m;
    float log_prior[3];
    float beta, tau, kappa;
};

// Order-preserving map float -> uint32 (larger float <=> larger key) and back.
__host__ __device__ __forceinline__ uint32_t ord_key(float f) {
#ifdef __CUDA_ARCH__
    uint32_t b = __float_as_uint(f);
#else
    uint32_t b;
    memcpy(&b, &f, 4);
#endif
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_float(uint32_t k) {
    uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(b);
}

// 16-byte chunk -> fp32 values.  bf16 and fp16: 8 values, fp32: 4 values.
template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerChunk = 8;
    static constexpr int kBytes = 2;
    __device__ __forceinline__ static void unpack(const uint4& q, float* v) {
        v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
        v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
        v[4] = __uint_as_float(q.z << 16); v[5] = __uint_as_float(q.z & 0xffff0000u);
        v[6] = __uint_as_float(q.w << 16); v[7] = __uint_as_float(q.w & 0xffff0000u);
    }
};
template <> struct Elem<__half> {
    static constexpr int kPerChunk = 8;
    static constexpr int kBytes = 2;
    __device__ __forceinline__ static void unpack(const uint4& q, float* v) {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
            v[2 * j] = f.x;
            v[2 * j + 1] = f.y;
        }
    }
};
template <> struct Elem<float> {
    static constexpr int kPerChunk = 4;
    static constexpr int kBytes = 4;
    __device__ __forceinline__ static void unpack(const uint4& q, float* v) {
        v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y);
        v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
    }
};

__device__ __forceinline__ float group8_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ void set_status(int* status, int code, int detail) {
    if (atomicCAS(&status[kStatusCode], 0, code) == 0) status[kStatusDetail] = detail;
}

// ---- launchers implemented in the .cu files (all enqueue on `stream`, return cudaError_t) ----
cudaError_t launch_threshold_scores(int units, const uint32_t* thr, float* out, cudaStream_t stream, int64_t* launches);
constexpr int kWaitProbeDetail = 799;   // status detail recorded by the wait probe
cudaError_t launch_wait_probe(int* status, uint32_t limit, cudaStream_t stream, int64_t* launches);
cudaError_t launch_anchor_sums(const TensorView& K, int dtype, int G, const ScoreParams& sp, float* block_sums,
                               float* inv_norm, cudaStream_t stream, int64_t* launches);
cudaError_t launch_anchor_means(int units, int N, int d, const ScoreParams& sp, float* mu_e_inout, float* mu_s,
                                cudaStream_t stream, int64_t* launches);
cudaError_t launch_window_means(const TensorView& K, int dtype, int G, const ScoreParams& sp, const float* inv_norm,
                                float* mu_c, cudaStream_t stream, int64_t* launches);
cudaError_t launch_anchor_norms(int units, int d, const ScoreParams& sp, const float* mu_s, const float* mu_e,
                                float* inv_mu_s_norm, float* inv_mu_e_norm, uint32_t* minmax_keys_to_reset_or_null,
                                cudaStream_t stream, int64_t* launches);
// streaming key passes (block size a multiple of 8)
bool stream_path_supported(const ScoreParams& sp);
cudaError_t launch_stream_a(const TensorView& K, int dtype, int G, const ScoreParams& sp, float* block_sums,
                            float* inv_norm, float* a_raw, uint32_t* mm, int* status, int sm_count,
                            cudaStream_t stream, int64_t* launches);
cudaError_t launch_stream_b(const TensorView& K, int dtype, int G, const ScoreParams& sp, const float* mu_s,
                            const float* mu_e, const float* inv_norm, const float* inv_s, const float* inv_e,
                            float* a_raw, uint32_t* mm, int* status, int sm_count, cudaStream_t stream,
                            int64_t* launches);
// first key pass on the tensor cores (bf16 keys, d = 128): same outputs as launch_stream_a
bool gram_pass_supported(const TensorView& K, int dtype, const ScoreParams& sp);
cudaError_t configure_gram_kernels();
cudaError_t launch_gram_pass(const TensorView& K, int G, const ScoreParams& sp, float* block_sums, float* inv_norm,
                             float* a_raw, uint32_t* mm, int* status, int sm_count, cudaStream_t stream,
                             int64_t* launches);
// second key pass on the tensor cores (bf16 keys, d = 128): same outputs as launch_stream_b
bool anchor_dots_supported(const TensorView& K, int dtype, const ScoreParams& sp);
cudaError_t configure_dots_kernels();
cudaError_t launch_anchor_dots(const TensorView& K, int G, const ScoreParams& sp, const float* mu_s, const float* mu_e,
                               const float* inv_norm, const float* inv_s, const float* inv_e, float* a_raw,
                               uint32_t* mm, int* status, int sm_count, cudaStream_t stream, int64_t* launches);
cudaError_t configure_select_kernels();
cudaError_t configure_scan_kernels();
cudaError_t configure_stream_kernels();
cudaError_t launch_scan_scores(const TensorView& K, int dtype, int G, const ScoreParams& sp, const float* mu_s,
                               const float* mu_e, const float* inv_norm, const float* inv_mu_s_norm,
                               const float* inv_mu_e_norm, float* a_raw, uint32_t* minmax_keys,
                               cudaStream_t stream, int64_t* launches);
size_t head_stat_bytes(int64_t units);   // scratch of launch_head_scores (`hstat`)
cudaError_t launch_head_scores(int units, int N, const ScoreParams& sp, const float* a_raw,
                               const uint32_t* minmax_keys, float* a_star, float* head_stats_opt, float* hstat,
                               int* status, cudaStream_t stream, int64_t* launches);
size_t budget_scratch_bytes(int64_t G, int64_t H);   // scratch of the parallel form of launch_budget
cudaError_t launch_budget(int G, int H, int N, int keep, int n_safe, const float* a_star, int32_t* budgets,
                          uint32_t* sel_thresholds, int* status, void* scratch_or_null, cudaStream_t stream,
                          int64_t* launches);
cudaError_t launch_select(int G, int H, int N, int64_t idx_capacity, const float* a_star, const int32_t* budgets,
                          const uint32_t* sel_thresholds_or_null, int32_t* idx, int32_t* head_offsets, int* status,
                          cudaStream_t stream, int64_t* launches);
cudaError_t launch_ranks(int units, int N, const float* a_star, int32_t* ranks, cudaStream_t stream,
                         int64_t* launches);
cudaError_t launch_gather(const TensorView& K, int k_elem_bytes, const TensorView& V, int v_elem_bytes, int G,
                          const int32_t* idx, const int32_t* head_offsets, int64_t idx_capacity, void* K_out,
                          void* V_out, int sm_count, cudaStream_t stream, int64_t* launches);
cudaError_t launch_gather_in_place(const TensorView& K, int k_elem_bytes, const TensorView& V, int v_elem_bytes, int G,
                                   const int32_t* idx, const int32_t* head_offsets, int64_t idx_capacity,
                                   cudaStream_t stream, int64_t* launches);

}  // namespace nkv
