// Anchor and anomaly kernels: the two passes over the keys.
//
//   anchor_sums   (Section 2.1, 2.2)  1/||k_i|| per token and the sum of normalised
//                                     keys of every episodic block
//   anchor_means  (Section 2.2)       block means and the stable mean
//   anchor_norms                      1/||mu_s||, 1/||mu_e[t]|| and min/max key reset
//   scan_scores   (Section 2.3)       a_s, a_e, a_c of every token from one staged
//                                     read of the key tile, plus per-head min/max
//   window_means  (Section 2.2)       explicit mu_c(i), for inspection only
//
// Thread mapping shared by the key passes: a row of d elements is split over an
// 8-lane group as 16-byte chunks, lane l owning chunks l, l+8, l+16, ...  A warp
// therefore reads four rows per instruction, each quarter-warp touching 128
// contiguous bytes (full sectors in global memory, all 32 banks once in shared
// memory), and a row-wise dot product needs three shuffle steps.
#include "nkv_common.cuh"

namespace nkv {

namespace {

template <typename T, int D>
struct RowMap {
    static constexpr int kRowBytes = D * (int)sizeof(T);
    static constexpr int kChunks = kRowBytes / 128;          // 16-byte chunks per lane
    static constexpr int kPerChunk = Elem<T>::kPerChunk;     // elements per chunk
    static constexpr int kCols = kChunks * kPerChunk;        // columns per lane (D/8)
    // column of element e of chunk j for lane l
    __device__ __forceinline__ static int col(int l, int j, int e) { return (l + 8 * j) * kPerChunk + e; }
};

template <typename T, int D>
__device__ __forceinline__ void load_row_chunks(const unsigned char* row, int l, float* v) {
    using M = RowMap<T, D>;
#pragma unroll
    for (int j = 0; j < M::kChunks; ++j) {
        uint4 q = *reinterpret_cast<const uint4*>(row + (l + 8 * j) * 16);
        Elem<T>::unpack(q, v + j * M::kPerChunk);
    }
}

// fp32 vector laid out by column (anchors, segment sums) -> the lane's columns
template <typename T, int D>
__device__ __forceinline__ void load_cols(const float* vec, int l, float* v) {
    using M = RowMap<T, D>;
#pragma unroll
    for (int j = 0; j < M::kChunks; ++j)
#pragma unroll
        for (int e = 0; e < M::kPerChunk; e += 4) {
            float4 f = *reinterpret_cast<const float4*>(vec + M::col(l, j, e));
            v[j * M::kPerChunk + e + 0] = f.x;
            v[j * M::kPerChunk + e + 1] = f.y;
            v[j * M::kPerChunk + e + 2] = f.z;
            v[j * M::kPerChunk + e + 3] = f.w;
        }
}
template <typename T, int D>
__device__ __forceinline__ void store_cols(float* vec, int l, const float* v) {
    using M = RowMap<T, D>;
#pragma unroll
    for (int j = 0; j < M::kChunks; ++j)
#pragma unroll
        for (int e = 0; e < M::kPerChunk; e += 4) {
            float4 f = make_float4(v[j * M::kPerChunk + e], v[j * M::kPerChunk + e + 1],
                                   v[j * M::kPerChunk + e + 2], v[j * M::kPerChunk + e + 3]);
            *reinterpret_cast<float4*>(vec + M::col(l, j, e)) = f;
        }
}

// ------------------------------------------------------------------------------------------
// anchor_sums: one CTA per (episodic block, head).
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) anchor_sums_kernel(TensorView K, ScoreParams sp, float* __restrict__ block_sums,
                                                          float* __restrict__ inv_norm) {
    using M = RowMap<T, D>;
    __shared__ float red[32][D];
    const int u = blockIdx.x / sp.nblocks, t = blockIdx.x - u * sp.nblocks;
    const int g = u / K.H, h = u % K.H;
    const unsigned char* base =
        reinterpret_cast<const unsigned char*>(K.ptr) + ((int64_t)g * K.stride_g + (int64_t)h * K.stride_h) * sizeof(T);
    const int row0 = t * sp.block;
    const int row1 = min(K.N, row0 + sp.block);
    const int grp = threadIdx.x >> 3, l = threadIdx.x & 7;

    float acc[M::kCols];
#pragma unroll
    for (int c = 0; c < M::kCols; ++c) acc[c] = 0.f;

    const int iters = (sp.block + 31) / 32;
#pragma unroll 2
    for (int it = 0; it < iters; ++it) {
        const int r = row0 + grp + 32 * it;
        const bool ok = r < row1;
        float v[M::kCols];
        if (ok) {
            load_row_chunks<T, D>(base + (int64_t)r * M::kRowBytes, l, v);
        } else {
#pragma unroll
            for (int c = 0; c < M::kCols; ++c) v[c] = 0.f;
        }
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < M::kCols; ++c) ss = fmaf(v[c], v[c], ss);
        ss = group8_sum(ss);
        const float inv = 1.0f / fmaxf(sqrtf(ss), kEps);
        if (ok) {
#pragma unroll
            for (int c = 0; c < M::kCols; ++c) acc[c] = fmaf(v[c], inv, acc[c]);
            if (l == 0) inv_norm[(int64_t)u * K.N + r] = inv;
        }
    }
    store_cols<T, D>(&red[grp][0], l, acc);
    __syncthreads();
    if (threadIdx.x < D) {
        float s = 0.f;
#pragma unroll 8
        for (int q = 0; q < 32; ++q) s += red[q][threadIdx.x];
        block_sums[((int64_t)u * sp.nblocks + t) * D + threadIdx.x] = s;
    }
}

// anchor_means: block sums -> block means (in place) and the stable mean (compensated sum over blocks).
__global__ void anchor_means_kernel(int N, int d, ScoreParams sp, float* __restrict__ mu_e, float* __restrict__ mu_s) {
    const int u = blockIdx.x, c = threadIdx.x;
    if (c >= d) return;
    float sum = 0.f, comp = 0.f;
    float* col = mu_e + (int64_t)u * sp.nblocks * d + c;
    for (int t0 = 0; t0 < sp.nblocks; t0 += 8) {   // eight block sums in flight, then added in block order
        float s[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) s[k] = t0 + k < sp.nblocks ? col[(int64_t)(t0 + k) * d] : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int t = t0 + k;
            if (t < sp.nblocks) {
                const float y = s[k] - comp;
                const float z = sum + y;
                comp = (z - sum) - y;
                sum = z;
                const int cnt = min(N, (t + 1) * sp.block) - t * sp.block;
                col[(int64_t)t * d] = s[k] / (float)cnt;
            }
        }
    }
    mu_s[(int64_t)u * d + c] = sum / (float)N;
}

// anchor_norms: reciprocal norms of the anchors; also resets the per-head min/max keys.
__global__ void __launch_bounds__(128) anchor_norms_kernel(int d, ScoreParams sp, const float* __restrict__ mu_s,
                                                           const float* __restrict__ mu_e, float* __restrict__ inv_s,
                                                           float* __restrict__ inv_e, uint32_t* __restrict__ mm) {
    const int u = blockIdx.x, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll 4
    for (int t = w - 1; t < sp.nblocks; t += 4) {
        const float* v = (t < 0) ? mu_s + (int64_t)u * d : mu_e + ((int64_t)u * sp.nblocks + t) * d;
        float ss = 0.f;
        for (int c = lane; c < d; c += 32) ss = fmaf(v[c], v[c], ss);
        ss = warp_sum(ss);
        if (lane == 0) {
            const float inv = 1.0f / fmaxf(sqrtf(ss), kEps);
            if (t < 0) inv_s[u] = inv;
            else inv_e[(int64_t)u * sp.nblocks + t] = inv;
        }
    }
    if (mm && threadIdx.x < 6) mm[(int64_t)u * 6 + threadIdx.x] = (threadIdx.x & 1) ? 0u : 0xffffffffu;  // [scale][min,max]
}

// ------------------------------------------------------------------------------------------
// scan_scores: one CTA per tile of 256 tokens (+64 rows of halo) of one head.
// ------------------------------------------------------------------------------------------
constexpr int kTile = 256;
constexpr int kRows = kTile + kMaxWindow;
constexpr int kSegs = kRows / kSeg;

template <typename T, int D>
constexpr size_t scan_smem_bytes() {
    return (size_t)kRows * D * sizeof(T) + kRows * sizeof(float) + (size_t)kSegs * D * sizeof(float) +
           3 * kTile * sizeof(float) + 8 * 6 * sizeof(float);
}

template <typename T, int D>
__global__ void __launch_bounds__(256, (sizeof(T) == 2 ? 2 : 1))
scan_scores_kernel(TensorView K, ScoreParams sp, const float* __restrict__ mu_s, const float* __restrict__ mu_e,
                   const float* __restrict__ inv_norm, const float* __restrict__ inv_s,
                   const float* __restrict__ inv_e, float* __restrict__ a_raw, uint32_t* __restrict__ mm) {
    using M = RowMap<T, D>;
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned char* tile = smem;
    float* invs = reinterpret_cast<float*>(smem + (size_t)kRows * M::kRowBytes);
    float* segsum = invs + kRows;
    float* outbuf = segsum + kSegs * D;
    float* red = outbuf + 3 * kTile;

    const int N = K.N;
    const int tiles = (N + kTile - 1) / kTile;
    const int u = blockIdx.x / tiles;
    const int g = u / K.H, h = u % K.H;
    const int i0 = (blockIdx.x - u * tiles) * kTile;
    const unsigned char* base =
        reinterpret_cast<const unsigned char*>(K.ptr) + ((int64_t)g * K.stride_g + (int64_t)h * K.stride_h) * sizeof(T);
    const int tid = threadIdx.x, grp = tid >> 3, l = tid & 7;

    // stage rows [i0-64, i0+256) and their reciprocal norms; rows outside [0, N) are zero
    constexpr int kChunksPerRow = M::kRowBytes / 16;
    for (int idx = tid; idx < kRows * kChunksPerRow; idx += 256) {
        const int sr = idx / kChunksPerRow;
        const int gr = i0 - kMaxWindow + sr;
        uint4 q = make_uint4(0u, 0u, 0u, 0u);
        if (gr >= 0 && gr < N)
            q = *reinterpret_cast<const uint4*>(base + (int64_t)gr * M::kRowBytes + (idx - sr * kChunksPerRow) * 16);
        *reinterpret_cast<uint4*>(tile + (size_t)idx * 16) = q;
    }
    for (int sr = tid; sr < kRows; sr += 256) {
        const int gr = i0 - kMaxWindow + sr;
        invs[sr] = (gr >= 0 && gr < N) ? inv_norm[(int64_t)u * N + gr] : 0.f;
    }
    __syncthreads();

    // sums of normalised keys over every 8-row segment of the staged rows
    for (int s = grp; s < kSegs; s += 32) {
        float acc[M::kCols];
#pragma unroll
        for (int c = 0; c < M::kCols; ++c) acc[c] = 0.f;
#pragma unroll
        for (int r = 0; r < kSeg; ++r) {
            const int sr = s * kSeg + r;
            float v[M::kCols];
            load_row_chunks<T, D>(tile + (size_t)sr * M::kRowBytes, l, v);
            const float inv = invs[sr];
#pragma unroll
            for (int c = 0; c < M::kCols; ++c) acc[c] = fmaf(v[c], inv, acc[c]);
        }
        store_cols<T, D>(segsum + s * D, l, acc);
    }
    __syncthreads();

    // each 8-lane group walks its own 8 tokens with a running window sum seeded from the segment sums
    const int W = sp.window;
    const int st = grp + kMaxWindow / kSeg;  // segment index of this group's tokens among the staged rows
    float Sw[M::kCols];
#pragma unroll
    for (int c = 0; c < M::kCols; ++c) Sw[c] = 0.f;
    {
        const int full = W / kSeg;
        for (int s = st - full; s < st; ++s) {
            float v[M::kCols];
            load_cols<T, D>(segsum + s * D, l, v);
#pragma unroll
            for (int c = 0; c < M::kCols; ++c) Sw[c] += v[c];
        }
        for (int sr = st * kSeg - W; sr < (st - full) * kSeg; ++sr) {
            float v[M::kCols];
            load_row_chunks<T, D>(tile + (size_t)sr * M::kRowBytes, l, v);
            const float inv = invs[sr];
#pragma unroll
            for (int c = 0; c < M::kCols; ++c) Sw[c] = fmaf(v[c], inv, Sw[c]);
        }
    }

    float ms[M::kCols], me[M::kCols];
    load_cols<T, D>(mu_s + (int64_t)u * D, l, ms);
    const float rs = inv_s[u];
    int cur_blk = -1;
    float re = 0.f;
    float lo[3] = {INFINITY, INFINITY, INFINITY}, hi[3] = {-INFINITY, -INFINITY, -INFINITY};

#pragma unroll 1
    for (int o = 0; o < kSeg; ++o) {
        const int sr = st * kSeg + o;
        const int gi = i0 + grp * kSeg + o;
        const bool valid = gi < N;
        const int blk = min(gi / sp.block, sp.nblocks - 1);
        if (blk != cur_blk) {
            cur_blk = blk;
            load_cols<T, D>(mu_e + ((int64_t)u * sp.nblocks + blk) * D, l, me);
            re = inv_e[(int64_t)u * sp.nblocks + blk];
        }
        float kn[M::kCols], ko[M::kCols];
        load_row_chunks<T, D>(tile + (size_t)sr * M::kRowBytes, l, kn);
        load_row_chunks<T, D>(tile + (size_t)(sr - W) * M::kRowBytes, l, ko);
        const float inv_n = invs[sr];
        const float ninv_o = -invs[sr - W];
        float dc = 0.f, nc = 0.f, ds = 0.f, de = 0.f;
#pragma unroll
        for (int c = 0; c < M::kCols; ++c) {
            float s = fmaf(inv_n, kn[c], Sw[c]);
            s = fmaf(ninv_o, ko[c], s);
            Sw[c] = s;
            dc = fmaf(kn[c], s, dc);
            nc = fmaf(s, s, nc);
            ds = fmaf(kn[c], ms[c], ds);
            de = fmaf(kn[c], me[c], de);
        }
        dc = group8_sum(dc);
        nc = group8_sum(nc);
        ds = group8_sum(ds);
        de = group8_sum(de);
        if (l == 0) {
            // a_k = -cos(k_hat_i, mu_k); adding +0 turns a -0 into +0
            const float a_s = -(ds * inv_n) * rs + 0.f;
            const float a_e = -(de * inv_n) * re + 0.f;
            const float a_c = -(dc * inv_n) / fmaxf(sqrtf(nc), kEps) + 0.f;
            const int j = grp * kSeg + o;
            outbuf[j] = a_s;
            outbuf[kTile + j] = a_e;
            outbuf[2 * kTile + j] = a_c;
            if (valid) {
                lo[0] = fminf(lo[0], a_s); hi[0] = fmaxf(hi[0], a_s);
                lo[1] = fminf(lo[1], a_e); hi[1] = fmaxf(hi[1], a_e);
                lo[2] = fminf(lo[2], a_c); hi[2] = fmaxf(hi[2], a_c);
            }
        }
    }

    // per-head min / max of each scale: warp -> CTA -> global ordered keys
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        lo[k] = warp_min(lo[k]);
        hi[k] = warp_max(hi[k]);
    }
    if ((tid & 31) == 0) {
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            red[(tid >> 5) * 6 + 2 * k] = lo[k];
            red[(tid >> 5) * 6 + 2 * k + 1] = hi[k];
        }
    }
    __syncthreads();
    if (tid < 6) {
        float v = red[tid];
        for (int w = 1; w < 8; ++w) v = (tid & 1) ? fmaxf(v, red[w * 6 + tid]) : fminf(v, red[w * 6 + tid]);
        if (tid & 1) atomicMax(&mm[(int64_t)u * 6 + tid], ord_key(v));
        else atomicMin(&mm[(int64_t)u * 6 + tid], ord_key(v));
    }
    for (int idx = tid; idx < 3 * kTile; idx += 256) {
        const int k = idx / kTile, j = idx - k * kTile;
        if (i0 + j < N) a_raw[((int64_t)u * 3 + k) * N + i0 + j] = outbuf[idx];
    }
}

// window_means: explicit current-memory mean of every token (inspection only).
template <typename T>
__global__ void window_means_kernel(TensorView K, ScoreParams sp, const float* __restrict__ inv_norm,
                                    float* __restrict__ mu_c) {
    const int u = blockIdx.x / K.N, g = u / K.H, h = u % K.H;
    const int i = blockIdx.x - u * K.N, c = threadIdx.x;
    if (c >= K.d) return;
    const T* base = reinterpret_cast<const T*>(K.ptr) + (int64_t)g * K.stride_g + (int64_t)h * K.stride_h;
    const int lft = max(0, i - sp.window + 1);
    float s = 0.f;
    for (int j = lft; j <= i; ++j) s = fmaf((float)base[(int64_t)j * K.d + c], inv_norm[(int64_t)u * K.N + j], s);
    mu_c[((int64_t)u * K.N + i) * K.d + c] = s / (float)(i - lft + 1);
}

template <typename T, int D>
cudaError_t set_scan_attr() {
    return cudaFuncSetAttribute(scan_scores_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)scan_smem_bytes<T, D>());
}

}  // namespace

cudaError_t configure_scan_kernels() {
    cudaError_t e;
    if ((e = set_scan_attr<__nv_bfloat16, 64>()) != cudaSuccess) return e;
    if ((e = set_scan_attr<__nv_bfloat16, 128>()) != cudaSuccess) return e;
    if ((e = set_scan_attr<__half, 64>()) != cudaSuccess) return e;
    if ((e = set_scan_attr<__half, 128>()) != cudaSuccess) return e;
    if ((e = set_scan_attr<float, 64>()) != cudaSuccess) return e;
    if ((e = set_scan_attr<float, 128>()) != cudaSuccess) return e;
    return cudaSuccess;
}

#define NKV_DISPATCH(dtype, d, CALL)                                   \
    do {                                                               \
        if ((dtype) == NKV_BF16 && (d) == 64) { CALL(__nv_bfloat16, 64); }  \
        else if ((dtype) == NKV_BF16 && (d) == 128) { CALL(__nv_bfloat16, 128); } \
        else if ((dtype) == NKV_F16 && (d) == 64) { CALL(__half, 64); }  \
        else if ((dtype) == NKV_F16 && (d) == 128) { CALL(__half, 128); } \
        else if ((dtype) == NKV_F32 && (d) == 64) { CALL(float, 64); }  \
        else if ((dtype) == NKV_F32 && (d) == 128) { CALL(float, 128); } \
        else return cudaErrorInvalidValue;                             \
    } while (0)

cudaError_t launch_anchor_sums(const TensorView& K, int dtype, int G, const ScoreParams& sp, float* block_sums,
                               float* inv_norm, cudaStream_t stream, int64_t* launches) {
    const unsigned grid = (unsigned)sp.nblocks * (unsigned)(G * K.H);
#define CALL(T, D) anchor_sums_kernel<T, D><<<grid, 256, 0, stream>>>(K, sp, block_sums, inv_norm)
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_anchor_means(int units, int N, int d, const ScoreParams& sp, float* mu_e_inout, float* mu_s,
                                cudaStream_t stream, int64_t* launches) {
    anchor_means_kernel<<<units, d, 0, stream>>>(N, d, sp, mu_e_inout, mu_s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_anchor_norms(int units, int d, const ScoreParams& sp, const float* mu_s, const float* mu_e,
                                float* inv_mu_s_norm, float* inv_mu_e_norm, uint32_t* minmax_keys,
                                cudaStream_t stream, int64_t* launches) {
    anchor_norms_kernel<<<units, 128, 0, stream>>>(d, sp, mu_s, mu_e, inv_mu_s_norm, inv_mu_e_norm, minmax_keys);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_scan_scores(const TensorView& K, int dtype, int G, const ScoreParams& sp, const float* mu_s,
                               const float* mu_e, const float* inv_norm, const float* inv_mu_s_norm,
                               const float* inv_mu_e_norm, float* a_raw, uint32_t* minmax_keys,
                               cudaStream_t stream, int64_t* launches) {
    const unsigned grid = (unsigned)((K.N + kTile - 1) / kTile) * (unsigned)(G * K.H);
#define CALL(T, D)                                                                                              \
    scan_scores_kernel<T, D><<<grid, 256, scan_smem_bytes<T, D>(), stream>>>(K, sp, mu_s, mu_e, inv_norm,       \
                                                                             inv_mu_s_norm, inv_mu_e_norm, a_raw, \
                                                                             minmax_keys)
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_window_means(const TensorView& K, int dtype, int G, const ScoreParams& sp, const float* inv_norm,
                                float* mu_c, cudaStream_t stream, int64_t* launches) {
    const unsigned grid = (unsigned)K.N * (unsigned)(G * K.H);
    if (dtype == NKV_BF16) window_means_kernel<__nv_bfloat16><<<grid, K.d, 0, stream>>>(K, sp, inv_norm, mu_c);
    else if (dtype == NKV_F16) window_means_kernel<__half><<<grid, K.d, 0, stream>>>(K, sp, inv_norm, mu_c);
    else window_means_kernel<float><<<grid, K.d, 0, stream>>>(K, sp, inv_norm, mu_c);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
