// Streaming key passes of the fused path (used when the episodic block size is a multiple of 8).
//
//   stream_a  (Sections 2.1-2.3)  one pass over the keys that needs no anchor: 1/||k_i||, the sums of
//                                 normalised keys of every episodic block, and the current-memory
//                                 anomaly a_c(i) = -cos(k_hat_i, mu_c(i)) with its per-head min/max
//   stream_b  (Section 2.3)       the pass that needs the anchors: a_s(i), a_e(i) and their min/max
//
// Both kernels are persistent (one CTA per SM, tiles taken round-robin) and stage key tiles in shared
// memory with bulk asynchronous copies (cp.async.bulk + mbarrier), double buffered so the copy of the
// next tile overlaps the arithmetic of the current one.  A row of d elements is split over d/8 lanes,
// 8 columns per lane; each lane group walks 8 consecutive tokens and the per-token partial sums of the
// group are combined with a transposed shuffle reduction (about one shuffle per token and quantity).
// The sliding-window sum is a running sum over the 8 tokens of a group, seeded from exact sums of
// 8-row segments, so no long prefix sum is ever differenced.  FP32 arithmetic uses the packed
// two-wide fma/add forms of sm_100.
#include "nkv_common.cuh"

namespace nkv {

namespace {

constexpr int kHalo = kMaxWindow;   // rows staged in front of a tile
constexpr uint32_t kSpinLimit = 1u << 22;

// ---------------------------------------------------------------------------- async copy helpers
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_global, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src_global), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false (after setting the device status) if the copy never lands.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status, int where) {
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    set_status(status, NKV_ERR_TIMEOUT, where);
    return false;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------------------- packed fp32 helpers
struct F2 {
    unsigned long long v;
};
__device__ __forceinline__ F2 pack2(float a, float b) {
    F2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(F2 x, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(x.v)); }
__device__ __forceinline__ F2 fma2(F2 a, F2 b, F2 c) {
    F2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v));
    return r;
}
__device__ __forceinline__ F2 add2(F2 a, F2 b) {
    F2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
    return r;
}
__device__ __forceinline__ float hsum2(F2 x) {
    float a, b;
    unpack2(x, a, b);
    return a + b;
}

// 16-byte chunk -> packed pairs.  bf16 and fp16: 4 pairs (8 values), fp32: 2 pairs (4 values).
template <typename T> struct Pairs;
template <> struct Pairs<__nv_bfloat16> {
    static constexpr int kPairs = 4;
    __device__ __forceinline__ static void unpack(const uint4& q, F2* p) {
        p[0] = pack2(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u));
        p[1] = pack2(__uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u));
        p[2] = pack2(__uint_as_float(q.z << 16), __uint_as_float(q.z & 0xffff0000u));
        p[3] = pack2(__uint_as_float(q.w << 16), __uint_as_float(q.w & 0xffff0000u));
    }
};
template <> struct Pairs<__half> {
    static constexpr int kPairs = 4;
    __device__ __forceinline__ static void unpack(const uint4& q, F2* p) {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
            p[j] = pack2(f.x, f.y);
        }
    }
};
template <> struct Pairs<float> {
    static constexpr int kPairs = 2;
    __device__ __forceinline__ static void unpack(const uint4& q, F2* p) {
        p[0] = pack2(__uint_as_float(q.x), __uint_as_float(q.y));
        p[1] = pack2(__uint_as_float(q.z), __uint_as_float(q.w));
    }
};

// Geometry of one staged row for element type T and head dimension D: 8 columns (4 pairs) per lane.
template <typename T, int D>
struct Geo {
    static constexpr int kLanes = D / 8;                        // lanes per row
    static constexpr int kRowBytes = D * (int)sizeof(T);
    static constexpr int kPerChunk = 16 / (int)sizeof(T);       // elements per 16-byte chunk
    static constexpr int kChunks = 8 / kPerChunk;               // chunks per lane
    // first column of chunk j of lane l
    __device__ __forceinline__ static int col0(int l, int j) { return (l + kLanes * j) * kPerChunk; }
    __device__ __forceinline__ static void load_row(const unsigned char* row, int l, F2* p) {
#pragma unroll
        for (int j = 0; j < kChunks; ++j) {
            const uint4 q = *reinterpret_cast<const uint4*>(row + (l + kLanes * j) * 16);
            Pairs<T>::unpack(q, p + j * Pairs<T>::kPairs);
        }
    }
    // the lane's 8 columns of an fp32 vector laid out by column
    __device__ __forceinline__ static void load_vec(const float* vec, int l, F2* p) {
#pragma unroll
        for (int j = 0; j < kChunks; ++j)
#pragma unroll
            for (int e = 0; e < kPerChunk; e += 4) {
                const float4 f = *reinterpret_cast<const float4*>(vec + col0(l, j) + e);
                p[(j * kPerChunk + e) / 2] = pack2(f.x, f.y);
                p[(j * kPerChunk + e) / 2 + 1] = pack2(f.z, f.w);
            }
    }
    __device__ __forceinline__ static void store_vec(float* vec, int l, const F2* p) {
#pragma unroll
        for (int j = 0; j < kChunks; ++j)
#pragma unroll
            for (int e = 0; e < kPerChunk; e += 4) {
                float4 f;
                unpack2(p[(j * kPerChunk + e) / 2], f.x, f.y);
                unpack2(p[(j * kPerChunk + e) / 2 + 1], f.z, f.w);
                *reinterpret_cast<float4*>(vec + col0(l, j) + e) = f;
            }
    }
};

// Transposed reduction of V per-lane partial values over a group of L lanes (L, V powers of two).
// Afterwards v[0 .. max(1, V/L)) hold complete sums: with V >= L lane l owns values l*(V/L)+j,
// with V < L lane l owns value l / (L/V) (shared by L/V lanes).
template <int V, int L>
__device__ __forceinline__ void treduce(float* v, int l) {
    int n = V;
#pragma unroll
    for (int o = L / 2; o >= 1; o >>= 1) {
        if (n > 1) {
            const int half = n / 2;
            const bool up = (l & o) != 0;
#pragma unroll
            for (int j = 0; j < V / 2; ++j) {
                if (j < half) {
                    const float send = up ? v[j] : v[j + half];
                    const float keep = up ? v[j + half] : v[j];
                    v[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
            }
            n = half;
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
        }
    }
}

__device__ __forceinline__ void cta_minmax_to_global(float lo, float hi, float* red, int nwarps, uint32_t* mm_lo,
                                                     uint32_t* mm_hi) {
    lo = warp_min(lo);
    hi = warp_max(hi);
    if ((threadIdx.x & 31) == 0) {
        red[(threadIdx.x >> 5) * 2] = lo;
        red[(threadIdx.x >> 5) * 2 + 1] = hi;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < nwarps; ++w) {
            lo = fminf(lo, red[w * 2]);
            hi = fmaxf(hi, red[w * 2 + 1]);
        }
        if (lo <= hi) {
            atomicMin(mm_lo, ord_key(lo));
            atomicMax(mm_hi, ord_key(hi));
        }
    }
}

// ============================================================================================
// stream_a
// ============================================================================================
template <typename T, int D, int TILE>
struct ACfg {
    using G = Geo<T, D>;
    static constexpr int kRows = TILE + kHalo;
    static constexpr int kSegs = kRows / kSeg;
    static constexpr int kHaloSegs = kHalo / kSeg;
    static constexpr int kThreads = kSegs * G::kLanes;            // one lane group per staged segment
    static constexpr int kChunks64 = kRows / 64;                  // 64-row chunks (prefix granularity)
    static constexpr size_t kTileBytes = (size_t)kRows * G::kRowBytes;
    static constexpr size_t kSmem = 2 * kTileBytes + (size_t)kSegs * D * 4 + kRows * 4 + TILE * 4 + 64 * 4 + 64;
    static_assert(kThreads == kChunks64 * D, "prefix tasks must equal threads");
    static_assert(kThreads % 32 == 0 && kThreads <= 1024, "bad CTA size");
};

// sum over staged segments [s0, s1) of the per-segment sums, from inclusive prefixes within 64-row chunks
template <typename T, int D>
__device__ __forceinline__ void range_sum(const float* pp, int l, int s0, int s1, F2* out) {
    using G = Geo<T, D>;
#pragma unroll
    for (int p = 0; p < 4; ++p) out[p] = pack2(0.f, 0.f);
    if (s1 <= s0) return;
    for (int c = s0 >> 3; c <= (s1 - 1) >> 3; ++c) {
        const int lo = max(s0, c * 8), hi = min(s1, c * 8 + 8);
        F2 a[4];
        G::load_vec(pp + (size_t)(hi - 1) * D, l, a);
#pragma unroll
        for (int p = 0; p < 4; ++p) out[p] = add2(out[p], a[p]);
        if (lo > c * 8) {
            G::load_vec(pp + (size_t)(lo - 1) * D, l, a);
            const F2 m1 = pack2(-1.f, -1.f);
#pragma unroll
            for (int p = 0; p < 4; ++p) out[p] = fma2(a[p], m1, out[p]);
        }
    }
}

template <typename T, int D, int TILE>
__global__ void __launch_bounds__(ACfg<T, D, TILE>::kThreads, 1)
stream_a_kernel(TensorView K, ScoreParams sp, int units, float* __restrict__ block_sums, float* __restrict__ inv_norm,
                float* __restrict__ a_raw, uint32_t* __restrict__ mm, int* status) {
    using C = ACfg<T, D, TILE>;
    using G = Geo<T, D>;
    constexpr int L = G::kLanes;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* tiles = smem;
    float* pp = reinterpret_cast<float*>(smem + 2 * C::kTileBytes);   // [kSegs][D] segment sums -> chunk prefixes
    float* invs = pp + C::kSegs * D;                                  // [kRows]
    float* outbuf = invs + C::kRows;                                  // [TILE] a_c
    float* red = outbuf + TILE;                                       // [64]
    uint64_t* full = reinterpret_cast<uint64_t*>(red + 64);           // [2]

    const int N = K.N;
    const int tiles_per_unit = (N + TILE - 1) / TILE;
    const long long total = (long long)units * tiles_per_unit;
    const int tid = threadIdx.x, grp = tid / L, l = tid % L;
    const int W = sp.window;

    if (tid == 0) {
        mbar_init(&full[0], 1);
        mbar_init(&full[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto issue = [&](long long t, int buf) {   // thread 0 only
        const int u = (int)(t / tiles_per_unit);
        const int i0 = (int)(t - (long long)u * tiles_per_unit) * TILE;
        const int g = u / K.H, h = u % K.H;
        const unsigned char* base = reinterpret_cast<const unsigned char*>(K.ptr) +
                                    ((int64_t)g * K.stride_g + (int64_t)h * K.stride_h) * sizeof(T);
        const int r0 = max(0, i0 - kHalo), r1 = min(N, i0 + TILE);
        const uint32_t bytes = (uint32_t)(r1 - r0) * G::kRowBytes;
        unsigned char* dst = tiles + (size_t)buf * C::kTileBytes + (size_t)(r0 - (i0 - kHalo)) * G::kRowBytes;
        const unsigned char* src = base + (int64_t)r0 * G::kRowBytes;
        fence_async_smem();
        mbar_expect_tx(&full[buf], bytes);
        for (uint32_t off = 0; off < bytes; off += 16384u)
            bulk_load(dst + off, src + off, min(16384u, bytes - off), &full[buf]);
    };

    long long t = blockIdx.x;
    if (t < total && tid == 0) issue(t, 0);
    int it = 0;
    for (; t < total; t += gridDim.x, ++it) {
        const int buf = it & 1;
        const long long tn = t + gridDim.x;
        if (tn < total && tid == 0) issue(tn, buf ^ 1);

        const int u = (int)(t / tiles_per_unit);
        const int i0 = (int)(t - (long long)u * tiles_per_unit) * TILE;
        unsigned char* tile = tiles + (size_t)buf * C::kTileBytes;
        // rows outside [0, N) are not copied: zero them (disjoint from the bytes in flight)
        {
            const int r0 = max(0, i0 - kHalo), r1 = min(N, i0 + TILE);
            const int head_rows = r0 - (i0 - kHalo);            // missing rows in front
            const int tail_row0 = r1 - (i0 - kHalo);            // first missing row at the back
            constexpr int cpr = G::kRowBytes / 16;
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            for (int c = tid; c < head_rows * cpr; c += C::kThreads) reinterpret_cast<uint4*>(tile)[c] = z;
            for (int c = tail_row0 * cpr + tid; c < C::kRows * cpr; c += C::kThreads) reinterpret_cast<uint4*>(tile)[c] = z;
        }
        if (!mbar_wait(&full[buf], (uint32_t)((it >> 1) & 1), status, 401)) return;
        __syncthreads();

        // ---- S1: reciprocal norms and the sum of normalised keys of every staged 8-row segment
        {
            F2 acc[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) acc[p] = pack2(0.f, 0.f);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                F2 x[4][4];
                float n2[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    G::load_row(tile + (size_t)(grp * kSeg + half * 4 + r) * G::kRowBytes, l, x[r]);
                    F2 s = pack2(0.f, 0.f);
#pragma unroll
                    for (int p = 0; p < 4; ++p) s = fma2(x[r][p], x[r][p], s);
                    n2[r] = hsum2(s);
                }
                treduce<4, L>(n2, l);
                // lane l now owns the squared norm of row l / (L/4) of this half
                const float inv = 1.0f / fmaxf(sqrtf(n2[0]), kEps);
                if ((l & (L / 4 - 1)) == 0) invs[grp * kSeg + half * 4 + l / (L / 4)] = inv;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const float ir = __shfl_sync(0xffffffffu, inv, r * (L / 4), L);
                    const F2 ir2 = pack2(ir, ir);
#pragma unroll
                    for (int p = 0; p < 4; ++p) acc[p] = fma2(x[r][p], ir2, acc[p]);
                }
            }
            G::store_vec(pp + (size_t)grp * D, l, acc);
        }
        __syncthreads();
        // ---- S1b: inclusive prefix of the segment sums inside every 64-row chunk (one column per thread)
        {
            const int c64 = tid / D, col = tid - c64 * D;
            float run = 0.f;
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                float* q = pp + (size_t)(c64 * 8 + p) * D + col;
                run += *q;
                *q = run;
            }
        }
        __syncthreads();

        // ---- S2: sliding-window anomaly of the tile's tokens; block sums; outputs
        float lo = INFINITY, hi = -INFINITY;
        if (grp >= C::kHaloSegs) {
            const int s = grp;                       // staged segment of this group's 8 tokens
            F2 Sw[4];
            range_sum<T, D>(pp, l, s - W / kSeg, s, Sw);
            for (int sr = s * kSeg - W; sr < (s - W / kSeg) * kSeg; ++sr) {   // the W % 8 oldest rows
                F2 x[4];
                G::load_row(tile + (size_t)sr * G::kRowBytes, l, x);
                const float iv = invs[sr];
                const F2 iv2 = pack2(iv, iv);
#pragma unroll
                for (int p = 0; p < 4; ++p) Sw[p] = fma2(x[p], iv2, Sw[p]);
            }
            float part[16];
#pragma unroll
            for (int o = 0; o < kSeg; ++o) {
                const int sr = s * kSeg + o;
                F2 kn[4], ko[4];
                G::load_row(tile + (size_t)sr * G::kRowBytes, l, kn);
                G::load_row(tile + (size_t)(sr - W) * G::kRowBytes, l, ko);
                const float in = invs[sr], io = -invs[sr - W];
                const F2 in2 = pack2(in, in), io2 = pack2(io, io);
                F2 dc = pack2(0.f, 0.f), nc = pack2(0.f, 0.f);
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    F2 w = fma2(in2, kn[p], Sw[p]);
                    w = fma2(io2, ko[p], w);
                    Sw[p] = w;
                    dc = fma2(kn[p], w, dc);
                    nc = fma2(w, w, nc);
                }
                part[2 * o] = hsum2(dc);
                part[2 * o + 1] = hsum2(nc);
            }
            treduce<16, L>(part, l);
            // L == 16: lane l owns value l (token l/2, quantity l%2).  L == 8: lane l owns token l, both quantities.
            float dcv, ncv;
            int o;
            bool writer;
            if (L == 16) {
                const float other = __shfl_xor_sync(0xffffffffu, part[0], 1);
                dcv = part[0];
                ncv = other;
                o = l >> 1;
                writer = (l & 1) == 0;
            } else {
                dcv = part[0];
                ncv = part[1];
                o = l;
                writer = true;
            }
            if (writer) {
                const int j = (s - C::kHaloSegs) * kSeg + o;
                const float a_c = -(dcv * invs[s * kSeg + o]) / fmaxf(sqrtf(ncv), kEps) + 0.f;
                outbuf[j] = a_c;
                if (i0 + j < N) {
                    lo = a_c;
                    hi = a_c;
                }
            }
        }
        // sums of normalised keys of the episodic blocks that overlap this tile (one column per thread)
        if (tid < D) {
            const int b = sp.block;
            const int row_end = min(N, i0 + TILE);
            for (int blk = i0 / b; blk * b < row_end; ++blk) {
                const int rlo = max(blk * b, i0), rhi = min(min((blk + 1) * b, i0 + TILE), ((N + 7) / 8) * 8);
                const int s0 = C::kHaloSegs + (rlo - i0) / kSeg, s1 = C::kHaloSegs + (rhi - i0 + kSeg - 1) / kSeg;
                float sum = 0.f;
                for (int c = s0 >> 3; c <= (s1 - 1) >> 3; ++c) {
                    const int a = max(s0, c * 8), e = min(s1, c * 8 + 8);
                    sum += pp[(size_t)(e - 1) * D + tid];
                    if (a > c * 8) sum -= pp[(size_t)(a - 1) * D + tid];
                }
                float* dst = block_sums + ((int64_t)u * sp.nblocks + blk) * D + tid;
                const bool whole = rlo == blk * b && (rhi >= min((blk + 1) * b, N));
                if (whole) *dst = sum;
                else atomicAdd(dst, sum);
            }
        }
        cta_minmax_to_global(lo, hi, red, C::kThreads / 32, &mm[(int64_t)u * 6 + 4], &mm[(int64_t)u * 6 + 5]);
        __syncthreads();
        for (int j = tid; j < TILE; j += C::kThreads) {
            if (i0 + j < N) {
                a_raw[((int64_t)u * 3 + 2) * N + i0 + j] = outbuf[j];
                inv_norm[(int64_t)u * N + i0 + j] = invs[kHalo + j];
            }
        }
        __syncthreads();   // the tile, pp, invs and outbuf may be overwritten from here on
    }
}

// ============================================================================================
// stream_b
// ============================================================================================
template <typename T, int D, int TILE>
struct BCfg {
    using G = Geo<T, D>;
    static constexpr int kThreads = (TILE / kSeg) * G::kLanes;
    static constexpr size_t kTileBytes = (size_t)TILE * G::kRowBytes;
    static constexpr size_t kSmem = 2 * kTileBytes + 2 * TILE * 4 + 64 * 4 + 64;
    static_assert(kThreads % 32 == 0 && kThreads <= 1024, "bad CTA size");
};

template <typename T, int D, int TILE>
__global__ void __launch_bounds__(BCfg<T, D, TILE>::kThreads, 1)
stream_b_kernel(TensorView K, ScoreParams sp, int units, const float* __restrict__ mu_s, const float* __restrict__ mu_e,
                const float* __restrict__ inv_norm, const float* __restrict__ inv_s, const float* __restrict__ inv_e,
                float* __restrict__ a_raw, uint32_t* __restrict__ mm, int* status) {
    using C = BCfg<T, D, TILE>;
    using G = Geo<T, D>;
    constexpr int L = G::kLanes;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* tiles = smem;
    float* outbuf = reinterpret_cast<float*>(smem + 2 * C::kTileBytes);   // [2][TILE]
    float* red = outbuf + 2 * TILE;
    uint64_t* full = reinterpret_cast<uint64_t*>(red + 64);

    const int N = K.N;
    const int tiles_per_unit = (N + TILE - 1) / TILE;
    const long long total = (long long)units * tiles_per_unit;
    const int tid = threadIdx.x, grp = tid / L, l = tid % L;

    if (tid == 0) {
        mbar_init(&full[0], 1);
        mbar_init(&full[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto issue = [&](long long t, int buf) {
        const int u = (int)(t / tiles_per_unit);
        const int i0 = (int)(t - (long long)u * tiles_per_unit) * TILE;
        const int g = u / K.H, h = u % K.H;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(K.ptr) +
                                   ((int64_t)g * K.stride_g + (int64_t)h * K.stride_h) * sizeof(T) +
                                   (int64_t)i0 * G::kRowBytes;
        const uint32_t bytes = (uint32_t)(min(N, i0 + TILE) - i0) * G::kRowBytes;
        unsigned char* dst = tiles + (size_t)buf * C::kTileBytes;
        fence_async_smem();
        mbar_expect_tx(&full[buf], bytes);
        for (uint32_t off = 0; off < bytes; off += 16384u)
            bulk_load(dst + off, src + off, min(16384u, bytes - off), &full[buf]);
    };

    long long t = blockIdx.x;
    if (t < total && tid == 0) issue(t, 0);
    int it = 0;
    int cur_u = -1;
    F2 ms[4];
    float rs = 0.f;
    for (; t < total; t += gridDim.x, ++it) {
        const int buf = it & 1;
        const long long tn = t + gridDim.x;
        if (tn < total && tid == 0) issue(tn, buf ^ 1);
        const int u = (int)(t / tiles_per_unit);
        const int i0 = (int)(t - (long long)u * tiles_per_unit) * TILE;
        unsigned char* tile = tiles + (size_t)buf * C::kTileBytes;
        {
            const int rows = min(N, i0 + TILE) - i0;
            constexpr int cpr = G::kRowBytes / 16;
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            for (int c = rows * cpr + tid; c < TILE * cpr; c += C::kThreads) reinterpret_cast<uint4*>(tile)[c] = z;
        }
        if (u != cur_u) {
            cur_u = u;
            G::load_vec(mu_s + (int64_t)u * D, l, ms);
            rs = inv_s[u];
        }
        // anchors and reciprocal norms of this group's 8 tokens (loaded while the copy is in flight)
        const int gi0 = i0 + grp * kSeg;
        const int blk = min(gi0 / sp.block, sp.nblocks - 1);
        F2 me[4];
        G::load_vec(mu_e + ((int64_t)u * sp.nblocks + blk) * D, l, me);
        const float re = inv_e[(int64_t)u * sp.nblocks + blk];
        // after the reduction lane l finishes token o_mine of the group
        const int o_mine = (L == 16) ? (l >> 1) : l;
        const float inv_mine = (gi0 + o_mine < N) ? inv_norm[(int64_t)u * N + gi0 + o_mine] : 0.f;

        if (!mbar_wait(&full[buf], (uint32_t)((it >> 1) & 1), status, 402)) return;
        __syncthreads();

        float part[16];
#pragma unroll
        for (int o = 0; o < kSeg; ++o) {
            F2 kn[4];
            G::load_row(tile + (size_t)(grp * kSeg + o) * G::kRowBytes, l, kn);
            F2 ds = pack2(0.f, 0.f), de = pack2(0.f, 0.f);
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                ds = fma2(kn[p], ms[p], ds);
                de = fma2(kn[p], me[p], de);
            }
            part[2 * o] = hsum2(ds);
            part[2 * o + 1] = hsum2(de);
        }
        treduce<16, L>(part, l);
        float lo_s = INFINITY, hi_s = -INFINITY, lo_e = INFINITY, hi_e = -INFINITY;
        if (L == 16) {
            // lane l owns value l: token l/2, quantity l%2 (0: stable, 1: episodic)
            const float scale = (l & 1) ? re : rs;
            const float a = -(part[0] * inv_mine) * scale + 0.f;
            outbuf[(l & 1) * TILE + grp * kSeg + o_mine] = a;
            if (gi0 + o_mine < N) {
                if (l & 1) { lo_e = a; hi_e = a; }
                else { lo_s = a; hi_s = a; }
            }
        } else {
            const float a_s = -(part[0] * inv_mine) * rs + 0.f;
            const float a_e = -(part[1] * inv_mine) * re + 0.f;
            outbuf[grp * kSeg + o_mine] = a_s;
            outbuf[TILE + grp * kSeg + o_mine] = a_e;
            if (gi0 + o_mine < N) {
                lo_s = hi_s = a_s;
                lo_e = hi_e = a_e;
            }
        }
        cta_minmax_to_global(lo_s, hi_s, red, C::kThreads / 32, &mm[(int64_t)u * 6 + 0], &mm[(int64_t)u * 6 + 1]);
        __syncthreads();
        cta_minmax_to_global(lo_e, hi_e, red, C::kThreads / 32, &mm[(int64_t)u * 6 + 2], &mm[(int64_t)u * 6 + 3]);
        __syncthreads();
        for (int j = tid; j < 2 * TILE; j += C::kThreads) {
            const int k = j / TILE, jj = j - k * TILE;
            if (i0 + jj < N) a_raw[((int64_t)u * 3 + k) * N + i0 + jj] = outbuf[j];
        }
        __syncthreads();
    }
}

// reset of the per-head min/max keys (and, when blocks straddle tiles, of the block sums)
__global__ void stream_init_kernel(int units, uint32_t* mm, float* block_sums, long long n_sums) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < (long long)units * 6) mm[i] = (i & 1) ? 0u : 0xffffffffu;
    if (block_sums)
        for (long long j = i; j < n_sums; j += (long long)gridDim.x * blockDim.x) block_sums[j] = 0.f;
}

// tile sizes per (type, head dim)
template <typename T, int D> struct Tiles;
template <> struct Tiles<__nv_bfloat16, 128> { static constexpr int A = 256, B = 256; };
template <> struct Tiles<__nv_bfloat16, 64> { static constexpr int A = 512, B = 512; };
template <> struct Tiles<__half, 128> { static constexpr int A = 256, B = 256; };
template <> struct Tiles<__half, 64> { static constexpr int A = 512, B = 512; };
template <> struct Tiles<float, 128> { static constexpr int A = 128, B = 128; };
template <> struct Tiles<float, 64> { static constexpr int A = 256, B = 256; };

template <typename T, int D>
cudaError_t set_attrs() {
    cudaError_t e = cudaFuncSetAttribute(stream_a_kernel<T, D, Tiles<T, D>::A>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)ACfg<T, D, Tiles<T, D>::A>::kSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(stream_b_kernel<T, D, Tiles<T, D>::B>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)BCfg<T, D, Tiles<T, D>::B>::kSmem);
}
}  // namespace

cudaError_t configure_stream_kernels() {
    cudaError_t e;
    if ((e = set_attrs<__nv_bfloat16, 64>()) != cudaSuccess) return e;
    if ((e = set_attrs<__nv_bfloat16, 128>()) != cudaSuccess) return e;
    if ((e = set_attrs<__half, 64>()) != cudaSuccess) return e;
    if ((e = set_attrs<__half, 128>()) != cudaSuccess) return e;
    if ((e = set_attrs<float, 64>()) != cudaSuccess) return e;
    if ((e = set_attrs<float, 128>()) != cudaSuccess) return e;
    return cudaSuccess;
}

bool stream_path_supported(const ScoreParams& sp) { return sp.block % kSeg == 0; }

#define NKV_DISPATCH(dtype, d, CALL)                                         \
    do {                                                                     \
        if ((dtype) == NKV_BF16 && (d) == 64) { CALL(__nv_bfloat16, 64); }   \
        else if ((dtype) == NKV_BF16 && (d) == 128) { CALL(__nv_bfloat16, 128); } \
        else if ((dtype) == NKV_F16 && (d) == 64) { CALL(__half, 64); }      \
        else if ((dtype) == NKV_F16 && (d) == 128) { CALL(__half, 128); }    \
        else if ((dtype) == NKV_F32 && (d) == 64) { CALL(float, 64); }       \
        else if ((dtype) == NKV_F32 && (d) == 128) { CALL(float, 128); }     \
        else return cudaErrorInvalidValue;                                   \
    } while (0)

cudaError_t launch_stream_a(const TensorView& K, int dtype, int G, const ScoreParams& sp, float* block_sums,
                            float* inv_norm, float* a_raw, uint32_t* mm, int* status, int sm_count,
                            cudaStream_t stream, int64_t* launches) {
    const int units = G * K.H;
    int tile = 0;
#define CALL(T, D) tile = Tiles<T, D>::A
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    const bool straddle = (tile % sp.block) != 0;
    const long long n_sums = (long long)units * sp.nblocks * K.d;
    int init_grid = (units * 6 + 255) / 256;
    if (straddle && init_grid < 1024) init_grid = 1024;
    stream_init_kernel<<<init_grid, 256, 0, stream>>>(units, mm, straddle ? block_sums : nullptr, n_sums);
    ++*launches;
    const long long total = (long long)units * ((K.N + tile - 1) / tile);
    const unsigned grid = (unsigned)(total < sm_count ? total : sm_count);
#define CALL(T, D)                                                                                         \
    stream_a_kernel<T, D, Tiles<T, D>::A><<<grid, ACfg<T, D, Tiles<T, D>::A>::kThreads,                       \
                                            ACfg<T, D, Tiles<T, D>::A>::kSmem, stream>>>(                    \
        K, sp, units, block_sums, inv_norm, a_raw, mm, status)
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_stream_b(const TensorView& K, int dtype, int G, const ScoreParams& sp, const float* mu_s,
                            const float* mu_e, const float* inv_norm, const float* inv_s, const float* inv_e,
                            float* a_raw, uint32_t* mm, int* status, int sm_count, cudaStream_t stream,
                            int64_t* launches) {
    const int units = G * K.H;
    int tile = 0;
#define CALL(T, D) tile = Tiles<T, D>::B
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    const long long total = (long long)units * ((K.N + tile - 1) / tile);
    const unsigned grid = (unsigned)(total < sm_count ? total : sm_count);
#define CALL(T, D)                                                                                         \
    stream_b_kernel<T, D, Tiles<T, D>::B><<<grid, BCfg<T, D, Tiles<T, D>::B>::kThreads,                       \
                                            BCfg<T, D, Tiles<T, D>::B>::kSmem, stream>>>(                    \
        K, sp, units, mu_s, mu_e, inv_norm, inv_s, inv_e, a_raw, mm, status)
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
