// Fused key scan of the compression path (Sections 2.1-2.3): one persistent kernel that makes both
// passes over the keys, interleaved head by head so that the second pass finds the keys in L2.
//
//   pass A (needs no anchor)   1/||k_i||, sums of normalised keys per 8-row segment and per episodic
//                              block, the current-memory anomaly a_c(i) and its per-head min/max
//   finalize (once per head)   stable mean, block means, reciprocal norms of the anchors; done by the
//                              CTA that finishes the head's last pass-A tile
//   pass B (needs the anchors) a_s(i), a_e(i) and their per-head min/max
//
// Pass-A tiles are handed out in ticket order (strips of consecutive tiles of one head) to the pass-A
// threads of the persistent CTAs; a control warp per CTA takes the tickets, issues the bulk copies into
// two tile buffers (one is always in flight) and does the per-item bookkeeping, so the compute threads
// never wait for a global atomic.  Pass B runs beside it on its own warp group with its own ticket
// counter and buffer: it waits (bounded) for a head's anchors and therefore trails pass A by as little
// as the anchors allow, which is what keeps its reads in L2.  Pass A never waits for pass B, so the two
// cannot deadlock.
//
// Pass A: a row of d elements is split over 8 or 16 lanes (16-byte chunks), each lane group owns one
// 8-row segment; per-token partial sums are combined with a transposed shuffle reduction.  The
// sliding-window sum is a running sum over the 8 tokens of a group, seeded from exact segment sums, so
// no long prefix is ever differenced.
#include "nkv_common.cuh"

namespace nkv {

namespace {

constexpr int kHalo = kMaxWindow;
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr unsigned long long kWaitLimitNs = 2000000000ULL;   // every device-side wait gives up after 2 s

// control words (ints) in the workspace: [0..1] 64-bit ticket counter of pass A, [2..3] of pass B,
// [8 + u] tiles of head u finished by pass A, [8 + units + u] anchors of head u published
constexpr int kCtrlHeader = 8;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_keep() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_stream() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_global, uint32_t bytes, uint64_t* bar,
                                          uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_addr(dst_smem)),
        "l"(src_global), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
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
__device__ __forceinline__ unsigned long long now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for a bulk copy; gives up at once when the CTA has already recorded a failure.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = now_ns();
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 63u &&
            (*reinterpret_cast<const volatile int*>(abort_flag) != 0 || now_ns() - t0 > kWaitLimitNs))
            return false;
    }
    return false;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void bar_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
constexpr int kBarCompute = 1;   // the compute threads only
constexpr int kBarEnd = 2;       // compute threads + control warp, once per item

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

template <typename T> struct Pairs;
template <> struct Pairs<__nv_bfloat16> {
    static constexpr int kPairs = 4;   // per 16-byte chunk
    __device__ __forceinline__ static void unpack(const uint4& q, F2* p) {
        p[0] = pack2(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u));
        p[1] = pack2(__uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u));
        p[2] = pack2(__uint_as_float(q.z << 16), __uint_as_float(q.z & 0xffff0000u));
        p[3] = pack2(__uint_as_float(q.w << 16), __uint_as_float(q.w & 0xffff0000u));
    }
};
template <> struct Pairs<float> {
    static constexpr int kPairs = 2;
    __device__ __forceinline__ static void unpack(const uint4& q, F2* p) {
        p[0] = pack2(__uint_as_float(q.x), __uint_as_float(q.y));
        p[1] = pack2(__uint_as_float(q.z), __uint_as_float(q.w));
    }
};

// Geometry for element type T and head dimension D.  A row is split over kL lanes (16 when the row
// has at least 256 bytes, else 8); lane l owns the 16-byte chunks l, l + kL, ...
template <typename T, int D>
struct Geo {
    static constexpr int kRowBytes = D * (int)sizeof(T);
    static constexpr int kL = kRowBytes >= 256 ? 16 : 8;       // lanes per row
    static constexpr int kChunks = kRowBytes / (16 * kL);      // 16-byte chunks per lane
    static constexpr int kPerChunk = 16 / (int)sizeof(T);      // elements per chunk
    static constexpr int kCols = D / kL;                       // columns per lane
    static constexpr int kNP = kCols / 2;                      // packed pairs per lane
    static constexpr int kTile = 65536 / kRowBytes;            // rows per tile (64 KB of keys)
    static constexpr int kRows = kTile + kHalo;
    static constexpr int kSegs = kRows / kSeg;
    static constexpr int kThreads = kSegs * kL;                // compute threads: one lane group per staged segment
    static constexpr size_t kTileBytes = (size_t)kRows * kRowBytes;
    static_assert(kChunks >= 1 && kThreads % 32 == 0 && kThreads + 32 <= 1024, "bad geometry");

    __device__ __forceinline__ static int col0(int l, int j) { return (l + kL * j) * kPerChunk; }
    __device__ __forceinline__ static void load_row(const unsigned char* row, int l, F2* p) {
#pragma unroll
        for (int j = 0; j < kChunks; ++j) {
            const uint4 q = *reinterpret_cast<const uint4*>(row + (l + kL * j) * 16);
            Pairs<T>::unpack(q, p + j * Pairs<T>::kPairs);
        }
    }
    // the lane's columns of an fp32 vector laid out by column
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

// Transposed reduction of V per-lane partial values over the L lanes of a group (L, V powers of two).
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

struct FusedArgs {
    TensorView K;
    ScoreParams sp;
    int units, lag, hints, strip;   // strip: consecutive tiles of one pass handed out per ticket
    float* block_sums;   // [units, nb, d]: block sums, turned into block means (mu_e) by finalize
    float* mu_s;         // [units, d]
    float* inv_s;        // [units]
    float* inv_e;        // [units, nb]
    float* inv_norm;     // [units, N]
    float* a_raw;        // [units, 3, N]
    uint32_t* mm;        // [units, 6] ordered keys: min/max of a_s, a_e, a_c
    int* ctrl;           // control words, see kCtrlHeader
    int* status;
};

// item descriptor written by the control warp: kind 0 = pass A, 1 = pass B, 2 = no more work
struct Item {
    int kind, unit, tile, pad;
};

// sum over staged segments [s0, s1) of the per-segment sums, from inclusive prefixes within 64-row chunks
template <typename T, int D>
__device__ __forceinline__ void range_sum(const float* pp, int l, int s0, int s1, F2* out) {
    using G = Geo<T, D>;
#pragma unroll
    for (int p = 0; p < G::kNP; ++p) out[p] = pack2(0.f, 0.f);
    if (s1 <= s0) return;
    for (int c = s0 >> 3; c <= (s1 - 1) >> 3; ++c) {
        const int lo = max(s0, c * 8), hi = min(s1, c * 8 + 8);
        F2 a[G::kNP];
        G::load_vec(pp + (size_t)(hi - 1) * D, l, a);
#pragma unroll
        for (int p = 0; p < G::kNP; ++p) out[p] = add2(out[p], a[p]);
        if (lo > c * 8) {
            G::load_vec(pp + (size_t)(lo - 1) * D, l, a);
            const F2 m1 = pack2(-1.f, -1.f);
#pragma unroll
            for (int p = 0; p < G::kNP; ++p) out[p] = fma2(a[p], m1, out[p]);
        }
    }
}

// ---------------------------------------------------------------------------- pass A on one tile
template <typename T, int D>
__device__ __forceinline__ void pass_a(const FusedArgs& A, int u, int tile_idx, unsigned char* tile, float* pp,
                                       float* invs, uint32_t* mmk, uint64_t* full, uint32_t parity, int* abort_flag) {
    using G = Geo<T, D>;
    constexpr int NP = G::kNP;
    constexpr int L = G::kL;
    const int N = A.K.N, W = A.sp.window;
    const int tid = threadIdx.x, grp = tid / L, l = tid % L;
    const int i0 = tile_idx * G::kTile;

    // rows outside [0, N) are not copied: zero them (disjoint from the bytes in flight)
    const int r0 = max(0, i0 - kHalo), r1 = min(N, i0 + G::kTile);
    const bool fill = (r0 != i0 - kHalo) || (r1 != i0 + G::kTile);
    if (fill) {
        const int head_rows = r0 - (i0 - kHalo), tail_row0 = r1 - (i0 - kHalo);
        constexpr int cpr = G::kRowBytes / 16;
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
        for (int c = tid; c < head_rows * cpr; c += G::kThreads) reinterpret_cast<uint4*>(tile)[c] = z;
        for (int c = tail_row0 * cpr + tid; c < G::kRows * cpr; c += G::kThreads) reinterpret_cast<uint4*>(tile)[c] = z;
    }
    if (!mbar_wait(full, parity, abort_flag)) {
        set_status(A.status, NKV_ERR_TIMEOUT, 501);
        *abort_flag = 1;
    }
    if (fill) bar_sync(kBarCompute, G::kThreads);

    // ---- S1: reciprocal norms and the sum of normalised keys of every staged 8-row segment
    {
        F2 acc[NP];
#pragma unroll
        for (int p = 0; p < NP; ++p) acc[p] = pack2(0.f, 0.f);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            F2 x[4][NP];
            float n2[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                G::load_row(tile + (size_t)(grp * kSeg + half * 4 + r) * G::kRowBytes, l, x[r]);
                F2 s = pack2(0.f, 0.f);
#pragma unroll
                for (int p = 0; p < NP; ++p) s = fma2(x[r][p], x[r][p], s);
                n2[r] = hsum2(s);
            }
            treduce<4, L>(n2, l);   // lane l: squared norm of row l / (L/4) of this half
            const float inv = 1.0f / fmaxf(sqrtf(n2[0]), kEps);
            if ((l & (L / 4 - 1)) == 0) {
                const int sr = grp * kSeg + half * 4 + l / (L / 4);
                invs[sr] = inv;
                const int gi = i0 - kHalo + sr;
                if (sr >= kHalo && gi < N) A.inv_norm[(int64_t)u * N + gi] = inv;
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float ir = __shfl_sync(0xffffffffu, inv, r * (L / 4), L);
                const F2 ir2 = pack2(ir, ir);
#pragma unroll
                for (int p = 0; p < NP; ++p) acc[p] = fma2(x[r][p], ir2, acc[p]);
            }
        }
        G::store_vec(pp + (size_t)grp * D, l, acc);
    }
    bar_sync(kBarCompute, G::kThreads);
    // ---- S1b: inclusive prefix of the segment sums inside every 64-row chunk (one column per task)
    for (int task = tid; task < (G::kRows / 64) * D; task += G::kThreads) {
        const int c64 = task / D, col = task - c64 * D;
        float run = 0.f;
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            float* q = pp + (size_t)(c64 * 8 + p) * D + col;
            run += *q;
            *q = run;
        }
    }
    bar_sync(kBarCompute, G::kThreads);

    // ---- S2: sliding-window anomaly of the tile's tokens
    constexpr int kHaloSegs = kHalo / kSeg;
    if (grp >= kHaloSegs) {
        const int s = grp;
        F2 Sw[NP];
        range_sum<T, D>(pp, l, s - W / kSeg, s, Sw);
        for (int sr = s * kSeg - W; sr < (s - W / kSeg) * kSeg; ++sr) {   // the W % 8 oldest rows
            F2 x[NP];
            G::load_row(tile + (size_t)sr * G::kRowBytes, l, x);
            const float iv = invs[sr];
            const F2 iv2 = pack2(iv, iv);
#pragma unroll
            for (int p = 0; p < NP; ++p) Sw[p] = fma2(x[p], iv2, Sw[p]);
        }
        float part[16];
#pragma unroll
        for (int o = 0; o < kSeg; ++o) {
            const int sr = s * kSeg + o;
            F2 kn[NP], ko[NP];
            G::load_row(tile + (size_t)sr * G::kRowBytes, l, kn);
            G::load_row(tile + (size_t)(sr - W) * G::kRowBytes, l, ko);
            const float in = invs[sr], io = -invs[sr - W];
            const F2 in2 = pack2(in, in), io2 = pack2(io, io);
            F2 dc = pack2(0.f, 0.f), nc = pack2(0.f, 0.f);
#pragma unroll
            for (int p = 0; p < NP; ++p) {
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
        // L == 8: lane l owns (dc, nc) of token l.  L == 16: lane l owns value l = (token l/2, quantity l%2).
        float dcv, ncv;
        int o;
        bool writer;
        if (L == 16) {
            const float other = __shfl_xor_sync(0xffffffffu, part[0], 1);
            dcv = (l & 1) ? other : part[0];
            ncv = (l & 1) ? part[0] : other;
            o = l >> 1;
            writer = (l & 1) == 0;
        } else {
            dcv = part[0];
            ncv = part[1];
            o = l;
            writer = true;
        }
        const int j = (s - kHaloSegs) * kSeg + o;
        const float a_c = -(dcv * invs[s * kSeg + o]) / fmaxf(sqrtf(ncv), kEps) + 0.f;
        float lo = INFINITY, hi = -INFINITY;
        if (writer && i0 + j < N) {
            A.a_raw[((int64_t)u * 3 + 2) * N + i0 + j] = a_c;
            lo = hi = a_c;
        }
        lo = warp_min(lo);
        hi = warp_max(hi);
        if ((tid & 31) == 0 && lo <= hi) {
            atomicMin(&mmk[4], ord_key(lo));
            atomicMax(&mmk[5], ord_key(hi));
        }
    }
    // ---- sums of normalised keys of the episodic blocks inside this tile (one column per thread);
    //      the tile size is a multiple of the block size, so every block is written by one tile
    if (tid < D) {
        const int b = A.sp.block;
        const int row_end = min(N, i0 + G::kTile);
        for (int blk = i0 / b; blk * b < row_end; ++blk) {
            const int rlo = blk * b, rhi = min((blk + 1) * b, ((N + 7) / 8) * 8);
            const int s0 = kHaloSegs + (rlo - i0) / kSeg, s1 = kHaloSegs + (rhi - i0 + kSeg - 1) / kSeg;
            float sum = 0.f;
            for (int c = s0 >> 3; c <= (s1 - 1) >> 3; ++c) {
                const int a = max(s0, c * 8), e = min(s1, c * 8 + 8);
                sum += pp[(size_t)(e - 1) * D + tid];
                if (a > c * 8) sum -= pp[(size_t)(a - 1) * D + tid];
            }
            A.block_sums[((int64_t)u * A.sp.nblocks + blk) * D + tid] = sum;
        }
        __threadfence();   // the block sums must be visible before this tile is counted as finished
    }
}

// ---------------------------------------------------------------------------- pass B (own warp group)
// Four warps beside the pass-A threads take pass-B tiles from their own ticket counter, wait (bounded)
// until the tile's head has published its anchors, and stream the tile through a private buffer in
// sub-tiles.  Pass A never waits for pass B, so the two cannot deadlock; pass B simply trails pass A as
// closely as the anchors allow, which is what keeps its reads in L2.
//
// bf16 keys with blocks of 16k rows: the two dots of a key against mu_s and mu_e are a skinny matrix
// product [16 keys x d] x [d x 8] on the tensor cores.  The fp32 anchors are split three ways into bf16
// (hi + mid + lo carries all 24 mantissa bits), products of bf16 numbers are exact in fp32 and the
// accumulation is fp32.  Columns: 0..2 = mu_s hi/mid/lo, 3..5 = mu_e hi/mid/lo, 6..7 = 0.  The
// contraction index may be visited in any order, so lane (g, t) takes the 16-byte chunks t, t+4, ... of
// rows g and g+8 straight from the staged rows and the right-hand side uses the same order.
// Other cases (fp32 keys, odd block sizes) use packed FMAs with the anchors read from L2.
constexpr int kBThreads = 128;
constexpr int kBarB = 3;

template <typename T, int D>
struct BGeo {
    using G = Geo<T, D>;
    static constexpr int kBytes = G::kRowBytes >= 512 ? 16384 : 32768;   // private buffer of the group
    static constexpr int kRows = kBytes / G::kRowBytes;                  // rows per sub-tile
    static constexpr int kAnchorBytes = sizeof(T) == 2 ? 4 * 8 * D * 2 : 0;   // split right-hand sides [4][8][D] bf16
};

template <typename T, int D>
__device__ __forceinline__ void pass_b_group(const FusedArgs& A, unsigned char* tileB, __nv_bfloat16* rhs, float* bsc,
                                             int* bslot, uint64_t* mbarB, int* abort_flag) {
    using G = Geo<T, D>;
    using B = BGeo<T, D>;
    constexpr int NP = G::kNP, L = G::kL;
    constexpr int kHalfRows = B::kRows / 2;                       // rows per sub-tile (one half of the buffer)
    constexpr int kHalfBytes = B::kBytes / 2;
    const int N = A.K.N, b = A.sp.block, nb = A.sp.nblocks;
    const int bt = threadIdx.x - (G::kThreads + 32), warp = bt >> 5, lane = bt & 31;
    const int tiles_per_unit = (N + G::kTile - 1) / G::kTile;
    const long long total = (long long)A.units * tiles_per_unit;
    unsigned long long* ticket = reinterpret_cast<unsigned long long*>(A.ctrl + 2);
    const uint64_t policy = A.hints ? l2_policy_stream() : l2_policy_normal();
    // a sub-tile overlaps at most ceil(kHalfRows / b) + 1 blocks; the staged right-hand sides hold four
    const bool mma_path = sizeof(T) == 2 && b % 16 == 0 && (kHalfRows + b - 1) / b + 1 <= 4;
    uint32_t used[2] = {0u, 0u};   // copies awaited so far per half (mbarrier parity)
    unsigned long long next_t = 0;
    if (bt == 0) next_t = atomicAdd(ticket, 1ULL);   // always one ticket ahead
    int staged_u = -1, staged_blk0 = -1, staged_n = 0;

    for (;;) {
        if (bt == 0) {
            int u = -1, tile = 0;
            const unsigned long long t = next_t;
            if ((long long)t < total && *reinterpret_cast<volatile int*>(abort_flag) == 0) {
                next_t = atomicAdd(ticket, 1ULL);
                u = (int)(t / (unsigned long long)tiles_per_unit);
                tile = (int)(t - (unsigned long long)u * tiles_per_unit);
                // wait (bounded) until the head's anchors have been published
                const int* ready = A.ctrl + kCtrlHeader + A.units + u;
                bool ok = ld_acquire(ready) != 0;
                if (!ok) {
                    const unsigned long long t0 = now_ns();
                    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
                        if (ld_acquire(ready) != 0) {
                            ok = true;
                            break;
                        }
                        __nanosleep(256);
                        if ((spin & 15u) == 15u &&
                            (*reinterpret_cast<volatile int*>(abort_flag) != 0 || now_ns() - t0 > kWaitLimitNs))
                            break;
                    }
                }
                if (!ok) {
                    set_status(A.status, NKV_ERR_TIMEOUT, 502);
                    *abort_flag = 1;
                    u = -1;
                }
            }
            bslot[0] = u;
            bslot[1] = tile;
        }
        bar_sync(kBarB, kBThreads);
        const int u = bslot[0], tile_idx = bslot[1];
        if (u < 0) break;
        const int g = u / A.K.H, h = u % A.K.H;
        const unsigned char* base = reinterpret_cast<const unsigned char*>(A.K.ptr) +
                                    ((int64_t)g * A.K.stride_g + (int64_t)h * A.K.stride_h) * (int64_t)sizeof(T);
        float lo_s = INFINITY, hi_s = -INFINITY, lo_e = INFINITY, hi_e = -INFINITY;
        const float rs = __ldcg(A.inv_s + u);
        const int row_begin = tile_idx * G::kTile, row_end = min(N, (tile_idx + 1) * G::kTile);
        auto issue = [&](int r0, int half) {   // thread 0 of the group
            const uint32_t bytes = (uint32_t)(min(row_end, r0 + kHalfRows) - r0) * G::kRowBytes;
            fence_async_smem();
            mbar_expect_tx(&mbarB[half], bytes);
            bulk_load(tileB + (size_t)half * kHalfBytes, base + (int64_t)r0 * G::kRowBytes, bytes, &mbarB[half], policy);
        };
        if (bt == 0) issue(row_begin, 0);

        int sub = 0;
        for (int r0 = row_begin; r0 < row_end; r0 += kHalfRows, ++sub) {
            const int half = sub & 1;
            const int rows = min(row_end, r0 + kHalfRows) - r0;
            // the other half was released by the barrier that ended the previous sub-tile
            if (bt == 0 && r0 + kHalfRows < row_end) issue(r0 + kHalfRows, half ^ 1);
            const unsigned char* buf = tileB + (size_t)half * kHalfBytes;
            const int blk0 = r0 / b;
            if (mma_path) {
                if constexpr (sizeof(T) == 2) {
                    constexpr int kCh = D / 32;
                    const int gq = lane >> 2, t = lane & 3;
                    const int row_in_block = gq + ((t & 2) ? 8 : 0);
                    // split right-hand sides of the sub-tile's blocks (restaged only when they change)
                    const int nblk = min(nb - 1, (r0 + rows - 1) / b) - blk0 + 1;
                    const bool restage = u != staged_u || blk0 != staged_blk0 || nblk > staged_n;
                    if (restage) {
                        if (bt < D) {
                            const float mu = __ldcg(A.mu_s + (int64_t)u * D + bt);
                            for (int q = 0; q < nblk; ++q) {
                                __nv_bfloat16* r = rhs + (size_t)q * 8 * D + bt;
                                split3_bf16(mu, r, D);
                                split3_bf16(__ldcg(A.block_sums + ((int64_t)u * nb + blk0 + q) * D + bt), r + 3 * D, D);
                                r[6 * D] = __float2bfloat16_rn(0.f);
                                r[7 * D] = __float2bfloat16_rn(0.f);
                            }
                            if (bt < nblk) bsc[bt] = __ldcg(A.inv_e + (int64_t)u * nb + blk0 + bt);
                        }
                        staged_u = u;
                        staged_blk0 = blk0;
                        staged_n = nblk;
                    }
                    // reciprocal norm of the key this lane finishes, fetched before the copy is awaited
                    constexpr int kIters = (kHalfRows / 16 + kBThreads / 32 - 1) / (kBThreads / 32);
                    float inv_pre[kIters];
#pragma unroll
                    for (int it = 0; it < kIters; ++it) {
                        const int gi = r0 + (warp + it * (kBThreads / 32)) * 16 + row_in_block;
                        inv_pre[it] = (warp + it * (kBThreads / 32)) * 16 < rows && gi < N
                                          ? __ldcg(A.inv_norm + (int64_t)u * N + gi)
                                          : 0.f;
                    }
                    if (restage) bar_sync(kBarB, kBThreads);   // right-hand sides visible (uniform condition)
                    if (!mbar_wait(&mbarB[half], used[half] & 1u, abort_flag)) {
                        set_status(A.status, NKV_ERR_TIMEOUT, 503);
                        *abort_flag = 1;
                    }
                    ++used[half];
#pragma unroll
                    for (int it = 0; it < kIters; ++it) {
                        const int rr = (warp + it * (kBThreads / 32)) * 16;
                        if (rr >= rows) break;
                        const int q = min((r0 + rr) / b, nb - 1) - blk0;
                        const float re = bsc[q];
                        const int gi = r0 + rr + row_in_block;
                        float c[4] = {0.f, 0.f, 0.f, 0.f};
                        const unsigned char* row_lo = buf + (size_t)(rr + gq) * G::kRowBytes;
                        const unsigned char* row_hi = row_lo + 8 * G::kRowBytes;
                        const __nv_bfloat16* rq = rhs + ((size_t)q * 8 + gq) * D;
#pragma unroll
                        for (int j = 0; j < kCh; ++j) {
                            const uint4 x = *reinterpret_cast<const uint4*>(row_lo + (t + 4 * j) * 16);
                            const uint4 y = *reinterpret_cast<const uint4*>(row_hi + (t + 4 * j) * 16);
                            const uint4 w = *reinterpret_cast<const uint4*>(rq + (t + 4 * j) * 8);
                            const uint32_t a_first[4] = {x.x, y.x, x.y, y.y};
                            const uint32_t a_second[4] = {x.z, y.z, x.w, y.w};
                            mma_bf16_16816(c, a_first, w.x, w.y);
                            mma_bf16_16816(c, a_second, w.z, w.w);
                        }
                        // columns 0,1 (t=0) and 2 (t=1, c[0]) belong to mu_s; 3 (t=1, c[1]) and 4,5 (t=2) to mu_e
                        float xs_lo = t == 0 ? c[0] + c[1] : (t == 1 ? c[0] : 0.f);
                        float xe_lo = t == 1 ? c[1] : (t == 2 ? c[0] + c[1] : 0.f);
                        float xs_hi = t == 0 ? c[2] + c[3] : (t == 1 ? c[2] : 0.f);
                        float xe_hi = t == 1 ? c[3] : (t == 2 ? c[2] + c[3] : 0.f);
#pragma unroll
                        for (int o = 1; o <= 2; o <<= 1) {
                            xs_lo += __shfl_xor_sync(0xffffffffu, xs_lo, o);
                            xe_lo += __shfl_xor_sync(0xffffffffu, xe_lo, o);
                            xs_hi += __shfl_xor_sync(0xffffffffu, xs_hi, o);
                            xe_hi += __shfl_xor_sync(0xffffffffu, xe_hi, o);
                        }
                        // each lane finishes one of its quad's four results: t=0: a_s(row g), t=1: a_e(row g),
                        // t=2: a_s(row g+8), t=3: a_e(row g+8)
                        const float dot = t == 0 ? xs_lo : (t == 1 ? xe_lo : (t == 2 ? xs_hi : xe_hi));
                        const float a = -(dot * inv_pre[it]) * ((t & 1) ? re : rs) + 0.f;
                        if (gi < N) {
                            A.a_raw[((int64_t)u * 3 + (t & 1)) * N + gi] = a;
                            if (t & 1) {
                                lo_e = fminf(lo_e, a);
                                hi_e = fmaxf(hi_e, a);
                            } else {
                                lo_s = fminf(lo_s, a);
                                hi_s = fmaxf(hi_s, a);
                            }
                        }
                    }
                }
            } else {
                // packed FMAs: an L-lane group walks 8 rows; whole warps run every iteration (groups past
                // the end compute on stale rows and write nothing); anchors come from L2
                if (!mbar_wait(&mbarB[half], used[half] & 1u, abort_flag)) {
                    set_status(A.status, NKV_ERR_TIMEOUT, 503);
                    *abort_flag = 1;
                }
                ++used[half];
                const int grp = bt / L, l = bt % L;
                F2 ms[NP];
                G::load_vec(A.mu_s + (int64_t)u * D, l, ms);
                for (int seg0 = 0; seg0 * kSeg < rows; seg0 += kBThreads / L) {
                    const int seg = seg0 + grp;
                    const int gi0 = r0 + seg * kSeg;
                    const int blk = min(gi0 / b, nb - 1);
                    F2 me[NP];
                    G::load_vec(A.block_sums + ((int64_t)u * nb + blk) * D, l, me);
                    const float re = __ldcg(A.inv_e + (int64_t)u * nb + blk);
                    const int o_mine = L == 16 ? (l >> 1) : l;
                    const float inv_mine = gi0 + o_mine < N ? __ldcg(A.inv_norm + (int64_t)u * N + gi0 + o_mine) : 0.f;
                    float part[16];
                    const int seg_c = min(seg, kHalfRows / kSeg - 1);   // stay inside the buffer
#pragma unroll
                    for (int o = 0; o < kSeg; ++o) {
                        F2 kn[NP];
                        G::load_row(buf + (size_t)(seg_c * kSeg + o) * G::kRowBytes, l, kn);
                        F2 ds = pack2(0.f, 0.f), de = pack2(0.f, 0.f);
#pragma unroll
                        for (int p = 0; p < NP; ++p) {
                            ds = fma2(kn[p], ms[p], ds);
                            de = fma2(kn[p], me[p], de);
                        }
                        part[2 * o] = hsum2(ds);
                        part[2 * o + 1] = hsum2(de);
                    }
                    treduce<16, L>(part, l);
                    const bool live = seg * kSeg < rows;
                    if (L == 16) {
                        const int o = l >> 1;
                        const float a = -(part[0] * inv_mine) * ((l & 1) ? re : rs) + 0.f;
                        if (live && gi0 + o < N) {
                            A.a_raw[((int64_t)u * 3 + (l & 1)) * N + gi0 + o] = a;
                            if (l & 1) {
                                lo_e = fminf(lo_e, a);
                                hi_e = fmaxf(hi_e, a);
                            } else {
                                lo_s = fminf(lo_s, a);
                                hi_s = fmaxf(hi_s, a);
                            }
                        }
                    } else {
                        const float a_s = -(part[0] * inv_mine) * rs + 0.f;
                        const float a_e = -(part[1] * inv_mine) * re + 0.f;
                        if (live && gi0 + l < N) {
                            A.a_raw[((int64_t)u * 3 + 0) * N + gi0 + l] = a_s;
                            A.a_raw[((int64_t)u * 3 + 1) * N + gi0 + l] = a_e;
                            lo_s = fminf(lo_s, a_s);
                            hi_s = fmaxf(hi_s, a_s);
                            lo_e = fminf(lo_e, a_e);
                            hi_e = fmaxf(hi_e, a_e);
                        }
                    }
                }
            }
            bar_sync(kBarB, kBThreads);   // this half (and, next time they change, the right-hand sides) is free
        }
        lo_s = warp_min(lo_s);
        hi_s = warp_max(hi_s);
        lo_e = warp_min(lo_e);
        hi_e = warp_max(hi_e);
        if (lane == 0) {
            if (lo_s <= hi_s) {
                atomicMin(&A.mm[(int64_t)u * 6 + 0], ord_key(lo_s));
                atomicMax(&A.mm[(int64_t)u * 6 + 1], ord_key(hi_s));
            }
            if (lo_e <= hi_e) {
                atomicMin(&A.mm[(int64_t)u * 6 + 2], ord_key(lo_e));
                atomicMax(&A.mm[(int64_t)u * 6 + 3], ord_key(hi_e));
            }
        }
    }
}

// ---------------------------------------------------------------------------- anchors of one head
// Block sums -> block means (in place), stable mean (compensated sums), reciprocal anchor norms.
// Called by all compute threads of the CTA that finished the head's last pass-A tile.
template <typename T, int D>
__device__ __forceinline__ void finalize_head(const FusedArgs& A, int u, float* pp, float* invs) {
    using G = Geo<T, D>;
    constexpr int Q = D / 4;                      // column quads
    constexpr int kParts = (G::kThreads / Q) < (G::kSegs / 2) ? (G::kThreads / Q) : (G::kSegs / 2);   // slices of the blocks
    static_assert(2 * kParts <= G::kSegs && D <= G::kRows, "finalize scratch does not fit");
    const int N = A.K.N, b = A.sp.block, nb = A.sp.nblocks;
    const int tid = threadIdx.x;
    const int part = tid / Q, q4 = (tid - part * Q) * 4;
    float* bs = A.block_sums + (int64_t)u * nb * D;
    if (part < kParts) {
        const int per = (nb + kParts - 1) / kParts;
        const int t0 = part * per, t1 = min(nb, t0 + per);
        float sum[4] = {0.f, 0.f, 0.f, 0.f}, comp[4] = {0.f, 0.f, 0.f, 0.f};
        for (int t = t0; t < t1; t += 4) {
            float4 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)   // four independent loads in flight
                v[j] = (t + j < t1) ? __ldcg(reinterpret_cast<const float4*>(bs + (size_t)(t + j) * D + q4))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (t + j < t1) {
                    const float s[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
                    const float cnt = (float)(min(N, (t + j + 1) * b) - (t + j) * b);
                    float m[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float y = s[e] - comp[e];
                        const float z = sum[e] + y;
                        comp[e] = (z - sum[e]) - y;
                        sum[e] = z;
                        m[e] = s[e] / cnt;
                    }
                    *reinterpret_cast<float4*>(bs + (size_t)(t + j) * D + q4) = make_float4(m[0], m[1], m[2], m[3]);
                }
            }
        }
        *reinterpret_cast<float4*>(pp + (size_t)(2 * part) * D + q4) = make_float4(sum[0], sum[1], sum[2], sum[3]);
        *reinterpret_cast<float4*>(pp + (size_t)(2 * part + 1) * D + q4) = make_float4(comp[0], comp[1], comp[2], comp[3]);
    }
    bar_sync(kBarCompute, G::kThreads);
    if (tid < D) {
        float sum = 0.f, comp = 0.f;
        for (int p = 0; p < kParts; ++p) {
            // add the partial sum, then its pending correction, both compensated
            const float v[2] = {pp[(2 * p) * D + tid], -pp[(2 * p + 1) * D + tid]};
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const float y = v[k] - comp;
                const float z = sum + y;
                comp = (z - sum) - y;
                sum = z;
            }
        }
        const float m = sum / (float)N;
        A.mu_s[(int64_t)u * D + tid] = m;
        invs[tid] = m;
    }
    bar_sync(kBarCompute, G::kThreads);
    // reciprocal norms: one warp per vector (vector -1 is the stable mean)
    const int w = tid >> 5, lane = tid & 31;
    for (int t = w - 1; t < nb; t += G::kThreads / 32) {
        const float* v = (t < 0) ? invs : bs + (size_t)t * D;
        float ss = 0.f;
        for (int cc = lane; cc < D; cc += 32) ss = fmaf(v[cc], v[cc], ss);
        ss = warp_sum(ss);
        if (lane == 0) {
            const float inv = 1.0f / fmaxf(sqrtf(ss), kEps);
            if (t < 0) A.inv_s[u] = inv;
            else A.inv_e[(int64_t)u * nb + t] = inv;
        }
    }
    __threadfence();
    bar_sync(kBarCompute, G::kThreads);
    if (tid == 0) st_release(A.ctrl + kCtrlHeader + A.units + u, 1);
}

// ---------------------------------------------------------------------------- the persistent kernel
// Thread roles: [0, kThreads) pass A; one control warp (tickets, copies and bookkeeping of pass A);
// kBThreads threads of pass B.  Small shared-memory state after the big arrays (byte offsets in `small`):
//   0  item[2]      descriptors of the pass-A items in the two tile buffers
//   32 mmk[2][6]    per-item ordered min/max keys (double buffered like the tiles; slots 4, 5 are used)
//   80 fin[2]       head whose anchors this CTA owes after item k (or -1), written by the control warp
//   88 abort_flag   a bounded wait ran out somewhere in this CTA
//   96 full[2]      mbarriers of the two pass-A tile buffers
//   112 mbarB[2]    mbarriers of the two halves of the pass-B buffer
//   128 bslot[2]    head and tile of the pass-B group's current ticket
//   136 bsc[8]      1/||mu_e|| of the blocks of the current pass-B sub-tile
template <typename T, int D>
struct Ctl {
    using G = Geo<T, D>;
    const FusedArgs& A;
    unsigned char* tiles;
    Item* item;
    uint64_t* full;
    int* abort_flag;
    int tiles_per_unit, strips;
    long long total;   // strip tickets of pass A
    uint64_t policy;

    __device__ __forceinline__ unsigned long long take_ticket() {
        return atomicAdd(reinterpret_cast<unsigned long long*>(A.ctrl), 1ULL);
    }
    // ticket number -> first tile of its strip (kind 2 when the tickets are used up)
    __device__ __forceinline__ Item decode(unsigned long long t) const {
        Item it;
        it.kind = 2;
        it.unit = it.tile = it.pad = 0;
        if ((long long)t >= total || *reinterpret_cast<volatile int*>(abort_flag) != 0) return it;
        it.kind = 0;
        it.unit = (int)(t / (unsigned long long)strips);
        it.tile = (int)(t - (unsigned long long)it.unit * strips) * A.strip;
        return it;
    }
    // tiles that follow `it` in its strip
    __device__ __forceinline__ int rest_of_strip(const Item& it) const {
        return it.kind == 2 ? 0 : min(A.strip, tiles_per_unit - it.tile) - 1;
    }
    // publish `it` in `slot` and start its copy (tile rows plus the 64 rows in front of them)
    __device__ __forceinline__ void issue(int slot, Item it) {
        item[slot] = it;
        if (it.kind == 2) return;
        const int N = A.K.N;
        const int g = it.unit / A.K.H, h = it.unit % A.K.H;
        const unsigned char* base = reinterpret_cast<const unsigned char*>(A.K.ptr) +
                                    ((int64_t)g * A.K.stride_g + (int64_t)h * A.K.stride_h) * (int64_t)sizeof(T);
        const int i0 = it.tile * G::kTile;
        const int r0 = max(0, i0 - kHalo), r1 = min(N, i0 + G::kTile);
        unsigned char* dst = tiles + (size_t)slot * G::kTileBytes + (size_t)(r0 - (i0 - kHalo)) * G::kRowBytes;
        const uint32_t bytes = (uint32_t)(r1 - r0) * G::kRowBytes;
        const unsigned char* src = base + (int64_t)r0 * G::kRowBytes;
        fence_async_smem();
        mbar_expect_tx(&full[slot], bytes);
        for (uint32_t off = 0; off < bytes; off += 32768u)
            bulk_load(dst + off, src + off, min(32768u, bytes - off), &full[slot], policy);
    }
};

template <typename T, int D>
constexpr size_t fused_smem_bytes() {
    using G = Geo<T, D>;
    return 2 * G::kTileBytes + BGeo<T, D>::kBytes + (size_t)G::kSegs * D * 4 + (size_t)G::kRows * 4 +
           BGeo<T, D>::kAnchorBytes + 256;
}

template <typename T, int D>
__global__ void __launch_bounds__(Geo<T, D>::kThreads + 32 + kBThreads, 1) fused_scan_kernel(FusedArgs A) {
    using G = Geo<T, D>;
    using B = BGeo<T, D>;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* tiles = smem;
    unsigned char* tileB = smem + 2 * G::kTileBytes;
    float* pp = reinterpret_cast<float*>(tileB + B::kBytes);                 // [kSegs][D]
    float* invs = pp + G::kSegs * D;                                         // [kRows]
    __nv_bfloat16* rhs = reinterpret_cast<__nv_bfloat16*>(invs + G::kRows);
    unsigned char* small = reinterpret_cast<unsigned char*>(rhs) + B::kAnchorBytes;
    Item* item = reinterpret_cast<Item*>(small);
    uint32_t* mmk = reinterpret_cast<uint32_t*>(small + 32);
    int* fin = reinterpret_cast<int*>(small + 80);
    int* abort_flag = reinterpret_cast<int*>(small + 88);
    uint64_t* full = reinterpret_cast<uint64_t*>(small + 96);
    uint64_t* mbarB = reinterpret_cast<uint64_t*>(small + 112);
    int* bslot = reinterpret_cast<int*>(small + 128);
    float* bsc = reinterpret_cast<float*>(small + 136);

    const int N = A.K.N;
    const int tiles_per_unit = (N + G::kTile - 1) / G::kTile;
    const int tid = threadIdx.x;
    constexpr int kAll = G::kThreads + 32;   // pass-A threads and the control warp share the item barrier

    if (tid == 0) {
        mbar_init(&full[0], 1);
        mbar_init(&full[1], 1);
        mbar_init(&mbarB[0], 1);
        mbar_init(&mbarB[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < 12; ++i) mmk[i] = (i & 1) ? 0u : 0xffffffffu;
        fin[0] = fin[1] = -1;
        *abort_flag = 0;
    }
    __syncthreads();

    if (tid >= kAll) {
        pass_b_group<T, D>(A, tileB, rhs, bsc, bslot, mbarB, abort_flag);
        return;
    }

    if (tid >= G::kThreads) {
        // ------------------------------------------------------------------ control warp
        // All 32 lanes run the loop together (the per-item barrier is warp-aligned); lane 0 works.
        const int lane = tid - G::kThreads;
        const int strips = (tiles_per_unit + A.strip - 1) / A.strip;
        Ctl<T, D> C{A, tiles, item, full, abort_flag, tiles_per_unit, strips, (long long)A.units * strips,
                    A.hints ? l2_policy_keep() : l2_policy_normal()};
        Item nxt;   // the next item to issue (lane 0), fetched ahead of time
        nxt.kind = 2;
        nxt.unit = nxt.tile = nxt.pad = 0;
        int left = 0;   // tiles that follow `nxt` in its strip
        auto advance = [&]() {
            if (left > 0) {
                ++nxt.tile;
                --left;
            } else {
                nxt = C.decode(C.take_ticket());
                left = C.rest_of_strip(nxt);
            }
        };
        if (lane == 0) {
            advance();
            C.issue(0, nxt);
            advance();
            C.issue(1, nxt);
            advance();
        }
        __syncwarp();
        bar_sync(kBarEnd, kAll);   // start: both descriptors are visible
        bool prev_done = false;
        for (int k = 0;; ++k) {
            const Item cur = item[k & 1];
            bar_sync(kBarEnd, kAll);   // the pass-A threads have finished item k
            const bool done = cur.kind == 2;
            if (done && prev_done) break;
            prev_done = done;
            if (lane == 0) {
                C.issue(k & 1, nxt);   // item k + 2 goes into the buffer that item k has released
                // Two global atomics, both in flight at once: the next ticket (needed at the next item
                // barrier) and the tile counter of the head.  No fence here: the pass-A threads fence
                // their block sums before the item barrier.
                const bool in_strip = left > 0;
                const bool more = !in_strip && nxt.kind != 2;
                unsigned long long t_raw = ~0ULL;
                if (more) t_raw = C.take_ticket();
                int fin_unit = -1;
                if (cur.kind == 0) {
                    const int prev = atomicAdd(A.ctrl + kCtrlHeader + cur.unit, 1);
                    if (prev == tiles_per_unit - 1) fin_unit = cur.unit;
                    // publish the tile's min/max of a_c and re-arm the slots
                    uint32_t* m = mmk + (k & 1) * 6;
                    if (m[4] != 0xffffffffu) atomicMin(&A.mm[(int64_t)cur.unit * 6 + 4], m[4]);
                    if (m[5] != 0u) atomicMax(&A.mm[(int64_t)cur.unit * 6 + 5], m[5]);
                    m[4] = 0xffffffffu;
                    m[5] = 0u;
                }
                fin[k & 1] = fin_unit;
                if (in_strip) {
                    ++nxt.tile;
                    --left;
                } else if (more) {
                    nxt = C.decode(t_raw);
                    left = C.rest_of_strip(nxt);
                } else {
                    nxt.kind = 2;
                }
            }
            __syncwarp();
        }
        return;
    }

    // ---------------------------------------------------------------------- pass-A threads
    bar_sync(kBarEnd, kAll);   // start
    bool prev_done = false;
    for (int k = 0;; ++k) {
        const Item cur = item[k & 1];
        const int buf = k & 1;
        if (cur.kind == 0)
            pass_a<T, D>(A, cur.unit, cur.tile, tiles + (size_t)buf * G::kTileBytes, pp, invs, mmk + buf * 6, &full[buf],
                         (uint32_t)((k >> 1) & 1), abort_flag);
        bar_sync(kBarEnd, kAll);   // end of item k
        const bool done = cur.kind == 2;
        if (done && prev_done) break;
        prev_done = done;
        // the head completed by item k - 1 (known since the control warp passed this barrier) gets its anchors
        if (k >= 1) {
            const int f = fin[(k - 1) & 1];
            if (f >= 0) finalize_head<T, D>(A, f, pp, invs);
        }
    }
}

__global__ void fused_init_kernel(int units, uint32_t* mm, int* ctrl) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < (long long)units * 6) mm[i] = (i & 1) ? 0u : 0xffffffffu;
    if (i < (long long)kCtrlHeader + 2LL * units) ctrl[i] = 0;
}

template <typename T, int D>
cudaError_t launch_one(const FusedArgs& A, int sm_count, cudaStream_t stream) {
    using G = Geo<T, D>;
    const long long tiles = (long long)A.units * ((A.K.N + G::kTile - 1) / G::kTile);
    const unsigned grid = (unsigned)(tiles < sm_count ? tiles : sm_count);
    fused_scan_kernel<T, D><<<grid, G::kThreads + 32 + kBThreads, fused_smem_bytes<T, D>(), stream>>>(A);
    return cudaGetLastError();
}

}  // namespace

#define NKV_DISPATCH(dtype, d, CALL)                                         \
    do {                                                                     \
        if ((dtype) == NKV_BF16 && (d) == 64) { CALL(__nv_bfloat16, 64); }   \
        else if ((dtype) == NKV_BF16 && (d) == 128) { CALL(__nv_bfloat16, 128); } \
        else if ((dtype) == NKV_F32 && (d) == 64) { CALL(float, 64); }       \
        else if ((dtype) == NKV_F32 && (d) == 128) { CALL(float, 128); }     \
        else return cudaErrorInvalidValue;                                   \
    } while (0)

cudaError_t configure_fused_kernels() {
    cudaError_t e = cudaSuccess;
#define CALL(T, D)                                                                                          \
    if (e == cudaSuccess)                                                                                   \
    e = cudaFuncSetAttribute(fused_scan_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,          \
                             (int)fused_smem_bytes<T, D>())
    CALL(__nv_bfloat16, 64);
    CALL(__nv_bfloat16, 128);
    CALL(float, 64);
    CALL(float, 128);
#undef CALL
    return e;
}

// The fused scan needs episodic blocks that are whole 8-row segments and tiles that are whole blocks.
bool fused_scan_supported(const ScoreParams& sp, int dtype, int d) {
    const int row_bytes = d * (dtype == NKV_BF16 ? 2 : 4);
    const int tile = 65536 / row_bytes;
    return sp.block % kSeg == 0 && tile % sp.block == 0;
}

size_t fused_ctrl_bytes(int64_t units) { return (size_t)(kCtrlHeader + 2 * units) * sizeof(int); }

cudaError_t launch_fused_scan(const TensorView& K, int dtype, int G, const ScoreParams& sp, float* block_sums,
                              float* mu_s, float* inv_s, float* inv_e, float* inv_norm, float* a_raw, uint32_t* mm,
                              int* ctrl, int* status, int sm_count, int lag, int hints, cudaStream_t stream,
                              int64_t* launches) {
    FusedArgs A;
    A.K = K;
    A.sp = sp;
    A.units = G * K.H;
    A.lag = lag < 1 ? 1 : lag;
    A.hints = hints;
    A.strip = 4;
    A.block_sums = block_sums;
    A.mu_s = mu_s;
    A.inv_s = inv_s;
    A.inv_e = inv_e;
    A.inv_norm = inv_norm;
    A.a_raw = a_raw;
    A.mm = mm;
    A.ctrl = ctrl;
    A.status = status;
    const long long words = (long long)kCtrlHeader + 2LL * A.units;
    const long long n_init = words > 6LL * A.units ? words : 6LL * A.units;
    fused_init_kernel<<<(unsigned)((n_init + 255) / 256), 256, 0, stream>>>(A.units, mm, ctrl);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
#define CALL(T, D) e = launch_one<T, D>(A, sm_count, stream)
    NKV_DISPATCH(dtype, K.d, CALL);
#undef CALL
    ++*launches;
    return e;
}

}  // namespace nkv
