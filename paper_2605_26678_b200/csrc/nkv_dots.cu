// Second key pass on the tensor cores (bf16 keys, d = 64 or 128): a_s(i) = -cos(k_hat_i, mu_s) and
// a_e(i) = -cos(k_hat_i, mu_e(block of i)) with their per-head min/max (Section 2.3).
//
// The dots of 128 keys with the anchors are one skinny product [128 x d] x [d x 16] per tile.  The fp32
// anchors enter as three bf16 columns each (hi + mid + lo carries all 24 mantissa bits; products of bf16
// numbers are exact in fp32 and tcgen05.mma accumulates in fp32), so a tile's right-hand side is
//     columns 0..2  mu_s        3..5  mu_e of the block the tile starts in        6..8  mu_e of the next block
// (a tile of 128 keys touches at most two blocks because a block has at least 128 keys).  Key tiles are
// staged by TMA (128-byte swizzle) several tiles ahead; the tensor core reads them from shared memory
// directly, so the SM issues a few dozen instructions per tile and the pass runs at the speed of the
// copy.  Warp roles: TMA producer, MMA issuer, four warps that build the right-hand sides, four warps
// that turn the accumulator into scores.  Every wait is bounded.
#include "nkv_sm100.cuh"

namespace nkv {

namespace {

using namespace sm100;

constexpr int kTile = 128;                        // keys per tile
constexpr int kTileHalfBytes = kTile * 128;       // one 64-column half of a tile
constexpr int kRhsHalfBytes = 16 * 128;           // 16 right-hand-side rows of 64 columns
constexpr int kStages = 4;                        // accumulators of 32 columns (16 used)
constexpr uint32_t kTmemCols = 128;
constexpr int kPrepWarp0 = 0, kEpiWarp0 = 4, kProducerWarp = 8, kMmaWarp = 9;
constexpr int kThreads = 10 * 32;
constexpr int kMaxSlots = 10;

// Sizes for head dimension D (64 or 128): a key row is D / 64 swizzled halves of 128 bytes.
template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kSlots = 640 / D;                       // key tiles staged at once (160 KB)
    static constexpr int kTileBytes = kHalves * kTileHalfBytes;
    static constexpr int kRhsBytes = kHalves * kRhsHalfBytes;
    static constexpr int kPrepWarps = D / 32;                    // one thread per column
    static_assert(kSlots <= kMaxSlots, "barrier arrays too small");
};

struct Smem {
    uint64_t full[kMaxSlots];   // key tile landed
    uint64_t rready[kMaxSlots]; // right-hand side written (one arrival per building warp)
    uint64_t kfree[kMaxSlots];  // tile and right-hand side consumed by the MMAs
    uint64_t tfull[kStages];    // accumulator written
    uint64_t tempty[kStages];   // accumulator read (one arrival per reading warp)
    uint64_t drain;             // products issued before a give-up have completed
    uint32_t tmem_base;
};
template <int D>
constexpr size_t smem_bytes() {
    return 1024 + (size_t)Cfg<D>::kSlots * (Cfg<D>::kTileBytes + Cfg<D>::kRhsBytes) + sizeof(Smem);
}

struct TileRange {
    long long first, last;      // this CTA's tiles [first, last)
    int tiles_per_unit;
};
__device__ __forceinline__ TileRange my_tiles(int units, int N) {
    TileRange r;
    r.tiles_per_unit = (N + kTile - 1) / kTile;
    const long long total = (long long)units * r.tiles_per_unit;
    r.first = total * blockIdx.x / gridDim.x;
    r.last = total * (blockIdx.x + 1) / gridDim.x;
    return r;
}

// ---------------------------------------------------------------------------- roles
template <int D>
__device__ void dots_producer(const CUtensorMap* tmap, unsigned char* tiles, Smem* s, TileRange tr, int H, int* status) {
    using C = Cfg<D>;
    long long n = 0;
    const uint64_t policy = l2_evict_first_policy();   // keys are read once per pass
    for (long long t = tr.first; t < tr.last; ++t, ++n) {
        const int slot = (int)(n % C::kSlots);
        const long long fill = n / C::kSlots;
        if (fill > 0 && !mbar_wait(&s->kfree[slot], (uint32_t)((fill - 1) & 1), status, 711)) {
            // giving up: the copies already armed still land in this CTA's shared memory, so stay (bounded)
            // until they have
            for (long long m = n > C::kSlots ? n - C::kSlots : 0; m < n; ++m)
                for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try_wait(&s->full[m % C::kSlots], (uint32_t)((m / C::kSlots) & 1)); ++spin)
                    __nanosleep(256);
            return;
        }
        const int u = (int)(t / tr.tiles_per_unit);
        const int i0 = (int)(t - (long long)u * tr.tiles_per_unit) * kTile;
        const int g = u / H, h = u - g * H;
        unsigned char* dst = tiles + (size_t)slot * C::kTileBytes;
        mbar_expect_tx(&s->full[slot], C::kTileBytes);
#pragma unroll
        for (int half = 0; half < C::kHalves; ++half)
            tma_load_4d(dst + half * kTileHalfBytes, tmap, 64 * half, i0, h, g, &s->full[slot], policy);
    }
}

template <int D>
__device__ void dots_mma(unsigned char* tiles, unsigned char* rhs, Smem* s, uint32_t tmem_base, TileRange tr,
                         int* status) {
    using C = Cfg<D>;
    constexpr uint32_t idesc = umma_idesc_bf16(kTile, 16);
    const uint32_t tiles_addr = smem_addr(tiles), rhs_addr = smem_addr(rhs);
    long long n = 0;
    for (long long t = tr.first; t < tr.last; ++t, ++n) {
        const int slot = (int)(n % C::kSlots), stage = (int)(n % kStages);
        const uint32_t fpar = (uint32_t)((n / C::kSlots) & 1), upar = (uint32_t)((n / kStages) & 1);
        if (!mbar_wait(&s->full[slot], fpar, status, 712) || !mbar_wait(&s->rready[slot], fpar, status, 713) ||
            !mbar_wait(&s->tempty[stage], upar ^ 1u, status, 714)) {
            // products already issued keep reading shared memory and writing tensor memory: wait (bounded)
            // for them before the CTA frees both
            umma_commit(&s->drain);
            for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try_wait(&s->drain, 0); ++spin) __nanosleep(256);
            return;
        }
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t a = tiles_addr + (uint32_t)slot * C::kTileBytes + (uint32_t)(kk >> 2) * kTileHalfBytes +
                               (uint32_t)(kk & 3) * 32u;
            const uint32_t b = rhs_addr + (uint32_t)slot * C::kRhsBytes + (uint32_t)(kk >> 2) * kRhsHalfBytes +
                               (uint32_t)(kk & 3) * 32u;
            umma_bf16(tmem_base + (uint32_t)stage * 32u, umma_desc_sw128(a), umma_desc_sw128(b), idesc, kk > 0);
        }
        umma_commit(&s->tfull[stage]);
        umma_commit(&s->kfree[slot]);
    }
}

// Thread k writes column k of the nine right-hand-side rows of every tile (rows 9..15 stay zero).
template <int D>
__device__ void dots_prep(unsigned char* rhs, Smem* s, ScoreParams sp, TileRange tr, const float* __restrict__ mu_s,
                          const float* __restrict__ mu_e, int* status) {
    using C = Cfg<D>;
    const int k = threadIdx.x - kPrepWarp0 * 32, lane = k & 31;
    if (k >= D) return;   // d = 64 needs two of the four warps
    const int half = k >> 6, kk = k & 63;
    float v[3] = {0.f, 0.f, 0.f};
    int cur_u = -1, cur_blk = -1;
    long long n = 0;
    for (long long t = tr.first; t < tr.last; ++t, ++n) {
        const int slot = (int)(n % C::kSlots);
        const long long fill = n / C::kSlots;
        if (fill > 0 && !mbar_wait(&s->kfree[slot], (uint32_t)((fill - 1) & 1), status, 715)) return;
        const int u = (int)(t / tr.tiles_per_unit);
        const int i0 = (int)(t - (long long)u * tr.tiles_per_unit) * kTile;
        const int blk0 = i0 / sp.block;
        if (u != cur_u || blk0 != cur_blk) {   // the anchors change every few tiles only
            if (u != cur_u) v[0] = mu_s[(int64_t)u * D + k];
            v[1] = mu_e[((int64_t)u * sp.nblocks + blk0) * D + k];
            v[2] = blk0 + 1 < sp.nblocks ? mu_e[((int64_t)u * sp.nblocks + blk0 + 1) * D + k] : 0.f;
            cur_u = u;
            cur_blk = blk0;
        }
        unsigned char* base = rhs + (size_t)slot * C::kRhsBytes + (size_t)half * kRhsHalfBytes + (kk & 7) * 2;
#pragma unroll
        for (int a = 0; a < 3; ++a) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(v[a]);
            const float r1 = v[a] - __bfloat162float(hi);
            const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
            const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
            const __nv_bfloat16 part[3] = {hi, mid, lo};
#pragma unroll
            for (int j = 0; j < 3; ++j) {
                const int row = 3 * a + j;   // row of the right-hand side, 8-row groups 1024 bytes apart
                *reinterpret_cast<__nv_bfloat16*>(base + (row >> 3) * 1024 + (row & 7) * 128 +
                                                  ((((kk >> 3) ^ (row & 7))) << 4)) = part[j];
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads these writes
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->rready[slot]);
    }
}

// Thread r reads row r of the accumulator: the key's dots with mu_s and with the two candidate mu_e.
__device__ void dots_epilogue(Smem* s, uint32_t tmem_base, ScoreParams sp, TileRange tr, int N,
                              const float* __restrict__ inv_norm, const float* __restrict__ inv_s,
                              const float* __restrict__ inv_e, float* __restrict__ a_raw, uint32_t* __restrict__ mm,
                              int* status) {
    const int r = threadIdx.x - kEpiWarp0 * 32, q = r >> 5, lane = r & 31;
    int cur_u = -1;
    float rs = 0.f;
    float lo_s = INFINITY, hi_s = -INFINITY, lo_e = INFINITY, hi_e = -INFINITY;
    auto flush = [&]() {   // the warp's min/max of the head it has been working on
        if (cur_u < 0) return;
        lo_s = warp_min(lo_s);
        hi_s = warp_max(hi_s);
        lo_e = warp_min(lo_e);
        hi_e = warp_max(hi_e);
        if (lane == 0 && lo_s <= hi_s) {
            atomicMin(&mm[(int64_t)cur_u * 6 + 0], ord_key(lo_s));
            atomicMax(&mm[(int64_t)cur_u * 6 + 1], ord_key(hi_s));
            atomicMin(&mm[(int64_t)cur_u * 6 + 2], ord_key(lo_e));
            atomicMax(&mm[(int64_t)cur_u * 6 + 3], ord_key(hi_e));
        }
        lo_s = lo_e = INFINITY;
        hi_s = hi_e = -INFINITY;
    };
    // per-tile inputs of this thread's row, fetched one tile ahead of their use
    struct RowIn {
        int u, i;
        bool second;
        float inv_i, re;
    };
    auto fetch = [&](long long t) {
        RowIn x;
        x.u = (int)(t / tr.tiles_per_unit);
        const int i0 = (int)(t - (long long)x.u * tr.tiles_per_unit) * kTile;
        const int blk0 = i0 / sp.block;
        x.i = i0 + r;
        x.second = x.i >= (blk0 + 1) * sp.block;   // the key lies in the block after the tile's first
        const int blk = min(blk0 + (x.second ? 1 : 0), sp.nblocks - 1);
        x.inv_i = x.i < N ? inv_norm[(int64_t)x.u * N + x.i] : 0.f;
        x.re = inv_e[(int64_t)x.u * sp.nblocks + blk];
        return x;
    };
    long long n = 0;
    RowIn nxt = {};
    if (tr.first < tr.last) nxt = fetch(tr.first);
    for (long long t = tr.first; t < tr.last; ++t, ++n) {
        const int stage = (int)(n % kStages);
        const RowIn cur = nxt;
        if (t + 1 < tr.last) nxt = fetch(t + 1);
        if (cur.u != cur_u) {
            flush();
            cur_u = cur.u;
            rs = inv_s[cur.u];
        }
        if (!mbar_wait(&s->tfull[stage], (uint32_t)((n / kStages) & 1), status, 716)) return;
        tc_fence_after();
        float d[16];
        tmem_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)stage * 32u, d);
        tmem_wait_ld(d);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s->tempty[stage]);
        const float ds = d[0] + d[1] + d[2];
        const float de = cur.second ? d[6] + d[7] + d[8] : d[3] + d[4] + d[5];
        const float a_s = -(ds * cur.inv_i) * rs + 0.f;
        const float a_e = -(de * cur.inv_i) * cur.re + 0.f;
        if (cur.i < N) {
            a_raw[((int64_t)cur.u * 3 + 0) * N + cur.i] = a_s;
            a_raw[((int64_t)cur.u * 3 + 1) * N + cur.i] = a_e;
            lo_s = fminf(lo_s, a_s);
            hi_s = fmaxf(hi_s, a_s);
            lo_e = fminf(lo_e, a_e);
            hi_e = fmaxf(hi_e, a_e);
        }
    }
    flush();
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
anchor_dots_kernel(const __grid_constant__ CUtensorMap tmap, ScoreParams sp, int units, int H, int N,
                   const float* __restrict__ mu_s, const float* __restrict__ mu_e, const float* __restrict__ inv_norm,
                   const float* __restrict__ inv_s, const float* __restrict__ inv_e, float* __restrict__ a_raw,
                   uint32_t* __restrict__ mm, int* status) {
    using C = Cfg<D>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* tiles = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    unsigned char* rhs = tiles + (size_t)C::kSlots * C::kTileBytes;
    Smem* s = reinterpret_cast<Smem*>(rhs + (size_t)C::kSlots * C::kRhsBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const TileRange tr = my_tiles(units, N);

    if (tid == 0) {
        for (int i = 0; i < C::kSlots; ++i) {
            mbar_init(&s->full[i], 1);
            mbar_init(&s->rready[i], C::kPrepWarps);
            mbar_init(&s->kfree[i], 1);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&s->tfull[i], 1);
            mbar_init(&s->tempty[i], 4);
        }
        mbar_init(&s->drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < C::kSlots * C::kRhsBytes / 16; i += kThreads) reinterpret_cast<uint4*>(rhs)[i] = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == kMmaWarp) tmem_alloc(&s->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s->tmem_base;

    if (warp == kProducerWarp) {
        if (lane == 0) dots_producer<D>(&tmap, tiles, s, tr, H, status);
        __syncwarp();
    } else if (warp == kMmaWarp) {
        if (lane == 0) dots_mma<D>(tiles, rhs, s, tmem_base, tr, status);
        __syncwarp();
    } else if (warp >= kEpiWarp0) {
        dots_epilogue(s, tmem_base, sp, tr, N, inv_norm, inv_s, inv_e, a_raw, mm, status);
    } else {
        dots_prep<D>(rhs, s, sp, tr, mu_s, mu_e, status);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

cudaError_t configure_dots_kernels() {
    cudaError_t e = cudaFuncSetAttribute(anchor_dots_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem_bytes<64>());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(anchor_dots_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)smem_bytes<128>());
}

// bf16 keys of 64 or 128 columns, strides a tensor map accepts, and blocks of at least 128 keys (a tile
// of 128 keys then touches at most two blocks).
bool anchor_dots_supported(const TensorView& K, int dtype, const ScoreParams& sp) {
    if (dtype != NKV_BF16 || (K.d != 64 && K.d != 128) || sp.block < kTile) return false;
    if (reinterpret_cast<uintptr_t>(K.ptr) % 16 != 0) return false;
    if (K.stride_h % 8 != 0 || K.stride_g % 8 != 0) return false;
    if (K.stride_h < (int64_t)K.N * K.d || K.stride_g < (int64_t)K.N * K.d) return false;
    CUtensorMap probe;   // the driver has the last word on what a tensor map can describe
    return encode_key_map(K, 1, kTile, &probe) == cudaSuccess;
}

cudaError_t launch_anchor_dots(const TensorView& K, int G, const ScoreParams& sp, const float* mu_s, const float* mu_e,
                               const float* inv_norm, const float* inv_s, const float* inv_e, float* a_raw,
                               uint32_t* mm, int* status, int sm_count, cudaStream_t stream, int64_t* launches) {
    CUtensorMap tmap;
    cudaError_t e = encode_key_map(K, G, kTile, &tmap);
    if (e != cudaSuccess) return e;
    const int units = G * K.H;
    const long long total = (long long)units * ((K.N + kTile - 1) / kTile);
    const unsigned grid = (unsigned)(total < sm_count ? total : sm_count);
    if (K.d == 128)
        anchor_dots_kernel<128><<<grid, kThreads, smem_bytes<128>(), stream>>>(tmap, sp, units, K.H, K.N, mu_s, mu_e,
                                                                               inv_norm, inv_s, inv_e, a_raw, mm, status);
    else
        anchor_dots_kernel<64><<<grid, kThreads, smem_bytes<64>(), stream>>>(tmap, sp, units, K.H, K.N, mu_s, mu_e,
                                                                             inv_norm, inv_s, inv_e, a_raw, mm, status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
