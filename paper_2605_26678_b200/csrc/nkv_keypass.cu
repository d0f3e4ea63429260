// The key scan (Sections 2.1-2.3) as one persistent kernel on the tensor cores: bf16 keys, d = 128, window
// W = 64, episodic blocks of 128 or 256 keys.
//
// What is computed: w_i = 1/||k_i||, the sum of the normalised keys of every episodic block and of the whole
// head, and the three anomalies
//     a_c(i) = -cos(k_hat_i, mu_c(i))     mu_c(i) = mean of the last W normalised keys
//     a_e(i) = -cos(k_hat_i, mu_e(block of i))
//     a_s(i) = -cos(k_hat_i, mu_s)
// with their per-head minima and maxima.  A cosine does not change when its anchor is scaled, so block sums
// and the head sum stand in for the means.
//
// First touch of a key ("A tiles", 128 keys each).  With g_ij = w_i w_j (k_i . k_j) and S_i the sum of the
// last W normalised keys,  k_hat_i . S_i = sum_{j in window(i)} g_ij  and  ||S_i||^2 = sum_{j,l in window(i)}
// g_jl: sums over a band of the keys' Gram matrix.  Per tile the tensor core forms
//     D      = K[tile rows] x K[64 rows before .. tile rows]^T     128 x 192, fp32 in tensor memory
//     corner = K[previous tile rows] x K[first 64 tile rows]^T     128 x 64 (its last 64 rows are used)
//     tsum   = K[tile rows]^T x [w hi | w mid | w lo]              128 (channels) x 16: sum_i w_i k_i
// bf16 products are exact in fp32 and the accumulation is fp32, so D holds fp32 dot products; w enters the
// last product as three bf16 numbers that add up to its 24 mantissa bits.  ||k_i||^2 is the diagonal of D.
// Row r of D gives the backward band sum c_r (k_hat . S) and, with the corner that arrives one tile later,
// the forward band sum f_r; ||S_i||^2 follows from
//     T_i = T_{i-1} + (2 c_i - g_ii) - (2 f_{i-W} - g_{i-W,i-W}),
// a prefix sum over the tile that restarts every tile from an exact value (the sum of the 64 x 64 Gram
// block of the previous tile's last rows).  No quantity looks ahead of the keys already loaded.
//
// Second touch ("B tiles"): the dots of 128 keys with the head sum and with the block sum are one product
// [128 x d] x [d x 16] (both anchors split three ways into bf16).  It needs the sums over the whole head,
// so it trails the first touch, closely enough to find the keys in L2.
//
// A head is cut into pieces of a few tiles (whole blocks).  Every CTA (one per SM) runs two independent
// pipelines, each drawing pieces from its own global counter: the first-touch pipeline never waits for the
// other one; a second-touch piece waits (bounded) for the flag of its head.  A first-touch piece starts
// with a "halo" tile of the 128 rows before it, which yields the restart value, the norms and the forward
// sums its first real tile needs.  Per-tile sums of normalised keys go to global memory; the CTA that
// completes the last piece of a head adds them up per block and per head, takes the norms of those anchors
// and raises the head's flag.  A flag wait that runs out records NKV_ERR_TIMEOUT and the call goes on with
// whatever the buffers hold.
//
// Warps of a CTA: two teams of 8 warps take the first-touch tiles in turn (4 warps: norms, backward sums,
// tile sums; 4 warps: forward sums, prefix scan, a_c), so two tiles are in flight and a team's chain of
// tensor-memory round trips overlaps the other team's; 4 warps build the split anchors of the second touch
// and turn its accumulators into a_s, a_e; one TMA producer thread and one MMA issuer warp per
// pipeline.  The teams keep pieces of the accumulators in registers, so after start-up the other warp groups
// hand registers over to them (setmaxnreg).
// Keys are staged by TMA in two rings of 128-row slots (64-row slabs, 128-byte swizzle); hand-overs are
// mbarriers and named barriers inside a team; every wait is bounded.
#include "nkv_sm100.cuh"

namespace nkv {

namespace {

using namespace sm100;

constexpr int kD = 128;                       // head dimension
constexpr int kTile = 128;                    // keys per tile
constexpr int kSlabRows = 64;                 // rows per staged slab
constexpr int kSlotsA = 3;                    // first-touch tiles staged at once
constexpr int kSlotsB = 2;                    // second-touch tiles staged at once
constexpr int kSlabsA = 2 * kSlotsA + 1;      // slab 0 is a copy of the slab before slot 0's tile
constexpr int kSlabs = kSlabsA + 2 * kSlotsB;
constexpr int kSlabHalfBytes = kSlabRows * 128;            // one 64-column half of a slab
constexpr int kHalfBytes = kSlabs * kSlabHalfBytes;        // all slabs of one half are contiguous
constexpr int kRingBytes = 2 * kHalfBytes;
constexpr int kOperandBytes = 2 * 16 * 128;   // a 16-row operand of 128 columns: two swizzled halves
constexpr int kQueue = 4;                     // piece descriptors in flight per pipeline
constexpr int kHist = 8;                      // first-touch tiles whose hand-over state is kept
constexpr int kWRing = kHist * kTile, kWMask = kWRing - 1;   // per-row scalars of those tiles
constexpr int kPrefetchTiles = 3;             // first-touch tiles requested from DRAM into L2 ahead of their slot

// tensor-memory columns
constexpr uint32_t kColMain0 = 0, kColCorner = 192, kColMain1 = 256, kColTsum = 448, kColDots = 480;
constexpr uint32_t kTmemCols = 512;

// warps: team 0 = 0..7, team 1 = 8..15 (first four backward, last four forward), second touch 16..19,
// then warps 20..23 (producers: one thread each; issuers: lane 0 issues)
constexpr int kTeamThreads = 256;
constexpr int kBWarp0 = 16, kProdAWarp = 20, kProdBWarp = 21, kMmaAWarp = 22, kMmaBWarp = 23;
constexpr int kThreads = 24 * 32;
constexpr int kConsumersA = 17, kConsumersB = 5;
constexpr int kLaunchRegs = 80;                    // 65536 / kThreads rounded down to a multiple of 8
constexpr int kTeamRegs = 96, kOtherRegs = 40;     // registers per thread after the warp groups rebalance them
// the CTA can only redistribute what it was given at launch; asking for more would wait forever
static_assert(16 * 32 * kTeamRegs + 8 * 32 * kOtherRegs <= kLaunchRegs * kThreads, "register pool exceeded");   // warps (or single threads) that read a pipeline's queue

struct Item {
    int end, u, g, h, row0, ntiles;
};

struct KeyPassArgs {
    ScoreParams sp;
    int units, H, N;
    int tiles_per_piece, pieces;       // pieces per head
    int hints;                         // bit 0: keep first-touch lines in L2, bit 1: second-touch lines leave first
    int debug;                         // bit 0 (tests): the head flags are never raised
    uint32_t flag_spin_limit;
    float* tile_sums;                  // [units][tiles][d] sums of normalised keys per 128-key tile
    float* block_sums;                 // [units][nblocks][d]
    float* head_sum;                   // [units][d]
    float* inv_s;                      // [units]          1 / ||head sum||
    float* inv_e;                      // [units][nblocks] 1 / ||block sum||
    float* inv_norm;                   // [units][N]
    float* a_raw;                      // [units][3][N]
    uint32_t* mm;                      // [units][6] ordered min/max keys
    unsigned long long* next_a;        // pieces handed out, first touch
    unsigned long long* next_b;        // pieces handed out, second touch
    int* head_count;                   // [units] first-touch pieces completed
    int* head_ready;                   // [units] anchors final
    int* status;
};

struct alignas(16) TeamSmem {
    float c[kTile];              // backward band sums of the team's tile
    float fcur[64];              // forward band sums of the tile's rows 0..63
    float fprev[64];             // forward band sums of the previous tile's rows 64..127
    float wtot[4];               // per-warp totals of the tile's prefix sum
    float red[8];                // min/max reduction at the end of a piece
    float fin[2][kD];            // column sums of the finaliser
    int fin_flag;
};

struct Smem {
    float w[kWRing];             // 1/||k|| by row (0 outside the head)
    float g[kWRing];             // g_ii by row
    float carry[kHist][64];          // rows 64..127 of a tile: forward sums over the tile's own columns (unscaled)
    float apart[kHist][2];           // per-warp parts of the next tile's restart value
    TeamSmem team[2];
    Item qa[kQueue], qb[kQueue];
    uint64_t qa_full[kQueue], qa_free[kQueue], qb_full[kQueue], qb_free[kQueue];
    uint64_t full_a[kSlotsA], free_a[kSlotsA];   // first-touch slot landed / no longer read
    uint64_t full_b[kSlotsB], free_b[kSlotsB];
    uint64_t tfull[2], tempty[2];       // Gram accumulators (one per team)
    uint64_t cempty;                    // corner accumulator read
    uint64_t wpub[kHist];                   // norms of a tile are in the ring
    uint64_t spub[kHist];                   // carry and restart parts of a tile are written
    uint64_t done[kHist];                   // the other team's global writes of a piece are fenced
    uint64_t wsready[2];                // split norms written
    uint64_t tsfull[2], tsempty[2];     // tile-sum accumulators
    uint64_t rready[2], rfree[2];       // split anchors
    uint64_t dfull[2], dempty[2];       // second-touch accumulators
    uint64_t drain_a, drain_b;
    uint32_t tmem_base;
    int abort;
};
constexpr size_t kSmemBytes = 1024 + kRingBytes + 4 * kOperandBytes + sizeof(Smem);

struct Waiter {
    int* status;
    volatile int* abort;
};

// Bounded wait that also leaves when another role of the CTA has given up.  The polling loop is kept out of
// line: the kernel's roles run side by side and share the instruction cache.
__device__ __forceinline__ bool bwait_slow(uint64_t* bar, uint32_t parity, int* status, volatile int* abort, int where) {
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if (spin >= 8) __nanosleep(spin < 64 ? 32 : 128);
    }
    set_status(status, NKV_ERR_TIMEOUT, where);
    *abort = 1;
    return false;
}
__device__ __forceinline__ bool bwait(uint64_t* bar, uint32_t parity, const Waiter& wt, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    return bwait_slow(bar, parity, wt.status, wt.abort, where);
}

// Descriptor `cnt` of a pipeline's queue.  kWarp: the whole warp calls (one release per warp); else one thread.
template <bool kWarp>
__device__ __forceinline__ bool get_item(const Item* q, uint64_t* qfull, uint64_t* qfree, long long cnt, Item& it,
                                         const Waiter& wt, int where) {
    const int k = (int)(cnt & (kQueue - 1));
    if (!bwait(&qfull[k], (uint32_t)((cnt / kQueue) & 1), wt, where)) return false;
    it = q[k];
    if (kWarp) {
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(&qfree[k]);
    } else {
        mbar_arrive(&qfree[k]);
    }
    return true;
}

// Piece `idx` of the call: heads in order, pieces of a head in order.
__device__ __forceinline__ Item decode_item(long long idx, const KeyPassArgs& p) {
    Item it;
    it.end = idx >= (long long)p.units * p.pieces;
    it.u = it.g = it.h = it.row0 = it.ntiles = 0;
    if (it.end) return it;
    it.u = (int)(idx / p.pieces);
    const int piece = (int)(idx - (long long)it.u * p.pieces);
    it.g = it.u / p.H;
    it.h = it.u - it.g * p.H;
    const int T = (p.N + kTile - 1) / kTile;
    it.row0 = piece * p.tiles_per_piece * kTile;
    it.ntiles = min(p.tiles_per_piece, T - piece * p.tiles_per_piece);
    return it;
}

// 1/sqrt(x) to fp32 rounding for x well inside the normal range (one Newton step on the hardware estimate)
__device__ __forceinline__ float fast_rsqrt(float x) {
    const float y = rsqrtf(x);
    return y * fmaf(-0.5f * x * y, y, 1.5f);
}

// ---------------------------------------------------------------------------- producers
__device__ __forceinline__ void load_slab(unsigned char* dst, const CUtensorMap* tmap, int row, int h, int g, uint64_t* bar,
                                          bool hint, uint64_t pol) {
    if (hint) {
        tma_load_4d_hint(dst, tmap, 0, row, h, g, bar, pol);
        tma_load_4d_hint(dst + kHalfBytes, tmap, 64, row, h, g, bar, pol);
    } else {
        tma_load_4d(dst, tmap, 0, row, h, g, bar);
        tma_load_4d(dst + kHalfBytes, tmap, 64, row, h, g, bar);
    }
}

// Copies already armed still land in this CTA's shared memory: after a give-up, stay until they have.
__device__ __forceinline__ void settle_loads(uint64_t* full, int slots, long long n) {
    for (long long m = n > slots ? n - slots : 0; m < n; ++m) {
        uint64_t* bar = &full[m % slots];
        const uint32_t par = (uint32_t)((m / slots) & 1);
        for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try_wait(bar, par); ++spin) __nanosleep(256);
    }
}

// First-touch producer (one thread): draws pieces, publishes them, stages halo + tiles.
__device__ __forceinline__ void producer_a(const CUtensorMap* tmap, unsigned char* ring, Smem* s, const KeyPassArgs& p, const Waiter& wt) {
    const uint64_t pol = l2_policy_evict_last();
    const bool hint = (p.hints & 1) != 0;
    long long n = 0, ic = 0;
    bool ok = true;
    while (ok) {
        const Item it = decode_item((long long)atomicAdd(p.next_a, 1ULL), p);
        const int k = (int)(ic & (kQueue - 1));
        if (!bwait(&s->qa_free[k], (uint32_t)(((ic / kQueue) & 1) ^ 1), wt, 731)) break;
        s->qa[k] = it;
        mbar_arrive(&s->qa_full[k]);
        ++ic;
        if (it.end) break;
        // the first rows are asked of DRAM now; further on every tile asks for the one kPrefetchTiles ahead
        for (int tl = 1; tl <= min(kPrefetchTiles, it.ntiles); ++tl) {
            tma_prefetch_4d(tmap, 0, it.row0 + (tl - 1) * kTile, it.h, it.g);
            tma_prefetch_4d(tmap, 0, it.row0 + (tl - 1) * kTile + kSlabRows, it.h, it.g);
            tma_prefetch_4d(tmap, 64, it.row0 + (tl - 1) * kTile, it.h, it.g);
            tma_prefetch_4d(tmap, 64, it.row0 + (tl - 1) * kTile + kSlabRows, it.h, it.g);
        }
        for (int tl = 0; tl <= it.ntiles; ++tl, ++n) {
            if (tl + kPrefetchTiles <= it.ntiles && tl > 0) {
                const int row = it.row0 + (tl + kPrefetchTiles - 1) * kTile;
                tma_prefetch_4d(tmap, 0, row, it.h, it.g);
                tma_prefetch_4d(tmap, 0, row + kSlabRows, it.h, it.g);
                tma_prefetch_4d(tmap, 64, row, it.h, it.g);
                tma_prefetch_4d(tmap, 64, row + kSlabRows, it.h, it.g);
            }
            const int slot = (int)(n % kSlotsA);
            if (!bwait(&s->free_a[slot], (uint32_t)(((n / kSlotsA) & 1) ^ 1), wt, 732)) {
                ok = false;
                break;
            }
            const int R = it.row0 + (tl - 1) * kTile;
            const bool before = tl > 0 && slot == 0;   // slot 0's tile keeps its own copy of the slab before it
            mbar_expect_tx(&s->full_a[slot], (before ? 3 : 2) * 2 * kSlabHalfBytes);
            for (int j = before ? -1 : 0; j < 2; ++j)
                load_slab(ring + (size_t)(j < 0 ? 0 : 1 + 2 * slot + j) * kSlabHalfBytes, tmap, R + j * kSlabRows, it.h,
                          it.g, &s->full_a[slot], hint, pol);
        }
    }
    if (*wt.abort) settle_loads(s->full_a, kSlotsA, n);
}

// Second-touch producer (one thread).
__device__ __forceinline__ void producer_b(const CUtensorMap* tmap, unsigned char* ring, Smem* s, const KeyPassArgs& p, const Waiter& wt) {
    const uint64_t pol = l2_policy_evict_first();
    const bool hint = (p.hints & 2) != 0;
    long long n = 0, ic = 0;
    bool ok = true;
    while (ok) {
        const Item it = decode_item((long long)atomicAdd(p.next_b, 1ULL), p);
        const int k = (int)(ic & (kQueue - 1));
        if (!bwait(&s->qb_free[k], (uint32_t)(((ic / kQueue) & 1) ^ 1), wt, 733)) break;
        s->qb[k] = it;
        mbar_arrive(&s->qb_full[k]);
        ++ic;
        if (it.end) break;
        for (int tl = 0; tl < it.ntiles; ++tl, ++n) {
            const int slot = (int)(n % kSlotsB);
            if (!bwait(&s->free_b[slot], (uint32_t)(((n / kSlotsB) & 1) ^ 1), wt, 734)) {
                ok = false;
                break;
            }
            const int R = it.row0 + tl * kTile;
            mbar_expect_tx(&s->full_b[slot], 2 * 2 * kSlabHalfBytes);
            for (int j = 0; j < 2; ++j)
                load_slab(ring + (size_t)(kSlabsA + 2 * slot + j) * kSlabHalfBytes, tmap, R + j * kSlabRows, it.h, it.g,
                          &s->full_b[slot], hint, pol);
        }
    }
    if (*wt.abort) settle_loads(s->full_b, kSlotsB, n);
}

// ---------------------------------------------------------------------------- MMA issuers
// Offset of K step kk (16 columns) in descriptor units of 16 bytes, for a K-major operand whose two
// 64-column halves are `half_bytes` apart.
__device__ __forceinline__ constexpr uint64_t kstep(int kk, uint32_t half_bytes) {
    return (uint64_t)(((uint32_t)(kk >> 2) * half_bytes + (uint32_t)(kk & 3) * 32u) >> 4);
}

// Lane 0's value in every lane; also tells the compiler that the value is the same across the warp, so
// that descriptor arithmetic can stay in the uniform datapath the MMA instruction reads its operands from.
__device__ __forceinline__ uint32_t uni(uint32_t x) { return __shfl_sync(0xffffffffu, x, 0); }
__device__ __forceinline__ uint64_t uni(uint64_t x) {
    return ((uint64_t)uni((uint32_t)(x >> 32)) << 32) | uni((uint32_t)x);
}

// Products of the first touch (one warp; lane 0 issues).  Tile n of the CTA goes to the accumulator of
// team n & 1.  After the Gram and corner products of tile n come the tile-sum product of tile n - 1 (its
// norms are known by then) and the release of that tile's slot, which the products of tile n still read.
__device__ __forceinline__ void mma_a(unsigned char* ring, unsigned char* wsplit, Smem* s, uint32_t tmem, const Waiter& wt) {
    constexpr uint32_t idesc192 = umma_idesc_bf16(kTile, 192), idesc128 = umma_idesc_bf16(kTile, 128);
    constexpr uint32_t idesc64 = umma_idesc_bf16(kTile, 64);
    constexpr uint32_t idesc_ts = umma_idesc_bf16(kD, 16) | kUmmaAMajorMN;
    const uint32_t ring_a = smem_addr(ring), ws_a = smem_addr(wsplit);
    const bool leader = (threadIdx.x & 31) == 0;
    long long n = 0, nC = 0, nS = 0, ic = 0;
    int prev_slot = -1;
    bool prev_real = false;
    // Tile sum of the previous tile (real tiles) and release of its slot.
    auto flush = [&]() -> bool {
        if (prev_slot < 0) return true;
        if (prev_real) {
            const int b = (int)(nS & 1);
            if (!bwait(&s->wsready[b], (uint32_t)((nS >> 1) & 1), wt, 741)) return false;
            if (!bwait(&s->tsempty[b], (uint32_t)(((nS >> 1) & 1) ^ 1), wt, 742)) return false;
            tc_fence_after();
            const uint64_t rows = uni(umma_desc_sw128_mn(ring_a + (uint32_t)(1 + 2 * prev_slot) * kSlabHalfBytes, kHalfBytes));
            const uint64_t wdesc = uni(umma_desc_sw128(ws_a + (uint32_t)b * kOperandBytes));
            const uint32_t dsum = uni(tmem + kColTsum + 16u * (uint32_t)b);
            if (leader) {
#pragma unroll
                for (int kk = 0; kk < kTile / 16; ++kk)
                    umma_bf16(dsum, rows + (uint64_t)(kk * (2048 >> 4)), wdesc + kstep(kk, 2048u), idesc_ts, kk > 0);
                umma_commit(&s->tsfull[b]);
            }
            ++nS;
        }
        if (leader) umma_commit(&s->free_a[prev_slot]);
        __syncwarp();
        prev_slot = -1;
        return true;
    };
    for (;;) {
        Item it;
        if (!get_item<true>(s->qa, s->qa_full, s->qa_free, ic++, it, wt, 743)) return;
        if (it.end) break;
        for (int tl = 0; tl <= it.ntiles; ++tl, ++n) {
            const int slot = (int)(n % kSlotsA), par = (int)(n & 1);
            if (!bwait(&s->full_a[slot], (uint32_t)((n / kSlotsA) & 1), wt, 744)) return;
            if (!bwait(&s->tempty[par], (uint32_t)(((n >> 1) & 1) ^ 1), wt, 745)) return;
            tc_fence_after();
            const uint32_t dmain = uni(tmem + (par ? kColMain1 : kColMain0));
            const uint64_t own = uni(umma_desc_sw128(ring_a + (uint32_t)(1 + 2 * slot) * kSlabHalfBytes));
            if (tl == 0) {
                // halo: Gram of the 128 rows with themselves, columns 64..191 of the accumulator
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        umma_bf16(dmain + 64u, own + kstep(kk, kHalfBytes), own + kstep(kk, kHalfBytes), idesc128, kk > 0);
                }
            } else {
                const uint64_t wide = uni(umma_desc_sw128(ring_a + (uint32_t)(2 * slot) * kSlabHalfBytes));   // from the slab before
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        umma_bf16(dmain, own + kstep(kk, kHalfBytes), wide + kstep(kk, kHalfBytes), idesc192, kk > 0);
                }
                if (!bwait(&s->cempty, (uint32_t)((nC & 1) ^ 1), wt, 746)) return;
                tc_fence_after();
                const uint64_t prev = uni(umma_desc_sw128(ring_a + (uint32_t)(1 + 2 * prev_slot) * kSlabHalfBytes));
                const uint32_t dcorner = uni(tmem + kColCorner);
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        umma_bf16(dcorner, prev + kstep(kk, kHalfBytes), own + kstep(kk, kHalfBytes), idesc64, kk > 0);
                }
                ++nC;
            }
            if (leader) umma_commit(&s->tfull[par]);
            __syncwarp();
            if (!flush()) return;
            prev_slot = slot;
            prev_real = tl > 0;
        }
    }
    if (!flush()) return;
    // every product issued has completed before the accumulators are given back
    if (leader) umma_commit(&s->drain_a);
    __syncwarp();
    bwait(&s->drain_a, 0, wt, 747);
}

// Second touch (one warp; lane 0 issues): the tiles of a block share one pair of split anchors.
__device__ __forceinline__ void mma_b(unsigned char* ring, unsigned char* rhs, Smem* s, uint32_t tmem, int tiles_per_block,
                      const Waiter& wt) {
    constexpr uint32_t idesc16 = umma_idesc_bf16(kTile, 16);
    const uint32_t ring_a = smem_addr(ring), rhs_a = smem_addr(rhs);
    const bool leader = (threadIdx.x & 31) == 0;
    long long n = 0, nR = 0, ic = 0;
    for (;;) {
        Item it;
        if (!get_item<true>(s->qb, s->qb_full, s->qb_free, ic++, it, wt, 748)) return;
        if (it.end) break;
        for (int tl = 0; tl < it.ntiles; ++tl, ++n) {
            const int slot = (int)(n % kSlotsB), b = (int)(n & 1), rb = (int)(nR & 1);
            if (tl % tiles_per_block == 0 && !bwait(&s->rready[rb], (uint32_t)((nR >> 1) & 1), wt, 749)) return;
            if (!bwait(&s->full_b[slot], (uint32_t)((n / kSlotsB) & 1), wt, 750)) return;
            if (!bwait(&s->dempty[b], (uint32_t)(((n >> 1) & 1) ^ 1), wt, 751)) return;
            tc_fence_after();
            const uint64_t rows = uni(umma_desc_sw128(ring_a + (uint32_t)(kSlabsA + 2 * slot) * kSlabHalfBytes));
            const uint64_t anchors = uni(umma_desc_sw128(rhs_a + (uint32_t)rb * kOperandBytes));
            const uint32_t ddots = uni(tmem + kColDots + 16u * (uint32_t)b);
            const bool last_of_block = (tl + 1) % tiles_per_block == 0 || tl + 1 == it.ntiles;
            if (leader) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    umma_bf16(ddots, rows + kstep(kk, kHalfBytes), anchors + kstep(kk, 2048u), idesc16, kk > 0);
                umma_commit(&s->dfull[b]);
                umma_commit(&s->free_b[slot]);
                if (last_of_block) umma_commit(&s->rfree[rb]);
            }
            __syncwarp();
            if (last_of_block) ++nR;
        }
    }
    if (leader) umma_commit(&s->drain_b);
    __syncwarp();
    bwait(&s->drain_b, 0, wt, 752);
}

// ---------------------------------------------------------------------------- first-touch teams
// Band sums of one row of D over three 32-column chunks: column o of chunk A counts when o >= thr, chunk B
// counts whole, column o of chunk C counts when o < thr.  Every column is weighted by its key's 1/||k||;
// iA, iB, iC are the ring indices (multiples of 32) of the chunks' first keys.
__device__ __forceinline__ void band_sums3(uint32_t tA, uint32_t tB, uint32_t tC, const float* wring, int iA, int iB,
                                           int iC, int thr, float& X, float& Y, float& Z) {
    const float* wA = wring + (iA & kWMask);
    const float* wB = wring + (iB & kWMask);
    const float* wC = wring + (iC & kWMask);
    // 16 columns of chunk A and the 16 columns at the same offset of chunk C share the diagonal test
    auto cut16 = [&](const float* a, const float* c, const float* wa, const float* wc, int col0, float& xa, float& xb,
                     float& za, float& zb) {
#pragma unroll
        for (int o4 = 0; o4 < 4; ++o4) {
            const float4 fa = *reinterpret_cast<const float4*>(wa + 4 * o4);
            const float4 fc = *reinterpret_cast<const float4*>(wc + 4 * o4);
            const float was[4] = {fa.x, fa.y, fa.z, fa.w}, wcs[4] = {fc.x, fc.y, fc.z, fc.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int o = 4 * o4 + e;
                float& x = (e & 1) ? xb : xa;
                float& z = (e & 1) ? zb : za;
                if (col0 + o >= thr) x = fmaf(a[o], was[e], x);
                else z = fmaf(c[o], wcs[e], z);
            }
        }
    };
    auto dot16 = [&](const float* v, const float* w, float& s0, float& s1) {
#pragma unroll
        for (int o4 = 0; o4 < 4; ++o4) {
            const float4 ww = *reinterpret_cast<const float4*>(w + 4 * o4);
            s0 = fmaf(v[4 * o4], ww.x, s0);
            s1 = fmaf(v[4 * o4 + 1], ww.y, s1);
            s0 = fmaf(v[4 * o4 + 2], ww.z, s0);
            s1 = fmaf(v[4 * o4 + 3], ww.w, s1);
        }
    };
    float x0 = 0.f, x1 = 0.f, y0 = 0.f, y1 = 0.f, z0 = 0.f, z1 = 0.f;
    float p0[16], p1[16], p2[16], p3[16];
    tmem_ld16(tA, p0);
    tmem_ld16(tC, p1);
    tmem_wait_ld(p0, p1);
    tmem_ld16(tA + 16, p2);
    tmem_ld16(tC + 16, p3);
    cut16(p0, p1, wA, wC, 0, x0, x1, z0, z1);
    tmem_wait_ld(p2, p3);
    tmem_ld16(tB, p0);
    tmem_ld16(tB + 16, p1);
    cut16(p2, p3, wA + 16, wC + 16, 16, x0, x1, z0, z1);
    tmem_wait_ld(p0, p1);
    dot16(p0, wB, y0, y1);
    dot16(p1, wB + 16, y0, y1);
    X = x0 + x1;
    Y = y0 + y1;
    Z = z0 + z1;
}

// v[lane] of 32 registers
__device__ __forceinline__ float select_lane(const float* v, int lane) {
    float a[16], b[8], c[4], d[2];
#pragma unroll
    for (int j = 0; j < 16; ++j) a[j] = (lane & 16) ? v[j + 16] : v[j];
#pragma unroll
    for (int j = 0; j < 8; ++j) b[j] = (lane & 8) ? a[j + 8] : a[j];
#pragma unroll
    for (int j = 0; j < 4; ++j) c[j] = (lane & 4) ? b[j + 4] : b[j];
#pragma unroll
    for (int j = 0; j < 2; ++j) d[j] = (lane & 2) ? c[j + 2] : c[j];
    return (lane & 1) ? d[1] : d[0];
}

// The team that completed a head's last piece: block sums, head sum and the reciprocals of their norms
// (256 threads, `tid` inside the team, `bar` the team's named barrier).
__device__ __forceinline__ void finalise_head(TeamSmem* ts, const KeyPassArgs& p, int u, int tid, int bar) {
    const int nb = p.sp.nblocks, T = (p.N + kTile - 1) / kTile, tpb = p.sp.block / kTile;
    const float* tsum = p.tile_sums + (size_t)u * T * kD;
    float* bs = p.block_sums + (size_t)u * nb * kD;
    const int c = tid & (kD - 1), half = tid >> 7, warp = tid >> 5, lane = tid & 31;
    float sum = 0.f, comp = 0.f;   // compensated: the head sum is the anchor of every key of the head
    for (int b = half; b < nb; b += 2) {
        float v = 0.f;
        for (int t = b * tpb; t < min((b + 1) * tpb, T); ++t) v += __ldcg(tsum + (size_t)t * kD + c);
        bs[(size_t)b * kD + c] = v;
        const float y = v - comp;
        const float t2 = sum + y;
        comp = (t2 - sum) - y;
        sum = t2;
    }
    ts->fin[half][c] = sum;
    bar_sync(bar, kTeamThreads);   // also orders this team's block-sum writes before its reads below
    if (tid < kD) {
        const float tot = ts->fin[0][c] + ts->fin[1][c];
        p.head_sum[(size_t)u * kD + c] = tot;
        ts->fin[0][c] = tot;
    }
    bar_sync(bar, kTeamThreads);
    if (warp == 0) {
        const float4 v = *reinterpret_cast<const float4*>(&ts->fin[0][4 * lane]);
        const float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
        if (lane == 0) p.inv_s[u] = 1.0f / fmaxf(sqrtf(ss), kEps);
    }
    for (int b = warp; b < nb; b += kTeamThreads / 32) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(bs + (size_t)b * kD) + lane);
        const float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
        if (lane == 0) p.inv_e[(size_t)u * nb + b] = 1.0f / fmaxf(sqrtf(ss), kEps);
    }
}

// One team (8 warps) takes every second first-touch tile of the CTA.
__device__ __forceinline__ void team_role(int team, unsigned char* wsplit, Smem* s, uint32_t tmem, const KeyPassArgs& p,
                          const Waiter& wt) {
    const int tid = threadIdx.x - team * kTeamThreads, warp = tid >> 5, lane = tid & 31;
    const int q = warp & 3, side = warp >> 2;   // quarter of the tile's rows; 0 backward band, 1 forward band
    const int r = q * 32 + lane;                // row of the tile
    const int N = p.N, T = (N + kTile - 1) / kTile;
    const int bar_team = 1 + team, bar_fwd = 3 + team;
    const uint32_t lane_base = (uint32_t)(32 * q) << 16;
    const uint32_t dmain = tmem + lane_base + (team ? kColMain1 : kColMain0);
    TeamSmem* ts = &s->team[team];
    long long ic = 0, n0 = 0, real0 = 0;   // pieces read, first-touch tiles and real tiles before the piece
    for (;;) {
        Item it;
        const bool got = get_item<true>(s->qa, s->qa_full, s->qa_free, ic++, it, wt, 753);
        if (bar_or(bar_team, kTeamThreads, !got)) return;   // the team leaves together or not at all
        if (it.end) return;
        const int u = it.u;
        const long long n_last = n0 + it.ntiles;
        float lo = INFINITY, hi = -INFINITY;
        bool ok = true;
        for (int tl = (int)((n0 ^ team) & 1); tl <= it.ntiles; tl += 2) {
            const long long n = n0 + tl, nW = real0 + tl - 1;   // tile of the CTA; real tile of the CTA
            const bool real = tl > 0;
            const int R = it.row0 + (tl - 1) * kTile, i = R + r;
            const int wbase = (int)(n & (kHist - 1)) * kTile;   // ring index of the tile's row 0
            const int slot4 = (int)(n & (kHist - 1)), prev4 = (int)((n - 1) & (kHist - 1));
            ok = bwait(&s->tfull[team], (uint32_t)((n >> 1) & 1), wt, 754) && ok;
            tc_fence_after();
            float wi = 0.f, gi = 0.f;
            if (side == 0) {
                // the diagonal of D is ||k_i||^2
                float v[32];
                tmem_ld32(dmain + (uint32_t)(32 * q + 64), v);
                tmem_wait_ld(v, v + 16);
                const float n2 = select_lane(v, lane);
                if (i >= 0 && i < N) wi = n2 > 1e-30f ? fast_rsqrt(n2) : 1.0f / fmaxf(sqrtf(n2), kEps);
                gi = wi * wi * n2;
                s->w[wbase + r] = wi;
                s->g[wbase + r] = gi;
                if (real) {
                    if (i < N) p.inv_norm[(size_t)u * N + i] = wi;
                    // w as hi + mid + lo in bf16: rows 0..2 of the tile-sum product's second operand
                    unsigned char* base = wsplit + (size_t)(nW & 1) * kOperandBytes + (size_t)(r >> 6) * 2048 + (r & 7) * 2;
                    const __nv_bfloat16 hi_ = __float2bfloat16_rn(wi);
                    const float r1 = wi - __bfloat162float(hi_);
                    const __nv_bfloat16 mid_ = __float2bfloat16_rn(r1);
                    const __nv_bfloat16 lo_ = __float2bfloat16_rn(r1 - __bfloat162float(mid_));
                    const __nv_bfloat16 part[3] = {hi_, mid_, lo_};
#pragma unroll
                    for (int j = 0; j < 3; ++j)
                        *reinterpret_cast<__nv_bfloat16*>(base + j * 128 + (((((r & 63) >> 3)) ^ j) << 4)) = part[j];
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads these writes
                }
            }
            if (bar_or(bar_team, kTeamThreads, !ok)) return;   // the tile's norms are in the ring
            if (side == 0 && lane == 0) {
                mbar_arrive(&s->wpub[slot4]);
                if (real) mbar_arrive(&s->wsready[nW & 1]);
            }
            // the previous tile belongs to the other team: its norms, then (below) its carry and restart parts
            if (real) ok = bwait(&s->wpub[prev4], (uint32_t)(((n - 1) / kHist) & 1), wt, 755) && ok;
            float X, Y, Z;
            if (side == 0) {
                const int c0 = 32 * q;
                band_sums3(dmain + c0, dmain + c0 + 32, dmain + c0 + 64, s->w, wbase - 64 + c0, wbase - 32 + c0,
                           wbase + c0, lane + 1, X, Y, Z);
                ts->c[r] = wi * (X + Y + Z);
                if (q >= 2) {
                    // Gram block of the tile's last 64 rows: the next tile's exact restart value
                    const float bp = wi * (q == 2 ? Z : Y + Z);
                    const float ap = warp_sum(2.f * bp - gi);
                    if (lane == 0) s->apart[slot4][q - 2] = ap;
                }
            } else {
                // forward band: three chunks from column 32 q + 64; columns past 191 are the corner that
                // arrives with this tile and belongs to the same row of the previous tile
                uint32_t ta[3];
                int ia[3];
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    const int col = 32 * q + 64 + 32 * j;
                    if (col < 192) {
                        ta[j] = dmain + (uint32_t)col;
                        ia[j] = wbase - 64 + col;
                    } else if (real) {
                        ta[j] = tmem + lane_base + kColCorner + (uint32_t)(col - 192);
                        ia[j] = wbase + (col - 192);
                    } else {   // no corner with a halo tile; the value is not used
                        ta[j] = dmain + 160u;
                        ia[j] = wbase;
                    }
                }
                band_sums3(ta[0], ta[1], ta[2], s->w, ia[0], ia[1], ia[2], lane, X, Y, Z);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&s->tempty[team]);
                if (side == 1 && q >= 2 && real) mbar_arrive(&s->cempty);
            }
            if (real) ok = bwait(&s->spub[prev4], (uint32_t)(((n - 1) / kHist) & 1), wt, 756) && ok;
            if (side == 1) {
                const float wr = s->w[wbase + r];
                if (q < 2) {
                    ts->fcur[r] = wr * (X + Y + Z);
                } else {
                    const float wprev = s->w[(wbase - kTile + r) & kWMask];
                    const float late = q == 2 ? Z : Y + Z, now = q == 2 ? X + Y : X;
                    ts->fprev[r - 64] = wprev * (s->carry[prev4][r - 64] + late);
                    s->carry[slot4][r - 64] = now;
                }
            }
            if (q >= 2) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&s->spub[slot4]);
            }
            if (bar_or(bar_team, kTeamThreads, !ok)) return;   // band sums of the tile are written
            if (side == 0) {
                if (real) {
                    // sum of the tile's normalised keys: thread r owns channel r
                    const int b = (int)(nW & 1);
                    ok = bwait(&s->tsfull[b], (uint32_t)((nW >> 1) & 1), wt, 757) && ok;
                    tc_fence_after();
                    float d[16];
                    tmem_ld16(tmem + lane_base + kColTsum + 16u * (uint32_t)b, d);
                    tmem_wait_ld(d);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s->tsempty[b]);
                    p.tile_sums[((size_t)u * T + R / kTile) * kD + r] = d[0] + d[1] + d[2];
                }
            } else {
                // T_i = restart + prefix of (2 c_i - g_ii) - (2 f_{i-64} - g_{i-64,i-64})
                const float ci = ts->c[r];
                const float g0 = s->g[wbase + r];
                const float fm = r < 64 ? ts->fprev[r] : ts->fcur[r - 64];
                const float gm = s->g[(wbase + r - 64) & kWMask];
                float x = 2.f * ci - g0 - (2.f * fm - gm);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float y = __shfl_up_sync(0xffffffffu, x, o);
                    if (lane >= o) x += y;
                }
                if (lane == 31) ts->wtot[q] = x;
                bar_sync(bar_fwd, 128);
                float base = s->apart[prev4][0] + s->apart[prev4][1];
                for (int w = 0; w < q; ++w) base += ts->wtot[w];
                const float Ti = base + x;
                if (real && i < N) {
                    const float a_c = (Ti > 1e-30f ? -ci * fast_rsqrt(Ti) : -ci / fmaxf(sqrtf(fmaxf(Ti, 0.f)), kEps)) + 0.f;
                    p.a_raw[((size_t)u * 3 + 2) * N + i] = a_c;
                    lo = fminf(lo, a_c);
                    hi = fmaxf(hi, a_c);
                }
            }
        }
        // ---- end of the piece: min/max of the team's tiles
        if (side == 1) {
            lo = warp_min(lo);
            hi = warp_max(hi);
            if (lane == 0) {
                ts->red[2 * q] = lo;
                ts->red[2 * q + 1] = hi;
            }
        }
        // every write of the piece is fenced before the piece is counted: the team that did not take the
        // last tile reports, the other one waits for that report
        const bool owner = (int)(n_last & 1) == team;
        const int pslot = (int)((ic - 1) & (kHist - 1));
        __threadfence();
        __syncwarp();
        if (!owner && lane == 0) mbar_arrive(&s->done[pslot]);
        if (owner) ok = bwait(&s->done[pslot], (uint32_t)(((ic - 1) / kHist) & 1), wt, 758) && ok;
        if (bar_or(bar_team, kTeamThreads, !ok)) return;
        if (tid == 128) {
            for (int w = 0; w < 4; ++w) {
                lo = fminf(lo, ts->red[2 * w]);
                hi = fmaxf(hi, ts->red[2 * w + 1]);
            }
            if (lo <= hi) {
                atomicMin(&p.mm[(size_t)u * 6 + 4], ord_key(lo));
                atomicMax(&p.mm[(size_t)u * 6 + 5], ord_key(hi));
            }
        }
        if (owner) {
            // both teams have fenced every write of the piece
            if (tid == 0) {
                __threadfence();
                ts->fin_flag = atomicAdd(&p.head_count[u], 1) == p.pieces - 1;
            }
            bar_sync(bar_team, kTeamThreads);
            if (ts->fin_flag) {   // every piece of the head is done, by this CTA or by others
                __threadfence();
                finalise_head(ts, p, u, tid, bar_team);
                __threadfence();
                bar_sync(bar_team, kTeamThreads);
                if (tid == 0 && !(p.debug & 1)) {
                    __threadfence();
                    atomicExch(&p.head_ready[u], 1);
                }
            }
        }
        n0 += it.ntiles + 1;
        real0 += it.ntiles;
    }
}

// ---------------------------------------------------------------------------- second touch
__device__ __forceinline__ int ld_acquire(const int* ptr) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// Four warps.  Thread k writes column k of the six anchor rows (rows 6..15 stay zero): the head sum and the
// sum of the block, each as hi + mid + lo in bf16; thread r reads row r of a tile's accumulator: the key's
// dots with the head sum and with its block's sum.
__device__ __forceinline__ void second_touch_role(unsigned char* rhs, Smem* s, uint32_t tmem, const KeyPassArgs& p, const Waiter& wt) {
    const int r = threadIdx.x - kBWarp0 * 32, q = r >> 5, lane = r & 31;
    const int half = r >> 6, kk = r & 63;
    const int N = p.N, nb = p.sp.nblocks, tpb = p.sp.block / kTile;
    long long ic = 0, n = 0, nR = 0;
    bool degraded = false, ok = true;
    for (;;) {
        Item it;
        if (!get_item<true>(s->qb, s->qb_full, s->qb_free, ic++, it, wt, 761)) return;
        if (it.end) return;
        const int u = it.u;
        if (!degraded) {
            uint32_t spin = 0;
            while (ld_acquire(&p.head_ready[u]) == 0) {
                if (*wt.abort) return;
                if (++spin > p.flag_spin_limit) {
                    set_status(p.status, NKV_ERR_TIMEOUT, 762);
                    degraded = true;   // go on with what the buffers hold, wait for no further flag
                    break;
                }
                __nanosleep(spin < 16 ? 64 : 512);
            }
        }
        // the head's anchors, norms and 1/||k|| are final from here on
        const float rs = __ldcg(&p.inv_s[u]);
        const float v0 = __ldcg(&p.head_sum[(size_t)u * kD + r]);
        const int blk0 = it.row0 / p.sp.block, nblk = (it.ntiles + tpb - 1) / tpb;
        float v1 = __ldcg(&p.block_sums[((size_t)u * nb + blk0) * kD + r]);
        auto build = [&](int b) {   // split anchors of block blk0 + b; fetches the next block's sum
            const int rb = (int)((nR + b) & 1);
            ok = bwait(&s->rfree[rb], (uint32_t)((((nR + b) >> 1) & 1) ^ 1), wt, 763) && ok;
            const float v[2] = {v0, v1};
            if (b + 1 < nblk) v1 = __ldcg(&p.block_sums[((size_t)u * nb + blk0 + b + 1) * kD + r]);
            unsigned char* base = rhs + (size_t)rb * kOperandBytes + (size_t)half * 2048 + (kk & 7) * 2;
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(v[a]);
                const float r1 = v[a] - __bfloat162float(hi);
                const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                const __nv_bfloat16 part[3] = {hi, mid, lo};
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    const int row = 3 * a + j;
                    *reinterpret_cast<__nv_bfloat16*>(base + row * 128 + (((kk >> 3) ^ row) << 4)) = part[j];
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&s->rready[rb]);
        };
        float lo_s = INFINITY, hi_s = -INFINITY, lo_e = INFINITY, hi_e = -INFINITY;
        build(0);
        int i = it.row0 + r;
        float wi = i < N ? __ldcg(&p.inv_norm[(size_t)u * N + i]) : 0.f;
        float re = __ldcg(&p.inv_e[(size_t)u * nb + blk0]);
        for (int tl = 0; tl < it.ntiles; ++tl, ++n) {
            if (tl % tpb == 0 && tl / tpb + 1 < nblk) build(tl / tpb + 1);   // one block ahead of the products
            // this tile's inputs are in registers; fetch the next tile's while the product runs
            const int i_cur = i;
            const float wi_cur = wi, re_cur = re;
            if (tl + 1 < it.ntiles) {
                i = it.row0 + (tl + 1) * kTile + r;
                wi = i < N ? __ldcg(&p.inv_norm[(size_t)u * N + i]) : 0.f;
                re = __ldcg(&p.inv_e[(size_t)u * nb + (it.row0 + (tl + 1) * kTile) / p.sp.block]);
            }
            const int b = (int)(n & 1);
            if (!bwait(&s->dfull[b], (uint32_t)((n >> 1) & 1), wt, 764)) return;
            tc_fence_after();
            float d[16];
            tmem_ld16(tmem + ((uint32_t)(32 * q) << 16) + kColDots + 16u * (uint32_t)b, d);
            tmem_wait_ld(d);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s->dempty[b]);
            const float a_s = -((d[0] + d[1] + d[2]) * wi_cur) * rs + 0.f;
            const float a_e = -((d[3] + d[4] + d[5]) * wi_cur) * re_cur + 0.f;
            if (i_cur < N) {
                p.a_raw[((size_t)u * 3 + 0) * N + i_cur] = a_s;
                p.a_raw[((size_t)u * 3 + 1) * N + i_cur] = a_e;
                lo_s = fminf(lo_s, a_s);
                hi_s = fmaxf(hi_s, a_s);
                lo_e = fminf(lo_e, a_e);
                hi_e = fmaxf(hi_e, a_e);
            }
        }
        if (!ok) return;
        nR += nblk;
        lo_s = warp_min(lo_s);
        hi_s = warp_max(hi_s);
        lo_e = warp_min(lo_e);
        hi_e = warp_max(hi_e);
        if (lane == 0 && lo_s <= hi_s) {
            atomicMin(&p.mm[(size_t)u * 6 + 0], ord_key(lo_s));
            atomicMax(&p.mm[(size_t)u * 6 + 1], ord_key(hi_s));
            atomicMin(&p.mm[(size_t)u * 6 + 2], ord_key(lo_e));
            atomicMax(&p.mm[(size_t)u * 6 + 3], ord_key(hi_e));
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
key_pass_kernel(const __grid_constant__ CUtensorMap tmap, const KeyPassArgs p) {
    extern __shared__ unsigned char smem_raw[];
    // the swizzle atoms (8 rows x 128 bytes) must start on 1024-byte boundaries
    unsigned char* ring = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    unsigned char* wsplit = ring + kRingBytes;
    unsigned char* rhs = wsplit + 2 * kOperandBytes;
    Smem* s = reinterpret_cast<Smem*>(rhs + 2 * kOperandBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < kQueue; ++i) {
            mbar_init(&s->qa_full[i], 1);
            mbar_init(&s->qa_free[i], kConsumersA);
            mbar_init(&s->qb_full[i], 1);
            mbar_init(&s->qb_free[i], kConsumersB);
        }
        for (int i = 0; i < kSlotsA; ++i) {
            mbar_init(&s->full_a[i], 1);
            mbar_init(&s->free_a[i], 1);
        }
        for (int i = 0; i < kSlotsB; ++i) {
            mbar_init(&s->full_b[i], 1);
            mbar_init(&s->free_b[i], 1);
        }
        for (int i = 0; i < kHist; ++i) {
            mbar_init(&s->wpub[i], 4);
            mbar_init(&s->spub[i], 4);
            mbar_init(&s->done[i], 8);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s->tfull[i], 1);
            mbar_init(&s->tempty[i], 8);
            mbar_init(&s->wsready[i], 4);
            mbar_init(&s->tsfull[i], 1);
            mbar_init(&s->tsempty[i], 4);
            mbar_init(&s->rready[i], 4);
            mbar_init(&s->rfree[i], 1);
            mbar_init(&s->dfull[i], 1);
            mbar_init(&s->dempty[i], 4);
        }
        mbar_init(&s->cempty, 2);
        mbar_init(&s->drain_a, 1);
        mbar_init(&s->drain_b, 1);
        s->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows of the two 16-row operands that are never written must read as zeros
    for (int i = tid; i < 4 * kOperandBytes / 16; i += kThreads) reinterpret_cast<uint4*>(wsplit)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < kWRing; i += kThreads) {
        s->w[i] = 0.f;
        s->g[i] = 0.f;
    }
    for (int i = tid; i < kHist * 64; i += kThreads) (&s->carry[0][0])[i] = 0.f;
    if (tid < kHist * 2) (&s->apart[0][0])[tid] = 0.f;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == kMmaAWarp) tmem_alloc(&s->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s->tmem_base;
    Waiter wt;
    wt.status = p.status;
    wt.abort = &s->abort;

    // The teams hold tiles of the accumulators in registers; the other two warp groups (warps 16..19 and
    // 20..23) give registers up for them.  Every warp of a warp group runs the same instruction here.
    if (warp < 16) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kTeamRegs));
    else asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp < 16) {
        team_role(warp >> 3, wsplit, s, tmem, p, wt);
    } else if (warp < kProdAWarp) {
        second_touch_role(rhs, s, tmem, p, wt);
    } else if (warp == kMmaAWarp) {
        mma_a(ring, wsplit, s, tmem, wt);
    } else if (warp == kMmaBWarp) {
        mma_b(ring, rhs, s, tmem, p.sp.block / kTile, wt);
    } else {
        if (lane == 0) {
            if (warp == kProdAWarp) producer_a(&tmap, ring, s, p, wt);
            else producer_b(&tmap, ring, s, p, wt);
        }
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaAWarp) tmem_dealloc(tmem, kTmemCols);
}

// reset of the per-head min/max keys and of the scheduling words
__global__ void key_pass_init_kernel(int units, uint32_t* mm, int* ctrl, int ctrl_words) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < units * 6) mm[i] = (i & 1) ? 0u : 0xffffffffu;
    if (i < ctrl_words) ctrl[i] = 0;
}

// block sums and head sum -> means (the staged outputs mu_e, mu_s)
__global__ void key_pass_means_kernel(int units, int N, int block, int nblocks, const float* block_sums,
                                      const float* head_sum, float* mu_e, float* mu_s) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t per_unit = (int64_t)(nblocks + 1) * kD;
    if (i >= units * per_unit) return;
    const int u = (int)(i / per_unit), rem = (int)(i - u * per_unit);
    const int b = rem / kD, c = rem - b * kD;
    if (b < nblocks) {
        const int cnt = min(block, N - b * block);
        mu_e[((int64_t)u * nblocks + b) * kD + c] = block_sums[((int64_t)u * nblocks + b) * kD + c] / (float)cnt;
    } else {
        mu_s[(int64_t)u * kD + c] = head_sum[(int64_t)u * kD + c] / (float)N;
    }
}

}  // namespace

cudaError_t configure_keypass_kernels() {
    return cudaFuncSetAttribute(key_pass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
}

size_t keypass_ctrl_bytes(int64_t units) { return (size_t)(2 * units + 4) * sizeof(int); }
size_t keypass_tile_sum_bytes(int64_t units, int64_t N) {
    return (size_t)units * (size_t)((N + kTile - 1) / kTile) * kD * sizeof(float);
}

// bf16 keys of 128 columns, the paper's window of 64, blocks of whole tiles, and strides a tensor map
// accepts (multiples of 16 bytes, base 16-byte aligned).
bool keypass_supported(const TensorView& K, int dtype, const ScoreParams& sp) {
    if (dtype != NKV_BF16 || K.d != kD || sp.window != 64 || sp.block % kTile != 0) return false;
    if (reinterpret_cast<uintptr_t>(K.ptr) % 16 != 0) return false;
    if (K.stride_h % 8 != 0 || K.stride_g % 8 != 0) return false;
    if (K.stride_h < (int64_t)K.N * kD || K.stride_g < (int64_t)K.N * kD) return false;
    CUtensorMap probe;   // the driver has the last word on what a tensor map can describe
    return encode_key_map(K, 1, kSlabRows, &probe) == cudaSuccess;
}

cudaError_t launch_keypass(const TensorView& K, int G, const ScoreParams& sp, const KeyPassOptions& opt,
                           float* tile_sums, float* block_sums, float* head_sum, float* inv_s, float* inv_e,
                           float* inv_norm, float* a_raw, uint32_t* mm, int* ctrl, int* status, int sm_count,
                           cudaStream_t stream, int64_t* launches) {
    const int units = G * K.H;
    CUtensorMap tmap;
    cudaError_t e = encode_key_map(K, G, kSlabRows, &tmap);
    if (e != cudaSuccess) return e;
    const int ctrl_words = 2 * units + 4;
    const int init_n = units * 6 > ctrl_words ? units * 6 : ctrl_words;
    key_pass_init_kernel<<<(init_n + 255) / 256, 256, 0, stream>>>(units, mm, ctrl, ctrl_words);
    ++*launches;

    KeyPassArgs a;
    a.sp = sp;
    a.units = units;
    a.H = K.H;
    a.N = K.N;
    const int T = (K.N + kTile - 1) / kTile;
    const int tiles_per_block = sp.block / kTile;
    // pieces are whole blocks; small calls take smaller pieces so that every SM gets several
    int tpp = opt.tiles_per_piece > 0 ? opt.tiles_per_piece : 16;
    if (opt.tiles_per_piece <= 0)
        while (tpp > tiles_per_block && (int64_t)units * ((T + tpp - 1) / tpp) < 4LL * sm_count) tpp >>= 1;
    tpp = (tpp + tiles_per_block - 1) / tiles_per_block * tiles_per_block;
    a.tiles_per_piece = tpp;
    a.pieces = (T + tpp - 1) / tpp;
    const int64_t total = (int64_t)units * a.pieces;
    const unsigned grid = (unsigned)(total < sm_count ? total : sm_count);
    a.hints = opt.hints;
    a.debug = opt.debug;
    a.flag_spin_limit = opt.flag_spin_limit > 0 ? (uint32_t)opt.flag_spin_limit : (1u << 21);
    a.tile_sums = tile_sums;
    a.block_sums = block_sums;
    a.head_sum = head_sum;
    a.inv_s = inv_s;
    a.inv_e = inv_e;
    a.inv_norm = inv_norm;
    a.a_raw = a_raw;
    a.mm = mm;
    a.next_a = reinterpret_cast<unsigned long long*>(ctrl);
    a.next_b = reinterpret_cast<unsigned long long*>(ctrl) + 1;
    a.head_count = ctrl + 4;
    a.head_ready = ctrl + 4 + units;
    a.status = status;
    key_pass_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tmap, a);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_keypass_means(int units, int N, const ScoreParams& sp, const float* block_sums,
                                 const float* head_sum, float* mu_e, float* mu_s, cudaStream_t stream,
                                 int64_t* launches) {
    const int64_t n = (int64_t)units * (sp.nblocks + 1) * kD;
    key_pass_means_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(units, N, sp.block, sp.nblocks, block_sums,
                                                                           head_sum, mu_e, mu_s);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
