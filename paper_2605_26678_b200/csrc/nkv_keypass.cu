// Both key passes in one persistent kernel on the tensor cores (bf16 keys, d = 128, window W = 64, episodic
// blocks of 128 or 256 keys).
//
// What is computed (Sections 2.1-2.3): w_i = 1/||k_i||, the sum of the normalised keys of every episodic
// block and of the whole head, and the three anomalies
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
//     bsum   = K[tile rows]^T x [w hi | w mid | w lo]              128 (channels) x 16: sum_i w_i k_i
// bf16 products are exact in fp32 and the accumulation is fp32, so D holds fp32 dot products; w enters the
// last product as three bf16 numbers that add up to its 24 mantissa bits.  ||k_i||^2 is the diagonal of D.
// Row r of D gives the backward band sum c_r (k_hat . S) and, with the corner that arrives one tile later,
// the forward band sum f_r; ||S_i||^2 follows from
//     T_i = T_{i-1} + (2 c_i - g_ii) - (2 f_{i-W} - g_{i-W,i-W}),
// a prefix sum over the tile that restarts every tile from an exact value (the sum of the 64 x 64 Gram
// block of the previous tile's last rows).  No quantity looks ahead of the keys already loaded.
//
// Second touch ("B tiles"): the dots of 128 keys with the head sum and with the block sum are one product
// [128 x d] x [d x 16] (both anchors split three ways into bf16).  It needs the sums over the whole head, so
// it trails the first touch; the work is ordered so that it finds the keys in L2.
//
// Work is cut into items: a piece of a head (a few tiles, whole blocks) for the first touch or for the
// second.  One global sequence interleaves them, second-touch items trailing first-touch items by a fixed
// number of items; CTAs (one per SM) draw from it with an atomic counter.  A first-touch item starts with a
// "halo" tile of the 128 rows before the piece, which yields the restart value, the norms and the forward
// sums the first real tile needs.  The CTA that completes the last piece of a head sums its block sums,
// takes the norms of the anchors and raises the head's flag; a second-touch item waits (bounded) for that
// flag.  Every item depends only on items earlier in the sequence, which running CTAs hold, so the waits
// end.  A flag wait that runs out records NKV_ERR_TIMEOUT and goes on with whatever the buffers hold.
//
// Warp roles in a CTA: 4 warps backward sums, norms and block sums; 4 warps forward sums, prefix scan and
// a_c; 4 warps that turn second-touch accumulators into a_s, a_e; 4 warps that build the split anchors;
// one TMA producer thread (also draws the items); one MMA issuer thread.  Keys are staged by TMA in a ring
// of 128-row slots (64-row slabs, 128-byte swizzle); hand-overs are mbarriers and two named barriers per
// tile; every wait is bounded.
#include "nkv_sm100.cuh"

namespace nkv {

namespace {

using namespace sm100;

constexpr int kD = 128;                       // head dimension
constexpr int kTile = 128;                    // keys per tile
constexpr int kSlabRows = 64;                 // rows per staged slab
constexpr int kSlots = 5;                     // tiles staged at once
constexpr int kSlabs = 2 * kSlots + 1;        // slab 0 is a copy of the slab before slot 0's tile
constexpr int kSlabHalfBytes = kSlabRows * 128;            // one 64-column half of a slab
constexpr int kHalfBytes = kSlabs * kSlabHalfBytes;        // all slabs of one half are contiguous
constexpr int kRingBytes = 2 * kHalfBytes;
constexpr int kOperandBytes = 2 * 16 * 128;   // a 16-row operand of 128 columns: two swizzled halves
constexpr int kQueue = 4;                     // item descriptors in flight inside a CTA
constexpr int kWRing = 512, kWMask = kWRing - 1;   // per-row scalars of the last four first-touch tiles

// tensor-memory columns
constexpr uint32_t kColMain0 = 0, kColCorner = 192, kColMain1 = 256, kColBsum = 448, kColDots = 480;
constexpr uint32_t kTmemCols = 512;

constexpr int kBandThreads = 256;             // warps 0-3 backward, 4-7 forward
constexpr int kEpiWarp0 = 8, kPrepWarp0 = 12, kProducerWarp = 16, kMmaWarp = 17;
constexpr int kThreads = 18 * 32;
constexpr int kConsumerWarps = 17;            // every warp but the producer reads the item queue
constexpr int kBarBand = 1, kBarFwd = 2;      // named barriers

enum { kItemA = 0, kItemB = 1, kItemEnd = 2 };

struct Item {
    int kind, u, g, h, row0, ntiles;
};

struct KeyPassArgs {
    ScoreParams sp;
    int units, H, N;
    int tiles_per_piece, pieces;       // pieces per head
    long long lag_items;               // first-touch items ahead of the first second-touch item
    int hints;                         // bit 0: keep first-touch lines in L2, bit 1: second-touch lines leave first
    int debug;                         // bit 0 (tests): the head flags are never raised
    uint32_t flag_spin_limit;
    float* block_sums;                 // [units][nblocks][d] sums of normalised keys
    float* head_sum;                   // [units][d]
    float* inv_s;                      // [units]          1 / ||head sum||
    float* inv_e;                      // [units][nblocks] 1 / ||block sum||
    float* inv_norm;                   // [units][N]
    float* a_raw;                      // [units][3][N]
    uint32_t* mm;                      // [units][6] ordered min/max keys
    unsigned long long* next_item;
    int* head_count;                   // [units] first-touch pieces completed
    int* head_ready;                   // [units] anchors final
    int* status;
};

struct Smem {
    float w[kWRing];             // 1/||k|| by row (0 outside the head)
    float g[kWRing];             // g_ii by row
    float c[2][kTile];           // backward band sums of a tile
    float fcur[2][64];           // forward band sums of the tile's rows 0..63
    float fprev[2][64];          // forward band sums of the previous tile's rows 64..127
    float apart[2][2];           // per-warp parts of the next tile's restart value
    float wtot[2][4];            // per-warp totals of a tile's prefix sum
    float red[8];                // min/max reduction at the end of an item
    float fin[2][kD];            // column sums of the finaliser
    Item items[kQueue];
    uint64_t qfull[kQueue], qfree[kQueue];
    uint64_t full[kSlots];       // slot landed
    uint64_t sfree[kSlots];      // slot no longer read
    uint64_t tfull[2], tempty[2];       // Gram accumulators
    uint64_t cempty;                    // corner accumulator read
    uint64_t wsready[2];                // split norms written
    uint64_t bsfull[2], bsempty[2];     // block-sum accumulators
    uint64_t rready[2], rfree[2];       // split anchors
    uint64_t dfull[2], dempty[2];       // second-touch accumulators
    uint64_t drain;
    uint32_t tmem_base;
    int abort;
    int fin_flag;
};
constexpr size_t kSmemBytes = 1024 + kRingBytes + 4 * kOperandBytes + sizeof(Smem);

struct Waiter {
    int* status;
    volatile int* abort;
};

// Bounded wait that also leaves when another role of the CTA has given up.
__device__ __forceinline__ bool bwait(uint64_t* bar, uint32_t parity, const Waiter& wt, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    uint32_t ns = 32;
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*wt.abort) return false;
        __nanosleep(ns);
        if (ns < 256) ns <<= 1;
    }
    set_status(wt.status, NKV_ERR_TIMEOUT, where);
    *wt.abort = 1;
    return false;
}

// Item `cnt` of the CTA's queue.  kWarp: the whole warp calls (one release per warp); else one thread.
template <bool kWarp>
__device__ __forceinline__ bool get_item(Smem* s, long long cnt, Item& it, const Waiter& wt, int where) {
    const int q = (int)(cnt & (kQueue - 1));
    if (!bwait(&s->qfull[q], (uint32_t)((cnt / kQueue) & 1), wt, where)) return false;
    it = s->items[q];
    if (kWarp) {
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(&s->qfree[q]);
    } else {
        mbar_arrive(&s->qfree[q]);
    }
    return true;
}

// Place `pos` of the global sequence: the first `lag` places are first-touch items, then second- and
// first-touch items alternate until the first-touch items are used up, then the rest.
__device__ __forceinline__ Item decode_item(long long pos, const KeyPassArgs& p) {
    Item it;
    it.kind = kItemEnd;
    it.u = it.g = it.h = it.row0 = it.ntiles = 0;
    const long long UP = (long long)p.units * p.pieces;
    if (pos >= 2 * UP) return it;
    const long long L = p.lag_items < UP ? p.lag_items : UP;
    long long idx;
    if (pos < L) {
        it.kind = kItemA;
        idx = pos;
    } else {
        const long long t = pos - L, RA = UP - L;
        if (t < 2 * RA) {
            it.kind = (t & 1) ? kItemA : kItemB;
            idx = (t & 1) ? L + (t >> 1) : (t >> 1);
        } else {
            it.kind = kItemB;
            idx = t - RA;
        }
    }
    it.u = (int)(idx / p.pieces);
    const int piece = (int)(idx - (long long)it.u * p.pieces);
    it.g = it.u / p.H;
    it.h = it.u - it.g * p.H;
    const int T = (p.N + kTile - 1) / kTile;
    it.row0 = piece * p.tiles_per_piece * kTile;
    it.ntiles = min(p.tiles_per_piece, T - piece * p.tiles_per_piece);
    return it;
}

// ---------------------------------------------------------------------------- producer
__device__ void producer_role(const CUtensorMap* tmap, unsigned char* ring, Smem* s, const KeyPassArgs& p,
                              const Waiter& wt) {
    const uint64_t pol_a = l2_policy_evict_last(), pol_b = l2_policy_evict_first();
    long long n = 0, ic = 0;
    bool ok = true;
    while (ok) {
        const long long pos = (long long)atomicAdd(p.next_item, 1ULL);
        const Item it = decode_item(pos, p);
        const int q = (int)(ic & (kQueue - 1));
        if (!bwait(&s->qfree[q], (uint32_t)(((ic / kQueue) & 1) ^ 1), wt, 731)) break;
        s->items[q] = it;
        mbar_arrive(&s->qfull[q]);
        ++ic;
        if (it.kind == kItemEnd) break;
        const bool first_touch = it.kind == kItemA;
        const int ntl = first_touch ? it.ntiles + 1 : it.ntiles;
        const bool hint = first_touch ? (p.hints & 1) != 0 : (p.hints & 2) != 0;
        const uint64_t pol = first_touch ? pol_a : pol_b;
        for (int tl = 0; tl < ntl; ++tl, ++n) {
            const int slot = (int)(n % kSlots);
            if (!bwait(&s->sfree[slot], (uint32_t)(((n / kSlots) & 1) ^ 1), wt, 732)) {
                ok = false;
                break;
            }
            const int R = first_touch ? it.row0 + (tl - 1) * kTile : it.row0 + tl * kTile;
            const bool before = first_touch && tl > 0 && slot == 0;
            mbar_expect_tx(&s->full[slot], (before ? 3 : 2) * 2 * kSlabHalfBytes);
            for (int j = before ? -1 : 0; j < 2; ++j) {
                unsigned char* dst = ring + (size_t)(j < 0 ? 0 : 1 + 2 * slot + j) * kSlabHalfBytes;
                const int row = R + j * kSlabRows;
                if (hint) {
                    tma_load_4d_hint(dst, tmap, 0, row, it.h, it.g, &s->full[slot], pol);
                    tma_load_4d_hint(dst + kHalfBytes, tmap, 64, row, it.h, it.g, &s->full[slot], pol);
                } else {
                    tma_load_4d(dst, tmap, 0, row, it.h, it.g, &s->full[slot]);
                    tma_load_4d(dst + kHalfBytes, tmap, 64, row, it.h, it.g, &s->full[slot]);
                }
            }
        }
    }
    if (*wt.abort) {
        // copies already armed still land in this CTA's shared memory: stay until they have
        for (long long m = n > kSlots ? n - kSlots : 0; m < n; ++m) {
            uint64_t* bar = &s->full[m % kSlots];
            const uint32_t par = (uint32_t)((m / kSlots) & 1);
            for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try_wait(bar, par); ++spin) __nanosleep(256);
        }
    }
}

// ---------------------------------------------------------------------------- MMA issuer
__device__ void mma_role(unsigned char* ring, unsigned char* wsplit, unsigned char* rhs, Smem* s, uint32_t tmem,
                         const Waiter& wt) {
    constexpr uint32_t idesc192 = umma_idesc_bf16(kTile, 192), idesc128 = umma_idesc_bf16(kTile, 128);
    constexpr uint32_t idesc64 = umma_idesc_bf16(kTile, 64), idesc16 = umma_idesc_bf16(kTile, 16);
    constexpr uint32_t idesc_bs = umma_idesc_bf16(kD, 16) | kUmmaAMajorMN;
    const uint32_t ring_a = smem_addr(ring), ws_a = smem_addr(wsplit), rhs_a = smem_addr(rhs);
    long long n = 0, nA = 0, nC = 0, nS = 0, nB = 0, ic = 0;
    int pend_slot = -1;
    bool pend_real = false;
    // The tile whose slot is still read: issue its block-sum product (real tiles) and release the slot.
    auto flush = [&]() -> bool {
        if (pend_slot < 0) return true;
        if (pend_real) {
            const int b = (int)(nS & 1);
            if (!bwait(&s->wsready[b], (uint32_t)((nS >> 1) & 1), wt, 741)) return false;
            if (!bwait(&s->bsempty[b], (uint32_t)(((nS >> 1) & 1) ^ 1), wt, 742)) return false;
            tc_fence_after();
            const uint32_t a0 = ring_a + (uint32_t)(1 + 2 * pend_slot) * kSlabHalfBytes;
#pragma unroll
            for (int kk = 0; kk < kTile / 16; ++kk) {
                const uint64_t adesc = umma_desc_sw128_mn(a0 + (uint32_t)kk * 2048u, kHalfBytes);
                const uint64_t bdesc = umma_desc_sw128(ws_a + (uint32_t)b * kOperandBytes + (uint32_t)(kk >> 2) * 2048u +
                                                       (uint32_t)(kk & 3) * 32u);
                umma_bf16(tmem + kColBsum + 16u * (uint32_t)b, adesc, bdesc, idesc_bs, kk > 0);
            }
            umma_commit(&s->bsfull[b]);
            ++nS;
        }
        umma_commit(&s->sfree[pend_slot]);
        pend_slot = -1;
        return true;
    };
    for (;;) {
        Item it;
        if (!get_item<false>(s, ic++, it, wt, 743)) return;
        if (it.kind == kItemEnd) {
            if (!flush()) return;
            break;
        }
        if (it.kind == kItemA) {
            for (int tl = 0; tl <= it.ntiles; ++tl, ++n, ++nA) {
                const int slot = (int)(n % kSlots), par = (int)(nA & 1);
                if (!bwait(&s->full[slot], (uint32_t)((n / kSlots) & 1), wt, 744)) return;
                if (!bwait(&s->tempty[par], (uint32_t)(((nA >> 1) & 1) ^ 1), wt, 745)) return;
                if (tl > 0 && !bwait(&s->cempty, (uint32_t)((nC & 1) ^ 1), wt, 746)) return;
                tc_fence_after();
                const uint32_t dmain = tmem + (par ? kColMain1 : kColMain0);
                const uint32_t a0 = ring_a + (uint32_t)(1 + 2 * slot) * kSlabHalfBytes;
                if (tl == 0) {
                    // halo: Gram of the 128 rows with themselves, columns 64..191 of the accumulator
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk) {
                        const uint32_t koff = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
                        umma_bf16(dmain + 64u, umma_desc_sw128(a0 + koff), umma_desc_sw128(a0 + koff), idesc128, kk > 0);
                    }
                } else {
                    const uint32_t b0 = ring_a + (uint32_t)(2 * slot) * kSlabHalfBytes;   // the slab before the tile
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk) {
                        const uint32_t koff = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
                        umma_bf16(dmain, umma_desc_sw128(a0 + koff), umma_desc_sw128(b0 + koff), idesc192, kk > 0);
                    }
                    const uint32_t pa = ring_a + (uint32_t)(1 + 2 * (int)((n - 1) % kSlots)) * kSlabHalfBytes;
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk) {
                        const uint32_t koff = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
                        umma_bf16(tmem + kColCorner, umma_desc_sw128(pa + koff), umma_desc_sw128(a0 + koff), idesc64,
                                  kk > 0);
                    }
                    ++nC;
                }
                umma_commit(&s->tfull[par]);
                if (!flush()) return;
                pend_slot = slot;
                pend_real = tl > 0;
            }
        } else {
            // nothing of a first-touch item may wait behind a second-touch tile
            if (!flush()) return;
            for (int tl = 0; tl < it.ntiles; ++tl, ++n, ++nB) {
                const int slot = (int)(n % kSlots), b = (int)(nB & 1);
                if (!bwait(&s->full[slot], (uint32_t)((n / kSlots) & 1), wt, 747)) return;
                if (!bwait(&s->rready[b], (uint32_t)((nB >> 1) & 1), wt, 748)) return;
                if (!bwait(&s->dempty[b], (uint32_t)(((nB >> 1) & 1) ^ 1), wt, 749)) return;
                tc_fence_after();
                const uint32_t a0 = ring_a + (uint32_t)(1 + 2 * slot) * kSlabHalfBytes;
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk) {
                    const uint32_t koff = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
                    const uint64_t bdesc = umma_desc_sw128(rhs_a + (uint32_t)b * kOperandBytes +
                                                           (uint32_t)(kk >> 2) * 2048u + (uint32_t)(kk & 3) * 32u);
                    umma_bf16(tmem + kColDots + 16u * (uint32_t)b, umma_desc_sw128(a0 + koff), bdesc, idesc16, kk > 0);
                }
                umma_commit(&s->dfull[b]);
                umma_commit(&s->rfree[b]);
                umma_commit(&s->sfree[slot]);
            }
        }
    }
    // every product issued has completed before the accumulators are given back
    umma_commit(&s->drain);
    bwait(&s->drain, 0, wt, 750);
}

// ---------------------------------------------------------------------------- band group
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

// The CTA that completed a head's last piece: head sum, 1/||head sum||, 1/||block sum|| (256 threads).
__device__ void finalise_head(Smem* s, const KeyPassArgs& p, int u, int tid) {
    const int nb = p.sp.nblocks;
    const float* bs = p.block_sums + (size_t)u * nb * kD;
    const int c = tid & (kD - 1), half = tid >> 7, warp = tid >> 5, lane = tid & 31;
    float sum = 0.f, comp = 0.f;   // compensated: the head sum is the anchor of every key of the head
    for (int b = half; b < nb; b += 2) {
        const float y = __ldcg(bs + (size_t)b * kD + c) - comp;
        const float t = sum + y;
        comp = (t - sum) - y;
        sum = t;
    }
    s->fin[half][c] = sum;
    bar_sync(kBarBand, kBandThreads);
    if (tid < kD) {
        const float tot = s->fin[0][c] + s->fin[1][c];
        p.head_sum[(size_t)u * kD + c] = tot;
        s->fin[0][c] = tot;
    }
    bar_sync(kBarBand, kBandThreads);
    if (warp == 0) {
        const float4 v = *reinterpret_cast<const float4*>(&s->fin[0][4 * lane]);
        const float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
        if (lane == 0) p.inv_s[u] = 1.0f / fmaxf(sqrtf(ss), kEps);
    }
    for (int b = warp; b < nb; b += kBandThreads / 32) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(bs + (size_t)b * kD) + lane);
        const float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
        if (lane == 0) p.inv_e[(size_t)u * nb + b] = 1.0f / fmaxf(sqrtf(ss), kEps);
    }
}

__device__ void band_role(unsigned char* wsplit, Smem* s, uint32_t tmem, const KeyPassArgs& p, const Waiter& wt) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q = warp & 3, side = warp >> 2;   // quarter of the tile's rows; 0 backward band, 1 forward band
    const int r = q * 32 + lane;                // row of the tile
    const int N = p.N, nb = p.sp.nblocks, blk_len = p.sp.block;
    const uint32_t lane_base = (uint32_t)(32 * q) << 16;
    long long ic = 0, nA = 0, nW = 0, nS = 0;   // items, first-touch tiles, split norms written, block sums read
    float carry = 0.f;   // forward sums of this thread's row of the previous tile over that tile's own columns
    for (;;) {
        Item it;
        const bool got = get_item<true>(s, ic++, it, wt, 751);
        if (bar_or(kBarBand, kBandThreads, !got)) return;   // the group leaves together or not at all
        if (it.kind == kItemEnd) return;
        if (it.kind == kItemB) continue;
        const int u = it.u;
        float lo = INFINITY, hi = -INFINITY, run = 0.f;
        bool ok = true;
        // block sums of the previous real tile (backward side): thread r owns channel r
        auto take_block_sum = [&](int tlp) {
            const int b = (int)(nS & 1);
            ok = bwait(&s->bsfull[b], (uint32_t)((nS >> 1) & 1), wt, 752) && ok;
            tc_fence_after();
            float d[16];
            tmem_ld16(tmem + lane_base + kColBsum + 16u * (uint32_t)b, d);
            tmem_wait_ld(d);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s->bsempty[b]);
            ++nS;
            run += d[0] + d[1] + d[2];
            const int Rp = it.row0 + (tlp - 1) * kTile, end = Rp + kTile;
            if (end % blk_len == 0 || end >= N || tlp == it.ntiles) {
                p.block_sums[((size_t)u * nb + Rp / blk_len) * kD + r] = run;
                run = 0.f;
            }
        };
        for (int tl = 0; tl <= it.ntiles; ++tl, ++nA) {
            const int par = (int)(nA & 1);
            const bool real = tl > 0;
            const int R = it.row0 + (tl - 1) * kTile, i = R + r;
            const int wbase = (int)(nA & 3) * kTile;   // ring index of the tile's row 0
            const uint32_t dmain = tmem + lane_base + (par ? kColMain1 : kColMain0);
            ok = bwait(&s->tfull[par], (uint32_t)((nA >> 1) & 1), wt, 753) && ok;
            tc_fence_after();
            float wi = 0.f, gi = 0.f;
            if (side == 0) {
                // the diagonal of D is ||k_i||^2
                float v[32];
                tmem_ld32(dmain + (uint32_t)(32 * q + 64), v);
                tmem_wait_ld(v, v + 16);
                const float n2 = select_lane(v, lane);
                wi = (i >= 0 && i < N) ? 1.0f / fmaxf(sqrtf(n2), kEps) : 0.f;
                gi = wi * wi * n2;
                s->w[wbase + r] = wi;
                s->g[wbase + r] = gi;
                if (real) {
                    if (i < N) p.inv_norm[(size_t)u * N + i] = wi;
                    // w as hi + mid + lo in bf16: rows 0..2 of the block-sum product's second operand
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
            if (bar_or(kBarBand, kBandThreads, !ok)) return;   // norms of the tile are in the ring
            float X, Y, Z;
            if (side == 0) {
                if (real && lane == 0) mbar_arrive(&s->wsready[nW & 1]);
                const int c0 = 32 * q;
                band_sums3(dmain + c0, dmain + c0 + 32, dmain + c0 + 64, s->w, wbase - 64 + c0, wbase - 32 + c0,
                           wbase + c0, lane + 1, X, Y, Z);
                s->c[par][r] = wi * (X + Y + Z);
                if (q >= 2) {
                    // Gram block of the tile's last 64 rows: the next tile's exact restart value
                    const float bp = wi * (q == 2 ? Z : Y + Z);
                    const float ap = warp_sum(2.f * bp - gi);
                    if (lane == 0) s->apart[par ^ 1][q - 2] = ap;
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
                const float wr = s->w[wbase + r];
                if (q < 2) {
                    s->fcur[par][r] = wr * (X + Y + Z);
                } else {
                    const float wprev = s->w[(wbase - kTile + r) & kWMask];
                    const float late = q == 2 ? Z : Y + Z, now = q == 2 ? X + Y : X;
                    s->fprev[par][r - 64] = wprev * (carry + late);
                    carry = now;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&s->tempty[par]);
                if (side == 1 && q >= 2 && real) mbar_arrive(&s->cempty);
            }
            if (bar_or(kBarBand, kBandThreads, !ok)) return;   // band sums of the tile are written
            if (real) ++nW;
            if (side == 0) {
                if (tl >= 2) take_block_sum(tl - 1);
            } else {
                // T_i = restart + prefix of (2 c_i - g_ii) - (2 f_{i-64} - g_{i-64,i-64})
                const float ci = s->c[par][r];
                const float g0 = s->g[wbase + r];
                const float fm = r < 64 ? s->fprev[par][r] : s->fcur[par][r - 64];
                const float gm = s->g[(wbase + r - 64) & kWMask];
                float x = 2.f * ci - g0 - (2.f * fm - gm);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float y = __shfl_up_sync(0xffffffffu, x, o);
                    if (lane >= o) x += y;
                }
                if (lane == 31) s->wtot[par][q] = x;
                bar_sync(kBarFwd, 128);
                float base = s->apart[par][0] + s->apart[par][1];
                for (int w = 0; w < q; ++w) base += s->wtot[par][w];
                const float Ti = base + x;
                if (real && i < N) {
                    const float a_c = -ci / fmaxf(sqrtf(fmaxf(Ti, 0.f)), kEps) + 0.f;
                    p.a_raw[((size_t)u * 3 + 2) * N + i] = a_c;
                    lo = fminf(lo, a_c);
                    hi = fmaxf(hi, a_c);
                }
            }
        }
        // ---- end of the piece
        if (side == 0) {
            take_block_sum(it.ntiles);
        } else {
            lo = warp_min(lo);
            hi = warp_max(hi);
            if (lane == 0) {
                s->red[2 * q] = lo;
                s->red[2 * q + 1] = hi;
            }
        }
        __threadfence();
        if (bar_or(kBarBand, kBandThreads, !ok)) return;
        if (tid == 128) {
            for (int w = 0; w < 4; ++w) {
                lo = fminf(lo, s->red[2 * w]);
                hi = fmaxf(hi, s->red[2 * w + 1]);
            }
            if (lo <= hi) {
                atomicMin(&p.mm[(size_t)u * 6 + 4], ord_key(lo));
                atomicMax(&p.mm[(size_t)u * 6 + 5], ord_key(hi));
            }
        }
        if (tid == 0) {
            __threadfence();
            s->fin_flag = atomicAdd(&p.head_count[u], 1) == p.pieces - 1;
        }
        bar_sync(kBarBand, kBandThreads);
        if (s->fin_flag) {   // every piece of the head is done, by this CTA or by others
            __threadfence();
            finalise_head(s, p, u, tid);
            __threadfence();
            bar_sync(kBarBand, kBandThreads);
            if (tid == 0 && !(p.debug & 1)) {
                __threadfence();
                atomicExch(&p.head_ready[u], 1);
            }
        }
    }
}

// ---------------------------------------------------------------------------- second touch
__device__ __forceinline__ int ld_acquire(const int* ptr) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// Thread k writes column k of the six anchor rows of every tile (rows 6..15 stay zero): the head sum and the
// sum of the tile's block, each as hi + mid + lo in bf16.
__device__ void prep_role(unsigned char* rhs, Smem* s, const KeyPassArgs& p, const Waiter& wt) {
    const int k = threadIdx.x - kPrepWarp0 * 32, lane = k & 31;
    const int half = k >> 6, kk = k & 63;
    long long ic = 0, nB = 0;
    bool degraded = false;
    for (;;) {
        Item it;
        if (!get_item<true>(s, ic++, it, wt, 761)) return;
        if (it.kind == kItemEnd) return;
        if (it.kind == kItemA) continue;
        if (!degraded) {
            uint32_t ns = 64;
            uint32_t spin = 0;
            while (ld_acquire(&p.head_ready[it.u]) == 0) {
                if (*wt.abort) return;
                if (++spin > p.flag_spin_limit) {
                    set_status(p.status, NKV_ERR_TIMEOUT, 762);
                    degraded = true;   // go on with what the buffers hold, wait for no further flag
                    break;
                }
                __nanosleep(ns);
                if (ns < 1024) ns <<= 1;
            }
        }
        float v[2] = {0.f, 0.f};
        v[0] = __ldcg(&p.head_sum[(size_t)it.u * kD + k]);
        int cur_blk = -1;
        for (int tl = 0; tl < it.ntiles; ++tl, ++nB) {
            const int b = (int)(nB & 1);
            if (!bwait(&s->rfree[b], (uint32_t)(((nB >> 1) & 1) ^ 1), wt, 763)) return;
            const int blk = (it.row0 + tl * kTile) / p.sp.block;
            if (blk != cur_blk) {
                v[1] = __ldcg(&p.block_sums[((size_t)it.u * p.sp.nblocks + blk) * kD + k]);
                cur_blk = blk;
            }
            unsigned char* base = rhs + (size_t)b * kOperandBytes + (size_t)half * 2048 + (kk & 7) * 2;
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
            if (lane == 0) mbar_arrive(&s->rready[b]);
        }
    }
}

// Thread r reads row r of the accumulator: the key's dots with the head sum and with its block's sum.
__device__ void epilogue_role(Smem* s, uint32_t tmem, const KeyPassArgs& p, const Waiter& wt) {
    const int r = threadIdx.x - kEpiWarp0 * 32, q = r >> 5, lane = r & 31;
    const int N = p.N, nb = p.sp.nblocks;
    long long ic = 0, nB = 0;
    for (;;) {
        Item it;
        if (!get_item<true>(s, ic++, it, wt, 771)) return;
        if (it.kind == kItemEnd) return;
        if (it.kind == kItemA) continue;
        const int u = it.u;
        float lo_s = INFINITY, hi_s = -INFINITY, lo_e = INFINITY, hi_e = -INFINITY;
        float rs = 0.f;
        for (int tl = 0; tl < it.ntiles; ++tl, ++nB) {
            const int b = (int)(nB & 1);
            if (!bwait(&s->dfull[b], (uint32_t)((nB >> 1) & 1), wt, 772)) return;
            tc_fence_after();
            // the accumulator exists, so the head's flag has been seen: its anchors and norms are final
            const int i = it.row0 + tl * kTile + r;
            const float wi = i < N ? __ldcg(&p.inv_norm[(size_t)u * N + i]) : 0.f;
            const float re = __ldcg(&p.inv_e[(size_t)u * nb + (it.row0 + tl * kTile) / p.sp.block]);
            if (tl == 0) rs = __ldcg(&p.inv_s[u]);
            float d[16];
            tmem_ld16(tmem + ((uint32_t)(32 * q) << 16) + kColDots + 16u * (uint32_t)b, d);
            tmem_wait_ld(d);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s->dempty[b]);
            const float a_s = -((d[0] + d[1] + d[2]) * wi) * rs + 0.f;
            const float a_e = -((d[3] + d[4] + d[5]) * wi) * re + 0.f;
            if (i < N) {
                p.a_raw[((size_t)u * 3 + 0) * N + i] = a_s;
                p.a_raw[((size_t)u * 3 + 1) * N + i] = a_e;
                lo_s = fminf(lo_s, a_s);
                hi_s = fmaxf(hi_s, a_s);
                lo_e = fminf(lo_e, a_e);
                hi_e = fmaxf(hi_e, a_e);
            }
        }
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
            mbar_init(&s->qfull[i], 1);
            mbar_init(&s->qfree[i], kConsumerWarps);
        }
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(&s->full[i], 1);
            mbar_init(&s->sfree[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s->tfull[i], 1);
            mbar_init(&s->tempty[i], 8);
            mbar_init(&s->wsready[i], 4);
            mbar_init(&s->bsfull[i], 1);
            mbar_init(&s->bsempty[i], 4);
            mbar_init(&s->rready[i], 4);
            mbar_init(&s->rfree[i], 1);
            mbar_init(&s->dfull[i], 1);
            mbar_init(&s->dempty[i], 4);
        }
        mbar_init(&s->cempty, 2);
        mbar_init(&s->drain, 1);
        s->abort = 0;
        s->fin_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows of the two 16-row operands that are never written must read as zeros
    for (int i = tid; i < 4 * kOperandBytes / 16; i += kThreads) reinterpret_cast<uint4*>(wsplit)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < kWRing; i += kThreads) {
        s->w[i] = 0.f;
        s->g[i] = 0.f;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == kMmaWarp) tmem_alloc(&s->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s->tmem_base;
    Waiter wt;
    wt.status = p.status;
    wt.abort = &s->abort;

    if (warp == kProducerWarp) {
        if (lane == 0) producer_role(&tmap, ring, s, p, wt);
        __syncwarp();
    } else if (warp == kMmaWarp) {
        if (lane == 0) mma_role(ring, wsplit, rhs, s, tmem, wt);
        __syncwarp();
    } else if (warp >= kPrepWarp0) {
        prep_role(rhs, s, p, wt);
    } else if (warp >= kEpiWarp0) {
        epilogue_role(s, tmem, p, wt);
    } else {
        band_role(wsplit, s, tmem, p, wt);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
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
                           float* block_sums, float* head_sum, float* inv_s, float* inv_e, float* inv_norm,
                           float* a_raw, uint32_t* mm, int* ctrl, int* status, int sm_count, cudaStream_t stream,
                           int64_t* launches) {
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
    int tpp = opt.tiles_per_piece > 0 ? opt.tiles_per_piece : 8;
    if (opt.tiles_per_piece <= 0)
        while (tpp > tiles_per_block && (int64_t)units * ((T + tpp - 1) / tpp) < 4LL * sm_count) tpp >>= 1;
    tpp = (tpp + tiles_per_block - 1) / tiles_per_block * tiles_per_block;
    a.tiles_per_piece = tpp;
    a.pieces = (T + tpp - 1) / tpp;
    const int64_t total = (int64_t)units * a.pieces;
    const unsigned grid = (unsigned)(total < sm_count ? total : sm_count);
    // the second touch of a head starts once its last piece has had time to finish: one head's pieces plus
    // one round of the grid behind the first touch
    a.lag_items = opt.lag_items > 0 ? opt.lag_items : (long long)a.pieces + (long long)grid + grid / 4;
    a.hints = opt.hints;
    a.debug = opt.debug;
    a.flag_spin_limit = opt.flag_spin_limit > 0 ? (uint32_t)opt.flag_spin_limit : (1u << 20);
    a.block_sums = block_sums;
    a.head_sum = head_sum;
    a.inv_s = inv_s;
    a.inv_e = inv_e;
    a.inv_norm = inv_norm;
    a.a_raw = a_raw;
    a.mm = mm;
    a.next_item = reinterpret_cast<unsigned long long*>(ctrl);
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
