// First key pass on the tensor cores (bf16 keys, d = 128, window W = 64).
//
// What the pass computes (Sections 2.1-2.3): 1/||k_i||, the sums of normalised keys of every episodic
// block, and the current-memory anomaly a_c(i) = -cos(k_hat_i, mu_c(i)) with its per-head min/max, where
// mu_c(i) is the mean of the last W normalised keys.  With S_i the sum of that window,
//     k_hat_i . S_i = sum_{j in window(i)} g_ij          g_ij = k_hat_i . k_hat_j
//     ||S_i||^2     = sum_{j, l in window(i)} g_jl
// so both are sums over a band of the Gram matrix of the keys.  The raw Gram entries G_ij = k_i . k_j are
// products of bf16 numbers summed in fp32, which is what tcgen05.mma does, so the band comes out of the
// tensor cores at no cost in instruction issue: g_ij = w_i w_j G_ij with w_i = 1/||k_i||.
//
// One CTA walks a head front to back in tiles of 128 keys.  Keys are staged by TMA in slabs of 64 rows
// (128-byte swizzle, two 64-column halves) in a ring of eight slabs (the first two have second copies behind
// the last, so that every run of four slabs is contiguous), so every key is fetched once.  For tile t the MMA
// warp forms D = K[tile rows] x K[64 rows before .. 64 rows after]^T (128 x 256, fp32 in tensor memory, double
// buffered, one N = 256 product per 16-wide K step).  The diagonal of D holds ||k||^2 of the tile's rows, so the
// norms cost no pass over the key values.  Row r of D gives
//     c_r = sum of g over the 64 columns ending at the diagonal       (= k_hat . S, backward band)
//     f_r = sum of g over the 64 columns starting at the diagonal     (forward band)
// and ||S_i||^2 follows from T_i = T_{i-1} + (2 c_i - g_ii) - (2 f_{i-W} - g_{i-W,i-W}), a prefix sum over
// the tile that restarts every tile from an exact value (the sum of the 64 x 64 Gram block that ends at
// the previous tile's last row, which is in that tile's D).  The forward band of a tile's rows 64..127 reaches
// 64 rows into the next tile, whose norms are not known yet: those Gram entries wait in shared memory and are
// added one tile later (f is read with a lag of 64 rows anyway).  Only the sums of normalised keys need the key
// values themselves and stay on the FMA pipes.
//
// The CTA is a pipeline of warp groups:
//     producer (1 thread)  TMA loads of the slabs
//     mma      (1 thread)  the Gram rectangle of the tile
//     diag     (4 warps)   1/||k|| and g_ii from the diagonal of D; block sums out of the segment sums
//     band     (8 warps)   c_r, f_r and the row's part of the next exact restart value from D
//     sums     (4 warps)   sums of normalised keys per eight-row segment
//     scan     (4 warps)   prefix sum, a_c, outputs, min/max
// Groups hand work to each other through mbarriers; every wait is bounded and a group that gives up
// records where and leaves, which makes the others give up in turn.  The busiest unit is the shared-memory
// data pipe (operand reads of the MMAs, the copies landing, the segment sums' key reads, barrier polls).  Outer
// loops are kept rolled and the kernel's code under 48 KB: with all groups running different code a kernel of
// 66 KB starved on instruction fetch.
#include "nkv_sm100.cuh"

namespace nkv {

namespace {

using namespace sm100;

constexpr int kD = 128;                       // head dimension
constexpr int kTile = 128;                    // keys per tile (rows of D)
constexpr int kSlabRows = 64;                 // rows per staged slab
constexpr int kRing = 8;                      // slabs in the ring
constexpr int kSlabHalfBytes = kSlabRows * 128;             // one 64-column half of a slab
constexpr int kMirror = 2;                                  // positions 8 and 9 hold second copies of positions 0 and 1,
                                                            // so that a run of up to four slabs that starts at
                                                            // position 6 or 7 is contiguous too
constexpr int kHalfBytes = (kRing + kMirror) * kSlabHalfBytes;   // all slabs of one half are contiguous
constexpr int kRingBytes = 2 * kHalfBytes;
constexpr int kBandThreads = 256, kDiagThreads = 128, kSumsThreads = 128, kScanThreads = 128;
constexpr int kDiagWarp0 = 8, kSumsWarp0 = 12, kScanWarp0 = 16, kProducerWarp = 20, kMmaWarp = 21;
constexpr int kThreads = 22 * 32;
constexpr int kWRing = 1024;                  // per-row scalars kept in rings of 1024 rows (band and scan are at most four tiles apart)
constexpr int kCfRing = 4;                    // band -> scan hand-over buffers
constexpr int kWReady = 8;                    // band -> sums hand-over barriers (1/||k|| of a tile published)
constexpr int kPpRing = 4, kPpShift = 2;      // sums -> diag hand-over buffers (segment sums of a tile)
constexpr int kStashFloats = 16 * 32 * 4;     // per warp: 16 four-float slots per lane
constexpr uint32_t kTmemCols = 512;           // two accumulators of 256 columns
constexpr int kBarDiag = 1, kBarBand = 2, kBarScan = 3, kBarSums = 4;   // named barriers

struct Smem {
    float pp[kPpRing][16 * kD];  // sums of normalised keys of the 16 eight-row segments of a tile
    float stash[2][kStashFloats];   // [lane quarter 2, 3] Gram entries whose column weights the next tile brings (forward band
                                    // of rows 64..127)
    float w[kWRing];             // 1/||k|| by row (0 outside the head)
    float g[kWRing];             // g_ii by row
    float c[kCfRing][kTile];     // backward band sums of a tile
    float f[kCfRing][kTile];     // forward band sums of a tile
    float bp[kCfRing][kTile];    // row's share of the Gram block of the tile's last 64 rows
    float anchor[2];             // exact ||S||^2 at the last row of the previous tile
    float wtot[2][4];            // per-warp totals of a tile's prefix sum
    float apart[2][4];           // per-warp parts of the next anchor
    float red[16];               // min/max reduction at the end of a head
    uint64_t full[kRing];        // slab landed
    uint64_t sfree[kRing];       // slab no longer needed (one arrival from the MMAs, one from the sums group)
    uint64_t tfull[2];           // accumulator written
    uint64_t tempty[2];          // accumulator read
    uint64_t wready[kWReady];    // 1/||k|| of a tile written
    uint64_t cready[kCfRing];    // band sums of a tile written
    uint64_t cfree[kCfRing];     // band sums of a tile consumed
    uint64_t ppfree[kPpRing];    // segment sums of a tile consumed
    uint64_t ppready[kPpRing];   // segment sums of a tile written
    uint64_t drain;              // products issued before a give-up have completed
    uint32_t tmem_base;
};
constexpr size_t kSmemBytes = 1024 + kRingBytes + sizeof(Smem);

// Slab q of a CTA's slab sequence sits at ring position p and is the fc-th use of that position.  A head
// starts at an even q, so the four slabs that a tile's product reads as B start at an even position and the
// two slabs of its own rows (A) at an odd one.
__device__ __forceinline__ void slab_slot(uint32_t q, int& p, uint32_t& fc) {
    p = (int)(q & 7);
    fc = (uint32_t)(q >> 3);
}

// The per-row rings (1/||k||, g_ii) are indexed by a row count that keeps running from head to head, so
// that the first rows of a head never land on entries the last tiles of the previous head still read.
// A head uses rows -64 .. 128 T + 127.
__device__ __forceinline__ int ring_advance(int T) { return kTile * (T + 2); }

// Transposed reduction of V per-lane partial values over a group of L lanes (L, V powers of two, V <= L):
// afterwards lane l holds in v[0] the complete sum of value l / (L/V).
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

// ---------------------------------------------------------------------------- producer and MMA
// TMA producer (one thread): the slabs of every head of this CTA, in order.  Slab lam of a head holds
// rows [64 (lam - 1), 64 lam); rows outside [0, N) arrive as zeros.
__device__ void producer_role(const CUtensorMap* tmap, unsigned char* ring, Smem* s, int units, int H, int T,
                              int* status) {
    uint32_t q = 0;
    const uint64_t policy = l2_evict_first_policy();   // keys are read once per pass
#pragma unroll 1
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        const int g = u / H, h = u - g * H;
#pragma unroll 1
        for (int lam = 0; lam < 2 * T + 2; ++lam, ++q) {
            int p;
            uint32_t fc;
            slab_slot(q, p, fc);
            if (fc > 0 && !mbar_wait(&s->sfree[p], (fc - 1) & 1u, status, 701)) {
                // giving up: the copies already armed still land in this CTA's shared memory, so stay (bounded)
                // until the last ring of them has
#pragma unroll 1
                for (uint32_t m = q > kRing ? q - kRing : 0; m < q; ++m) {
                    int pm;
                    uint32_t fm;
                    slab_slot(m, pm, fm);
#pragma unroll 1
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try_wait(&s->full[pm], fm & 1u); ++spin) __nanosleep(256);
                }
                return;
            }
            mbar_expect_tx(&s->full[p], (p < kMirror ? 4 : 2) * kSlabHalfBytes);
#pragma unroll 1
            for (int copy = 0; copy < (p < kMirror ? 2 : 1); ++copy) {
                unsigned char* dst = ring + (size_t)(copy ? kRing + p : p) * kSlabHalfBytes;
                tma_load_4d(dst, tmap, 0, kSlabRows * (lam - 1), h, g, &s->full[p], policy);
                tma_load_4d(dst + kHalfBytes, tmap, 64, kSlabRows * (lam - 1), h, g, &s->full[p], policy);
            }
        }
    }
}

// MMA issuer (one thread).  Tile tau of a head: A = slabs 2 tau + 1, 2 tau + 2 (the tile's rows),
// B = slabs 2 tau .. 2 tau + 3, one MMA of N = 256 per 16-wide K step (half the operand reads of A and half the
// instructions of two N = 128 products).
// Products already issued keep reading shared memory and writing tensor memory: a role that gives up
// waits (bounded) for them before the CTA frees both.
__device__ __forceinline__ void drain_products(Smem* s) {
    umma_commit(&s->drain);
#pragma unroll 1
    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try_wait(&s->drain, 0); ++spin) __nanosleep(256);
}

__device__ void mma_role(unsigned char* ring, Smem* s, uint32_t tmem_base, int units, int T, int* status) {
    constexpr uint32_t idesc = umma_idesc_bf16(kTile, 256);
    const uint32_t ring_addr = smem_addr(ring);
    uint32_t hb = 0, gt = 0;
#pragma unroll 1
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
#pragma unroll 1
        for (int tau = 0; tau < T; ++tau, ++gt) {
            int p;
            uint32_t fc;
#pragma unroll 1
            for (int lam = tau == 0 ? 0 : 2 * tau + 2; lam <= 2 * tau + 3; ++lam) {
                slab_slot(hb + lam, p, fc);
                if (!mbar_wait(&s->full[p], fc & 1u, status, 702)) return drain_products(s);
            }
            const int st = (int)(gt & 1);
            if (!mbar_wait(&s->tempty[st], (uint32_t)(((gt >> 1) & 1) ^ 1), status, 703)) return drain_products(s);
            tc_fence_after();
            int pa, pb;   // odd and even; what follows position 7 is read from the copies at positions 8 and 9
            slab_slot(hb + 2 * tau + 1, pa, fc);
            slab_slot(hb + 2 * tau, pb, fc);
            // the address field of a descriptor counts 16-byte units: a K step moves it by a constant
            const uint64_t adesc = umma_desc_sw128(ring_addr + (uint32_t)pa * kSlabHalfBytes);
            const uint64_t bdesc = umma_desc_sw128(ring_addr + (uint32_t)pb * kSlabHalfBytes);
#pragma unroll
            for (int kk = 0; kk < kD / 16; ++kk) {
                constexpr uint32_t kHalfUnits = kHalfBytes >> 4;
                const uint64_t koff = (uint64_t)((uint32_t)(kk >> 2) * kHalfUnits + (uint32_t)(kk & 3) * 2u);
                umma_bf16(tmem_base + (uint32_t)st * 256u, adesc + koff, bdesc + koff, idesc, kk > 0);
            }
            umma_commit(&s->tfull[st]);
#pragma unroll 1
            for (int lam = 2 * tau; lam <= (tau == T - 1 ? 2 * tau + 3 : 2 * tau + 1); ++lam) {
                slab_slot(hb + lam, p, fc);
                umma_commit(&s->sfree[p]);
            }
        }
        hb += 2 * T + 2;
    }
}

// ---------------------------------------------------------------------------- sums group
// Segment sums of normalised keys of the tile's 128 rows, held by ring positions p0 (first 64 rows) and p1.
// Lane group grp (16 lanes, 8 columns per lane) takes the 8 rows of segment grp; 1/||k|| of the rows comes from
// the ring the band group has filled from the diagonal of the tile's Gram block.
__device__ __forceinline__ void tile_segment_sums(const unsigned char* ring, int p0, int p1, const float* wring, float* pp,
                                                  int wrow_tile, int grp, int l) {
    const int pos = grp < 8 ? p0 : p1;
    const unsigned char* base = ring + (size_t)(l >> 3) * kHalfBytes + (size_t)pos * kSlabHalfBytes;
    const int w0 = (wrow_tile + grp * 8) & (kWRing - 1);   // a multiple of 8: the eight weights are contiguous
    const float4 wa = *reinterpret_cast<const float4*>(wring + w0), wb = *reinterpret_cast<const float4*>(wring + w0 + 4);
    const float ir[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
    F2 acc[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) acc[p] = pack2(0.f, 0.f);
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const int rs = (grp & 7) * 8 + r;   // row inside the slab
        const uint4 q = *reinterpret_cast<const uint4*>(base + rs * 128 + (((l & 7) ^ (rs & 7)) << 4));
        F2 x[4];
        unpack_bf16x8(q, x);
        const F2 ir2 = pack2(ir[r], ir[r]);
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[p] = fma2(x[p], ir2, acc[p]);
    }
    float* dst = pp + grp * kD + l * 8;
    float4 o0, o1;
    unpack2(acc[0], o0.x, o0.y);
    unpack2(acc[1], o0.z, o0.w);
    unpack2(acc[2], o1.x, o1.y);
    unpack2(acc[3], o1.z, o1.w);
    *reinterpret_cast<float4*>(dst) = o0;
    *reinterpret_cast<float4*>(dst + 4) = o1;
}

// 1/||k|| and g_ii of the tile's rows from the diagonal of its Gram block: row lr of lane quarter q has its
// diagonal at column 64 + 32 q + lr of D, which in the fragment layout is held by the thread with
// t % 4 == t / 8 (element e = (t / 4) % 2 of the column pair k == J).
__device__ __forceinline__ void publish_norms(Smem* s, uint32_t tq, int q, int t, int wrow_tile, int R0, int N) {
    const bool owner = (t & 3) == (t >> 3);
    const int e = (t >> 2) & 1;
    float cc[2][16];
    tmem_ld_frag32(tq + (uint32_t)(64 + 32 * q), cc[0]);
    tmem_ld_frag32(tq + (16u << 16) + (uint32_t)(64 + 32 * q), cc[1]);
    tmem_wait_ld(cc[0], cc[1]);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const float* c = cc[half];
        if (owner) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int J = 2 * half + j;
                const float G = e ? c[4 * J + 2 * j + 1] : c[4 * J + 2 * j];
                const int row = 32 * q + 8 * J + (t >> 2);
                const float inv = R0 + row < N ? rsqrtf(fmaxf(G, kEps * kEps)) : 0.f;   // 1 / max(||k||, eps)
                s->w[(wrow_tile + row) & (kWRing - 1)] = inv;
                s->g[(wrow_tile + row) & (kWRing - 1)] = inv * inv * G;
            }
        }
    }
}

// sum of v[sg] over a <= sg < b (16 segment sums in registers), as a tree
__device__ __forceinline__ float segment_range_sum(const float* v, int a, int b) {
    float p[16];
#pragma unroll
    for (int sg = 0; sg < 16; ++sg) p[sg] = (sg >= a && sg < b) ? v[sg] : 0.f;
#pragma unroll
    for (int w = 8; w >= 1; w >>= 1)
#pragma unroll
        for (int sg = 0; sg < w; ++sg) p[sg] += p[sg + w];
    return p[0];
}

// Block sums of column `col` over one span (rows [R1, R1 + 128), 16 segment sums in pp): a block that closes
// inside the span is written out, the rest of the span starts the next one (rows outside the head are zeros).
struct BlockWalk {
    float run;     // running sum of the open block
    int blk;       // the open block
    int blk_end;   // the row it ends before
};

__device__ __noinline__ BlockWalk span_block_sums(const float* pp, int R1, int col, int nblocks, int block, int N,
                                                  float* __restrict__ head_sums, BlockWalk bw) {
    // everything by value: a walk kept behind a reference would live in local memory, which this kernel's
    // shared-memory carve-out leaves almost no L1 for
    float v[16], tr[16];
#pragma unroll
    for (int sg = 0; sg < 16; ++sg) tr[sg] = v[sg] = pp[sg * kD + col];
#pragma unroll
    for (int w = 8; w >= 1; w >>= 1)
#pragma unroll
        for (int sg = 0; sg < w; ++sg) tr[sg] += tr[sg + w];
    const float total = tr[0];   // the same tree as segment_range_sum(v, 0, 16)
    int s0 = 0;   // first segment not yet added
#pragma unroll 1
    while (bw.blk < nblocks && bw.blk_end <= R1 + kTile) {
        const int s1 = (bw.blk_end - R1 + kSeg - 1) / kSeg;   // segments [s0, s1) close the block
        // blocks of 128 or 256 rows end where tiles end: the whole tile, no masks
        bw.run += (s0 == 0 && s1 == 16) ? total : segment_range_sum(v, s0, s1);
        head_sums[bw.blk * kD + col] = bw.run;
        bw.run = 0.f;
        ++bw.blk;
        bw.blk_end = min(bw.blk_end + block, N);
        s0 = s1;
    }
    if (s0 == 0) bw.run += total;
    else if (s0 < 16) bw.run += segment_range_sum(v, s0, 16);
    return bw;
}

// Diagonal group (four warps, one per lane quarter): as soon as a tile's Gram rectangle is complete it reads the
// diagonal and publishes 1/||k|| of the tile's rows; the band group and the sums group wait for that.  In the time
// left it adds the segment sums of the previous tile up into block sums (one thread per column; the sums group
// runs a tile behind), and those of the head's last tile once they are there.
__device__ void diag_role(Smem* s, uint32_t tmem_base, ScoreParams sp, int units, int N, int T, float* __restrict__ block_sums,
                          int* status) {
    const int t = threadIdx.x - kDiagWarp0 * 32;
    const int q = t >> 5;
    uint32_t gt = 0;
    int rb = 64;   // ring index of the head's row 0 (see ring_advance)
#pragma unroll 1
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        BlockWalk bw = {0.f, 0, min(sp.block, N)};
        float* head_sums = block_sums + (int64_t)u * sp.nblocks * kD;
#pragma unroll 1
        for (int tau = 0; tau < T; ++tau, ++gt) {
            const bool ok = mbar_wait(&s->tfull[gt & 1], (uint32_t)((gt >> 1) & 1), status, 705);
            tc_fence_after();
            publish_norms(s, tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)((gt & 1) * 256), q, t & 31, rb + kTile * tau,
                          kTile * tau, N);
            if (tau == 0 && t < 64) {   // the 64 rows before a head weigh nothing
                s->w[(rb - 64 + t) & (kWRing - 1)] = 0.f;
                s->g[(rb - 64 + t) & (kWRing - 1)] = 0.f;
            }
            tc_fence_before();
            if (bar_or(kBarDiag, kDiagThreads, !ok)) return;
            if (t == 0) mbar_arrive(&s->wready[gt & (kWReady - 1)]);
            bool ok2 = true;
            if (tau > 0) {
                ok2 = mbar_wait(&s->ppready[(gt - 1) & (kPpRing - 1)], (uint32_t)(((gt - 1) >> kPpShift) & 1), status, 710);
                bw = span_block_sums(s->pp[(gt - 1) & (kPpRing - 1)], kTile * (tau - 1), t, sp.nblocks, sp.block, N, head_sums, bw);
            }
            if (tau == T - 1) {
                ok2 = ok2 && mbar_wait(&s->ppready[gt & (kPpRing - 1)], (uint32_t)((gt >> kPpShift) & 1), status, 710);
                bw = span_block_sums(s->pp[gt & (kPpRing - 1)], kTile * tau, t, sp.nblocks, sp.block, N, head_sums, bw);
            }
            if (tau > 0 || tau == T - 1) {
                if (bar_or(kBarDiag, kDiagThreads, !ok2)) return;
                if (t == 0) {   // every column of the segment sums has been read
                    if (tau > 0) mbar_arrive(&s->ppfree[(gt - 1) & (kPpRing - 1)]);
                    if (tau == T - 1) mbar_arrive(&s->ppfree[gt & (kPpRing - 1)]);
                }
            }
        }
        rb = (rb + ring_advance(T)) & (kWRing - 1);
    }
}

// Sums group (four warps).  Tile tau of a head: rows [128 tau, 128 tau + 128) = slabs 2 tau + 1 and 2 tau + 2; a
// lane group takes one segment of each slab.  The segment sums go to the scan group, which adds them up into block
// sums.  The slabs of a head that hold no rows of a tile (the first and the last) are released here too.
__device__ void sums_role(const unsigned char* ring, Smem* s, int units, int T, int* status) {
    const int t = threadIdx.x - kSumsWarp0 * 32;
    const int grp = t >> 4, l = t & 15;
    uint32_t hb = 0, gt = 0;
    int rb = 64;
#pragma unroll 1
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
#pragma unroll 1
        for (int tau = 0; tau < T; ++tau, ++gt) {
            int p0, p1;
            uint32_t fc0, fc1;
            slab_slot(hb + 2 * tau + 1, p0, fc0);
            slab_slot(hb + 2 * tau + 2, p1, fc1);
            const int pi = (int)(gt & (kPpRing - 1));
            bool ok = mbar_wait(&s->ppfree[pi], (uint32_t)(((gt >> kPpShift) & 1) ^ 1), status, 709);
            ok = ok && mbar_wait(&s->wready[gt & (kWReady - 1)], (uint32_t)((gt >> 3) & 1), status, 712);
            ok = ok && mbar_wait(&s->full[p0], fc0 & 1u, status, 704);   // complete long ago: makes the copies visible here
            ok = ok && mbar_wait(&s->full[p1], fc1 & 1u, status, 704);
#pragma unroll 1
            for (int sg = grp; sg < 16; sg += 8) tile_segment_sums(ring, p0, p1, s->w, s->pp[pi], rb + kTile * tau, sg, l);
            if (bar_or(kBarSums, kSumsThreads, !ok)) return;
            if (t == 0) {   // every thread is done with the two slabs and has written its segment sums
                mbar_arrive(&s->sfree[p0]);
                mbar_arrive(&s->sfree[p1]);
                mbar_arrive(&s->ppready[pi]);
                int pe;
                uint32_t fe;
                if (tau == 0) {
                    slab_slot(hb, pe, fe);
                    mbar_arrive(&s->sfree[pe]);
                }
                if (tau == T - 1) {
                    slab_slot(hb + 2 * T + 1, pe, fe);
                    mbar_arrive(&s->sfree[pe]);
                }
            }
        }
        hb += 2 * T + 2;
        rb = (rb + ring_advance(T)) & (kWRing - 1);
    }
}

// ---------------------------------------------------------------------------- band group
// Band sums of the 32 rows of one lane quarter of D.  Row lr of the quarter has its diagonal at column
// 64 + 32 q + lr.  side 0 sums the 64 columns that end at the diagonal, side 1 the 64 columns that start there;
// both live in three 32-column chunks starting at the column `taddr` points to, of which the first and the last
// are cut by the diagonal: column o of the first chunk counts when o >= lr + (side == 0), column o of the last
// when it does not.  Every column is weighted by its key's 1/||k||; row0 is the ring index of the first column's key.
//
// The accumulator is read in the fragment layout (tmem_ld_frag32): a thread holds columns 8 k + b0 + e
// (b0 = 2 (t % 4), k = 0..3, e = 0, 1) of the four rows lr = 8 J + t / 4.  The weights of its eight columns per
// chunk are two-float loads that eight lanes share, which costs a twelfth of the shared-memory wavefronts that a
// thread-per-row walk spends on broadcasting every weight to every row.  With r0 = t / 4 + (side == 0) the cut
// 8 k + b0 + e >= 8 J + r0 is decided by k alone unless k == J (0 <= b0 + e <= 7, 0 <= r0 <= 8): columns with
// k > J lie past the cut, columns with k < J before it, and the pair k == J is tested against r0.
// Afterwards lane t holds the three chunk sums of row 8 (t % 4) + t / 4 of the quarter.
struct ChunkSums {
    float x[2][2], y[2][2], z[2][2];   // [row pair j][column parity e] of the half being read
};

__device__ __forceinline__ void load_w8(const float* wring, int idx, float2* w) {
#pragma unroll
    for (int k = 0; k < 4; ++k) w[k] = *reinterpret_cast<const float2*>(wring + ((idx + 8 * k) & (kWRing - 1)));
}

template <int kChunk>
__device__ __forceinline__ void chunk_fma(const float* v, const float2* w, int half, bool p0, bool p1, ChunkSums& cs) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float v0 = v[4 * k + 2 * j], v1 = v[4 * k + 2 * j + 1];
            if (kChunk == 1) {
                cs.y[j][0] = fmaf(v0, w[k].x, cs.y[j][0]);
                cs.y[j][1] = fmaf(v1, w[k].y, cs.y[j][1]);
            } else {
                // J = 2 half + j is known only at run time as far as `half` goes; both halves are unrolled by the caller
                const int J = 2 * half + j;
                const bool past = k > J, at = k == J;
                if (kChunk == 0) {
                    if (past || at) {
                        cs.x[j][0] = fmaf((past || p0) ? v0 : 0.f, w[k].x, cs.x[j][0]);
                        cs.x[j][1] = fmaf((past || p1) ? v1 : 0.f, w[k].y, cs.x[j][1]);
                    }
                } else {
                    if (k < J || at) {
                        cs.z[j][0] = fmaf((k < J || !p0) ? v0 : 0.f, w[k].x, cs.z[j][0]);
                        cs.z[j][1] = fmaf((k < J || !p1) ? v1 : 0.f, w[k].y, cs.z[j][1]);
                    }
                }
            }
        }
    }
}

// X, Y, Z[J]: chunk sums of row 8 J + t / 4 over this thread's columns (to be added up over the four lanes t % 4).
// The weights of the last `deferred` chunks are not known yet (they belong to rows of the next tile): those Gram
// entries go to the thread's stash instead and finish_forward() adds them one tile later.
__device__ __forceinline__ void band_sums(int side, uint32_t taddr, const float* wring, int row0, int t, int deferred,
                                          float4* stash, float* X, float* Y, float* Z) {
    const int b0 = 2 * (t & 3), r0 = (t >> 2) + (side == 0 ? 1 : 0);
    const bool p0 = b0 >= r0, p1 = b0 + 1 >= r0;
    const int i0 = (row0 + b0) & (kWRing - 1);
    float a[16], b[16], c[16];
    float2 w[4];
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const uint32_t ta = taddr + ((uint32_t)(16 * half) << 16);
        ChunkSums cs;
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) cs.x[j][e] = cs.y[j][e] = cs.z[j][e] = 0.f;
        tmem_ld_frag32(ta, a);
        tmem_ld_frag32(ta + 32, b);
        tmem_wait_ld(a, b);
        tmem_ld_frag32(ta + 64, c);
        load_w8(wring, i0, w);
        chunk_fma<0>(a, w, half, p0, p1, cs);
        if (deferred < 2) {
            load_w8(wring, i0 + 32, w);
            chunk_fma<1>(b, w, half, p0, p1, cs);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) stash[(half * 8 + 4 + i) * 32] = make_float4(b[4 * i], b[4 * i + 1], b[4 * i + 2], b[4 * i + 3]);
        }
        tmem_wait_ld(c);
        if (deferred < 1) {
            load_w8(wring, i0 + 64, w);
            chunk_fma<2>(c, w, half, p0, p1, cs);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) stash[(half * 8 + i) * 32] = make_float4(c[4 * i], c[4 * i + 1], c[4 * i + 2], c[4 * i + 3]);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            X[2 * half + j] = cs.x[j][0] + cs.x[j][1];
            Y[2 * half + j] = cs.y[j][0] + cs.y[j][1];
            Z[2 * half + j] = cs.z[j][0] + cs.z[j][1];
        }
    }
}

// The stashed part of the previous tile's forward band (rows 64 .. 127 of that tile, lane quarter q = 2 or 3): its
// columns are this tile's rows 0 .. 31 (and 32 .. 63 for q = 3), whose 1/||k|| the ring holds now.  Returns in F[0]
// the sum for row 8 (t % 4) + t / 4 of the quarter.
__device__ __forceinline__ float finish_forward(const float4* stash, const float* wring, int wrow_tile, int q, int t) {
    const int b0 = 2 * (t & 3), r0 = t >> 2;
    const bool p0 = b0 >= r0, p1 = b0 + 1 >= r0;
    float F[4];
    float v[16];
    float2 w[4];
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        ChunkSums cs;
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) cs.x[j][e] = cs.y[j][e] = cs.z[j][e] = 0.f;
        if (q == 3) {   // the middle chunk: all of its columns count
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 f = stash[(half * 8 + 4 + i) * 32];
                v[4 * i] = f.x, v[4 * i + 1] = f.y, v[4 * i + 2] = f.z, v[4 * i + 3] = f.w;
            }
            load_w8(wring, wrow_tile + b0, w);
            chunk_fma<1>(v, w, half, p0, p1, cs);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = stash[(half * 8 + i) * 32];
            v[4 * i] = f.x, v[4 * i + 1] = f.y, v[4 * i + 2] = f.z, v[4 * i + 3] = f.w;
        }
        load_w8(wring, wrow_tile + (q == 3 ? 32 : 0) + b0, w);
        chunk_fma<2>(v, w, half, p0, p1, cs);
#pragma unroll
        for (int j = 0; j < 2; ++j) F[2 * half + j] = (cs.y[j][0] + cs.y[j][1]) + (cs.z[j][0] + cs.z[j][1]);
    }
    treduce<4, 4>(F, t & 3);
    return F[0];
}

__device__ __forceinline__ void band_tile(int side, Smem* s, uint32_t taddr, int wrow0, int wrow_tile, int q, int lane, int cb) {
    float X[4], Y[4], Z[4];
    const int deferred = side == 1 && q >= 2 ? q - 1 : 0;
    float4* stash = reinterpret_cast<float4*>(s->stash[q & 1]) + lane;
    band_sums(side, taddr, s->w, wrow0, lane, deferred, stash, X, Y, Z);
    float tot[4], part[4];
#pragma unroll
    for (int J = 0; J < 4; ++J) {
        tot[J] = X[J] + Y[J] + Z[J];
        part[J] = q == 2 ? Z[J] : Y[J] + Z[J];
    }
    treduce<4, 4>(tot, lane & 3);
    const int r = 32 * q + 8 * (lane & 3) + (lane >> 2);   // the row whose sums this lane now holds
    const float wi = s->w[(wrow_tile + r) & (kWRing - 1)];
    if (side == 0) {
        treduce<4, 4>(part, lane & 3);
        s->c[cb][r] = wi * tot[0];
        // Gram block of the tile's last 64 rows: columns 128 .. diagonal of rows 64 .. 127
        s->bp[cb][r] = q >= 2 ? wi * part[0] : 0.f;
    } else {
        s->f[cb][r] = wi * tot[0];
    }
}

// Per tile, once the sums group has published 1/||k|| of the tile's rows, every warp sums its band with those
// weights.  The forward band of rows 64 .. 127 reaches into the
// next tile: that part waits in the stash and is added to the row's forward sum when the next tile is here (the
// scan group reads those sums one tile later anyway; behind a head's last tile lie zero rows, nothing to add).
__device__ void band_role(Smem* s, uint32_t tmem_base, int units, int T, int* status) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q = warp & 3, side = warp >> 2;   // quarter of the tile's rows, backward / forward band
    uint32_t gt = 0;
    int rb = 64;
#pragma unroll 1
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
#pragma unroll 1
        for (int tau = 0; tau < T; ++tau, ++gt) {
            const int st = (int)(gt & 1), cb = (int)(gt & (kCfRing - 1));
            bool ok = mbar_wait(&s->cfree[cb], (uint32_t)(((gt >> 2) & 1) ^ 1), status, 706);
            ok = ok && mbar_wait(&s->tfull[st], (uint32_t)((gt >> 1) & 1), status, 707);
            ok = ok && mbar_wait(&s->wready[gt & (kWReady - 1)], (uint32_t)((gt >> 3) & 1), status, 711);
            tc_fence_after();
            const int R0 = kTile * tau;
            const uint32_t tq = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(st * 256);
            const int cA = 32 * q + 64 * side;   // first column of the first chunk
            if (side == 1 && q >= 2 && tau > 0) {   // before this tile's entries take the stash over
                const float F = finish_forward(reinterpret_cast<const float4*>(s->stash[q & 1]) + lane, s->w, rb + R0, q, lane);
                const int r = 32 * q + 8 * (lane & 3) + (lane >> 2);
                s->f[(gt - 1) & (kCfRing - 1)][r] += s->w[(rb + R0 - kTile + r) & (kWRing - 1)] * F;
            }
            band_tile(side, s, tq + (uint32_t)cA, rb + R0 - 64 + cA, rb + R0, q, lane, cb);
            tc_fence_before();
            if (bar_or(kBarBand, kBandThreads, !ok)) return;
            if (tid == 0) {
                mbar_arrive(&s->tempty[st]);
                mbar_arrive(&s->cready[cb]);
            }
        }
        rb = (rb + ring_advance(T)) & (kWRing - 1);
    }
}

// ---------------------------------------------------------------------------- scan group
// Thread r owns row r of the tile: T_i = anchor + prefix of (2 c_i - g_ii) - (2 f_{i-64} - g_{i-64,i-64}).
__device__ void scan_role(Smem* s, int units, int N, int T, float* __restrict__ inv_norm, float* __restrict__ a_raw,
                          uint32_t* __restrict__ mm, int* status) {
    const int r = threadIdx.x - kScanWarp0 * 32;
    const int q = r >> 5, lane = r & 31;
    uint32_t gt = 0;
    int rb = 64;
#pragma unroll 1
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        float lo = INFINITY, hi = -INFINITY;
        if (r == 0) s->anchor[gt & 1] = 0.f;
#pragma unroll 1
        for (int tau = 0; tau < T; ++tau, ++gt) {
            const int cb = (int)(gt & (kCfRing - 1)), pb = (int)((gt - 1) & (kCfRing - 1)), par = (int)(gt & 1);
            const bool ok = mbar_wait(&s->cready[cb], (uint32_t)((gt >> 2) & 1), status, 708);
            const int R0 = kTile * tau;
            const float gi = s->g[(rb + R0 + r) & (kWRing - 1)];
            const float wi = s->w[(rb + R0 + r) & (kWRing - 1)];
            const float ci = s->c[cb][r];
            float rem = 0.f;
            if (r >= 64) rem = 2.f * s->f[cb][r - 64] - s->g[(rb + R0 + r - 64) & (kWRing - 1)];
            else if (tau > 0) rem = 2.f * s->f[pb][r + 64] - s->g[(rb + R0 + r - 64) & (kWRing - 1)];
            float x = 2.f * ci - gi - rem;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float y = __shfl_up_sync(0xffffffffu, x, o);
                if (lane >= o) x += y;
            }
            const float ap = warp_sum(q >= 2 ? 2.f * s->bp[cb][r] - gi : 0.f);
            if (lane == 31) s->wtot[par][q] = x;
            if (lane == 0) s->apart[par][q] = ap;
            if (bar_or(kBarScan, kScanThreads, !ok)) return;
            // the previous tile's forward sums have been read by now
            if (r == 0 && gt > 0) mbar_arrive(&s->cfree[pb]);
            float base = s->anchor[par];
            for (int w = 0; w < q; ++w) base += s->wtot[par][w];
            const float Ti = base + x;
            const int i = R0 + r;
            if (i < N) {
                const float a_c = -ci * rsqrtf(fmaxf(Ti, kEps * kEps)) + 0.f;   // -c / max(||S||, eps)
                a_raw[((int64_t)u * 3 + 2) * N + i] = a_c;
                inv_norm[(int64_t)u * N + i] = wi;
                lo = fminf(lo, a_c);
                hi = fmaxf(hi, a_c);
            }
            if (r == 0) s->anchor[par ^ 1] = s->apart[par][2] + s->apart[par][3];
        }
        // ---- per-head min/max of a_c
        lo = warp_min(lo);
        hi = warp_max(hi);
        if (lane == 0) {
            s->red[2 * q] = lo;
            s->red[2 * q + 1] = hi;
        }
        bar_sync(kBarScan, kScanThreads);
        if (r == 0) {
            for (int w = 1; w < 4; ++w) {
                lo = fminf(lo, s->red[2 * w]);
                hi = fmaxf(hi, s->red[2 * w + 1]);
            }
            if (lo <= hi) {
                atomicMin(&mm[(int64_t)u * 6 + 4], ord_key(lo));
                atomicMax(&mm[(int64_t)u * 6 + 5], ord_key(hi));
            }
        }
        rb = (rb + ring_advance(T)) & (kWRing - 1);
    }
}

__global__ void __launch_bounds__(kThreads, 1)
gram_pass_kernel(const __grid_constant__ CUtensorMap tmap, ScoreParams sp, int units, int H, int N,
                 float* __restrict__ block_sums, float* __restrict__ inv_norm, float* __restrict__ a_raw,
                 uint32_t* __restrict__ mm, int* status) {
    extern __shared__ unsigned char smem_raw[];
    // the swizzle atoms (8 rows x 128 bytes) must start on 1024-byte boundaries
    unsigned char* ring = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    Smem* s = reinterpret_cast<Smem*>(ring + kRingBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = (N + kTile - 1) / kTile;

    if (tid == 0) {
        for (int i = 0; i < kRing; ++i) {
            mbar_init(&s->full[i], 1);
            mbar_init(&s->sfree[i], 2);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s->tfull[i], 1);
            mbar_init(&s->tempty[i], 1);
        }
        mbar_init(&s->drain, 1);
        for (int i = 0; i < kWReady; ++i) mbar_init(&s->wready[i], 1);
        for (int i = 0; i < kCfRing; ++i) {
            mbar_init(&s->cready[i], 1);
            mbar_init(&s->cfree[i], 1);
        }
        for (int i = 0; i < kPpRing; ++i) {
            mbar_init(&s->ppfree[i], 1);
            mbar_init(&s->ppready[i], 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) tmem_alloc(&s->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s->tmem_base;

    if (warp == kProducerWarp) {
        if (lane == 0) producer_role(&tmap, ring, s, units, H, T, status);
        __syncwarp();
    } else if (warp == kMmaWarp) {
        if (lane == 0) mma_role(ring, s, tmem_base, units, T, status);
        __syncwarp();
    } else if (warp >= kScanWarp0) {
        scan_role(s, units, N, T, inv_norm, a_raw, mm, status);
    } else if (warp >= kSumsWarp0) {
        sums_role(ring, s, units, T, status);
    } else if (warp >= kDiagWarp0) {
        diag_role(s, tmem_base, sp, units, N, T, block_sums, status);
    } else {
        band_role(s, tmem_base, units, T, status);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// reset of the per-head min/max keys
__global__ void gram_init_kernel(int units, uint32_t* mm) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < units * 6) mm[i] = (i & 1) ? 0u : 0xffffffffu;
}

}  // namespace

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once (the library does not link against the driver).
EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

// Tensor map of the keys [G][H][N][128] bf16 for boxes of 64 columns x box_rows rows, 128-byte swizzle.
cudaError_t encode_key_map(const TensorView& K, int G, int box_rows, CUtensorMap* out) {
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return cudaErrorNotSupported;
    const cuuint64_t dims[4] = {(cuuint64_t)K.d, (cuuint64_t)K.N, (cuuint64_t)K.H, (cuuint64_t)G};
    const cuuint64_t strides[3] = {(cuuint64_t)K.d * 2, (cuuint64_t)K.stride_h * 2, (cuuint64_t)K.stride_g * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(K.ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    return cudaSuccess;
}

cudaError_t configure_gram_kernels() {
    return cudaFuncSetAttribute(gram_pass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
}

// bf16 keys of 128 columns, the paper's window of 64, a block size the segment sums can follow, and
// strides a tensor map accepts (multiples of 16 bytes, base 16-byte aligned).
bool gram_pass_supported(const TensorView& K, int dtype, const ScoreParams& sp) {
    if (dtype != NKV_BF16 || K.d != kD || sp.window != 64 || sp.block % kSeg != 0) return false;
    if (reinterpret_cast<uintptr_t>(K.ptr) % 16 != 0) return false;
    if (K.stride_h % 8 != 0 || K.stride_g % 8 != 0) return false;
    if (K.stride_h < (int64_t)K.N * kD || K.stride_g < (int64_t)K.N * kD) return false;
    CUtensorMap probe;   // the driver has the last word on what a tensor map can describe
    return encode_key_map(K, 1, kSlabRows, &probe) == cudaSuccess;
}

cudaError_t launch_gram_pass(const TensorView& K, int G, const ScoreParams& sp, float* block_sums, float* inv_norm,
                             float* a_raw, uint32_t* mm, int* status, int sm_count, cudaStream_t stream,
                             int64_t* launches) {
    const int units = G * K.H;
    CUtensorMap tmap;
    cudaError_t e = encode_key_map(K, G, kSlabRows, &tmap);
    if (e != cudaSuccess) return e;
    gram_init_kernel<<<(units * 6 + 255) / 256, 256, 0, stream>>>(units, mm);
    ++*launches;
    const unsigned grid = (unsigned)(units < sm_count ? units : sm_count);
    gram_pass_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tmap, sp, units, K.H, K.N, block_sums, inv_norm, a_raw, mm,
                                                             status);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
