// Score-side kernels: everything that works on the per-token score arrays.
//
//   head_scores  (Sections 2.3-2.4)  min-max, reliability gaps (exact top/bottom-m sums),
//                                    softmax weights, surprise, gate, routed score, sink pin
//   budget       (Section 2.6)       per-head safeguard thresholds, cross-head competition
//   select       (Section 2.5)       TopB_h as an ordered stream compaction
//   ranks                            place of every token in its head's order (diagnostic)
//
// All order statistics are exact.  The selection primitive finds the rank-th largest
// element of a multiset of floats by counting into 2048 value-linear bins, refining the
// chosen bin up to three times (each level splits it 2048 ways again), and finishing on
// the at most kCap candidates that remain by direct rank counting.  If a bin still holds
// more than kCap elements after three levels (massive ties), an 8-bit most-significant-
// digit radix select over the ordered key bits finishes the job.  Only monotonicity of the
// binning function is needed for exactness, so float rounding inside it is harmless.
#include "nkv_common.cuh"

namespace nkv {

namespace {

constexpr int kThreads = 1024;
constexpr int kBins = 2048;
constexpr int kCap = 2048;
constexpr int kLevels = 3;
constexpr int kMaxCorr = 64;   // heads per group supported by the budget kernel

struct SelectShared {
    int hist[kBins];
    uint32_t cand[kCap];
    int cand_n;
    int bin, above, nbin;
    uint32_t theta;
    int gt, eq;
    int found;
    float red_f[32];
    int red_i[32];
    int scan_w[32];   // per-warp totals of find_bin_desc
    // elements to remove from the multiset (value, multiplicity)
    float corr_v[kMaxCorr];
    int corr_m[kMaxCorr];
    int ncorr;
};

struct Levels {
    float lo[kLevels], sc[kLevels];
    int bin[kLevels];
    int n;  // levels fixed so far
};

__device__ __forceinline__ int bin_of(float v, float lo, float sc) {
    int b = __float2int_rz((v - lo) * sc);
    return min(max(b, 0), kBins - 1);
}
__device__ __forceinline__ bool matches(const Levels& L, float v) {
    for (int i = 0; i < L.n; ++i)
        if (bin_of(v, L.lo[i], L.sc[i]) != L.bin[i]) return false;
    return true;
}

// The bin holding the `need`-th element counted from the top, and the count above it (S.bin, S.above,
// S.nbin).  Whole CTA: thread t sums the kBins / blockDim.x bins below bin kBins - 1 - t * per, a scan over
// the threads finds the owner, which walks its own bins.  The caller synchronises before reading S.*.
__device__ __forceinline__ void find_bin_desc(SelectShared& S, int need) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = kBins / (int)blockDim.x;   // 8 or 2 (CTAs of 256 or 1024 threads)
    const int top = kBins - 1 - tid * per;      // thread 0 owns the highest bins
    int c[8], sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        c[j] = j < per ? S.hist[top - j] : 0;
        sum += c[j];
    }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) S.scan_w[warp] = incl;
    __syncthreads();
    int excl = incl - sum;
    for (int w = 0; w < warp; ++w) excl += S.scan_w[w];
    if (need > excl && need <= excl + sum) {
        int run = excl;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j < per && need > run && need <= run + c[j]) {
                S.bin = top - j;
                S.above = run;
                S.nbin = c[j];
            }
            run += c[j];
        }
    }
}

__device__ __forceinline__ int block_sum_int(SelectShared& S, int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) S.red_i[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = (threadIdx.x < (blockDim.x >> 5)) ? S.red_i[threadIdx.x] : 0;
    if (threadIdx.x < 32) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (threadIdx.x == 0) S.red_i[0] = t;
    }
    __syncthreads();
    return S.red_i[0];
}

// Exact selection of the rank-th largest (1-based) element of { src(j) : j in [0,n), src.get true }
// minus the S.corr multiset.  Results in S.theta (ordered key), S.gt (#elements > theta),
// S.eq (#elements == theta).  lo/scale give the level-0 binning.  Must be called by all threads.
template <class Src>
__device__ __noinline__ void block_select_desc(SelectShared& S, const Src& src, int n, int rank, float lo0, float sc0, int* status) {
    Levels L;
    L.n = 0;
    float lo = lo0, sc = sc0;
    int need = rank, above_total = 0;
    bool small = false;
    for (int level = 0; level < kLevels; ++level) {
        for (int b = threadIdx.x; b < kBins; b += blockDim.x) S.hist[b] = 0;
        if (threadIdx.x == 0) {
            S.bin = 0;
            S.above = 0;
            S.nbin = 0;
        }
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += blockDim.x) {
            float v;
            if (src.get(j, v) && matches(L, v)) atomicAdd(&S.hist[bin_of(v, lo, sc)], 1);
        }
        __syncthreads();
        if (threadIdx.x < S.ncorr) {
            const float v = S.corr_v[threadIdx.x];
            if (S.corr_m[threadIdx.x] > 0 && matches(L, v)) atomicSub(&S.hist[bin_of(v, lo, sc)], S.corr_m[threadIdx.x]);
        }
        __syncthreads();
        find_bin_desc(S, need);
        __syncthreads();
        above_total += S.above;
        need -= S.above;
        L.lo[level] = lo;
        L.sc[level] = sc;
        L.bin[level] = S.bin;
        L.n = level + 1;
        if (S.nbin <= kCap) {
            small = true;
            break;
        }
        lo = lo + (float)S.bin / sc;
        sc = sc * (float)kBins;
        __syncthreads();
    }

    if (small) {
        if (threadIdx.x == 0) {
            S.cand_n = 0;
            S.found = 0;
        }
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += blockDim.x) {
            float v;
            if (src.get(j, v) && matches(L, v)) {
                const int pos = atomicAdd(&S.cand_n, 1);
                if (pos < kCap) S.cand[pos] = ord_key(v);
            }
        }
        __syncthreads();
        const int cn = min(S.cand_n, kCap);
        for (int a = threadIdx.x; a < cn; a += blockDim.x) {
            const uint32_t x = S.cand[a];
            int gt = 0, eq = 0;
            for (int b = 0; b < cn; ++b) {
                const uint32_t y = S.cand[b];
                gt += (y > x);
                eq += (y == x);
            }
            for (int c = 0; c < S.ncorr; ++c) {
                if (S.corr_m[c] > 0 && matches(L, S.corr_v[c])) {
                    const uint32_t y = ord_key(S.corr_v[c]);
                    if (y > x) gt -= S.corr_m[c];
                    if (y == x) eq -= S.corr_m[c];
                }
            }
            if (gt < need && need <= gt + eq) {
                S.theta = x;
                S.gt = above_total + gt;
                S.eq = eq;
                S.found = 1;
            }
        }
        __syncthreads();
        if (!S.found && threadIdx.x == 0) set_status(status, NKV_ERR_DEVICE_CHECK, 101);
        __syncthreads();
        return;
    }

    // radix fallback over the ordered key bits of the elements of the last chosen bin
    if (threadIdx.x == 0) atomicAdd(&status[kStatusFallbacks], 1);
    uint32_t prefix = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        const uint32_t himask = (shift == 24) ? 0u : (0xffffffffu << (shift + 8));
        for (int b = threadIdx.x; b < 256; b += blockDim.x) S.hist[b] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += blockDim.x) {
            float v;
            if (src.get(j, v) && matches(L, v)) {
                const uint32_t key = ord_key(v);
                if (((key ^ prefix) & himask) == 0) atomicAdd(&S.hist[(key >> shift) & 255], 1);
            }
        }
        __syncthreads();
        if (threadIdx.x < S.ncorr) {
            const float v = S.corr_v[threadIdx.x];
            const uint32_t key = ord_key(v);
            if (S.corr_m[threadIdx.x] > 0 && matches(L, v) && ((key ^ prefix) & himask) == 0)
                atomicSub(&S.hist[(key >> shift) & 255], S.corr_m[threadIdx.x]);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int run = 0, dsel = 0;
            for (int dgt = 255; dgt >= 0; --dgt) {
                const int c = S.hist[dgt];
                if (need <= run + c) {
                    dsel = dgt;
                    S.nbin = c;
                    break;
                }
                run += c;
            }
            S.bin = dsel;
            S.above = run;
        }
        __syncthreads();
        above_total += S.above;
        need -= S.above;
        prefix |= ((uint32_t)S.bin) << shift;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        S.theta = prefix;
        S.gt = above_total;
        S.eq = S.nbin;
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------
// head_scores: one CTA per head.
// ------------------------------------------------------------------------------------------
// A source yields element j of a multiset (get returns false for an element it leaves out).  A source
// with kVec also yields four consecutive elements at once when vec_ok() says its rows are 16-byte aligned
// (get4: values in x, bit e of the result set when element 4 j4 + e belongs to the multiset).
struct ScaleSrc {      // values of one scale of one head; `flip` turns bottom-m into top-m of the negated values
    static constexpr bool kVec = false;
    const float* a;
    float sign;
    __device__ __forceinline__ bool get(int j, float& v) const {
        v = sign * a[j];
        return true;
    }
};

// Min-max normalisation with the reciprocal of the range taken once per head (0 for a constant sequence): the
// per-token kernels are bound by instruction issue, and an IEEE division costs ten instructions.
__device__ __forceinline__ float inv_range(float range) { return range > 0.f ? 1.0f / range : 0.f; }
__device__ __forceinline__ float norm01(float a, float lo, float inv) { return (a - lo) * inv; }

__device__ __forceinline__ float surprise3(float x0, float x1, float x2) {
    constexpr float kThird = 1.0f / 3.0f;
    const float mean = (x0 + x1 + x2) * kThird;
    const float d0 = x0 - mean, d1 = x1 - mean, d2 = x2 - mean;
    return sqrtf((d0 * d0 + d1 * d1 + d2 * d2) * kThird);
}

__device__ __forceinline__ float block_reduce_f(SelectShared& S, float v, int op) {  // 0 sum, 1 min, 2 max
    if (op == 0) v = warp_sum(v);
    else if (op == 1) v = warp_min(v);
    else v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) S.red_f[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        const int nw = blockDim.x >> 5;
        float t = (threadIdx.x < nw) ? S.red_f[threadIdx.x] : (op == 0 ? 0.f : (op == 1 ? INFINITY : -INFINITY));
        if (op == 0) t = warp_sum(t);
        else if (op == 1) t = warp_min(t);
        else t = warp_max(t);
        if (threadIdx.x == 0) S.red_f[0] = t;
    }
    __syncthreads();
    const float r = S.red_f[0];
    __syncthreads();
    return r;
}

// ------------------------------------------------------------------------------------------
// Bracketed selection.  block_select_desc touches a shared-memory histogram once per element and
// pass, which serialises on the crowded bins.  Here a strided sample of the source first brackets
// the wanted order statistic between two pivots P_lo <= theta <= P_hi (a few standard deviations of
// the sample's rank error on either side); one pass then counts (and optionally sums) the elements
// above P_hi in registers and appends only the elements inside the bracket, a few percent of the
// source, to a shared list; block_select_desc finishes exactly on that list.  Whenever the bracket
// turns out wrong (rank outside the list, list overflow) the full-histogram path runs instead, so the
// result is always exact.
// ------------------------------------------------------------------------------------------
constexpr int kSampleMin = 1024, kSampleMax = 32768;   // sample positions: n / 8 (n / 4 for long inputs), clamped
// The bracket that one sample rank error of 4 sigma spans grows with n / positions: beyond 64k elements a
// denser sample keeps it inside the candidate buffers.
__device__ __forceinline__ int sample_positions(int n) { return min(max(n > 65536 ? n / 4 : n / 8, kSampleMin), kSampleMax); }
// Sample position i of `positions` over n elements is floor(i * step / 2^16) with step = floor(n * 2^16 / positions):
// one 64-bit division per thread instead of one per sample (positions <= n, so the index stays below n).
__device__ __forceinline__ unsigned long long sample_step(int n, int positions) {
    return ((unsigned long long)n << 16) / (unsigned long long)positions;
}
__device__ __forceinline__ int sample_index(int i, unsigned long long step) { return (int)(((unsigned long long)i * step) >> 16); }
constexpr int kCandSmall = 4096;                       // bracket capacity of the per-head kernels
constexpr int kCandLarge = 12288;                      // ... of the per-group kernel (dynamic shared memory)

template <int CAP>
struct BracketShared {
    float cand[CAP];
    int cand_n, cnt_gt, ok;
    float sum_gt;
    float p_lo, p_hi;
    float save_v[kMaxCorr];
    int save_m[kMaxCorr], save_n;
};

struct SmemSrc {
    static constexpr bool kVec = false;
    const float* p;
    __device__ __forceinline__ bool get(int j, float& v) const {
        v = p[j];
        return true;
    }
};

// Same contract as block_select_desc (results in S.theta / S.gt / S.eq, S.corr honoured).  `n_eff` is the
// number of elements the source really yields (n minus those its get() rejects).  If `sum_above` is not
// null it receives the sum of the elements strictly greater than theta.
template <int CAP, class Src>
__device__ void block_select_bracket(SelectShared& S, BracketShared<CAP>& X, const Src& src, int n, long long n_eff,
                                     int rank, float lo0, float sc0, int* status, float* sum_above) {
    constexpr int kCandCap = CAP;
    const int tid = threadIdx.x, nt = blockDim.x;
    bool use_bracket = n > kCandCap && n_eff > 0;
    if (use_bracket) {
        // 1. histogram of a strided sample (rejected elements are skipped)
        const int positions = sample_positions(n);
        const unsigned long long step = sample_step(n, positions);
        for (int b = tid; b < kBins; b += nt) S.hist[b] = 0;
        __syncthreads();
        int mine = 0;
        for (int i0 = 0; i0 < positions; i0 += 4 * nt) {   // four loads in flight per thread
            float sv[4];
            bool sk[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = i0 + k * nt + tid;
                sv[k] = 0.f;
                sk[k] = i < positions && src.get(sample_index(i, step), sv[k]);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (sk[k]) {
                    atomicAdd(&S.hist[bin_of(sv[k], lo0, sc0)], 1);
                    ++mine;
                }
        }
        const int sn = block_sum_int(S, mine);
        // 2. pivots: sample ranks around rank * sn / n_eff, four standard deviations of the rank error apart
        const float q = (float)rank * (float)sn / (float)n_eff;
        const float sd = sqrtf(fmaxf(q * (1.0f - q / fmaxf((float)sn, 1.0f)), 1.0f));
        const int r_hi = (int)floorf(q - 4.0f * sd - 4.0f), r_lo = (int)ceilf(q + 4.0f * sd + 4.0f);
        // save the correction multiset: the sample selections below must not see it
        if (tid == 0) {
            X.save_n = S.ncorr;
            for (int c = 0; c < S.ncorr; ++c) {
                X.save_v[c] = S.corr_v[c];
                X.save_m[c] = S.corr_m[c];
            }
            S.ncorr = 0;
            X.p_hi = INFINITY;
            X.p_lo = -INFINITY;
        }
        __syncthreads();
        // pivots = edges of the value-linear bins that hold the r_hi-th and r_lo-th largest sample elements
        if (sn >= 64) {
            if (r_hi >= 1) {
                find_bin_desc(S, r_hi);
                __syncthreads();
                if (tid == 0) X.p_hi = lo0 + (float)(S.bin + 1) / sc0;
                __syncthreads();
            }
            if (r_lo <= sn) {
                find_bin_desc(S, r_lo);
                __syncthreads();
                if (tid == 0) X.p_lo = lo0 + (float)S.bin / sc0;
                __syncthreads();
            }
        }
        const float p_hi = X.p_hi, p_lo = X.p_lo;
        // 3. one pass: count / sum above the bracket, collect the bracket
        if (tid == 0) {
            X.cand_n = 0;
            X.cnt_gt = 0;
            X.sum_gt = 0.f;
        }
        __syncthreads();
        int cnt = 0;
        float sum = 0.f;
        // one element: counted (and summed) above the bracket, appended to the list inside it
        auto consume = [&](float v, bool in) {
            const bool above = in && v > p_hi;
            const bool inside = in && !above && v >= p_lo;
            cnt += above;
            if (above) sum += v;
            // a few percent of the elements: every thread appends its own (a warp-wide vote per element would
            // send nearly every warp down the append path, which is what this pass spent its time on)
            if (inside) {
                const int pos = atomicAdd(&X.cand_n, 1);
                if (pos < kCandCap) X.cand[pos] = v;
            }
        };
        bool vec = false;
        if constexpr (Src::kVec) vec = src.vec_ok() && (n & 3) == 0;
        if (vec) {
            if constexpr (Src::kVec) {
                const int n4 = n >> 2;
                for (int jb = 0; jb < n4; jb += 4 * nt) {   // sixteen elements in flight per thread
                    float4 q[4];
                    unsigned keep[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int j = jb + k * nt + tid;
                        keep[k] = 0u;
                        q[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (j < n4) keep[k] = src.get4(j, q[k]);
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        consume(q[k].x, (keep[k] & 1u) != 0);
                        consume(q[k].y, (keep[k] & 2u) != 0);
                        consume(q[k].z, (keep[k] & 4u) != 0);
                        consume(q[k].w, (keep[k] & 8u) != 0);
                    }
                }
            }
        } else {
            for (int jb = 0; jb < n; jb += 4 * nt) {   // four loads in flight per thread
                float vv[4];
                bool vk[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int j = jb + k * nt + tid;
                    vv[k] = 0.f;
                    vk[k] = j < n && src.get(j, vv[k]);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) consume(vv[k], vk[k]);
            }
        }
        cnt = block_sum_int(S, cnt);
        __syncthreads();
        const float total_sum = sum_above ? block_reduce_f(S, sum, 0) : 0.f;
        // 4. move the correction multiset inside / above the bracket
        if (tid == 0) {
            int above_corr = 0, ncorr = 0;
            for (int c = 0; c < X.save_n; ++c) {
                if (X.save_m[c] <= 0) continue;
                if (X.save_v[c] > p_hi) above_corr += X.save_m[c];
                else if (X.save_v[c] >= p_lo) {
                    S.corr_v[ncorr] = X.save_v[c];
                    S.corr_m[ncorr] = X.save_m[c];
                    ++ncorr;
                }
            }
            S.ncorr = ncorr;
            X.cnt_gt = cnt - above_corr;
            X.sum_gt = total_sum;
            int inner = X.cand_n;
            for (int c = 0; c < ncorr; ++c) inner -= S.corr_m[c];
            const int r2 = rank - X.cnt_gt;
            X.ok = (X.cand_n <= kCandCap && r2 >= 1 && r2 <= inner) ? 1 : 0;
        }
        __syncthreads();
        if (X.ok) {
            const int cn = X.cand_n, r2 = rank - X.cnt_gt;
            const float width = p_hi - p_lo;
            const bool own_bins = width > 0.f && isfinite(width) && isfinite(p_lo);
            SmemSrc csrc{X.cand};
            block_select_desc(S, csrc, cn, r2, own_bins ? p_lo : lo0, own_bins ? (float)kBins / width : sc0, status);
            if (sum_above) {
                const uint32_t theta = S.theta;
                float part = 0.f;
                for (int j = tid; j < cn; j += nt)
                    if (ord_key(X.cand[j]) > theta) part += X.cand[j];
                const float inner_sum = block_reduce_f(S, part, 0);
                if (tid == 0) *sum_above = X.sum_gt + inner_sum;
            }
            __syncthreads();
            if (tid == 0) {
                S.gt += X.cnt_gt;
                // restore the caller's correction multiset
                S.ncorr = X.save_n;
                for (int c = 0; c < X.save_n; ++c) {
                    S.corr_v[c] = X.save_v[c];
                    S.corr_m[c] = X.save_m[c];
                }
            }
            __syncthreads();
            return;
        }
        if (tid == 0) {
            S.ncorr = X.save_n;
            for (int c = 0; c < X.save_n; ++c) {
                S.corr_v[c] = X.save_v[c];
                S.corr_m[c] = X.save_m[c];
            }
        }
        __syncthreads();
    }
    // full-histogram path
    block_select_desc(S, src, n, rank, lo0, sc0, status);
    if (sum_above) {
        const uint32_t theta = S.theta;
        __syncthreads();
        float part = 0.f;
        for (int j = tid; j < n; j += nt) {
            float v;
            if (src.get(j, v) && ord_key(v) > theta) part += v;
        }
        const float above = block_reduce_f(S, part, 0);
        if (tid == 0) *sum_above = above;
        __syncthreads();
    }
}

// Sums of the m largest and of the m smallest of a[0..n) with both tails bracketed from one sample
// histogram and collected in one pass (the two halves of X.cand hold the two brackets).  Returns false,
// having computed nothing, when a bracket misses or the two overlap; the caller then selects each tail
// on its own.  lo0 / sc0: value-linear binning of the whole range.
template <int CAP>
__device__ bool two_tail_sums(SelectShared& S, BracketShared<CAP>& X, const float* __restrict__ a, int n, int m,
                              float lo0, float sc0, int* status, float* top_sum, float* bot_sum) {
    constexpr int kHalf = CAP / 2;
    __shared__ int sh_n[2], sh_cnt[2], sh_ok;
    __shared__ float sh_piv[4], sh_sum[2], sh_res[2];
    const int tid = threadIdx.x, nt = blockDim.x;
    if (n <= CAP || 2 * m >= n) return false;
    // 1. histogram of a strided sample
    const int positions = sample_positions(n);
    const unsigned long long step = sample_step(n, positions);
    for (int b = tid; b < kBins; b += nt) S.hist[b] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < positions; i0 += 4 * nt) {   // four loads in flight per thread
        float sv[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = i0 + k * nt + tid;
            sv[k] = i < positions ? a[sample_index(i, step)] : 0.f;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (i0 + k * nt + tid < positions) atomicAdd(&S.hist[bin_of(sv[k], lo0, sc0)], 1);
    }
    __syncthreads();
    const int sn = positions;
    // 2. four pivots: ranks (counted from the top) around m and around n - m + 1
    const float qt = (float)m * (float)sn / (float)n, qb = (float)(n - m + 1) * (float)sn / (float)n;
    const float sdt = sqrtf(fmaxf(qt * (1.0f - qt / (float)sn), 1.0f)), sdb = sqrtf(fmaxf(qb * (1.0f - qb / (float)sn), 1.0f));
    const int r[4] = {(int)floorf(qt - 4.0f * sdt - 4.0f), (int)ceilf(qt + 4.0f * sdt + 4.0f),
                      (int)floorf(qb - 4.0f * sdb - 4.0f), (int)ceilf(qb + 4.0f * sdb + 4.0f)};
    if (tid == 0) {
        sh_piv[0] = INFINITY;    // top bracket: (piv[1], piv[0]]
        sh_piv[3] = -INFINITY;   // bottom bracket: [piv[3], piv[2])
    }
    if (r[1] > sn || r[2] < 1) return false;   // uniform: depends on n and m only
    __syncthreads();
    for (int k = 0; k < 4; ++k) {
        if (r[k] >= 1 && r[k] <= sn) {
            find_bin_desc(S, r[k]);
            __syncthreads();
            // upper pivots take the upper edge of their bin, lower pivots the lower edge
            if (tid == 0) sh_piv[k] = lo0 + (float)(S.bin + ((k & 1) ? 0 : 1)) / sc0;
            __syncthreads();
        }
    }
    const float pt_hi = sh_piv[0], pt_lo = sh_piv[1], pb_hi = sh_piv[2], pb_lo = sh_piv[3];
    if (!(pt_lo > pb_hi)) return false;   // uniform
    // 3. one pass: count and sum beyond the brackets, collect inside them
    if (tid == 0) sh_n[0] = sh_n[1] = 0;
    __syncthreads();
    int cnt_t = 0, cnt_b = 0;
    float sum_t = 0.f, sum_b = 0.f;
    auto take = [&](float v, bool in) {
        const bool above = in && v > pt_hi, below = in && v < pb_lo;
        const bool in_t = in && !above && v >= pt_lo, in_b = in && !below && v <= pb_hi;
        cnt_t += above;
        cnt_b += below;
        if (above) sum_t += v;
        if (below) sum_b += v;
        if (in_t || in_b) {   // a few percent of the values: every thread appends its own
            const int side = in_t ? 0 : 1;
            const int pos = atomicAdd(&sh_n[side], 1);
            if (pos < kHalf) X.cand[side * kHalf + pos] = v;
        }
    };
    if ((n & 3) == 0 && (reinterpret_cast<uintptr_t>(a) & 15) == 0) {
        // rows are 16-byte aligned: four values per load, four loads in flight per thread
        const float4* a4 = reinterpret_cast<const float4*>(a);
        const int n4 = n >> 2;
        for (int jb = 0; jb < n4; jb += 4 * nt) {
            float4 q[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) q[k] = jb + k * nt + tid < n4 ? a4[jb + k * nt + tid] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const bool in = jb + k * nt + tid < n4;
                take(q[k].x, in);
                take(q[k].y, in);
                take(q[k].z, in);
                take(q[k].w, in);
            }
        }
    } else {
        for (int jb = 0; jb < n; jb += 4 * nt) {   // four loads in flight per thread
            float vv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) vv[k] = jb + k * nt + tid < n ? a[jb + k * nt + tid] : 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) take(vv[k], jb + k * nt + tid < n);
        }
    }
    cnt_t = block_sum_int(S, cnt_t);
    __syncthreads();
    cnt_b = block_sum_int(S, cnt_b);
    __syncthreads();
    sum_t = block_reduce_f(S, sum_t, 0);
    sum_b = block_reduce_f(S, sum_b, 0);
    if (tid == 0) {
        const int rt = m - cnt_t, rb = m - cnt_b;   // ranks wanted inside the brackets (largest / smallest)
        sh_ok = sh_n[0] <= kHalf && sh_n[1] <= kHalf && rt >= 1 && rt <= sh_n[0] && rb >= 1 && rb <= sh_n[1];
        sh_cnt[0] = cnt_t;
        sh_cnt[1] = cnt_b;
        sh_sum[0] = sum_t;
        sh_sum[1] = sum_b;
    }
    __syncthreads();
    if (!sh_ok) return false;
    // 4. finish exactly inside each bracket
    for (int side = 0; side < 2; ++side) {
        const int cn = sh_n[side];
        const float* c = X.cand + side * kHalf;
        const int want = m - sh_cnt[side];
        const int rank_desc = side == 0 ? want : cn - want + 1;
        const float blo = side == 0 ? pt_lo : pb_lo, bhi = side == 0 ? pt_hi : pb_hi, width = bhi - blo;
        const bool own = width > 0.f && isfinite(width) && isfinite(blo);
        SmemSrc csrc{c};
        block_select_desc(S, csrc, cn, rank_desc, own ? blo : lo0, own ? (float)kBins / width : sc0, status);
        const uint32_t theta = S.theta;
        __syncthreads();
        float part = 0.f;
        int beyond = 0;   // bracket elements strictly beyond theta on this side
        for (int j = tid; j < cn; j += nt) {
            const uint32_t key = ord_key(c[j]);
            const bool b = side == 0 ? key > theta : key < theta;
            if (b) {
                part += c[j];
                ++beyond;
            }
        }
        const float inner = block_reduce_f(S, part, 0);
        beyond = block_sum_int(S, beyond);
        if (tid == 0) sh_res[side] = sh_sum[side] + inner + (float)(want - beyond) * ord_float(theta);
        __syncthreads();
    }
    if (tid == 0) {
        *top_sum = sh_res[0];
        *bot_sum = sh_res[1];
    }
    __syncthreads();
    return true;
}

// Layout of the per-head statistics scratch written by scale_stats_kernel (floats per head).
constexpr int kHeadStat = 8;   // Delta_s, Delta_e, Delta_c, min s, max s, sum s, unused, unused
constexpr int kStatThreads = 256;

// scale_stats: one CTA per (head, task).  Tasks 0..2: the reliability gap of one scale (exact sums of
// the m largest and m smallest values); task 3: min, max and sum of the surprise over the head.
template <int kT>
__global__ void __launch_bounds__(kT, kT == 256 ? 4 : 1) scale_stats_kernel(int N, ScoreParams sp, const float* __restrict__ a_raw,
                                                                   const uint32_t* __restrict__ mm,
                                                                   float* __restrict__ hstat, int* status) {
    __shared__ SelectShared S;
    __shared__ BracketShared<kCandSmall> X;
    __shared__ float sh_above;
    const int u = blockIdx.x >> 2, task = blockIdx.x & 3;
    const float* a[3] = {a_raw + ((int64_t)u * 3 + 0) * N, a_raw + ((int64_t)u * 3 + 1) * N,
                         a_raw + ((int64_t)u * 3 + 2) * N};
    float lo[3], range[3], inv[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        lo[k] = ord_float(mm[(int64_t)u * 6 + 2 * k]);
        range[k] = ord_float(mm[(int64_t)u * 6 + 2 * k + 1]) - lo[k];
        inv[k] = inv_range(range[k]);
    }
    if (threadIdx.x == 0) S.ncorr = 0;
    __syncthreads();
    float* out = hstat + (int64_t)u * kHeadStat;

    if (task < 3) {
        // reliability gap: (sum of the m largest - sum of the m smallest) / (m * range)
        const int k = task, m = sp.top_m;
        const float lok = k == 0 ? lo[0] : (k == 1 ? lo[1] : lo[2]);
        const float rk = k == 0 ? range[0] : (k == 1 ? range[1] : range[2]);
        const float* ak = k == 0 ? a[0] : (k == 1 ? a[1] : a[2]);
        float gap = 0.f;
        if (rk > 0.f) {
            __shared__ float sh_top, sh_bot;
            if (two_tail_sums(S, X, ak, N, m, lok, (float)kBins / rk, status, &sh_top, &sh_bot)) {
                gap = (sh_top - sh_bot) / ((float)m * rk);
            } else {
                float side_sum[2];
                for (int side = 0; side < 2; ++side) {
                    ScaleSrc src{ak, side == 0 ? 1.f : -1.f};
                    const float lo0 = side == 0 ? lok : -(lok + rk);
                    block_select_bracket(S, X, src, N, (long long)N, m, lo0, (float)kBins / rk, status, &sh_above);
                    __syncthreads();
                    side_sum[side] = sh_above + (float)(m - S.gt) * ord_float(S.theta);
                    __syncthreads();
                }
                // side 1 summed the negated values: top_sum - bot_sum = side_sum[0] + side_sum[1]
                gap = (side_sum[0] + side_sum[1]) / ((float)m * rk);
            }
        }
        if (threadIdx.x == 0) out[k] = gap;
    } else {
        float smin = INFINITY, smax = -INFINITY, ssum = 0.f;
        auto take = [&](float r0, float r1, float r2) {
            const float s = surprise3(norm01(r0, lo[0], inv[0]), norm01(r1, lo[1], inv[1]), norm01(r2, lo[2], inv[2]));
            smin = fminf(smin, s);
            smax = fmaxf(smax, s);
            ssum += s;
        };
        if ((N & 3) == 0 && (reinterpret_cast<uintptr_t>(a_raw) & 15) == 0) {
            // rows are 16-byte aligned: four tokens per load, two sets of loads in flight
            const float4* q0 = reinterpret_cast<const float4*>(a[0]);
            const float4* q1 = reinterpret_cast<const float4*>(a[1]);
            const float4* q2 = reinterpret_cast<const float4*>(a[2]);
            const int n4 = N >> 2, nt = blockDim.x;
            for (int jb = 0; jb < n4; jb += 2 * nt) {
                float4 r[2][3];
                bool in[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const int j = jb + k * nt + threadIdx.x;
                    in[k] = j < n4;
                    if (in[k]) {
                        r[k][0] = q0[j];
                        r[k][1] = q1[j];
                        r[k][2] = q2[j];
                    }
                }
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    if (in[k]) {
                        take(r[k][0].x, r[k][1].x, r[k][2].x);
                        take(r[k][0].y, r[k][1].y, r[k][2].y);
                        take(r[k][0].z, r[k][1].z, r[k][2].z);
                        take(r[k][0].w, r[k][1].w, r[k][2].w);
                    }
            }
        } else {
            for (int j = threadIdx.x; j < N; j += blockDim.x) take(a[0][j], a[1][j], a[2][j]);
        }
        smin = block_reduce_f(S, smin, 1);
        smax = block_reduce_f(S, smax, 2);
        ssum = block_reduce_f(S, ssum, 0);
        if (threadIdx.x == 0) {
            out[3] = smin;
            out[4] = smax;
            out[5] = ssum;
        }
    }
}

// mix: elementwise.  Every CTA recomputes its head's three weights and surprise constants (a handful of
// flops) and routes a chunk of tokens: a* = (1 - alpha) * blend + alpha * max, sinks pinned to +inf.
constexpr int kMixThreads = 256;
constexpr int kMixPerThread = 16;
__global__ void __launch_bounds__(kMixThreads) mix_kernel(int N, ScoreParams sp, const float* __restrict__ a_raw,
                                                          const uint32_t* __restrict__ mm,
                                                          const float* __restrict__ hstat, float* __restrict__ a_star,
                                                          float* __restrict__ stats_out) {
    const int u = blockIdx.y;
    const float* a0 = a_raw + ((int64_t)u * 3 + 0) * N;
    const float* a1 = a0 + N;
    const float* a2 = a1 + N;
    float lo[3], range[3], inv[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        lo[k] = ord_float(mm[(int64_t)u * 6 + 2 * k]);
        range[k] = ord_float(mm[(int64_t)u * 6 + 2 * k + 1]) - lo[k];
        inv[k] = inv_range(range[k]);
    }
    const float* hs = hstat + (int64_t)u * kHeadStat;
    float z[3], zmax = -INFINITY, wsum = 0.f, w[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        z[k] = sp.log_prior[k] + sp.beta * hs[k];
        zmax = fmaxf(zmax, z[k]);
    }
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        z[k] = expf(z[k] - zmax);
        wsum += z[k];
    }
#pragma unroll
    for (int k = 0; k < 3; ++k) w[k] = z[k] / wsum;
    const float s_lo = hs[3], s_inv = inv_range(hs[4] - hs[3]);
    const float s_mean = norm01(hs[5] / (float)N, s_lo, s_inv);

    const int base = blockIdx.x * (kMixThreads * kMixPerThread);
    // one token: min-max normalise, blend, gate, pin the sinks
    auto route = [&](float r0, float r1, float r2, int j) {
        const float x0 = norm01(r0, lo[0], inv[0]);
        const float x1 = norm01(r1, lo[1], inv[1]);
        const float x2 = norm01(r2, lo[2], inv[2]);
        const float blend = w[0] * x0 + w[1] * x1 + w[2] * x2;
        const float win = fmaxf(x0, fmaxf(x1, x2));
        float alpha;
        if (sp.gate_mode == NKV_GATE_AVERAGE) alpha = 0.f;
        else if (sp.gate_mode == NKV_GATE_MAX) alpha = 1.f;
        else {
            const float sn = norm01(surprise3(x0, x1, x2), s_lo, s_inv);
            const float sprime = fmaxf(0.f, sn - s_mean);
            alpha = __fdividef(1.0f, 1.0f + __expf(-sp.kappa * (sprime - sp.tau)));   // both within 2 ulp here
        }
        const float v = (1.0f - alpha) * blend + alpha * win + 0.f;
        return j < sp.n_sink ? INFINITY : v;
    };
    if ((N & 3) == 0 && ((reinterpret_cast<uintptr_t>(a_raw) | reinterpret_cast<uintptr_t>(a_star)) & 15) == 0) {
        // rows are 16-byte aligned: four tokens per load
        const float4* q0 = reinterpret_cast<const float4*>(a0);
        const float4* q1 = reinterpret_cast<const float4*>(a1);
        const float4* q2 = reinterpret_cast<const float4*>(a2);
        float4* out4 = reinterpret_cast<float4*>(a_star + (int64_t)u * N);
#pragma unroll
        for (int e = 0; e < kMixPerThread / 4; ++e) {
            const int j4 = base / 4 + e * kMixThreads + threadIdx.x;
            if (4 * j4 < N) {
                const float4 r0 = q0[j4], r1 = q1[j4], r2 = q2[j4];
                float4 o;
                o.x = route(r0.x, r1.x, r2.x, 4 * j4);
                o.y = route(r0.y, r1.y, r2.y, 4 * j4 + 1);
                o.z = route(r0.z, r1.z, r2.z, 4 * j4 + 2);
                o.w = route(r0.w, r1.w, r2.w, 4 * j4 + 3);
                out4[j4] = o;
            }
        }
    } else {
#pragma unroll
        for (int e = 0; e < kMixPerThread; ++e) {
            const int j = base + e * kMixThreads + threadIdx.x;
            if (j < N) a_star[(int64_t)u * N + j] = route(a0[j], a1[j], a2[j], j);
        }
    }
    if (stats_out && blockIdx.x == 0 && threadIdx.x == 0) {
        float* o = stats_out + (int64_t)u * NKV_HEAD_STATS;
        for (int k = 0; k < 3; ++k) {
            o[k] = lo[k];
            o[3 + k] = lo[k] + range[k];
            o[6 + k] = hs[k];
            o[9 + k] = w[k];
        }
        o[12] = s_lo;
        o[13] = hs[4];
        o[14] = s_mean;
        o[15] = (float)sp.top_m;
    }
}

// ------------------------------------------------------------------------------------------
// budget: one CTA per layer group.
// ------------------------------------------------------------------------------------------
struct HeadSrc {
    static constexpr bool kVec = true;
    const float* v;
    int n;
    __device__ __forceinline__ bool get(int j, float& x) const {
        x = v[j];
        return true;
    }
    __device__ __forceinline__ bool vec_ok() const { return (n & 3) == 0 && (reinterpret_cast<uintptr_t>(v) & 15) == 0; }
    __device__ __forceinline__ unsigned get4(int j4, float4& x) const {
        x = reinterpret_cast<const float4*>(v)[j4];
        return 15u;
    }
};
struct PoolSrc {       // all (head, token) pairs of a group whose key does not exceed the head's safeguard threshold
    const float* v;    // [H, N]
    const uint32_t* T; // per-head safeguard threshold keys (shared memory)
    int N;
    float invN;
    static constexpr bool kVec = true;
    // head of element j without an integer division: the float quotient is off by one at most
    __device__ __forceinline__ int head_of(int j) const {
        int h = (int)((float)j * invN);
        if ((h + 1) * N <= j) ++h;
        if (h * N > j) --h;
        return h;
    }
    __device__ __forceinline__ bool get(int j, float& x) const {
        x = v[j];
        return ord_key(x) <= T[head_of(j)];
    }
    __device__ __forceinline__ bool vec_ok() const { return (N & 3) == 0 && (reinterpret_cast<uintptr_t>(v) & 15) == 0; }
    __device__ __forceinline__ unsigned get4(int j4, float4& x) const {
        x = reinterpret_cast<const float4*>(v)[j4];
        const uint32_t t = T[head_of(4 * j4)];   // N is a multiple of 4: the four share a head
        return (ord_key(x.x) <= t ? 1u : 0u) | (ord_key(x.y) <= t ? 2u : 0u) | (ord_key(x.z) <= t ? 4u : 0u) |
               (ord_key(x.w) <= t ? 8u : 0u);
    }
};

// safeguard: one CTA per head.  The n_safe best tokens of each head are kept unconditionally:
// thr[2u] = ordered key of the n_safe-th best score, thr[2u+1] = how many tokens tied at that key
// belong to the safeguard.  (The group kernel below overwrites both words with the final threshold.)
template <int kT>
__global__ void __launch_bounds__(kT, kT == 256 ? 4 : 1) safeguard_kernel(int N, int n_safe, const float* __restrict__ a_star,
                                                                 uint32_t* __restrict__ thr, int* status) {
    __shared__ SelectShared S;
    __shared__ BracketShared<kCandSmall> X;
    const int u = blockIdx.x;
    if (threadIdx.x == 0) S.ncorr = 0;
    __syncthreads();
    if (n_safe > 0) {
        HeadSrc src{a_star + (int64_t)u * N, N};
        block_select_bracket(S, X, src, N, (long long)N, n_safe, 0.f, (float)kBins, status, nullptr);
        if (threadIdx.x == 0) {
            thr[(int64_t)u * 2] = S.theta;
            thr[(int64_t)u * 2 + 1] = (uint32_t)(n_safe - S.gt);
        }
    } else if (threadIdx.x == 0) {
        thr[(int64_t)u * 2] = 0xffffffffu;
        thr[(int64_t)u * 2 + 1] = 0u;
    }
}

// budget: one CTA per layer group, after safeguard_kernel.
__global__ void __launch_bounds__(kThreads) budget_kernel(int H, int N, int keep, int n_safe,
                                                          const float* __restrict__ a_star,
                                                          int32_t* __restrict__ budgets, uint32_t* __restrict__ thr,
                                                          int* status, const int* __restrict__ only_flagged) {
    // after the parallel form: only the groups it left over
    if (only_flagged && only_flagged[blockIdx.x * 4 + 3] == 0) return;
    __shared__ SelectShared S;
    extern __shared__ __align__(16) unsigned char budget_dyn[];
    BracketShared<kCandLarge>& X = *reinterpret_cast<BracketShared<kCandLarge>*>(budget_dyn);
    __shared__ uint32_t T[kMaxCorr];
    __shared__ int corr[kMaxCorr], cnt_mid[kMaxCorr], cnt_eq[kMaxCorr];
    const int g = blockIdx.x;
    const float* v = a_star + (int64_t)g * H * N;
    if (threadIdx.x == 0) S.ncorr = 0;
    if (threadIdx.x < H) {
        T[threadIdx.x] = thr[((int64_t)g * H + threadIdx.x) * 2];
        corr[threadIdx.x] = (int)thr[((int64_t)g * H + threadIdx.x) * 2 + 1];
    }
    __syncthreads();

    // cross-head competition for the remaining slots
    const int rest = H * keep - H * n_safe;
    uint32_t tau = 0xffffffffu;
    if (rest > 0) {
        if (threadIdx.x < H) {
            S.corr_v[threadIdx.x] = ord_float(T[threadIdx.x]);
            S.corr_m[threadIdx.x] = corr[threadIdx.x];
        }
        if (threadIdx.x == 0) S.ncorr = H;
        __syncthreads();
        PoolSrc src{v, T, N, 1.0f / (float)N};
        block_select_bracket(S, X, src, H * N, (long long)H * N - (long long)H * n_safe, rest, 0.f, (float)kBins, status,
                             nullptr);
        tau = S.theta;
        __syncthreads();
    }
    for (int h = 0; h < H; ++h) {
        int mid = 0, eq = 0;
        const uint32_t Th = T[h];
        const float* vh = v + (int64_t)h * N;
        auto tally = [&](float x) {
            const uint32_t key = ord_key(x);
            mid += (key > tau && key <= Th);
            eq += (key == tau && key <= Th);
        };
        if ((N & 3) == 0 && (reinterpret_cast<uintptr_t>(a_star) & 15) == 0) {
            // rows are 16-byte aligned: four tokens per load, four loads in flight
            const float4* q = reinterpret_cast<const float4*>(vh);
            const int n4 = N >> 2, nt = blockDim.x;
            for (int jb = 0; jb < n4; jb += 4 * nt) {
                float4 r[4];
                bool in[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int j = jb + k * nt + threadIdx.x;
                    in[k] = j < n4;
                    if (in[k]) r[k] = q[j];
                }
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (in[k]) {
                        tally(r[k].x);
                        tally(r[k].y);
                        tally(r[k].z);
                        tally(r[k].w);
                    }
            }
        } else {
            for (int j = threadIdx.x; j < N; j += blockDim.x) tally(vh[j]);
        }
        mid = block_sum_int(S, mid);
        __syncthreads();
        eq = block_sum_int(S, eq);
        if (threadIdx.x == 0) {
            cnt_mid[h] = mid;
            cnt_eq[h] = eq;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int taken_gt = 0;
        for (int h = 0; h < H; ++h) taken_gt += cnt_mid[h] - (T[h] > tau ? corr[h] : 0);
        int remaining = rest - taken_gt;
        int total = 0;
        for (int h = 0; h < H; ++h) {
            const int pool_eq = cnt_eq[h] - (T[h] == tau ? corr[h] : 0);
            const int t = max(0, min(pool_eq, remaining));
            remaining -= t;
            const int B = n_safe + cnt_mid[h] - (T[h] > tau ? corr[h] : 0) + t;
            budgets[(int64_t)g * H + h] = B;
            total += B;
            uint32_t theta, q;
            if (tau < T[h]) {
                theta = tau;
                q = (uint32_t)t;
            } else {
                theta = T[h];
                q = (uint32_t)(corr[h] + t);
            }
            thr[((int64_t)g * H + h) * 2] = theta;
            thr[((int64_t)g * H + h) * 2 + 1] = q;
        }
        if (total != H * keep || remaining != 0) set_status(status, NKV_ERR_DEVICE_CHECK, 201);
    }
}

// ------------------------------------------------------------------------------------------
// budget, parallel form: the cross-head competition of a group as a histogram over all of its
// heads, so that the streaming work is spread over many CTAs and only a small candidate list
// is finished by one CTA per group.
// ------------------------------------------------------------------------------------------
constexpr int kBudgetCand = 8192;    // candidates per group (the scores that share the threshold's bin)
constexpr int kBudgetChunk = 8192;   // scores per CTA of the two streaming steps
constexpr int kBudgetMeta = 4;       // per group: threshold bin, rank wanted inside it, candidates, needs the one-CTA kernel

// final scores lie in [0, 1] (sinks: +inf): 2048 value-linear bins, monotone in the score
__device__ __forceinline__ int score_bin(float v) { return min(max(__float2int_rz(v * (float)kBins), 0), kBins - 1); }

// step 1: per head, the histogram of its pool (scores at or below the head's safeguard threshold)
__global__ void __launch_bounds__(256) budget_hist_kernel(int N, const float* __restrict__ a_star,
                                                          const uint32_t* __restrict__ thr, int* __restrict__ bhist) {
    __shared__ int hist[kBins];
    const int u = blockIdx.y, j0 = blockIdx.x * kBudgetChunk, j1 = min(N, j0 + kBudgetChunk);
    for (int b = threadIdx.x; b < kBins; b += blockDim.x) hist[b] = 0;
    __syncthreads();
    const uint32_t T = thr[(int64_t)u * 2];
    const float* v = a_star + (int64_t)u * N;
    for (int j = j0 + threadIdx.x; j < j1; j += blockDim.x) {
        const float x = v[j];
        if (ord_key(x) <= T) atomicAdd(&hist[score_bin(x)], 1);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kBins; b += blockDim.x)
        if (hist[b]) atomicAdd(&bhist[(int64_t)u * kBins + b], hist[b]);
}

// step 2: per group, the bin that holds the rank the competition stops at
__global__ void __launch_bounds__(256) budget_find_kernel(int H, int keep, int n_safe, const uint32_t* __restrict__ thr,
                                                          const int* __restrict__ bhist, int* __restrict__ bmeta) {
    __shared__ SelectShared S;
    const int g = blockIdx.x;
    const int rest = H * keep - H * n_safe;
    if (rest <= 0) {
        if (threadIdx.x == 0) bmeta[g * kBudgetMeta] = -1;
        return;
    }
    for (int b = threadIdx.x; b < kBins; b += blockDim.x) {
        int c = 0;
        for (int h = 0; h < H; ++h) {
            const int64_t u = (int64_t)g * H + h;
            c += bhist[u * kBins + b];
            // of the scores tied at the safeguard threshold, thr[2u+1] belong to the safeguard, not to the pool
            if (score_bin(ord_float(thr[u * 2])) == b) c -= (int)thr[u * 2 + 1];
        }
        S.hist[b] = c;
    }
    if (threadIdx.x == 0) {
        S.bin = -1;
        S.above = 0;
    }
    __syncthreads();
    find_bin_desc(S, rest);
    __syncthreads();
    if (threadIdx.x == 0) {
        bmeta[g * kBudgetMeta] = S.bin;                 // -1: fewer pool scores than slots (cannot happen: rest <= pool)
        bmeta[g * kBudgetMeta + 1] = rest - S.above;    // rank wanted among the bin's scores, from the top
    }
}

// step 3: the pool scores of that bin, with their heads, into the group's candidate list
__global__ void __launch_bounds__(256) budget_collect_kernel(int H, int N, const float* __restrict__ a_star,
                                                             const uint32_t* __restrict__ thr, int* __restrict__ bmeta,
                                                             float* __restrict__ cand_v, unsigned char* __restrict__ cand_h) {
    const int u = blockIdx.y, g = u / H, h = u - g * H;
    const int bin = bmeta[g * kBudgetMeta];
    if (bin < 0) return;
    const int j0 = blockIdx.x * kBudgetChunk, j1 = min(N, j0 + kBudgetChunk);
    const uint32_t T = thr[(int64_t)u * 2];
    const float* v = a_star + (int64_t)u * N;
    const int lane = threadIdx.x & 31;
    for (int jb = j0; jb < j1; jb += blockDim.x) {
        const int j = jb + threadIdx.x;
        const float x = j < j1 ? v[j] : 0.f;
        const bool mine = j < j1 && ord_key(x) <= T && score_bin(x) == bin;
        const unsigned ballot = __ballot_sync(0xffffffffu, mine);
        if (ballot) {
            int base = 0;
            if (lane == 0) base = atomicAdd(&bmeta[g * kBudgetMeta + 2], __popc(ballot));
            base = __shfl_sync(0xffffffffu, base, 0);
            const int pos = base + __popc(ballot & ((1u << lane) - 1u));
            if (mine && pos < kBudgetCand) {
                cand_v[(int64_t)g * kBudgetCand + pos] = x;
                cand_h[(int64_t)g * kBudgetCand + pos] = (unsigned char)h;
            }
        }
    }
}

// step 4: one CTA per group finishes exactly on the candidates and turns counts into budgets.  A group whose
// candidate list overflowed (scores packed into one bin) is left to budget_kernel.
__global__ void __launch_bounds__(kThreads) budget_finish_kernel(int H, int keep, int n_safe,
                                                                 const int* __restrict__ bhist, int* __restrict__ bmeta,
                                                                 const float* __restrict__ cand_v,
                                                                 const unsigned char* __restrict__ cand_h,
                                                                 int32_t* __restrict__ budgets, uint32_t* __restrict__ thr,
                                                                 int* status) {
    __shared__ SelectShared S;
    extern __shared__ __align__(16) unsigned char finish_dyn[];
    float* cv = reinterpret_cast<float*>(finish_dyn);
    unsigned char* ch = finish_dyn + kBudgetCand * sizeof(float);
    __shared__ uint32_t T[kMaxCorr];
    __shared__ int corr[kMaxCorr], cnt_mid[kMaxCorr], cnt_eq[kMaxCorr];
    const int g = blockIdx.x, tid = threadIdx.x;
    const int bin = bmeta[g * kBudgetMeta], need = bmeta[g * kBudgetMeta + 1], nc = bmeta[g * kBudgetMeta + 2];
    if (bin >= 0 && nc > kBudgetCand) {
        if (tid == 0) bmeta[g * kBudgetMeta + 3] = 1;
        return;
    }
    if (tid < H) {
        T[tid] = thr[((int64_t)g * H + tid) * 2];
        corr[tid] = (int)thr[((int64_t)g * H + tid) * 2 + 1];
    }
    if (tid == 0) S.ncorr = 0;
    __syncthreads();
    const int rest = H * keep - H * n_safe;
    uint32_t tau = 0xffffffffu;
    if (bin >= 0) {
        for (int j = tid; j < nc; j += blockDim.x) {
            cv[j] = cand_v[(int64_t)g * kBudgetCand + j];
            ch[j] = cand_h[(int64_t)g * kBudgetCand + j];
        }
        if (tid == 0) {
            // safeguard ties that sit among the candidates do not compete
            int n = 0;
            for (int h = 0; h < H; ++h)
                if (corr[h] > 0 && score_bin(ord_float(T[h])) == bin) {
                    S.corr_v[n] = ord_float(T[h]);
                    S.corr_m[n] = corr[h];
                    ++n;
                }
            S.ncorr = n;
        }
        __syncthreads();
        SmemSrc src{cv};
        block_select_desc(S, src, nc, need, (float)bin / (float)kBins, (float)kBins * (float)kBins, status);
        tau = S.theta;
        __syncthreads();
    }
    // per head: pool scores above tau (whole bins above the threshold's bin plus candidates) and equal to it
    for (int h = 0; h < H; ++h) {
        int mid = 0, eq = 0;
        if (bin >= 0) {
            const int* hh = bhist + ((int64_t)g * H + h) * kBins;
            for (int b = bin + 1 + tid; b < kBins; b += blockDim.x) mid += hh[b];
            for (int j = tid; j < nc; j += blockDim.x)
                if (ch[j] == h) {
                    const uint32_t key = ord_key(cv[j]);
                    mid += key > tau;
                    eq += key == tau;
                }
        }
        mid = block_sum_int(S, mid);
        __syncthreads();
        eq = block_sum_int(S, eq);
        if (tid == 0) {
            cnt_mid[h] = mid;
            cnt_eq[h] = eq;
        }
        __syncthreads();
    }
    if (tid == 0) {
        int taken_gt = 0;
        for (int h = 0; h < H; ++h) taken_gt += cnt_mid[h] - (T[h] > tau ? corr[h] : 0);
        int remaining = rest - taken_gt;
        int total = 0;
        for (int h = 0; h < H; ++h) {
            const int pool_eq = cnt_eq[h] - (T[h] == tau ? corr[h] : 0);
            const int t = max(0, min(pool_eq, remaining));
            remaining -= t;
            const int B = n_safe + cnt_mid[h] - (T[h] > tau ? corr[h] : 0) + t;
            budgets[(int64_t)g * H + h] = B;
            total += B;
            uint32_t theta, q;
            if (tau < T[h]) {
                theta = tau;
                q = (uint32_t)t;
            } else {
                theta = T[h];
                q = (uint32_t)(corr[h] + t);
            }
            thr[((int64_t)g * H + h) * 2] = theta;
            thr[((int64_t)g * H + h) * 2 + 1] = q;
        }
        if (total != H * keep || remaining != 0) set_status(status, NKV_ERR_DEVICE_CHECK, 202);
    }
}

// ------------------------------------------------------------------------------------------
// select: one CTA per head, ordered compaction of the retained positions.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) warp_tot[w] = incl;
    __syncthreads();
    if (w == 0) {
        int t = warp_tot[lane];
        int ti = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, ti, o);
            if (lane >= o) ti += y;
        }
        warp_tot[lane] = ti - t;
        if (lane == 31) *total = ti;
    }
    __syncthreads();
    return warp_tot[w] + incl - v;
}

__global__ void __launch_bounds__(kThreads) select_kernel(int H, int N, int64_t cap, const float* __restrict__ a_star,
                                                          const int32_t* __restrict__ budgets,
                                                          const uint32_t* __restrict__ thr, int32_t* __restrict__ idx,
                                                          int32_t* __restrict__ head_offsets, int* status) {
    __shared__ SelectShared S;
    __shared__ int warp_tot[32];
    __shared__ int tot;
    const int u = blockIdx.x, g = u / H, h = u % H;
    const float* v = a_star + (int64_t)u * N;
    const int B = budgets[u];
    int off = 0;
    for (int hh = 0; hh < h; ++hh) off += budgets[(int64_t)g * H + hh];
    if (threadIdx.x == 0) {
        head_offsets[(int64_t)g * (H + 1) + h] = off;
        if (h == H - 1) head_offsets[(int64_t)g * (H + 1) + H] = off + B;
        S.ncorr = 0;
    }
    __syncthreads();
    if (B <= 0) return;
    if (B > N || off + B > cap) {
        if (threadIdx.x == 0) set_status(status, NKV_ERR_DEVICE_CHECK, 301);
        return;
    }
    uint32_t theta;
    int q;
    if (thr) {
        theta = thr[(int64_t)u * 2];
        q = (int)thr[(int64_t)u * 2 + 1];
    } else {
        HeadSrc src{v, N};
        block_select_desc(S, src, N, B, 0.f, (float)kBins, status);
        theta = S.theta;
        q = B - S.gt;
        __syncthreads();
    }
    int run_eq = 0, run_sel = 0;
    // the four scores of the next round are fetched before the scans of this one
    float nxt[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) nxt[e] = (threadIdx.x * 4 + e < N) ? v[threadIdx.x * 4 + e] : 0.f;
    for (int base = 0; base < N; base += kThreads * 4) {
        const int j0 = base + threadIdx.x * 4;
        uint32_t key[4];
        int eq_cnt = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            key[e] = (j0 + e < N) ? ord_key(nxt[e]) : 0u;
            eq_cnt += (j0 + e < N && key[e] == theta);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int jn = j0 + kThreads * 4 + e;
            nxt[e] = jn < N ? v[jn] : 0.f;
        }
        // ties at the threshold are rare: their ranks need a scan only in rounds that hold one
        int t_eq = 0, tie_rank = run_eq;
        if (__syncthreads_or(eq_cnt)) {
            tie_rank += block_exclusive_scan(eq_cnt, warp_tot, &tot);
            t_eq = tot;
            __syncthreads();
        }
        int sel[4], sel_cnt = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool in = j0 + e < N;
            const bool is_eq = in && key[e] == theta;
            sel[e] = in && (key[e] > theta || (is_eq && tie_rank < q));
            tie_rank += is_eq;
            sel_cnt += sel[e];
        }
        int pos = run_sel + block_exclusive_scan(sel_cnt, warp_tot, &tot);
        const int t_sel = tot;
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (sel[e]) {
                if (pos < B) idx[(int64_t)g * cap + off + pos] = j0 + e;
                ++pos;
            }
        run_eq += t_eq;
        run_sel += t_sel;
    }
    if (threadIdx.x == 0 && run_sel != B) set_status(status, NKV_ERR_DEVICE_CHECK, 302);
}

// ranks: place of token i in its head's order (score descending, position ascending).  O(N^2).
__global__ void __launch_bounds__(256) ranks_kernel(int N, const float* __restrict__ a_star, int32_t* __restrict__ ranks) {
    __shared__ uint32_t tile[1024];
    const int u = blockIdx.y;
    const float* v = a_star + (int64_t)u * N;
    const int i = blockIdx.x * 256 + threadIdx.x;
    const uint32_t mine = i < N ? ord_key(v[i]) : 0u;
    int r = 0;
    for (int base = 0; base < N; base += 1024) {
        __syncthreads();
        for (int t = threadIdx.x; t < 1024; t += 256) tile[t] = (base + t < N) ? ord_key(v[base + t]) : 0u;
        __syncthreads();
        const int lim = min(1024, N - base);
        for (int t = 0; t < lim; ++t) {
            const uint32_t y = tile[t];
            r += (y > mine) || (y == mine && base + t < i);
        }
    }
    if (i < N) ranks[(int64_t)u * N + i] = r;
}

}  // namespace

cudaError_t launch_head_scores(int units, int N, const ScoreParams& sp, const float* a_raw,
                               const uint32_t* minmax_keys, float* a_star, float* head_stats_opt, float* hstat,
                               int* status, cudaStream_t stream, int64_t* launches) {
    // long heads: four times the threads per head (the per-head work is one CTA's)
    if (N >= 65536) scale_stats_kernel<1024><<<units * 4, 1024, 0, stream>>>(N, sp, a_raw, minmax_keys, hstat, status);
    else scale_stats_kernel<kStatThreads><<<units * 4, kStatThreads, 0, stream>>>(N, sp, a_raw, minmax_keys, hstat, status);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dim3 grid((N + kMixThreads * kMixPerThread - 1) / (kMixThreads * kMixPerThread), units);
    mix_kernel<<<grid, kMixThreads, 0, stream>>>(N, sp, a_raw, minmax_keys, hstat, a_star, head_stats_opt);
    ++*launches;
    return cudaGetLastError();
}

size_t head_stat_bytes(int64_t units) { return (size_t)units * kHeadStat * sizeof(float); }

// Raises the dynamic shared-memory limit of the group kernel on the current device (once per device;
// callers without a handle reach the kernel through launch_budget, which calls this too).
cudaError_t configure_select_kernels() {
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(budget_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)sizeof(BracketShared<kCandLarge>));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(budget_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBudgetCand * 5);
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

namespace {
// the score of a head's last retained token, from the ordered key the budget kernels leave per head
__global__ void threshold_scores_kernel(int units, const uint32_t* __restrict__ thr, float* __restrict__ out) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u < units) out[u] = ord_float(thr[2 * (int64_t)u]);
}
}  // namespace

cudaError_t launch_threshold_scores(int units, const uint32_t* thr, float* out, cudaStream_t stream, int64_t* launches) {
    threshold_scores_kernel<<<(units + 255) / 256, 256, 0, stream>>>(units, thr, out);
    ++*launches;
    return cudaGetLastError();
}

size_t budget_scratch_bytes(int64_t G, int64_t H) {
    return (size_t)G * H * kBins * sizeof(int) + (size_t)G * 256 + (size_t)G * kBudgetCand * 5;
}

// `scratch` (budget_scratch_bytes, 256-byte aligned) or null: with it, calls large enough to pay for the extra
// launches run the parallel form of the group competition.
cudaError_t launch_budget(int G, int H, int N, int keep, int n_safe, const float* a_star, int32_t* budgets,
                          uint32_t* sel_thresholds, int* status, void* scratch, cudaStream_t stream,
                          int64_t* launches) {
    if (H > kMaxCorr) return cudaErrorInvalidValue;
    cudaError_t cfg = configure_select_kernels();
    if (cfg != cudaSuccess) return cfg;
    if (N >= 65536) safeguard_kernel<1024><<<G * H, 1024, 0, stream>>>(N, n_safe, a_star, sel_thresholds, status);
    else safeguard_kernel<kStatThreads><<<G * H, kStatThreads, 0, stream>>>(N, n_safe, a_star, sel_thresholds, status);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int* flagged = nullptr;
    // with a group per SM or so the one-CTA kernel already fills the GPU and reads the scores once
    if (scratch && (int64_t)H * N >= 200000 && G <= 64) {
        unsigned char* base = static_cast<unsigned char*>(scratch);
        int* bhist = reinterpret_cast<int*>(base);
        int* bmeta = reinterpret_cast<int*>(base + (size_t)G * H * kBins * sizeof(int));
        float* cand_v = reinterpret_cast<float*>(base + (size_t)G * H * kBins * sizeof(int) + (size_t)G * 256);
        unsigned char* cand_h = reinterpret_cast<unsigned char*>(cand_v + (size_t)G * kBudgetCand);
        e = cudaMemsetAsync(base, 0, (size_t)G * H * kBins * sizeof(int) + (size_t)G * 256, stream);
        if (e != cudaSuccess) return e;
        const dim3 grid((unsigned)((N + kBudgetChunk - 1) / kBudgetChunk), (unsigned)(G * H));
        budget_hist_kernel<<<grid, 256, 0, stream>>>(N, a_star, sel_thresholds, bhist);
        budget_find_kernel<<<G, 256, 0, stream>>>(H, keep, n_safe, sel_thresholds, bhist, bmeta);
        budget_collect_kernel<<<grid, 256, 0, stream>>>(H, N, a_star, sel_thresholds, bmeta, cand_v, cand_h);
        budget_finish_kernel<<<G, kThreads, kBudgetCand * 5, stream>>>(H, keep, n_safe, bhist, bmeta, cand_v, cand_h, budgets,
                                                                      sel_thresholds, status);
        *launches += 4;
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        flagged = bmeta;
    }
    budget_kernel<<<G, kThreads, sizeof(BracketShared<kCandLarge>), stream>>>(H, N, keep, n_safe, a_star, budgets,
                                                                                 sel_thresholds, status, flagged);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_select(int G, int H, int N, int64_t idx_capacity, const float* a_star, const int32_t* budgets,
                          const uint32_t* sel_thresholds_or_null, int32_t* idx, int32_t* head_offsets, int* status,
                          cudaStream_t stream, int64_t* launches) {
    select_kernel<<<G * H, kThreads, 0, stream>>>(H, N, idx_capacity, a_star, budgets, sel_thresholds_or_null, idx,
                                                  head_offsets, status);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_ranks(int units, int N, const float* a_star, int32_t* ranks, cudaStream_t stream,
                         int64_t* launches) {
    dim3 grid((N + 255) / 256, units);
    ranks_kernel<<<grid, 256, 0, stream>>>(N, a_star, ranks);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv
