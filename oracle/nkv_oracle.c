/*
 * NestedKV compression oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU statement of what the compression path
 * computes, written from the paper's definitions in the paper's order.  All
 * floating point is double; inputs (bf16, fp16 or fp32 bytes) are widened exactly.
 * There is no blocking, fusion, running sum or reordering: the sliding-window
 * mean is summed directly for every token and ranks come from full sorts.
 *
 * It shares no code with the CUDA library and must never be called from the
 * product path: only tests, the smoke check and the bench's CPU-baseline legs
 * may use it.
 *
 * Readings taken where the paper is silent (each is also a special case the
 * tests exercise):
 *   - eps: a norm used as a denominator is max(norm, 1e-12);
 *   - min-max of a constant sequence is identically 0;
 *   - sinks take part in every per-head statistic with their natural values and
 *     are pinned to +inf only on the final score (Section 2.3, last sentence);
 *   - top_p / bot_p use m = max(1, floor(p*N)) tokens;
 *   - std over the three scales is the population form (the following per-head
 *     min-max removes any constant factor);
 *   - surprise is min-max normalised per head, then mean-centred, then rectified
 *     (Appendix A, Hyperparameters), and the gate threshold acts on that value;
 *   - cross-head competition uses the final pinned score, with the total order
 *     (score descending, head ascending, position ascending);
 *   - layer budget is H * floor((1-r)*N); safeguard floor(0.20 * floor((1-r)N)).
 *
 * Pins: tests/test_oracle_*.py (closed forms, invariants, textbook special
 * cases and brute force on tiny inputs).  The paper prints no worked example;
 * the surprise -> gate -> final-score chain is pinned by a head constructed so
 * that every quantity has a closed form.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define NKVO_BF16 0
#define NKVO_F16 2
#define NKVO_F32 1

#define NKVO_GATE_SURPRISE 0
#define NKVO_GATE_AVERAGE 1
#define NKVO_GATE_MAX 2

typedef struct {
    int32_t window;       /* W, Eq. for the current memory (Section 2.2) */
    int32_t n_sink;       /* pinned prefix (Section 2.3) */
    int32_t block_div;    /* 32 in b = clip(floor(N/32), 128, 256) */
    int32_t block_min;
    int32_t block_max;
    int32_t gate_mode;    /* surprise gate, or the "only average"/"only max" ablations */
    double top_frac;      /* p = 10% */
    double prior[3];      /* (w_s^0, w_e^0, w_c^0) */
    double beta;
    double tau;
    double kappa;
    double safeguard;     /* alpha_s = 0.20 */
} nkvo_params;

void nkvo_default_params(nkvo_params* p) {
    /* Appendix A, Hyperparameters. */
    p->window = 64;
    p->n_sink = 4;
    p->block_div = 32;
    p->block_min = 128;
    p->block_max = 256;
    p->gate_mode = NKVO_GATE_SURPRISE;
    p->top_frac = 0.10;
    p->prior[0] = 0.4;
    p->prior[1] = 0.4;
    p->prior[2] = 0.2;
    p->beta = 3.0;
    p->tau = 0.60;
    p->kappa = 10.0;
    p->safeguard = 0.20;
}

static double widen(const void* base, int dtype, int64_t index) {
    if (dtype == NKVO_F32) {
        return (double)((const float*)base)[index];
    } else if (dtype == NKVO_F16) {
        /* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits; every value is exact in double */
        uint16_t h = ((const uint16_t*)base)[index];
        int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
        double v;
        if (e == 0) v = ldexp((double)f, -24);
        else if (e == 31) v = f ? NAN : INFINITY;
        else v = ldexp((double)(1024 + f), e - 25);
        return sign ? -v : v;
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t*)base)[index]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* Section 2.2, block size of the episodic memory. */
int64_t nkvo_block_size(int64_t N, const nkvo_params* p) {
    int64_t b = N / p->block_div;
    if (b < p->block_min) b = p->block_min;
    if (b > p->block_max) b = p->block_max;
    return b;
}

int64_t nkvo_num_blocks(int64_t N, const nkvo_params* p) {
    int64_t b = nkvo_block_size(N, p);
    return (N + b - 1) / b;
}

/* Section 2.6 / Appendix A: k = floor((1-r) N), n_safe = floor(alpha_s * k). */
int64_t nkvo_keep_per_head(int64_t N, double r) { return (int64_t)floor((1.0 - r) * (double)N); }
int64_t nkvo_safeguard_count(int64_t N, double r, const nkvo_params* p) {
    return (int64_t)floor(p->safeguard * (double)nkvo_keep_per_head(N, r));
}
int64_t nkvo_top_count(int64_t N, const nkvo_params* p) {
    int64_t m = (int64_t)floor(p->top_frac * (double)N);
    return m < 1 ? 1 : m;
}

static double norm2(const double* v, int64_t d) {
    double s = 0.0;
    for (int64_t c = 0; c < d; ++c) s += v[c] * v[c];
    return sqrt(s);
}

static double neg_cos(const double* a, const double* b, int64_t d) {
    /* a_k(i) = -cos(k_hat_i, mu_k)   (Section 2.3) */
    double dot = 0.0;
    for (int64_t c = 0; c < d; ++c) dot += a[c] * b[c];
    double na = norm2(a, d), nb = norm2(b, d);
    if (na < 1e-12) na = 1e-12;
    if (nb < 1e-12) nb = 1e-12;
    return -dot / (na * nb);
}

static int cmp_double_asc(const void* x, const void* y) {
    double a = *(const double*)x, b = *(const double*)y;
    return (a > b) - (a < b);
}

static void minmax_normalise(const double* a, int64_t N, double* out, double* lo_out, double* hi_out) {
    double lo = a[0], hi = a[0];
    for (int64_t i = 1; i < N; ++i) {
        if (a[i] < lo) lo = a[i];
        if (a[i] > hi) hi = a[i];
    }
    for (int64_t i = 0; i < N; ++i) out[i] = (hi > lo) ? (a[i] - lo) / (hi - lo) : 0.0;
    *lo_out = lo;
    *hi_out = hi;
}

/*
 * One (layer, KV head): Sections 2.1-2.4.
 *
 * K: N rows of d elements, row stride `stride_n` elements.
 * Outputs (any may be NULL except a_star):
 *   inv_norm[N]           1 / max(||k_i||, eps)
 *   mu_s[d], mu_e[nb*d], mu_c[N*d]
 *   a_raw[3*N]            a_s, a_e, a_c (scale-major)
 *   stats[16]             lo_s,lo_e,lo_c, hi_s,hi_e,hi_c, D_s,D_e,D_c, w_s,w_e,w_c,
 *                         min s, max s, mean of normalised s, m
 *   a_star[N]             final score rounded once to fp32, sinks = +inf
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int nkvo_score_head(const void* K, int dtype, int64_t N, int64_t d, int64_t stride_n,
                    const nkvo_params* p, double* inv_norm, double* mu_s_out, double* mu_e_out,
                    double* mu_c_out, double* a_raw_out, double* stats_out, float* a_star) {
    if (!K || !p || !a_star || N < 1 || d < 1) return -1;
    const int64_t b = nkvo_block_size(N, p);
    const int64_t nb = (N + b - 1) / b;
    const int64_t W = p->window;

    double* khat = (double*)malloc(sizeof(double) * (size_t)(N * d));
    double* mu_s = (double*)calloc((size_t)d, sizeof(double));
    double* mu_e = (double*)calloc((size_t)(nb * d), sizeof(double));
    double* mu_c = (double*)malloc(sizeof(double) * (size_t)d);
    double* a = (double*)malloc(sizeof(double) * (size_t)(3 * N));
    double* an = (double*)malloc(sizeof(double) * (size_t)(3 * N));
    double* s = (double*)malloc(sizeof(double) * (size_t)N);
    double* sn = (double*)malloc(sizeof(double) * (size_t)N);
    double* sorted = (double*)malloc(sizeof(double) * (size_t)N);
    if (!khat || !mu_s || !mu_e || !mu_c || !a || !an || !s || !sn || !sorted) {
        free(khat); free(mu_s); free(mu_e); free(mu_c); free(a); free(an); free(s); free(sn); free(sorted);
        return -1;
    }

    /* k_hat_i = k_i / ||k_i||_2   (Section 2.1) */
    for (int64_t i = 0; i < N; ++i) {
        double ss = 0.0;
        for (int64_t c = 0; c < d; ++c) {
            double x = widen(K, dtype, i * stride_n + c);
            khat[i * d + c] = x;
            ss += x * x;
        }
        double n = sqrt(ss);
        if (n < 1e-12) n = 1e-12;
        for (int64_t c = 0; c < d; ++c) khat[i * d + c] /= n;
        if (inv_norm) inv_norm[i] = 1.0 / n;
    }

    /* mu_s = (1/N) sum_j k_hat_j   (stable memory) */
    for (int64_t i = 0; i < N; ++i)
        for (int64_t c = 0; c < d; ++c) mu_s[c] += khat[i * d + c];
    for (int64_t c = 0; c < d; ++c) mu_s[c] /= (double)N;

    /* mu_e(i) = mean of k_hat over the block containing i   (episodic memory) */
    for (int64_t t = 0; t < nb; ++t) {
        int64_t lo = t * b, hi = lo + b < N ? lo + b : N;
        for (int64_t i = lo; i < hi; ++i)
            for (int64_t c = 0; c < d; ++c) mu_e[t * d + c] += khat[i * d + c];
        for (int64_t c = 0; c < d; ++c) mu_e[t * d + c] /= (double)(hi - lo);
    }

    /* anomalies, with mu_c(i) = mean over j = max(first, i-W+1) .. i   (current memory) */
    for (int64_t i = 0; i < N; ++i) {
        int64_t l = i - W + 1;
        if (l < 0) l = 0;
        for (int64_t c = 0; c < d; ++c) mu_c[c] = 0.0;
        for (int64_t j = l; j <= i; ++j)
            for (int64_t c = 0; c < d; ++c) mu_c[c] += khat[j * d + c];
        for (int64_t c = 0; c < d; ++c) mu_c[c] /= (double)(i - l + 1);
        if (mu_c_out) memcpy(mu_c_out + i * d, mu_c, sizeof(double) * (size_t)d);
        a[0 * N + i] = neg_cos(khat + i * d, mu_s, d);
        a[1 * N + i] = neg_cos(khat + i * d, mu_e + (i / b) * d, d);
        a[2 * N + i] = neg_cos(khat + i * d, mu_c, d);
    }

    /* per-head min-max normalisation of each scale (Section 2.3) */
    double lo[3], hi[3];
    for (int k = 0; k < 3; ++k) minmax_normalise(a + k * N, N, an + k * N, &lo[k], &hi[k]);

    /* reliability gaps: mean of the top p minus mean of the bottom p (Section 2.4) */
    const int64_t m = nkvo_top_count(N, p);
    double delta[3];
    for (int k = 0; k < 3; ++k) {
        memcpy(sorted, an + k * N, sizeof(double) * (size_t)N);
        qsort(sorted, (size_t)N, sizeof(double), cmp_double_asc);
        double top = 0.0, bot = 0.0;
        for (int64_t j = 0; j < m; ++j) {
            bot += sorted[j];
            top += sorted[N - 1 - j];
        }
        delta[k] = top / (double)m - bot / (double)m;
    }

    /* w = softmax(log w0 + beta * Delta) */
    double z[3], zmax, w[3], wsum = 0.0;
    for (int k = 0; k < 3; ++k) z[k] = log(p->prior[k]) + p->beta * delta[k];
    zmax = z[0];
    for (int k = 1; k < 3; ++k) if (z[k] > zmax) zmax = z[k];
    for (int k = 0; k < 3; ++k) { w[k] = exp(z[k] - zmax); wsum += w[k]; }
    for (int k = 0; k < 3; ++k) w[k] /= wsum;

    /* surprise: std over the three normalised readings, then per-head min-max,
       mean-centre, rectify (Appendix A) */
    for (int64_t i = 0; i < N; ++i) {
        double x0 = an[i], x1 = an[N + i], x2 = an[2 * N + i];
        double mean = (x0 + x1 + x2) / 3.0;
        double var = ((x0 - mean) * (x0 - mean) + (x1 - mean) * (x1 - mean) + (x2 - mean) * (x2 - mean)) / 3.0;
        s[i] = sqrt(var);
    }
    double s_lo, s_hi, s_mean = 0.0;
    minmax_normalise(s, N, sn, &s_lo, &s_hi);
    for (int64_t i = 0; i < N; ++i) s_mean += sn[i];
    s_mean /= (double)N;

    /* routed score, rounded once to fp32; then sink pinning */
    for (int64_t i = 0; i < N; ++i) {
        double x0 = an[i], x1 = an[N + i], x2 = an[2 * N + i];
        double blend = w[0] * x0 + w[1] * x1 + w[2] * x2;
        double win = x0;
        if (x1 > win) win = x1;
        if (x2 > win) win = x2;
        double sp = sn[i] - s_mean;
        if (sp < 0.0) sp = 0.0;
        double alpha;
        if (p->gate_mode == NKVO_GATE_AVERAGE) alpha = 0.0;
        else if (p->gate_mode == NKVO_GATE_MAX) alpha = 1.0;
        else alpha = 1.0 / (1.0 + exp(-p->kappa * (sp - p->tau)));
        a_star[i] = (float)((1.0 - alpha) * blend + alpha * win);
    }
    for (int64_t i = 0; i < N && i < p->n_sink; ++i) a_star[i] = INFINITY;

    if (mu_s_out) memcpy(mu_s_out, mu_s, sizeof(double) * (size_t)d);
    if (mu_e_out) memcpy(mu_e_out, mu_e, sizeof(double) * (size_t)(nb * d));
    if (a_raw_out) memcpy(a_raw_out, a, sizeof(double) * (size_t)(3 * N));
    if (stats_out) {
        for (int k = 0; k < 3; ++k) {
            stats_out[k] = lo[k];
            stats_out[3 + k] = hi[k];
            stats_out[6 + k] = delta[k];
            stats_out[9 + k] = w[k];
        }
        stats_out[12] = s_lo;
        stats_out[13] = s_hi;
        stats_out[14] = s_mean;
        stats_out[15] = (double)m;
    }
    free(khat); free(mu_s); free(mu_e); free(mu_c); free(a); free(an); free(s); free(sn); free(sorted);
    return 0;
}

typedef struct {
    float score;
    int32_t head;
    int32_t pos;
} pair_t;

/* total order: larger score first, then smaller head, then smaller position */
static int cmp_pair(const void* x, const void* y) {
    const pair_t* a = (const pair_t*)x;
    const pair_t* b = (const pair_t*)y;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    if (a->head != b->head) return a->head < b->head ? -1 : 1;
    if (a->pos != b->pos) return a->pos < b->pos ? -1 : 1;
    return 0;
}

/*
 * One layer group (H heads of one sequence): Sections 2.5-2.6.
 *
 * a_star: [H, N] fp32 final scores (sinks already +inf).
 * budgets[H]; idx[H*k] retained positions, ascending inside each head, heads
 * concatenated; offsets[H+1]; ranks[H*N] (optional) = place of each token in
 * its head's order.  Returns 0, or -1 on bad arguments.
 */
int nkvo_budget_select(const float* a_star, int64_t H, int64_t N, double r, const nkvo_params* p,
                       int32_t* budgets, int32_t* idx, int32_t* offsets, int32_t* ranks) {
    if (!a_star || !p || !budgets || H < 1 || N < 1) return -1;
    const int64_t k = nkvo_keep_per_head(N, r);
    if (k < 1 || k > N) return -1;
    int64_t n_safe = nkvo_safeguard_count(N, r, p);
    if (n_safe > k) n_safe = k;
    const int64_t layer_budget = H * k;

    pair_t* all = (pair_t*)malloc(sizeof(pair_t) * (size_t)(H * N));
    pair_t* pool = (pair_t*)malloc(sizeof(pair_t) * (size_t)(H * N));
    if (!all || !pool) { free(all); free(pool); return -1; }

    /* each head's own order; its first n_safe pairs are the safeguard */
    int64_t n_pool = 0;
    for (int64_t h = 0; h < H; ++h) {
        pair_t* row = all + h * N;
        for (int64_t i = 0; i < N; ++i) {
            row[i].score = a_star[h * N + i];
            row[i].head = (int32_t)h;
            row[i].pos = (int32_t)i;
        }
        qsort(row, (size_t)N, sizeof(pair_t), cmp_pair);
        if (ranks)
            for (int64_t j = 0; j < N; ++j) ranks[h * N + row[j].pos] = (int32_t)j;
        budgets[h] = (int32_t)n_safe;
        for (int64_t j = n_safe; j < N; ++j) pool[n_pool++] = row[j];
    }

    /* the rest of the layer budget goes to the globally largest unmarked pairs */
    qsort(pool, (size_t)n_pool, sizeof(pair_t), cmp_pair);
    const int64_t rest = layer_budget - H * n_safe;
    for (int64_t j = 0; j < rest; ++j) budgets[pool[j].head] += 1;

    /* each head keeps its top B_h, reported in ascending position */
    if (idx && offsets) {
        int64_t o = 0;
        for (int64_t h = 0; h < H; ++h) {
            offsets[h] = (int32_t)o;
            const pair_t* row = all + h * N;
            const int64_t B = budgets[h];
            unsigned char* keep = (unsigned char*)calloc((size_t)N, 1);
            if (!keep) { free(all); free(pool); return -1; }
            for (int64_t j = 0; j < B; ++j) keep[row[j].pos] = 1;
            for (int64_t i = 0; i < N; ++i)
                if (keep[i]) idx[o++] = (int32_t)i;
            free(keep);
        }
        offsets[H] = (int32_t)o;
    }
    free(all);
    free(pool);
    return 0;
}

/*
 * Compaction: retained rows copied verbatim, heads concatenated per group.
 * src: [H, N, row_bytes] with head stride `stride_h_bytes`; dst: [sum B_h, row_bytes].
 */
int nkvo_compact(const void* src, int64_t H, int64_t N, int64_t row_bytes, int64_t stride_h_bytes,
                 int64_t stride_n_bytes, const int32_t* idx, const int32_t* offsets, void* dst) {
    if (!src || !idx || !offsets || !dst) return -1;
    for (int64_t h = 0; h < H; ++h)
        for (int64_t j = offsets[h]; j < offsets[h + 1]; ++j) {
            if (idx[j] < 0 || idx[j] >= N) return -1;
            memcpy((char*)dst + j * row_bytes,
                   (const char*)src + h * stride_h_bytes + (int64_t)idx[j] * stride_n_bytes,
                   (size_t)row_bytes);
        }
    return 0;
}
