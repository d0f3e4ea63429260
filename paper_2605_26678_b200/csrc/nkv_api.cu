// C ABI of the nkv library: argument checking, workspace carving and launch order.
#include <math.h>
#include <new>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "nkv_common.cuh"

using namespace nkv;

struct nkv_handle {
    int device;
    int sm_count;
    int l2_bytes;
    int64_t launches;
    int timing;
    int timing_valid;
    int key_pass;     // NKV_KEY_PASS_*: which kernels make the two key passes
    cudaEvent_t ev[NKV_NUM_STAGES + 1];
    cudaStream_t copy_streams[2];
    cudaEvent_t slot_done[2];
    int* chunk_status;   // pinned host copy of every chunk's status words (nkv_compress_host)
    int inject_status;   // tests: status code planted in chunk `inject_chunk` of nkv_compress_host
    int inject_chunk;
};

constexpr int kMaxHostChunks = 4096;

namespace {

constexpr size_t kAlign = 256;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool params_ok(const nkv_params* p) {
    if (!p) return false;
    if (p->n_sink < 0 || p->block_div < 1 || p->block_min < 1 || p->block_max < p->block_min) return false;
    if (!(p->top_frac > 0.0 && p->top_frac <= 1.0)) return false;
    // a prior of zero switches its scale off (the single-anchor and no-current ablations); one must remain
    double prior_sum = 0.0;
    for (int k = 0; k < 3; ++k) {
        if (!(p->prior[k] >= 0.0) || !isfinite(p->prior[k])) return false;
        prior_sum += p->prior[k];
    }
    if (!(prior_sum > 0.0)) return false;
    if (!isfinite(p->beta) || !isfinite(p->tau) || !isfinite(p->kappa)) return false;
    if (!(p->safeguard >= 0.0 && p->safeguard <= 1.0)) return false;
    if (p->gate_mode < NKV_GATE_SURPRISE || p->gate_mode > NKV_GATE_MAX) return false;
    return true;
}

int64_t block_size(int64_t N, const nkv_params* p) {
    int64_t b = N / p->block_div;
    if (b < p->block_min) b = p->block_min;
    if (b > p->block_max) b = p->block_max;
    return b;
}

int64_t keep_count(int64_t N, double r) { return (int64_t)floor((1.0 - r) * (double)N); }

// Workspace carving shared by every entry point.
struct Layout {
    size_t status, inv_norm, mu_s, mu_e, inv_s, inv_e, mm, a_raw, a_star, thr, hstat, bscr, total;
};

Layout make_layout(int64_t G, int64_t units, int64_t N, int64_t d, int64_t nb) {
    Layout L;
    size_t o = 0;
    auto take = [&](size_t bytes) {
        size_t at = o;
        o += align_up(bytes);
        return at;
    };
    L.status = take(kStatusWords * sizeof(int));
    L.inv_norm = take((size_t)units * N * 4);
    L.mu_s = take((size_t)units * d * 4);
    L.mu_e = take((size_t)units * nb * d * 4);
    L.inv_s = take((size_t)units * 4);
    L.inv_e = take((size_t)units * nb * 4);
    L.mm = take((size_t)units * 6 * 4);
    L.a_raw = take((size_t)units * 3 * N * 4);
    L.a_star = take((size_t)units * N * 4);
    L.thr = take((size_t)units * 2 * 4);
    L.hstat = take(head_stat_bytes(units));
    L.bscr = take(budget_scratch_bytes(G, units / G));   // the heads per group divide the units
    L.total = o;
    return L;
}

int check_tensor(const nkv_tensor* t) {
    if (!t || !t->ptr) return NKV_ERR_INVALID_ARG;
    if (t->dtype != NKV_BF16 && t->dtype != NKV_F32 && t->dtype != NKV_F16) return NKV_ERR_UNSUPPORTED;
    if (t->d != 64 && t->d != 128) return NKV_ERR_UNSUPPORTED;
    if (t->G < 1 || t->H < 1 || t->N < 1) return NKV_ERR_INVALID_ARG;
    if (t->N > (int64_t)1 << 24 || t->G * t->H > (int64_t)1 << 24) return NKV_ERR_UNSUPPORTED;
    if (t->stride_n != t->d) return NKV_ERR_UNSUPPORTED;
    const int64_t eb = t->dtype == NKV_F32 ? 4 : 2;
    if (t->stride_h < t->N * t->d || t->stride_g < t->H * t->N * t->d) {
        // strides may be permuted (for instance heads outermost); only require non-overlap of rows
        if (t->stride_h < 1 || t->stride_g < 1) return NKV_ERR_INVALID_ARG;
    }
    if (((uintptr_t)t->ptr) % 16 != 0 || (t->stride_h * eb) % 16 != 0 || (t->stride_g * eb) % 16 != 0)
        return NKV_ERR_INVALID_ARG;
    return NKV_OK;
}

// Some score-side kernels put the heads on gridDim.y.
int check_units(int64_t units) { return units > 65535 ? NKV_ERR_UNSUPPORTED : NKV_OK; }

TensorView view_of(const nkv_tensor* t) {
    TensorView v;
    v.ptr = t->ptr;
    v.stride_g = t->stride_g;
    v.stride_h = t->stride_h;
    v.H = (int)t->H;
    v.N = (int)t->N;
    v.d = (int)t->d;
    return v;
}

int resolve_params(const nkv_params* p, int64_t N, ScoreParams* sp) {
    if (!params_ok(p)) return NKV_ERR_INVALID_ARG;
    // W = 1 makes the current anchor the key itself: a_c is the constant -1 and its per-head min-max would
    // normalise rounding noise, so the smallest window is 2
    if (p->window < 2 || p->window > kMaxWindow) return NKV_ERR_UNSUPPORTED;
    sp->window = p->window;
    sp->n_sink = p->n_sink;
    sp->block = (int)block_size(N, p);
    sp->nblocks = (int)((N + sp->block - 1) / sp->block);
    sp->gate_mode = p->gate_mode;
    int64_t m = (int64_t)floor(p->top_frac * (double)N);
    sp->top_m = (int)(m < 1 ? 1 : m);
    for (int k = 0; k < 3; ++k) sp->log_prior[k] = (float)log(p->prior[k]);
    sp->beta = (float)p->beta;
    sp->tau = (float)p->tau;
    sp->kappa = (float)p->kappa;
    return NKV_OK;
}

int check_ws(const void* ws, size_t ws_bytes, size_t need) {
    if (!ws || ((uintptr_t)ws) % kAlign != 0 || ws_bytes < need) return NKV_ERR_WORKSPACE;
    return NKV_OK;
}

template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(reinterpret_cast<unsigned char*>(ws) + off); }

// With NKV_TRACE set in the environment a failing CUDA call is named on stderr.
int cuda_failed(cudaError_t e, const char* what, int line) {
    static const bool trace = getenv("NKV_TRACE") != nullptr;
    if (trace) fprintf(stderr, "nkv: %s (nkv_api.cu:%d): %s\n", what, line, cudaGetErrorString(e));
    return NKV_ERR_CUDA;
}

#define CU(expr)                                                     \
    do {                                                             \
        cudaError_t e__ = (expr);                                    \
        if (e__ != cudaSuccess) return cuda_failed(e__, #expr, __LINE__); \
    } while (0)

// The workspace arrays of a run of groups that starts at group g0 (unit u0 = g0 * H).
struct Bufs {
    float *inv_norm, *mu_s, *mu_e, *inv_s, *inv_e, *a_raw, *hstat;
    uint32_t *mm, *thr;
    unsigned char* bscr;
};
Bufs bufs_at(void* ws, const Layout& L, int64_t g0, int64_t H, int64_t N, int64_t d, int64_t nb) {
    const int64_t u0 = g0 * H;
    Bufs b;
    b.inv_norm = at<float>(ws, L.inv_norm) + u0 * N;
    b.mu_s = at<float>(ws, L.mu_s) + u0 * d;
    b.mu_e = at<float>(ws, L.mu_e) + u0 * nb * d;
    b.inv_s = at<float>(ws, L.inv_s) + u0;
    b.inv_e = at<float>(ws, L.inv_e) + u0 * nb;
    b.a_raw = at<float>(ws, L.a_raw) + u0 * 3 * N;
    b.hstat = at<float>(ws, L.hstat) + head_stat_bytes(u0) / sizeof(float);
    b.mm = at<uint32_t>(ws, L.mm) + u0 * 6;
    b.thr = at<uint32_t>(ws, L.thr) + u0 * 2;
    b.bscr = at<unsigned char>(ws, L.bscr) + (g0 ? budget_scratch_bytes(g0, H) : 0);   // every term is linear in G
    return b;
}

// The two passes over the keys (Sections 2.1-2.3): afterwards the workspace holds 1/||k||, the anchors, the
// three raw anomalies and their per-head min/max keys.  `mark` is called once between the passes (stage
// timing).
template <typename Mark>
int key_scan(nkv_handle* h, const TensorView& kv, int dtype, int G, const ScoreParams& sp, const Bufs& B, int* status,
             cudaStream_t st, Mark&& mark) {
    const int units = G * kv.H, N = kv.N, d = kv.d;
    if (stream_path_supported(sp)) {
        // pass A: norms, block sums and the current-memory anomaly; pass B: the two anchor anomalies
        // the tensor-core form walks whole heads, one CTA each: by default it runs when the heads fill
        // the SMs to at least 85 % over its waves (below that the FMA form, which splits heads, is faster)
        const int waves = (units + h->sm_count - 1) / h->sm_count;
        const bool fills = (double)units >= 0.85 * (double)waves * (double)h->sm_count;
        const bool tensor_ok = h->key_pass != NKV_KEY_PASS_FMA && gram_pass_supported(kv, dtype, sp) &&
                               (h->key_pass == NKV_KEY_PASS_TENSOR || fills);
        if (tensor_ok)
            CU(launch_gram_pass(kv, G, sp, B.mu_e, B.inv_norm, B.a_raw,
                                B.mm, status, h->sm_count, st, &h->launches));
        else
            CU(launch_stream_a(kv, dtype, G, sp, B.mu_e, B.inv_norm,
                               B.a_raw, B.mm, status, h->sm_count, st,
                               &h->launches));
        CU(launch_anchor_means(units, N, d, sp, B.mu_e, B.mu_s, st, &h->launches));
        CU(launch_anchor_norms(units, d, sp, B.mu_s, B.mu_e, B.inv_s,
                               B.inv_e, nullptr, st, &h->launches));
        CU(mark());
        // d = 64 tiles are too small to pay for the per-tile hand-overs: the FMA form is faster there
        const bool dots_wanted = h->key_pass == NKV_KEY_PASS_TENSOR || (h->key_pass == NKV_KEY_PASS_AUTO && d == 128);
        if (dots_wanted && anchor_dots_supported(kv, dtype, sp))
            CU(launch_anchor_dots(kv, G, sp, B.mu_s, B.mu_e, B.inv_norm,
                                  B.inv_s, B.inv_e, B.a_raw,
                                  B.mm, status, h->sm_count, st, &h->launches));
        else
            CU(launch_stream_b(kv, dtype, G, sp, B.mu_s, B.mu_e,
                               B.inv_norm, B.inv_s, B.inv_e,
                               B.a_raw, B.mm, status, h->sm_count, st,
                               &h->launches));
    } else {
        CU(launch_anchor_sums(kv, dtype, G, sp, B.mu_e, B.inv_norm, st, &h->launches));
        CU(launch_anchor_means(units, N, d, sp, B.mu_e, B.mu_s, st, &h->launches));
        CU(launch_anchor_norms(units, d, sp, B.mu_s, B.mu_e, B.inv_s,
                               B.inv_e, B.mm, st, &h->launches));
        CU(mark());
        CU(launch_scan_scores(kv, dtype, G, sp, B.mu_s, B.mu_e,
                              B.inv_norm, B.inv_s, B.inv_e,
                              B.a_raw, B.mm, st, &h->launches));
    }
    return NKV_OK;
}

// ordered min/max keys -> floats (lo_s, hi_s, lo_e, hi_e, lo_c, hi_c per head)
__global__ void minmax_floats_kernel(int n, const uint32_t* keys, float* out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = ord_float(keys[i]);
}

}  // namespace

extern "C" {

const char* nkv_version(void) { return "nkv 0.1 (sm_100a)"; }

const char* nkv_status_string(int status) {
    switch (status) {
        case NKV_OK: return "ok";
        case NKV_ERR_INVALID_ARG: return "invalid argument";
        case NKV_ERR_UNSUPPORTED: return "unsupported dtype, head_dim, window or layout";
        case NKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case NKV_ERR_CUDA: return "CUDA runtime error";
        case NKV_ERR_TIMEOUT: return "device-side bounded wait ran out";
        case NKV_ERR_DEVICE_CHECK: return "device-side self-check failed";
        default: return "unknown status";
    }
}

int nkv_default_params(nkv_params* p) {
    if (!p) return NKV_ERR_INVALID_ARG;
    p->window = 64;
    p->n_sink = 4;
    p->block_div = 32;
    p->block_min = 128;
    p->block_max = 256;
    p->gate_mode = NKV_GATE_SURPRISE;
    p->top_frac = 0.10;
    p->prior[0] = 0.4;
    p->prior[1] = 0.4;
    p->prior[2] = 0.2;
    p->beta = 3.0;
    p->tau = 0.60;
    p->kappa = 10.0;
    p->safeguard = 0.20;
    return NKV_OK;
}

int64_t nkv_block_size(int64_t N, const nkv_params* p) {
    if (N < 1 || !params_ok(p)) return -1;
    return block_size(N, p);
}
int64_t nkv_num_blocks(int64_t N, const nkv_params* p) {
    if (N < 1 || !params_ok(p)) return -1;
    const int64_t b = block_size(N, p);
    return (N + b - 1) / b;
}
int64_t nkv_keep_per_head(int64_t N, double r) {
    if (N < 1 || !(r >= 0.0 && r < 1.0)) return -1;
    return keep_count(N, r);
}
int64_t nkv_safeguard_count(int64_t N, double r, const nkv_params* p) {
    if (N < 1 || !(r >= 0.0 && r < 1.0) || !params_ok(p)) return -1;
    const int64_t k = keep_count(N, r);
    int64_t s = (int64_t)floor(p->safeguard * (double)k);
    return s > k ? k : s;
}
int64_t nkv_top_count(int64_t N, const nkv_params* p) {
    if (N < 1 || !params_ok(p)) return -1;
    int64_t m = (int64_t)floor(p->top_frac * (double)N);
    return m < 1 ? 1 : m;
}

int nkv_create(nkv_handle** out, int device) {
    if (!out) return NKV_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0, previous = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return NKV_ERR_CUDA;
    CU(cudaGetDevice(&previous));
    CU(cudaSetDevice(device));
    struct Restore {   // the caller's current device is left as it was
        int dev;
        ~Restore() { cudaSetDevice(dev); }
    } restore{previous};
    nkv_handle* h = new (std::nothrow) nkv_handle();
    if (!h) return NKV_ERR_INVALID_ARG;
    memset(h, 0, sizeof(*h));
    h->device = device;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
        delete h;
        return NKV_ERR_CUDA;
    }
    h->sm_count = prop.multiProcessorCount;
    h->l2_bytes = prop.l2CacheSize;
    h->key_pass = NKV_KEY_PASS_AUTO;
    if (configure_scan_kernels() != cudaSuccess || configure_stream_kernels() != cudaSuccess ||
        configure_gram_kernels() != cudaSuccess ||
        configure_dots_kernels() != cudaSuccess || configure_select_kernels() != cudaSuccess) {
        delete h;
        return NKV_ERR_CUDA;
    }
    for (int i = 0; i <= NKV_NUM_STAGES; ++i)
        if (cudaEventCreate(&h->ev[i]) != cudaSuccess) {
            delete h;
            return NKV_ERR_CUDA;
        }
    if (cudaMallocHost(reinterpret_cast<void**>(&h->chunk_status), kMaxHostChunks * 4 * sizeof(int)) != cudaSuccess) {
        delete h;
        return NKV_ERR_CUDA;
    }
    for (int i = 0; i < 2; ++i) {
        if (cudaStreamCreateWithFlags(&h->copy_streams[i], cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->slot_done[i], cudaEventDisableTiming) != cudaSuccess) {
            delete h;
            return NKV_ERR_CUDA;
        }
    }
    *out = h;
    return NKV_OK;
}

int nkv_destroy(nkv_handle* h) {
    if (!h) return NKV_ERR_INVALID_ARG;
    for (int i = 0; i <= NKV_NUM_STAGES; ++i) cudaEventDestroy(h->ev[i]);
    for (int i = 0; i < 2; ++i) {
        cudaStreamDestroy(h->copy_streams[i]);
        cudaEventDestroy(h->slot_done[i]);
    }
    cudaFreeHost(h->chunk_status);
    delete h;
    return NKV_OK;
}

int nkv_workspace_bytes(const nkv_handle* h, int64_t G, int64_t H, int64_t N, int64_t d, int32_t dtype,
                        const nkv_params* params, size_t* out_bytes) {
    (void)dtype;
    if (!h || !out_bytes || G < 1 || H < 1 || N < 1 || d < 1 || !params_ok(params)) return NKV_ERR_INVALID_ARG;
    const int64_t b = block_size(N, params);
    *out_bytes = make_layout(G, G * H, N, d, (N + b - 1) / b).total;
    return NKV_OK;
}

int nkv_anchors(nkv_handle* h, const nkv_tensor* K, const nkv_params* params, float* mu_s, float* mu_e,
                float* inv_norm, float* mu_c_opt, void* ws, size_t ws_bytes, void* stream) {
    if (!h || !mu_s || !mu_e || !inv_norm) return NKV_ERR_INVALID_ARG;
    int rc = check_tensor(K);
    if (rc) return rc;
    ScoreParams sp;
    if ((rc = resolve_params(params, K->N, &sp))) return rc;
    if ((rc = check_ws(ws, ws_bytes, align_up(kStatusWords * sizeof(int))))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const TensorView kv = view_of(K);
    const int units = (int)(K->G * K->H);
    CU(launch_anchor_sums(kv, K->dtype, (int)K->G, sp, mu_e, inv_norm, st, &h->launches));
    CU(launch_anchor_means(units, (int)K->N, (int)K->d, sp, mu_e, mu_s, st, &h->launches));
    if (mu_c_opt) CU(launch_window_means(kv, K->dtype, (int)K->G, sp, inv_norm, mu_c_opt, st, &h->launches));
    return NKV_OK;
}

int nkv_score(nkv_handle* h, const nkv_tensor* K, const float* mu_s, const float* mu_e, const float* inv_norm,
              const nkv_params* params, float* a_raw_opt, float* a_star, float* head_stats_opt, void* ws,
              size_t ws_bytes, void* stream) {
    if (!h || !mu_s || !mu_e || !inv_norm || !a_star) return NKV_ERR_INVALID_ARG;
    int rc = check_tensor(K);
    if (rc) return rc;
    if ((rc = check_units(K->G * K->H))) return rc;
    ScoreParams sp;
    if ((rc = resolve_params(params, K->N, &sp))) return rc;
    const int units = (int)(K->G * K->H);
    const Layout L = make_layout(K->G, units, K->N, K->d, sp.nblocks);
    if ((rc = check_ws(ws, ws_bytes, L.total))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const TensorView kv = view_of(K);
    float* a_raw = a_raw_opt ? a_raw_opt : at<float>(ws, L.a_raw);
    CU(cudaMemsetAsync(at<int>(ws, L.status), 0, kStatusWords * sizeof(int), st));
    CU(launch_anchor_norms(units, (int)K->d, sp, mu_s, mu_e, at<float>(ws, L.inv_s), at<float>(ws, L.inv_e),
                           at<uint32_t>(ws, L.mm), st, &h->launches));
    CU(launch_scan_scores(kv, K->dtype, (int)K->G, sp, mu_s, mu_e, inv_norm, at<float>(ws, L.inv_s),
                          at<float>(ws, L.inv_e), a_raw, at<uint32_t>(ws, L.mm), st, &h->launches));
    CU(launch_head_scores(units, (int)K->N, sp, a_raw, at<uint32_t>(ws, L.mm), a_star, head_stats_opt,
                          at<float>(ws, L.hstat), at<int>(ws, L.status), st, &h->launches));
    return NKV_OK;
}

int nkv_budget(nkv_handle* h, const float* a_star, int64_t G, int64_t H, int64_t N, double r,
               const nkv_params* params, int32_t* budgets, float* thresholds_opt, void* ws, size_t ws_bytes,
               void* stream) {
    if (!h || !a_star || !budgets || G < 1 || H < 1 || N < 1 || !params_ok(params)) return NKV_ERR_INVALID_ARG;
    if (!(r >= 0.0 && r < 1.0)) return NKV_ERR_INVALID_ARG;
    if (H > 64 || N > (int64_t)1 << 24 || H * N > (int64_t)1 << 30) return NKV_ERR_UNSUPPORTED;
    const int64_t k = keep_count(N, r);
    if (k < 1 || k > N) return NKV_ERR_INVALID_ARG;
    const int64_t n_safe = nkv_safeguard_count(N, r, params);
    const size_t thr_off = align_up(kStatusWords * sizeof(int));
    int rc = check_ws(ws, ws_bytes, thr_off + align_up((size_t)G * H * 8));
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaMemsetAsync(ws, 0, kStatusWords * sizeof(int), st));
    const size_t scr_off = thr_off + align_up((size_t)G * H * 8);
    void* scratch = ws_bytes >= scr_off + budget_scratch_bytes(G, H) ? at<unsigned char>(ws, scr_off) : nullptr;
    CU(launch_budget((int)G, (int)H, (int)N, (int)k, (int)n_safe, a_star, budgets, at<uint32_t>(ws, thr_off),
                     at<int>(ws, 0), scratch, st, &h->launches));
    if (thresholds_opt)
        CU(launch_threshold_scores((int)(G * H), at<uint32_t>(ws, thr_off), thresholds_opt, st, &h->launches));
    return NKV_OK;
}

int nkv_select(nkv_handle* h, const float* a_star, const int32_t* budgets, int64_t G, int64_t H, int64_t N,
               int64_t idx_capacity, int32_t* idx, int32_t* head_offsets, int32_t* ranks_opt, void* ws,
               size_t ws_bytes, void* stream) {
    if (!h || !a_star || !budgets || !idx || !head_offsets || G < 1 || H < 1 || N < 1 || idx_capacity < 1)
        return NKV_ERR_INVALID_ARG;
    if (N > (int64_t)1 << 24 || G * H > (int64_t)1 << 24) return NKV_ERR_UNSUPPORTED;
    int rc = check_ws(ws, ws_bytes, align_up(kStatusWords * sizeof(int)));
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaMemsetAsync(ws, 0, kStatusWords * sizeof(int), st));
    CU(launch_select((int)G, (int)H, (int)N, idx_capacity, a_star, budgets, nullptr, idx, head_offsets,
                     at<int>(ws, 0), st, &h->launches));
    if (ranks_opt) {
        if (G * H > 65535) return NKV_ERR_UNSUPPORTED;
        CU(launch_ranks((int)(G * H), (int)N, a_star, ranks_opt, st, &h->launches));
    }
    return NKV_OK;
}

int nkv_compact(nkv_handle* h, const nkv_tensor* K, const nkv_tensor* V, const int32_t* idx,
                const int32_t* head_offsets, int64_t idx_capacity, void* K_out, void* V_out, int32_t mode, void* ws,
                size_t ws_bytes, void* stream) {
    (void)ws;
    (void)ws_bytes;
    if (!h || !idx || !head_offsets || idx_capacity < 1) return NKV_ERR_INVALID_ARG;
    int rc = check_tensor(K);
    if (rc) return rc;
    if ((rc = check_tensor(V))) return rc;
    if (V->G != K->G || V->H != K->H || V->N != K->N) return NKV_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int kb = K->dtype == NKV_F32 ? 4 : 2, vb = V->dtype == NKV_F32 ? 4 : 2;
    if (mode == NKV_OUT_OF_PLACE) {
        if (!K_out || !V_out || ((uintptr_t)K_out) % 16 || ((uintptr_t)V_out) % 16) return NKV_ERR_INVALID_ARG;
        CU(launch_gather(view_of(K), kb, view_of(V), vb, (int)K->G, idx, head_offsets, idx_capacity, K_out, V_out,
                         h->sm_count, st, &h->launches));
    } else if (mode == NKV_IN_PLACE) {
        if (K_out || V_out) return NKV_ERR_INVALID_ARG;
        CU(launch_gather_in_place(view_of(K), kb, view_of(V), vb, (int)K->G, idx, head_offsets, idx_capacity, st,
                                  &h->launches));
    } else {
        return NKV_ERR_INVALID_ARG;
    }
    return NKV_OK;
}

int nkv_compress(nkv_handle* h, const nkv_tensor* K, const nkv_tensor* V, double r, const nkv_params* params,
                 void* K_out, void* V_out, int32_t* idx, int32_t* head_offsets, int32_t* budgets,
                 float* a_star_opt, void* ws, size_t ws_bytes, void* stream) {
    if (!h || !K_out || !V_out || !idx || !head_offsets || !budgets) return NKV_ERR_INVALID_ARG;
    int rc = check_tensor(K);
    if (rc) return rc;
    if ((rc = check_tensor(V))) return rc;
    if (V->G != K->G || V->H != K->H || V->N != K->N) return NKV_ERR_INVALID_ARG;
    if (!(r >= 0.0 && r < 1.0)) return NKV_ERR_INVALID_ARG;
    if (K->H > 64 || K->H * K->N > (int64_t)1 << 30) return NKV_ERR_UNSUPPORTED;
    if ((rc = check_units(K->G * K->H))) return rc;
    if (((uintptr_t)K_out) % 16 || ((uintptr_t)V_out) % 16) return NKV_ERR_INVALID_ARG;
    ScoreParams sp;
    if ((rc = resolve_params(params, K->N, &sp))) return rc;
    const int64_t keep = keep_count(K->N, r);
    if (keep < 1 || keep > K->N) return NKV_ERR_INVALID_ARG;
    const int64_t n_safe = nkv_safeguard_count(K->N, r, params);
    const int G = (int)K->G, H = (int)K->H, N = (int)K->N, d = (int)K->d;
    const int units = G * H;
    const Layout L = make_layout(G, units, N, d, sp.nblocks);
    if ((rc = check_ws(ws, ws_bytes, L.total))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const TensorView kv = view_of(K), vv = view_of(V);
    const int kb = K->dtype == NKV_F32 ? 4 : 2, vb = V->dtype == NKV_F32 ? 4 : 2;
    float* a_star = a_star_opt ? a_star_opt : at<float>(ws, L.a_star);
    int* status = at<int>(ws, L.status);
    const bool timing = h->timing != 0;
    int stage = 0;
    auto mark = [&]() -> cudaError_t {
        if (!timing) return cudaSuccess;
        return cudaEventRecord(h->ev[stage++], st);
    };

    CU(cudaMemsetAsync(status, 0, kStatusWords * sizeof(int), st));
    CU(mark());
    // One run of groups: the key scan on `ks`, everything after it on `ss`.
    auto run = [&](int g0, int gc, cudaStream_t ks, cudaStream_t ss, cudaEvent_t scanned) -> int {
        const Bufs B = bufs_at(ws, L, g0, H, N, d, sp.nblocks);
        TensorView kc = kv, vc = vv;
        kc.ptr = static_cast<const unsigned char*>(kv.ptr) + (size_t)g0 * kv.stride_g * kb;
        vc.ptr = static_cast<const unsigned char*>(vv.ptr) + (size_t)g0 * vv.stride_g * vb;
        float* as = a_star + (size_t)g0 * H * N;
        int32_t* bud = budgets + (size_t)g0 * H;
        int32_t* ix = idx + (size_t)g0 * H * keep;
        int32_t* ho = head_offsets + (size_t)g0 * (H + 1);
        int rc2 = key_scan(h, kc, K->dtype, gc, sp, B, status, ks, mark);
        if (rc2) return rc2;
        CU(mark());
        if (ss != ks) {
            CU(cudaEventRecord(scanned, ks));
            CU(cudaStreamWaitEvent(ss, scanned, 0));
        }
        CU(launch_head_scores(gc * H, N, sp, B.a_raw, B.mm, as, nullptr, B.hstat, status, ss, &h->launches));
        CU(mark());
        CU(launch_budget(gc, H, N, (int)keep, (int)n_safe, as, bud, B.thr, status, B.bscr, ss, &h->launches));
        CU(mark());
        CU(launch_select(gc, H, N, (int64_t)H * keep, as, bud, B.thr, ix, ho, status, ss, &h->launches));
        CU(mark());
        CU(launch_gather(kc, kb, vc, vb, gc, ix, ho, (int64_t)H * keep,
                         static_cast<unsigned char*>(K_out) + (size_t)g0 * H * keep * kv.d * kb,
                         static_cast<unsigned char*>(V_out) + (size_t)g0 * H * keep * vv.d * vb, h->sm_count, ss,
                         &h->launches));
        CU(mark());
        return NKV_OK;
    };
    // Running a call as two halves on two streams (the score side of one half beside the second key pass and
    // the compaction of the other) measured no faster: the first key pass leaves no registers for a second
    // kernel on its SMs, and beside the second pass the score kernels get a quarter of their CTAs.
    if ((rc = run(0, G, st, st, nullptr))) return rc;
    if (timing) h->timing_valid = 1;
    return NKV_OK;
}

int nkv_host_staging_bytes(const nkv_handle* h, int64_t H, int64_t N, int64_t d, int32_t dtype, double r,
                           const nkv_params* params, int64_t groups_per_chunk, size_t* out_bytes) {
    if (!h || !out_bytes || H < 1 || N < 1 || d < 1 || groups_per_chunk < 1 || !params_ok(params))
        return NKV_ERR_INVALID_ARG;
    if (!(r >= 0.0 && r < 1.0)) return NKV_ERR_INVALID_ARG;
    const int64_t keep = keep_count(N, r);
    if (keep < 1) return NKV_ERR_INVALID_ARG;
    const size_t eb = dtype == NKV_F32 ? 4 : 2;
    const int64_t b = block_size(N, params);
    const size_t c = (size_t)groups_per_chunk;
    size_t slot = 0;
    slot += 2 * align_up(c * H * N * d * eb);        // K, V
    slot += 2 * align_up(c * H * keep * d * eb);     // K_out, V_out
    slot += align_up(c * H * keep * 4);              // idx
    slot += align_up(c * (H + 1) * 4);               // head_offsets
    slot += align_up(c * H * 4);                     // budgets
    slot += make_layout(c, c * H, N, d, (N + b - 1) / b).total;
    *out_bytes = 2 * slot;
    return NKV_OK;
}

int nkv_compress_host(nkv_handle* h, const nkv_tensor* Kh, const nkv_tensor* Vh, double r, const nkv_params* params,
                      void* K_out_host, void* V_out_host, int32_t* idx_host, int32_t* head_offsets_host,
                      int32_t* budgets_host, int64_t groups_per_chunk, void* dev, size_t dev_bytes) {
    if (!h || !K_out_host || !V_out_host || !idx_host || !head_offsets_host || !budgets_host) return NKV_ERR_INVALID_ARG;
    int rc = check_tensor(Kh);
    if (rc) return rc;
    if ((rc = check_tensor(Vh))) return rc;
    if (Vh->G != Kh->G || Vh->H != Kh->H || Vh->N != Kh->N || Vh->d != Kh->d || Vh->dtype != Kh->dtype)
        return NKV_ERR_INVALID_ARG;
    // the host path copies whole groups: require densely packed groups
    if (Kh->stride_h != Kh->N * Kh->d || Kh->stride_g != Kh->H * Kh->N * Kh->d || Vh->stride_h != Kh->stride_h ||
        Vh->stride_g != Kh->stride_g)
        return NKV_ERR_UNSUPPORTED;
    size_t need = 0;
    if ((rc = nkv_host_staging_bytes(h, Kh->H, Kh->N, Kh->d, Kh->dtype, r, params, groups_per_chunk, &need))) return rc;
    if ((rc = check_ws(dev, dev_bytes, need))) return rc;
    const int64_t G = Kh->G, H = Kh->H, N = Kh->N, d = Kh->d;
    const int64_t keep = keep_count(N, r);
    const size_t eb = Kh->dtype == NKV_F32 ? 4 : 2;
    const int64_t b = block_size(N, params);
    const size_t c = (size_t)groups_per_chunk;
    const size_t slot_bytes = need / 2;
    const size_t kv_bytes = align_up(c * H * N * d * eb), out_bytes = align_up(c * H * keep * d * eb);
    const size_t idx_bytes = align_up(c * H * keep * 4), off_bytes = align_up(c * (H + 1) * 4),
                 bud_bytes = align_up(c * H * 4);
    const size_t ws_need = make_layout(c, c * H, N, d, (N + b - 1) / b).total;

    int result = NKV_OK;
    int chunk_index = 0;
    for (int64_t g0 = 0; g0 < G && result == NKV_OK; g0 += groups_per_chunk, ++chunk_index) {
        const int slot = chunk_index & 1;
        cudaStream_t st = h->copy_streams[slot];
        const int64_t gc = (G - g0 < groups_per_chunk) ? (G - g0) : groups_per_chunk;
        unsigned char* base = reinterpret_cast<unsigned char*>(dev) + slot * slot_bytes;
        unsigned char* dK = base;
        unsigned char* dV = dK + kv_bytes;
        unsigned char* dKo = dV + kv_bytes;
        unsigned char* dVo = dKo + out_bytes;
        int32_t* dIdx = reinterpret_cast<int32_t*>(dVo + out_bytes);
        int32_t* dOff = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(dIdx) + idx_bytes);
        int32_t* dBud = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(dOff) + off_bytes);
        void* dWs = reinterpret_cast<unsigned char*>(dBud) + bud_bytes;
        const size_t grp_in = (size_t)H * N * d * eb, grp_out = (size_t)H * keep * d * eb;
        // the slot's previous chunk finished all its copies before this stream reaches here (same stream)
        if (cudaMemcpyAsync(dK, (const unsigned char*)Kh->ptr + g0 * grp_in, gc * grp_in, cudaMemcpyHostToDevice, st) !=
                cudaSuccess ||
            cudaMemcpyAsync(dV, (const unsigned char*)Vh->ptr + g0 * grp_in, gc * grp_in, cudaMemcpyHostToDevice, st) !=
                cudaSuccess) {
            result = NKV_ERR_CUDA;
            break;
        }
        nkv_tensor dk = *Kh, dv = *Vh;
        dk.ptr = dK;
        dv.ptr = dV;
        dk.G = dv.G = gc;
        rc = nkv_compress(h, &dk, &dv, r, params, dKo, dVo, dIdx, dOff, dBud, nullptr, dWs, ws_need, st);
        if (rc) {
            result = rc;
            break;
        }
        if (h->inject_status && chunk_index == h->inject_chunk &&
            cudaMemcpyAsync(dWs, &h->inject_status, sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess) {
            result = NKV_ERR_CUDA;
            break;
        }
        if (cudaMemcpyAsync((unsigned char*)K_out_host + g0 * grp_out, dKo, gc * grp_out, cudaMemcpyDeviceToHost, st) !=
                cudaSuccess ||
            cudaMemcpyAsync((unsigned char*)V_out_host + g0 * grp_out, dVo, gc * grp_out, cudaMemcpyDeviceToHost, st) !=
                cudaSuccess ||
            cudaMemcpyAsync(idx_host + g0 * H * keep, dIdx, gc * H * keep * 4, cudaMemcpyDeviceToHost, st) !=
                cudaSuccess ||
            cudaMemcpyAsync(head_offsets_host + g0 * (H + 1), dOff, gc * (H + 1) * 4, cudaMemcpyDeviceToHost, st) !=
                cudaSuccess ||
            cudaMemcpyAsync(budgets_host + g0 * H, dBud, gc * H * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            (chunk_index < kMaxHostChunks &&
             cudaMemcpyAsync(h->chunk_status + chunk_index * 4, dWs, 16, cudaMemcpyDeviceToHost, st) != cudaSuccess)) {
            result = NKV_ERR_CUDA;
            break;
        }
    }
    for (int i = 0; i < 2; ++i)
        if (cudaStreamSynchronize(h->copy_streams[i]) != cudaSuccess) result = result ? result : NKV_ERR_CUDA;
    // every chunk's device status words were copied out before its slot was reused: report the first failure
    for (int c2 = 0; c2 < chunk_index && c2 < kMaxHostChunks && result == NKV_OK; ++c2)
        if (h->chunk_status[c2 * 4 + kStatusCode] != 0)
            result = h->chunk_status[c2 * 4 + kStatusCode] == NKV_ERR_TIMEOUT ? NKV_ERR_TIMEOUT : NKV_ERR_DEVICE_CHECK;
    return result;
}

int nkv_last_device_status(nkv_handle* h, const void* ws, void* stream) {
    if (!h || !ws) return NKV_ERR_INVALID_ARG;
    int words[4] = {0, 0, 0, 0};
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return NKV_ERR_CUDA;
    if (cudaMemcpy(words, ws, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess) return NKV_ERR_CUDA;
    if (words[kStatusCode] == NKV_ERR_TIMEOUT) return NKV_ERR_TIMEOUT;
    if (words[kStatusCode] != 0) return NKV_ERR_DEVICE_CHECK;
    return NKV_OK;
}

int nkv_set_timing(nkv_handle* h, int enable) {
    if (!h) return NKV_ERR_INVALID_ARG;
    h->timing = enable ? 1 : 0;
    h->timing_valid = 0;
    return NKV_OK;
}

int nkv_get_stage_ms(nkv_handle* h, float* ms_out) {
    if (!h || !ms_out || !h->timing_valid) return NKV_ERR_INVALID_ARG;
    if (cudaEventSynchronize(h->ev[NKV_NUM_STAGES]) != cudaSuccess) return NKV_ERR_CUDA;
    for (int i = 0; i < NKV_NUM_STAGES; ++i)
        if (cudaEventElapsedTime(&ms_out[i], h->ev[i], h->ev[i + 1]) != cudaSuccess) return NKV_ERR_CUDA;
    return NKV_OK;
}

int64_t nkv_launch_count(const nkv_handle* h) { return h ? h->launches : -1; }

int nkv_key_scan(nkv_handle* h, const nkv_tensor* K, const nkv_params* params, float* inv_norm, float* mu_s,
                 float* mu_e, float* a_raw, float* minmax, void* ws, size_t ws_bytes, void* stream) {
    if (!h || !inv_norm || !mu_s || !mu_e || !a_raw || !minmax) return NKV_ERR_INVALID_ARG;
    int rc = check_tensor(K);
    if (rc) return rc;
    if ((rc = check_units(K->G * K->H))) return rc;
    ScoreParams sp;
    if ((rc = resolve_params(params, K->N, &sp))) return rc;
    const int G = (int)K->G, N = (int)K->N, d = (int)K->d, units = (int)(K->G * K->H);
    const Layout L = make_layout(G, units, N, d, sp.nblocks);
    if ((rc = check_ws(ws, ws_bytes, L.total))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaMemsetAsync(at<int>(ws, L.status), 0, kStatusWords * sizeof(int), st));
    auto no_mark = []() -> cudaError_t { return cudaSuccess; };
    if ((rc = key_scan(h, view_of(K), K->dtype, G, sp, bufs_at(ws, L, 0, K->H, N, d, sp.nblocks), at<int>(ws, L.status), st,
                       no_mark)))
        return rc;
    CU(cudaMemcpyAsync(mu_s, at<float>(ws, L.mu_s), (size_t)units * d * 4, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(mu_e, at<float>(ws, L.mu_e), (size_t)units * sp.nblocks * d * 4, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(inv_norm, at<float>(ws, L.inv_norm), (size_t)units * N * 4, cudaMemcpyDeviceToDevice, st));
    CU(cudaMemcpyAsync(a_raw, at<float>(ws, L.a_raw), (size_t)units * 3 * N * 4, cudaMemcpyDeviceToDevice, st));
    minmax_floats_kernel<<<(units * 6 + 255) / 256, 256, 0, st>>>(units * 6, at<uint32_t>(ws, L.mm), minmax);
    ++h->launches;
    CU(cudaGetLastError());
    return NKV_OK;
}

int nkv_debug_set(nkv_handle* h, int what, int64_t value) {
    if (!h) return NKV_ERR_INVALID_ARG;
    switch (what) {
        case NKV_DEBUG_INJECT_HOST_STATUS:   // value = chunk * 16 + status code (0 clears)
            if (value < 0) return NKV_ERR_INVALID_ARG;
            h->inject_status = (int)(value & 15);
            h->inject_chunk = (int)(value >> 4);
            return NKV_OK;
        default:
            return NKV_ERR_INVALID_ARG;
    }
}

int nkv_debug_wait_probe(nkv_handle* h, int64_t polls, void* ws, size_t ws_bytes, void* stream) {
    if (!h || polls < 1 || polls > (1 << 16)) return NKV_ERR_INVALID_ARG;
    int rc = check_ws(ws, ws_bytes, align_up(kStatusWords * sizeof(int)));
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaMemsetAsync(ws, 0, kStatusWords * sizeof(int), st));
    CU(launch_wait_probe(static_cast<int*>(ws), (uint32_t)polls, st, &h->launches));
    return NKV_OK;
}

int nkv_set_key_passes(nkv_handle* h, int mode) {
    if (!h || mode < NKV_KEY_PASS_AUTO || mode > NKV_KEY_PASS_TENSOR) return NKV_ERR_INVALID_ARG;
    h->key_pass = mode;
    return NKV_OK;
}

}  // extern "C"
