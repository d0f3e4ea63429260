/*
 * nkv -- NestedKV key-value cache compression on one B200 (sm_100a), C ABI.
 *
 * The library implements the per-(layer, KV-head) compression operator
 * C_phi(K, V; B_h) of the paper (Section 2.1) together with the head-wise
 * budget competition that couples the KV heads of one layer (Section 2.6):
 *
 *   anchors  (Section 2.2)  stable mean, episodic block means, current
 *                           sliding-window mean of the L2-normalised keys
 *   score    (Sections 2.3-2.4) three cosine anomalies per token, per-head
 *                           min-max, head-adaptive softmax blend, surprise-
 *                           gated routing, sink pinning -> a_star
 *   budget   (Section 2.6, Appendix A) per-head safeguard + cross-head
 *                           competition -> B_h with sum_h B_h = H*floor((1-r)N)
 *   select   (Section 2.5)  TopB_h(a_star) per head -> ascending positions
 *   compact  (Section 2.1)  (K_S, V_S): retained rows copied verbatim
 *
 * Conventions
 *   - A cache is [G, H, N, d]: G = sequences x layers "groups" (the H heads of a
 *     group compete for one layer budget), N tokens, d channels, positions
 *     0-based.  All pointers in nkv_tensor and all array arguments are DEVICE
 *     pointers unless an argument says "host".  Strides are in elements; d is
 *     contiguous, stride_n must equal d, every row start is 16-byte aligned.
 *     d is 64 or 128, dtype bf16, fp16 or fp32 (fp16 keys run the FMA form of the key passes), 2 <= window <= 64 (with a window of one key the
 *     current anchor is the key itself and that scale carries no information).
 *   - Every buffer is caller-owned.  No entry point except nkv_create,
 *     nkv_destroy and nkv_compress_host allocates, frees or synchronises; work
 *     is enqueued on the given stream (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and the call returns.
 *   - `ws` is caller-provided device scratch of at least nkv_workspace_bytes()
 *     bytes, 256-byte aligned.  Its first bytes hold a device status word that
 *     kernels set when a bounded wait runs out or a self-check fails; read it
 *     with nkv_last_device_status after synchronising the stream.
 *   - Every function returns an nkv_status.  Argument errors are detected on
 *     the host before anything is launched; nothing throws or aborts.
 *   - Keys are assumed finite.  Non-finite keys are not detected.
 *   - r is the fraction of entries REMOVED (Section 3.1), 0 <= r < 1, and
 *     k = floor((1-r)*N) >= 1 must hold (evaluated in double).
 */
#ifndef NKV_H
#define NKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define NKV_API __attribute__((visibility("default")))
#else
#define NKV_API
#endif

typedef enum nkv_status {
    NKV_OK = 0,
    NKV_ERR_INVALID_ARG = 1,  /* null pointer, bad shape/stride/alignment, r or params out of range */
    NKV_ERR_UNSUPPORTED = 2,  /* dtype / head_dim / window outside the supported set */
    NKV_ERR_WORKSPACE = 3,    /* workspace missing, misaligned or too small */
    NKV_ERR_CUDA = 4,         /* a CUDA runtime call failed (launch or copy) */
    NKV_ERR_TIMEOUT = 5,      /* device status: a bounded device-side wait ran out */
    NKV_ERR_DEVICE_CHECK = 6  /* device status: a kernel self-check failed */
} nkv_status;

typedef enum nkv_dtype { NKV_BF16 = 0, NKV_F32 = 1, NKV_F16 = 2 } nkv_dtype;

/* Routing rule (Section 2.4); AVERAGE and MAX are the router-ablation variants. */
typedef enum nkv_gate_mode { NKV_GATE_SURPRISE = 0, NKV_GATE_AVERAGE = 1, NKV_GATE_MAX = 2 } nkv_gate_mode;

typedef enum nkv_compact_mode {
    NKV_OUT_OF_PLACE = 0, /* packed [G, H*k, d] output, heads concatenated per group */
    NKV_IN_PLACE = 1      /* each head's retained rows moved to the front of its own [N, d] slab */
} nkv_compact_mode;

/* Constants of the method (Appendix A, "Hyperparameters"). */
typedef struct nkv_params {
    int32_t window;     /* W of the current memory, 64 */
    int32_t n_sink;     /* pinned leading positions, 4 */
    int32_t block_div;  /* b = clip(floor(N / block_div), block_min, block_max): 32, 128, 256 */
    int32_t block_min;
    int32_t block_max;
    int32_t gate_mode;  /* nkv_gate_mode */
    double top_frac;    /* p of the reliability gap, 0.10 */
    double prior[3];    /* (w_s^0, w_e^0, w_c^0) = (0.4, 0.4, 0.2); entries >= 0, not all 0; a zero
                           switches its scale off (single-anchor and no-current ablations) */
    double beta;        /* 3.0 */
    double tau;         /* 0.60 */
    double kappa;       /* 10.0 */
    double safeguard;   /* alpha_s = 0.20, in [0, 1] */
} nkv_params;

/* A [G, H, N, d] device tensor. */
typedef struct nkv_tensor {
    void* ptr;
    int32_t dtype; /* nkv_dtype */
    int32_t reserved;
    int64_t G, H, N, d;
    int64_t stride_g, stride_h, stride_n; /* elements */
} nkv_tensor;

typedef struct nkv_handle nkv_handle;

/* Number of floats per head in the optional head_stats output of nkv_score:
 * lo_s,lo_e,lo_c, hi_s,hi_e,hi_c, Delta_s,Delta_e,Delta_c, w_s,w_e,w_c,
 * min s, max s, mean of the min-max-normalised s, m (top/bottom count). */
#define NKV_HEAD_STATS 16

/* Stages whose device time nkv_compress records when timing is enabled. */
#define NKV_STAGE_ANCHORS 0
#define NKV_STAGE_SCORE 1
#define NKV_STAGE_HEAD 2
#define NKV_STAGE_BUDGET 3
#define NKV_STAGE_SELECT 4
#define NKV_STAGE_COMPACT 5
#define NKV_NUM_STAGES 6

NKV_API const char* nkv_version(void);
NKV_API const char* nkv_status_string(int status);

/* Fills the defaults of Appendix A (host pointer). */
NKV_API int nkv_default_params(nkv_params* params);

/* Derived sizes, on the host, exactly as the kernels use them.
 * block size b (Section 2.2), number of blocks ceil(N/b), per-head nominal
 * budget k = floor((1-r)N), safeguard floor(safeguard*k), top/bottom count
 * m = max(1, floor(top_frac*N)).  Each returns -1 on invalid arguments. */
NKV_API int64_t nkv_block_size(int64_t N, const nkv_params* params);
NKV_API int64_t nkv_num_blocks(int64_t N, const nkv_params* params);
NKV_API int64_t nkv_keep_per_head(int64_t N, double r);
NKV_API int64_t nkv_safeguard_count(int64_t N, double r, const nkv_params* params);
NKV_API int64_t nkv_top_count(int64_t N, const nkv_params* params);

/* Creates a handle bound to CUDA device `device` (caches SM count, L2 size and
 * raises the kernels' dynamic shared-memory limits).  Allocates host memory
 * and CUDA events only.  `*out` is NULL on failure. */
NKV_API int nkv_create(nkv_handle** out, int device);
NKV_API int nkv_destroy(nkv_handle* h);

/* Bytes of device scratch that any entry point below needs for a cache of this
 * shape (an upper bound valid for every r and every stage).  `out_bytes`: host. */
NKV_API int nkv_workspace_bytes(const nkv_handle* h, int64_t G, int64_t H, int64_t N, int64_t d, int32_t dtype,
                        const nkv_params* params, size_t* out_bytes);

/*
 * Section 2.1 (key normalisation) and Section 2.2 (continuum memory state).
 *   K         keys [G,H,N,d]
 *   mu_s      out f32 [G,H,d]      stable mean of the normalised keys
 *   mu_e      out f32 [G,H,nb,d]   episodic block means, nb = nkv_num_blocks(N)
 *                                   (the last block averages its actual members)
 *   inv_norm  out f32 [G,H,N]      1 / max(||k_i||, 1e-12)
 *   mu_c_opt  out f32 [G,H,N,d] or NULL: the current sliding-window mean of every
 *             token (window of min(i+1, W) keys ending at i).  For inspection
 *             and tests only; the scoring kernel never materialises it.
 */
NKV_API int nkv_anchors(nkv_handle* h, const nkv_tensor* K, const nkv_params* params, float* mu_s, float* mu_e,
                float* inv_norm, float* mu_c_opt, void* ws, size_t ws_bytes, void* stream);

/*
 * Sections 2.3-2.4: per-scale anomalies a_k(i) = -cos(k_hat_i, mu_k), per-head
 * min-max, reliability gaps over the top/bottom p, softmax weights, surprise,
 * gate, routed score; then sink pinning (+inf on the first n_sink positions).
 *   mu_s, mu_e, inv_norm   as produced by nkv_anchors
 *   a_raw_opt   out f32 [G,H,3,N] or NULL: a_s, a_e, a_c before normalisation
 *   a_star      out f32 [G,H,N]
 *   head_stats_opt out f32 [G,H,NKV_HEAD_STATS] or NULL
 */
NKV_API int nkv_score(nkv_handle* h, const nkv_tensor* K, const float* mu_s, const float* mu_e,
              const float* inv_norm, const nkv_params* params, float* a_raw_opt, float* a_star,
              float* head_stats_opt, void* ws, size_t ws_bytes, void* stream);

/*
 * Section 2.6 with Appendix A's safeguard: every head first keeps its
 * floor(safeguard*k) best tokens, the remaining H*k - H*n_safe slots go to the
 * globally largest remaining (head, token) pairs under the total order
 * (a_star descending, head ascending, position ascending).
 *   a_star   f32 [G,H,N] (sinks already +inf)
 *   budgets  out i32 [G,H], sum over H = H*k
 *   thresholds_opt  out f32 [G,H] or NULL: the head's selection threshold: the head retains every token that
 *            scores above it and, in position order, as many of the tokens that score exactly it as its
 *            budget still allows (+inf while the sinks alone fill the head's budget)
 *   ws       at least 256 + 8*G*H bytes (rounded up to 256); with 8192*G*H + 42000*G bytes more, large calls
 *            spread the cross-head competition of a group over many thread blocks (same result)
 */
NKV_API int nkv_budget(nkv_handle* h, const float* a_star, int64_t G, int64_t H, int64_t N, double r,
               const nkv_params* params, int32_t* budgets, float* thresholds_opt, void* ws, size_t ws_bytes,
               void* stream);

/*
 * Section 2.5: TopB_h(a_star) per head under (a_star descending, position
 * ascending); positions are written in ascending order.
 *   budgets       i32 [G,H] with 0 <= B_h <= N and sum over H <= idx_capacity
 *   idx           out i32 [G, idx_capacity]: head h of group g occupies
 *                 idx[g, head_offsets[g,h] .. head_offsets[g,h+1])
 *   head_offsets  out i32 [G,H+1] (exclusive prefix sums of budgets)
 *   ranks_opt     out i32 [G,H,N] or NULL: place of every token in its head's
 *                 order (0 = best).  Diagnostic, quadratic time, small N only.
 */
NKV_API int nkv_select(nkv_handle* h, const float* a_star, const int32_t* budgets, int64_t G, int64_t H, int64_t N,
               int64_t idx_capacity, int32_t* idx, int32_t* head_offsets, int32_t* ranks_opt, void* ws,
               size_t ws_bytes, void* stream);

/*
 * Section 2.1: M^B = (K_S, V_S).  Rows are copied byte for byte.
 *   OUT_OF_PLACE: K_out/V_out are [G, idx_capacity, d] / [G, idx_capacity, d_v]
 *                 in the dtype of K / V; row j of group g is the row idx[g,j].
 *   IN_PLACE:     K_out/V_out must be NULL; row idx[g, off+j] of head h moves to
 *                 row j of the same head; rows >= B_h are left unspecified.
 * V may have a different d (64 or 128) and dtype than K, same G, H, N.
 */
NKV_API int nkv_compact(nkv_handle* h, const nkv_tensor* K, const nkv_tensor* V, const int32_t* idx,
                const int32_t* head_offsets, int64_t idx_capacity, void* K_out, void* V_out, int32_t mode,
                void* ws, size_t ws_bytes, void* stream);

/*
 * The whole path (all five stages above) in one call, the timed entry point.
 * Output layout as in nkv_select / nkv_compact with idx_capacity = H*k,
 * k = nkv_keep_per_head(N, r); out-of-place compaction.
 *   K_out, V_out  out [G, H*k, d]      idx out i32 [G, H*k]
 *   head_offsets  out i32 [G, H+1]     budgets out i32 [G, H]
 *   a_star_opt    out f32 [G,H,N] or NULL (a copy of the final scores)
 */
NKV_API int nkv_compress(nkv_handle* h, const nkv_tensor* K, const nkv_tensor* V, double r, const nkv_params* params,
                 void* K_out, void* V_out, int32_t* idx, int32_t* head_offsets, int32_t* budgets,
                 float* a_star_opt, void* ws, size_t ws_bytes, void* stream);

/*
 * The same path for a cache that lives in HOST memory (pinned memory makes the
 * copies asynchronous).  K, V are described by nkv_tensor with HOST pointers;
 * K_out, V_out, idx, head_offsets, budgets are HOST buffers with the layout of
 * nkv_compress.  The call stages `groups_per_chunk` groups at a time through
 * the caller-provided device staging area `dev` (at least
 * nkv_host_staging_bytes() bytes, 256-byte aligned), overlapping the copies of
 * one chunk with the kernels of the previous one on two internal streams, and
 * returns after everything has arrived on the host (it synchronises).
 */
NKV_API int nkv_host_staging_bytes(const nkv_handle* h, int64_t H, int64_t N, int64_t d, int32_t dtype, double r,
                           const nkv_params* params, int64_t groups_per_chunk, size_t* out_bytes);
NKV_API int nkv_compress_host(nkv_handle* h, const nkv_tensor* K_host, const nkv_tensor* V_host, double r,
                      const nkv_params* params, void* K_out_host, void* V_out_host, int32_t* idx_host,
                      int32_t* head_offsets_host, int32_t* budgets_host, int64_t groups_per_chunk, void* dev,
                      size_t dev_bytes);

/* Reads the device status word of `ws` (synchronises `stream` first).
 * Returns NKV_OK, NKV_ERR_TIMEOUT, NKV_ERR_DEVICE_CHECK or NKV_ERR_CUDA. */
NKV_API int nkv_last_device_status(nkv_handle* h, const void* ws, void* stream);

/* Per-stage device timing of nkv_compress (CUDA events on the call's stream).
 * When enabled, every nkv_compress call records events around each stage;
 * nkv_get_stage_ms synchronises on them and returns the milliseconds of the
 * most recent call (host array of NKV_NUM_STAGES floats). */
NKV_API int nkv_set_timing(nkv_handle* h, int enable);
NKV_API int nkv_get_stage_ms(nkv_handle* h, float* ms_out);

/* Number of kernels this handle has launched since creation. */
NKV_API int64_t nkv_launch_count(const nkv_handle* h);

/*
 * Choice of the kernels that make the two passes over the keys of nkv_compress (Sections 2.1-2.3).  The
 * first pass yields 1/||k||, the block sums of normalised keys and the current-memory anomaly a_c; the
 * second, which needs the anchors of the whole head, the anomalies a_s and a_e.
 *   NKV_KEY_PASS_FMA     both passes with fp32 FMAs on staged key tiles (any supported dtype and d).
 *   NKV_KEY_PASS_TENSOR  (bf16 keys) forms on the tensor cores what is a contraction: in the first pass
 *       (d = 128, W = 64, one CTA per head) k_hat_i . S_i and ||S_i||^2 as sums over a band of the keys'
 *       Gram matrix, and ||k_i||^2 as its diagonal; in the second pass (d = 64 or 128) the dots of the keys with the anchors, the fp32
 *       anchors split three ways into bf16.  A pass whose inputs do not allow the tensor form runs the
 *       FMA kernel.
 *   NKV_KEY_PASS_AUTO (default) takes the tensor form of the second pass when d = 128, and of the first
 *       pass when in addition the call's heads, dealt one per SM, keep at least 85 % of the SMs busy over
 *       the rounds that takes.
 * The forms agree to fp32 rounding.
 */
enum { NKV_KEY_PASS_AUTO = 0, NKV_KEY_PASS_FMA = 1, NKV_KEY_PASS_TENSOR = 2 };
NKV_API int nkv_set_key_passes(nkv_handle* h, int mode);

/*
 * Sections 2.1-2.3 exactly as nkv_compress runs them (same kernels, same choice), with the intermediates
 * copied out for inspection and tests:
 *   inv_norm out f32 [G,H,N]     mu_s out f32 [G,H,d]     mu_e out f32 [G,H,nb,d]
 *   a_raw    out f32 [G,H,3,N]   a_s, a_e, a_c before normalisation
 *   minmax   out f32 [G,H,6]     lo_s, hi_s, lo_e, hi_e, lo_c, hi_c of the head
 * `ws` as for nkv_compress.  Enqueues on `stream` and returns.
 */
NKV_API int nkv_key_scan(nkv_handle* h, const nkv_tensor* K, const nkv_params* params, float* inv_norm, float* mu_s,
                         float* mu_e, float* a_raw, float* minmax, void* ws, size_t ws_bytes, void* stream);

/*
 * Test hook (no counterpart in the paper).
 *   NKV_DEBUG_INJECT_HOST_STATUS  value = chunk * 16 + code: nkv_compress_host plants device status `code`
 *       in that chunk's status words before reading them back, so that the reporting of a device-side
 *       failure in any chunk can be tested without provoking one (0 clears).
 */
enum { NKV_DEBUG_INJECT_HOST_STATUS = 5 };
NKV_API int nkv_debug_set(nkv_handle* h, int what, int64_t value);

/*
 * Test hook (no counterpart in the paper): runs the bounded wait that the tensor-core key passes use for their
 * hand-overs on a barrier that nothing arrives at.  One warp polls `polls` times (1 .. 65536; a poll takes well
 * under a microsecond), gives up and records NKV_ERR_TIMEOUT in the status words at the start of `ws` (device,
 * >= 256 bytes, 256-byte aligned), which nkv_last_device_status then reports.  The kernel touches nothing else,
 * so the device stays usable: this is how a wait that runs out is tested without a kernel that hangs.
 * Enqueues on `stream` and returns.
 */
NKV_API int nkv_debug_wait_probe(nkv_handle* h, int64_t polls, void* ws, size_t ws_bytes, void* stream);

/*
 * nkv_budget for callers that cannot allocate device memory (the paper has no
 * counterpart: this is a packaging variant of nkv_budget, same arithmetic,
 * same kernel).  A host that runs inside a memory pool fixed at start-up, a
 * plugin that receives nothing but its inputs and outputs, or a step that runs
 * while the process may not grow its footprint has no scratch buffer to hand
 * to nkv_budget.  Here the scratch (status words and the per-head selection
 * thresholds, 256 + 8 * NKV_STATIC_MAX_UNITS bytes) is a fixed array inside
 * the library image; every GPU that loads the library holds it until the
 * process exits.  No handle and no workspace are needed, and the call makes no
 * cudaMalloc, cudaFree or other allocating call.
 *   a_star, r, params, budgets, stream   exactly as in nkv_budget
 *   G * H <= NKV_STATIC_MAX_UNITS, otherwise NKV_ERR_WORKSPACE is returned and
 *   nothing is launched (use nkv_budget with your own workspace instead).
 * The first call made with a given device current looks up the array's device
 * address (once per device); make that first call before any stream capture.
 * All calls on a device share the one array, which still holds what the last
 * call left: the status words are cleared on the stream at the start of each
 * call, the threshold slots of the call's G * H heads are all rewritten.  Two
 * calls whose work overlaps on the GPU (different streams) race on the array:
 * keep calls on one device ordered.  Device-side self-check results are not
 * readable through this entry point.
 */
#define NKV_STATIC_MAX_UNITS 4096
NKV_API int nkv_budget_static(const float* a_star, int64_t G, int64_t H, int64_t N, double r,
                              const nkv_params* params, int32_t* budgets, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NKV_H */
