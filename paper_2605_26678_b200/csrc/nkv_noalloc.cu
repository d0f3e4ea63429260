// nkv_budget_static: the head-wise budget competition for callers that cannot allocate.
//
// Some hosts of this library may not create device memory at the point where they need budgets:
// code running inside a memory pool whose size was fixed at start-up, a plugin that is handed
// only its inputs and outputs, or a step that runs while the process is forbidden to grow its
// footprint.  nkv_budget needs a small scratch area (status words and per-head selection
// thresholds) that such a caller has no way to provide, so this variant keeps that scratch in a
// fixed array that is part of the library image on every GPU that loads it.
//
// The array's name is only a host-side stand-in in host code; the device address is looked up
// with cudaGetSymbolAddress, once per device, by the first call made with that device current.
#include <mutex>

#include "nkv_common.cuh"

namespace {

constexpr int kStaticMaxUnits = NKV_STATIC_MAX_UNITS;
constexpr size_t kStatusBytes = nkv::kStatusWords * sizeof(int);              // 256
constexpr size_t kStaticBytes = kStatusBytes + (size_t)kStaticMaxUnits * 8;   // status words + (threshold, quota) pairs

// Scratch shared by every nkv_budget_static call on a device; lives until the process exits.
static __device__ __align__(256) unsigned char g_budget_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
void* g_scratch_addr[kMaxDevices];   // device address of g_budget_scratch, per device (null = not looked up yet)

// Device address of the scratch array on the current device (looked up on first use).
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return NKV_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return NKV_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_budget_scratch) != cudaSuccess || !p) return NKV_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return NKV_OK;
}

}  // namespace

extern "C" int nkv_budget_static(const float* a_star, int64_t G, int64_t H, int64_t N, double r,
                                 const nkv_params* params, int32_t* budgets, void* stream) {
    if (!a_star || !budgets || !params || G < 1 || H < 1 || N < 1) return NKV_ERR_INVALID_ARG;
    if (!(r >= 0.0 && r < 1.0)) return NKV_ERR_INVALID_ARG;
    if (H > 64 || N > (int64_t)1 << 24 || H * N > (int64_t)1 << 30) return NKV_ERR_UNSUPPORTED;
    if (G > kStaticMaxUnits || G * H > kStaticMaxUnits) return NKV_ERR_WORKSPACE;   // beyond the fixed scratch
    const int64_t keep = nkv_keep_per_head(N, r);
    if (keep < 1 || keep > N) return NKV_ERR_INVALID_ARG;
    const int64_t n_safe = nkv_safeguard_count(N, r, params);   // -1 when a parameter is out of range
    if (n_safe < 0) return NKV_ERR_INVALID_ARG;

    void* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != NKV_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the scratch keeps the previous call's contents: the status words must start at zero, the
    // threshold pairs of the G*H heads of this call are all rewritten by the kernel
    if (cudaMemsetAsync(scratch, 0, kStatusBytes, st) != cudaSuccess) return NKV_ERR_CUDA;
    int64_t launches = 0;
    unsigned char* base = reinterpret_cast<unsigned char*>(scratch);
    if (nkv::launch_budget((int)G, (int)H, (int)N, (int)keep, (int)n_safe, a_star, budgets,
                           reinterpret_cast<uint32_t*>(base + kStatusBytes), reinterpret_cast<int*>(base), nullptr, st,
                           &launches) != cudaSuccess)
        return NKV_ERR_CUDA;
    return NKV_OK;
}
