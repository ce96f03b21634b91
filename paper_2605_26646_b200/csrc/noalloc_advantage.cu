// unity_role_advantage_noalloc: the role-level advantage stage for callers that must not allocate.
//
// The regular entry point keeps two per-invocation scratch vectors (combined reward, segment id) and a table of
// per-segment accumulators in the workspace of a context, and creating a context calls cudaMalloc /
// cudaMallocHost.  Some hosts of this library cannot do that: a trainer that has handed every byte of device memory to its framework's caching
// allocator, a plug-in running under a memory budget enforced by its host process, or code that sits on a
// latency-critical path where the implicit device synchronisation of cudaMalloc is not acceptable.  For them
// the scratch lives in the fixed device array below, which exists once per GPU for as long as the library
// is loaded, and this entry point needs neither a context nor a workspace.
#include <cstdio>
#include <cstring>
#include <mutex>

#include "internal.h"

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kStatusBytes = 256;
constexpr size_t kInvBytes = 2 * sizeof(float) * UNITY_NOALLOC_MAX_INV;
constexpr size_t kTableBytes = 256 + 32 * static_cast<size_t>(UNITY_NOALLOC_MAX_SEG);   // advantage_table_bytes(MAX_SEG)
constexpr size_t kScratchBytes = kStatusBytes + kInvBytes + kTableBytes;

// [0, 256): status word (bit set when an id in the data is out of range); then r[MAX_INV]; then seg[MAX_INV]; then
// the table of the statistics passes (a 256-byte header and 32 bytes of accumulators per segment, up to MAX_SEG).
static __device__ __align__(256) unsigned char g_adv_scratch[kScratchBytes];

std::mutex g_mu;
unsigned char* g_dev_ptr[kMaxDevices];   // device address of g_adv_scratch on each device, looked up once

void say(char* err, size_t err_len, const char* msg) {
    if (err && err_len > 0) snprintf(err, err_len, "%s", msg);
}

}  // namespace

extern "C" int unity_role_advantage_noalloc(int device, void* cuda_stream, int32_t n_inv, int32_t n_traj,
                                            int32_t n_roles, int32_t n_groups, const int32_t* inv_role,
                                            const int32_t* inv_group, const int32_t* inv_traj, const float* r_node,
                                            const float* r_turn, const float* r_traj, const float* lam,
                                            const unity_adv_params* params, int64_t n_tok,
                                            const int64_t* cu_seqlens, const uint8_t* tok_mask, float* adv_inv,
                                            float* adv_tok, float* seg_mean, float* seg_std, int32_t* bad_index_out,
                                            char* err, size_t err_len) {
    using namespace unity;
    if (err && err_len > 0) err[0] = '\0';
    if (device < 0 || device >= kMaxDevices) { say(err, err_len, "device index outside [0, 64)"); return UNITY_ERR_INVALID_ARG; }
    if (n_inv < 0 || n_traj < 0 || n_tok < 0) { say(err, err_len, "negative size"); return UNITY_ERR_INVALID_ARG; }
    if (n_inv > UNITY_NOALLOC_MAX_INV) {
        char msg[160];
        snprintf(msg, sizeof(msg), "n_inv=%d exceeds UNITY_NOALLOC_MAX_INV=%d: use unity_role_advantage with a workspace",
                 n_inv, UNITY_NOALLOC_MAX_INV);
        say(err, err_len, msg);
        return UNITY_ERR_SHAPE;
    }
    if (n_roles < 1 || n_roles > UNITY_MAX_ROLES) { say(err, err_len, "n_roles outside [1, UNITY_MAX_ROLES]"); return UNITY_ERR_SHAPE; }
    if (n_groups < 1 || static_cast<long long>(n_groups) * n_roles > UNITY_NOALLOC_MAX_SEG) {
        say(err, err_len, "n_groups*n_roles outside [1, UNITY_NOALLOC_MAX_SEG]: use unity_role_advantage with a workspace");
        return UNITY_ERR_SHAPE;
    }
    if (n_inv > 0 && (!inv_role || !inv_group || !adv_inv)) { say(err, err_len, "inv_role / inv_group / adv_inv is NULL"); return UNITY_ERR_INVALID_ARG; }
    if (r_traj && n_inv > 0 && !inv_traj) { say(err, err_len, "r_traj given without inv_traj"); return UNITY_ERR_INVALID_ARG; }
    if (n_tok > 0 && (!cu_seqlens || !adv_tok || n_inv < 1)) { say(err, err_len, "cu_seqlens / adv_tok is NULL or n_inv < 1"); return UNITY_ERR_INVALID_ARG; }
    const float eps = params ? params->eps : 1e-6f;
    const int ddof = params ? params->ddof : 0;
    if (!(eps >= 0.f) || (ddof != 0 && ddof != 1)) { say(err, err_len, "eps must be >= 0 and ddof 0 or 1"); return UNITY_ERR_INVALID_ARG; }

    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); say(err, err_len, "cudaSetDevice failed"); return UNITY_ERR_CUDA; }
    unsigned char* base = nullptr;
    {
        // First call on this device: ask the runtime where the array lives on the device.  The array's name is
        // only a host-side handle; a kernel must be given the address looked up here.
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_dev_ptr[device]) {
            void* p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&p, g_adv_scratch);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                say(err, err_len, "cudaGetSymbolAddress failed for the static scratch array");
                return UNITY_ERR_CUDA;
            }
            g_dev_ptr[device] = static_cast<unsigned char*>(p);
        }
        base = g_dev_ptr[device];
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    AdvArgs a;
    memset(&a, 0, sizeof(a));
    a.status = reinterpret_cast<int*>(base);
    a.r_scratch = reinterpret_cast<float*>(base + kStatusBytes);
    a.seg_scratch = reinterpret_cast<int*>(base + kStatusBytes + sizeof(float) * UNITY_NOALLOC_MAX_INV);
    a.seg_table = base + kStatusBytes + kInvBytes;
    if (advantage_table_bytes(UNITY_NOALLOC_MAX_SEG) > kTableBytes) { say(err, err_len, "internal: static table too small"); return UNITY_ERR_CUDA; }
    a.n_inv = n_inv; a.n_traj = n_traj; a.n_roles = n_roles; a.n_groups = n_groups;
    a.inv_role = inv_role; a.inv_group = inv_group; a.inv_traj = inv_traj;
    a.r_node = r_node; a.r_turn = r_turn; a.r_traj = r_traj;
    a.has_lam = lam != nullptr;
    if (lam) memcpy(a.lam, lam, sizeof(float) * 3 * n_roles);
    a.eps = eps; a.ddof = ddof; a.n_tok = n_tok; a.cu_seqlens = cu_seqlens; a.tok_mask = tok_mask;
    a.adv_inv = adv_inv; a.adv_tok = adv_tok; a.seg_mean = seg_mean; a.seg_std = seg_std;

    // The array keeps whatever the previous call left.  The status word must start at zero, and so must the
    // accumulators of the n_groups*n_roles segments (launch_advantage clears those on the stream); the reward and
    // segment vectors are fully rewritten for [0, n_inv) before anything reads them.
    if (cudaMemsetAsync(a.status, 0, sizeof(int), st) != cudaSuccess) { cudaGetLastError(); say(err, err_len, "cudaMemsetAsync failed"); return UNITY_ERR_CUDA; }
    int nl = 0;
    if (launch_advantage(a, st, &nl) != cudaSuccess) { cudaGetLastError(); say(err, err_len, "kernel launch failed"); return UNITY_ERR_CUDA; }
    if (bad_index_out &&
        cudaMemcpyAsync(bad_index_out, a.status, sizeof(int), cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        say(err, err_len, "cudaMemcpyAsync failed");
        return UNITY_ERR_CUDA;
    }
    return UNITY_OK;
}
