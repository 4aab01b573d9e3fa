// Forward pass for callers that cannot provide (or allocate) a workspace: the per-call scratch lives in a
// file-scope device array that every GPU loading this library holds until the process exits.
//
// Who needs this: code that runs where device allocation is off the table -- a serving loop whose memory pool was
// frozen at start-up, a plug-in that is handed only its input and output buffers, a real-time path where
// cudaMalloc's implicit device synchronisation (or its failure under a tight memory budget) is not acceptable.
// Such a caller still owns x, W, y and the adapter pool; only the scratch the layer needs between its kernels
// (per-token slots, the low-rank intermediates, the expand operand) comes from here.
#include <mutex>

#include "internal.cuh"

namespace marlaas {

constexpr size_t STATIC_WS_BYTES = 8u << 20;   // 8 MiB: enough for 256 tokens on a pool of 32 slots of rank <= 64

// In host code this name is only a stand-in for the device array: its device address comes from
// cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_static_ws[STATIC_WS_BYTES];

static void* g_static_ws_addr[64] = {};
static std::mutex g_static_ws_mutex;      // two host threads may make the first call on a device at the same time

// Device address of the array on `device` (which must be current).  Resolved on first use per device: that lookup
// makes the CUDA runtime load this module on the device, which is when the device's copy of the array comes into being.
static marlaas_status_t static_ws_address(int device, void** out) {
    if (device < 0 || device >= 64)
        return fail(MARLAAS_ERR_INVALID_ARG, "lora_forward_static_ws: device index %d is outside [0,64)", device);
    std::lock_guard<std::mutex> lock(g_static_ws_mutex);
    if (!g_static_ws_addr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_ws);
        if (e != cudaSuccess || !p)
            return fail(MARLAAS_ERR_CUDA, "cudaGetSymbolAddress for the static workspace failed: %s", cudaGetErrorString(e));
        g_static_ws_addr[device] = p;
    }
    *out = g_static_ws_addr[device];
    return MARLAAS_OK;
}

}  // namespace marlaas

using namespace marlaas;

extern "C" {

size_t marlaas_lora_static_workspace_limit(void) { return STATIC_WS_BYTES; }

marlaas_status_t marlaas_lora_forward_static_ws(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx,
                                                const void* W, int64_t ldw, void* y, int64_t ldy,
                                                const marlaas_segments_t* seg, float* h_save, uint32_t flags,
                                                void* cuda_stream) {
    const char* fn = "lora_forward_static_ws";
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: pool is NULL", fn);
    if (T < 0 || T >= (1ll << 31)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: T out of range", fn);
    if (flags & MARLAAS_FLAG_OVERLAP_PREVIOUS)
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: MARLAAS_FLAG_OVERLAP_PREVIOUS needs a workspace of the call's own; every call "
                    "through this entry uses the one built-in array", fn);
    if (T == 0) return MARLAAS_OK;
    // forward's share of the workspace, without the scratch only the kernels that exchange partial sums use
    const size_t need = marlaas_lora_forward_workspace_min_bytes(pool, T);
    if (need == 0 || need > STATIC_WS_BYTES)
        return fail(MARLAAS_ERR_WORKSPACE_TOO_SMALL,
                    "%s: a batch of %lld tokens on this pool needs %zu bytes of scratch, the built-in array holds %zu; "
                    "use marlaas_lora_forward with a caller workspace",
                    fn, (long long)T, need, (size_t)STATIC_WS_BYTES);
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    void* ws = nullptr;
    marlaas_status_t rc = static_ws_address(pool->device, &ws);
    if (rc != MARLAAS_OK) return rc;
    // Every intermediate in the scratch is written by this call before it is read, so nothing has to be cleared.
    return marlaas_lora_forward(pool, T, x, ldx, W, ldw, y, ldy, seg, h_save, ws, STATIC_WS_BYTES, flags, cuda_stream);
}

}  // extern "C"
