// Pooled adapter store: one slot per tenant, holding the tenant's current policy version
// (paper: Methods, "Multi-Task Manager": per-task LoRA parameters theta_t^(v) and version counter;
// Algorithm 1: "Commit updated parameters to M").
#include <stdarg.h>
#include <stdio.h>

#include <new>

#include "sm100_ptx.cuh"

namespace marlaas {

// One CTA waits, with the tensor-core kernels' own bounded wait, on a barrier that nobody arrives on, gives up after
// limit_ns and reports it the way those kernels do (abort word -> status word); then it returns normally.
__global__ void k_wait_runs_out(int32_t* status, unsigned long long limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_word;
    const uint32_t b = sm100::smem_u32(&bar);
    if (threadIdx.x == 0) {
        sm100::mbar_init(b, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = sm100::mbar_wait_limit(b, 0, &abort_word, 99, limit_ns);
    __syncthreads();
    // every other thread sees the abort word, as the other roles of a kernel would, and leaves
    if (threadIdx.x == 0 && !ok && abort_word != 0) {
        if (atomicCAS(status, 0, DEV_TIMEOUT) == 0) status[1] = abort_word * 1000000 + (int)blockIdx.x;
    }
}

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_launches{0};

marlaas_status_t fail(marlaas_status_t code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

TimedLaunch::TimedLaunch(marlaas_pool* p, cudaStream_t s) : pool(p), st(s), on(false) {
    if (!p->timing) return;
    if (p->timing_used + 2 > p->timing_events.size()) {
        cudaEvent_t a, b;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
        p->timing_events.push_back(a);
        p->timing_events.push_back(b);
    }
    on = cudaEventRecord(p->timing_events[p->timing_used], st) == cudaSuccess;
}
TimedLaunch::~TimedLaunch() {
    if (!on) return;
    cudaEventRecord(pool->timing_events[pool->timing_used + 1], st);
    pool->timing_used += 2;
}

void part_view(const marlaas_pool* pool, int p, marlaas_pool* v) {
    v->device = pool->device;
    v->K = pool->K;
    v->N = pool->part_begin[p + 1] - pool->part_begin[p];
    v->max_rank = pool->max_rank; v->RP = pool->RP; v->cap = pool->cap;
    v->P = 1;
    v->part_begin[0] = 0; v->part_begin[1] = v->N;
    v->ldB = pool->ldB;
    v->storage = pool->storage; v->storage_bytes = pool->storage_bytes;
    v->d_status = pool->d_status; v->d_sync = pool->d_sync; v->d_rank = pool->d_rank; v->d_scale = pool->d_scale;
    v->d_At = pool->d_At + (size_t)p * pool->cap * pool->RP * (size_t)pool->K;
    v->d_Bs = pool->d_Bs + pool->part_begin[p];
    v->sm_count = pool->sm_count;
    v->slots = pool->slots;
}

StorageLayout storage_layout(int64_t K, int64_t N, int32_t RP, int32_t cap, int32_t parts) {
    StorageLayout L;
    size_t o = 0;
    L.off_status = o; o += 256;
    L.off_sync = o;   o += DECODE_SYNC_BYTES;
    L.off_rank = o;   o += align_up(sizeof(int32_t) * (size_t)cap, 256);
    L.off_scale = o;  o += align_up(sizeof(float) * (size_t)cap, 256);
    L.off_At = o;     o += align_up(sizeof(bf16) * (size_t)parts * cap * RP * (size_t)K, 256);
    L.off_Bs = o;     o += align_up(sizeof(bf16) * (size_t)cap * RP * (size_t)N, 256);
    L.total = o;
    return L;
}

static bool pool_args_ok(int64_t K, int64_t N, int32_t max_rank, int32_t cap) {
    return K > 0 && N > 0 && (K % 8) == 0 && (N % 8) == 0 && max_rank >= 1 && max_rank <= 128 && cap >= 1 &&
           cap <= 4096 && K < (1ll << 31) && N < (1ll << 31);
}

// A [K][r] row-major -> At rows (slot*RP + j)[k]; B [r][N] -> Bs rows (pitch ldB); rows r..RP-1 cleared.
__global__ void k_register(const bf16* __restrict__ A, const bf16* __restrict__ B, bf16* __restrict__ At,
                           bf16* __restrict__ Bs, int32_t* d_rank, float* d_scale, int slot, int r, int RP,
                           int64_t K, int64_t N, int64_t ldB, float scale) {
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x;
    bf16* at = At + (size_t)slot * RP * K;
    bf16* bs = Bs + (size_t)slot * RP * ldB;
    const bf16 zero = __float2bfloat16(0.f);
    for (int64_t e = tid; e < (int64_t)RP * K; e += nth) {
        const int64_t j = e / K, k = e - j * K;
        at[e] = (j < r) ? A[k * r + j] : zero;
    }
    for (int64_t e = tid; e < (int64_t)RP * N; e += nth) {
        const int64_t j = e / N, c = e - j * N;
        bs[j * ldB + c] = (j < r) ? B[e] : zero;
    }
    if (tid == 0) {
        d_rank[slot] = r;
        d_scale[slot] = scale;
    }
}

__global__ void k_export(const bf16* __restrict__ At, const bf16* __restrict__ Bs, bf16* A_out, bf16* B_out,
                         int slot, int r, int RP, int64_t K, int64_t N, int64_t ldB) {
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x;
    const bf16* at = At + (size_t)slot * RP * K;
    const bf16* bs = Bs + (size_t)slot * RP * ldB;
    if (A_out)
        for (int64_t e = tid; e < (int64_t)r * K; e += nth) {
            const int64_t k = e / r, j = e - k * r;
            A_out[e] = at[j * K + k];
        }
    if (B_out)
        for (int64_t e = tid; e < (int64_t)r * N; e += nth) {
            const int64_t j = e / N;
            B_out[e] = bs[j * ldB + (e - j * N)];
        }
}

}  // namespace marlaas

using namespace marlaas;

extern "C" {

const char* marlaas_last_error(void) { return g_err; }
uint64_t marlaas_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

// part widths of a pool over several projections: 1..MARLAAS_MAX_PARTS parts, each a positive multiple of 256 columns
// (no 256-column output tile of the fused kernels may straddle two projections)
static bool parts_ok(int32_t n_parts, const int64_t* part_d_out, int64_t* total) {
    if (n_parts < 1 || n_parts > MARLAAS_MAX_PARTS || !part_d_out) return false;
    int64_t sum = 0;
    for (int p = 0; p < n_parts; ++p) {
        if (part_d_out[p] <= 0 || (part_d_out[p] % 256) != 0) return false;
        sum += part_d_out[p];
    }
    *total = sum;
    return true;
}

size_t marlaas_adapter_pool_storage_bytes(int64_t d_in, int64_t d_out, int32_t max_rank, int32_t capacity) {
    if (!pool_args_ok(d_in, d_out, max_rank, capacity)) return 0;
    return storage_layout(d_in, d_out, (max_rank + 15) / 16 * 16, capacity).total;
}

size_t marlaas_adapter_pool_storage_bytes_segmented(int64_t d_in, int32_t n_parts, const int64_t* part_d_out,
                                                    int32_t max_rank, int32_t capacity) {
    int64_t d_out = 0;
    if (!parts_ok(n_parts, part_d_out, &d_out) || !pool_args_ok(d_in, d_out, max_rank, capacity)) return 0;
    return storage_layout(d_in, d_out, (max_rank + 15) / 16 * 16, capacity, n_parts).total;
}

static marlaas_status_t create_impl(const char* fn, marlaas_pool_t** out, int device, int64_t d_in, int32_t n_parts,
                                    const int64_t* part_d_out, int32_t max_rank, int32_t capacity, void* storage,
                                    size_t storage_bytes, void* cuda_stream) {
    if (!out) return fail(MARLAAS_ERR_INVALID_ARG, "%s: out is NULL", fn);
    *out = nullptr;
    int64_t d_out = 0;      // (the segmented entry has checked the part widths; a plain pool has one part of any width)
    for (int q = 0; q < n_parts; ++q) d_out += part_d_out[q];
    if (!pool_args_ok(d_in, d_out, max_rank, capacity))
        return fail(MARLAAS_ERR_INVALID_ARG,
                    "%s: need d_in, d_out > 0 and multiples of 8, max_rank in [1,128], capacity in [1,4096]", fn);
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        cudaGetLastError();
        return fail(MARLAAS_ERR_UNSUPPORTED_DEVICE, "%s: no CUDA device %d", fn, device);
    }
    int major = 0, sms = 0;
    MARLAAS_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    MARLAAS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    if (major != 10)
        return fail(MARLAAS_ERR_UNSUPPORTED_DEVICE, "%s: device %d is sm_%d0, this library is sm_100a only", fn, device, major);
    const int32_t RP = (max_rank + 15) / 16 * 16;
    const StorageLayout L = storage_layout(d_in, d_out, RP, capacity, n_parts);
    if (!storage || ((uintptr_t)storage & 255) != 0)
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: storage must be a 256-byte aligned device pointer", fn);
    if (storage_bytes < L.total)
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: storage_bytes %zu < required %zu", fn, storage_bytes, L.total);
    MARLAAS_CUDA_TRY(cudaSetDevice(device));
    MARLAAS_CUDA_TRY(cudaMemsetAsync(storage, 0, L.total, (cudaStream_t)cuda_stream));
    marlaas_pool* p = new (std::nothrow) marlaas_pool();
    if (!p) return fail(MARLAAS_ERR_INVALID_ARG, "%s: out of host memory", fn);
    p->device = device;
    p->K = d_in;
    p->N = d_out;
    p->ldB = d_out;
    p->P = n_parts;
    for (int q = 0; q < n_parts; ++q) p->part_begin[q + 1] = p->part_begin[q] + part_d_out[q];
    p->max_rank = max_rank;
    p->RP = RP;
    p->cap = capacity;
    p->storage = (char*)storage;
    p->storage_bytes = storage_bytes;
    p->d_status = (int32_t*)(p->storage + L.off_status);
    p->d_sync = (int32_t*)(p->storage + L.off_sync);
    p->d_rank = (int32_t*)(p->storage + L.off_rank);
    p->d_scale = (float*)(p->storage + L.off_scale);
    p->d_At = (bf16*)(p->storage + L.off_At);
    p->d_Bs = (bf16*)(p->storage + L.off_Bs);
    p->slots.resize((size_t)capacity);
    p->sm_count = sms;
    *out = p;
    return MARLAAS_OK;
}

marlaas_status_t marlaas_adapter_pool_create(marlaas_pool_t** out, int device, int64_t d_in, int64_t d_out,
                                             int32_t max_rank, int32_t capacity, void* storage,
                                             size_t storage_bytes, void* cuda_stream) {
    return create_impl("pool_create", out, device, d_in, 1, &d_out, max_rank, capacity, storage, storage_bytes, cuda_stream);
}

marlaas_status_t marlaas_adapter_pool_create_segmented(marlaas_pool_t** out, int device, int64_t d_in, int32_t n_parts,
                                                       const int64_t* part_d_out, int32_t max_rank, int32_t capacity,
                                                       void* storage, size_t storage_bytes, void* cuda_stream) {
    int64_t total = 0;
    if (out) *out = nullptr;
    if (!parts_ok(n_parts, part_d_out, &total))
        return fail(MARLAAS_ERR_INVALID_ARG, "pool_create_segmented: need 1 to %d parts, each a positive multiple of 256 columns",
                    MARLAAS_MAX_PARTS);
    return create_impl("pool_create_segmented", out, device, d_in, n_parts, part_d_out, max_rank, capacity, storage, storage_bytes,
                       cuda_stream);
}

int32_t marlaas_adapter_pool_parts(const marlaas_pool_t* pool) { return pool ? pool->P : 0; }

marlaas_status_t marlaas_kernel_timing_begin(marlaas_pool_t* pool) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "kernel_timing_begin: pool is NULL");
    pool->timing = true;
    pool->timing_used = 0;
    return MARLAAS_OK;
}

marlaas_status_t marlaas_kernel_timing_end(marlaas_pool_t* pool, float* gemm_ms, int32_t* gemm_launches) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "kernel_timing_end: pool is NULL");
    pool->timing = false;
    float total = 0.f;
    for (size_t i = 0; i + 1 < pool->timing_used; i += 2) {
        MARLAAS_CUDA_TRY(cudaEventSynchronize(pool->timing_events[i + 1]));
        float ms = 0.f;
        MARLAAS_CUDA_TRY(cudaEventElapsedTime(&ms, pool->timing_events[i], pool->timing_events[i + 1]));
        total += ms;
    }
    if (gemm_ms) *gemm_ms = total;
    if (gemm_launches) *gemm_launches = (int32_t)(pool->timing_used / 2);
    pool->timing_used = 0;
    return MARLAAS_OK;
}

marlaas_status_t marlaas_adapter_pool_destroy(marlaas_pool_t* pool) {
    if (pool) {
        for (cudaEvent_t e : pool->timing_events) cudaEventDestroy(e);
        if (pool->ev_fork) cudaEventDestroy(pool->ev_fork);
        if (pool->ev_join) cudaEventDestroy(pool->ev_join);
        if (pool->side) cudaStreamDestroy(pool->side);
    }
    delete pool;
    return MARLAAS_OK;
}

int32_t marlaas_adapter_pool_rank_stride(const marlaas_pool_t* pool) { return pool ? pool->RP : 0; }

marlaas_status_t marlaas_adapter_pool_register(marlaas_pool_t* pool, uint64_t tenant_id, uint64_t version,
                                               int32_t rank, float alpha, const void* A, const void* B,
                                               int32_t* slot_out, void* cuda_stream) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "pool_register: pool is NULL");
    if (rank < 0) return fail(MARLAAS_ERR_INVALID_ARG, "pool_register: negative rank");
    if (rank > pool->max_rank)
        return fail(MARLAAS_ERR_RANK_TOO_LARGE, "pool_register: rank %d > pool max_rank %d", rank, pool->max_rank);
    if (rank > 0 && (!A || !B)) return fail(MARLAAS_ERR_INVALID_ARG, "pool_register: A or B is NULL");
    if (rank > 0 && ((((uintptr_t)A) | ((uintptr_t)B)) & 1))
        return fail(MARLAAS_ERR_INVALID_ARG, "pool_register: A and B must be 2-byte aligned");
    int slot = -1, free_slot = -1;
    for (int s = 0; s < pool->cap; ++s) {
        if (pool->slots[s].used && pool->slots[s].tenant_id == tenant_id) { slot = s; break; }
        if (!pool->slots[s].used && free_slot < 0) free_slot = s;
    }
    if (slot < 0) slot = free_slot;
    if (slot < 0) return fail(MARLAAS_ERR_POOL_FULL, "pool_register: all %d slots in use", pool->cap);
    const float scale = rank > 0 ? alpha / (float)rank : 0.f;
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    // one launch per part: A block p is [K][rank], B block p is [rank][width of part p]
    for (int p = 0; p < pool->P; ++p) {
        const int64_t Np = pool->part_begin[p + 1] - pool->part_begin[p];
        const int64_t work = (int64_t)pool->RP * (pool->K > Np ? pool->K : Np);
        const int blocks = (int)(cdiv(work, 256) < 4 * pool->sm_count ? cdiv(work, 256) : 4 * pool->sm_count);
        const bf16* Ap = rank > 0 ? (const bf16*)A + (size_t)p * pool->K * rank : nullptr;
        const bf16* Bp = rank > 0 ? (const bf16*)B + (size_t)rank * pool->part_begin[p] : nullptr;
        k_register<<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(Ap, Bp, pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K,
                                                                  pool->d_Bs + pool->part_begin[p], pool->d_rank, pool->d_scale,
                                                                  slot, rank, pool->RP, pool->K, Np, pool->ldB, scale);
        MARLAAS_LAUNCH_CHECK("k_register");
    }
    SlotMeta& m = pool->slots[slot];
    m.used = true;
    m.tenant_id = tenant_id;
    m.version = version;
    m.rank = rank;
    m.alpha = alpha;
    m.scale = scale;
    if (slot_out) *slot_out = slot;
    return MARLAAS_OK;
}

marlaas_status_t marlaas_adapter_pool_unregister(marlaas_pool_t* pool, uint64_t tenant_id, void* cuda_stream) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "pool_unregister: pool is NULL");
    for (int s = 0; s < pool->cap; ++s) {
        if (pool->slots[s].used && pool->slots[s].tenant_id == tenant_id) {
            MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
            for (int p = 0; p < pool->P; ++p) {
                k_register<<<1, 256, 0, (cudaStream_t)cuda_stream>>>(nullptr, nullptr,
                                                                     pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K,
                                                                     pool->d_Bs + pool->part_begin[p], pool->d_rank, pool->d_scale, s, 0,
                                                                     pool->RP, pool->K, pool->part_begin[p + 1] - pool->part_begin[p],
                                                                     pool->ldB, 0.f);
                MARLAAS_LAUNCH_CHECK("k_register(unregister)");
            }
            pool->slots[s] = SlotMeta();
            return MARLAAS_OK;
        }
    }
    return fail(MARLAAS_ERR_UNKNOWN_TENANT, "pool_unregister: tenant %llu is not registered",
                (unsigned long long)tenant_id);
}

marlaas_status_t marlaas_adapter_pool_lookup(const marlaas_pool_t* pool, uint64_t tenant_id, int32_t* slot_out,
                                             int32_t* rank_out, float* scale_out, uint64_t* version_out) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "pool_lookup: pool is NULL");
    for (int s = 0; s < pool->cap; ++s) {
        const SlotMeta& m = pool->slots[s];
        if (m.used && m.tenant_id == tenant_id) {
            if (slot_out) *slot_out = s;
            if (rank_out) *rank_out = m.rank;
            if (scale_out) *scale_out = m.scale;
            if (version_out) *version_out = m.version;
            return MARLAAS_OK;
        }
    }
    return fail(MARLAAS_ERR_UNKNOWN_TENANT, "pool_lookup: tenant %llu is not registered", (unsigned long long)tenant_id);
}

marlaas_status_t marlaas_adapter_pool_export(marlaas_pool_t* pool, int32_t slot, void* A_out, void* B_out,
                                             void* cuda_stream) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "pool_export: pool is NULL");
    if (slot < 0 || slot >= pool->cap || !pool->slots[slot].used)
        return fail(MARLAAS_ERR_UNKNOWN_TENANT, "pool_export: slot %d is not in use", slot);
    const int r = pool->slots[slot].rank;
    if (r == 0 || (!A_out && !B_out)) return MARLAAS_OK;
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    for (int p = 0; p < pool->P; ++p) {
        const int64_t Np = pool->part_begin[p + 1] - pool->part_begin[p];
        const int64_t work = (int64_t)r * (pool->K > Np ? pool->K : Np);
        const int blocks = (int)(cdiv(work, 256) < 4 * pool->sm_count ? cdiv(work, 256) : 4 * pool->sm_count);
        k_export<<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K,
                                                                pool->d_Bs + pool->part_begin[p],
                                                                A_out ? (bf16*)A_out + (size_t)p * pool->K * r : nullptr,
                                                                B_out ? (bf16*)B_out + (size_t)r * pool->part_begin[p] : nullptr, slot, r,
                                                                pool->RP, pool->K, Np, pool->ldB);
        MARLAAS_LAUNCH_CHECK("k_export");
    }
    return MARLAAS_OK;
}

marlaas_status_t marlaas_debug_wait_runs_out(marlaas_pool_t* pool, uint64_t limit_ns, void* cuda_stream) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "debug_wait_runs_out: pool is NULL");
    if (limit_ns == 0 || limit_ns > 100ull * 1000 * 1000)
        return fail(MARLAAS_ERR_INVALID_ARG, "debug_wait_runs_out: limit must be in (0, 100 ms]");
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    k_wait_runs_out<<<1, 64, 0, (cudaStream_t)cuda_stream>>>(pool->d_status, (unsigned long long)limit_ns);
    MARLAAS_LAUNCH_CHECK("k_wait_runs_out");
    return MARLAAS_OK;
}

marlaas_status_t marlaas_check_status(marlaas_pool_t* pool, void* cuda_stream) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "check_status: pool is NULL");
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    int32_t w[4] = {0, 0, 0, 0};
    MARLAAS_CUDA_TRY(cudaMemcpyAsync(w, pool->d_status, sizeof(w), cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream));
    MARLAAS_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    if (w[0] == DEV_OK) return MARLAAS_OK;
    MARLAAS_CUDA_TRY(cudaMemsetAsync(pool->d_status, 0, 16, (cudaStream_t)cuda_stream));
    // a call that gave up may have left the decode path's counters and flags behind
    if (w[0] == DEV_TIMEOUT) MARLAAS_CUDA_TRY(cudaMemsetAsync(pool->d_sync, 0, DECODE_SYNC_BYTES, (cudaStream_t)cuda_stream));
    MARLAAS_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    switch (w[0]) {
        case DEV_BAD_TABLE:
            return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "device check: malformed segment table (detail %d)", w[1]);
        case DEV_BAD_INDEX:
            return fail(MARLAAS_ERR_DEVICE_BAD_INDEX, "device check: slot outside [-1, capacity) at token %d", w[1]);
        case DEV_TIMEOUT:
            return fail(MARLAAS_ERR_DEVICE_TIMEOUT, "device check: a bounded wait ran out (site %d)", w[1]);
        default:
            return fail(MARLAAS_ERR_CUDA, "device check: unknown status word %d", w[0]);
    }
}

}  // extern "C"
