// Policy update and commit (Algorithm 1: "PolicyUpdate" followed by the commit of the new adapter version): AdamW on
// the fp32 master copies of the listed tenants' adapters, fused with the write of their bf16 rounding into the pooled
// store in the store's own layout (At rows = columns of A, Bs rows = rows of B), one launch for up to
// OPT_MAX_TENANTS tenants.  Bound by HBM: per element 4 fp32 reads (gradient, master, two moments), 3 fp32 writes and
// one bf16 write = 30 bytes.
#include "internal.cuh"

#include <cmath>

namespace marlaas {

constexpr int OPT_MAX_TENANTS = 16;     // pointer sets passed by value per launch
constexpr int OPT_THREADS = 256;
constexpr int OPT_TILE_K = 64;          // rows of A per transposed tile

struct OptTenant {
    const float* dA;
    const float* dB;
    float* A;
    float* B;
    float* mA;
    float* vA;
    float* mB;
    float* vB;
    int32_t slot, rank;
    int32_t vec;        // all eight pointers are 16-byte aligned: four elements per access
};
struct OptArgs {
    OptTenant t[OPT_MAX_TENANTS];
    int n, RP;
    int64_t K, N, ldB;     // ldB: elements between rows of Bs (N unless the pool holds several projections side by side)
    float lr, b1, b2, eps, wd, gscale, c1, c2;      // c1 = 1 / (1 - beta1^step), c2 = 1 / (1 - beta2^step)
    bf16* At;
    bf16* Bs;
};

__device__ __forceinline__ float adamw_update(float theta, float grad, float& m, float& v, const OptArgs& g) {
    const float gr = g.gscale * grad;
    m = g.b1 * m + (1.f - g.b1) * gr;
    v = g.b2 * v + (1.f - g.b2) * gr * gr;
    const float mh = m * g.c1, vh = v * g.c2;
    return theta - g.lr * (mh / (sqrtf(vh) + g.eps) + g.wd * theta);
}

// grid = (blocks, tenants).  The blocks of a tenant first walk B (r x N, stored as the pool stores it: same linear
// index), then A in tiles of OPT_TILE_K rows, transposed through shared memory so that both the reads of A [K][r] and
// the writes of the pool's At rows [r][K] are contiguous.
__global__ void __launch_bounds__(OPT_THREADS) k_adamw_commit(const OptArgs g) {
    __shared__ bf16 tile[OPT_TILE_K][128 + 2];
    const OptTenant& t = g.t[blockIdx.y];
    const int r = t.rank;
    // ---- B ----
    {
        bf16* bs = g.Bs + (size_t)t.slot * g.RP * g.ldB;
        const int64_t nB = (int64_t)r * g.N;
        if (g.ldB != g.N) {
            // rows of the store are further apart than rows of B
            for (int64_t e = (int64_t)blockIdx.x * OPT_THREADS + threadIdx.x; e < nB; e += (int64_t)gridDim.x * OPT_THREADS) {
                float m = t.mB[e], v = t.vB[e];
                const float th = adamw_update(t.B[e], t.dB[e], m, v, g);
                t.mB[e] = m;
                t.vB[e] = v;
                t.B[e] = th;
                const int64_t j = e / g.N;
                bs[j * g.ldB + (e - j * g.N)] = __float2bfloat16_rn(th);
            }
        } else if (t.vec && (g.N & 3) == 0) {
            // four elements per thread and access (r * N is a multiple of 4, rows of the store start 8-byte aligned)
            const int64_t n4 = nB >> 2;
            for (int64_t e = (int64_t)blockIdx.x * OPT_THREADS + threadIdx.x; e < n4; e += (int64_t)gridDim.x * OPT_THREADS) {
                float4 m = reinterpret_cast<const float4*>(t.mB)[e], v = reinterpret_cast<const float4*>(t.vB)[e];
                const float4 th0 = reinterpret_cast<const float4*>(t.B)[e], gr = __ldcs(reinterpret_cast<const float4*>(t.dB) + e);
                float4 th;
                th.x = adamw_update(th0.x, gr.x, m.x, v.x, g);
                th.y = adamw_update(th0.y, gr.y, m.y, v.y, g);
                th.z = adamw_update(th0.z, gr.z, m.z, v.z, g);
                th.w = adamw_update(th0.w, gr.w, m.w, v.w, g);
                reinterpret_cast<float4*>(t.mB)[e] = m;
                reinterpret_cast<float4*>(t.vB)[e] = v;
                reinterpret_cast<float4*>(t.B)[e] = th;
                __nv_bfloat162 p0 = __floats2bfloat162_rn(th.x, th.y), p1 = __floats2bfloat162_rn(th.z, th.w);
                uint2 o;
                o.x = *reinterpret_cast<uint32_t*>(&p0);
                o.y = *reinterpret_cast<uint32_t*>(&p1);
                reinterpret_cast<uint2*>(bs)[e] = o;
            }
        } else
        for (int64_t e = (int64_t)blockIdx.x * OPT_THREADS + threadIdx.x; e < nB; e += (int64_t)gridDim.x * OPT_THREADS) {
            float m = t.mB[e], v = t.vB[e];
            const float th = adamw_update(t.B[e], t.dB[e], m, v, g);
            t.mB[e] = m;
            t.vB[e] = v;
            t.B[e] = th;
            bs[e] = __float2bfloat16_rn(th);
        }
    }
    // ---- A ----
    bf16* at = g.At + (size_t)t.slot * g.RP * g.K;
    const int64_t ntiles = (g.K + OPT_TILE_K - 1) / OPT_TILE_K;
    for (int64_t tl = blockIdx.x; tl < ntiles; tl += gridDim.x) {
        const int64_t k0 = tl * OPT_TILE_K;
        const int kn = (int)min((int64_t)OPT_TILE_K, g.K - k0);
        if (t.vec && (r & 3) == 0) {
            for (int e4 = threadIdx.x; e4 < (kn * r) >> 2; e4 += OPT_THREADS) {
                const int64_t i4 = ((k0 * r) >> 2) + e4;
                float4 m = reinterpret_cast<const float4*>(t.mA)[i4], v = reinterpret_cast<const float4*>(t.vA)[i4];
                const float4 th0 = reinterpret_cast<const float4*>(t.A)[i4], gr = __ldcs(reinterpret_cast<const float4*>(t.dA) + i4);
                float4 th;
                th.x = adamw_update(th0.x, gr.x, m.x, v.x, g);
                th.y = adamw_update(th0.y, gr.y, m.y, v.y, g);
                th.z = adamw_update(th0.z, gr.z, m.z, v.z, g);
                th.w = adamw_update(th0.w, gr.w, m.w, v.w, g);
                reinterpret_cast<float4*>(t.mA)[i4] = m;
                reinterpret_cast<float4*>(t.vA)[i4] = v;
                reinterpret_cast<float4*>(t.A)[i4] = th;
                const int e = e4 << 2, kk = e / r, j = e - kk * r;     // four ranks of one row of A
                tile[kk][j] = __float2bfloat16_rn(th.x);
                tile[kk][j + 1] = __float2bfloat16_rn(th.y);
                tile[kk][j + 2] = __float2bfloat16_rn(th.z);
                tile[kk][j + 3] = __float2bfloat16_rn(th.w);
            }
        } else
        for (int e = threadIdx.x; e < kn * r; e += OPT_THREADS) {
            const int64_t idx = k0 * r + e;         // A is [K][r]: the tile's elements are contiguous
            float m = t.mA[idx], v = t.vA[idx];
            const float th = adamw_update(t.A[idx], t.dA[idx], m, v, g);
            t.mA[idx] = m;
            t.vA[idx] = v;
            t.A[idx] = th;
            tile[e / r][e % r] = __float2bfloat16_rn(th);
        }
        __syncthreads();
        for (int e = threadIdx.x; e < kn * r; e += OPT_THREADS) {
            const int j = e / kn, kk = e - j * kn;
            at[(size_t)j * g.K + k0 + kk] = tile[kk][j];
        }
        __syncthreads();
    }
}

}  // namespace marlaas

using namespace marlaas;

extern "C" marlaas_status_t marlaas_adapter_pool_adamw_commit(marlaas_pool_t* pool, int32_t n, const uint64_t* tenant_ids,
                                                              const uint64_t* new_versions, const float* const* dA,
                                                              const float* const* dB, float* const* A, float* const* B,
                                                              float* const* m_A, float* const* v_A, float* const* m_B,
                                                              float* const* v_B, const marlaas_adamw_t* hp,
                                                              void* cuda_stream) {
    const char* fn = "pool_adamw_commit";
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: pool is NULL", fn);
    if (n < 0) return fail(MARLAAS_ERR_INVALID_ARG, "%s: negative tenant count", fn);
    if (n == 0) return MARLAAS_OK;
    if (!tenant_ids || !dA || !dB || !A || !B || !m_A || !v_A || !m_B || !v_B || !hp)
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: a table or the hyper-parameters are NULL", fn);
    if (hp->step < 1) return fail(MARLAAS_ERR_INVALID_ARG, "%s: step %lld < 1", fn, (long long)hp->step);
    if (!(hp->beta1 >= 0.f && hp->beta1 < 1.f && hp->beta2 >= 0.f && hp->beta2 < 1.f))
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: beta1, beta2 must lie in [0, 1)", fn);
    std::vector<int> slot_of(n);
    for (int i = 0; i < n; ++i) {
        int slot = -1;
        for (int s = 0; s < pool->cap; ++s)
            if (pool->slots[s].used && pool->slots[s].tenant_id == tenant_ids[i]) { slot = s; break; }
        if (slot < 0)
            return fail(MARLAAS_ERR_UNKNOWN_TENANT, "%s: tenant %llu is not registered", fn, (unsigned long long)tenant_ids[i]);
        if (pool->slots[slot].rank <= 0)
            return fail(MARLAAS_ERR_INVALID_ARG, "%s: tenant %llu has rank 0", fn, (unsigned long long)tenant_ids[i]);
        for (int k = 0; k < i; ++k)
            if (slot_of[k] == slot)
                return fail(MARLAAS_ERR_INVALID_ARG, "%s: tenant %llu is listed twice", fn, (unsigned long long)tenant_ids[i]);
        const void* ps[8] = {dA[i], dB[i], A[i], B[i], m_A[i], v_A[i], m_B[i], v_B[i]};
        for (const void* q : ps)
            if (!q || ((uintptr_t)q & 3))
                return fail(MARLAAS_ERR_INVALID_ARG, "%s: tenant %llu: a pointer is NULL or not 4-byte aligned", fn,
                            (unsigned long long)tenant_ids[i]);
        slot_of[i] = slot;
    }
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    OptArgs g;
    g.RP = pool->RP; g.K = pool->K; g.ldB = pool->ldB;
    g.lr = hp->lr; g.b1 = hp->beta1; g.b2 = hp->beta2; g.eps = hp->eps; g.wd = hp->weight_decay; g.gscale = hp->grad_scale;
    g.c1 = (float)(1.0 / (1.0 - std::pow((double)hp->beta1, (double)hp->step)));
    g.c2 = (float)(1.0 / (1.0 - std::pow((double)hp->beta2, (double)hp->step)));
    // a pool over several projections: one pass per part (its A block, its columns of Bs, block p of every array)
    for (int p = 0; p < pool->P; ++p)
    for (int i0 = 0; i0 < n; i0 += OPT_MAX_TENANTS) {
        g.N = pool->part_begin[p + 1] - pool->part_begin[p];
        g.At = pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K;
        g.Bs = pool->d_Bs + pool->part_begin[p];
        g.n = std::min(OPT_MAX_TENANTS, n - i0);
        int max_rank = 1;
        for (int i = 0; i < g.n; ++i) {
            OptTenant& t = g.t[i];
            const int ii = i0 + i;
            const int32_t r = pool->slots[slot_of[ii]].rank;
            const size_t oa = (size_t)p * pool->K * r, ob = (size_t)r * pool->part_begin[p];
            t.dA = dA[ii] + oa; t.dB = dB[ii] + ob; t.A = A[ii] + oa; t.B = B[ii] + ob;
            t.mA = m_A[ii] + oa; t.vA = v_A[ii] + oa; t.mB = m_B[ii] + ob; t.vB = v_B[ii] + ob;
            t.slot = slot_of[ii]; t.rank = r;
            t.vec = ((((uintptr_t)t.dA | (uintptr_t)t.dB | (uintptr_t)t.A | (uintptr_t)t.B | (uintptr_t)t.mA | (uintptr_t)t.vA |
                       (uintptr_t)t.mB | (uintptr_t)t.vB) & 15) == 0);
            max_rank = std::max(max_rank, (int)t.rank);
        }
        // enough blocks per tenant to cover its larger matrix once, within a few waves over all tenants
        const int64_t elems = (int64_t)max_rank * std::max(pool->K, g.N);
        const int64_t want = std::max<int64_t>(cdiv(elems, (int64_t)OPT_THREADS * 8), cdiv(pool->K, (int64_t)OPT_TILE_K));
        const int bx = (int)std::max<int64_t>(1, std::min<int64_t>(want, (int64_t)8 * pool->sm_count / g.n + 1));
        k_adamw_commit<<<dim3((unsigned)bx, (unsigned)g.n), OPT_THREADS, 0, (cudaStream_t)cuda_stream>>>(g);
        MARLAAS_LAUNCH_CHECK("k_adamw_commit");
    }
    for (int i = 0; i < n; ++i) {
        SlotMeta& m = pool->slots[slot_of[i]];
        m.version = new_versions ? new_versions[i] : m.version + 1;
    }
    return MARLAAS_OK;
}
