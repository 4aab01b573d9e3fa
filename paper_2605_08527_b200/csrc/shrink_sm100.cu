// Segmented shrink on the tensor cores (sm_100a): per 128-token tile (half of a 256-token plan tile), h = x A_t (or g = dy B_t^T) for every tenant
// present in the tile at once.
//
// The tile's unit list (16 ranks of one tenant per unit, built by the plan kernel) names the adapter rows to
// gather from the pooled store; TMA brings each unit's [16][64] slab next to the tile's [128][64] slab of x, one
// tcgen05.mma of N = 16 * units multiplies them, and the epilogue keeps, for every token, only the columns of its
// own tenant: fp32 into out[T][RP] (the h / g the gradient reductions and h_save need) and bf16(s_t * value)
// into the block-diagonal operand hd the base GEMM's extra k-steps consume (zeros in the other tenants' columns).
// Same warp roles, pipeline and bounded waits as the base GEMM.
#include "sm100_ptx.cuh"

namespace marlaas {
namespace sm100 {

constexpr int SHRINK_THREADS = 192;
constexpr int SHRINK_STAGES = 4;
constexpr int GROUP_UNITS = 16;                          // units per pass: N = 256 accumulator columns
constexpr uint32_t SB_STAGE_BYTES = GROUP_UNITS * UNIT_BYTES;

struct ShrinkArgs {
    int T, D;
    int num_m_tiles, num_kb;
    int RP, cap;
    const int32_t* tok_slot;
    const int32_t* tok_uoff;
    const int32_t* tile_nunits;
    const int32_t* tile_units;
    int umax;
    const int32_t* d_rank;
    const float* d_scale;
    float* out;       // [T][RP], zero-filled before the launch
    bf16* hd;         // [T][hd_cols]
    int hd_cols;
    int32_t* status;
};

__device__ __forceinline__ void tc_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

__global__ void __launch_bounds__(SHRINK_THREADS, 1)
k_shrink_sm100(const __grid_constant__ CUtensorMap tmSrc, const __grid_constant__ CUtensorMap tmStore,
               const ShrinkArgs g) {
    constexpr int STAGES = SHRINK_STAGES;
    constexpr uint32_t TMEM_COLS = 512;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sA = smem_u32(smem);
    const uint32_t sB = sA + STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STAGE_BYTES + SB_STAGE_BYTES));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 5);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, 4);
        }
        mbar_init(bar_drain, 1);
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        prefetch_tmap(&tmSrc);
        prefetch_tmap(&tmStore);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {   // ---- TMA producer
            uint32_t it = 0;
            bool ok = true;
            for (int m = blockIdx.x; m < g.num_m_tiles && ok; m += gridDim.x) {
                const int nun = g.tile_nunits[m >> 1];
                for (int g0 = 0; g0 < nun && ok; g0 += GROUP_UNITS) {
                    const int nug = min(GROUP_UNITS, nun - g0);
                    const int32_t* rows = g.tile_units + (size_t)(m >> 1) * g.umax + g0;
                    for (int kb = 0; kb < g.num_kb && ok; ++kb, ++it) {
                        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                        if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 11))) break;
                        const uint32_t full = bar_full + 8 * s;
                        mbar_expect_tx(full, A_STAGE_BYTES + nug * UNIT_BYTES);
                        tma_load_2d(sA + s * A_STAGE_BYTES, &tmSrc, full, kb * BK, m * BM);
                        for (int u = 0; u < nug; ++u)
                            tma_load_2d(sB + s * SB_STAGE_BYTES + u * UNIT_BYTES, &tmStore, full, kb * BK, rows[u]);
                    }
                }
            }
            if (!ok) {
                const uint32_t back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                for (uint32_t j = 0; j < back; ++j) {
                    const uint32_t jt = it - 1 - j;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * (jt % STAGES), (jt / STAGES) & 1) &&
                           global_ns() - t0 < WAIT_LIMIT_NS) {
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {   // ---- MMA issuer
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int m = blockIdx.x; m < g.num_m_tiles && ok; m += gridDim.x) {
                const int nun = g.tile_nunits[m >> 1];
                for (int g0 = 0; g0 < nun && ok; g0 += GROUP_UNITS, ++lt) {
                    const int nug = min(GROUP_UNITS, nun - g0);
                    const uint32_t idesc = make_idesc(nug * 16, 0);
                    const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
                    if (!(ok = mbar_wait(bar_tempty + 8 * b, aph ^ 1, abort_word, 13))) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + b * 256;
                    uint32_t acc = 0;
                    for (int kb = 0; kb < g.num_kb && ok; ++kb, ++it) {
                        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                        if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 14))) break;
                        tc_fence_after();
                        const uint32_t a0 = sA + s * A_STAGE_BYTES, b0 = sB + s * SB_STAGE_BYTES;
#pragma unroll
                        for (int j = 0; j < BK / 16; ++j) {
                            tc_mma_bf16(d_tmem, desc_k_major(a0 + j * 32), desc_k_major(b0 + j * 32), idesc, acc);
                            acc = 1;
                        }
                        tc_commit(bar_empty + 8 * s);
                    }
                    if (ok) tc_commit(bar_tfull + 8 * b);
                }
            }
            if (!ok) {
                tc_commit(bar_drain);
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {
                }
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue: keep each token's own tenant columns
        const int q = warp & 3;
        uint32_t lt = 0;
        bool ok = true;
        for (int m = blockIdx.x; m < g.num_m_tiles && ok; m += gridDim.x) {
            const int nun = g.tile_nunits[m >> 1];
            const int row = m * BM + q * 32 + lane;
            int uo = -1, nu = 0;
            float sc = 0.f;
            if (row < g.T && nun > 0) {
                const int t = g.tok_slot[row];
                const int r = (t >= 0 && t < g.cap) ? g.d_rank[t] : 0;
                if (r > 0) {
                    uo = g.tok_uoff[row];
                    nu = (r + 15) >> 4;
                    sc = g.d_scale[t];
                }
            }
            for (int g0 = 0; g0 < nun && ok; g0 += GROUP_UNITS, ++lt) {
                const int nug = min(GROUP_UNITS, nun - g0);
                const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
                ok = mbar_wait(bar_tfull + 8 * b, aph, abort_word, 16);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int u = 0; u < nug; ++u) {
                    uint32_t v[16];
                    tc_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + b * 256 + u * 16, v);
                    tc_wait_ld();
                    if (row < g.T) {
                        const int gu = g0 + u;
                        const bool own = uo >= 0 && gu >= uo && gu < uo + nu;
                        uint4 o0 = make_uint4(0u, 0u, 0u, 0u), o1 = o0;
                        if (own) {
                            __nv_bfloat162 p[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                p[e] = __floats2bfloat162_rn(sc * __uint_as_float(v[2 * e]), sc * __uint_as_float(v[2 * e + 1]));
                            o0 = make_uint4(*reinterpret_cast<uint32_t*>(&p[0]), *reinterpret_cast<uint32_t*>(&p[1]),
                                            *reinterpret_cast<uint32_t*>(&p[2]), *reinterpret_cast<uint32_t*>(&p[3]));
                            o1 = make_uint4(*reinterpret_cast<uint32_t*>(&p[4]), *reinterpret_cast<uint32_t*>(&p[5]),
                                            *reinterpret_cast<uint32_t*>(&p[6]), *reinterpret_cast<uint32_t*>(&p[7]));
                            float4* dst = reinterpret_cast<float4*>(g.out + (size_t)row * g.RP + (gu - uo) * 16);
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]),
                                                     __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                        }
                        uint4* hdst = reinterpret_cast<uint4*>(g.hd + (size_t)row * g.hd_cols + gu * 16);
                        hdst[0] = o0;
                        hdst[1] = o1;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * b);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
}

}  // namespace sm100

marlaas_status_t launch_shrink_sm100(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                                     const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st) {
    using namespace sm100;
    if (T <= 0) return MARLAAS_OK;
    ShrinkArgs g;
    g.T = (int)T;
    g.D = (int)D;
    g.num_m_tiles = (int)cdiv(T, BM);
    g.num_kb = (int)cdiv(D, BK);
    g.RP = pool->RP;
    g.cap = pool->cap;
    g.tok_slot = ws.tok_slot;
    g.tok_uoff = ws.tok_uoff;
    g.tile_nunits = ws.tile_nunits;
    g.tile_units = ws.tile_units;
    g.umax = ws.umax;
    g.d_rank = pool->d_rank;
    g.d_scale = pool->d_scale;
    g.out = out;
    g.hd = ws.hd;
    g.hd_cols = ws.umax * 16;
    g.status = pool->d_status;
    alignas(64) CUtensorMap tmSrc, tmStore;
    marlaas_status_t rc;
    if ((rc = make_map(&tmSrc, src, T, D, ld, BK, BM)) != MARLAAS_OK) return rc;
    if ((rc = make_map(&tmStore, store, (int64_t)pool->cap * pool->RP, D, sld, BK, 16)) != MARLAAS_OK) return rc;
    MARLAAS_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(float) * (size_t)T * pool->RP, st));
    constexpr size_t smem_bytes = 1024 + (size_t)SHRINK_STAGES * (A_STAGE_BYTES + SB_STAGE_BYTES) + 256;
    static bool attr_set[64] = {};
    if (pool->device >= 64 || !attr_set[pool->device]) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_shrink_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        if (pool->device < 64) attr_set[pool->device] = true;
    }
    const int grid = g.num_m_tiles < pool->sm_count ? g.num_m_tiles : pool->sm_count;
    k_shrink_sm100<<<grid, SHRINK_THREADS, smem_bytes, st>>>(tmSrc, tmStore, g);
    MARLAAS_LAUNCH_CHECK("k_shrink_sm100");
    return MARLAAS_OK;
}

}  // namespace marlaas
