// Base GEMM with the LoRA expand fused in as extra k-steps, for sm_100a: TMA-fed, tcgen05.mma with fp32
// accumulators in tensor memory, warp-specialised (1 TMA producer warp, 1 MMA issuer warp, 4 epilogue warps),
// persistent over output tiles with two accumulator buffers so that the epilogue of one tile overlaps the
// main loop of the next.
//
//   C[M][Nout] = bf16( A[M][Kc] * B  +  XA[M][units*16] * XB[units*16][Nout] )
//
// forward : A = x,  B = W        (W is [Kc][Nout] row-major: an MN-major B operand),  XA = bf16(s_t h), XB = B_t rows
// backward: A = dy, B = W^T      (W is [Nout][Kc] row-major: a K-major B operand),    XA = bf16(s_t g), XB = A_t^T rows
//
// The low-rank term rides in the same accumulator: every 256-row plan tile carries a list of 16-deep "units" (one per
// 16 ranks of each tenant present in the tile); XA holds, per token, its own tenant's scaled h (or g) in that
// tenant's unit columns and zeros elsewhere, so one extra MMA per unit adds s_t h_i B_t for all rows of the tile.
#include "sm100_ptx.cuh"

namespace marlaas {
namespace sm100 {

constexpr int NUM_THREADS = 192;

struct GemmArgs {
    int M, Nout, Kc;
    int num_m_tiles, num_n_tiles, num_kb;
    int group_m;
    int b_mn;                      // 1: B is MN-major in memory ([Kc][Nout]); 0: K-major ([Nout][Kc])
    const int32_t* tile_nunits;    // [ceil(M/256)] (one list per 256-row plan tile) or nullptr
    const int32_t* tile_units;     // [ceil(M/256)][umax]: first row of the unit in the XB store
    int umax;
    bf16* C;
    int64_t ldc;
    int32_t* status;
};

__device__ __forceinline__ void decode_tile(const GemmArgs& g, int tile, int& m_idx, int& n_idx) {
    const int per_band = g.group_m * g.num_n_tiles;
    const int band = tile / per_band;
    const int rem = tile - band * per_band;
    const int m_first = band * g.group_m;
    const int gm = min(g.group_m, g.num_m_tiles - m_first);
    n_idx = rem / gm;
    m_idx = m_first + (rem - n_idx * gm);
}

template <int BN, int STAGES>
__global__ void __launch_bounds__(NUM_THREADS, 1)
k_gemm_sm100(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const __grid_constant__ CUtensorMap tmXA, const __grid_constant__ CUtensorMap tmXB, const GemmArgs g) {
    constexpr uint32_t B_STAGE_BYTES = BN * BK * 2;
    constexpr uint32_t TMEM_COLS = 2 * BN;   // two accumulator buffers; a power of two >= 32
    constexpr int NCHUNK = BN / 64;
    static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "tensor memory allocation size");

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sA = smem_u32(smem);
    const uint32_t sB = sA + STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 5);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = g.num_m_tiles * g.num_n_tiles;

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
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (g.tile_nunits) {
            prefetch_tmap(&tmXA);
            prefetch_tmap(&tmXB);
        }
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
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int m_idx, n_idx;
                decode_tile(g, tile, m_idx, n_idx);
                const int m0 = m_idx * BM, n0 = n_idx * BN;
                const int nchunk = min(NCHUNK, (g.Nout - n0 + 63) / 64);
                for (int kb = 0; kb < g.num_kb && ok; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 1))) break;
                    const uint32_t full = bar_full + 8 * s;
                    if (g.b_mn) {
                        mbar_expect_tx(full, A_STAGE_BYTES + nchunk * CHUNK_BYTES);
                        tma_load_2d(sA + s * A_STAGE_BYTES, &tmA, full, kb * BK, m0);
                        for (int c = 0; c < nchunk; ++c)
                            tma_load_2d(sB + s * B_STAGE_BYTES + c * CHUNK_BYTES, &tmB, full, n0 + c * 64, kb * BK);
                    } else {
                        mbar_expect_tx(full, A_STAGE_BYTES + B_STAGE_BYTES);
                        tma_load_2d(sA + s * A_STAGE_BYTES, &tmA, full, kb * BK, m0);
                        tma_load_2d(sB + s * B_STAGE_BYTES, &tmB, full, kb * BK, n0);
                    }
                }
                const int nun = g.tile_nunits ? g.tile_nunits[m_idx >> 1] : 0;
                for (int x0 = 0; x0 < nun && ok; x0 += 4, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 2))) break;
                    const uint32_t full = bar_full + 8 * s;
                    const int nv = min(4, nun - x0);
                    mbar_expect_tx(full, A_STAGE_BYTES + nv * nchunk * UNIT_BYTES);
                    tma_load_2d(sA + s * A_STAGE_BYTES, &tmXA, full, x0 * 16, m0);
                    for (int u = 0; u < nv; ++u) {
                        const int row = g.tile_units[(size_t)(m_idx >> 1) * g.umax + x0 + u];
                        for (int c = 0; c < nchunk; ++c)
                            tma_load_2d(sB + s * B_STAGE_BYTES + c * CHUNK_BYTES + u * UNIT_BYTES, &tmXB, full,
                                        n0 + c * 64, row);
                    }
                }
            }
            if (!ok) {
                // let the copies already issued land (bounded) before the CTA's shared memory is released
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
        // ================= MMA issuer =================
        if (lane == 0) {
            constexpr uint32_t idesc_mn = make_idesc(BN, 1);
            const uint32_t idesc_main = make_idesc(BN, g.b_mn);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
                int m_idx, n_idx;
                decode_tile(g, tile, m_idx, n_idx);
                const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
                if (!(ok = mbar_wait(bar_tempty + 8 * b, aph ^ 1, abort_word, 3))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * BN;
                uint32_t acc = 0;
                for (int kb = 0; kb < g.num_kb && ok; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 4))) break;
                    tc_fence_after();
                    const uint32_t a0 = sA + s * A_STAGE_BYTES, b0 = sB + s * B_STAGE_BYTES;
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        const uint64_t da = desc_k_major(a0 + j * 32);
                        const uint64_t db = g.b_mn ? desc_mn_major(b0 + j * UNIT_BYTES, CHUNK_BYTES)
                                                   : desc_k_major(b0 + j * 32);
                        tc_mma_bf16(d_tmem, da, db, idesc_main, acc);
                        acc = 1;
                    }
                    tc_commit(bar_empty + 8 * s);
                }
                const int nun = g.tile_nunits ? g.tile_nunits[m_idx >> 1] : 0;
                for (int x0 = 0; x0 < nun && ok; x0 += 4, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 5))) break;
                    tc_fence_after();
                    const uint32_t a0 = sA + s * A_STAGE_BYTES, b0 = sB + s * B_STAGE_BYTES;
                    const int nv = min(4, nun - x0);
                    for (int u = 0; u < nv; ++u) {
                        tc_mma_bf16(d_tmem, desc_k_major(a0 + u * 32), desc_mn_major(b0 + u * UNIT_BYTES, CHUNK_BYTES),
                                    idesc_mn, acc);
                        acc = 1;
                    }
                    tc_commit(bar_empty + 8 * s);
                }
                if (ok) tc_commit(bar_tfull + 8 * b);
            }
            if (!ok) {
                // wait (bounded) for the MMAs already issued before tensor memory is released
                tc_commit(bar_drain);
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {
                }
            }
        }
        __syncwarp();
    } else {
        // ================= epilogue: tensor memory -> registers -> bf16 -> global =================
        const int q = warp & 3;   // this warp may touch tensor-memory lanes [32q, 32q+32)
        uint32_t lt = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
            int m_idx, n_idx;
            decode_tile(g, tile, m_idx, n_idx);
            const int m0 = m_idx * BM, n0 = n_idx * BN;
            const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
            ok = mbar_wait(bar_tfull + 8 * b, aph, abort_word, 6);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            bf16* crow = g.C + (size_t)row * g.ldc + n0;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + b * BN + c * 32, v);
                tc_wait_ld();
                if (row < g.M) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int col = n0 + c * 32 + e * 8;
                        if (col < g.Nout) {
                            uint4 o;
                            __nv_bfloat162 p0 = __floats2bfloat162_rn(__uint_as_float(v[e * 8 + 0]), __uint_as_float(v[e * 8 + 1]));
                            __nv_bfloat162 p1 = __floats2bfloat162_rn(__uint_as_float(v[e * 8 + 2]), __uint_as_float(v[e * 8 + 3]));
                            __nv_bfloat162 p2 = __floats2bfloat162_rn(__uint_as_float(v[e * 8 + 4]), __uint_as_float(v[e * 8 + 5]));
                            __nv_bfloat162 p3 = __floats2bfloat162_rn(__uint_as_float(v[e * 8 + 6]), __uint_as_float(v[e * 8 + 7]));
                            o.x = *reinterpret_cast<uint32_t*>(&p0);
                            o.y = *reinterpret_cast<uint32_t*>(&p1);
                            o.z = *reinterpret_cast<uint32_t*>(&p2);
                            o.w = *reinterpret_cast<uint32_t*>(&p3);
                            *reinterpret_cast<uint4*>(crow + c * 32 + e * 8) = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * b);
        }
    }

    // ---- teardown: every role has left its loop (normally, or after a bounded wait ran out) -------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
}

// ---- host side -----------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

marlaas_status_t make_map(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int64_t ld,
                                 uint32_t box_cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(MARLAAS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstr[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(MARLAAS_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) for a %lld x %lld tensor, pitch %lld", (int)r,
                    (long long)rows, (long long)cols, (long long)ld);
    return MARLAAS_OK;
}

template <int BN, int STAGES>
static marlaas_status_t launch_t(const marlaas_pool* pool, const GemmOperands& o, cudaStream_t st) {
    GemmArgs g;
    g.M = (int)o.M;
    g.Nout = (int)o.Nout;
    g.Kc = (int)o.Kc;
    g.num_m_tiles = (int)cdiv(o.M, BM);
    g.num_n_tiles = (int)cdiv(o.Nout, BN);
    g.num_kb = (int)cdiv(o.Kc, BK);
    g.group_m = 16;
    g.b_mn = o.b_mn ? 1 : 0;
    g.tile_nunits = o.tile_nunits;
    g.tile_units = o.tile_units;
    g.umax = o.umax;
    g.C = o.C;
    g.ldc = o.ldc;
    g.status = pool->d_status;

    alignas(64) CUtensorMap tmA, tmB, tmXA, tmXB;
    marlaas_status_t rc;
    if ((rc = make_map(&tmA, o.A, o.M, o.Kc, o.lda, BK, BM)) != MARLAAS_OK) return rc;
    if (o.b_mn) {
        if ((rc = make_map(&tmB, o.B, o.Kc, o.Nout, o.ldb, 64, BK)) != MARLAAS_OK) return rc;
    } else {
        if ((rc = make_map(&tmB, o.B, o.Nout, o.Kc, o.ldb, BK, BN)) != MARLAAS_OK) return rc;
    }
    if (o.tile_nunits) {
        if ((rc = make_map(&tmXA, o.XA, o.M, o.xa_cols, o.xa_cols, BK, BM)) != MARLAAS_OK) return rc;
        if ((rc = make_map(&tmXB, o.XB, o.xb_rows, o.Nout, o.xb_ld, 64, 16)) != MARLAAS_OK) return rc;
    } else {
        tmXA = tmA;
        tmXB = tmB;
    }
    constexpr size_t smem_bytes = 1024 + (size_t)STAGES * (A_STAGE_BYTES + BN * BK * 2) + 256;
    static bool attr_set[64] = {};
    if (pool->device >= 64 || !attr_set[pool->device]) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_gemm_sm100<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem_bytes));
        if (pool->device < 64) attr_set[pool->device] = true;
    }
    const int tiles = g.num_m_tiles * g.num_n_tiles;
    const int grid = tiles < pool->sm_count ? tiles : pool->sm_count;
    k_gemm_sm100<BN, STAGES><<<grid, NUM_THREADS, smem_bytes, st>>>(tmA, tmB, tmXA, tmXB, g);
    MARLAAS_LAUNCH_CHECK("k_gemm_sm100");
    return MARLAAS_OK;
}

}  // namespace sm100

marlaas_status_t launch_gemm_sm100(const marlaas_pool* pool, const GemmOperands& o, cudaStream_t st) {
    if (o.M <= 0) return MARLAAS_OK;
    return sm100::launch_t<256, 4>(pool, o, st);
}

}  // namespace marlaas
