// Base GEMM with the fused LoRA expand, 2-CTA form (sm_100a): a cluster of two CTAs owns one 256 x 256 output
// tile.  Each CTA stages its own 128 rows of A and its own 128 columns of B; one tcgen05.mma.cta_group::2 issued by
// the leader CTA (cluster rank 0) multiplies the pair's operands into both CTAs' tensor memory, so each SM moves
// and re-reads only half of B -- the single-CTA kernel is limited by shared-memory bandwidth (TMA writes plus
// operand reads), this one is not.  Same operand conventions and extra k-steps as gemm_sm100.cu:
//
//   C[M][Nout] = bf16( A[M][Kc] * B  +  XA[M][units*16] * XB[units*16][Nout] )
//
// Synchronisation (all waits bounded):
//   full[s]   leader's barrier; the leader's producer posts the expected bytes of BOTH CTAs, both CTAs' TMA loads
//             (cta_group::2 form, no multicast) complete on it
//   empty[s]  one per CTA; the leader's tcgen05.commit (multicast to both CTAs) releases the stage in both
//   tfull[b]  one per CTA, same multicast commit after the tile's last MMA
//   tempty[b] leader's barrier, 8 arrivals: the four epilogue warps of each CTA (the peer's arrive remotely)
#include "sm100_ptx.cuh"

namespace marlaas {
namespace sm100 {

constexpr int G2_THREADS = 192;
constexpr int G2_STAGES = 6;
constexpr int G2_BN = 256;                               // tile columns; each CTA stages 128 of them
constexpr uint32_t G2_B_STAGE_BYTES = 128 * BK * 2;      // 16 KB
constexpr uint32_t G2_STAGE_BYTES = A_STAGE_BYTES + G2_B_STAGE_BYTES;

struct Gemm2Args {
    int M, Nout, Kc;
    int num_m_tiles, num_n_tiles, num_kb;   // 256 x 256 tiles
    int group_m;
    int b_mn;
    const int32_t* tile_nunits;             // per 256-row tile
    const int32_t* tile_units;
    int umax;
    // A pool over several projections (parts > 1): XA holds one plane of M rows per part; an output tile of the forward
    // product (all_parts = 0) takes the plane of the part its columns lie in (part_end: the parts' last columns + 1),
    // the dx product (all_parts = 1) sums over every part's plane against that part's block of XB rows.
    int parts, all_parts;
    int part_end[4];
    int xb_part_rows;
    bf16* C;
    int64_t ldc;
    int32_t* status;
};

// the parts whose low-rank term enters output columns n0 ...
__device__ __forceinline__ void tile_parts(const Gemm2Args& g, int n0, int& p_lo, int& p_hi) {
    p_lo = 0;
    p_hi = 1;
    if (g.parts > 1) {
        if (g.all_parts) p_hi = g.parts;
        else {      // constant indices: a variable one would move the kernel's arguments to local memory
            p_lo = (int)(n0 >= g.part_end[0]) + (int)(g.parts > 2 && n0 >= g.part_end[1]) + (int)(g.parts > 3 && n0 >= g.part_end[2]);
            p_hi = p_lo + 1;
        }
    }
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load whose completion is signalled on a barrier that may live in the peer CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0,
                                                 int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(mask)
                 : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// M = 256 across the pair, N = 256, bf16 x bf16 -> fp32, A K-major.
__host__ __device__ constexpr uint32_t make_idesc_pair(int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(G2_BN >> 3) << 17) |
           ((uint32_t)(256 >> 4) << 24);
}

__device__ __forceinline__ void decode_tile2(const Gemm2Args& g, int tile, int& m_idx, int& n_idx) {
    const int per_band = g.group_m * g.num_n_tiles;
    const int band = tile / per_band;
    const int rem = tile - band * per_band;
    const int m_first = band * g.group_m;
    const int gm = min(g.group_m, g.num_m_tiles - m_first);
    n_idx = rem / gm;
    m_idx = m_first + (rem - n_idx * gm);
}

// bytes CTA `r` of the pair stages for one k-block of tile (m0, n0)
__device__ __forceinline__ int half_chunks(const Gemm2Args& g, int n0, int r) {
    return max(0, min(2, (g.Nout - (n0 + r * 128) + 63) / 64));
}
__device__ __forceinline__ uint32_t main_bytes(const Gemm2Args& g, int m0, int n0, int r, uint32_t kp) {
    const uint32_t a = (m0 + r * 128 < g.M) ? A_STAGE_BYTES : 0u;
    const uint32_t b = g.b_mn ? (uint32_t)half_chunks(g, n0, r) * CHUNK_BYTES
                              : ((n0 + r * 128 < g.Nout) ? G2_B_STAGE_BYTES : 0u);
    return kp * (a + b);      // kp 64-deep panels per pipeline step
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ uint32_t extra_bytes(const Gemm2Args& g, int m0, int n0, int r, int nv) {
    const uint32_t a = (m0 + r * 128 < g.M) ? A_STAGE_BYTES : 0u;
    return a + (uint32_t)(nv * half_chunks(g, n0, r)) * UNIT_BYTES;
}

// KP = 64-deep panels per pipeline step.  KP = 2 (contraction depth a multiple of 64): x / dy and a K-major W are viewed as
// 3-D tensors so that ONE TMA instruction brings both panels, and the barrier wait / expect / commit of the two issuing
// threads is paid once per 128 of depth; KP = 1 is the plain 2-D form for any depth.
template <int KP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(G2_THREADS, 1)
k_gemm2_sm100(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmXA, const __grid_constant__ CUtensorMap tmXB, const Gemm2Args g) {
    constexpr int STAGES = G2_STAGES / KP;
    constexpr uint32_t A_ST = KP * A_STAGE_BYTES, B_ST = KP * G2_B_STAGE_BYTES;
    constexpr uint32_t TMEM_COLS = 512;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sA = smem_u32(smem);
    const uint32_t sB = sA + STAGES * A_ST;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_ST + B_ST));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 5);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();      // 0 = leader
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = g.num_m_tiles * g.num_n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, 8);
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
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // both CTAs' barriers are initialised before any remote arrive or TMA completion
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================= TMA producer (both CTAs) =================
        if (lane == 0) {
            uint32_t it = 0, s = 0, ph = 0;     // blocks issued; stage and phase bit of the next block
            bool ok = true, waited = false;
            const uint32_t full0 = map_to_cta(bar_full, 0);      // the leader's full barriers (8 bytes apart)
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                int m_idx, n_idx;
                decode_tile2(g, tile, m_idx, n_idx);
                const int m0 = m_idx * 256, n0 = n_idx * G2_BN;
                const int my_m = m0 + (int)rank * 128, my_n = n0 + (int)rank * 128;
                const bool have_rows = my_m < g.M;
                const int nchunk = half_chunks(g, n0, (int)rank);
                const uint32_t stage_tx = main_bytes(g, m0, n0, 0, KP) + main_bytes(g, m0, n0, 1, KP);
                for (int kb = 0; kb < g.num_kb && ok; ++kb, ++it) {
                    if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 31))) break;
                    const uint32_t full = full0 + 8 * s;
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                    if (have_rows) {
                        if (KP == 1) tma_load_2d_pair(sA + s * A_ST, &tmA, full, kb * BK, my_m);
                        else tma_load_3d_pair(sA + s * A_ST, &tmA, full, 0, my_m, kb * KP);
                    }
                    if (g.b_mn) {      // box: 64 columns x (KP * 64) rows of W
                        for (int c = 0; c < nchunk; ++c)
                            tma_load_2d_pair(sB + s * B_ST + c * (KP * CHUNK_BYTES), &tmB, full, my_n + c * 64, kb * KP * BK);
                    } else if (my_n < g.Nout) {
                        if (KP == 1) tma_load_2d_pair(sB + s * B_ST, &tmB, full, kb * BK, my_n);
                        else tma_load_3d_pair(sB + s * B_ST, &tmB, full, 0, my_n, kb * KP);
                    }
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
                }
                if (!waited) {      // the plan and hd come from the kernels this one was launched behind
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    waited = true;
                }
                const int nun = g.tile_nunits ? g.tile_nunits[m_idx] : 0;
                int p_lo, p_hi;
                tile_parts(g, n0, p_lo, p_hi);
                for (int p = p_lo; p < p_hi; ++p)
                for (int x0 = 0; x0 < nun && ok; x0 += 4, ++it) {
                    if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 32))) break;
                    const uint32_t full = full0 + 8 * s;
                    const int nv = min(4, nun - x0);
                    if (rank == 0)
                        mbar_expect_tx(bar_full + 8 * s, extra_bytes(g, m0, n0, 0, nv) + extra_bytes(g, m0, n0, 1, nv));
                    if (have_rows) tma_load_2d_pair(sA + s * A_ST, &tmXA, full, x0 * 16, my_m + p * g.M);
                    for (int u = 0; u < nv; ++u) {
                        const int row = g.tile_units[(size_t)m_idx * g.umax + x0 + u] + (g.all_parts ? p * g.xb_part_rows : 0);
                        for (int c = 0; c < nchunk; ++c)
                            tma_load_2d_pair(sB + s * B_ST + c * CHUNK_BYTES + u * UNIT_BYTES, &tmXB, full,
                                             my_n + c * 64, row);
                    }
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
                }
            }
            if (!ok && rank == 0) {
                // let the copies already issued land (bounded) before shared memory is released
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
        // ================= MMA issuer (leader CTA only) =================
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc_mn = make_idesc_pair(1);
            const uint32_t idesc_main = make_idesc_pair(g.b_mn);
            uint32_t lt = 0, s = 0, ph = 0;     // stage and phase bit of the next k-block (running counters: no division)
            bool ok = true, waited = false;
            // descriptors of a stage's operands differ from stage 0's, and those of successive 16-deep slices from the
            // first slice's, only in the start-address field (16-byte units): they are stepped, not rebuilt
            const uint64_t da_base = desc_k_major(sA);
            const uint64_t db_base = g.b_mn ? desc_mn_major(sB, KP * CHUNK_BYTES) : desc_k_major(sB);
            const uint64_t db_step = g.b_mn ? (uint64_t)(UNIT_BYTES >> 4) : 2ull;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++lt) {
                int m_idx, n_idx;
                decode_tile2(g, tile, m_idx, n_idx);
                const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
                if (!(ok = mbar_wait(bar_tempty + 8 * b, aph ^ 1, abort_word, 33))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * G2_BN;
                uint32_t acc = 0;
                for (int kb = 0; kb < g.num_kb && ok; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 34))) break;
                    const uint64_t da = da_base + (uint64_t)(s * (A_ST >> 4));
                    const uint64_t db = db_base + (uint64_t)(s * (B_ST >> 4));
#pragma unroll
                    for (int p = 0; p < KP; ++p) {
                        // panel p: A tile 16 KB further; B rows 64 further down a chunk (MN-major) or tile 16 KB further (K-major)
                        const uint64_t dap = da + (uint64_t)(p * (A_STAGE_BYTES >> 4));
                        const uint64_t dbp = db + (g.b_mn ? (uint64_t)(p * (CHUNK_BYTES >> 4)) : (uint64_t)(p * (G2_B_STAGE_BYTES >> 4)));
#pragma unroll
                        for (int j = 0; j < BK / 16; ++j) {
                            tc_mma_bf16_pair(d_tmem, dap + (uint64_t)(2 * j), dbp + (uint64_t)j * db_step, idesc_main, acc);
                            acc = 1;
                        }
                    }
                    tc_commit_pair(bar_empty + 8 * s);
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
                }
                if (!waited) {
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    waited = true;
                }
                const int nun = g.tile_nunits ? g.tile_nunits[m_idx] : 0;
                int p_lo, p_hi;
                tile_parts(g, n_idx * G2_BN, p_lo, p_hi);
                for (int p = p_lo; p < p_hi; ++p)
                for (int x0 = 0; x0 < nun && ok; x0 += 4) {
                    if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 35))) break;
                    tc_fence_after();
                    const uint32_t a0 = sA + s * A_ST, b0 = sB + s * B_ST;
                    const int nv = min(4, nun - x0);
                    for (int u = 0; u < nv; ++u) {
                        tc_mma_bf16_pair(d_tmem, desc_k_major(a0 + u * 32),
                                         desc_mn_major(b0 + u * UNIT_BYTES, CHUNK_BYTES), idesc_mn, acc);
                        acc = 1;
                    }
                    tc_commit_pair(bar_empty + 8 * s);
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
                }
                if (ok) tc_commit_pair(bar_tfull + 8 * b);
            }
            if (!ok) {
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_drain)
                             : "memory");
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {
                }
            }
        }
        __syncwarp();
    } else {
        // ================= epilogue (both CTAs): own 128 rows of the tile =================
        const int q = warp & 3;
        const uint32_t tempty_leader0 = map_to_cta(bar_tempty, 0);
        uint32_t lt = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++lt) {
            int m_idx, n_idx;
            decode_tile2(g, tile, m_idx, n_idx);
            const int m0 = m_idx * 256 + (int)rank * 128, n0 = n_idx * G2_BN;
            const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
            ok = mbar_wait(bar_tfull + 8 * b, aph, abort_word, 36);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            bf16* crow = g.C + (size_t)row * g.ldc + n0;
#pragma unroll 1
            for (int c = 0; c < G2_BN / 32; ++c) {
                uint32_t v[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + b * G2_BN + c * 32, v);
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
            if (lane == 0) mbar_arrive_cluster(tempty_leader0 + 8 * b);
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    if (threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");   // never complete before the kernels it was launched behind
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // neither CTA leaves while its pair may still signal its barriers or use its operands
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
}

}  // namespace sm100

bool gemm2_sm100_eligible(const marlaas_pool* pool, int64_t M) { return M >= 1024 && pool->sm_count >= 2; }

template <int KP>
static marlaas_status_t launch_gemm2_t(const marlaas_pool* pool, const GemmOperands& o, cudaStream_t st) {
    using namespace sm100;
    Gemm2Args g;
    g.M = (int)o.M;
    g.Nout = (int)o.Nout;
    g.Kc = (int)o.Kc;
    g.num_m_tiles = (int)cdiv(o.M, 256);
    g.num_n_tiles = (int)cdiv(o.Nout, G2_BN);
    g.num_kb = (int)cdiv(o.Kc, (int64_t)BK * KP);      // pipeline steps
    g.group_m = g.num_m_tiles >= 32 ? 16 : 8;      // row tiles per band (measured: 8-16 best; 32 loses the band's x rows from L2)
    // A band's rows of A should stay in L2 while the band's column tiles pass over them: with a deep contraction (the dx
    // launch: 11008) sixteen row tiles are 90 MB and are read again by every wave of the band; eight are 45 MB.
    while (g.group_m > 4 && (int64_t)g.group_m * 256 * o.Kc * 2 > (int64_t)48 << 20) g.group_m >>= 1;
    g.b_mn = o.b_mn ? 1 : 0;
    g.tile_nunits = o.tile_nunits;
    g.tile_units = o.tile_units;
    g.umax = o.umax;
    g.parts = o.parts > 1 ? o.parts : 1;
    g.all_parts = o.all_parts ? 1 : 0;
    for (int p = 0; p < 4; ++p) g.part_end[p] = p < o.parts ? (int)o.part_end[p] : 0;
    g.xb_part_rows = (int)(o.xb_rows / g.parts);
    g.C = o.C;
    g.ldc = o.ldc;
    g.status = pool->d_status;

    alignas(64) CUtensorMap tmA, tmB, tmXA, tmXB;
    marlaas_status_t rc;
    if (KP == 1) rc = make_map(&tmA, o.A, o.M, o.Kc, o.lda, BK, BM);
    else rc = make_panel_map(&tmA, o.A, o.M, o.Kc, o.lda, KP);
    if (rc != MARLAAS_OK) return rc;
    if (o.b_mn) rc = make_map(&tmB, o.B, o.Kc, o.Nout, o.ldb, 64, BK * KP);
    else if (KP == 1) rc = make_map(&tmB, o.B, o.Nout, o.Kc, o.ldb, BK, 128);
    else rc = make_panel_map(&tmB, o.B, o.Nout, o.Kc, o.ldb, KP);
    if (rc != MARLAAS_OK) return rc;
    if (o.tile_nunits) {
        if ((rc = make_map(&tmXA, o.XA, o.M * g.parts, o.xa_cols, o.xa_cols, BK, BM)) != MARLAAS_OK) return rc;
        if ((rc = make_map(&tmXB, o.XB, o.xb_rows, o.Nout, o.xb_ld, 64, 16)) != MARLAAS_OK) return rc;
    } else {
        tmXA = tmA;
        tmXB = tmB;
    }
    constexpr size_t smem_bytes = 1024 + (size_t)G2_STAGES * G2_STAGE_BYTES + 256;
    static int max_clusters[64] = {};
    int& mc = max_clusters[pool->device < 64 ? pool->device : 63];
    if (mc == 0 || pool->device >= 64) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_gemm2_sm100<KP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * (unsigned)(pool->sm_count / 2));
        cfg.blockDim = dim3(G2_THREADS);
        cfg.dynamicSmemBytes = smem_bytes;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = 2;
        at.val.clusterDim.y = 1;
        at.val.clusterDim.z = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        int n = 0;
        MARLAAS_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, k_gemm2_sm100<KP>, &cfg));
        if (n < 1) return fail(MARLAAS_ERR_CUDA, "no 2-CTA cluster of the GEMM kernel fits on this device");
        mc = n;
    }
    const int tiles = g.num_m_tiles * g.num_n_tiles;
    const int pairs = tiles < mc ? tiles : mc;
    // launched as a programmatic dependent: its main loop (x and W only) may start while the shrink's last CTAs run
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)pairs);
    cfg.blockDim = dim3(G2_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_gemm2_sm100<KP>, tmA, tmB, tmXA, tmXB, g));
    count_launch();
    return MARLAAS_OK;
}

marlaas_status_t launch_gemm2_sm100(const marlaas_pool* pool, const GemmOperands& o, cudaStream_t st) {
    if (o.M <= 0) return MARLAAS_OK;
    // two panels per step need the contraction depth in whole 64-deep panels (3-D views of the row-major operands)
    return (o.Kc % 64) == 0 ? launch_gemm2_t<2>(pool, o, st) : launch_gemm2_t<1>(pool, o, st);
}

}  // namespace marlaas
