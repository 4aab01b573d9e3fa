// Segmented shrink with the contraction split over a cluster (sm_100a).  Same outputs as shrink_sm100.cu
// (h = x A_t or g = dy B_t^T per token, fp32, plus the bf16 block-diagonal expand operand hd), for batches with too
// few 128-token tiles to occupy the SMs one tile per CTA: a cluster of C CTAs owns one tile, each CTA streams 1/C of
// the contraction dimension through the same TMA / tcgen05 pipeline, and every CTA's epilogue sends, for each token,
// only the columns of the token's own tenant (at most RP floats) to the cluster's first CTA, which adds the C
// partial vectors in rank order and writes the results.  No atomics: the sum order is fixed.
//
// A pool over several projections that read the same activations (P blocks of adapter rows, one per projection) is served
// by ONE pass over the activations: an item's slab holds its units' rows of every block (virtual unit p * n + u = unit u
// of block p, so items take 8 / P units), the accumulator one group of 16 columns per virtual unit, and the results go
// to plane p of the outputs.
#include "sm100_ptx.cuh"

namespace marlaas {
namespace sm100 {

constexpr int SS_THREADS = 192;
constexpr int SS_SUB_UNITS = 8;                              // units per work item: N = 128 accumulator columns
constexpr int SS_KP = 2;                                     // 64-deep panels per pipeline step
constexpr uint32_t SS_STEP_BYTES = SS_KP * (A_STAGE_BYTES + SS_SUB_UNITS * UNIT_BYTES);   // 64 KB
constexpr int SS_MAX_C = 8;
constexpr int SS_MAX_STAGES = 8;
constexpr int SS_MAX_TILES = 160;

struct ShrinkSplitArgs {
    int T, D;
    int num_kb, num_m_tiles;
    int RP, cap;
    int C;
    uint32_t stage_area;   // bytes of shared memory for the pipeline stages (and, between items, the gather buffer)
    const int32_t* tok_slot;
    const int32_t* tok_uoff;
    const int32_t* tile_nunits;
    const int32_t* tile_units;
    int umax;
    const int32_t* d_rank;
    const float* d_scale;
    float* out;       // [P][T][RP], zero-filled before the launch
    bf16* hd;         // [P][T][hd_cols]
    int hd_cols;
    int P;            // blocks of adapter rows (projections of the pool) served by this pass
    int sub;          // units per work item: SS_SUB_UNITS / P
    int part_rows;    // store rows from one block to the next
    long long out_plane, hd_plane;   // elements from one plane of out / hd to the next
    int32_t* status;
};

__device__ __forceinline__ void ss_tc_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ uint32_t ss_cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t ss_cluster_id_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t ss_map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void ss_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void ss_st_cluster_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Adapter rows are fetched in runs: consecutive units of the tile's list that are also consecutive in the store (a
// tenant's own units always are, and so are neighbouring slots) move with one TMA instruction of 16 * 2^i rows, since
// the issuing thread pays about a hundred cycles per instruction whatever its size.
struct StoreMaps {
    CUtensorMap m[4];     // boxes of 16, 32, 64, 128 rows x 64 k
};

// Cuts a group's unit list into runs; run i covers 2^lg units starting at list position pos, store row `row`.
struct UnitRun { int row; short pos; short lg; };
__device__ __forceinline__ int ss_plan_runs(const int32_t* units, int nug, UnitRun* runs) {
    int u = 0, n = 0;
    while (u < nug) {
        const int r0 = units[u];
        int run = 1;
        while (u + run < nug && units[u + run] == r0 + 16 * run) ++run;
        int lg = 31 - __clz(run);                 // largest power of two <= run, at most 8 units
        if (lg > 3) lg = 3;
        runs[n].row = r0; runs[n].pos = (short)u; runs[n].lg = (short)lg;
        ++n;
        u += 1 << lg;
    }
    return n;
}

// Work items: a 128-token tile's unit list is cut into sub-groups of at most SS_SUB_UNITS units, and one item =
// (tile, sub-group).  Items, not tiles, are what costs alike (the tile of x plus a bounded slab of adapter rows per
// 64 k), so a tile that mixes many tenants is spread over several clusters instead of holding everyone up.  The
// clusters walk the item list with a fixed stride; every CTA derives the same list from the per-tile unit counts.
//
// Shared memory: [pipeline stages] [barriers].  What an SM takes in from HBM is its bytes in flight over the memory
// latency (about 2 us beside 135 other streaming CTAs), so shared memory is spent on stages and on nothing else:
//  - a stage is kp x (A panel 16 KB + the item's OWN unit slab, 2 KB per unit), so an item with one or two units (the
//    common case) runs 5-6 stages deep where a slab sized for 8 units allowed 2-3; the stage count is per item (the
//    pipeline is drained between items anyway), and each role keeps the phase of every stage barrier in a bit mask;
//  - the gather buffer (C x 128 rows x RP floats, in the cluster's first CTA) lies over the stages: once every CTA of the
//    cluster has seen its last MMA complete (one more cluster barrier per item) nothing touches them until the next item.
__global__ void __launch_bounds__(SS_THREADS, 1)
k_shrink_split_sm100(const __grid_constant__ CUtensorMap tmSrc, const __grid_constant__ StoreMaps tmStore,
                     const ShrinkSplitArgs g) {
    constexpr uint32_t TMEM_COLS = 128;
    constexpr int KP = SS_KP;
    constexpr uint32_t A_STEP = KP * A_STAGE_BYTES, B_PANEL = SS_SUB_UNITS * UNIT_BYTES, B_STEP = KP * B_PANEL;
    extern __shared__ uint8_t smem_raw[];
    __shared__ UnitRun s_runs[SS_SUB_UNITS];
    __shared__ int s_first[SS_MAX_TILES + 1];        // first item of every tile (exclusive scan of the sub-group counts)
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = ss_cluster_ctarank();
    const int cid = (int)ss_cluster_id_x(), ncl = (int)(gridDim.x / g.C);

    const uint32_t sS = smem_u32(smem);
    const uint32_t sG = sS;       // the gather buffer lies over the stages
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + g.stage_area);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * SS_MAX_STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * SS_MAX_STAGES;
    const uint32_t bar_drain = bar_tfull + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * SS_MAX_STAGES + 2);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < SS_MAX_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_drain, 1);
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        prefetch_tmap(&tmSrc);
        for (int i = 0; i < 4; ++i) prefetch_tmap(&tmStore.m[i]);
    }
    // Launched as a programmatic dependent of the plan kernel: everything above overlapped its tail; the plan's
    // outputs are read only from here on.  The base GEMM that follows may be launched in turn.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // items per tile, then their exclusive scan (one warp, five tiles per lane)
    for (int m = threadIdx.x; m < SS_MAX_TILES; m += SS_THREADS)
        s_first[m] = m < g.num_m_tiles ? (g.tile_nunits[m >> 1] + g.sub - 1) / g.sub : 0;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        constexpr int PER = SS_MAX_TILES / 32;
        int c[PER], sum = 0;
#pragma unroll
        for (int i = 0; i < PER; ++i) { c[i] = s_first[lane * PER + i]; sum += c[i]; }
        int inc = sum;
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        int run = inc - sum;
#pragma unroll
        for (int i = 0; i < PER; ++i) { s_first[lane * PER + i] = run; run += c[i]; }
        if (lane == 31) s_first[SS_MAX_TILES] = inc;
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int num_items = s_first[SS_MAX_TILES];
    const int num_steps = (g.num_kb + KP - 1) / KP;
    const int ks0 = (int)((int64_t)crank * num_steps / g.C), ks1 = (int)((int64_t)(crank + 1) * num_steps / g.C);

    // role-local pipeline state lives across items
    uint32_t p_mask = 0, p_issued = 0, p_stages = 1;     // producer: phase bit of every stage's next use; loads of this item
    uint32_t m_mask = 0;                                 // MMA issuer: likewise
    uint32_t done = 0;                        // items finished by this cluster (parity of bar_tfull)
    bool ok = true;

    for (int item = cid; item < num_items; item += ncl, ++done) {
        // item -> (tile, sub-group): the last tile whose first item is <= item
        int lo = 0, hi = g.num_m_tiles - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (s_first[mid] <= item) lo = mid; else hi = mid - 1;
        }
        const int m = lo, u0 = (item - s_first[lo]) * g.sub;
        const int nun = g.tile_nunits[m >> 1];
        const int nug = min(g.sub, nun - u0);
        const int nvu = nug * g.P;                // virtual units: the item's units in every block of adapter rows
        const int32_t* units = g.tile_units + (size_t)(m >> 1) * g.umax + u0;
        // this item's stage geometry
        const uint32_t b_panel = (uint32_t)nvu * UNIT_BYTES, stage_bytes = KP * (A_STAGE_BYTES + b_panel);
        const uint32_t nst = min((uint32_t)SS_MAX_STAGES, g.stage_area / stage_bytes);

        // per-row routing (epilogue threads): the row's units within the tile's list
        const int q = warp & 3;
        const int rl = q * 32 + lane;
        const int row = m * BM + rl;
        int uo = -1, nu = 0;
        float sc = 0.f;
        if (warp >= 2 && row < g.T) {
            const int t = g.tok_slot[row];
            const int r = (t >= 0 && t < g.cap) ? g.d_rank[t] : 0;
            if (r > 0) {
                uo = g.tok_uoff[row];
                nu = (r + 15) >> 4;
                sc = g.d_scale[t];
            }
        }

        if (warp == 0) {
            if (lane == 0 && ok) {   // ---- TMA producer: this CTA's slice of the contraction
                int32_t vunits[SS_SUB_UNITS];
                for (int p = 0; p < g.P; ++p)
                    for (int u = 0; u < nug; ++u) vunits[p * nug + u] = units[u] + p * g.part_rows;
                const int nruns = ss_plan_runs(vunits, nvu, s_runs);
                uint32_t p_s = 0;
                p_issued = 0;
                p_stages = nst;
                for (int ks = ks0; ks < ks1 && ok; ++ks) {
                    if (!(ok = mbar_wait(bar_empty + 8 * p_s, ((p_mask >> p_s) & 1u) ^ 1u, abort_word, 51))) break;
                    const uint32_t full = bar_full + 8 * p_s;
                    const uint32_t a0 = sS + p_s * stage_bytes, b0 = a0 + A_STEP;
                    mbar_expect_tx(full, A_STEP + KP * b_panel);
                    tma_load_3d(a0, &tmSrc, full, 0, m * BM, ks * KP);
                    for (int p = 0; p < KP; ++p)
                        for (int i = 0; i < nruns; ++i)
                            tma_load_2d(b0 + p * b_panel + s_runs[i].pos * UNIT_BYTES, &tmStore.m[s_runs[i].lg],
                                        full, (ks * KP + p) * BK, s_runs[i].row);
                    p_mask ^= 1u << p_s;
                    ++p_issued;
                    if (++p_s == nst) p_s = 0;
                }
            }
            __syncwarp();
        } else if (warp == 1) {
            if (lane == 0 && ok) {   // ---- MMA issuer
                const uint32_t idesc = make_idesc(nvu * 16, 0);
                uint32_t acc = 0, m_s = 0;
                for (int ks = ks0; ks < ks1 && ok; ++ks) {
                    if (!(ok = mbar_wait(bar_full + 8 * m_s, (m_mask >> m_s) & 1u, abort_word, 54))) break;
                    tc_fence_after();
                    const uint32_t a0 = sS + m_s * stage_bytes, b0 = a0 + A_STEP;
#pragma unroll
                    for (int p = 0; p < KP; ++p) {
                        const uint64_t da0 = desc_k_major(a0 + p * A_STAGE_BYTES), db0 = desc_k_major(b0 + p * b_panel);
#pragma unroll
                        for (int j = 0; j < BK / 16; ++j) {
                            tc_mma_bf16(tmem_base, da0 + (uint64_t)(2 * j), db0 + (uint64_t)(2 * j), idesc, acc);
                            acc = 1;
                        }
                    }
                    tc_commit(bar_empty + 8 * m_s);
                    m_mask ^= 1u << m_s;
                    if (++m_s == nst) m_s = 0;
                }
                if (ok) tc_commit(bar_tfull);
            }
            __syncwarp();
        } else {
            // ---- epilogue warps: wait for this CTA's accumulator
            bool eok = mbar_wait(bar_tfull, done & 1, abort_word, 56);
            eok = __all_sync(0xffffffffu, eok);
            ok = eok;
        }
        // every CTA's MMAs have completed: the stages of the first CTA may now take the partial vectors
        tc_fence_before();
        __syncthreads();
        ss_cluster_sync();
        tc_fence_after();
        if (warp >= 2) {
            // ---- this CTA's partial values of the row's own tenant columns -> gather buffer of CTA 0
            if (ok) {
                const uint32_t gdst = ss_map_to_cta(sG, 0) + ((crank * 128u + (uint32_t)rl) * (uint32_t)(g.P * g.RP)) * 4u;
                const bool empty_slice = ks0 >= ks1;      // no step: the accumulator was never written
#pragma unroll 1
                for (int vu = 0; vu < nvu; ++vu) {
                    uint32_t v[16];
                    ss_tc_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + vu * 16, v);
                    tc_wait_ld();
                    const int p = vu / nug, gu = u0 + (vu - p * nug);
                    if (uo >= 0 && gu >= uo && gu < uo + nu) {
                        const uint32_t a = gdst + (uint32_t)(p * g.RP) * 4u + (uint32_t)(gu - uo) * 64u;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (empty_slice) ss_st_cluster_v4(a + e * 16, 0u, 0u, 0u, 0u);
                            else ss_st_cluster_v4(a + e * 16, v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                        }
                    }
                }
            }
        }

        // ---- every CTA's partial vectors are in CTA 0: add them in rank order and write the results ------------
        tc_fence_before();
        __syncthreads();
        ss_cluster_sync();
        tc_fence_after();
        if (crank == 0 && warp >= 2 && row < g.T && ok) {
            const float* gbuf = reinterpret_cast<const float*>(smem);
            const int prp = g.P * g.RP;
            for (int vu = 0; vu < nvu; ++vu) {
                const int p = vu / nug, gu = u0 + (vu - p * nug);
                bf16* hrow = g.hd + (size_t)p * g.hd_plane + (size_t)row * g.hd_cols;
                uint4 o0 = make_uint4(0u, 0u, 0u, 0u), o1 = o0;
                if (uo >= 0 && gu >= uo && gu < uo + nu) {
                    float v[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) v[e] = 0.f;
                    for (int c = 0; c < g.C; ++c) {      // fixed order
                        const float4* src4 = reinterpret_cast<const float4*>(gbuf + ((size_t)c * 128 + rl) * prp + p * g.RP + (gu - uo) * 16);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float4 t4 = src4[e];
                            v[4 * e] += t4.x; v[4 * e + 1] += t4.y; v[4 * e + 2] += t4.z; v[4 * e + 3] += t4.w;
                        }
                    }
                    __nv_bfloat162 pk[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) pk[e] = __floats2bfloat162_rn(sc * v[2 * e], sc * v[2 * e + 1]);
                    o0 = make_uint4(*reinterpret_cast<uint32_t*>(&pk[0]), *reinterpret_cast<uint32_t*>(&pk[1]),
                                    *reinterpret_cast<uint32_t*>(&pk[2]), *reinterpret_cast<uint32_t*>(&pk[3]));
                    o1 = make_uint4(*reinterpret_cast<uint32_t*>(&pk[4]), *reinterpret_cast<uint32_t*>(&pk[5]),
                                    *reinterpret_cast<uint32_t*>(&pk[6]), *reinterpret_cast<uint32_t*>(&pk[7]));
                    float4* dst = reinterpret_cast<float4*>(g.out + (size_t)p * g.out_plane + (size_t)row * g.RP + (gu - uo) * 16);
#pragma unroll
                    for (int e = 0; e < 4; ++e) dst[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                }
                uint4* hdst = reinterpret_cast<uint4*>(hrow + gu * 16);
                hdst[0] = o0;
                hdst[1] = o1;
            }
        }
        // the gather buffer and the accumulator are free for the cluster's next item, whose copies (async proxy) will
        // overwrite shared memory that generic loads and stores have just used
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        tc_fence_before();
        ss_cluster_sync();
        tc_fence_after();
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    if (threadIdx.x == 0 && *abort_word != 0) {
        // let the copies already issued land (bounded) before shared memory is released
        const uint32_t back = p_issued < p_stages ? p_issued : p_stages;
        for (uint32_t j = 0; j < back; ++j) {
            const uint32_t st = (p_issued - 1 - j) % p_stages;      // its phase bit was flipped when the load went out
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_full + 8 * st, ((p_mask >> st) & 1u) ^ 1u) && global_ns() - t0 < WAIT_LIMIT_NS) {
            }
        }
    }
    if (warp == 1 && lane == 0 && *abort_word != 0) {
        tc_commit(bar_drain);
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {
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

// Cluster width for T tokens: as many CTAs per tile as keep one cluster per tile resident in a single wave (0 = this
// kernel does not apply: more tiles than SMs, where the persistent one-CTA-per-tile kernel is the better fit).
static int split_width(const marlaas_pool* pool, int64_t tiles, int64_t num_kb, size_t* smem_out, int* stages_out,
                       int* clusters_out, int P = 1) {
    using namespace sm100;
    if (tiles > pool->sm_count || tiles > SS_MAX_TILES) return 0;
    static int max_active[64][SS_MAX_C + 1] = {};
    for (int C = SS_MAX_C; C >= 1; --C) {
        if ((int64_t)C * tiles > pool->sm_count || (C > 1 && num_kb < 16 * C)) continue;
        const size_t gather = (size_t)C * 128 * pool->RP * 4 * (size_t)P;
        const size_t area = (222 * 1024 - 1024 - 256) / 1024 * 1024;      // stages; the gather buffer lies over them
        if (gather > area) continue;
        const int stages = (int)area;
        const size_t smem = 1024 + area + 256;
        int mc = pool->device < 64 ? max_active[pool->device][C] : 0;
        if (mc == 0) {
            if (cudaFuncSetAttribute(k_shrink_split_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024) != cudaSuccess) return 0;
            cudaLaunchConfig_t qc = {};
            qc.gridDim = dim3((unsigned)(C * 64));
            qc.blockDim = dim3(SS_THREADS);
            qc.dynamicSmemBytes = 200 * 1024;
            cudaLaunchAttribute qa;
            qa.id = cudaLaunchAttributeClusterDimension;
            qa.val.clusterDim.x = (unsigned)C; qa.val.clusterDim.y = 1; qa.val.clusterDim.z = 1;
            qc.attrs = &qa; qc.numAttrs = 1;
            if (cudaOccupancyMaxActiveClusters(&mc, k_shrink_split_sm100, &qc) != cudaSuccess || mc < 1) mc = -1;
            cudaGetLastError();
            if (pool->device < 64) max_active[pool->device][C] = mc;
        }
        if (mc < tiles) continue;
        *smem_out = smem;
        *stages_out = stages;
        *clusters_out = mc < pool->sm_count / C ? mc : pool->sm_count / C;     // all resident clusters walk the item list
        return C;
    }
    return 0;
}

bool shrink_split_sm100_eligible(const marlaas_pool* pool, int64_t T, int64_t D) {
    size_t smem; int stages, clusters;
    return T > 0 && (D % 64) == 0 && split_width(pool, cdiv(T, sm100::BM), cdiv(D, sm100::BK), &smem, &stages, &clusters) > 0;
}

// All P blocks of adapter rows of a pool over several projections in one pass over the activations (the blocks lie one
// after the other in the store, cap * RP rows each; out and hd are P planes of T rows).
bool shrink_split_sm100_parts_eligible(const marlaas_pool* pool, int64_t T, int64_t D, int P) {
    size_t smem; int stages, clusters;
    return T > 0 && P >= 1 && P <= 4 && (D % 64) == 0 &&
           split_width(pool, cdiv(T, sm100::BM), cdiv(D, sm100::BK), &smem, &stages, &clusters, P) > 0;
}

marlaas_status_t launch_shrink_split_sm100(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                                           const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st,
                                           bool out_is_zero, int P) {
    using namespace sm100;
    if (T <= 0) return MARLAAS_OK;
    const int64_t tiles = cdiv(T, BM);
    size_t smem_bytes = 0;
    int stages = 0, clusters = 0;
    const int C = split_width(pool, tiles, cdiv(D, BK), &smem_bytes, &stages, &clusters, P);
    if (C <= 0) return fail(MARLAAS_ERR_INVALID_ARG, "shrink_split: %lld tiles do not fit one wave", (long long)tiles);
    ShrinkSplitArgs g;
    g.T = (int)T; g.D = (int)D;
    g.num_kb = (int)cdiv(D, BK);
    g.num_m_tiles = (int)tiles;
    g.RP = pool->RP; g.cap = pool->cap;
    g.C = C; g.stage_area = (uint32_t)stages;
    g.tok_slot = ws.tok_slot; g.tok_uoff = ws.tok_uoff;
    g.tile_nunits = ws.tile_nunits; g.tile_units = ws.tile_units; g.umax = ws.umax;
    g.d_rank = pool->d_rank; g.d_scale = pool->d_scale;
    g.out = out; g.hd = ws.hd; g.hd_cols = ws.umax * 16;
    g.P = P; g.sub = SS_SUB_UNITS / P; g.part_rows = pool->cap * pool->RP;
    g.out_plane = (long long)T * pool->RP; g.hd_plane = (long long)T * g.hd_cols;
    g.status = pool->d_status;
    alignas(64) CUtensorMap tmSrc;
    alignas(64) StoreMaps maps;
    marlaas_status_t rc;
    if ((rc = make_panel_map(&tmSrc, src, T, D, ld, SS_KP)) != MARLAAS_OK) return rc;
    for (int i = 0; i < 4; ++i)
        if ((rc = make_map(&maps.m[i], store, (int64_t)P * pool->cap * pool->RP, D, sld, BK, 16u << i)) != MARLAAS_OK) return rc;
    if (!out_is_zero) MARLAAS_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(float) * (size_t)P * T * pool->RP, st));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(clusters * C));
    cfg.blockDim = dim3(SS_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_shrink_split_sm100, tmSrc, maps, g));
    count_launch();
    return MARLAAS_OK;
}

}  // namespace marlaas
