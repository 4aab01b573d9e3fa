// Decode-shaped forward (up to four 256-token tiles, typically one token per sequence, tenants unsorted): the call is
// bound by the one pass over W from HBM (or, from about 300 tokens, by the tensor cores on a grid of few tiles), so the
// work is cut to keep every SM busy and the launch count to two overlapping kernels.
//
//   k_decode_shrink  (CUDA cores + warp-level MMA)  per tenant: h_i = x_i A_t for the tenant's tokens, gathered from
//                    the pooled store; a cluster of CTAs splits K and sums its partial products through distributed
//                    shared memory in a fixed order.  Writes tok_slot, h (fp32) and the dense expand operand
//                    hd[i][t*RP + j] = bf16(s_t h_i[j]) (zeros in every other tenant's columns).
//   k_decode_gemm    (tcgen05, TMA)  y = bf16( [x | hd] * [W ; Bs] ): the base product and the expand as one
//                    contraction over K + cap*RP.  A cluster owns one strip of output columns; its S CTA pairs
//                    (cta_group::2, 256 rows) each take a slice of the contraction and the partial accumulators are
//                    summed through distributed shared memory, again in a fixed order.  Launched as a programmatic
//                    dependent of the shrink: it streams W while the shrink runs and waits for hd only before the
//                    expand k-blocks.
#include "sm100_ptx.cuh"
#include "sm100_cluster.cuh"

namespace marlaas {
namespace sm100 {

// ---------------------------------------------------------------------------------------------------------------
// k_decode_shrink
// ---------------------------------------------------------------------------------------------------------------
constexpr int DS_THREADS = 128;
constexpr int DS_MAX_T = 1024;         // tokens per call
constexpr int DS_ROUNDS = DS_MAX_T / DS_THREADS;
constexpr int DS_PASS = 16;            // tokens per pass (one m16 MMA tile)
constexpr int DS_MAX_CS = 8;
constexpr int DS_TABLE_SMEM = 1032;    // the segment table is staged in shared memory when S + 1 <= this
constexpr int DS_UB = 4;               // 32-deep k-blocks whose loads are in flight together per warp

struct DecodeShrinkArgs {
    int T, K, RP, cap;
    int S;                              // segments; < 0: tok_slot already holds the per-token slots
    int G;                              // clusters per tenant: cluster (t, i) takes the 16-token passes i, i + G, ...
    const int32_t* seg_offsets;
    const int32_t* seg_slot;
    const bf16* x;
    int64_t ldx;
    const bf16* At;                     // [cap*RP][K]
    const int32_t* d_rank;
    const float* d_scale;
    int32_t* tok_slot;                  // [T]
    float* h_out;                       // [T][RP]
    bf16* hd;                           // [T][hd_cols]
    int hd_cols;
    int32_t* status;
};

// Shared memory: the fixed part below, then (dynamic, sized by the launch) slot[T'], off_tab[max(S + 1, T')] whose
// space the cluster's token list takes over once every token has its slot, and slot_tab[S]; T' = T rounded up to 32.
// Keeping this small matters: two of these CTAs share an SM with a GEMM CTA, whose pipeline gets what is left.
struct __align__(16) DecodeShrinkSmem {
    float wpart[4][256];                // per-warp [16 tokens][16 ranks] partial products
    float part[DS_MAX_CS][256];         // per-CTA partials, gathered in cluster rank 0
    int32_t cnt[DS_ROUNDS * 4];
};
static size_t decode_shrink_dyn_smem(int64_t T, int32_t S) {
    const size_t Tp = (size_t)((T + 31) / 32 * 32);
    const bool staged = S >= 0 && S + 1 <= DS_TABLE_SMEM;
    return 4 * (Tp + std::max<size_t>(staged ? (size_t)S + 1 : 0, Tp) + (staged ? (size_t)S : 0));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// grid = (cap + 1) clusters of CS CTAs; cluster t < cap serves tenant slot t, cluster cap the tokens routed to no
// adapter (slot -1, or a slot outside the pool, which is reported).  The cluster's CTAs (and their warps) split K.
//
// Operand fragments of the m16n8k16 MMA come straight from global memory with 16-byte loads: within a 32-deep
// k-block lane (g, t) reads elements 8t .. 8t+7 of its rows, and the same element-to-position permutation is used
// for the token rows (A fragment) and the adapter rows (B fragment), so every product pairs matching k.
__global__ void __launch_bounds__(DS_THREADS, 4) k_decode_shrink(const DecodeShrinkArgs g) {
    __shared__ DecodeShrinkSmem sm;
    extern __shared__ int32_t ds_dyn[];
    const int Tp = (g.T + 31) / 32 * 32;
    const bool staged_tab = g.S >= 0 && g.S + 1 <= DS_TABLE_SMEM;
    int32_t* const s_slot = ds_dyn;
    int32_t* const s_off = ds_dyn + Tp;             // the segment offsets, later the token list
    int32_t* const s_list = s_off;
    int32_t* const s_stab = s_off + max(staged_tab ? g.S + 1 : 0, Tp);
    dk_launch_dependents();      // the GEMM may start streaming W now; it waits for this grid before the expand
    // blockIdx.y = the projection of a pool that holds several: its block of A rows, its plane of h and of hd
    const bf16* const At = g.At + (size_t)blockIdx.y * g.cap * g.RP * g.K;
    float* const h_out = g.h_out + (size_t)blockIdx.y * g.T * g.RP;
    bf16* const hd = g.hd + (size_t)blockIdx.y * g.T * g.hd_cols;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int crank = (int)dk_cluster_ctarank();
    int cs;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(cs));
    const int t = (int)dk_cluster_id_x() / g.G;     // tenant slot served by this cluster; == cap: no adapter
    const int gi = (int)dk_cluster_id_x() % g.G;    // which of the tenant's 16-token passes
    const bool first = (dk_cluster_id_x() == 0 && crank == 0 && blockIdx.y == 0);      // one CTA also publishes tok_slot and checks the table
    const int r_t = t < g.cap ? g.d_rank[t] : 0;
    const float sc = t < g.cap ? g.d_scale[t] : 0.f;

    // This warp's share of K: the cluster's CTAs split the 32-deep k-blocks, then each CTA's warps do.  The adapter rows
    // of the tenant's first rank group do not depend on the token list, and a load issued beside the GEMM's stream takes
    // microseconds to come back: they are requested before anything else.
    const int nb32 = (g.K + 31) >> 5;
    const int cb0 = crank * nb32 / cs, cb1 = (crank + 1) * nb32 / cs;        // (32-bit: 64-bit division is slow, and these
    const int wb0 = cb0 + warp * (cb1 - cb0) / 4, wb1 = cb0 + (warp + 1) * (cb1 - cb0) / 4;   // precede the first loads)
    const int gq = lane >> 2, tq = lane & 3;
    uint4 ba[DS_UB], bb[DS_UB];     // adapter fragments; held_jg / held_b0 say of which rank group and k-block batch
    int held_jg = 0, held_b0 = wb0;
    {
        const bf16* ar0 = At + ((size_t)(t < g.cap ? t : 0) * g.RP + gq) * g.K;
        const bf16* ar1 = ar0 + (size_t)8 * g.K;
#pragma unroll
        for (int u = 0; u < DS_UB; ++u) {
            const int k = (wb0 + u) * 32 + tq * 8;
            const bool in = t < g.cap && (wb0 + u) < wb1 && k < g.K;
            ba[u] = in ? ldg_nc_v4(ar0 + k) : make_uint4(0u, 0u, 0u, 0u);
            bb[u] = in ? ldg_nc_v4(ar1 + k) : make_uint4(0u, 0u, 0u, 0u);
        }
    }

    // ---- per-token slot ------------------------------------------------------------------------------------
    if (g.S >= 0) {
        const bool staged = staged_tab;
        if (staged) {
            for (int s = tid; s <= g.S; s += DS_THREADS) {
                s_off[s] = g.seg_offsets[s];
                if (s < g.S) s_stab[s] = g.seg_slot[s];
            }
            __syncthreads();
        }
        if (first) {
            for (int s = tid; s < g.S; s += DS_THREADS) {
                const int a = staged ? s_off[s] : g.seg_offsets[s], b = staged ? s_off[s + 1] : g.seg_offsets[s + 1];
                if (b < a || a < 0 || b > g.T) dk_report(g.status, DEV_BAD_TABLE, s);
                if (s == 0 && a != 0) dk_report(g.status, DEV_BAD_TABLE, -1);
                if (s == g.S - 1 && b != g.T) dk_report(g.status, DEV_BAD_TABLE, -2);
            }
            if (tid == 0 && g.S == 0 && g.T != 0) dk_report(g.status, DEV_BAD_TABLE, -3);
        }
        for (int i = tid; i < g.T; i += DS_THREADS) {
            int lo = 0, hi = g.S;
            while (lo < hi) {       // first s with seg_offsets[s + 1] > i
                const int mid = (lo + hi) >> 1;
                const int v = staged ? s_off[mid + 1] : g.seg_offsets[mid + 1];
                if (v > i) hi = mid; else lo = mid + 1;
            }
            s_slot[i] = lo < g.S ? (staged ? s_stab[lo] : g.seg_slot[lo]) : -1;
        }
    } else {
        for (int i = tid; i < g.T; i += DS_THREADS) s_slot[i] = g.tok_slot[i];
    }
    __syncthreads();
    if (first)
        for (int i = tid; i < g.T; i += DS_THREADS) {
            int s = s_slot[i];
            if (s < -1 || s >= g.cap) {
                dk_report(g.status, DEV_BAD_INDEX, i);
                s = -1;
            }
            g.tok_slot[i] = s;
        }

    // ---- this cluster's tokens, ascending --------------------------------------------------------------------
    unsigned bal[DS_ROUNDS];
    bool mine[DS_ROUNDS];
#pragma unroll
    for (int r = 0; r < DS_ROUNDS; ++r) {
        const int i = r * DS_THREADS + tid;
        bool m = false;
        if (i < g.T) {
            const int s = s_slot[i];
            m = (t < g.cap) ? (s == t) : (s < 0 || s >= g.cap);
        }
        mine[r] = m;
        bal[r] = __ballot_sync(0xffffffffu, m);
        if (lane == 0) sm.cnt[r * 4 + warp] = __popc(bal[r]);
    }
    __syncthreads();
    int n_t = 0;
#pragma unroll
    for (int e = 0; e < DS_ROUNDS * 4; ++e) n_t += sm.cnt[e];
#pragma unroll
    for (int r = 0; r < DS_ROUNDS; ++r) {
        if (mine[r]) {
            int off = __popc(bal[r] & ((1u << lane) - 1u));
            for (int e = 0; e < r * 4 + warp; ++e) off += sm.cnt[e];
            s_list[off] = r * DS_THREADS + tid;
        }
    }
    __syncthreads();
    if (gi * DS_PASS >= n_t) {           // nothing for this cluster (uniform over it)
        if (threadIdx.x == 0) dk_wait_prerequisites();
        return;
    }

    const int own0 = r_t > 0 ? t * g.RP : 0, own1 = r_t > 0 ? own0 + g.RP : 0;   // hd columns written by the MMA part
    const int ngroups = (r_t + 15) >> 4;

    // ---- partial products over this warp's share of K --------------------------------------------------------
    const uint32_t part_rank0 = dk_map_to_cta(smem_u32(&sm.part[0][0]), 0);

    // zero the other tenants' columns of this cluster's hd rows (and, with no adapter, the h rows): one warp per row
    for (int e = crank * 4 + warp; e < n_t; e += cs * 4) {
        if ((e / DS_PASS) % g.G != gi) continue;     // another cluster's pass
        const int tok = s_list[e];
        bf16* row = hd + (size_t)tok * g.hd_cols;
        for (int c = lane * 8; c < g.hd_cols; c += 256)
            if (c < own0 || c >= own1) *reinterpret_cast<uint4*>(row + c) = make_uint4(0u, 0u, 0u, 0u);
        if (r_t == 0)
            for (int j = lane; j < g.RP; j += 32) h_out[(size_t)tok * g.RP + j] = 0.f;
    }
    if (r_t == 0) {              // uniform over the cluster
        if (threadIdx.x == 0) dk_wait_prerequisites();
        return;
    }

    for (int p0 = gi * DS_PASS; p0 < n_t; p0 += DS_PASS * g.G) {
        const int np = min(DS_PASS, n_t - p0);
        const bf16* xr0 = gq < np ? g.x + (size_t)s_list[p0 + gq] * g.ldx : nullptr;
        const bf16* xr1 = gq + 8 < np ? g.x + (size_t)s_list[p0 + gq + 8] * g.ldx : nullptr;
        for (int jg = 0; jg < ngroups; ++jg) {
            float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
            const bf16* ar0 = At + ((size_t)t * g.RP + jg * 16 + gq) * g.K;
            const bf16* ar1 = ar0 + (size_t)8 * g.K;
            for (int b0 = wb0; b0 < wb1; b0 += DS_UB) {
                uint4 xa[DS_UB], xb[DS_UB];
                const bool held = held_jg == jg && held_b0 == b0;     // the adapter fragments are in registers already
#pragma unroll
                for (int u = 0; u < DS_UB; ++u) {
                    const int k = (b0 + u) * 32 + tq * 8;
                    const bool in = (b0 + u) < wb1 && k < g.K;
                    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                    xa[u] = (in && xr0) ? ldg_nc_v4(xr0 + k) : z;
                    xb[u] = (in && xr1) ? ldg_nc_v4(xr1 + k) : z;
                    if (!held) {
                        ba[u] = in ? ldg_nc_v4(ar0 + k) : z;
                        bb[u] = in ? ldg_nc_v4(ar1 + k) : z;
                    }
                }
                held_jg = jg;
                held_b0 = b0;
#pragma unroll
                for (int u = 0; u < DS_UB; ++u) {
                    mma_bf16_16816(c0, xa[u].x, xb[u].x, xa[u].y, xb[u].y, ba[u].x, ba[u].y);
                    mma_bf16_16816(c1, xa[u].x, xb[u].x, xa[u].y, xb[u].y, bb[u].x, bb[u].y);
                    mma_bf16_16816(c0, xa[u].z, xb[u].z, xa[u].w, xb[u].w, ba[u].z, ba[u].w);
                    mma_bf16_16816(c1, xa[u].z, xb[u].z, xa[u].w, xb[u].w, bb[u].z, bb[u].w);
                }
            }
            // warp partials -> CTA partial (fixed order) -> cluster rank 0
            const bool first_round = p0 == gi * DS_PASS && jg == 0;
            const bool last_round = p0 + DS_PASS * g.G >= n_t && jg == ngroups - 1;
            if (!first_round) __syncthreads();      // wpart of the previous group has been consumed
            {
                float* wp = sm.wpart[warp];
                wp[gq * 16 + 2 * tq] = c0[0];
                wp[gq * 16 + 2 * tq + 1] = c0[1];
                wp[(gq + 8) * 16 + 2 * tq] = c0[2];
                wp[(gq + 8) * 16 + 2 * tq + 1] = c0[3];
                wp[gq * 16 + 8 + 2 * tq] = c1[0];
                wp[gq * 16 + 8 + 2 * tq + 1] = c1[1];
                wp[(gq + 8) * 16 + 8 + 2 * tq] = c1[2];
                wp[(gq + 8) * 16 + 8 + 2 * tq + 1] = c1[3];
            }
            __syncthreads();
            for (int e = tid; e < 256; e += DS_THREADS) {
                const float v = ((sm.wpart[0][e] + sm.wpart[1][e]) + sm.wpart[2][e]) + sm.wpart[3][e];
                dk_st_cluster_f32(part_rank0 + (uint32_t)(crank * 256 + e) * 4, v);
            }
            dk_cluster_sync();
            if (crank == 0) {
                for (int e = tid; e < 256; e += DS_THREADS) {
                    const int i = e >> 4, j = e & 15;
                    if (i < np) {
                        float v = 0.f;
                        for (int s = 0; s < cs; ++s) v += sm.part[s][e];   // fixed order
                        const int tok = s_list[p0 + i];
                        h_out[(size_t)tok * g.RP + jg * 16 + j] = v;
                        hd[(size_t)tok * g.hd_cols + own0 + jg * 16 + j] = __float2bfloat16_rn(sc * v);
                    }
                }
            }
            if (!last_round) dk_cluster_sync();     // rank 0 has read the partials before they are overwritten (its own
                                                    // shared memory: after the last round the other CTAs may leave)
        }
        // ranks beyond the tenant's true rank (rounded up to 16) stay zero
        if (crank == 0) {
            const int rest = g.RP - ngroups * 16;
            for (int e = tid; e < np * rest; e += DS_THREADS) {
                const int i = e / rest, j = ngroups * 16 + e % rest;
                const int tok = s_list[p0 + i];
                h_out[(size_t)tok * g.RP + j] = 0.f;
                hd[(size_t)tok * g.hd_cols + own0 + j] = __float2bfloat16_rn(0.f);
            }
        }
    }
    // With MARLAAS_FLAG_OVERLAP_PREVIOUS this grid was launched behind the previous call's GEMM without waiting for it:
    // it must not complete first (what follows in the stream relies on stream order).  A no-op otherwise.
    if (threadIdx.x == 0) dk_wait_prerequisites();
}

// ---------------------------------------------------------------------------------------------------------------
// k_decode_gemm
// ---------------------------------------------------------------------------------------------------------------
constexpr int DG_THREADS = 192;
constexpr int DG_KP = 2;               // 64-deep panels per pipeline step

struct DecodeGemmArgs {
    int T, Nout;
    int nstrips;         // column strips; cluster c works on strip c mod nstrips of 256-row tile c / nstrips
    int num_ks;          // pipeline steps (kp * 64 deep) over K
    int num_xs;          // pipeline steps over the expand rows (cap*RP, or up to the last slot in use)
    int S;               // contraction slices = CTA pairs per cluster
    int nch;             // 64-column chunks of the B operand staged per CTA: the pair's strip is 128 * nch columns
    int kp;              // 64-deep panels per pipeline step: one TMA instruction per operand moves all of them
    int stages;
    int parts;           // projections held by the pool: hd is [parts][T][..] and strip n0 takes the plane of its projection
    int part_end[4];     // last column + 1 of each projection
    bf16* C;
    int64_t ldc;
    int32_t* status;
};

// Operand staging per pipeline step (kp panels of 64 k):
//   A  [kp][128 rows][64 k]      one 3-D TMA over x viewed as (64 k, rows, K / 64): K-major tiles, 128-byte swizzle
//   B  [nch][kp * 64 k][64 n]    one 2-D TMA per 64-column chunk: MN-major, chunks kp * 8 KB apart
// A single thread issues the loads and a single thread the MMAs, and each of their instructions costs tens to a
// hundred cycles of issue latency, so the steps are made deep: with 64-deep steps the issue loop, not HBM, set the pace.
__global__ void __launch_bounds__(DG_THREADS, 1)
k_decode_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmXA, const __grid_constant__ CUtensorMap tmXB, const DecodeGemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int STAGES = g.stages;
    const uint32_t a_stage_bytes = (uint32_t)g.kp * A_STAGE_BYTES;
    const uint32_t b_chunk_bytes = (uint32_t)g.kp * CHUNK_BYTES;
    const uint32_t b_stage_bytes = (uint32_t)g.nch * b_chunk_bytes;
    const uint32_t sA = smem_u32(smem);
    const uint32_t sB = sA + STAGES * a_stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (a_stage_bytes + b_stage_bytes));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_drain = bar_tfull + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NP = 128 * g.nch;                 // columns of the cluster's strip
    const uint32_t tmem_cols = (uint32_t)NP;    // 128 or 256
    // set-up first (one thread the barriers, one the descriptor prefetches, one warp the tensor-memory allocation): the
    // index arithmetic below holds a dozen integer divisions, a microsecond if it came before
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_drain, 1);
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x == 64) {
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (g.num_xs > 0) {
            prefetch_tmap(&tmXA);
            prefetch_tmap(&tmXB);
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    const uint32_t crank = dk_cluster_ctarank();
    const uint32_t half = crank & 1;            // which 128 rows of the 256-row tile
    const uint32_t pairi = crank >> 1;          // which slice of the contraction
    const uint32_t leader = crank & ~1u;
    const int n0 = ((int)dk_cluster_id_x() % g.nstrips) * NP;
    const int m0 = ((int)dk_cluster_id_x() / g.nstrips) * 256;      // first row of the cluster's token tile
    const int my_m = m0 + (int)half * 128, my_n = n0 + (int)half * 64 * g.nch;
    // the projection whose columns the strip lies in (constant indices: a variable one would move the arguments to local memory)
    const int part = (g.parts > 1 ? (int)(n0 >= g.part_end[0]) + (int)(g.parts > 2 && n0 >= g.part_end[1]) + (int)(g.parts > 3 && n0 >= g.part_end[2]) : 0);
    const int xa_m = my_m + part * g.T;         // this half's rows of the projection's plane of hd

    const int ks0 = (int)pairi * g.num_ks / g.S, ks1 = ((int)pairi + 1) * g.num_ks / g.S;
    const int xs0 = (int)pairi * g.num_xs / g.S, xs1 = ((int)pairi + 1) * g.num_xs / g.S;

    const int qper = 4 / g.S;
    // bit p set: slice p has at least one step (computed once: integer division is slow in these short loops)
    uint32_t live = 0;
    for (int p = 0; p < g.S; ++p) {
        const int n = ((p + 1) * g.num_ks / g.S - p * g.num_ks / g.S) + ((p + 1) * g.num_xs / g.S - p * g.num_xs / g.S);
        if (n > 0) live |= 1u << p;
    }
    const uint32_t box_bytes = (uint32_t)NP * 4u * 32u;      // one quarter from one pair
    tc_fence_before();
    dk_cluster_sync();      // every CTA's barriers exist before any remote arrive or TMA completion
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // bytes the two CTAs of the pair stage per step (rows and columns outside the tensors are skipped entirely;
    // partly outside boxes are filled with zeros and count in full)
    auto a_bytes = [&](int r) -> uint32_t { return (m0 + r * 128 < g.T) ? a_stage_bytes : 0u; };
    auto b_chunks = [&](int r) -> int { return max(0, min(g.nch, (g.Nout - (n0 + r * 64 * g.nch) + 63) / 64)); };
    const uint32_t stage_tx = a_bytes(0) + a_bytes(1) + (uint32_t)(b_chunks(0) + b_chunks(1)) * b_chunk_bytes;
    const int my_chunks = b_chunks((int)half);
    const bool have_rows = my_m < g.T;

    bool epi_ok = true;
    if (warp == 0) {
        // ================= TMA producer (every CTA) =================
        if (lane == 0) {
            uint32_t it = 0, s = 0, ph = 0;     // steps issued; stage and phase bit of the next step
            bool ok = true;
            const uint32_t full0 = dk_map_to_cta(bar_full, leader);
            for (int ks = ks0; ks < ks1 && ok; ++ks, ++it) {
                if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 41))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                if (have_rows) dg_tma_pair_3d(sA + s * a_stage_bytes, &tmA, full0 + 8 * s, 0, my_m, ks * g.kp);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + s * b_stage_bytes + c * b_chunk_bytes, &tmB, full0 + 8 * s, my_n + c * 64, ks * g.kp * BK);
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
            // the expand's adapter rows Bs do not depend on the shrink grid: the first steps' B operands are fetched
            // before the wait for it, their hd tiles after
            const int npre = (xs1 - xs0) < STAGES ? (xs1 - xs0) : STAGES;
            {
                uint32_t b_s = s, b_ph = ph;
                for (int i = 0; i < npre && ok; ++i) {
                    if (!(ok = mbar_wait(bar_empty + 8 * b_s, b_ph ^ 1, abort_word, 42))) break;
                    if (half == 0) mbar_expect_tx(bar_full + 8 * b_s, stage_tx);
                    for (int c = 0; c < my_chunks; ++c)
                        dg_tma_pair(sB + b_s * b_stage_bytes + c * b_chunk_bytes, &tmXB, full0 + 8 * b_s, my_n + c * 64,
                                    (xs0 + i) * g.kp * BK);
                    if (++b_s == (uint32_t)STAGES) { b_s = 0; b_ph ^= 1; }
                }
            }
            if (ok && xs0 < xs1) dk_wait_prerequisites();     // hd comes from the shrink grid
            for (int i = 0; i < npre && ok; ++i, ++it) {
                if (have_rows) dg_tma_pair_3d(sA + s * a_stage_bytes, &tmXA, full0 + 8 * s, 0, xa_m, (xs0 + i) * g.kp);
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
            for (int xs = xs0 + npre; xs < xs1 && ok; ++xs, ++it) {
                if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 42))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                if (have_rows) dg_tma_pair_3d(sA + s * a_stage_bytes, &tmXA, full0 + 8 * s, 0, xa_m, xs * g.kp);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + s * b_stage_bytes + c * b_chunk_bytes, &tmXB, full0 + 8 * s, my_n + c * 64, xs * g.kp * BK);
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
            if (!ok && half == 0) {
                // let the copies already issued land (bounded) before shared memory is reused or released
                const uint32_t back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                for (uint32_t j = 0; j < back; ++j) {
                    const uint32_t jt = it - 1 - j;
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * (jt % (uint32_t)STAGES), (jt / (uint32_t)STAGES) & 1) &&
                           global_ns() - t0 < WAIT_LIMIT_NS) {
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= MMA issuer (the pair's leader CTA) =================
        if (lane == 0 && half == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(NP >> 3) << 17) |
                                   ((uint32_t)(256 >> 4) << 24);    // fp32 acc, bf16 x bf16, B MN-major, M = 256, N = NP
            const uint16_t mask = (uint16_t)(3u << leader);
            uint32_t acc = 0, s = 0, ph = 0;
            bool ok = true;
            const int nstep = (ks1 - ks0) + (xs1 - xs0);
            for (int b = 0; b < nstep && ok; ++b) {
                if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 44))) break;
                tc_fence_after();
                const uint32_t a0 = sA + s * a_stage_bytes, b0 = sB + s * b_stage_bytes;
                for (int q = 0; q < g.kp; ++q) {
                    // descriptors of successive 16-deep slices differ only in the start-address field (16-byte units)
                    const uint64_t da0 = desc_k_major(a0 + q * A_STAGE_BYTES), db0 = desc_mn_major(b0 + q * CHUNK_BYTES, b_chunk_bytes);
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        dg_mma_pair(tmem_base, da0 + (uint64_t)(2 * j), db0 + (uint64_t)(j * (UNIT_BYTES >> 4)), idesc, acc);
                        acc = 1;
                    }
                }
                dg_commit_pair(bar_empty + 8 * s, mask);
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
            if (ok) {
                dg_commit_pair(bar_tfull, mask);
            } else {
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_drain)
                             : "memory");
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {
                }
            }
        }
        __syncwarp();
    } else {
        // ================= epilogue warps: wait for the pair's accumulator =================
        // Idle until then, one of them hands over to the next call: once the shrink grid has completed (and with it
        // whatever that grid was launched behind), a next call launched with MARLAAS_FLAG_OVERLAP_PREVIOUS may start its
        // shrink beside the rest of this kernel.  Every CTA does this, so the hand-over happens as early as it may.
        if (warp == 2 && lane == 0) {
            dk_wait_prerequisites();
            dk_launch_dependents();
        }
        __syncwarp();
        epi_ok = mbar_wait(bar_tfull, 0, abort_word, 46);
        epi_ok = __all_sync(0xffffffffu, epi_ok);
        tc_fence_after();
    }

    // ---- sum the S slices through distributed shared memory ---------------------------------------------------
    // Row quarter q (32 rows) of each half is finished by pair (q mod S).  The other pairs' warps holding that
    // quarter send their partial accumulators to a mailbox in the finishing CTA (thread to thread: the same
    // tensor-memory lane on both sides, [column group][lane] 16-byte slots), and the finishing warp adds them to
    // its own accumulator in ascending pair order.  The mailboxes reuse the pipeline stages.
    const int q = warp & 3;
    const uint32_t own = (uint32_t)(q % g.S);
    if (g.S > 1) {
        tc_fence_before();
        dk_cluster_sync();      // every pair's MMAs are complete: the pipeline stages may be overwritten
        tc_fence_after();
        if (warp >= 2 && epi_ok && own != pairi && ((live >> pairi) & 1u)) {
            const uint32_t si = pairi < own ? pairi : pairi - 1;
            const uint32_t dst = dk_map_to_cta(sA, 2 * own + half) + (si * (uint32_t)qper + (uint32_t)(q / g.S)) * box_bytes +
                                 (uint32_t)lane * 16u;
#pragma unroll 1
            for (int c = 0; c < NP / 32; ++c) {
                uint32_t v[32];
                tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, v);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    dk_st_cluster_v4(dst + (uint32_t)(c * 8 + e) * 512u, v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
            }
        }
        tc_fence_before();
        dk_cluster_sync();      // all partial accumulators have landed
        tc_fence_after();
    }
    if (warp >= 2 && epi_ok && own == pairi) {
        const int row = my_m + q * 32 + lane;
        bf16* crow = g.C + (size_t)row * g.ldc + n0;
        const uint32_t mbox = sA + (uint32_t)(q / g.S) * box_bytes + (uint32_t)lane * 16u;
#pragma unroll 1
        for (int c = 0; c < NP / 32; ++c) {
            uint32_t v[32];
            tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, v);
            tc_wait_ld();
            float acc[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] = 0.f;
            for (uint32_t src = 0; src < (uint32_t)g.S; ++src) {      // ascending pair order
                if (!((live >> src) & 1u)) continue;                  // a slice without steps never wrote its accumulator
                if (src == pairi) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) acc[e] += __uint_as_float(v[e]);
                } else {
                    const uint32_t si = src < pairi ? src : src - 1;
                    const uint32_t a = mbox + si * (uint32_t)qper * box_bytes + (uint32_t)(c * 8) * 512u;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float4 p;
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(p.x), "=f"(p.y), "=f"(p.z), "=f"(p.w)
                                     : "r"(a + (uint32_t)e * 512u));
                        acc[4 * e] += p.x; acc[4 * e + 1] += p.y; acc[4 * e + 2] += p.z; acc[4 * e + 3] += p.w;
                    }
                }
            }
            if (row < g.T) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = n0 + c * 32 + e * 8;
                    if (col < g.Nout) {
                        uint4 o;
                        __nv_bfloat162 p0 = __floats2bfloat162_rn(acc[e * 8 + 0], acc[e * 8 + 1]);
                        __nv_bfloat162 p1 = __floats2bfloat162_rn(acc[e * 8 + 2], acc[e * 8 + 3]);
                        __nv_bfloat162 p2 = __floats2bfloat162_rn(acc[e * 8 + 4], acc[e * 8 + 5]);
                        __nv_bfloat162 p3 = __floats2bfloat162_rn(acc[e * 8 + 6], acc[e * 8 + 7]);
                        o.x = *reinterpret_cast<uint32_t*>(&p0);
                        o.y = *reinterpret_cast<uint32_t*>(&p1);
                        o.z = *reinterpret_cast<uint32_t*>(&p2);
                        o.w = *reinterpret_cast<uint32_t*>(&p3);
                        *reinterpret_cast<uint4*>(crow + c * 32 + e * 8) = o;
                    }
                }
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    tc_fence_before();
    dk_cluster_sync();      // the pair leaves together (its barriers and tensor memory are shared)
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (threadIdx.x == 0) dk_wait_prerequisites();   // this grid never completes before the shrink grid it depends on
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
}

// x (or hd) viewed as a 3-D tensor (64 k, rows, K / 64) so that one copy brings `panels` K-major tiles of box_rows rows
marlaas_status_t make_panel_map(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int64_t ld, uint32_t panels,
                                uint32_t box_rows) {
    typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            return fail(MARLAAS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        fn = (EncodeTiledFn)p;
    }
    cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
    cuuint64_t gstr[2] = {(cuuint64_t)ld * 2, 128};
    cuuint32_t box[3] = {64, box_rows, panels};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(MARLAAS_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) for a %lld x %lld panel view, pitch %lld", (int)r,
                    (long long)rows, (long long)cols, (long long)ld);
    return MARLAAS_OK;
}

}  // namespace sm100

// ---------------------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------------------
bool decode_sm100_eligible(const marlaas_pool* pool, int64_t T) {
    if (!(T > 0 && T <= sm100::DS_MAX_T && (int64_t)pool->cap * pool->RP <= 2048 && pool->sm_count >= 8 && (pool->K % 64) == 0))
        return false;
    // beyond one 256-token tile only while all (token tile, 256-column strip) pairs make a single wave of CTA pairs
    return T <= 256 || cdiv(T, 256) * cdiv(pool->N, 256) <= pool->sm_count / 2;
}

// Shared memory one shrink CTA holds (static + dynamic + the system's 1 KB): a GEMM that wants shrink CTAs beside it on
// its SMs leaves room for two of them.
size_t decode_shrink_smem_bytes(int64_t T, int32_t S) { return sizeof(sm100::DecodeShrinkSmem) + sm100::decode_shrink_dyn_smem(T, S) + 1024; }

// The shrink kernel alone: (cap + 1) * G clusters, K split over the CTAs of a cluster.  Writes tok_slot, h and hd; its
// CTAs are small (four per SM), so they fit on whatever SMs a GEMM launched as its programmatic dependent leaves free.
marlaas_status_t launch_decode_shrink(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, int32_t S,
                                      const int32_t* seg_offsets, const int32_t* seg_slot, const Workspace& ws, float* h_out,
                                      cudaStream_t st) {
    using namespace sm100;
    const int64_t K = pool->K;
    const int hd_cols = (int)align_up((size_t)pool->cap * pool->RP, 64);     // pitch of hd: whole 64-deep panels
    DecodeShrinkArgs a;
    a.T = (int)T; a.K = (int)K; a.RP = pool->RP; a.cap = pool->cap;
    a.S = S; a.seg_offsets = seg_offsets; a.seg_slot = seg_slot;
    a.x = x; a.ldx = ldx; a.At = pool->d_At; a.d_rank = pool->d_rank; a.d_scale = pool->d_scale;
    a.tok_slot = ws.tok_slot; a.h_out = h_out; a.hd = ws.hd; a.hd_cols = hd_cols; a.status = pool->d_status;
    int cs = DS_MAX_CS;
    while (cs > 1 && K / cs < 32 * 4 * DS_UB) cs >>= 1;      // a full batch of loads per warp
    // with few tenants a tenant has many 16-token passes: several clusters share them, as many as keep the grid
    // within two CTAs per SM
    const int passes = (int)cdiv(T, DS_PASS);
    a.G = std::max(1, std::min(passes, (2 * pool->sm_count) / ((pool->cap + 1) * cs * pool->P)));
    static bool carveout_set[64] = {};
    if (pool->device >= 64 || !carveout_set[pool->device]) {
        // same shared-memory configuration as the GEMM, so that CTAs of both kernels can share an SM
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_shrink, cudaFuncAttributePreferredSharedMemoryCarveout,
                                              (int)cudaSharedmemCarveoutMaxShared));
        if (pool->device < 64) carveout_set[pool->device] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((pool->cap + 1) * a.G * cs), (unsigned)pool->P);     // y: the pool's projections
    cfg.blockDim = dim3(DS_THREADS);
    cfg.dynamicSmemBytes = decode_shrink_dyn_smem(T, S);
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    // the caller has stated that the previous call on the stream is independent of this one: the shrink starts once that
    // call's GEMM has let its dependents go (after its own shrink has completed) and runs beside it
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = ws.early_shrink ? 2 : 1;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_shrink, a));
    count_launch();
    return MARLAAS_OK;
}

marlaas_status_t launch_decode_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                     int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                     const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st) {
    using namespace sm100;
    const int64_t K = pool->K, N = pool->N;
    const int hd_cols = (int)align_up((size_t)pool->cap * pool->RP, 64);     // pitch of hd: whole 64-deep panels

    {
        marlaas_status_t rcs = launch_decode_shrink(pool, T, x, ldx, S, seg_offsets, seg_slot, ws, h_out, st);
        if (rcs != MARLAAS_OK) return rcs;
    }

    // ---- GEMM with the expand as extra steps of the contraction ----
    int last_used = -1;
    for (int s = 0; s < pool->cap; ++s)
        if (pool->slots[s].used && pool->slots[s].rank > 0) last_used = s;
    DecodeGemmArgs g;
    g.T = (int)T; g.Nout = (int)N;
    g.C = y; g.ldc = ldy; g.status = pool->d_status;
    g.parts = pool->P;
    for (int p = 0; p < 4; ++p) g.part_end[p] = p < pool->P ? (int)pool->part_begin[p + 1] : 0;
    // strip width and contraction slices: fill the SMs with one wave of clusters of 2 * S CTAs
    struct Shape { int nch, S; };
    const Shape shapes[] = {{1, 2}, {2, 2}, {1, 1}, {2, 1}, {1, 4}, {2, 4}};
    Shape pick = {2, 1};
    int64_t best = -1;
    const int64_t mtiles = cdiv(T, 256);
    static int max_clusters[64][3] = {};      // per device, cluster size 2 / 4 / 8
    constexpr int DG_SMEM = 200 * 1024;
    for (const Shape& sh : shapes) {
        const int csz = 2 * sh.S;
        const int ci = sh.S == 1 ? 0 : sh.S == 2 ? 1 : 2;
        int mc = pool->device < 64 ? max_clusters[pool->device][ci] : 0;
        if (mc == 0) {
            MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            cudaLaunchConfig_t qc = {};
            qc.gridDim = dim3((unsigned)(csz * 64));
            qc.blockDim = dim3(DG_THREADS);
            qc.dynamicSmemBytes = DG_SMEM;
            cudaLaunchAttribute qa;
            qa.id = cudaLaunchAttributeClusterDimension;
            qa.val.clusterDim.x = (unsigned)csz; qa.val.clusterDim.y = 1; qa.val.clusterDim.z = 1;
            qc.attrs = &qa; qc.numAttrs = 1;
            MARLAAS_CUDA_TRY(cudaOccupancyMaxActiveClusters(&mc, k_decode_gemm, &qc));
            if (mc < 1) mc = -1;
            if (pool->device < 64) max_clusters[pool->device][ci] = mc;
        }
        if (mc < 1) continue;
        const int64_t clusters = cdiv(N, 128 * sh.nch) * mtiles;
        if (clusters > mc) continue;                    // one wave only
        if (cdiv(K, (int64_t)DG_KP * BK) < sh.S) continue;     // every slice needs at least one step
        const int64_t ctas = clusters * csz;
        // more CTAs streaming is better; among equals fewer slices (no exchange of partial sums: 512 tokens run 28 us
        // as 128-column strips without slices against 34 us as 256-column strips cut in two), then wider strips
        const int64_t score = ctas * 16 - sh.S * 4 + sh.nch;
        if (score > best) { best = score; pick = sh; }
    }
    g.S = pick.S; g.nch = pick.nch;
    g.kp = DG_KP;
    const size_t step_bytes = (size_t)g.kp * (A_STAGE_BYTES + g.nch * CHUNK_BYTES);
    // leave room for two shrink CTAs (their static and dynamic shared memory + 1 KB system reservation each) on the same
    // SM: the shrink then overlaps the GEMM's main loop instead of delaying its start (measured: 23 us per call against
    // 29 us); what is left of the SM's 227 KB goes to the pipeline (4 steps at 256 tokens, 3 at 1024)
    const size_t shrink_smem = sizeof(DecodeShrinkSmem) + decode_shrink_dyn_smem(T, S) + 1024;
    g.stages = (int)std::min<size_t>(6, ((size_t)227 * 1024 - 2 * shrink_smem - 1024 - 256 - 1024) / step_bytes);
    if (g.stages < 2) g.stages = 2;
    g.num_ks = (int)cdiv(K, (int64_t)g.kp * BK);
    g.num_xs = (int)cdiv((int64_t)(last_used + 1) * pool->RP, (int64_t)g.kp * BK);
    const int NP = 128 * g.nch;

    alignas(64) CUtensorMap tmA, tmB, tmXA, tmXB;
    marlaas_status_t rc;
    if ((rc = make_panel_map(&tmA, x, T, K, ldx, (uint32_t)g.kp)) != MARLAAS_OK) return rc;
    if ((rc = make_map(&tmB, W, K, N, ldw, 64, (uint32_t)(g.kp * BK))) != MARLAAS_OK) return rc;
    if (g.num_xs > 0) {
        if ((rc = make_panel_map(&tmXA, ws.hd, T * pool->P, hd_cols, hd_cols, (uint32_t)g.kp)) != MARLAAS_OK) return rc;
        if ((rc = make_map(&tmXB, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, pool->ldB, 64, (uint32_t)(g.kp * BK))) != MARLAAS_OK) return rc;
    } else {
        tmXA = tmA;
        tmXB = tmB;
    }
    const size_t smem_bytes = 1024 + (size_t)g.stages * step_bytes + 256;
    cudaLaunchConfig_t cfg = {};
    g.nstrips = (int)cdiv(N, NP);
    cfg.gridDim = dim3((unsigned)(g.nstrips * mtiles * 2 * g.S));
    cfg.blockDim = dim3(DG_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)(2 * g.S); at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_gemm, tmA, tmB, tmXA, tmXB, g));
    count_launch();
    return MARLAAS_OK;
}

}  // namespace marlaas
