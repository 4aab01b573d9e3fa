// Decode-shaped forward (at most 256 tokens, one per sequence, tenants unsorted): the call is bound by the one pass
// over W from HBM, so the work is cut to keep every SM streaming and the launch count to two overlapping kernels.
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

namespace marlaas {
namespace sm100 {

// ---------------------------------------------------------------------------------------------------------------
// shared helpers
// ---------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t dk_cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t dk_cluster_id_x() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t dk_map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void dk_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void dk_st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void dk_st_cluster_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void dk_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void dk_wait_prerequisites() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void dk_report(int32_t* status, int code, int detail) {
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// ---------------------------------------------------------------------------------------------------------------
// k_decode_shrink
// ---------------------------------------------------------------------------------------------------------------
constexpr int DS_THREADS = 128;
constexpr int DS_MAX_T = 256;          // tokens per call
constexpr int DS_PASS = 16;            // tokens per pass (one m16 MMA tile)
constexpr int DS_SUB_OCT = 64;         // 16-byte octets (8 bf16) of K per staged sub-chunk: 512 elements
constexpr int DS_PITCH = (DS_SUB_OCT + 1) * 16;   // bytes per staged row (padded: conflict-free ldmatrix)
constexpr int DS_MAX_CS = 8;
constexpr int DS_TABLE_SMEM = 1024;    // segment offsets staged in shared memory when S + 1 <= this

struct DecodeShrinkArgs {
    int T, K, RP, cap;
    int S;                              // segments; < 0: tok_slot already holds the per-token slots
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

struct __align__(16) DecodeShrinkSmem {
    uint8_t sx[DS_PASS * DS_PITCH];
    uint8_t sa[16 * DS_PITCH];
    float part[DS_MAX_CS * 4 * 256];    // [cluster rank][warp][16 tokens x 16 ranks] (used in cluster rank 0)
    int32_t slot[DS_MAX_T];
    int32_t list[DS_MAX_T];
    int32_t table[DS_TABLE_SMEM];
    int32_t cnt[8];
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// grid = (cap + 1) clusters of CS CTAs; cluster t < cap serves tenant slot t, cluster cap the tokens routed to no
// adapter (slot -1, or a slot outside the pool, which is reported).
__global__ void __launch_bounds__(DS_THREADS) k_decode_shrink(const DecodeShrinkArgs g) {
    extern __shared__ uint8_t ds_raw[];
    DecodeShrinkSmem& sm = *reinterpret_cast<DecodeShrinkSmem*>((reinterpret_cast<uintptr_t>(ds_raw) + 15) & ~uintptr_t(15));
    dk_launch_dependents();      // the GEMM may start streaming W now; it waits for this grid before the expand

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int crank = (int)dk_cluster_ctarank();
    int cs;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(cs));
    const int t = (int)dk_cluster_id_x();           // tenant slot served by this cluster; == cap: no adapter
    const bool first = (t == 0 && crank == 0);      // one CTA also publishes tok_slot and checks the table

    // ---- per-token slot ------------------------------------------------------------------------------------
    if (g.S >= 0) {
        const bool staged = g.S + 1 <= DS_TABLE_SMEM;
        if (staged) {
            for (int s = tid; s <= g.S; s += DS_THREADS) sm.table[s] = g.seg_offsets[s];
            __syncthreads();
        }
        if (first) {
            for (int s = tid; s < g.S; s += DS_THREADS) {
                const int a = g.seg_offsets[s], b = g.seg_offsets[s + 1];
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
                const int v = staged ? sm.table[mid + 1] : g.seg_offsets[mid + 1];
                if (v > i) hi = mid; else lo = mid + 1;
            }
            sm.slot[i] = lo < g.S ? g.seg_slot[lo] : -1;
        }
    } else {
        for (int i = tid; i < g.T; i += DS_THREADS) sm.slot[i] = g.tok_slot[i];
    }
    __syncthreads();
    if (first)
        for (int i = tid; i < g.T; i += DS_THREADS) {
            int s = sm.slot[i];
            if (s < -1 || s >= g.cap) {
                dk_report(g.status, DEV_BAD_INDEX, i);
                s = -1;
            }
            g.tok_slot[i] = s;
        }

    // ---- this cluster's tokens, ascending --------------------------------------------------------------------
    unsigned bal[2];
    bool mine[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int i = r * DS_THREADS + tid;
        bool m = false;
        if (i < g.T) {
            const int s = sm.slot[i];
            m = (t < g.cap) ? (s == t) : (s < 0 || s >= g.cap);
        }
        mine[r] = m;
        bal[r] = __ballot_sync(0xffffffffu, m);
        if (lane == 0) sm.cnt[r * 4 + warp] = __popc(bal[r]);
    }
    __syncthreads();
    int n_t = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) n_t += sm.cnt[e];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        if (mine[r]) {
            int off = __popc(bal[r] & ((1u << lane) - 1u));
            for (int e = 0; e < r * 4 + warp; ++e) off += sm.cnt[e];
            sm.list[off] = r * DS_THREADS + tid;
        }
    }
    __syncthreads();
    if (n_t == 0) return;        // uniform over the cluster

    const int r_t = t < g.cap ? g.d_rank[t] : 0;
    const float sc = r_t > 0 ? g.d_scale[t] : 0.f;
    const int own0 = r_t > 0 ? t * g.RP : 0, own1 = r_t > 0 ? own0 + g.RP : 0;   // hd columns written by the MMA part

    // zero the other tenants' columns of this cluster's hd rows (and, with no adapter, the h rows): one warp per row
    for (int e = crank * 4 + warp; e < n_t; e += cs * 4) {
        const int tok = sm.list[e];
        bf16* row = g.hd + (size_t)tok * g.hd_cols;
        for (int c = lane * 8; c < g.hd_cols; c += 256)
            if (c < own0 || c >= own1) *reinterpret_cast<uint4*>(row + c) = make_uint4(0u, 0u, 0u, 0u);
        if (r_t == 0)
            for (int j = lane; j < g.RP; j += 32) g.h_out[(size_t)tok * g.RP + j] = 0.f;
    }
    if (r_t == 0) return;        // uniform over the cluster

    // ---- partial products over this CTA's share of K ---------------------------------------------------------
    const int oct_total = g.K >> 3;
    const int oct0 = (int)((int64_t)crank * oct_total / cs), oct1 = (int)((int64_t)(crank + 1) * oct_total / cs);
    const uint32_t sx_u = smem_u32(sm.sx), sa_u = smem_u32(sm.sa);
    const uint32_t part_rank0 = dk_map_to_cta(smem_u32(sm.part), 0);
    const int ngroups = (r_t + 15) >> 4;

    for (int p0 = 0; p0 < n_t; p0 += DS_PASS) {
        const int np = min(DS_PASS, n_t - p0);
        for (int jg = 0; jg < ngroups; ++jg) {
            float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
            const bf16* arow = g.At + ((size_t)t * g.RP + jg * 16) * g.K;
            for (int o0 = oct0; o0 < oct1; o0 += DS_SUB_OCT) {
                const int no = min(DS_SUB_OCT, oct1 - o0);
                __syncthreads();    // the previous sub-chunk has been consumed
#pragma unroll
                for (int e = tid; e < 16 * DS_SUB_OCT; e += DS_THREADS) {
                    const int row = e / DS_SUB_OCT, o = e - row * DS_SUB_OCT;
                    uint4 xv = make_uint4(0u, 0u, 0u, 0u), av = xv;
                    if (o < no) {
                        av = *reinterpret_cast<const uint4*>(arow + (size_t)row * g.K + (size_t)(o0 + o) * 8);
                        if (row < np)
                            xv = *reinterpret_cast<const uint4*>(g.x + (size_t)sm.list[p0 + row] * g.ldx + (size_t)(o0 + o) * 8);
                    }
                    *reinterpret_cast<uint4*>(sm.sx + row * DS_PITCH + o * 16) = xv;
                    *reinterpret_cast<uint4*>(sm.sa + row * DS_PITCH + o * 16) = av;
                }
                __syncthreads();
                // warp w multiplies k16 steps w, w + 4, ... of the sub-chunk (each step = two octets)
                const int steps = (no + 1) >> 1;
                for (int ks = warp; ks < steps; ks += 4) {
                    uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
                    ldmatrix_x4(sx_u + ((lane & 7) + ((lane >> 3) & 1) * 8) * DS_PITCH + (ks * 2 + (lane >> 4)) * 16, a0, a1, a2, a3);
                    ldmatrix_x4(sa_u + ((lane & 7) + (lane >> 4) * 8) * DS_PITCH + (ks * 2 + ((lane >> 3) & 1)) * 16, b0, b1, b2, b3);
                    mma_bf16_16816(c0, a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(c1, a0, a1, a2, a3, b2, b3);
                }
            }
            // this warp's 16 x 16 partial -> cluster rank 0, slot (crank, warp)
            {
                const int gq = lane >> 2, tq = lane & 3;
                const uint32_t base = part_rank0 + (uint32_t)((crank * 4 + warp) * 256) * 4;
                dk_st_cluster_f32(base + (gq * 16 + 2 * tq) * 4, c0[0]);
                dk_st_cluster_f32(base + (gq * 16 + 2 * tq + 1) * 4, c0[1]);
                dk_st_cluster_f32(base + ((gq + 8) * 16 + 2 * tq) * 4, c0[2]);
                dk_st_cluster_f32(base + ((gq + 8) * 16 + 2 * tq + 1) * 4, c0[3]);
                dk_st_cluster_f32(base + (gq * 16 + 8 + 2 * tq) * 4, c1[0]);
                dk_st_cluster_f32(base + (gq * 16 + 8 + 2 * tq + 1) * 4, c1[1]);
                dk_st_cluster_f32(base + ((gq + 8) * 16 + 8 + 2 * tq) * 4, c1[2]);
                dk_st_cluster_f32(base + ((gq + 8) * 16 + 8 + 2 * tq + 1) * 4, c1[3]);
            }
            dk_cluster_sync();
            if (crank == 0) {
                for (int e = tid; e < 256; e += DS_THREADS) {
                    const int i = e >> 4, j = e & 15;
                    if (i < np) {
                        float v = 0.f;
                        for (int s = 0; s < cs * 4; ++s) v += sm.part[s * 256 + e];   // fixed order
                        const int tok = sm.list[p0 + i];
                        g.h_out[(size_t)tok * g.RP + jg * 16 + j] = v;
                        g.hd[(size_t)tok * g.hd_cols + own0 + jg * 16 + j] = __float2bfloat16_rn(sc * v);
                    }
                }
            }
            dk_cluster_sync();      // rank 0 has read the partials before they are overwritten
        }
        // ranks beyond the tenant's true rank (rounded up to 16) stay zero
        if (crank == 0)
            for (int e = tid; e < np * (g.RP - ngroups * 16); e += DS_THREADS) {
                const int i = e / (g.RP - ngroups * 16), j = ngroups * 16 + e % (g.RP - ngroups * 16);
                const int tok = sm.list[p0 + i];
                g.h_out[(size_t)tok * g.RP + j] = 0.f;
                g.hd[(size_t)tok * g.hd_cols + own0 + j] = __float2bfloat16_rn(0.f);
            }
    }
}

// ---------------------------------------------------------------------------------------------------------------
// k_decode_gemm
// ---------------------------------------------------------------------------------------------------------------
constexpr int DG_THREADS = 192;

struct DecodeGemmArgs {
    int T, Nout;
    int num_kb;          // k-blocks of 64 over K
    int num_xb;          // k-blocks of 64 over the expand rows (cap*RP, or up to the last slot in use)
    int S;               // contraction slices = CTA pairs per cluster
    int nch;             // 64-column chunks of the B operand staged per CTA: the pair's strip is 128 * nch columns
    int stages;
    bf16* C;
    int64_t ldc;
    int32_t* status;
};

__device__ __forceinline__ void dg_tma_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void dg_commit_pair(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(mask)
                 : "memory");
}
__device__ __forceinline__ void dg_mma_pair(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

__global__ void __launch_bounds__(DG_THREADS, 1)
k_decode_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmXA, const __grid_constant__ CUtensorMap tmXB, const DecodeGemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int STAGES = g.stages;
    const uint32_t b_stage_bytes = (uint32_t)g.nch * CHUNK_BYTES;
    const uint32_t sA = smem_u32(smem);
    const uint32_t sB = sA + STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STAGE_BYTES + b_stage_bytes));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_drain = bar_tfull + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = dk_cluster_ctarank();
    const uint32_t half = crank & 1;            // which 128 rows of the 256-row tile
    const uint32_t pairi = crank >> 1;          // which slice of the contraction
    const uint32_t leader = crank & ~1u;
    const int NP = 128 * g.nch;                 // columns of the cluster's strip
    const int n0 = (int)dk_cluster_id_x() * NP;
    const int my_m = (int)half * 128, my_n = n0 + (int)half * 64 * g.nch;
    const uint32_t tmem_cols = (uint32_t)NP;    // 128 or 256

    const int kb0 = (int)((int64_t)pairi * g.num_kb / g.S), kb1 = (int)((int64_t)(pairi + 1) * g.num_kb / g.S);
    const int xb0 = (int)((int64_t)pairi * g.num_xb / g.S), xb1 = (int)((int64_t)(pairi + 1) * g.num_xb / g.S);

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
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (g.num_xb > 0) {
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
    tc_fence_before();
    __syncthreads();
    dk_cluster_sync();      // every CTA's barriers exist before any remote arrive or TMA completion
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // bytes the two CTAs of the pair stage per k-block (rows and columns outside the tensors are skipped entirely)
    auto a_bytes = [&](int r) -> uint32_t { return (r * 128 < g.T) ? A_STAGE_BYTES : 0u; };
    auto b_chunks = [&](int r) -> int { return max(0, min(g.nch, (g.Nout - (n0 + r * 64 * g.nch) + 63) / 64)); };
    const uint32_t stage_tx = a_bytes(0) + a_bytes(1) + (uint32_t)(b_chunks(0) + b_chunks(1)) * CHUNK_BYTES;
    const int my_chunks = b_chunks((int)half);
    const bool have_rows = my_m < g.T;

    bool epi_ok = true;
    if (warp == 0) {
        // ================= TMA producer (every CTA) =================
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t full0 = dk_map_to_cta(bar_full, leader);
            for (int kb = kb0; kb < kb1 && ok; ++kb, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 41))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                if (have_rows) dg_tma_pair(sA + s * A_STAGE_BYTES, &tmA, full0 + 8 * s, kb * BK, my_m);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + s * b_stage_bytes + c * CHUNK_BYTES, &tmB, full0 + 8 * s, my_n + c * 64, kb * BK);
            }
            if (ok && xb0 < xb1) dk_wait_prerequisites();     // hd comes from the shrink grid
            for (int xb = xb0; xb < xb1 && ok; ++xb, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 42))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                if (have_rows) dg_tma_pair(sA + s * A_STAGE_BYTES, &tmXA, full0 + 8 * s, xb * BK, my_m);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + s * b_stage_bytes + c * CHUNK_BYTES, &tmXB, full0 + 8 * s, my_n + c * 64, xb * BK);
            }
            if (!ok && half == 0) {
                // let the copies already issued land (bounded) before shared memory is reused or released
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
        // ================= MMA issuer (the pair's leader CTA) =================
        if (lane == 0 && half == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(NP >> 3) << 17) |
                                   ((uint32_t)(256 >> 4) << 24);    // fp32 acc, bf16 x bf16, B MN-major, M = 256, N = NP
            const uint16_t mask = (uint16_t)(3u << leader);
            uint32_t it = 0, acc = 0;
            bool ok = true;
            const int nblk = (kb1 - kb0) + (xb1 - xb0);
            for (int b = 0; b < nblk && ok; ++b, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 44))) break;
                tc_fence_after();
                const uint32_t a0 = sA + s * A_STAGE_BYTES, b0 = sB + s * b_stage_bytes;
#pragma unroll
                for (int j = 0; j < BK / 16; ++j) {
                    dg_mma_pair(tmem_base, desc_k_major(a0 + j * 32), desc_mn_major(b0 + j * UNIT_BYTES, CHUNK_BYTES), idesc, acc);
                    acc = 1;
                }
                dg_commit_pair(bar_empty + 8 * s, mask);
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
        epi_ok = mbar_wait(bar_tfull, 0, abort_word, 46);
        epi_ok = __all_sync(0xffffffffu, epi_ok);
        tc_fence_after();
    }

    // ---- sum the S slices through distributed shared memory ---------------------------------------------------
    // Row quarter q (32 rows) of each half is summed by pair (q mod S); that CTA's buffer holds, for each of its
    // 4 / S quarters, one [32][NP] fp32 block per source pair.  16-byte chunks are XOR-swizzled by the row so that
    // both the row-per-lane writes and the column-per-lane reads are conflict-free.
    tc_fence_before();
    __syncthreads();
    dk_cluster_sync();      // every pair's MMAs are complete: the pipeline stages may be overwritten
    tc_fence_after();
    const int qper = 4 / g.S;
    const uint32_t blk_bytes = 32u * (uint32_t)NP * 4u;
    const uint32_t row_bytes = (uint32_t)NP * 4u;
    if (warp >= 2 && epi_ok) {
        const int q = warp & 3;
        const uint32_t dst_rank = (uint32_t)(2 * (q % g.S)) + half;
        const uint32_t dst = dk_map_to_cta(sA, dst_rank) + (pairi * qper + (uint32_t)(q / g.S)) * blk_bytes + (uint32_t)lane * row_bytes;
#pragma unroll 1
        for (int c = 0; c < NP / 32; ++c) {
            uint32_t v[32];
            tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t c4 = (uint32_t)(c * 8 + e);
                dk_st_cluster_v4(dst + ((c4 ^ (uint32_t)(lane & 7)) << 4), v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
            }
        }
    }
    tc_fence_before();
    dk_cluster_sync();      // all partial blocks have landed
    if (warp >= 2 && epi_ok) {
        const int ew = warp - 2;
        for (int qs = 0; qs < qper; ++qs) {
            const int q = qs * g.S + (int)pairi;
            for (int rr = ew; rr < 32; rr += 4) {
                const int row = my_m + q * 32 + rr;
                if (row >= g.T) continue;
                for (int c4 = lane; c4 < NP / 4; c4 += 32) {
                    const int col = n0 + c4 * 4;
                    if (col >= g.Nout) continue;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int src = 0; src < g.S; ++src) {      // fixed order
                        const float4 p = *reinterpret_cast<const float4*>(
                            smem + (size_t)(src * qper + qs) * blk_bytes + (size_t)rr * row_bytes + ((c4 ^ (rr & 7)) << 4));
                        acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
                    }
                    __nv_bfloat162 p0 = __floats2bfloat162_rn(acc.x, acc.y), p1 = __floats2bfloat162_rn(acc.z, acc.w);
                    uint2 o;
                    o.x = *reinterpret_cast<uint32_t*>(&p0);
                    o.y = *reinterpret_cast<uint32_t*>(&p1);
                    *reinterpret_cast<uint2*>(g.C + (size_t)row * g.ldc + col) = o;
                }
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (threadIdx.x == 0) dk_wait_prerequisites();   // this grid never completes before the shrink grid it depends on
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
}

}  // namespace sm100

// ---------------------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------------------
bool decode_sm100_eligible(const marlaas_pool* pool, int64_t T) {
    return T > 0 && T <= sm100::DS_MAX_T && (int64_t)pool->cap * pool->RP <= 1024 && pool->sm_count >= 8;
}

marlaas_status_t launch_decode_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                     int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                     const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st) {
    using namespace sm100;
    const int64_t K = pool->K, N = pool->N;
    const int hd_cols = pool->cap * pool->RP;

    // ---- shrink: (cap + 1) clusters, K split over the CTAs of a cluster ----
    {
        DecodeShrinkArgs a;
        a.T = (int)T; a.K = (int)K; a.RP = pool->RP; a.cap = pool->cap;
        a.S = S; a.seg_offsets = seg_offsets; a.seg_slot = seg_slot;
        a.x = x; a.ldx = ldx; a.At = pool->d_At; a.d_rank = pool->d_rank; a.d_scale = pool->d_scale;
        a.tok_slot = ws.tok_slot; a.h_out = h_out; a.hd = ws.hd; a.hd_cols = hd_cols; a.status = pool->d_status;
        int cs = 8;
        while (cs > 1 && K / cs < 512) cs >>= 1;      // at least one full sub-chunk per CTA
        const size_t smem_bytes = sizeof(DecodeShrinkSmem) + 16;
        static bool attr_set[64] = {};
        if (pool->device >= 64 || !attr_set[pool->device]) {
            MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_shrink, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
            if (pool->device < 64) attr_set[pool->device] = true;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((pool->cap + 1) * cs));
        cfg.blockDim = dim3(DS_THREADS);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_shrink, a));
        count_launch();
    }

    // ---- GEMM with the expand as extra k-blocks ----
    int last_used = -1;
    for (int s = 0; s < pool->cap; ++s)
        if (pool->slots[s].used && pool->slots[s].rank > 0) last_used = s;
    DecodeGemmArgs g;
    g.T = (int)T; g.Nout = (int)N;
    g.num_kb = (int)cdiv(K, BK);
    g.num_xb = (int)cdiv((int64_t)(last_used + 1) * pool->RP, BK);
    g.C = y; g.ldc = ldy; g.status = pool->d_status;
    // strip width and contraction slices: fill the SMs with clusters of 2 * S CTAs
    struct Shape { int nch, S; };
    const Shape shapes[] = {{1, 2}, {2, 2}, {1, 1}, {2, 1}, {1, 4}, {2, 4}};
    Shape pick = {2, 1};
    int64_t best = -1;
    static int max_clusters[64][3] = {};      // per device, cluster size 2 / 4 / 8
    for (const Shape& sh : shapes) {
        const int csz = 2 * sh.S;
        const int ci = sh.S == 1 ? 0 : sh.S == 2 ? 1 : 2;
        const int stages_try = sh.nch == 1 ? 6 : 5;
        const size_t smem_try = 1024 + (size_t)stages_try * (A_STAGE_BYTES + sh.nch * CHUNK_BYTES) + 256;
        int mc = pool->device < 64 ? max_clusters[pool->device][ci] : 0;
        if (mc == 0) {
            MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
            cudaLaunchConfig_t qc = {};
            qc.gridDim = dim3((unsigned)(csz * 64));
            qc.blockDim = dim3(DG_THREADS);
            qc.dynamicSmemBytes = 200 * 1024;
            cudaLaunchAttribute qa;
            qa.id = cudaLaunchAttributeClusterDimension;
            qa.val.clusterDim.x = (unsigned)csz; qa.val.clusterDim.y = 1; qa.val.clusterDim.z = 1;
            qc.attrs = &qa; qc.numAttrs = 1;
            MARLAAS_CUDA_TRY(cudaOccupancyMaxActiveClusters(&mc, k_decode_gemm, &qc));
            if (mc < 1) mc = -1;
            if (pool->device < 64) max_clusters[pool->device][ci] = mc;
        }
        (void)smem_try;
        if (mc < 1) continue;
        const int64_t clusters = cdiv(N, 128 * sh.nch);
        if (clusters > mc) continue;                    // one wave only
        if (cdiv(K, BK) < sh.S) continue;
        const int64_t ctas = clusters * csz;
        // more CTAs streaming is better; among equals prefer fewer slices and wider strips (less re-read of x)
        const int64_t score = ctas * 16 - sh.S * 2 + sh.nch;
        if (score > best) { best = score; pick = sh; }
    }
    g.S = pick.S; g.nch = pick.nch;
    g.stages = pick.nch == 1 ? 6 : 5;
    const int NP = 128 * g.nch;

    alignas(64) CUtensorMap tmA, tmB, tmXA, tmXB;
    marlaas_status_t rc;
    if ((rc = make_map(&tmA, x, T, K, ldx, BK, BM)) != MARLAAS_OK) return rc;
    if ((rc = make_map(&tmB, W, K, N, ldw, 64, BK)) != MARLAAS_OK) return rc;
    if (g.num_xb > 0) {
        if ((rc = make_map(&tmXA, ws.hd, T, hd_cols, hd_cols, BK, BM)) != MARLAAS_OK) return rc;
        if ((rc = make_map(&tmXB, pool->d_Bs, hd_cols, N, N, 64, BK)) != MARLAAS_OK) return rc;
    } else {
        tmXA = tmA;
        tmXB = tmB;
    }
    const size_t smem_bytes = 1024 + (size_t)g.stages * (A_STAGE_BYTES + g.nch * CHUNK_BYTES) + 256;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cdiv(N, NP) * 2 * g.S));
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
