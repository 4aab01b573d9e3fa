// Decode-shaped forward as ONE kernel (at most 256 tokens, one per sequence, tenants unsorted).
//
//   y = bf16( [x | hd] * [W ; Bs] ),   hd[i][t*RP + j] = bf16(s_t (x_i A_t)[j]) for the token's own tenant t, else 0
//
// A cluster of S CTA pairs (cta_group::2, 256 token rows) owns one strip of output columns; the pairs split the
// contraction over K.  The shrink h = x A_t rides the same stream: the cluster is also given a few 16-rank units
// of the pooled adapter store, and every pipeline step adds one narrow MMA (N = 16 per unit) of the x tile that is
// in shared memory anyway against those adapter rows.  That product is dense (all 256 tokens against the unit),
// which costs nothing on a path bound by the pass over W; the token's own tenant is selected when hd is written.
//
//   phase A   every pair streams its slice of K: base accumulator [256][strip] and shrink accumulator [256][16 u]
//   sync 1    the other pairs' shrink partials are in the first pair's shared memory (fixed order sum)
//   phase C   first pair: writes its units' columns of hd (and h, tok_slot) and arrives at a grid-wide counter;
//             every pair: fetches its share of the expand's adapter rows, waits until every cluster has arrived,
//             fetches hd and adds its share of hd x Bs to its accumulator
//   exchange  row quarter q is finished by pair q mod S: the others send that quarter of their accumulators
//             through distributed shared memory; own + mailboxes in ascending pair order -> y
//
// The clusters wait on one another, so the launch is cooperative (all CTAs resident); every wait is bounded.  The
// grid-wide counter pair lives in the pool's status block and is left at zero by the last CTA to finish.
#include "sm100_ptx.cuh"
#include "sm100_cluster.cuh"

namespace marlaas {
namespace sm100 {

constexpr int DF_THREADS = 224;         // TMA producer, base MMA issuer, 4 epilogue warps, shrink MMA issuer
constexpr int DF_KP = 2;               // 64-deep panels per pipeline step
constexpr int DF_MAX_UPC = 8;          // 16-rank units per cluster
constexpr int DF_TABLE = 320;          // the segment table is staged in shared memory when S + 1 <= this
constexpr uint32_t DF_HROWS_BYTES = 8 * 128;   // one CTA's 8 adapter rows of a unit, one 64-deep panel

struct DecodeFusedArgs {
    int T, Nout;
    int num_ks;          // pipeline steps (kp * 64 deep) over K
    int num_xs;          // pipeline steps over the expand rows
    int S;               // contraction slices = CTA pairs per cluster
    int nch;             // 64-column chunks of W staged per CTA: the strip is 128 * nch columns
    int kp, stages;
    int RP, cap;
    int n_units;         // 16-rank units that hold adapter rows: (last slot in use + 1) * RP / 16
    int n_units_all;     // units the expand steps read (>= n_units; the rest are written as zeros)
    int upc;             // units per cluster: unit u belongs to cluster u mod (number of clusters)
    int nseg;            // segments; < 0: tok_slot already holds the per-token slots
    const int32_t* seg_offsets;
    const int32_t* seg_slot;
    int32_t* tok_slot;   // [T]
    const int32_t* d_rank;
    const float* d_scale;
    float* h_out;        // [T][RP]
    bf16* hd;            // [T][hd_cols]
    int hd_cols;
    bf16* C;
    int64_t ldc;
    int32_t* status;
    int32_t* sync;       // [0] arrivals of this call, [1] CTAs that have finished; both zero between calls
    int n_arrive, n_ctas;
};

__device__ __forceinline__ void df_tc_ld_32x8(uint32_t taddr, uint32_t (&v)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void df_bar_epi() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void df_fence_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ int df_ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void df_red_release(int32_t* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// K-major descriptor whose 8-row groups are `sbo_bytes` apart
__device__ __forceinline__ uint64_t df_desc_k_major(uint32_t saddr, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Bounded wait until the counter reaches `target`; false on abort (records the site like mbar_wait).
__device__ __forceinline__ bool df_wait_counter(const int32_t* p, int target, volatile int* abort_word, int site) {
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (df_ld_acquire(p) < target) {
        if (((++spins) & 63u) == 0) {
            if (*abort_word != 0) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                atomicCAS((int*)abort_word, 0, site);
                return false;
            }
        }
    }
    return true;
}

// Shared memory: [stages x A step] [stages x B step] [stages x unit-row step] [shrink partials (S-1) x 128 rows x 16 upc]
//                [segment table] [unit rank / scale] [barriers]; the exchange mailboxes reuse the stages
__global__ void __launch_bounds__(DF_THREADS, 1)
k_decode_fused(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmXA,
               const __grid_constant__ CUtensorMap tmXB, const DecodeFusedArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int STAGES = g.stages;
    const int NP = 128 * g.nch;                 // columns of the cluster's strip
    const uint32_t a_stage_bytes = (uint32_t)g.kp * A_STAGE_BYTES;
    const uint32_t b_chunk_bytes = (uint32_t)g.kp * CHUNK_BYTES;
    const uint32_t b_stage_bytes = (uint32_t)g.nch * b_chunk_bytes;
    const uint32_t h_unit_bytes = (uint32_t)g.kp * DF_HROWS_BYTES;
    const uint32_t h_stage_bytes = (uint32_t)g.upc * h_unit_bytes;
    const uint32_t box_bytes = (uint32_t)NP * 128u;                      // one 32-row quarter of one pair's partial
    const uint32_t hbox_bytes = (uint32_t)(g.S - 1) * (uint32_t)(4 * g.upc) * 2048u;
    const uint32_t sA = smem_u32(smem);
    const uint32_t sB = sA + STAGES * a_stage_bytes;
    const uint32_t sH = sB + STAGES * b_stage_bytes;
    const uint32_t sX = sH + STAGES * h_stage_bytes;
    uint8_t* after = smem + (sX - sA) + hbox_bytes;
    int32_t* off_tab = reinterpret_cast<int32_t*>(after);               // [DF_TABLE]
    int32_t* slot_tab = off_tab + DF_TABLE;                             // [DF_TABLE]
    int32_t* unit_rank = slot_tab + DF_TABLE;                           // [DF_MAX_UPC] rank and scale of the tenants of
    float* unit_scale = reinterpret_cast<float*>(unit_rank + DF_MAX_UPC);   // [DF_MAX_UPC] this cluster's units
    uint64_t* bars = reinterpret_cast<uint64_t*>(unit_scale + DF_MAX_UPC);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_hfull = bar_empty + 8 * STAGES;
    const uint32_t bar_tfull = bar_hfull + 8;
    const uint32_t bar_drain = bar_tfull + 8;
    const uint32_t bar_mail = bar_drain + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = dk_cluster_ctarank();
    const uint32_t half = crank & 1;            // which 128 rows of the 256-row tile
    const uint32_t pairi = crank >> 1;          // which slice of the contraction
    const uint32_t leader = crank & ~1u;
    const int cid = (int)dk_cluster_id_x();
    const int ncl = (int)gridDim.x / (2 * g.S);
    const int n0 = cid * NP;
    const int my_m = (int)half * 128, my_n = n0 + (int)half * 64 * g.nch;
    // this cluster's units: cid, cid + ncl, ...; those below n_units hold adapter rows, the rest are zero columns
    int nud = 0, nua = 0;
    for (int i = 0; i < g.upc; ++i) {
        const int u = cid + i * ncl;
        nud += u < g.n_units;
        nua += u < g.n_units_all;
    }
    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)(NP + 16 * g.upc)) tmem_cols <<= 1;

    const int ks0 = (int)((int64_t)pairi * g.num_ks / g.S), ks1 = (int)((int64_t)(pairi + 1) * g.num_ks / g.S);
    const int xs0 = (int)((int64_t)pairi * g.num_xs / g.S), xs1 = (int)((int64_t)(pairi + 1) * g.num_xs / g.S);
    const bool expander = xs1 > xs0;            // this pair adds its share of hd x Bs
    // The exchange of partial accumulators at the end (row quarter q is finished by pair q mod S).  Fast form: after
    // sync 1 every CTA of the cluster has finished the MMAs of phase A, so the two stages after a pair's last expand
    // step are free: the first is its inbox, the second its outbox.  A sending warp copies its quarter from tensor
    // memory to the outbox and one bulk copy moves it to the receiver's inbox, completing on the receiver's
    // barrier.  Otherwise the mailboxes take the first stages, the warps store to them directly, and a cluster
    // barrier on each side brackets the transfer.
    const int qper = 4 / g.S;
    const uint32_t mail_total = (uint32_t)((g.S - 1) * qper) * box_bytes;
    const uint32_t out_total = (uint32_t)(4 - qper) * box_bytes;
    const int nx_max = (g.num_xs + g.S - 1) / g.S;
    const bool fast_mail = g.S > 1 && mail_total <= a_stage_bytes && out_total <= a_stage_bytes && nx_max + 2 <= STAGES;
    auto mail_stage = [&](uint32_t pr) -> uint32_t {       // the stage after pair pr's last expand step
        const int k0 = (int)((int64_t)pr * g.num_ks / g.S), k1 = (int)((int64_t)(pr + 1) * g.num_ks / g.S);
        const int x0 = (int)((int64_t)pr * g.num_xs / g.S), x1 = (int)((int64_t)(pr + 1) * g.num_xs / g.S);
        return (uint32_t)(((k1 - k0) + (x1 - x0)) % STAGES);
    };
    const uint32_t mail_here = fast_mail ? sA + mail_stage(pairi) * a_stage_bytes : sA;
    const uint32_t out_here = sA + ((mail_stage(pairi) + 1) % (uint32_t)STAGES) * a_stage_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, nud > 0 ? 2 : 1);     // the base and the shrink MMA issuers both release a stage
        }
        mbar_init(bar_hfull, nud > 0 ? 2 : 1);
        mbar_init(bar_tfull, 1);
        mbar_init(bar_drain, 1);
        mbar_init(bar_mail, 1);
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (fast_mail) mbar_expect_tx(bar_mail, mail_total);      // armed for the other pairs' bulk copies
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (nud > 0) prefetch_tmap(&tmH);
        if (expander) {
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
    const uint32_t tmem_h = tmem_base + (uint32_t)NP;      // shrink accumulator: 16 * nud columns

    auto a_bytes = [&](int r) -> uint32_t { return (r * 128 < g.T) ? a_stage_bytes : 0u; };
    auto b_chunks = [&](int r) -> int { return max(0, min(g.nch, (g.Nout - (n0 + r * 64 * g.nch) + 63) / 64)); };
    const uint32_t base_tx = a_bytes(0) + a_bytes(1) + (uint32_t)(b_chunks(0) + b_chunks(1)) * b_chunk_bytes;
    const uint32_t stream_tx = base_tx + 2u * (uint32_t)nud * h_unit_bytes;
    const int my_chunks = b_chunks((int)half);
    const bool have_rows = my_m < g.T;
    const uint16_t pair_mask = (uint16_t)(3u << leader);
    const uint32_t full0 = dk_map_to_cta(bar_full, leader);

    // role state that lives across the phases
    uint32_t p_it = 0, p_s = 0, p_ph = 0;       // producer: steps issued, stage and phase of the next step
    uint32_t m_s = 0, m_ph = 0, m_acc = 0;      // MMA issuer
    bool ok = true;                             // this thread's role has not given up
    const int q = warp & 3;                     // epilogue warps: 32-row quarter = the warp's tensor-memory lanes
    const int erow = q * 32 + lane;             // row within this CTA's half
    const int row = my_m + erow;                // token
    int my_slot = -1;

    // =========================================== phase A ===========================================
    if (warp == 0) {
        if (lane == 0) {
            for (int ks = ks0; ks < ks1 && ok; ++ks, ++p_it) {
                if (!(ok = mbar_wait(bar_empty + 8 * p_s, p_ph ^ 1, abort_word, 41))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * p_s, stream_tx);
                if (have_rows) dg_tma_pair_3d(sA + p_s * a_stage_bytes, &tmA, full0 + 8 * p_s, 0, my_m, ks * g.kp);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + p_s * b_stage_bytes + c * b_chunk_bytes, &tmB, full0 + 8 * p_s, my_n + c * 64, ks * g.kp * BK);
                for (int i = 0; i < nud; ++i)
                    dg_tma_pair_3d(sH + p_s * h_stage_bytes + i * h_unit_bytes, &tmH, full0 + 8 * p_s, 0,
                                   16 * (cid + i * ncl) + 8 * (int)half, ks * g.kp);
                if (++p_s == (uint32_t)STAGES) { p_s = 0; p_ph ^= 1; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && half == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(NP >> 3) << 17) |
                                   ((uint32_t)(256 >> 4) << 24);    // fp32 acc, bf16 x bf16, B MN-major, M = 256, N = NP
            for (int b = ks0; b < ks1 && ok; ++b) {
                if (!(ok = mbar_wait(bar_full + 8 * m_s, m_ph, abort_word, 44))) break;
                tc_fence_after();
                const uint32_t a0 = sA + m_s * a_stage_bytes, b0 = sB + m_s * b_stage_bytes;
                for (int p = 0; p < g.kp; ++p) {
                    const uint64_t da0 = desc_k_major(a0 + p * A_STAGE_BYTES), db0 = desc_mn_major(b0 + p * CHUNK_BYTES, b_chunk_bytes);
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        dg_mma_pair(tmem_base, da0 + (uint64_t)(2 * j), db0 + (uint64_t)(j * (UNIT_BYTES >> 4)), idesc, m_acc);
                        m_acc = 1;
                    }
                }
                dg_commit_pair(bar_empty + 8 * m_s, pair_mask);
                if (++m_s == (uint32_t)STAGES) { m_s = 0; m_ph ^= 1; }
            }
            if (ok) dg_commit_pair(bar_hfull, pair_mask);     // this slice's base accumulator is complete
        }
        __syncwarp();
    } else if (warp == 6) {
        // shrink MMA issuer: its own thread, because a thread issues one MMA per ~80 cycles whatever its size, and the
        // narrow products would otherwise double the time of every step
        if (lane == 0 && half == 0 && nud > 0) {
            const uint32_t idesc_h = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((16 * nud) >> 3) << 17) |
                                     ((uint32_t)(256 >> 4) << 24);  // fp32 acc, bf16 x bf16, B K-major, M = 256, N = 16 per unit
            uint32_t h_s = 0, h_ph = 0, acc_h = 0;
            for (int b = ks0; b < ks1 && ok; ++b) {
                if (!(ok = mbar_wait(bar_full + 8 * h_s, h_ph, abort_word, 49))) break;
                tc_fence_after();
                const uint32_t a0 = sA + h_s * a_stage_bytes, h0 = sH + h_s * h_stage_bytes;
                for (int p = 0; p < g.kp; ++p) {
                    const uint64_t da0 = desc_k_major(a0 + p * A_STAGE_BYTES);
                    const uint64_t dh0 = df_desc_k_major(h0 + p * DF_HROWS_BYTES, h_unit_bytes);
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        dg_mma_pair(tmem_h, da0 + (uint64_t)(2 * j), dh0 + (uint64_t)(2 * j), idesc_h, acc_h);
                        acc_h = 1;
                    }
                }
                dg_commit_pair(bar_empty + 8 * h_s, pair_mask);
                if (++h_s == (uint32_t)STAGES) { h_s = 0; h_ph ^= 1; }
            }
            if (ok) dg_commit_pair(bar_hfull, pair_mask);     // this slice's shrink accumulator is complete
        }
        __syncwarp();
    } else {
        // epilogue warps of the first pair: the token's slot, while the stream runs
        if (pairi == 0) {
            const int te = (warp - 2) * 32 + lane;
            if (te < nud) {
                const int t = (16 * (cid + te * ncl)) / g.RP;
                unit_rank[te] = g.d_rank[t];
                unit_scale[te] = g.d_scale[t];
            }
            if (g.nseg >= 0) {
                const bool staged = g.nseg + 1 <= DF_TABLE;
                if (staged) {
                    for (int s = te; s <= g.nseg; s += 128) {
                        off_tab[s] = g.seg_offsets[s];
                        if (s < g.nseg) slot_tab[s] = g.seg_slot[s];
                    }
                    df_bar_epi();
                }
                if (cid == 0 && half == 0) {
                    for (int s = te; s < g.nseg; s += 128) {
                        const int a = staged ? off_tab[s] : g.seg_offsets[s], b = staged ? off_tab[s + 1] : g.seg_offsets[s + 1];
                        if (b < a || a < 0 || b > g.T) dk_report(g.status, DEV_BAD_TABLE, s);
                        if (s == 0 && a != 0) dk_report(g.status, DEV_BAD_TABLE, -1);
                        if (s == g.nseg - 1 && b != g.T) dk_report(g.status, DEV_BAD_TABLE, -2);
                    }
                    if (te == 0 && g.nseg == 0 && g.T != 0) dk_report(g.status, DEV_BAD_TABLE, -3);
                }
                if (row < g.T) {
                    int lo = 0, hi = g.nseg;
                    while (lo < hi) {       // first s with seg_offsets[s + 1] > row
                        const int mid = (lo + hi) >> 1;
                        const int v = staged ? off_tab[mid + 1] : g.seg_offsets[mid + 1];
                        if (v > row) hi = mid; else lo = mid + 1;
                    }
                    my_slot = lo < g.nseg ? (staged ? slot_tab[lo] : g.seg_slot[lo]) : -1;
                }
            } else if (row < g.T) {
                my_slot = g.tok_slot[row];
            }
            if (row < g.T) {
                if (my_slot < -1 || my_slot >= g.cap) {
                    if (cid == 0) dk_report(g.status, DEV_BAD_INDEX, row);
                    my_slot = -1;
                }
                if (cid == 0) {
                    g.tok_slot[row] = my_slot;
                    // tokens routed to no adapter: their row of h is zero
                    if (my_slot < 0 || g.d_rank[my_slot] <= 0) {
                        float4* hr = reinterpret_cast<float4*>(g.h_out + (size_t)row * g.RP);
                        for (int j = 0; j < g.RP / 4; ++j) hr[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
        }
        if (pairi == 0) df_bar_epi();      // unit_rank / unit_scale are written
        ok = mbar_wait(bar_hfull, 0, abort_word, 45);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        // the other pairs' shrink partials go to the first pair (same half), raw accumulator columns
        if (pairi != 0 && ok && nud > 0) {
            const uint32_t dst = dk_map_to_cta(sX, half) + (pairi - 1) * (uint32_t)(4 * g.upc) * 2048u + (uint32_t)erow * 16u;
            for (int c8 = 0; c8 < 2 * nud; ++c8) {
                uint32_t v[8];
                df_tc_ld_32x8(tmem_h + ((uint32_t)(q * 32) << 16) + c8 * 8, v);
                tc_wait_ld();
                dk_st_cluster_v4(dst + (uint32_t)(2 * c8) * 2048u, v[0], v[1], v[2], v[3]);
                dk_st_cluster_v4(dst + (uint32_t)(2 * c8 + 1) * 2048u, v[4], v[5], v[6], v[7]);
            }
        }
    }

    // =========================================== sync 1 ===========================================
    if (g.S > 1) {
        tc_fence_before();
        dk_cluster_sync();      // shrink partials have landed in the first pair
        tc_fence_after();
    }

    // =========================================== phase C ===========================================
    if (warp == 0) {
        if (lane == 0 && expander) {
            // the adapter rows Bs do not depend on hd: the first steps' B operands are fetched before the wait
            const int nx = xs1 - xs0;
            const int npre = nx < STAGES ? nx : STAGES;
            uint32_t b_s = p_s, b_ph = p_ph;
            for (int i = 0; i < npre && ok; ++i) {
                if (!(ok = mbar_wait(bar_empty + 8 * b_s, b_ph ^ 1, abort_word, 42))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * b_s, base_tx);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + b_s * b_stage_bytes + c * b_chunk_bytes, &tmXB, full0 + 8 * b_s, my_n + c * 64,
                                (xs0 + i) * g.kp * BK);
                if (++b_s == (uint32_t)STAGES) { b_s = 0; b_ph ^= 1; }
            }
            // hd is complete when every cluster's first pair has arrived (two CTAs each)
            if (ok) ok = df_wait_counter(g.sync, g.n_arrive, abort_word, 47);
            df_fence_async();       // the other CTAs' generic-proxy stores to hd, before this thread's TMA reads
            for (int i = 0; i < npre && ok; ++i, ++p_it) {
                if (have_rows) dg_tma_pair_3d(sA + p_s * a_stage_bytes, &tmXA, full0 + 8 * p_s, 0, my_m, (xs0 + i) * g.kp);
                if (++p_s == (uint32_t)STAGES) { p_s = 0; p_ph ^= 1; }
            }
            for (int xs = xs0 + npre; xs < xs1 && ok; ++xs, ++p_it) {
                if (!(ok = mbar_wait(bar_empty + 8 * p_s, p_ph ^ 1, abort_word, 42))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * p_s, base_tx);
                if (have_rows) dg_tma_pair_3d(sA + p_s * a_stage_bytes, &tmXA, full0 + 8 * p_s, 0, my_m, xs * g.kp);
                for (int c = 0; c < my_chunks; ++c)
                    dg_tma_pair(sB + p_s * b_stage_bytes + c * b_chunk_bytes, &tmXB, full0 + 8 * p_s, my_n + c * 64, xs * g.kp * BK);
                if (++p_s == (uint32_t)STAGES) { p_s = 0; p_ph ^= 1; }
            }
        }
        if (lane == 0 && half == 0 && *abort_word != 0) {
            // let the copies already issued land (bounded) before shared memory is released
            const uint32_t back = p_it < (uint32_t)STAGES ? p_it : (uint32_t)STAGES;
            for (uint32_t j = 0; j < back; ++j) {
                const uint32_t jt = p_it - 1 - j;
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_full + 8 * (jt % (uint32_t)STAGES), (jt / (uint32_t)STAGES) & 1) &&
                       global_ns() - t0 < WAIT_LIMIT_NS) {
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && half == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(NP >> 3) << 17) |
                                   ((uint32_t)(256 >> 4) << 24);
            for (int b = xs0; b < xs1 && ok; ++b) {
                if (!(ok = mbar_wait(bar_full + 8 * m_s, m_ph, abort_word, 48))) break;
                tc_fence_after();
                const uint32_t a0 = sA + m_s * a_stage_bytes, b0 = sB + m_s * b_stage_bytes;
                for (int p = 0; p < g.kp; ++p) {
                    const uint64_t da0 = desc_k_major(a0 + p * A_STAGE_BYTES), db0 = desc_mn_major(b0 + p * CHUNK_BYTES, b_chunk_bytes);
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        dg_mma_pair(tmem_base, da0 + (uint64_t)(2 * j), db0 + (uint64_t)(j * (UNIT_BYTES >> 4)), idesc, m_acc);
                        m_acc = 1;
                    }
                }
                dg_commit_pair(bar_empty + 8 * m_s, pair_mask);
                if (nud > 0) dg_commit_pair(bar_empty + 8 * m_s, pair_mask);     // the shrink issuer's arrival
                if (++m_s == (uint32_t)STAGES) { m_s = 0; m_ph ^= 1; }
            }
            if (ok) {
                dg_commit_pair(bar_tfull, pair_mask);
            } else {
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_drain)
                             : "memory");
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar_drain, 0) && global_ns() - t0 < WAIT_LIMIT_NS) {
                }
            }
        }
        __syncwarp();
    } else if (warp < 6) {
        if (pairi == 0) {
            // ---- this cluster's columns of hd (all 256 tokens), h for the tokens of the units' tenants ----
            for (int i = 0; i < nua; ++i) {
                const int u = cid + i * ncl;
                uint4 o0 = make_uint4(0u, 0u, 0u, 0u), o1 = o0;
                if (i < nud) {
                    uint32_t lo[8], hi[8];
                    df_tc_ld_32x8(tmem_h + ((uint32_t)(q * 32) << 16) + 8 * i, lo);
                    df_tc_ld_32x8(tmem_h + ((uint32_t)(q * 32) << 16) + 8 * nud + 8 * i, hi);
                    tc_wait_ld();
                    float v[16];
#pragma unroll
                    for (int e = 0; e < 8; ++e) { v[e] = __uint_as_float(lo[e]); v[8 + e] = __uint_as_float(hi[e]); }
                    for (int si = 0; si + 1 < g.S; ++si) {      // ascending pair order
                        const uint32_t a = sX + (uint32_t)si * (uint32_t)(4 * g.upc) * 2048u + (uint32_t)erow * 16u;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint32_t cg = (e < 2) ? (uint32_t)(2 * i + e) : (uint32_t)(2 * nud + 2 * i + (e - 2));
                            float4 p;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                         : "=f"(p.x), "=f"(p.y), "=f"(p.z), "=f"(p.w)
                                         : "r"(a + cg * 2048u));
                            v[4 * e] += p.x; v[4 * e + 1] += p.y; v[4 * e + 2] += p.z; v[4 * e + 3] += p.w;
                        }
                    }
                    const int t = (16 * u) / g.RP, j0 = (16 * u) - t * g.RP;
                    if (ok && row < g.T && my_slot == t && unit_rank[i] > 0) {
                        const float sc = unit_scale[i];
                        float4* hr = reinterpret_cast<float4*>(g.h_out + (size_t)row * g.RP + j0);
#pragma unroll
                        for (int e = 0; e < 4; ++e) hr[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            __nv_bfloat162 pk = __floats2bfloat162_rn(sc * v[2 * e], sc * v[2 * e + 1]);
                            w[e] = *reinterpret_cast<uint32_t*>(&pk);
                        }
                        o0 = make_uint4(w[0], w[1], w[2], w[3]);
                        o1 = make_uint4(w[4], w[5], w[6], w[7]);
                    }
                }
                if (row < g.T && 16 * u + 16 <= g.hd_cols) {
                    uint4* hp = reinterpret_cast<uint4*>(g.hd + (size_t)row * g.hd_cols + 16 * u);
                    hp[0] = o0;
                    hp[1] = o1;
                }
            }
            // the CTA's stores, then one release at GPU scope: the barrier orders the other threads' stores before it
            df_bar_epi();
            if (warp == 2 && lane == 0) df_red_release(g.sync, 1);
        }
        ok = mbar_wait(bar_tfull, 0, abort_word, 46) && ok;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
    }

    // ---- sum the S slices through distributed shared memory ---------------------------------------------------
    // Row quarter q (32 rows) of each half is finished by pair (q mod S).  The other pairs' warps holding that
    // quarter send their partial accumulators to a mailbox in the finishing CTA (thread to thread: the same
    // tensor-memory lane on both sides, [column group][lane] 16-byte slots), and the finishing warp adds them to
    // its own accumulator in ascending pair order.  The mailboxes reuse the pipeline stages.
    const uint32_t own = (uint32_t)(q % g.S);
    const bool epi = warp >= 2 && warp < 6;
    if (g.S > 1) {
        if (!fast_mail) {
            tc_fence_before();
            __syncthreads();
            dk_cluster_sync();      // every pair's MMAs are complete: the pipeline stages may be overwritten
            tc_fence_after();
        }
        if (epi && ok && own != pairi) {
            const uint32_t si = pairi < own ? pairi : pairi - 1;
            const uint32_t box = (si * (uint32_t)qper + (uint32_t)(q / g.S)) * box_bytes;     // place in the receiver's inbox
            if (fast_mail) {
                int oi = 0;     // which of this CTA's outgoing quarters
                for (int qq = 0; qq < q; ++qq) oi += (uint32_t)(qq % g.S) != pairi;
                const uint32_t src = out_here + (uint32_t)oi * box_bytes;
#pragma unroll 1
                for (int c = 0; c < NP / 32; ++c) {
                    uint32_t v[32];
                    tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(src + (uint32_t)lane * 16u + (uint32_t)(c * 8 + e) * 512u),
                                     "r"(v[4 * e]), "r"(v[4 * e + 1]), "r"(v[4 * e + 2]), "r"(v[4 * e + 3])
                                     : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the stores above, before the bulk copy reads
                __syncwarp();
                if (lane == 0) {
                    const uint32_t rcta = 2 * own + half;
                    const uint32_t dst = dk_map_to_cta(sA + mail_stage(own) * a_stage_bytes + box, rcta);
                    asm volatile(
                        "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                        "r"(src), "r"(box_bytes), "r"(dk_map_to_cta(bar_mail, rcta))
                        : "memory");
                }
            } else {
                const uint32_t dst = dk_map_to_cta(sA, 2 * own + half) + box + (uint32_t)lane * 16u;
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
        }
        if (!fast_mail) {
            tc_fence_before();
            dk_cluster_sync();      // all partial accumulators have landed
            tc_fence_after();
        } else if (epi && own == pairi) {
            ok = mbar_wait(bar_mail, 0, abort_word, 50) && ok;     // the other pairs' copies are complete
            ok = __all_sync(0xffffffffu, ok);
        }
    }
    if (epi && ok && own == pairi) {
        bf16* crow = g.C + (size_t)row * g.ldc + n0;
        const uint32_t mbox = mail_here + (uint32_t)(q / g.S) * box_bytes + (uint32_t)lane * 16u;
#pragma unroll 1
        for (int c = 0; c < NP / 32; ++c) {
            uint32_t v[32];
            tc_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, v);
            tc_wait_ld();
            float acc[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] = 0.f;
            for (uint32_t src = 0; src < (uint32_t)g.S; ++src) {      // ascending pair order
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
    __syncthreads();
    dk_cluster_sync();      // the pair leaves together (its barriers and tensor memory are shared)
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (threadIdx.x == 0) {
        if (*abort_word != 0) {
            if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
        }
        // the last CTA to finish leaves both counters at zero for the next call (every arrival of a CTA precedes
        // its own count here)
        __threadfence();
        if (atomicAdd(g.sync + 1, 1) == g.n_ctas - 1) {
            g.sync[0] = 0;
            g.sync[1] = 0;
            __threadfence();
        }
    }
}

}  // namespace sm100

// ---------------------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------------------
namespace {
constexpr int DF_SMEM_MAX = 227 * 1024;
struct FusedShape { int nch, S, upc, stages; size_t smem; };

// most clusters of `csz` CTAs with `smem` bytes each that can be resident at once (cached per device)
int fused_max_clusters(int device, int csz, size_t smem) {
    struct Entry { int device, csz; size_t smem; int mc; };
    static std::vector<Entry> cache;
    for (const Entry& e : cache)
        if (e.device == device && e.csz == csz && e.smem == smem) return e.mc;
    cudaLaunchConfig_t qc = {};
    qc.gridDim = dim3((unsigned)(csz * 64));
    qc.blockDim = dim3(sm100::DF_THREADS);
    qc.dynamicSmemBytes = smem;
    cudaLaunchAttribute qa;
    qa.id = cudaLaunchAttributeClusterDimension;
    qa.val.clusterDim.x = (unsigned)csz; qa.val.clusterDim.y = 1; qa.val.clusterDim.z = 1;
    qc.attrs = &qa; qc.numAttrs = 1;
    int mc = 0;
    if (cudaOccupancyMaxActiveClusters(&mc, sm100::k_decode_fused, &qc) != cudaSuccess) {
        (void)cudaGetLastError();
        mc = 0;
    }
    cache.push_back({device, csz, smem, mc});
    return mc;
}
}  // namespace

// Launches the single-kernel decode forward when the batch and the pool allow it; *launched tells the caller
// whether it did (otherwise nothing was issued and the two-kernel path should run).
marlaas_status_t launch_decode_fused_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                           int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                           const int32_t* seg_slot, const Workspace& ws, float* h_out, const void* ws_key,
                                           cudaStream_t st, bool* launched) {
    using namespace sm100;
    *launched = false;
    const int64_t K = pool->K, N = pool->N;
    const int RP = pool->RP;
    const int hd_cols = (int)align_up((size_t)pool->cap * RP, 64);
    int last_used = -1;
    for (int s = 0; s < pool->cap; ++s)
        if (pool->slots[s].used && pool->slots[s].rank > 0) last_used = s;
    const int kp = DF_KP;
    const int num_xs = (int)cdiv((int64_t)(last_used + 1) * RP, (int64_t)kp * BK);
    const int n_units = (last_used + 1) * RP / 16;
    const int n_units_all = std::min(num_xs * kp * 4, hd_cols / 16);

    static bool attr_set[64] = {};
    if (pool->device >= 64 || !attr_set[pool->device]) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, DF_SMEM_MAX));
        if (pool->device < 64) attr_set[pool->device] = true;
    }

    // strip width and contraction slices: one wave of clusters of 2 * S CTAs, as many CTAs streaming as possible
    const FusedShape shapes[] = {{1, 2}, {2, 2}, {1, 1}, {2, 1}, {1, 4}, {2, 4}};
    FusedShape pick = {};
    int64_t best = -1;
    for (FusedShape sh : shapes) {
        const int NP = 128 * sh.nch;
        const int64_t ncl = cdiv(N, NP);
        sh.upc = (int)std::max<int64_t>(1, cdiv(n_units_all, ncl));
        if (sh.upc > DF_MAX_UPC || NP + 16 * sh.upc > 512) continue;
        if (cdiv(K, (int64_t)kp * BK) < sh.S) continue;        // every slice needs at least one step
        const size_t fixed = 1024 + (size_t)(sh.S - 1) * 4 * sh.upc * 2048 +
                             (size_t)DF_TABLE * 8 + 256;
        const size_t step = (size_t)kp * (A_STAGE_BYTES + sh.nch * CHUNK_BYTES + sh.upc * DF_HROWS_BYTES);
        if (fixed + 2 * step > (size_t)DF_SMEM_MAX) continue;
        sh.stages = (int)std::min<size_t>(8, ((size_t)DF_SMEM_MAX - fixed) / step);
        sh.smem = fixed + (size_t)sh.stages * step;
        const int mc = fused_max_clusters(pool->device, 2 * sh.S, sh.smem);
        if (ncl > mc) continue;                                 // all clusters must be resident together
        const int64_t score = ncl * 2 * sh.S * 16 - sh.S * 2 + sh.nch;
        if (score > best) { best = score; pick = sh; }
    }
    if (best < 0) return MARLAAS_OK;

    // the grid-wide counter pair of this workspace (two calls in flight use two workspaces, hence two pairs)
    int set = -1;
    for (int i = 0; i < MARLAAS_SYNC_SETS; ++i)
        if (pool->sync_owner[i] == ws_key) { set = i; break; }
    if (set < 0)
        for (int i = 0; i < MARLAAS_SYNC_SETS; ++i)
            if (pool->sync_owner[i] == nullptr) { pool->sync_owner[i] = ws_key; set = i; break; }
    if (set < 0) return MARLAAS_OK;     // more workspaces in use with this pool than counter pairs: two-kernel path

    const int NP = 128 * pick.nch;
    const int ncl = (int)cdiv(N, NP);
    DecodeFusedArgs g;
    g.T = (int)T; g.Nout = (int)N;
    g.num_ks = (int)cdiv(K, (int64_t)kp * BK);
    g.num_xs = num_xs;
    g.S = pick.S; g.nch = pick.nch; g.kp = kp; g.stages = pick.stages;
    g.RP = RP; g.cap = pool->cap;
    g.n_units = n_units; g.n_units_all = n_units_all; g.upc = pick.upc;
    g.nseg = S; g.seg_offsets = seg_offsets; g.seg_slot = seg_slot;
    g.tok_slot = ws.tok_slot; g.d_rank = pool->d_rank; g.d_scale = pool->d_scale;
    g.h_out = h_out; g.hd = ws.hd; g.hd_cols = hd_cols;
    g.C = y; g.ldc = ldy; g.status = pool->d_status;
    g.sync = pool->d_status + 16 + 2 * set;
    g.n_arrive = 2 * ncl; g.n_ctas = ncl * 2 * pick.S;

    alignas(64) CUtensorMap tmA, tmB, tmH, tmXA, tmXB;
    marlaas_status_t rc;
    if ((rc = make_panel_map(&tmA, x, T, K, ldx, (uint32_t)kp)) != MARLAAS_OK) return rc;
    if ((rc = make_map(&tmB, W, K, N, ldw, 64, (uint32_t)(kp * BK))) != MARLAAS_OK) return rc;
    if (num_xs > 0) {
        if ((rc = make_panel_map(&tmH, pool->d_At, (int64_t)pool->cap * RP, K, K, (uint32_t)kp, 8)) != MARLAAS_OK) return rc;
        if ((rc = make_panel_map(&tmXA, ws.hd, T, hd_cols, hd_cols, (uint32_t)kp)) != MARLAAS_OK) return rc;
        if ((rc = make_map(&tmXB, pool->d_Bs, (int64_t)pool->cap * RP, N, N, 64, (uint32_t)(kp * BK))) != MARLAAS_OK) return rc;
    } else {
        tmH = tmA; tmXA = tmA; tmXB = tmB;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)g.n_ctas);
    cfg.blockDim = dim3(DF_THREADS);
    cfg.dynamicSmemBytes = pick.smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)(2 * pick.S); at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeCooperative;
    at[1].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_fused, tmA, tmB, tmH, tmXA, tmXB, g));
    count_launch();
    *launched = true;
    return MARLAAS_OK;
}

}  // namespace marlaas
