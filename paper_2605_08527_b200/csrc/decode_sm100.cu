// Decode-shaped forward (up to four 256-token tiles, typically one token per sequence, tenants unsorted): the call is
// bound by the one pass over W from HBM, so the work is cut to keep the memory system busy from the first microsecond
// to the last and the launch count to two kernels that run side by side on disjoint SMs.
//
//   k_decode_gemm    (tcgen05, TMA)  y^T = [W ; Bs]^T * [x | hd]^T: the base product and the expand as ONE contraction
//                    over K + cap*RP, with the operand roles swapped against the training GEMM: 256 columns of W are the
//                    M side of a cta_group::2 MMA (128 per CTA, read as an MN-major A operand straight from the row-major
//                    weight), the 256 tokens its N side (128 per CTA).  A 64-deep step therefore brings as many bytes of
//                    W as of x into a CTA (16 KB each), half the activation re-reads of a token-major tile.  A tile's
//                    contraction is cut into S slices (1, 2 or 4 CTA pairs); the partial accumulators are summed in a
//                    fixed tree: the two pairs of a 4-CTA cluster exchange token halves through distributed shared
//                    memory, the two clusters of a tile exchange token quarters through an L2-resident scratch buffer.
//   k_decode_shrink  (mma.sync, bulk copies)  per tenant and 16-token pass: h_i = x_i A_t from the pooled store.  Runs on
//                    the SMs the GEMM's clusters leave free (its CTAs take work units from a counter, so any number of
//                    resident CTAs is correct), writes tok_slot, fp32 h and the dense expand operand
//                    hd[i][t*RP + j] = bf16(s_t h_i[j]) (zeros in every other tenant's columns), and counts finished units;
//                    the GEMM's expand steps wait for that count.
//
// Launch order: the GEMM first (it triggers its dependents at once), the shrink second as its programmatic dependent.
// The shrink grid ends with a wait for the GEMM grid and then clears the counters and flags, so a kernel ordered after
// the pair sees both complete, and a replay of a captured call finds the counters at zero.
#include "sm100_ptx.cuh"
#include "sm100_cluster.cuh"

#include <algorithm>

namespace marlaas {
namespace sm100 {

// words of the pool's synchronisation area
constexpr int SY_TICKET = 0;        // next shrink work unit
constexpr int SY_DONE = 1;          // finished shrink work units
constexpr int SY_EXIT = 2;          // shrink CTAs that have reached their end
constexpr int SY_FLAGS = 16;        // split-K exchange flags, one per (tile, destination cluster, CTA, epilogue warp)

__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int32_t* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded wait for a global word to reach `target` (acquire); gives up like mbar_wait.
__device__ __forceinline__ bool wait_word_ge(const int32_t* p, int target, volatile int* abort_word, int site) {
    if (ld_acquire_gpu(p) >= target) return true;
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (true) {
        if (ld_acquire_gpu(p) >= target) return true;
        __nanosleep(40);
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
}

// ---------------------------------------------------------------------------------------------------------------
// k_decode_gemm
// ---------------------------------------------------------------------------------------------------------------
constexpr int DG_THREADS = 320;        // warp 0: TMA producer, warp 1: MMA issuer + tensor memory, warps 2..9: epilogue
constexpr int DG_TN = 256;             // tokens per tile = N of the MMA
constexpr int DG_TM = 256;             // W columns per tile = M of the MMA (128 per CTA)
constexpr uint32_t DG_MBOX_BYTES = 64 * 1024;   // one token half of a CTA's accumulator: 128 lanes x 128 columns fp32

struct DecodeGemmArgs {
    int T, Nout;
    int nstrips;         // 256-column strips of W; tile = (token tile, strip)
    int num_ks;          // 64-deep pipeline steps over K
    int num_xs;          // 64-deep pipeline steps over the expand rows (up to the last slot in use)
    int S;               // contraction slices per tile: 1 (clusters of one CTA pair), 2 or 4 (clusters of two pairs)
    int stages;
    int w3d;             // the W-side operand moves with one 3-D copy per step (N a multiple of 64), else one per chunk
    int n_units;         // shrink work units that must be finished before hd is read
    int n_flags;         // exchange flags in use (S = 4)
    int reset_at_end;    // serial order (shrink grid first): this grid ends last and clears the counters and flags
    bf16* C;
    int64_t ldc;
    int32_t* status;
    int32_t* sync;
    float* xbuf;         // S = 4: exchange buffer between the two clusters of a tile
};

__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ void mbar_arrive_remote_release(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ uint4 ld_cg_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// Operand staging per 64-deep pipeline step and CTA:
//   Wt [2 chunks][64 k][64 n]   the CTA's 128 columns of W (or of the adapter rows Bs): MN-major A operand, 128-byte
//                               swizzle, chunks 8 KB apart
//   Xt [128 tokens][64 k]       the CTA's half of the token tile of x (or of hd): K-major B operand
__global__ void __launch_bounds__(DG_THREADS, 1)
k_decode_gemm(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
              const __grid_constant__ CUtensorMap tmXW, const __grid_constant__ CUtensorMap tmXX, const DecodeGemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int STAGES = g.stages;
    constexpr uint32_t W_BYTES = 2 * CHUNK_BYTES, X_BYTES = A_STAGE_BYTES, STAGE_BYTES = W_BYTES + X_BYTES;
    const uint32_t sStage = smem_u32(smem);
    const uint32_t mbox_off = (uint32_t)STAGES * STAGE_BYTES;
    const uint32_t sMbox = sStage + mbox_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + mbox_off + (g.S > 1 ? DG_MBOX_BYTES : 0u));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_drain = bar_tfull + 8;
    const uint32_t bar_mbox = bar_drain + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 3);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t TMEM_COLS = DG_TN;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_drain, 1);
        mbar_init(bar_mbox, DG_THREADS - 64);       // every epilogue thread of the partner CTA arrives once
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x == 64) {
        prefetch_tmap(&tmW);
        prefetch_tmap(&tmX);
        if (g.num_xs > 0) {
            prefetch_tmap(&tmXW);
            prefetch_tmap(&tmXX);
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    const uint32_t crank = dk_cluster_ctarank();
    const uint32_t half = crank & 1;            // which 128 W columns and which 128 tokens this CTA stages
    const uint32_t pi = crank >> 1;             // pair within the cluster
    const uint32_t leader = crank & ~1u;
    const int C2 = g.S > 2 ? 2 : 1;             // clusters per tile
    const int cid = (int)dk_cluster_id_x();
    const int tile = cid / C2, cs = cid % C2;
    const int sl = cs * 2 + (int)pi;            // contraction slice of this pair
    const int n0 = (tile % g.nstrips) * DG_TM;
    const int m0 = (tile / g.nstrips) * DG_TN;
    const int my_n = n0 + (int)half * 128, my_tok = m0 + (int)half * 128;
    const int ks0 = sl * g.num_ks / g.S, ks1 = (sl + 1) * g.num_ks / g.S;
    const int xs0 = sl * g.num_xs / g.S, xs1 = (sl + 1) * g.num_xs / g.S;
    const int nbase = ks1 - ks0, nstep = nbase + (xs1 - xs0);

    // Everything above touches no global memory; from here on the kernels ordered before this one are complete.  The
    // shrink grid (this grid's dependent) may start as soon as every CTA has passed this point.
    dk_wait_prerequisites();
    dk_launch_dependents();

    tc_fence_before();
    dk_cluster_sync();      // every CTA's barriers exist before any remote arrive or TMA completion
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // bytes the two CTAs of the pair stage per step (boxes wholly outside the tensors are skipped; partly outside boxes
    // are filled with zeros and count in full)
    auto x_tx = [&](int r) -> uint32_t { return (m0 + r * 128 < g.T) ? X_BYTES : 0u; };
    auto w_chunks = [&](int r) -> int { return max(0, min(2, (g.Nout - (n0 + r * 128) + 63) / 64)); };
    auto w_tx = [&](int r) -> uint32_t { const int c = w_chunks(r); return (g.w3d ? (c > 0 ? 2u : 0u) : (uint32_t)c) * CHUNK_BYTES; };
    const uint32_t stage_tx = x_tx(0) + x_tx(1) + w_tx(0) + w_tx(1);
    const int my_chunks = w_chunks((int)half);
    const bool have_rows = my_tok < g.T;

    bool epi_ok = true;
    if (warp == 0) {
        // ================= TMA producer (every CTA) =================
        if (lane == 0) {
            uint32_t it = 0, s = 0, ph = 0;
            bool ok = true, hd_ready = false;
            const uint32_t full0 = dk_map_to_cta(bar_full, leader);
            for (int b = 0; b < nstep && ok; ++b, ++it) {
                const bool ex = b >= nbase;
                const int step = ex ? xs0 + (b - nbase) : ks0 + b;
                const CUtensorMap* mw = ex ? &tmXW : &tmW;
                const CUtensorMap* mx = ex ? &tmXX : &tmX;
                if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 41))) break;
                if (half == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                const uint32_t dw = sStage + s * STAGE_BYTES, dx = dw + W_BYTES;
                if (g.w3d) {
                    if (my_chunks > 0) dg_tma_pair_3d(dw, mw, full0 + 8 * s, 0, step * BK, my_n >> 6);
                } else {
                    for (int c = 0; c < my_chunks; ++c) dg_tma_pair(dw + c * CHUNK_BYTES, mw, full0 + 8 * s, my_n + c * 64, step * BK);
                }
                if (ex && !hd_ready) {
                    // the adapter rows above do not depend on the shrink grid; hd does
                    if (!(ok = wait_word_ge(g.sync + SY_DONE, g.n_units, abort_word, 43))) break;
                    fence_proxy_async_all();
                    hd_ready = true;
                }
                if (have_rows) dg_tma_pair_3d(dx, mx, full0 + 8 * s, 0, my_tok, step);
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
            if (!ok && half == 0) {
                // let the copies already issued land (bounded) before shared memory is released
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
            // fp32 accumulate, bf16 x bf16, A MN-major (W columns), B K-major (tokens), M = 256, N = 256
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(DG_TN >> 3) << 17) |
                                       ((uint32_t)(DG_TM >> 4) << 24);
            const uint16_t mask = (uint16_t)(3u << leader);
            uint32_t acc = 0, s = 0, ph = 0;
            bool ok = true;
            for (int b = 0; b < nstep && ok; ++b) {
                if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 44))) break;
                tc_fence_after();
                const uint32_t dw = sStage + s * STAGE_BYTES, dx = dw + W_BYTES;
                // descriptors of successive 16-deep slices differ only in the start-address field (16-byte units)
                const uint64_t da0 = desc_mn_major(dw, CHUNK_BYTES), db0 = desc_k_major(dx);
#pragma unroll
                for (int j = 0; j < BK / 16; ++j) {
                    dg_mma_pair(tmem_base, da0 + (uint64_t)(j * (UNIT_BYTES >> 4)), db0 + (uint64_t)(2 * j), idesc, acc);
                    acc = 1;
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
        // ================= epilogue warps =================
        // Thread (q, lane) owns W column n = my_n + 32 q + lane (tensor-memory lane 32 q + lane); the accumulator's
        // columns are the tile's tokens.  The two warps of a lane quarter split the token columns between them.
        const int ew = warp - 2, q = warp & 3, ch = ew >> 2;
        epi_ok = mbar_wait(bar_tfull, 0, abort_word, 46);
        epi_ok = __all_sync(0xffffffffu, epi_ok);
        tc_fence_after();
        const uint32_t tl = tmem_base + ((uint32_t)(q * 32) << 16);
        uint8_t* stg = smem + ew * 2048;            // the pipeline stages are free: every MMA of the pair has completed
        const int ncol = my_n + q * 32;             // first W column of this warp
        // 32 tokens x this warp's 32 columns, fp32 in registers (one column per thread) -> bf16 rows of y
        auto store_chunk = [&](const float (&v)[32], int tok0) {
#pragma unroll
            for (int j = 0; j < 32; ++j) reinterpret_cast<bf16*>(stg)[j * 32 + lane] = __float2bfloat16_rn(v[j]);
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int tk = i * 8 + (lane >> 2), sg = lane & 3;
                const uint4 o = *reinterpret_cast<const uint4*>(stg + tk * 64 + sg * 16);
                const int tok = tok0 + tk, col = ncol + sg * 8;
                if (tok < g.T && col < g.Nout) *reinterpret_cast<uint4*>(g.C + (size_t)tok * g.ldc + col) = o;
            }
            __syncwarp();
        };
        if (g.S == 1) {
            if (epi_ok) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t v[32];
                    tc_ld_32x32(tl + ch * 128 + c * 32, v);
                    tc_wait_ld();
                    float f[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
                    store_chunk(f, m0 + ch * 128 + c * 32);
                }
            }
        } else {
            // ---- level 1: the cluster's two pairs (slices 2 cs and 2 cs + 1) exchange token halves through
            // distributed shared memory.  Pair pi keeps tokens [128 pi, 128 pi + 128) and sends the other half to the
            // CTA of the other pair that stages the same W columns, thread to thread ([column group][lane] 16-byte
            // slots).  The mailbox is dedicated memory, so nobody waits before sending.
            const int keep = (int)pi, send = 1 - keep;
            if (epi_ok) {
                const uint32_t dst = dk_map_to_cta(sMbox, crank ^ 2u) + (uint32_t)(q * 32 + lane) * 16u;
#pragma unroll 1
                for (int e = 0; e < 2; ++e) {
                    uint32_t v[32];
                    tc_ld_32x32(tl + send * 128 + ch * 64 + e * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int gq = 0; gq < 8; ++gq)
                        dk_st_cluster_v4(dst + (uint32_t)((ch * 2 + e) * 8 + gq) * 2048u, v[4 * gq], v[4 * gq + 1], v[4 * gq + 2],
                                         v[4 * gq + 3]);
                }
            }
            mbar_arrive_remote_release(dk_map_to_cta(bar_mbox, crank ^ 2u));      // also on abort: the partner must not wait
            {
                bool ok = true;
                if (!mbar_try_wait_cluster(bar_mbox, 0)) {
                    unsigned long long t0 = 0;
                    uint32_t spins = 0;
                    while (!mbar_try_wait_cluster(bar_mbox, 0)) {
                        if (((++spins) & 255u) == 0) {
                            if (*abort_word != 0) { ok = false; break; }
                            const unsigned long long now = global_ns();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > WAIT_LIMIT_NS) { atomicCAS((int*)abort_word, 0, 47); ok = false; break; }
                        }
                    }
                }
                epi_ok = __all_sync(0xffffffffu, epi_ok && ok);
            }
            if (epi_ok) {
                const uint32_t mb = sMbox + (uint32_t)(q * 32 + lane) * 16u;
                // sum of the two slices of this cluster for 32 token columns (fp32 addition commutes, so both pairs
                // form the same bits whichever of them adds)
                auto level1 = [&](int e, float (&f)[32]) {
                    uint32_t v[32];
                    tc_ld_32x32(tl + keep * 128 + ch * 64 + e * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int gq = 0; gq < 8; ++gq) {
                        float4 p;
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(p.x), "=f"(p.y), "=f"(p.z), "=f"(p.w)
                                     : "r"(mb + (uint32_t)((ch * 2 + e) * 8 + gq) * 2048u));
                        f[4 * gq] = __uint_as_float(v[4 * gq]) + p.x;
                        f[4 * gq + 1] = __uint_as_float(v[4 * gq + 1]) + p.y;
                        f[4 * gq + 2] = __uint_as_float(v[4 * gq + 2]) + p.z;
                        f[4 * gq + 3] = __uint_as_float(v[4 * gq + 3]) + p.w;
                    }
                };
                const int tok_keep = m0 + keep * 128 + ch * 64;
                if (g.S == 2) {
#pragma unroll 1
                    for (int e = 0; e < 2; ++e) {
                        float f[32];
                        level1(e, f);
                        store_chunk(f, tok_keep + e * 32);
                    }
                } else {
                    // ---- level 2: the tile's two clusters (slices {0,1} and {2,3}) exchange token quarters through
                    // global memory: cluster cs finishes chunk cs of each warp's 64 columns and sends the other chunk,
                    // thread to thread, to the same CTA and warp of the other cluster.
                    const int slot_out = ((tile * 2 + (1 - cs)) * 4 + (int)crank) * 8 + ew;
                    const int slot_in = ((tile * 2 + cs) * 4 + (int)crank) * 8 + ew;
                    {
                        float f[32];
                        level1(1 - cs, f);
                        float* o = g.xbuf + (size_t)slot_out * 1024 + lane * 4;
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq)
                            *reinterpret_cast<float4*>(o + gq * 128) = make_float4(f[4 * gq], f[4 * gq + 1], f[4 * gq + 2], f[4 * gq + 3]);
                        __syncwarp();
                        if (lane == 0) st_release_gpu(g.sync + SY_FLAGS + slot_out, 1);
                    }
                    float f[32];
                    level1(cs, f);
                    bool ok = true;
                    if (lane == 0) ok = wait_word_ge(g.sync + SY_FLAGS + slot_in, 1, abort_word, 48);
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (ok) {
                        const float* in = g.xbuf + (size_t)slot_in * 1024 + lane * 4;
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) {
                            const uint4 p = ld_cg_v4(in + gq * 128);
                            f[4 * gq] += __uint_as_float(p.x);
                            f[4 * gq + 1] += __uint_as_float(p.y);
                            f[4 * gq + 2] += __uint_as_float(p.z);
                            f[4 * gq + 3] += __uint_as_float(p.w);
                        }
                        store_chunk(f, tok_keep + cs * 32);
                    }
                }
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    tc_fence_before();
    dk_cluster_sync();      // the cluster leaves together (barriers, mailboxes and tensor memory are shared)
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
    if (g.reset_at_end && threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(g.sync + SY_EXIT, 1) == (int)gridDim.x - 1) {
            for (int i = 0; i < g.n_flags; ++i) g.sync[SY_FLAGS + i] = 0;
            g.sync[SY_TICKET] = 0;
            g.sync[SY_DONE] = 0;
            __threadfence();
            g.sync[SY_EXIT] = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------------------------
// k_decode_shrink
// ---------------------------------------------------------------------------------------------------------------
constexpr int SH_THREADS = 288;        // warp 0: producer (work units, bulk copies), warps 1..8: MMA + output
constexpr int SH_CONS = 8;
constexpr int SH_KC = 512;             // elements of the contraction per pipeline stage
constexpr int SH_PITCH = SH_KC * 2 + 16;     // bytes between staged rows: 16 B of padding keeps ldmatrix conflict-free
constexpr int SH_RG = 32;              // ranks per streaming group
constexpr int SH_PASS = 16;            // tokens per pass (one m16 MMA tile)
constexpr int SH_MAX_T = 1024;
constexpr int SH_TABLE_SMEM = 1032;    // the segment table is staged in shared memory when S + 1 <= this

struct ShrinkStageMeta {
    int t;              // tenant slot; == cap: tokens routed to no adapter
    int jg0, rg;        // first rank and number of ranks (16 or 32) of this streaming group; rg == 0: nothing to compute
    int np;             // tokens of the pass
    int kel;            // elements of the contraction in this stage
    int first_chunk, last_chunk;    // of the (pass, rank group)
    int pass_first;     // first stage of the pass: the pass's rows of hd / h are cleared outside the tenant's columns
    int unit_last;      // last stage of the work unit
    int stop;           // no more work
    int rpt;            // tenant's rank rounded up to 16
    float scale;
    int tok[SH_PASS];
};

struct DecodeShrinkArgs {
    int T, K, RP, cap;
    int S;                              // segments; < 0: tok_slot already holds the per-token slots
    int G;                              // work units per tenant: unit (t, i) takes the tenant's 16-token passes i, i + G, ...
    int n_units;                        // (cap + 1) * G
    int nbuf;                           // pipeline stages
    int n_flags;                        // exchange flags of the GEMM to clear at the end
    int reset_at_end;                   // normal order (GEMM grid first): this grid ends last and clears counters and flags
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
    int32_t* sync;
};

static size_t decode_shrink_stage_bytes(int RP) { return (size_t)(SH_PASS + std::min(RP, SH_RG)) * SH_PITCH; }
static size_t decode_shrink_fixed_smem(int64_t T, int32_t S) {
    const size_t Tp = (size_t)((T + 31) / 32 * 32);
    const bool staged = S >= 0 && S + 1 <= SH_TABLE_SMEM;
    return 1024 /* alignment */ + 4 * (2 * Tp + (staged ? (size_t)(2 * S + 1) : 0)) + 16 +
           sizeof(float) * 2 * SH_CONS * SH_PASS * SH_RG + 8 * sizeof(ShrinkStageMeta) + 256;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Work unit u = (tenant t = u / G, share i = u % G): the tenant's tokens in ascending order are cut into passes of 16,
// and the unit takes passes i, i + G, ...  For each pass and each group of up to 32 ranks the token rows of x and the
// adapter rows of At stream through shared memory in 512-deep stages (one bulk copy per row, issued by the lanes of the
// producer warp); the eight consumer warps take the 16-deep slices of a stage in turn (m16n8k16 fragments by ldmatrix)
// and their partial products are added in warp order.  Nothing here depends on which CTA takes which unit.
__global__ void __launch_bounds__(SH_THREADS, 1) k_decode_shrink(const DecodeShrinkArgs g) {
    extern __shared__ uint8_t sh_raw[];
    uint8_t* sh = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(sh_raw) + 1023) & ~uintptr_t(1023));
    const int Tp = (g.T + 31) / 32 * 32;
    const bool staged_tab = g.S >= 0 && g.S + 1 <= SH_TABLE_SMEM;
    const size_t stage_bytes = (size_t)(SH_PASS + min(g.RP, SH_RG)) * SH_PITCH;
    uint8_t* bufs = sh;                                                  // [nbuf][rows][SH_PITCH]
    float* red = reinterpret_cast<float*>(sh + (size_t)g.nbuf * stage_bytes);       // [2][8 warps][16 tokens][32 ranks]
    ShrinkStageMeta* metas = reinterpret_cast<ShrinkStageMeta*>(red + 2 * SH_CONS * SH_PASS * SH_RG);
    uint64_t* bars = reinterpret_cast<uint64_t*>(metas + 8);
    int32_t* s_slot = reinterpret_cast<int32_t*>(bars + 16);            // [Tp]
    int32_t* s_list = s_slot + Tp;                                      // [Tp] producer's token list of the current unit
    int32_t* s_off = s_list + Tp;                                       // [S + 1] staged table
    int32_t* s_stab = s_off + (staged_tab ? g.S + 1 : 0);
    volatile int* abort_word = reinterpret_cast<volatile int*>(bars + 16) - 1;
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 64;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    dk_launch_dependents();     // whatever follows this call in the stream may be scheduled; it waits for this grid's end
    if (tid == 0) {
        for (int s = 0; s < g.nbuf; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, SH_CONS);
        }
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    // ---- per-token slot (every CTA, redundantly: the table is tiny) ---------------------------------------------
    if (g.S >= 0) {
        if (staged_tab) {
            for (int s = tid; s <= g.S; s += SH_THREADS) {
                s_off[s] = g.seg_offsets[s];
                if (s < g.S) s_stab[s] = g.seg_slot[s];
            }
            __syncthreads();
        }
        if (blockIdx.x == 0) {
            for (int s = tid; s < g.S; s += SH_THREADS) {
                const int a = staged_tab ? s_off[s] : g.seg_offsets[s], b = staged_tab ? s_off[s + 1] : g.seg_offsets[s + 1];
                if (b < a || a < 0 || b > g.T) dk_report(g.status, DEV_BAD_TABLE, s);
                if (s == 0 && a != 0) dk_report(g.status, DEV_BAD_TABLE, -1);
                if (s == g.S - 1 && b != g.T) dk_report(g.status, DEV_BAD_TABLE, -2);
            }
            if (tid == 0 && g.S == 0 && g.T != 0) dk_report(g.status, DEV_BAD_TABLE, -3);
        }
        for (int i = tid; i < g.T; i += SH_THREADS) {
            int lo = 0, hi = g.S;
            while (lo < hi) {       // first s with seg_offsets[s + 1] > i
                const int mid = (lo + hi) >> 1;
                const int v = staged_tab ? s_off[mid + 1] : g.seg_offsets[mid + 1];
                if (v > i) hi = mid; else lo = mid + 1;
            }
            s_slot[i] = lo < g.S ? (staged_tab ? s_stab[lo] : g.seg_slot[lo]) : -1;
        }
    } else {
        for (int i = tid; i < g.T; i += SH_THREADS) s_slot[i] = g.tok_slot[i];
    }
    __syncthreads();
    for (int i = tid; i < g.T; i += SH_THREADS) {
        int s = s_slot[i];
        if (s < -1 || s >= g.cap) {
            if (blockIdx.x == 0) dk_report(g.status, DEV_BAD_INDEX, i);
            s = -1;
        }
        s_slot[i] = s;
        if (blockIdx.x == 0) g.tok_slot[i] = s;
    }
    __syncthreads();

    if (warp == 0) {
        // ================= producer =================
        uint32_t s = 0, ph = 0;
        bool ok = true;
        // one stage: wait for its buffer, publish its description, then one bulk copy per row
        auto emit = [&](const ShrinkStageMeta& m, int p0, int k0) {
            if (!ok) return;
            bool w = true;
            if (lane == 0) w = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 51);
            ok = __shfl_sync(0xffffffffu, (int)w, 0) != 0;
            if (!ok) return;
            ShrinkStageMeta* d = metas + s;
            if (lane == 0) {
                d->t = m.t; d->jg0 = m.jg0; d->rg = m.rg; d->np = m.np; d->kel = m.kel; d->first_chunk = m.first_chunk;
                d->last_chunk = m.last_chunk; d->pass_first = m.pass_first; d->unit_last = m.unit_last; d->stop = m.stop;
                d->rpt = m.rpt; d->scale = m.scale;
            }
            if (lane < SH_PASS) d->tok[lane] = lane < m.np ? s_list[p0 + lane] : -1;
            __syncwarp();
            const int nrows = m.rg > 0 ? m.np + m.rg : 0;
            const uint32_t rowbytes = (uint32_t)m.kel * 2u;
            if (lane == 0) mbar_expect_tx(bar_full + 8 * s, (uint32_t)nrows * rowbytes);
            __syncwarp();
            uint8_t* buf = bufs + (size_t)s * stage_bytes;
            for (int r = lane; r < nrows; r += 32) {
                const bf16* src;
                uint32_t dst;
                if (r < m.np) {
                    src = g.x + (size_t)s_list[p0 + r] * g.ldx + k0;
                    dst = smem_u32(buf + (size_t)r * SH_PITCH);
                } else {
                    src = g.At + ((size_t)m.t * g.RP + m.jg0 + (r - m.np)) * g.K + k0;
                    dst = smem_u32(buf + (size_t)(SH_PASS + r - m.np) * SH_PITCH);
                }
                bulk_load_row(dst, src, rowbytes, bar_full + 8 * s);
            }
            if (++s == (uint32_t)g.nbuf) { s = 0; ph ^= 1; }
        };
        while (ok) {
            int u = 0;
            if (lane == 0) u = atomicAdd(g.sync + SY_TICKET, 1);
            u = __shfl_sync(0xffffffffu, u, 0);
            if (u >= g.n_units) break;
            const int t = u / g.G, gi = u % g.G;
            // the unit's tokens: token number e of the tenant (ascending) belongs to pass e / 16
            int seen = 0, mine = 0;
            for (int i0 = 0; i0 < g.T; i0 += 32) {
                const int i = i0 + lane;
                bool m = false;
                if (i < g.T) {
                    const int sl = s_slot[i];
                    m = t < g.cap ? sl == t : sl < 0;
                }
                const unsigned bal = __ballot_sync(0xffffffffu, m);
                const int e = seen + __popc(bal & ((1u << lane) - 1u));
                const bool take = m && ((e / SH_PASS) % g.G) == gi;
                const unsigned balt = __ballot_sync(0xffffffffu, take);
                if (take) s_list[mine + __popc(balt & ((1u << lane) - 1u))] = i;
                seen += __popc(bal);
                mine += __popc(balt);
            }
            __syncwarp();
            if (mine == 0) {
                if (lane == 0) atomicAdd(g.sync + SY_DONE, 1);
                continue;
            }
            const int r_t = t < g.cap ? g.d_rank[t] : 0;
            ShrinkStageMeta m;
            m.t = t; m.stop = 0;
            m.rpt = (r_t + 15) & ~15;
            m.scale = t < g.cap ? g.d_scale[t] : 0.f;
            const int ngroups = (m.rpt + SH_RG - 1) / SH_RG;
            const int nchunk = (g.K + SH_KC - 1) / SH_KC;
            for (int p0 = 0; p0 < mine && ok; p0 += SH_PASS) {
                m.np = min(SH_PASS, mine - p0);
                const bool last_pass = p0 + SH_PASS >= mine;
                if (ngroups == 0) {
                    m.jg0 = 0; m.rg = 0; m.kel = 0; m.first_chunk = 1; m.last_chunk = 1; m.pass_first = 1; m.unit_last = last_pass;
                    emit(m, p0, 0);
                    continue;
                }
                for (int jg = 0; jg < ngroups && ok; ++jg) {
                    m.jg0 = jg * SH_RG;
                    m.rg = min(SH_RG, m.rpt - m.jg0);
                    for (int c = 0; c < nchunk && ok; ++c) {
                        m.kel = min(SH_KC, g.K - c * SH_KC);
                        m.first_chunk = c == 0;
                        m.last_chunk = c == nchunk - 1;
                        m.pass_first = jg == 0 && c == 0;
                        m.unit_last = last_pass && jg == ngroups - 1 && m.last_chunk;
                        emit(m, p0, c * SH_KC);
                    }
                }
            }
        }
        {
            ShrinkStageMeta m;
            m.t = 0; m.jg0 = 0; m.rg = 0; m.np = 0; m.kel = 0; m.first_chunk = 0; m.last_chunk = 0; m.pass_first = 0; m.unit_last = 0;
            m.stop = 1; m.rpt = 0; m.scale = 0.f;
            emit(m, 0, 0);
        }
        if (!ok && lane == 0) {
            // the consumers may be waiting for a stage that will never come: they poll the abort word and leave.  Let the
            // copies already issued land (bounded) before shared memory is released.
            for (int j = 0; j < g.nbuf; ++j) {
                const unsigned long long t0 = global_ns();
                (void)j;
                while (global_ns() - t0 < 20000ull) {
                }
            }
        }
    } else {
        // ================= consumers =================
        const int cw = warp - 1, ctid = tid - 32;
        const int gq = lane >> 2, tq = lane & 3;
        uint32_t s = 0, ph = 0, par = 0;
        float acc[SH_RG / 8][4];
        while (true) {
            if (!mbar_wait(bar_full + 8 * s, ph, abort_word, 52)) break;
            const ShrinkStageMeta m = metas[s];
            if (m.stop) break;
            const uint8_t* buf = bufs + (size_t)s * stage_bytes;
            if (m.first_chunk) {
#pragma unroll
                for (int a = 0; a < SH_RG / 8; ++a) acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
            }
            if (m.pass_first) {
                // clear the pass's rows of hd outside the tenant's own columns, and h beyond its padded rank: two rows per warp
                const int own0 = m.rpt > 0 ? m.t * g.RP : 0, own1 = own0 + m.rpt;
                for (int rr = cw; rr < m.np; rr += SH_CONS) {
                    const int tok = m.tok[rr];
                    bf16* row = g.hd + (size_t)tok * g.hd_cols;
                    for (int c = lane * 8; c < g.hd_cols; c += 256)
                        if (c < own0 || c >= own1) *reinterpret_cast<uint4*>(row + c) = make_uint4(0u, 0u, 0u, 0u);
                    for (int j = m.rpt + lane; j < g.RP; j += 32) g.h_out[(size_t)tok * g.RP + j] = 0.f;
                }
            }
            if (m.rg > 0) {
                const uint32_t xb = smem_u32(buf), ab = xb + SH_PASS * SH_PITCH;
                const uint32_t x_lane = xb + (uint32_t)(((lane & 7) + ((lane >> 3) & 1) * 8) * SH_PITCH + (lane >> 4) * 16);
                const uint32_t a_lane = ab + (uint32_t)(((lane & 7) + ((lane >> 4) & 1) * 8) * SH_PITCH + ((lane >> 3) & 1) * 16);
                const int nk16 = m.kel >> 4;
                for (int ks = cw; ks < nk16; ks += SH_CONS) {
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(x_lane + ks * 32, a0, a1, a2, a3);
#pragma unroll
                    for (int jj = 0; jj < SH_RG / 16; ++jj) {
                        if (jj * 16 < m.rg) {
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4(a_lane + jj * 16 * SH_PITCH + ks * 32, b0, b1, b2, b3);
                            mma_bf16_16816(acc[2 * jj], a0, a1, a2, a3, b0, b1);
                            mma_bf16_16816(acc[2 * jj + 1], a0, a1, a2, a3, b2, b3);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * s);
            if (m.last_chunk && m.rg > 0) {
                // warp partials -> sum in warp order -> h (fp32) and the tenant's columns of hd
                float* rp = red + (size_t)par * SH_CONS * SH_PASS * SH_RG;
                float* wp = rp + cw * SH_PASS * SH_RG;
#pragma unroll
                for (int a = 0; a < SH_RG / 8; ++a) {
                    if (a * 8 < m.rg) {
                        wp[gq * SH_RG + a * 8 + 2 * tq] = acc[a][0];
                        wp[gq * SH_RG + a * 8 + 2 * tq + 1] = acc[a][1];
                        wp[(gq + 8) * SH_RG + a * 8 + 2 * tq] = acc[a][2];
                        wp[(gq + 8) * SH_RG + a * 8 + 2 * tq + 1] = acc[a][3];
                    }
                }
                bar_consumers();
                for (int e = ctid; e < SH_PASS * m.rg; e += SH_CONS * 32) {
                    const int i = e / m.rg, j = e - i * m.rg;
                    if (i < m.np) {
                        float v = 0.f;
#pragma unroll
                        for (int w = 0; w < SH_CONS; ++w) v += rp[w * SH_PASS * SH_RG + i * SH_RG + j];      // fixed order
                        const int tok = m.tok[i];
                        g.h_out[(size_t)tok * g.RP + m.jg0 + j] = v;
                        g.hd[(size_t)tok * g.hd_cols + m.t * g.RP + m.jg0 + j] = __float2bfloat16_rn(m.scale * v);
                    }
                }
                par ^= 1;
            }
            if (m.unit_last) {
                __threadfence();
                bar_consumers();
                if (ctid == 0) atomicAdd(g.sync + SY_DONE, 1);
            }
            if (++s == (uint32_t)g.nbuf) { s = 0; ph ^= 1; }
        }
    }

    // ---- end: this grid completes after the GEMM grid; the last CTA to get here clears the counters and flags -------
    __syncthreads();
    if (tid == 0) {
        if (*abort_word != 0 && atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
        dk_wait_prerequisites();
        __threadfence();
        if (g.reset_at_end && atomicAdd(g.sync + SY_EXIT, 1) == (int)gridDim.x - 1) {
            for (int i = 0; i < g.n_flags; ++i) g.sync[SY_FLAGS + i] = 0;
            g.sync[SY_TICKET] = 0;
            g.sync[SY_DONE] = 0;
            __threadfence();
            g.sync[SY_EXIT] = 0;
        }
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
namespace {

struct DecodeShape {
    int S;          // contraction slices per tile
    int clusters;   // GEMM clusters
    int csz;        // CTAs per cluster
    bool ok;
};

// Largest number of co-resident clusters of `csz` CTAs of the GEMM kernel with `smem` bytes each (cached per device).
marlaas_status_t decode_max_clusters(int device, int csz, size_t smem, int* out) {
    static int cache[64][2] = {};
    const int ci = csz == 2 ? 0 : 1;
    if (device >= 0 && device < 64 && cache[device][ci] != 0) {
        *out = cache[device][ci];
        return MARLAAS_OK;
    }
    MARLAAS_CUDA_TRY(cudaFuncSetAttribute(sm100::k_decode_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    cudaLaunchConfig_t qc = {};
    qc.gridDim = dim3((unsigned)(csz * 64));
    qc.blockDim = dim3(sm100::DG_THREADS);
    qc.dynamicSmemBytes = smem;
    cudaLaunchAttribute qa;
    qa.id = cudaLaunchAttributeClusterDimension;
    qa.val.clusterDim.x = (unsigned)csz; qa.val.clusterDim.y = 1; qa.val.clusterDim.z = 1;
    qc.attrs = &qa; qc.numAttrs = 1;
    int mc = 0;
    MARLAAS_CUDA_TRY(cudaOccupancyMaxActiveClusters(&mc, sm100::k_decode_gemm, &qc));
    if (mc < 1) mc = -1;
    if (device >= 0 && device < 64) cache[device][ci] = mc;
    *out = mc;
    return MARLAAS_OK;
}

constexpr int DECODE_MIN_SHRINK_SMS = 8;       // SMs the GEMM's grid must leave to the shrink grid
constexpr int DECODE_MAX_SHRINK_CTAS = 20;

// Slices per tile: as many as fill the SMs with one wave of clusters while leaving room for the shrink grid.  Uses only
// the pool's dimensions and the SM count, so that the workspace size and the launch agree.
DecodeShape decode_shape(const marlaas_pool* pool, int64_t T) {
    DecodeShape d = {1, 0, 2, false};
    const int64_t tiles = cdiv(T, sm100::DG_TN) * cdiv(pool->N, sm100::DG_TM);
    const int64_t num_ks = pool->K / sm100::BK;
    const int room = pool->sm_count - DECODE_MIN_SHRINK_SMS;
    // clusters of 4 pack less densely than pairs: 33 are co-resident on a 148-SM part (the launch checks the real figure)
    const int mc4 = (pool->sm_count - 16) / 4;
    if (num_ks >= 4 && tiles * 2 <= mc4 && tiles * 8 <= room) { d.S = 4; d.clusters = (int)tiles * 2; d.csz = 4; d.ok = true; }
    else if (num_ks >= 2 && tiles <= mc4 && tiles * 4 <= room) { d.S = 2; d.clusters = (int)tiles; d.csz = 4; d.ok = true; }
    else if (tiles * 2 <= room) { d.S = 1; d.clusters = (int)tiles; d.csz = 2; d.ok = true; }
    return d;
}

}  // namespace

bool decode_sm100_eligible(const marlaas_pool* pool, int64_t T) {
    if (!(T > 0 && T <= sm100::SH_MAX_T && (int64_t)pool->cap * pool->RP <= 2048 && pool->sm_count >= 16 && (pool->K % 64) == 0))
        return false;
    return decode_shape(pool, T).ok;
}

size_t decode_sm100_xbuf_bytes(const marlaas_pool* pool, int64_t T) {
    if (!decode_sm100_eligible(pool, T)) return 0;
    const DecodeShape d = decode_shape(pool, T);
    return d.S == 4 ? (size_t)(d.clusters / 2) * 2 * 4 * 8 * 4096 : 0;
}

marlaas_status_t launch_decode_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                     int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                     const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st, bool serial) {
    using namespace sm100;
    const int64_t K = pool->K, N = pool->N;
    const int hd_cols = (int)align_up((size_t)pool->cap * pool->RP, 64);     // pitch of hd: whole 64-deep panels
    const DecodeShape shape = decode_shape(pool, T);

    int last_used = -1;
    for (int s = 0; s < pool->cap; ++s)
        if (pool->slots[s].used && pool->slots[s].rank > 0) last_used = s;

    // ---- GEMM with the expand as extra steps of the contraction ----
    DecodeGemmArgs g;
    g.T = (int)T; g.Nout = (int)N;
    g.C = y; g.ldc = ldy; g.status = pool->d_status; g.sync = pool->d_sync; g.xbuf = ws.xbuf;
    g.S = shape.S;
    g.nstrips = (int)cdiv(N, DG_TM);
    g.num_ks = (int)(K / BK);
    g.num_xs = (int)cdiv((int64_t)(last_used + 1) * pool->RP, (int64_t)BK);
    g.w3d = (N % 64) == 0;
    constexpr size_t stage_bytes = 2 * CHUNK_BYTES + A_STAGE_BYTES;
    const size_t fixed = 1024 + (g.S > 1 ? DG_MBOX_BYTES : 0) + 512;
    g.stages = (int)std::min<size_t>(7, ((size_t)227 * 1024 - fixed) / stage_bytes);
    const size_t gemm_smem = fixed + (size_t)g.stages * stage_bytes;
    int mc = 0;
    marlaas_status_t rc;
    if ((rc = decode_max_clusters(pool->device, shape.csz, gemm_smem, &mc)) != MARLAAS_OK) return rc;
    if (mc < shape.clusters)
        return fail(MARLAAS_ERR_UNSUPPORTED_DEVICE, "lora_forward: %d clusters of %d CTAs are not co-resident on this device (%d are)",
                    shape.clusters, shape.csz, mc);

    // ---- shrink: work units (tenant, share) handed to the CTAs that fit beside the GEMM's clusters ----
    DecodeShrinkArgs a;
    a.T = (int)T; a.K = (int)K; a.RP = pool->RP; a.cap = pool->cap;
    a.S = S; a.seg_offsets = seg_offsets; a.seg_slot = seg_slot;
    a.x = x; a.ldx = ldx; a.At = pool->d_At; a.d_rank = pool->d_rank; a.d_scale = pool->d_scale;
    a.tok_slot = ws.tok_slot; a.h_out = h_out; a.hd = ws.hd; a.hd_cols = hd_cols; a.status = pool->d_status; a.sync = pool->d_sync;
    const int shrink_ctas = std::max(1, std::min(DECODE_MAX_SHRINK_CTAS, pool->sm_count - shape.clusters * shape.csz));
    const int passes = (int)cdiv(T, SH_PASS);
    a.G = std::max(1, std::min(passes, (2 * shrink_ctas + pool->cap) / (pool->cap + 1)));
    a.n_units = (pool->cap + 1) * a.G;
    a.n_flags = g.S == 4 ? shape.clusters * 4 * 8 : 0;
    a.reset_at_end = serial ? 0 : 1;
    g.n_flags = a.n_flags;
    g.reset_at_end = serial ? 1 : 0;
    const size_t sh_fixed = decode_shrink_fixed_smem(T, S), sh_stage = decode_shrink_stage_bytes(pool->RP);
    a.nbuf = (int)std::min<size_t>(6, ((size_t)200 * 1024 - sh_fixed) / sh_stage);
    // at least 120 KB, so that two of these CTAs never share an SM (and none fits beside a GEMM CTA)
    const size_t shrink_smem = std::max<size_t>(sh_fixed + (size_t)a.nbuf * sh_stage, 120 * 1024);
    g.n_units = a.n_units;

    alignas(64) CUtensorMap tmW, tmX, tmXW, tmXX;
    if ((rc = make_panel_map(&tmX, x, T, K, ldx, 1, 128)) != MARLAAS_OK) return rc;
    if (g.w3d) rc = make_panel_map(&tmW, W, K, N, ldw, 2, BK);
    else rc = make_map(&tmW, W, K, N, ldw, 64, BK);
    if (rc != MARLAAS_OK) return rc;
    if (g.num_xs > 0) {
        if ((rc = make_panel_map(&tmXX, ws.hd, T, hd_cols, hd_cols, 1, 128)) != MARLAAS_OK) return rc;
        if (g.w3d) rc = make_panel_map(&tmXW, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, N, 2, BK);
        else rc = make_map(&tmXW, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, N, 64, BK);
        if (rc != MARLAAS_OK) return rc;
    } else {
        tmXX = tmX;
        tmXW = tmW;
    }

    static bool attrs_set[64] = {};
    if (pool->device >= 64 || !attrs_set[pool->device]) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_shrink, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        if (pool->device < 64) attrs_set[pool->device] = true;
    }
    // Normal order: the GEMM grid first (its clusters take the SMs they need), the shrink grid as its programmatic
    // dependent on the SMs left over; the two run side by side and the GEMM's expand steps wait for the shrink's work-unit
    // count.  Serial order (for tools that run one kernel at a time): the shrink grid, then the GEMM grid, plainly ordered.
    auto launch_gemm = [&]() -> marlaas_status_t {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(shape.clusters * shape.csz));
        cfg.blockDim = dim3(DG_THREADS);
        cfg.dynamicSmemBytes = gemm_smem;
        cfg.stream = st;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)shape.csz; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = serial ? 1 : 2;
        MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_gemm, tmW, tmX, tmXW, tmXX, g));
        count_launch();
        return MARLAAS_OK;
    };
    auto launch_shrink = [&]() -> marlaas_status_t {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)shrink_ctas);
        cfg.blockDim = dim3(SH_THREADS);
        cfg.dynamicSmemBytes = shrink_smem;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = serial ? 0 : 1;
        MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_shrink, a));
        count_launch();
        return MARLAAS_OK;
    };
    if (serial) {
        if ((rc = launch_shrink()) != MARLAAS_OK) return rc;
        if ((rc = launch_gemm()) != MARLAAS_OK) return rc;
    } else {
        if ((rc = launch_gemm()) != MARLAAS_OK) return rc;
        if ((rc = launch_shrink()) != MARLAAS_OK) return rc;
    }
    return MARLAAS_OK;
}

}  // namespace marlaas
