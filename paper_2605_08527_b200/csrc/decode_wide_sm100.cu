// Decode-shaped forward over a LARGE weight (a 7B decoder's gate / up / down projections, or q + k + v side by side):
// at most 1024 tokens, typically one per sequence, tenants unsorted.  The call is bound by the one pass over W from HBM.
//
//   k_decode_shrink      (the kernel of decode_sm100.cu)  h_i = x_i A_t, the expand operand hd, tok_slot.  Launched first;
//                        its small CTAs run on the SMs the GEMM's pairs leave free.
//   k_decode_gemm_wide   (tcgen05, TMA)  y^T = [W ; Bs]^T * [x | hd]^T: the base product and the expand as ONE contraction
//                        over K + cap*RP, with the operand roles swapped against the training GEMM: 256 columns of W are
//                        the M side of a cta_group::2 MMA (128 per CTA, read as an MN-major A operand straight from the
//                        row-major weight), the 256 tokens its N side (128 per CTA).  A 64-deep step brings as many bytes
//                        of W as of x into a CTA (16 KB each), and one MMA covers 256 x 256 outputs, so the single
//                        MMA-issuing thread is not the limit.  Launched as a programmatic dependent of the shrink: it
//                        streams W at once and waits for the shrink grid only before its first read of hd.  A batch of
//                        fewer than 256 tokens whose contraction is not cut runs with token tiles of 64, 128 or 192 (the
//                        N of the MMA): fewer token rows per step, more steps in flight, no tensor work on empty rows.
//
// With at least 33 tiles (token tile x 256-column strip) every tile's contraction stays in one CTA pair and nothing is
// exchanged.  With fewer tiles the contraction is cut into S = 2 or 4 slices and the partial accumulators meet through an
// L2-resident scratch buffer: slice j finishes token columns [256 j / S, 256 (j + 1) / S) and receives those columns from
// the other slices, thread to thread, in a fixed order.  That exchange costs about 5 us at S = 4 (a CTA pushes 96 KB out
// and pulls 96 KB in; distributed shared memory is no faster at about 15 bytes per clock and SM), which a long stream
// (K = 11008) can carry and a 4096 x 4096 weight cannot: such weights stay with decode_sm100.cu.  Exchange flags live in
// the pool's synchronisation area and hold an epoch that the last CTA of every call advances, so a replay of a captured
// call needs no reset from outside.
#include "sm100_ptx.cuh"
#include "sm100_cluster.cuh"

#include <algorithm>

namespace marlaas {
namespace sm100 {

// words of the pool's synchronisation area
constexpr int SY_EXIT = 2;          // CTAs that have reached their end
constexpr int SY_EPOCH = 3;         // calls completed on this pool; exchange flags of a call hold epoch + 1
constexpr int SY_FLAGS = 16;        // split-K exchange flags, one per (tile, destination slice, source, CTA, epilogue warp)

__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int32_t* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ uint4 ld_cg_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// Bounded wait for a global word (acquire): until it is >= target (eq = false) or == target (eq = true).
__device__ __forceinline__ bool wait_word(const int32_t* p, int target, bool eq, volatile int* abort_word, int site) {
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (true) {
        const int v = ld_acquire_gpu(p);
        if (eq ? v == target : v >= target) return true;
        __nanosleep(32);
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

constexpr int DK_THREADS = 320;        // warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 epilogue
constexpr int DG_TN = 256;             // tokens per tile = N of the MMA
constexpr int DG_TM = 256;             // W columns per tile = M of the MMA (128 per CTA)

struct DecodeArgs {
    int T, Nout;
    int nstrips;         // 256-column strips of W; tile = (token tile, strip)
    int num_ks;          // 64-deep pipeline steps over K
    int num_xs;          // 64-deep pipeline steps over the expand rows (up to the last slot in use)
    int S;               // contraction slices per tile: 1, 2 or 4 CTA pairs
    int tn;              // tokens per tile = N of the MMA: 256, or 64 / 128 / 192 for smaller batches whose contraction is not cut
                         // (less of every stage is token rows, less tensor work on rows that hold no token)
    int stages;
    int w3d;             // the W-side operand moves with one 3-D copy per step (N a multiple of 64), else one per chunk
    int parts;           // projections held by the pool: hd is [parts][T][..] and a strip takes the plane of its projection
    int part_end[4];     // last column + 1 of each projection
    bf16* C;
    int64_t ldc;
    float* xbuf;         // exchange buffer between the slices of a tile
    int32_t* status;
    int32_t* sync;
};

// ---------------------------------------------------------------------------------------------------------------
// Operand staging per 64-deep pipeline step and CTA:
//   Wt [2 chunks][64 k][64 n]   the CTA's 128 columns of W (or of the adapter rows Bs): MN-major A operand, 128-byte
//                               swizzle, chunks 8 KB apart
//   Xt [128 tokens][64 k]       the CTA's half of the token tile of x (or of hd): K-major B operand
// ---------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DK_THREADS, 1)
k_decode_gemm_wide(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                   const __grid_constant__ CUtensorMap tmXW, const __grid_constant__ CUtensorMap tmXX, const DecodeArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int STAGES = g.stages;
    constexpr uint32_t W_BYTES = 2 * CHUNK_BYTES;
    const int XH = g.tn / 2;                         // token rows a CTA stages: its half of the tile's tokens
    const uint32_t X_BYTES = (uint32_t)XH * 128u, STAGE_BYTES = W_BYTES + X_BYTES;
    const uint32_t sStage = smem_u32(smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;
    const uint32_t bar_drain = bar_tfull + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2);
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
    const uint32_t half = dk_cluster_ctarank();      // which 128 W columns and which 128 tokens this CTA stages
    const int gp = (int)dk_cluster_id_x();           // CTA pair
    const int tile = gp / g.S, sl = gp % g.S;        // contraction slice of this pair
    const int n0 = (tile % g.nstrips) * DG_TM;
    const int m0 = (tile / g.nstrips) * g.tn;
    const int my_n = n0 + (int)half * 128, my_tok = m0 + (int)half * XH;
    // the projection whose columns the strip lies in (constant indices: a variable one would move the arguments to local memory)
    const int part = (g.parts > 1 ? (int)(n0 >= g.part_end[0]) + (int)(g.parts > 2 && n0 >= g.part_end[1]) + (int)(g.parts > 3 && n0 >= g.part_end[2]) : 0);
    const int hd_tok = my_tok + part * g.T;          // this half's rows of the projection's plane of hd
    const int ks0 = sl * g.num_ks / g.S, ks1 = (sl + 1) * g.num_ks / g.S;
    const int xs0 = sl * g.num_xs / g.S, xs1 = (sl + 1) * g.num_xs / g.S;
    const int nbase = ks1 - ks0, nstep = nbase + (xs1 - xs0);

    // The shrink grid this kernel depends on was launched in plain stream order, so everything ordered before the call
    // is complete; only the shrink's own outputs (hd) need the wait further down.  The epoch was written by the previous
    // call on this pool.
    const int epoch1 = g.S > 1 ? ld_acquire_gpu(g.sync + SY_EPOCH) + 1 : 0;

    tc_fence_before();
    dk_cluster_sync();      // both CTAs' barriers exist before any remote arrive or TMA completion
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // bytes the two CTAs of the pair stage per step (boxes wholly outside the tensors are skipped; partly outside boxes
    // are filled with zeros and count in full)
    auto x_tx = [&](int r) -> uint32_t { return (m0 + r * XH < g.T) ? X_BYTES : 0u; };
    auto w_chunks = [&](int r) -> int { return max(0, min(2, (g.Nout - (n0 + r * 128) + 63) / 64)); };
    auto w_tx = [&](int r) -> uint32_t { const int c = w_chunks(r); return (g.w3d ? (c > 0 ? 2u : 0u) : (uint32_t)c) * CHUNK_BYTES; };
    const uint32_t stage_tx = x_tx(0) + x_tx(1) + w_tx(0) + w_tx(1);
    const int my_chunks = w_chunks((int)half);
    const bool have_rows = my_tok < g.T;

    if (warp == 0) {
        // ================= TMA producer (both CTAs) =================
        if (lane == 0) {
            uint32_t it = 0, s = 0, ph = 0;
            bool ok = true, hd_ready = false;
            const uint32_t full0 = dk_map_to_cta(bar_full, 0);
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
                    dk_wait_prerequisites();
                    fence_proxy_async_all();
                    hd_ready = true;
                }
                if (have_rows) dg_tma_pair_3d(dx, mx, full0 + 8 * s, 0, ex ? hd_tok : my_tok, step);
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
        // ================= MMA issuer (the pair's first CTA) =================
        if (lane == 0 && half == 0) {
            // fp32 accumulate, bf16 x bf16, A MN-major (W columns), B K-major (tokens), M = 256, N = 256
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(g.tn >> 3) << 17) |
                                   ((uint32_t)(DG_TM >> 4) << 24);
            const uint16_t mask = 3;
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
        // columns are the tile's tokens.  Slice j finishes token columns [j Wd, (j + 1) Wd), Wd = 256 / S; the two warps
        // of a lane quarter split each such range in halves of nch chunks of 32 columns.
        const int ew = warp - 2, q = warp & 3, ch = ew >> 2;
        // Idle until the accumulator is complete, one epilogue thread hands over to the next call: once the shrink grid
        // has completed (and with it whatever that grid was launched behind), a next call launched with
        // MARLAAS_FLAG_OVERLAP_PREVIOUS may start its shrink beside the rest of this kernel.  Every CTA does this.
        if (ew == 0 && lane == 0) {
            dk_wait_prerequisites();
            dk_launch_dependents();
        }
        __syncwarp();
        bool epi_ok = mbar_wait(bar_tfull, 0, abort_word, 46);
        epi_ok = __all_sync(0xffffffffu, epi_ok);
        tc_fence_after();
        const uint32_t tl = tmem_base + ((uint32_t)(q * 32) << 16);
        uint8_t* stg = smem + ew * 2048;            // the pipeline stages are free: every MMA of the pair has completed
        const int ncol = my_n + q * 32;             // first W column of this warp
        const int Wd = g.tn / g.S, nch = Wd / 64;   // nch: 4, 2, 1 for 256 tokens and S = 1, 2, 4; 3, 2, 1 for 192, 128, 64 tokens
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
        // exchange slot of (destination slice j, source slice s != j) for this CTA and warp: nch blocks of 4 KB, each
        // [8 column groups][32 lanes][4 floats]
        auto slot_of = [&](int j, int s) -> int {
            const int si = s < j ? s : s - 1;
            return ((((tile * g.S + j) * (g.S - 1) + si) * 2 + (int)half) * 8 + ew);
        };
        if (epi_ok && g.S > 1) {
            // ---- send: the columns the other slices finish.  All stores first, one fence, then the flags: a release
            // per destination would wait for its own stores' acknowledgements, one round trip after the other.
            for (int j = 0; j < g.S; ++j) {
                if (j == sl) continue;
                float* o = g.xbuf + (size_t)slot_of(j, sl) * nch * 1024 + lane * 4;
                for (int c = 0; c < nch; ++c) {
                    uint32_t v[32];
                    tc_ld_32x32(tl + j * Wd + ch * (Wd / 2) + c * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int gq = 0; gq < 8; ++gq)
                        *reinterpret_cast<uint4*>(o + c * 1024 + gq * 128) = make_uint4(v[4 * gq], v[4 * gq + 1], v[4 * gq + 2], v[4 * gq + 3]);
                }
            }
            __threadfence();
            __syncwarp();
            if (lane < g.S && lane != sl) st_release_gpu(g.sync + SY_FLAGS + slot_of(lane, sl), epoch1);
        }
        if (epi_ok) {
            // ---- receive and finish the own columns: own partial first, then the other slices in ascending order
            bool ok = true;
            if (g.S > 1) {
                bool mine = true;
                if (lane < g.S && lane != sl) mine = wait_word(g.sync + SY_FLAGS + slot_of(sl, lane), epoch1, true, abort_word, 48);
                ok = __all_sync(0xffffffffu, mine);
            }
            for (int c = 0; c < nch && ok; ++c) {
                uint32_t v[32];
                tc_ld_32x32(tl + sl * Wd + ch * (Wd / 2) + c * 32, v);
                float f[32];
                if (g.S == 4) {
                    // three sources: all 24 loads in flight together
                    uint4 p[3][8];
#pragma unroll
                    for (int si = 0; si < 3; ++si) {
                        const float* in = g.xbuf + (size_t)((((tile * 4 + sl) * 3 + si) * 2 + (int)half) * 8 + ew) * 1024 + lane * 4;
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) p[si][gq] = ld_cg_v4(in + gq * 128);
                    }
                    tc_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
#pragma unroll
                    for (int si = 0; si < 3; ++si)
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) {
                            f[4 * gq] += __uint_as_float(p[si][gq].x);
                            f[4 * gq + 1] += __uint_as_float(p[si][gq].y);
                            f[4 * gq + 2] += __uint_as_float(p[si][gq].z);
                            f[4 * gq + 3] += __uint_as_float(p[si][gq].w);
                        }
                } else {
                    tc_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
                    for (int s = 0; s < g.S; ++s) {
                        if (s == sl) continue;
                        const float* in = g.xbuf + (size_t)slot_of(sl, s) * nch * 1024 + c * 1024 + lane * 4;
                        uint4 p[8];
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) p[gq] = ld_cg_v4(in + gq * 128);
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) {
                            f[4 * gq] += __uint_as_float(p[gq].x);
                            f[4 * gq + 1] += __uint_as_float(p[gq].y);
                            f[4 * gq + 2] += __uint_as_float(p[gq].z);
                            f[4 * gq + 3] += __uint_as_float(p[gq].w);
                        }
                    }
                }
                store_chunk(f, m0 + sl * Wd + ch * (Wd / 2) + c * 32);
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    tc_fence_before();
    dk_cluster_sync();      // the pair leaves together (its barriers and tensor memory are shared)
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
    if (threadIdx.x == 0) dk_wait_prerequisites();   // this grid never completes before the shrink grid it depends on
    // ---- the last CTA to get here opens the next epoch of the exchange flags -----------------------------------------
    if (g.S > 1 && threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(g.sync + SY_EXIT, 1) == (int)gridDim.x - 1) {
            g.sync[SY_EPOCH] = g.sync[SY_EPOCH] + 1;
            __threadfence();
            g.sync[SY_EXIT] = 0;
        }
    }
}


// ---------------------------------------------------------------------------------------------------------------
// k_decode_gemm_stream: the same product when there are MORE tiles than CTA pairs (gate and up side by side: 86 strips
// on 74 pairs).  One tile per pair would take two rounds with the second nearly empty; instead the tiles' pipeline steps
// (64 of depth each, base steps then expand steps) are laid end to end and cut into one equal range per pair.  A pair's
// range covers the tail of one tile, possibly whole tiles, and the head of another; it works through them from the
// LAST tile to the first, so that
//   - a head piece (first steps of a tile, base steps only: needs nothing from the shrink grid) is finished early, its
//     partial accumulator pushed to an L2-resident slot while the pair's remaining steps stream on (two accumulators
//     in tensor memory: the epilogue of one piece overlaps the main loop of the next);
//   - the tail piece (last steps of a tile, expand steps included) comes last; its pair owns the tile: it adds the
//     partials of the pairs holding the tile's earlier steps in ascending pair order (fixed order: results do not depend
//     on timing) and writes y.
// A pair waits only for pairs of LOWER index.  Every wait is bounded.
// ---------------------------------------------------------------------------------------------------------------
struct StreamArgs {
    int T, Nout;
    int nstrips;         // 256-column strips of W; tile = (token tile, strip)
    int num_ks, num_xs;  // 64-deep steps over K and over the expand rows
    int nstep;           // steps per tile = num_ks + num_xs
    int total;           // steps of all tiles
    int npairs;
    int tn;              // tokens per tile = N of the MMA: 256, or 64 / 128 / 192 when the whole batch fits
    int stages;
    int w3d;
    int parts;
    int part_end[4];
    bf16* C;
    int64_t ldc;
    float* xbuf;         // [npairs][2 CTAs][8 warps][4 blocks of 4 KB]
    int32_t* status;
    int32_t* sync;
};

__device__ __forceinline__ void dk_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// The pieces of a pair's step range [g0, g1), last tile first.
struct PieceIter {
    int ge, g0, nstep;
    __device__ __forceinline__ bool next(int& tile, int& s0, int& s1) {
        if (ge <= g0) return false;
        tile = (ge - 1) / nstep;
        const int lo = max(g0, tile * nstep);
        s0 = lo - tile * nstep;
        s1 = ge - tile * nstep;
        ge = lo;
        return true;
    }
};

__global__ void __launch_bounds__(DK_THREADS, 1)
k_decode_gemm_stream(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                     const __grid_constant__ CUtensorMap tmXW, const __grid_constant__ CUtensorMap tmXX, const StreamArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int STAGES = g.stages;
    constexpr uint32_t W_BYTES = 2 * CHUNK_BYTES;
    const int XH = g.tn / 2;                         // token rows a CTA stages: its half of the tile's tokens
    const uint32_t X_BYTES = (uint32_t)XH * 128u, STAGE_BYTES = W_BYTES + X_BYTES;
    constexpr uint32_t STG_BYTES = 8 * 2048;        // epilogue staging, one 2 KB block per warp (the stages stay busy)
    const uint32_t sStage = smem_u32(smem);
    uint8_t* stg_base = smem + (size_t)STAGES * STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(stg_base + STG_BYTES);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;      // two accumulators
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 5);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t TMEM_COLS = 2 * DG_TN;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, 16);      // the eight epilogue warps of both CTAs
        }
        mbar_init(bar_drain, 1);
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
    const uint32_t half = dk_cluster_ctarank();
    const int gp = (int)dk_cluster_id_x();
    const int g0 = (int)((int64_t)gp * g.total / g.npairs), g1 = (int)((int64_t)(gp + 1) * g.total / g.npairs);
    const int epoch1 = ld_acquire_gpu(g.sync + SY_EPOCH) + 1;

    tc_fence_before();
    dk_cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================= TMA producer (both CTAs) =================
        if (lane == 0) {
            uint32_t it = 0, s = 0, ph = 0;
            bool ok = true, hd_ready = false;
            const uint32_t full0 = dk_map_to_cta(bar_full, 0);
            PieceIter pi = {g1, g0, g.nstep};
            int tile, s0, s1;
            while (ok && pi.next(tile, s0, s1)) {
                const int n0 = (tile % g.nstrips) * DG_TM, m0 = (tile / g.nstrips) * g.tn;
                const int my_n = n0 + (int)half * 128, my_tok = m0 + (int)half * XH;
                const int part = (g.parts > 1 ? (int)(n0 >= g.part_end[0]) + (int)(g.parts > 2 && n0 >= g.part_end[1]) + (int)(g.parts > 3 && n0 >= g.part_end[2]) : 0);
                const int hd_tok = my_tok + part * g.T;
                auto x_tx = [&](int r) -> uint32_t { return (m0 + r * XH < g.T) ? X_BYTES : 0u; };
                auto w_chunks = [&](int r) -> int { return max(0, min(2, (g.Nout - (n0 + r * 128) + 63) / 64)); };
                auto w_tx = [&](int r) -> uint32_t { const int c = w_chunks(r); return (g.w3d ? (c > 0 ? 2u : 0u) : (uint32_t)c) * CHUNK_BYTES; };
                const uint32_t stage_tx = x_tx(0) + x_tx(1) + w_tx(0) + w_tx(1);
                const int my_chunks = w_chunks((int)half);
                const bool have_rows = my_tok < g.T;
                for (int st = s0; st < s1 && ok; ++st, ++it) {
                    const bool ex = st >= g.num_ks;
                    const int step = ex ? st - g.num_ks : st;
                    const CUtensorMap* mw = ex ? &tmXW : &tmW;
                    const CUtensorMap* mx = ex ? &tmXX : &tmX;
                    if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 61))) break;
                    if (half == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
                    const uint32_t dw = sStage + s * STAGE_BYTES, dx = dw + W_BYTES;
                    if (g.w3d) {
                        if (my_chunks > 0) dg_tma_pair_3d(dw, mw, full0 + 8 * s, 0, step * BK, my_n >> 6);
                    } else {
                        for (int c = 0; c < my_chunks; ++c) dg_tma_pair(dw + c * CHUNK_BYTES, mw, full0 + 8 * s, my_n + c * 64, step * BK);
                    }
                    if (ex && !hd_ready) {
                        // the adapter rows above do not depend on the shrink grid; hd does
                        dk_wait_prerequisites();
                        fence_proxy_async_all();
                        hd_ready = true;
                        // the shrink grid has completed (and with it whatever it was launched behind): a next call launched
                        // with MARLAAS_FLAG_OVERLAP_PREVIOUS may start its shrink beside the rest of this kernel (here the
                        // epilogue warps are busy with early pieces, so the producer hands over)
                        dk_launch_dependents();
                    }
                    if (have_rows) dg_tma_pair_3d(dx, mx, full0 + 8 * s, 0, ex ? hd_tok : my_tok, step);
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
                }
            }
            if (ok && !hd_ready) {
                dk_wait_prerequisites();
                dk_launch_dependents();
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
        // ================= MMA issuer (the pair's first CTA) =================
        if (lane == 0 && half == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(g.tn >> 3) << 17) |
                                   ((uint32_t)(DG_TM >> 4) << 24);
            const uint16_t mask = 3;
            uint32_t s = 0, ph = 0, k = 0;
            bool ok = true;
            PieceIter pi = {g1, g0, g.nstep};
            int tile, s0, s1;
            while (ok && pi.next(tile, s0, s1)) {
                const uint32_t b = k & 1, aph = (k >> 1) & 1;
                if (!(ok = mbar_wait(bar_tempty + 8 * b, aph ^ 1, abort_word, 63))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * DG_TN;
                uint32_t acc = 0;
                for (int st = s0; st < s1 && ok; ++st) {
                    if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 64))) break;
                    tc_fence_after();
                    const uint32_t dw = sStage + s * STAGE_BYTES, dx = dw + W_BYTES;
                    const uint64_t da0 = desc_mn_major(dw, CHUNK_BYTES), db0 = desc_k_major(dx);
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        dg_mma_pair(d_tmem, da0 + (uint64_t)(j * (UNIT_BYTES >> 4)), db0 + (uint64_t)(2 * j), idesc, acc);
                        acc = 1;
                    }
                    dg_commit_pair(bar_empty + 8 * s, mask);
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
                }
                if (ok) dg_commit_pair(bar_tfull + 8 * b, mask);
                ++k;
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
        // ================= epilogue warps =================
        // Thread (q, lane) owns W column n = my_n + 32 q + lane (tensor-memory lane 32 q + lane); the accumulator's columns
        // are the tile's tokens, and warp (q, ch) takes its half of them, token columns [ch tn / 2, (ch + 1) tn / 2), in
        // chunks of 32 (four at 256 tokens a tile).
        const int ew = warp - 2, q = warp & 3, ch = ew >> 2;
        const int nchk = g.tn / 64;
        uint8_t* stg = stg_base + ew * 2048;
        const uint32_t tempty0 = dk_map_to_cta(bar_tempty, 0);
        auto slot_of = [&](int pair) -> size_t { return ((size_t)pair * 2 + half) * 8 + ew; };      // 16 KB each
        PieceIter pi = {g1, g0, g.nstep};
        int tile, s0, s1;
        uint32_t k = 0;
        bool ok = true;
        while (ok && pi.next(tile, s0, s1)) {
            const uint32_t b = k & 1, aph = (k >> 1) & 1;
            ok = mbar_wait(bar_tfull + 8 * b, aph, abort_word, 66);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int n0 = (tile % g.nstrips) * DG_TM, m0 = (tile / g.nstrips) * g.tn;
            const int ncol = n0 + (int)half * 128 + q * 32;
            const uint32_t tl = tmem_base + ((uint32_t)(q * 32) << 16) + b * DG_TN + ch * XH;
            if (s1 < g.nstep) {
                // ---- not the tile's last steps: the partial sums go to this pair's slot
                float* o = g.xbuf + slot_of(gp) * 4096 + lane * 4;
                for (int c = 0; c < nchk; ++c) {
                    uint32_t v[32];
                    tc_ld_32x32(tl + c * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int gq = 0; gq < 8; ++gq)
                        *reinterpret_cast<uint4*>(o + c * 1024 + gq * 128) = make_uint4(v[4 * gq], v[4 * gq + 1], v[4 * gq + 2], v[4 * gq + 3]);
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_gpu(g.sync + SY_FLAGS + (int)slot_of(gp), epoch1);
            } else {
                // ---- the tile's last steps: this pair owns the tile.  Earlier steps, if any, were taken by the pairs
                // pf .. gp - 1; their partial sums are added in ascending order.
                int pf = gp;
                if (s0 > 0) {
                    const int64_t gfirst = (int64_t)tile * g.nstep;
                    pf = (int)(((gfirst + 1) * g.npairs - 1) / g.total);
                    bool mine = true;
                    for (int src = pf + lane; src < gp; src += 32)
                        mine = mine && wait_word(g.sync + SY_FLAGS + (int)slot_of(src), epoch1, true, abort_word, 68);
                    ok = __all_sync(0xffffffffu, mine);
                    __syncwarp();
                    if (!ok) break;
                }
                for (int c = 0; c < nchk; ++c) {
                    uint32_t v[32];
                    tc_ld_32x32(tl + c * 32, v);
                    tc_wait_ld();
                    float f[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
                    for (int src = pf; src < gp; ++src) {
                        const float* in = g.xbuf + slot_of(src) * 4096 + c * 1024 + lane * 4;
                        uint4 p[8];
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) p[gq] = ld_cg_v4(in + gq * 128);
#pragma unroll
                        for (int gq = 0; gq < 8; ++gq) {
                            f[4 * gq] += __uint_as_float(p[gq].x);
                            f[4 * gq + 1] += __uint_as_float(p[gq].y);
                            f[4 * gq + 2] += __uint_as_float(p[gq].z);
                            f[4 * gq + 3] += __uint_as_float(p[gq].w);
                        }
                    }
                    // 32 tokens x this warp's 32 columns, fp32 in registers (one column per thread) -> bf16 rows of y
                    const int tok0 = m0 + ch * XH + c * 32;
#pragma unroll
                    for (int j = 0; j < 32; ++j) reinterpret_cast<bf16*>(stg)[j * 32 + lane] = __float2bfloat16_rn(f[j]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tk = i * 8 + (lane >> 2), sg = lane & 3;
                        const uint4 o4 = *reinterpret_cast<const uint4*>(stg + tk * 64 + sg * 16);
                        const int tok = tok0 + tk, col = ncol + sg * 8;
                        if (tok < g.T && col < g.Nout) *reinterpret_cast<uint4*>(g.C + (size_t)tok * g.ldc + col) = o4;
                    }
                    __syncwarp();
                }
            }
            // this accumulator may be overwritten by the pair's next piece but one
            tc_fence_before();
            __syncwarp();
            if (lane == 0) dk_arrive_remote(tempty0 + 8 * b);
            ++k;
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------------
    tc_fence_before();
    dk_cluster_sync();      // the pair leaves together (its barriers and tensor memory are shared)
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_word != 0) {
        if (atomicCAS(g.status, 0, DEV_TIMEOUT) == 0) g.status[1] = *abort_word * 1000000 + (int)blockIdx.x;
    }
    if (threadIdx.x == 0) dk_wait_prerequisites();   // this grid never completes before the shrink grid it depends on
    // ---- the last CTA to get here opens the next epoch of the exchange flags -----------------------------------------
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(g.sync + SY_EXIT, 1) == (int)gridDim.x - 1) {
            g.sync[SY_EPOCH] = g.sync[SY_EPOCH] + 1;
            __threadfence();
            g.sync[SY_EXIT] = 0;
        }
    }
}

}  // namespace sm100

// ---------------------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------------------
namespace {

struct DecodeShape {
    int S;          // contraction slices per tile
    int pairs;      // CTA pairs = tiles * S
    bool ok;
};

// Slices per tile: as many as fill the part with one wave of CTA pairs.  Uses only the pool's dimensions and the SM count,
// so that the workspace size and the launch agree.
DecodeShape decode_shape(const marlaas_pool* pool, int64_t T) {
    DecodeShape d = {1, 0, false};
    const int64_t tiles = cdiv(T, sm100::DG_TN) * cdiv(pool->N, sm100::DG_TM);
    const int64_t num_ks = pool->K / sm100::BK;
    const int room = pool->sm_count / 2;
    if (tiles > room) return d;
    d.S = (num_ks >= 4 && tiles * 4 <= room) ? 4 : (num_ks >= 2 && tiles * 2 <= room) ? 2 : 1;
    d.pairs = (int)tiles * d.S;
    d.ok = true;
    return d;
}

}  // namespace

// Large weights only: the stream must be long enough to carry the exchange of a split contraction (none with 33 tiles or
// more), and the shrink kernel's own limits apply.
bool decode_wide_sm100_eligible(const marlaas_pool* pool, int64_t T) {
    if (!decode_sm100_eligible(pool, T) || pool->sm_count < 32) return false;
    if ((int64_t)pool->K * pool->N * 2 < (int64_t)64 << 20) return false;
    return decode_shape(pool, T).ok;
}

// More tiles than CTA pairs (and at most 1024 tokens, a large weight, the shrink kernel's limits): the tiles' steps are
// spread evenly over all pairs (k_decode_gemm_stream).
bool decode_stream_sm100_eligible(const marlaas_pool* pool, int64_t T) {
    if (!(T > 0 && T <= 1024 && (int64_t)pool->cap * pool->RP <= 2048 && pool->sm_count >= 32 && (pool->K % 64) == 0)) return false;
    if ((int64_t)pool->K * pool->N * 2 < (int64_t)64 << 20) return false;
    const int64_t tiles = cdiv(T, sm100::DG_TN) * cdiv(pool->N, sm100::DG_TM), room = pool->sm_count / 2;
    // also where one tile per pair could only cut the contraction in two although three pairs per tile are there (a third
    // or more of the SMs would idle) and the contraction is deep enough to carry the exchange of three or four pieces
    // per tile: 17408 x 5120, 256 tokens: 68.4 against 71.1 us; 25600 x 5120: 87.2 against 95.7 us
    const bool deep_few = tiles * 4 > room && tiles * 3 <= room && pool->K / sm100::BK >= 256;
    // and for batches of up to 64 tokens over 16 to 44 tiles: partial sums of 64 tokens are cheap to pass on, and an even
    // share of the steps on every pair beats one tile per pair, cut in 1, 2 or 4 (11008 x 4096: 34.6 against 36.5 us;
    // 4096 x 8192: 27.8 against 29.9; 4096 x 11008: 31.6 against 33.3; from 48 tiles on it is no faster, then slower)
    const bool small_batch = T <= 64 && tiles >= 16 && tiles * 5 <= room * 3;
    return (tiles > room || deep_few || small_batch) && tiles * ((pool->K + pool->cap * pool->RP) / sm100::BK + 1) < (1ll << 30);
}

// Whether the one-tile-per-pair kernel would cut the contraction (and so need the exchange scratch) for this batch.
bool decode_wide_sm100_splits(const marlaas_pool* pool, int64_t T) { return decode_shape(pool, T).S > 1; }

size_t decode_wide_sm100_xbuf_bytes(const marlaas_pool* pool, int64_t T) {
    if (decode_stream_sm100_eligible(pool, T)) return (size_t)(pool->sm_count / 2) * 2 * 8 * 16384;     // a slot per pair, CTA, warp
    if (!decode_wide_sm100_eligible(pool, T)) return 0;
    const DecodeShape d = decode_shape(pool, T);
    // per tile: S destinations x (S - 1) sources x 2 CTAs x 8 warps x (256 / S / 64) blocks of 4 KB
    return d.S > 1 ? (size_t)(d.pairs / d.S) * d.S * (d.S - 1) * 2 * 8 * (256 / d.S / 64) * 4096 : 0;
}

marlaas_status_t launch_decode_wide_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                          int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                          const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st) {
    using namespace sm100;
    const int64_t K = pool->K, N = pool->N;
    const int hd_cols = (int)align_up((size_t)pool->cap * pool->RP, 64);     // pitch of hd: whole 64-deep panels
    const DecodeShape shape = decode_shape(pool, T);

    int last_used = -1;
    for (int s = 0; s < pool->cap; ++s)
        if (pool->slots[s].used && pool->slots[s].rank > 0) last_used = s;

    DecodeArgs g;
    g.T = (int)T; g.Nout = (int)N;
    g.C = y; g.ldc = ldy; g.status = pool->d_status; g.sync = pool->d_sync; g.xbuf = ws.xbuf;
    g.S = shape.S;
    g.tn = shape.S == 1 && T < DG_TN ? (int)cdiv(T, 64) * 64 : DG_TN;
    g.nstrips = (int)cdiv(N, DG_TM);
    g.num_ks = (int)(K / BK);
    g.num_xs = (int)cdiv((int64_t)(last_used + 1) * pool->RP, (int64_t)BK);
    g.w3d = (N % 64) == 0;
    g.parts = pool->P;
    for (int p = 0; p < 4; ++p) g.part_end[p] = p < pool->P ? (int)pool->part_begin[p + 1] : 0;
    const size_t stage_bytes = 2 * CHUNK_BYTES + (size_t)(g.tn / 2) * 128;
    // The shrink kernel's CTAs are spread over all SMs (two apiece) when this kernel's CTAs arrive: the pipeline takes
    // what two of them leave of an SM's 227 KB, so that neither kernel waits for the other's shared memory.
    const size_t room = (size_t)227 * 1024 - 2 * decode_shrink_smem_bytes(T, S) - 1024;
    g.stages = (int)std::max<size_t>(2, std::min<size_t>(9, (room - 1024 - 512) / stage_bytes));
    const size_t smem_bytes = 1024 + 512 + (size_t)g.stages * stage_bytes;
    if ((size_t)SY_FLAGS + (size_t)(shape.pairs / shape.S) * shape.S * (shape.S - 1) * 16 > DECODE_SYNC_BYTES / 4)
        return fail(MARLAAS_ERR_INVALID_ARG, "lora_forward: the decode path needs more exchange flags than the pool holds");

    marlaas_status_t rc;
    if ((rc = launch_decode_shrink(pool, T, x, ldx, S, seg_offsets, seg_slot, ws, h_out, st)) != MARLAAS_OK) return rc;

    alignas(64) CUtensorMap tmW, tmX, tmXW, tmXX;
    if ((rc = make_panel_map(&tmX, x, T, K, ldx, 1, (uint32_t)(g.tn / 2))) != MARLAAS_OK) return rc;
    if (g.w3d) rc = make_panel_map(&tmW, W, K, N, ldw, 2, BK);
    else rc = make_map(&tmW, W, K, N, ldw, 64, BK);
    if (rc != MARLAAS_OK) return rc;
    if (g.num_xs > 0) {
        if ((rc = make_panel_map(&tmXX, ws.hd, T * pool->P, hd_cols, hd_cols, 1, (uint32_t)(g.tn / 2))) != MARLAAS_OK) return rc;
        if (g.w3d) rc = make_panel_map(&tmXW, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, pool->ldB, 2, BK);
        else rc = make_map(&tmXW, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, pool->ldB, 64, BK);
        if (rc != MARLAAS_OK) return rc;
    } else {
        tmXX = tmX;
        tmXW = tmW;
    }

    // the largest dynamic shared memory asked for so far on the device (raised when a call needs more)
    static size_t smem_set[64] = {};
    if (pool->device >= 64 || smem_set[pool->device] < smem_bytes) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_gemm_wide, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        if (pool->device < 64) smem_set[pool->device] = smem_bytes;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * shape.pairs));
    cfg.blockDim = dim3(DK_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_gemm_wide, tmW, tmX, tmXW, tmXX, g));
    count_launch();
    return MARLAAS_OK;
}

marlaas_status_t launch_decode_stream_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                            int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                            const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st) {
    using namespace sm100;
    const int64_t K = pool->K, N = pool->N;
    const int hd_cols = (int)align_up((size_t)pool->cap * pool->RP, 64);     // pitch of hd: whole 64-deep panels

    int last_used = -1;
    for (int s = 0; s < pool->cap; ++s)
        if (pool->slots[s].used && pool->slots[s].rank > 0) last_used = s;

    StreamArgs g;
    g.T = (int)T; g.Nout = (int)N;
    g.C = y; g.ldc = ldy; g.status = pool->d_status; g.sync = pool->d_sync; g.xbuf = ws.xbuf;
    g.nstrips = (int)cdiv(N, DG_TM);
    g.num_ks = (int)(K / BK);
    g.num_xs = (int)cdiv((int64_t)(last_used + 1) * pool->RP, (int64_t)BK);
    g.nstep = g.num_ks + g.num_xs;
    g.tn = T < DG_TN ? (int)cdiv(T, 64) * 64 : DG_TN;  // one token tile whenever it is narrower than 256
    const int64_t tiles = cdiv(T, DG_TN) * g.nstrips;
    g.total = (int)(tiles * g.nstep);
    g.w3d = (N % 64) == 0;
    g.parts = pool->P;
    for (int p = 0; p < 4; ++p) g.part_end[p] = p < pool->P ? (int)pool->part_begin[p + 1] : 0;
    const size_t stage_bytes = 2 * CHUNK_BYTES + (size_t)(g.tn / 2) * 128;
    // as in the one-tile-per-pair kernel, two shrink CTAs share each SM with a CTA of this kernel
    const size_t room = (size_t)227 * 1024 - 2 * decode_shrink_smem_bytes(T, S) - 1024;
    g.stages = (int)std::max<size_t>(2, std::min<size_t>(9, (room - 1024 - 512 - 8 * 2048) / stage_bytes));
    const size_t smem_bytes = 1024 + 512 + 8 * 2048 + (size_t)g.stages * stage_bytes;

    // every pair must be resident at once only in so far as a pair waits for pairs of lower index, which are placed first;
    // the grid is nevertheless kept within what fits beside nothing else
    static int max_clusters[64] = {};
    int mc = pool->device < 64 ? max_clusters[pool->device] : 0;
    if (mc == 0) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_decode_gemm_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        cudaLaunchConfig_t qc = {};
        qc.gridDim = dim3(2 * 64);
        qc.blockDim = dim3(DK_THREADS);
        qc.dynamicSmemBytes = 200 * 1024;
        cudaLaunchAttribute qa;
        qa.id = cudaLaunchAttributeClusterDimension;
        qa.val.clusterDim.x = 2; qa.val.clusterDim.y = 1; qa.val.clusterDim.z = 1;
        qc.attrs = &qa; qc.numAttrs = 1;
        MARLAAS_CUDA_TRY(cudaOccupancyMaxActiveClusters(&mc, k_decode_gemm_stream, &qc));
        if (mc < 1) return fail(MARLAAS_ERR_CUDA, "no CTA pair of the decode kernel fits on this device");
        if (pool->device < 64) max_clusters[pool->device] = mc;
    }
    g.npairs = std::min(mc, pool->sm_count / 2);
    if ((size_t)SY_FLAGS + (size_t)g.npairs * 16 > DECODE_SYNC_BYTES / 4)
        return fail(MARLAAS_ERR_INVALID_ARG, "lora_forward: the decode path needs more exchange flags than the pool holds");

    marlaas_status_t rc;
    if ((rc = launch_decode_shrink(pool, T, x, ldx, S, seg_offsets, seg_slot, ws, h_out, st)) != MARLAAS_OK) return rc;

    alignas(64) CUtensorMap tmW, tmX, tmXW, tmXX;
    if ((rc = make_panel_map(&tmX, x, T, K, ldx, 1, (uint32_t)(g.tn / 2))) != MARLAAS_OK) return rc;
    if (g.w3d) rc = make_panel_map(&tmW, W, K, N, ldw, 2, BK);
    else rc = make_map(&tmW, W, K, N, ldw, 64, BK);
    if (rc != MARLAAS_OK) return rc;
    if (g.num_xs > 0) {
        if ((rc = make_panel_map(&tmXX, ws.hd, T * pool->P, hd_cols, hd_cols, 1, (uint32_t)(g.tn / 2))) != MARLAAS_OK) return rc;
        if (g.w3d) rc = make_panel_map(&tmXW, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, pool->ldB, 2, BK);
        else rc = make_map(&tmXW, pool->d_Bs, (int64_t)pool->cap * pool->RP, N, pool->ldB, 64, BK);
        if (rc != MARLAAS_OK) return rc;
    } else {
        tmXX = tmX;
        tmXW = tmW;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * g.npairs));
    cfg.blockDim = dim3(DK_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_decode_gemm_stream, tmW, tmX, tmXW, tmXX, g));
    count_launch();
    return MARLAAS_OK;
}

}  // namespace marlaas
