// Per-tenant adapter-gradient reductions on the tensor cores (sm_100a):
//     dB_t[j][n] (+)= s_t * sum_{i in t} h_i[j] * dy_i[n]          dA_t[k][j] (+)= s_t * sum_{i in t} x_i[k] * g_i[j]
// Both are "sum over a tenant's tokens of (fp32 r-vector) x (bf16 row)".  The contraction runs over tokens, so the
// streamed operand (dy or x, [tokens][C], C contiguous) is an MN-major A operand and the r-vectors an MN-major B
// operand.  The r-vectors must stay fp32-accurate (a bf16 rounding of h or g would show up as a random walk in
// sums over thousands of tokens), so each is split into bf16 hi + bf16 lo and both halves ride in the same MMA
// (N = 2 * RP columns); the epilogue adds the two column halves.
//
// Tokens are taken in aligned blocks of 64 (one k-block).  For every (block, tenant present in it) there is one
// "copy" of the block's r-vectors in which the rows of other tenants are zero, so a tenant's sum is simply the
// sum over its copies, whatever the segment structure: no atomics, fixed summation order, deterministic.
// One work item = (tenant, 128 output columns); a CTA walks the tenant's copy list accumulating in tensor memory
// and writes the slot's gradient once.  If the batch interleaves tenants so finely that the copies would not
// fit the workspace, a device flag routes the call to the CUDA-core reduction instead.
#include "sm100_ptx.cuh"

namespace marlaas {
namespace sm100 {

constexpr int GRAD_THREADS = 192;
constexpr int GRAD_STAGES = 4;          // at most: as many steps as fit the shared-memory budget (see the launch)
constexpr int GRAD_BPS = 2;              // 64-token blocks per pipeline step: one barrier round trip and one commit for both
constexpr int GRAD_INLINE_SLOTS = 64;
constexpr int GRAD_QN = 4;               // depth of the CTA's work-item queue
constexpr uint32_t GB_STAGE_BYTES = 4 * CHUNK_BYTES;   // up to 256 columns of split r-vectors

__device__ __forceinline__ void tc_ld_32x16g(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

// ---- plan: which tenants are present in each 64-token block ----------------------------------------------------
__global__ void __launch_bounds__(64) k_grad_presence(int T, int cap, const int32_t* __restrict__ tok_slot,
                                                      const int32_t* __restrict__ d_rank,
                                                      int32_t* __restrict__ blk_np, int32_t* __restrict__ blk_rank) {
    __shared__ int pres[256];
    const int blk = blockIdx.x, tid = threadIdx.x;
    for (int t = tid; t < cap; t += 64) pres[t] = 0;
    __syncthreads();
    const int i = blk * 64 + tid;
    if (i < T) {
        const int t = tok_slot[i];
        if (t >= 0 && t < cap && d_rank[t] > 0) pres[t] = 1;
    }
    __syncthreads();
    if (tid == 0) {
        int n = 0;
        for (int t = 0; t < cap; ++t) {
            blk_rank[(size_t)blk * cap + t] = pres[t] ? n : -1;
            n += pres[t];
        }
        blk_np[blk] = n;
    }
}

// One CTA per tenant: position of every copy (exclusive scan of the per-block counts) and the tenant's copy list in
// ascending block order.  CTA 0 also publishes the scan and decides whether the copies fit.
__global__ void __launch_bounds__(256) k_grad_lists(int nblk, int cap, int max_copies,
                                                    const int32_t* __restrict__ blk_np,
                                                    const int32_t* __restrict__ blk_rank,
                                                    int32_t* __restrict__ blk_base, int32_t* __restrict__ ten_nblk,
                                                    int32_t* __restrict__ ten_blks, int32_t* __restrict__ ten_pos,
                                                    int32_t* __restrict__ gflag) {
    __shared__ int base[4096 + 1];
    __shared__ int s_warp[8];
    __shared__ int s_run;
    const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // exclusive scan of blk_np into base[]
    const int per = (nblk + 255) / 256;
    const int b0 = tid * per, b1 = min(nblk, b0 + per);
    int loc = 0;
    for (int b = b0; b < b1; ++b) loc += blk_np[b];
    int inc = loc;
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    int off = inc - loc;
    for (int w = 0; w < warp; ++w) off += s_warp[w];
    int total = 0;
    for (int w = 0; w < 8; ++w) total += s_warp[w];
    for (int b = b0; b < b1; ++b) {
        base[b] = off;
        off += blk_np[b];
    }
    if (tid == 0) s_run = 0;
    __syncthreads();
    if (t == 0) {
        for (int b = tid; b < nblk; b += 256) blk_base[b] = base[b];
        if (tid == 0) {
            blk_base[nblk] = total;
            gflag[0] = total > max_copies ? 1 : 0;
            gflag[1] = total;
            gflag[2] = 0;      // work-item counters of the two reduction launches (dB, dA)
            gflag[3] = 0;
        }
    }
    // this tenant's copies, ascending block order
    for (int c0 = 0; c0 < nblk; c0 += 256) {
        const int b = c0 + tid;
        const int rk = b < nblk ? blk_rank[(size_t)b * cap + t] : -1;
        const bool hit = rk >= 0;
        const unsigned bal = __ballot_sync(0xffffffffu, hit);
        __syncthreads();
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int before = s_run;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        if (hit) {
            const int n = before + __popc(bal & ((1u << lane) - 1u));
            ten_blks[(size_t)t * nblk + n] = b;
            ten_pos[(size_t)t * nblk + n] = base[b] + rk;
        }
        __syncthreads();
        if (tid == 0) {
            int v = s_run;
            for (int w = 0; w < 8; ++w) v += s_warp[w];
            s_run = v;
        }
    }
    __syncthreads();
    if (tid == 0) ten_nblk[t] = s_run;
}

// One CTA per 64-token block: writes the block's copies, hm[(copy*64 + row)][HW] = [ hi(v) | lo(v) | 0 ] for rows of
// the copy's tenant and zero rows for the other tokens of the block.
__global__ void __launch_bounds__(256) k_pad_split(int T, int cap, int RP, int HW, const float* __restrict__ src,
                                                   const int32_t* __restrict__ tok_slot,
                                                   const int32_t* __restrict__ blk_base,
                                                   const int32_t* __restrict__ blk_rank,
                                                   const int32_t* __restrict__ gflag, bf16* __restrict__ hm) {
    if (gflag[0] != 0) return;
    const int blk = blockIdx.x, tid = threadIdx.x;
    const int base = blk_base[blk];
    const int chunks_per_row = HW / 8;
    for (int t = 0; t < cap; ++t) {
        const int rk = blk_rank[(size_t)blk * cap + t];
        if (rk < 0) continue;
        bf16* dst = hm + (size_t)(base + rk) * 64 * HW;
        for (int e = tid; e < 64 * chunks_per_row; e += 256) {
            const int row = e / chunks_per_row, c = (e - row * chunks_per_row) * 8;
            const int i = blk * 64 + row;
            uint4 o = make_uint4(0u, 0u, 0u, 0u);
            if (i < T && tok_slot[i] == t && c < 2 * RP) {
                const bool lo_half = c >= RP;
                const float* s = src + (size_t)i * RP + (lo_half ? c - RP : c);
                __nv_bfloat162 p[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float v0 = s[2 * q], v1 = s[2 * q + 1];
                    const bf16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
                    if (lo_half)
                        p[q] = __floats2bfloat162_rn(v0 - __bfloat162float(h0), v1 - __bfloat162float(h1));
                    else
                        p[q] = __halves2bfloat162(h0, h1);
                }
                o = make_uint4(*reinterpret_cast<uint32_t*>(&p[0]), *reinterpret_cast<uint32_t*>(&p[1]),
                               *reinterpret_cast<uint32_t*>(&p[2]), *reinterpret_cast<uint32_t*>(&p[3]));
            }
            *reinterpret_cast<uint4*>(dst + (size_t)row * HW + c) = o;
        }
    }
}

struct GradArgs {
    int C;                 // columns of the streamed operand (N for dB, K for dA)
    int num_c_tiles;
    int cap, RP, HW, nblk;
    const int32_t* d_rank;
    const float* d_scale;
    const int32_t* ten_nblk;
    const int32_t* ten_blks;
    const int32_t* ten_pos;
    const int32_t* gflag;
    int32_t* counter;      // next work item (zeroed by the plan kernel before every pair of launches)
    float* const* out_ptrs;   // per-slot outputs in device memory, or nullptr: the table is inl[] below
    int transpose_out, accumulate;
    int stages;            // pipeline steps in flight
    int32_t* status;
    float* inl[GRAD_INLINE_SLOTS];   // small pools: the pointer table travels with the launch (no host-to-device copy)
};

__global__ void __launch_bounds__(GRAD_THREADS, 1)
k_grad_sm100(const __grid_constant__ CUtensorMap tmSrc, const __grid_constant__ CUtensorMap tmHm, const GradArgs g) {
    constexpr int MAX_STAGES = GRAD_STAGES;
    const int STAGES = g.stages;
    constexpr uint32_t TMEM_COLS = 512;
    // A second reduction launched behind this one as a programmatic dependent (it reads nothing this one writes) may
    // take over every SM a CTA of this grid leaves.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (g.gflag[0] != 0) return;   // copies did not fit: the CUDA-core reduction handles this call

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sA = smem_u32(smem);
    const int hw_chunks = g.HW / 64;
    const uint32_t B_BLOCK = (uint32_t)hw_chunks * CHUNK_BYTES;      // one block's split r-vectors
    const uint32_t A_STEP = GRAD_BPS * A_STAGE_BYTES, B_STEP = GRAD_BPS * B_BLOCK;
    const uint32_t sB = sA + STAGES * A_STEP;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STEP + B_STEP));
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * MAX_STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * MAX_STAGES;
    const uint32_t bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;
    const uint32_t bar_qfull = bar_drain + 8, bar_qempty = bar_qfull + 8 * GRAD_QN;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 5 + 2 * GRAD_QN);
    volatile int* abort_word = reinterpret_cast<volatile int*>(tmem_slot + 1);
    __shared__ int s_cnt[256], s_order[256];
    __shared__ volatile int s_q[GRAD_QN];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_items = g.num_c_tiles * g.cap;

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
        for (int i = 0; i < GRAD_QN; ++i) {
            mbar_init(bar_qfull + 8 * i, 1);
            mbar_init(bar_qempty + 8 * i, 5);     // the MMA thread and the four epilogue warps
        }
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        prefetch_tmap(&tmSrc);
        prefetch_tmap(&tmHm);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Work items are handed out dynamically, heaviest tenants first (an item's cost is its tenant's copy count), so that
    // skewed batches still finish together; which CTA computes an item does not change its value.
    for (int t = threadIdx.x; t < g.cap; t += GRAD_THREADS) s_cnt[t] = ((g.out_ptrs ? g.out_ptrs[t] : g.inl[t]) != nullptr && g.d_rank[t] > 0) ? g.ten_nblk[t] : -1;
    tc_fence_before();
    __syncthreads();
    for (int t = threadIdx.x; t < g.cap; t += GRAD_THREADS) {
        const int c = s_cnt[t];
        int rk = 0;
        for (int u = 0; u < g.cap; ++u) rk += (s_cnt[u] > c) || (s_cnt[u] == c && u < t);
        s_order[rk] = t;
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // an item does tensor work only if its slot has an output, a rank and at least one copy
    auto item_blocks = [&](int item, int& t, int& c0) -> int {
        t = s_order[item / g.num_c_tiles];
        c0 = (item % g.num_c_tiles) * 128;
        return s_cnt[t];      // -1: no output or no rank
    };

    if (warp == 0) {
        if (lane == 0) {   // ---- TMA producer
            uint32_t it = 0, qi = 0, ps = 0, pph = 0;    // steps issued; stage and phase of the next step
            bool ok = true;
            while (ok) {
                const uint32_t qs = qi % GRAD_QN, qph = (qi / GRAD_QN) & 1;
                if (!(ok = mbar_wait(bar_qempty + 8 * qs, qph ^ 1, abort_word, 27))) break;
                int item = atomicAdd(g.counter, 1);
                if (item >= num_items) item = -1;
                s_q[qs] = item;
                mbar_arrive(bar_qfull + 8 * qs);
                ++qi;
                if (item < 0) break;
                int t, c0;
                const int nb = item_blocks(item, t, c0);
                if (nb <= 0) continue;
                const int a_chunks = min(2, (g.C - c0 + 63) / 64);
                for (int k = 0; k < nb && ok; k += GRAD_BPS, ++it) {
                    const uint32_t s = ps, ph = pph;
                    if (!(ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_word, 21))) break;
                    if (++ps == (uint32_t)STAGES) { ps = 0; pph ^= 1; }
                    const int nj = min(GRAD_BPS, nb - k);
                    const uint32_t full = bar_full + 8 * s;
                    mbar_expect_tx(full, (uint32_t)nj * (a_chunks + hw_chunks) * CHUNK_BYTES);
                    for (int j = 0; j < nj; ++j) {
                        const int blk = g.ten_blks[(size_t)t * g.nblk + k + j];
                        const int pos = g.ten_pos[(size_t)t * g.nblk + k + j];
                        for (int c = 0; c < a_chunks; ++c)
                            tma_load_2d(sA + s * A_STEP + j * A_STAGE_BYTES + c * CHUNK_BYTES, &tmSrc, full, c0 + c * 64, blk * 64);
                        for (int c = 0; c < hw_chunks; ++c)
                            tma_load_2d(sB + s * B_STEP + j * B_BLOCK + c * CHUNK_BYTES, &tmHm, full, c * 64, pos * 64);
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
        if (lane == 0) {   // ---- MMA issuer: A and B both MN-major, M = 128, N = HW
            const uint32_t idesc = make_idesc(g.HW, 1) | (1u << 15);
            uint32_t it = 0, lt = 0, ms = 0, mph = 0;
            bool ok = true;
            uint32_t qi = 0;
            while (ok) {
                const uint32_t qs = qi % GRAD_QN, qph = (qi / GRAD_QN) & 1;
                if (!(ok = mbar_wait(bar_qfull + 8 * qs, qph, abort_word, 28))) break;
                const int item = s_q[qs];
                mbar_arrive(bar_qempty + 8 * qs);
                ++qi;
                if (item < 0) break;
                int t, c0;
                const int nb = item_blocks(item, t, c0);
                if (nb <= 0) continue;
                const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
                if (!(ok = mbar_wait(bar_tempty + 8 * b, aph ^ 1, abort_word, 23))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * 256;
                uint32_t acc = 0;
                for (int k = 0; k < nb && ok; k += GRAD_BPS, ++it) {
                    const uint32_t s = ms, ph = mph;
                    if (!(ok = mbar_wait(bar_full + 8 * s, ph, abort_word, 24))) break;
                    if (++ms == (uint32_t)STAGES) { ms = 0; mph ^= 1; }
                    tc_fence_after();
                    const int nj = min(GRAD_BPS, nb - k);
                    for (int jb = 0; jb < nj; ++jb) {
                        const uint32_t a0 = sA + s * A_STEP + jb * A_STAGE_BYTES, b0 = sB + s * B_STEP + jb * B_BLOCK;
                        // descriptors of successive 16-token slices differ only in the start-address field (16-byte units)
                        const uint64_t da0 = desc_mn_major(a0, CHUNK_BYTES), db0 = desc_mn_major(b0, CHUNK_BYTES);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            tc_mma_bf16(d_tmem, da0 + (uint64_t)(j * (UNIT_BYTES >> 4)), db0 + (uint64_t)(j * (UNIT_BYTES >> 4)), idesc, acc);
                            acc = 1;
                        }
                    }
                    tc_commit(bar_empty + 8 * s);
                }
                if (ok) tc_commit(bar_tfull + 8 * b);
                ++lt;
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
        // ---- epilogue: out = s_t * (hi part + lo part)
        const int q = warp & 3;
        uint32_t lt = 0;
        bool ok = true;
        uint32_t qi = 0;
        while (ok) {
            const uint32_t qs = qi % GRAD_QN, qph = (qi / GRAD_QN) & 1;
            ok = mbar_wait(bar_qfull + 8 * qs, qph, abort_word, 29);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int item = s_q[qs];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_qempty + 8 * qs);
            ++qi;
            if (item < 0) break;
            int t, c0;
            const int nb = item_blocks(item, t, c0);
            if (nb < 0) continue;
            float* out = g.out_ptrs ? g.out_ptrs[t] : g.inl[t];
            const int r = g.d_rank[t];
            const int c = c0 + q * 32 + lane;
            if (nb == 0) {   // tenant without tokens: exact zeros unless accumulating
                if (!g.accumulate && c < g.C)
                    for (int j = 0; j < r; ++j) {
                        if (g.transpose_out) out[(size_t)c * r + j] = 0.f;
                        else out[(size_t)j * g.C + c] = 0.f;
                    }
                continue;
            }
            const float sc = g.d_scale[t];
            const uint32_t b = lt & 1, aph = (lt >> 1) & 1;
            ok = mbar_wait(bar_tfull + 8 * b, aph, abort_word, 26);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + b * 256;
#pragma unroll 1
            for (int j0 = 0; j0 < r; j0 += 16) {
                uint32_t hi[16], lo[16];
                tc_ld_32x16g(trow + j0, hi);
                tc_ld_32x16g(trow + g.RP + j0, lo);
                tc_wait_ld();
                if (c < g.C && g.transpose_out && (r & 3) == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0) {
                    // out is [C][r]: the thread's 16 ranks are contiguous, four per store
                    float4* dst = reinterpret_cast<float4*>(out + (size_t)c * r + j0);
#pragma unroll
                    for (int e4 = 0; e4 < 4; ++e4) {
                        if (j0 + 4 * e4 < r) {
                            float4 v;
                            v.x = sc * (__uint_as_float(hi[4 * e4]) + __uint_as_float(lo[4 * e4]));
                            v.y = sc * (__uint_as_float(hi[4 * e4 + 1]) + __uint_as_float(lo[4 * e4 + 1]));
                            v.z = sc * (__uint_as_float(hi[4 * e4 + 2]) + __uint_as_float(lo[4 * e4 + 2]));
                            v.w = sc * (__uint_as_float(hi[4 * e4 + 3]) + __uint_as_float(lo[4 * e4 + 3]));
                            if (g.accumulate) {
                                const float4 o = dst[e4];
                                v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                            }
                            dst[e4] = v;
                        }
                    }
                } else if (c < g.C) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int j = j0 + e;
                        if (j < r) {
                            const float v = sc * (__uint_as_float(hi[e]) + __uint_as_float(lo[e]));
                            float* dst = g.transpose_out ? out + (size_t)c * r + j : out + (size_t)j * g.C + c;
                            *dst = g.accumulate ? *dst + v : v;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * b);
            ++lt;
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
    // launched early behind another reduction: never complete before it (what follows in the stream relies on both)
    if (threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace sm100

bool grad_sm100_eligible(const marlaas_pool* pool, int64_t T) { return pool->cap <= 256 && T > 0 && cdiv(T, 64) <= 4096; }

marlaas_status_t launch_grad_plan(const marlaas_pool* pool, int64_t T, const Workspace& ws, cudaStream_t st) {
    using namespace sm100;
    const int nblk = (int)cdiv(T, 64);
    k_grad_presence<<<nblk, 64, 0, st>>>((int)T, pool->cap, ws.tok_slot, pool->d_rank, ws.blk_np, ws.blk_rank);
    MARLAAS_LAUNCH_CHECK("k_grad_presence");
    k_grad_lists<<<pool->cap, 256, 0, st>>>(nblk, pool->cap, ws.max_copies, ws.blk_np, ws.blk_rank, ws.blk_base,
                                            ws.ten_nblk, ws.ten_blks, ws.ten_pos, ws.gflag);
    MARLAAS_LAUNCH_CHECK("k_grad_lists");
    return MARLAAS_OK;
}

marlaas_status_t launch_grad_sm100(const marlaas_pool* pool, int64_t T, int64_t C, const bf16* src, int64_t ld,
                                   const float* hg, float* const* out_ptrs, float* const* host_ptrs, bool transpose_out,
                                   bool accumulate,
                                   const Workspace& ws, cudaStream_t st, bf16* hm, int phases) {
    using namespace sm100;
    const int nblk = (int)cdiv(T, 64);
    if (phases & GRAD_PHASE_COPIES) {
        k_pad_split<<<nblk, 256, 0, st>>>((int)T, pool->cap, pool->RP, ws.HW, hg, ws.tok_slot, ws.blk_base, ws.blk_rank,
                                          ws.gflag, hm);
        MARLAAS_LAUNCH_CHECK("k_pad_split");
    }
    if (!(phases & GRAD_PHASE_REDUCE)) return MARLAAS_OK;
    GradArgs g;
    g.C = (int)C;
    g.num_c_tiles = (int)cdiv(C, 128);
    g.cap = pool->cap;
    g.RP = pool->RP;
    g.HW = ws.HW;
    g.nblk = nblk;
    g.d_rank = pool->d_rank;
    g.d_scale = pool->d_scale;
    g.ten_nblk = ws.ten_nblk;
    g.ten_blks = ws.ten_blks;
    g.ten_pos = ws.ten_pos;
    g.gflag = ws.gflag;
    g.counter = ws.gflag + (transpose_out ? 3 : 2);
    g.out_ptrs = out_ptrs;
    if (host_ptrs && pool->cap <= GRAD_INLINE_SLOTS) {
        g.out_ptrs = nullptr;
        for (int t = 0; t < GRAD_INLINE_SLOTS; ++t) g.inl[t] = t < pool->cap ? host_ptrs[t] : nullptr;
    }
    g.transpose_out = transpose_out ? 1 : 0;
    g.accumulate = accumulate ? 1 : 0;
    g.status = pool->d_status;
    alignas(64) CUtensorMap tmSrc, tmHm;
    marlaas_status_t rc;
    if ((rc = make_map(&tmSrc, src, T, C, ld, 64, 64)) != MARLAAS_OK) return rc;
    if ((rc = make_map(&tmHm, hm, (int64_t)ws.max_copies * 64, ws.HW, ws.HW, 64, 64)) != MARLAAS_OK) return rc;
    // as many steps of GRAD_BPS blocks as fit what four single-block steps of the widest r-vectors take
    constexpr size_t smem_bytes = 1024 + (size_t)4 * (A_STAGE_BYTES + GB_STAGE_BYTES) + 256;
    const size_t step_bytes = (size_t)GRAD_BPS * (A_STAGE_BYTES + (size_t)(ws.HW / 64) * CHUNK_BYTES);
    g.stages = (int)std::min<size_t>(GRAD_STAGES, (smem_bytes - 1024 - 256) / step_bytes);
    static bool attr_set[64] = {};
    if (pool->device >= 64 || !attr_set[pool->device]) {
        MARLAAS_CUDA_TRY(cudaFuncSetAttribute(k_grad_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        if (pool->device < 64) attr_set[pool->device] = true;
    }
    const int items = g.num_c_tiles * g.cap;
    const int grid = items < pool->sm_count ? items : pool->sm_count;
    if (phases & GRAD_PHASE_EARLY) {
        // the caller states that this launch reads nothing the kernel before it in the stream writes: its CTAs may start
        // on SMs that kernel's CTAs have left
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(GRAD_THREADS);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        MARLAAS_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_grad_sm100, tmSrc, tmHm, g));
    } else {
        k_grad_sm100<<<grid, GRAD_THREADS, smem_bytes, st>>>(tmSrc, tmHm, g);
    }
    MARLAAS_LAUNCH_CHECK("k_grad_sm100");
    return MARLAAS_OK;
}

}  // namespace marlaas
