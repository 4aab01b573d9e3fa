// Plain CUDA-core kernels for every step of the layer.  They are the diagnostic path
// (MARLAAS_FLAG_CUDA_CORE_PATH) and serve shapes the tensor-core kernels do not take; fp32 FMA throughout.
#include "internal.cuh"

namespace marlaas {

__device__ __forceinline__ float bf2f(bf16 v) { return __bfloat162float(v); }

// ---- shrink: out[i][j] = <src_i , store[slot_i*RP + j]> -------------------------------------------------
// One CTA per token, one warp per rank index (strided); 16-byte loads along the contiguous dimension,
// warp-shuffle reduction.  Used for h = x A_t (store = At, D = K) and g = dy B_t^T (store = Bs, D = N).
__global__ void __launch_bounds__(128) k_rowdot(int64_t D, const bf16* __restrict__ src, int64_t ld,
                                                const bf16* __restrict__ store, int64_t sld, const int32_t* __restrict__ tok_slot,
                                                const int32_t* __restrict__ d_rank, int RP, int cap,
                                                float* __restrict__ out) {
    const int64_t i = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = tok_slot[i];
    const int r = (t >= 0 && t < cap) ? d_rank[t] : 0;
    const bf16* row = src + i * ld;
    for (int j = warp; j < RP; j += 4) {
        float acc = 0.f;
        if (j < r) {
            const bf16* a = store + ((size_t)t * RP + j) * sld;
            for (int64_t d = (int64_t)lane * 8; d < D; d += 256) {
                const uint4 xv = *reinterpret_cast<const uint4*>(row + d);
                const uint4 av = *reinterpret_cast<const uint4*>(a + d);
                const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xv);
                const __nv_bfloat162* ap = reinterpret_cast<const __nv_bfloat162*>(&av);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 xf = __bfloat1622float2(xp[q]);
                    const float2 af = __bfloat1622float2(ap[q]);
                    acc = fmaf(xf.x, af.x, acc);
                    acc = fmaf(xf.y, af.y, acc);
                }
            }
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        }
        if (lane == 0) out[i * RP + j] = acc;
    }
}

// Same dot products, plus the token's row of the block-diagonal bf16 operand the tensor-core GEMM multiplies with
// the adapter rows: bf16(s_t * h) in the columns of the token's own tenant units, zeros in the tile's other units.
__global__ void __launch_bounds__(128) k_shrink_hd(int64_t D, const bf16* __restrict__ src, int64_t ld,
                                                   const bf16* __restrict__ store, int64_t sld, const int32_t* __restrict__ tok_slot,
                                                   const int32_t* __restrict__ tok_uoff,
                                                   const int32_t* __restrict__ tile_nunits,
                                                   const int32_t* __restrict__ d_rank, const float* __restrict__ d_scale,
                                                   int RP, int cap, int hd_cols, float* __restrict__ out,
                                                   bf16* __restrict__ hd) {
    __shared__ float sh[128];
    const int64_t i = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = tok_slot[i];
    const int r = (t >= 0 && t < cap) ? d_rank[t] : 0;
    const bf16* row = src + i * ld;
    for (int j = warp; j < RP; j += 4) {
        float acc = 0.f;
        if (j < r) {
            const bf16* a = store + ((size_t)t * RP + j) * sld;
            for (int64_t d = (int64_t)lane * 8; d < D; d += 256) {
                const uint4 xv = *reinterpret_cast<const uint4*>(row + d);
                const uint4 av = *reinterpret_cast<const uint4*>(a + d);
                const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xv);
                const __nv_bfloat162* ap = reinterpret_cast<const __nv_bfloat162*>(&av);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 xf = __bfloat1622float2(xp[q]);
                    const float2 af = __bfloat1622float2(ap[q]);
                    acc = fmaf(xf.x, af.x, acc);
                    acc = fmaf(xf.y, af.y, acc);
                }
            }
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        }
        if (lane == 0) {
            out[i * RP + j] = acc;
            sh[j] = acc;
        }
    }
    __syncthreads();
    const int nun = tile_nunits[i >> 8];
    const int uo = r > 0 ? tok_uoff[i] : -1;
    const float s = r > 0 ? d_scale[t] : 0.f;
    const int own0 = uo * 16, own1 = own0 + ((r + 15) >> 4) * 16;
    for (int c8 = threadIdx.x; c8 * 8 < nun * 16; c8 += 128) {
        uint4 o = make_uint4(0u, 0u, 0u, 0u);
        const int c = c8 * 8;
        if (uo >= 0 && c >= own0 && c < own1) {
            __nv_bfloat162 p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
                p[e] = __floats2bfloat162_rn(s * sh[c - own0 + 2 * e], s * sh[c - own0 + 2 * e + 1]);
            o.x = *reinterpret_cast<uint32_t*>(&p[0]);
            o.y = *reinterpret_cast<uint32_t*>(&p[1]);
            o.z = *reinterpret_cast<uint32_t*>(&p[2]);
            o.w = *reinterpret_cast<uint32_t*>(&p[3]);
        }
        *reinterpret_cast<uint4*>(hd + i * hd_cols + c) = o;
    }
}

// ---- base GEMM + fused low-rank term ----------------------------------------------------------------------
// C[i][c] = bf16( sum_k A[i][k] * Wop[k][c] + s_t * sum_p sum_j hg[p][i][j] * store[((p*cap + t)*RP+j)][c] )
// (nparts = 1 but for the dx of a pool over several projections, whose low-rank term sums over all of them: hg planes
// hg_plane floats apart, store rows sld elements apart).  64x64 tile, 16-deep k slab, 256 threads x (4x4) outputs.
template <bool TRANS_W>
__global__ void __launch_bounds__(256) k_gemm_cuda_core(int64_t T, int64_t Nout, int64_t Kc, const bf16* __restrict__ A,
                                                        int64_t lda, const bf16* __restrict__ W, int64_t ldw,
                                                        bf16* __restrict__ C, int64_t ldc, const float* __restrict__ hg,
                                                        const bf16* __restrict__ store, int64_t sld, int nparts,
                                                        int64_t hg_plane, const int32_t* __restrict__ tok_slot,
                                                        const int32_t* __restrict__ d_rank,
                                                        const float* __restrict__ d_scale, int RP, int cap) {
    __shared__ float sA[16][64 + 1];
    __shared__ float sB[16][64 + 1];
    const int tid = threadIdx.x;
    const int64_t row0 = (int64_t)blockIdx.y * 64, col0 = (int64_t)blockIdx.x * 64;
    const int ty = tid / 16, tx = tid % 16;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    for (int64_t k0 = 0; k0 < Kc; k0 += 16) {
        for (int e = tid; e < 64 * 16; e += 256) {
            {   // A tile: 64 rows x 16 k, k fastest in memory
                const int rr = e / 16, kk = e % 16;
                const int64_t gi = row0 + rr, gk = k0 + kk;
                sA[kk][rr] = (gi < T && gk < Kc) ? bf2f(A[gi * lda + gk]) : 0.f;
            }
            if (!TRANS_W) {   // W[k][c], c fastest
                const int kk = e / 64, cc = e % 64;
                const int64_t gk = k0 + kk, gc = col0 + cc;
                sB[kk][cc] = (gk < Kc && gc < Nout) ? bf2f(W[gk * ldw + gc]) : 0.f;
            } else {          // W stored [c][k], k fastest
                const int cc = e / 16, kk = e % 16;
                const int64_t gk = k0 + kk, gc = col0 + cc;
                sB[kk][cc] = (gk < Kc && gc < Nout) ? bf2f(W[gc * ldw + gk]) : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                a[q] = sA[kk][ty * 4 + q];
                b[q] = sB[kk][tx * 4 + q];
            }
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(a[p], b[q], acc[p][q]);
        }
        __syncthreads();
    }
    for (int p = 0; p < 4; ++p) {
        const int64_t gi = row0 + ty * 4 + p;
        if (gi >= T) continue;
        const int t = tok_slot ? tok_slot[gi] : -1;
        const int r = (t >= 0 && t < cap) ? d_rank[t] : 0;
        const float s = r > 0 ? d_scale[t] : 0.f;
        for (int q = 0; q < 4; ++q) {
            const int64_t gc = col0 + tx * 4 + q;
            if (gc >= Nout) continue;
            float d = 0.f;
            for (int p = 0; p < nparts; ++p)
                for (int j = 0; j < r; ++j)
                    d = fmaf(hg[p * hg_plane + gi * RP + j], bf2f(store[(((size_t)p * cap + t) * RP + j) * sld + gc]), d);
            C[gi * ldc + gc] = __float2bfloat16_rn(acc[p][q] + s * d);
        }
    }
}

// ---- adapter-gradient reductions ---------------------------------------------------------------------------
// out_t[j][c] (+)= s_t * sum over tenant t's tokens (ascending token order) of hg[i][j] * src[i][c]
// grid = (ceil(C/128), capacity, RP/16); one thread per column c holding 16 rank accumulators.
// Deterministic: fixed summation order, no atomics.
__global__ void __launch_bounds__(128) k_grad_reduce(int64_t C, const bf16* __restrict__ src, int64_t ld,
                                                     const float* __restrict__ hg, const int32_t* __restrict__ perm,
                                                     const int32_t* __restrict__ slot_offset,
                                                     const int32_t* __restrict__ d_rank,
                                                     const float* __restrict__ d_scale, int RP,
                                                     float* const* __restrict__ out_ptrs, int transpose_out,
                                                     int accumulate, const int32_t* __restrict__ run_flag) {
    if (run_flag != nullptr && run_flag[0] == 0) return;
    const int t = blockIdx.y;
    float* out = out_ptrs[t];
    const int r = d_rank[t];
    const int j0 = blockIdx.z * 16;
    if (out == nullptr || j0 >= r) return;
    const int64_t c = (int64_t)blockIdx.x * 128 + threadIdx.x;
    const int p0 = slot_offset[t], p1 = slot_offset[t + 1];
    __shared__ float sh[32][16];
    float acc[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) acc[j] = 0.f;
    for (int pb = p0; pb < p1; pb += 32) {
        const int nb = min(32, p1 - pb);
        __syncthreads();
        for (int e = threadIdx.x; e < nb * 16; e += 128) {
            const int q = e / 16, j = e % 16;
            sh[q][j] = hg[(int64_t)perm[pb + q] * RP + j0 + j];
        }
        __syncthreads();
        if (c < C) {
            for (int q = 0; q < nb; ++q) {
                const float v = bf2f(src[(int64_t)perm[pb + q] * ld + c]);
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = fmaf(sh[q][j], v, acc[j]);
            }
        }
    }
    if (c >= C) return;
    const float s = d_scale[t];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        if (j0 + j >= r) break;
        float* dst = transpose_out ? (out + c * r + (j0 + j)) : (out + (int64_t)(j0 + j) * C + c);
        const float v = s * acc[j];
        *dst = accumulate ? (*dst + v) : v;
    }
}

marlaas_status_t launch_rowdot(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                               const bf16* store, int64_t sld, const int32_t* tok_slot, float* out, cudaStream_t st) {
    if (T <= 0) return MARLAAS_OK;
    k_rowdot<<<(unsigned)T, 128, 0, st>>>(D, src, ld, store, sld, tok_slot, pool->d_rank, pool->RP, pool->cap, out);
    MARLAAS_LAUNCH_CHECK("k_rowdot");
    return MARLAAS_OK;
}

marlaas_status_t launch_shrink_hd(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                                  const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st) {
    if (T <= 0) return MARLAAS_OK;
    k_shrink_hd<<<(unsigned)T, 128, 0, st>>>(D, src, ld, store, sld, ws.tok_slot, ws.tok_uoff, ws.tile_nunits, pool->d_rank,
                                             pool->d_scale, pool->RP, pool->cap, ws.umax * 16, out, ws.hd);
    MARLAAS_LAUNCH_CHECK("k_shrink_hd");
    return MARLAAS_OK;
}

marlaas_status_t launch_gemm_cuda_core(const marlaas_pool* pool, int64_t T, int64_t Nout, int64_t Kc,
                                       const bf16* A, int64_t lda, const bf16* W, int64_t ldw, bool trans_w,
                                       bf16* C, int64_t ldc, const float* hg, const bf16* store, int64_t sld,
                                       const int32_t* tok_slot, cudaStream_t st, int nparts, int64_t hg_plane) {
    if (T <= 0) return MARLAAS_OK;
    dim3 grid((unsigned)cdiv(Nout, 64), (unsigned)cdiv(T, 64));
    if (trans_w)
        k_gemm_cuda_core<true><<<grid, 256, 0, st>>>(T, Nout, Kc, A, lda, W, ldw, C, ldc, hg, store, sld, nparts, hg_plane, tok_slot,
                                                     pool->d_rank, pool->d_scale, pool->RP, pool->cap);
    else
        k_gemm_cuda_core<false><<<grid, 256, 0, st>>>(T, Nout, Kc, A, lda, W, ldw, C, ldc, hg, store, sld, nparts, hg_plane, tok_slot,
                                                      pool->d_rank, pool->d_scale, pool->RP, pool->cap);
    MARLAAS_LAUNCH_CHECK("k_gemm_cuda_core");
    return MARLAAS_OK;
}

marlaas_status_t launch_grad_reduce(const marlaas_pool* pool, int64_t C, const bf16* src, int64_t ld,
                                    const float* hg, const int32_t* perm, const int32_t* slot_offset,
                                    float* const* out_ptrs, bool transpose_out, bool accumulate, cudaStream_t st,
                                    const int32_t* run_flag) {
    dim3 grid((unsigned)cdiv(C, 128), (unsigned)pool->cap, (unsigned)(pool->RP / 16));
    k_grad_reduce<<<grid, 128, 0, st>>>(C, src, ld, hg, perm, slot_offset, pool->d_rank, pool->d_scale, pool->RP,
                                        out_ptrs, transpose_out ? 1 : 0, accumulate ? 1 : 0, run_flag);
    MARLAAS_LAUNCH_CHECK("k_grad_reduce");
    return MARLAAS_OK;
}

}  // namespace marlaas
