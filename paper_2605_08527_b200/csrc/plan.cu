// Index build: token-to-adapter segment table -> per-token slot, per-slot counts / offsets and the
// stable token permutation grouped by slot.  Pure integer work; its outputs are an exact contract
// (the same table always gives the same four arrays).
#include "internal.cuh"

namespace marlaas {

__device__ __forceinline__ void report(int32_t* status, int code, int detail) {
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// One thread per token: the segment of token i is the last s with seg_offsets[s] <= i < seg_offsets[s+1]
// (zero-length segments are skipped by construction).  Threads < S also check the table itself.
__global__ void k_tok_slot(int T, int S, const int32_t* __restrict__ seg_offsets,
                           const int32_t* __restrict__ seg_slot, int cap, int32_t* __restrict__ tok_slot,
                           int32_t* status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < S) {
        const int a = seg_offsets[i], b = seg_offsets[i + 1];
        if (b < a || a < 0 || b > T) report(status, DEV_BAD_TABLE, i);
        if (i == 0 && a != 0) report(status, DEV_BAD_TABLE, -1);
        if (i == S - 1 && b != T) report(status, DEV_BAD_TABLE, -2);
    }
    if (i == 0 && S == 0 && T != 0) report(status, DEV_BAD_TABLE, -3);
    if (i >= T) return;
    // first index s in [0,S) with seg_offsets[s+1] > i
    int lo = 0, hi = S;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (seg_offsets[mid + 1] > i) hi = mid; else lo = mid + 1;
    }
    int slot = -1;
    if (lo < S) {
        slot = seg_slot[lo];
        if (slot < -1 || slot >= cap) {
            report(status, DEV_BAD_INDEX, i);
            slot = -1;
        }
    }
    tok_slot[i] = slot;
}

// One CTA per key (slot 0..cap-1, then key cap = slot -1): count the tokens below and at this key, then place
// this key's tokens in ascending token order.  Stable by construction.
__global__ void __launch_bounds__(256) k_slot_sort(int T, int cap, const int32_t* __restrict__ tok_slot,
                                                   int32_t* __restrict__ slot_count,
                                                   int32_t* __restrict__ slot_offset, int32_t* __restrict__ perm,
                                                   const int32_t* __restrict__ run_flag) {
    if (run_flag != nullptr && run_flag[0] == 0) return;
    const int key = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ int s_warp[8];
    __shared__ int s_less, s_base;
    int less = 0;
    for (int i = tid; i < T; i += 256) {
        const int t = tok_slot[i];
        const int k = t < 0 ? cap : t;
        less += (k < key);
    }
    for (int o = 16; o > 0; o >>= 1) less += __shfl_xor_sync(0xffffffffu, less, o);
    if (lane == 0) s_warp[warp] = less;
    __syncthreads();
    if (tid == 0) {
        int v = 0;
        for (int w = 0; w < 8; ++w) v += s_warp[w];
        s_less = v;
        s_base = 0;
    }
    __syncthreads();
    const int start = s_less;
    for (int i0 = 0; i0 < T; i0 += 256) {
        const int i = i0 + tid;
        bool match = false;
        if (i < T) {
            const int t = tok_slot[i];
            match = ((t < 0 ? cap : t) == key);
        }
        const unsigned bal = __ballot_sync(0xffffffffu, match);
        __syncthreads();                       // s_warp / s_base of the previous chunk fully consumed
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int before = s_base;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        if (match && perm) perm[start + before + __popc(bal & ((1u << lane) - 1u))] = i;
        __syncthreads();
        if (tid == 0) {
            int v = s_base;
            for (int w = 0; w < 8; ++w) v += s_warp[w];
            s_base = v;
        }
    }
    __syncthreads();
    if (tid == 0) {
        if (slot_count) slot_count[key] = s_base;
        if (slot_offset) {
            slot_offset[key] = start;
            if (key == cap) slot_offset[cap + 1] = T;
        }
    }
}

// One CTA of 256 threads per 256-token plan tile.  Besides tok_slot it lists, for the tile, the 16-deep rank units of
// every tenant present (ascending slot order) and tells each token where its tenant's units start.
__global__ void __launch_bounds__(256) k_plan_tiles(int T, int S, const int32_t* __restrict__ seg_offsets,
                                                    const int32_t* __restrict__ seg_slot, int cap, int RP,
                                                    const int32_t* __restrict__ d_rank, int32_t* __restrict__ tok_slot,
                                                    int32_t* __restrict__ tok_uoff, int32_t* __restrict__ tile_nunits,
                                                    int32_t* __restrict__ tile_units, int umax, int32_t* status) {
    __shared__ int s_u[4096];
    __shared__ int s_warp[8];
    // the next kernel of the call may be launched now: it waits (griddepcontrol.wait) before it reads the plan
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = blockIdx.x;
    const int i = m * 256 + tid;
    if (S >= 0) {   // table checks, spread over the grid
        for (int s = blockIdx.x * 256 + tid; s < S; s += gridDim.x * 256) {
            const int a = seg_offsets[s], b = seg_offsets[s + 1];
            if (b < a || a < 0 || b > T) report(status, DEV_BAD_TABLE, s);
            if (s == 0 && a != 0) report(status, DEV_BAD_TABLE, -1);
            if (s == S - 1 && b != T) report(status, DEV_BAD_TABLE, -2);
        }
        if (i == 0 && S == 0 && T != 0) report(status, DEV_BAD_TABLE, -3);
    }
    int slot = -1;
    if (i < T) {
        if (S >= 0) {
            int lo = 0, hi = S;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (seg_offsets[mid + 1] > i) hi = mid; else lo = mid + 1;
            }
            if (lo < S) slot = seg_slot[lo];
        } else {
            slot = tok_slot[i];
        }
        if (slot < -1 || slot >= cap) {
            report(status, DEV_BAD_INDEX, i);
            slot = -1;
        }
        tok_slot[i] = slot;
    }
    for (int t = tid; t < cap; t += 256) s_u[t] = 0;
    __syncthreads();
    const int r = slot >= 0 ? d_rank[slot] : 0;
    if (r > 0) s_u[slot] = (r + 15) >> 4;
    __syncthreads();
    // exclusive scan of the per-slot unit counts; each thread owns a contiguous run of slots
    const int per = (cap + 255) / 256;
    const int t0 = tid * per, t1 = min(cap, t0 + per);
    int loc = 0;
    for (int t = t0; t < t1; ++t) loc += s_u[t];
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
    for (int t = t0; t < t1; ++t) {
        const int u = s_u[t];
        for (int j = 0; j < u; ++j)
            if (off + j < umax) tile_units[(size_t)m * umax + off + j] = t * RP + j * 16;
        s_u[t] = off;
        off += u;
    }
    __syncthreads();
    if (i < T) tok_uoff[i] = r > 0 ? s_u[slot] : -1;
    if (tid == 0) tile_nunits[m] = min(total, umax);
}

marlaas_status_t launch_plan_tiles(const marlaas_pool* pool, int64_t T, int32_t S, const int32_t* seg_offsets,
                                   const int32_t* seg_slot, const Workspace& ws, cudaStream_t st) {
    if (T <= 0) return MARLAAS_OK;
    k_plan_tiles<<<(unsigned)cdiv(T, 256), 256, 0, st>>>((int)T, S, seg_offsets, seg_slot, pool->cap, pool->RP,
                                                         pool->d_rank, ws.tok_slot, ws.tok_uoff, ws.tile_nunits,
                                                         ws.tile_units, ws.umax, pool->d_status);
    MARLAAS_LAUNCH_CHECK("k_plan_tiles");
    return MARLAAS_OK;
}

marlaas_status_t launch_tok_slot(const marlaas_pool* pool, int64_t T, int32_t S, const int32_t* seg_offsets,
                                 const int32_t* seg_slot, int32_t* tok_slot, cudaStream_t st) {
    const int64_t n = T > S ? T : S;
    if (n <= 0) return MARLAAS_OK;
    k_tok_slot<<<(unsigned)cdiv(n, 256), 256, 0, st>>>((int)T, S, seg_offsets, seg_slot, pool->cap, tok_slot,
                                                       pool->d_status);
    MARLAAS_LAUNCH_CHECK("k_tok_slot");
    return MARLAAS_OK;
}

marlaas_status_t launch_slot_sort(const marlaas_pool* pool, int64_t T, const int32_t* tok_slot,
                                  int32_t* slot_count, int32_t* slot_offset, int32_t* perm, cudaStream_t st,
                                  const int32_t* run_flag) {
    k_slot_sort<<<pool->cap + 1, 256, 0, st>>>((int)T, pool->cap, tok_slot, slot_count, slot_offset, perm, run_flag);
    MARLAAS_LAUNCH_CHECK("k_slot_sort");
    return MARLAAS_OK;
}

}  // namespace marlaas
