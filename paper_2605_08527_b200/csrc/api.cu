// The exported layer calls: argument validation on the host, then the kernel sequence on the caller's stream.
#include <string.h>

#include <mutex>

#include "internal.cuh"

namespace marlaas {

Workspace carve_workspace(const marlaas_pool* pool, int64_t T, void* base) {
    Workspace w;
    char* p = (char*)base;
    size_t o = 0;
    const size_t Tn = (size_t)(T > 0 ? T : 1);
    auto take = [&](size_t bytes) { char* q = p ? p + o : nullptr; o += align_up(bytes, 256); return q; };
    // 1. The plan of the batch (forward and backward): its layout depends on T, the capacity and the rank stride only, so
    //    that pools of one layer (same capacity and max_rank, whatever their widths and however many projections they hold)
    //    find one another's plan in a shared workspace (MARLAAS_FLAG_REUSE_PLAN).
    w.tok_slot = (int32_t*)take(sizeof(int32_t) * Tn);
    const size_t ntiles = (Tn + 255) / 256;
    w.umax = (pool->cap < 256 ? pool->cap : 256) * (pool->RP / 16);
    w.tok_uoff = (int32_t*)take(sizeof(int32_t) * Tn);
    w.tile_nunits = (int32_t*)take(sizeof(int32_t) * ntiles);
    w.tile_units = (int32_t*)take(sizeof(int32_t) * ntiles * (size_t)w.umax);
    w.perm = (int32_t*)take(sizeof(int32_t) * Tn);
    w.slot_count = (int32_t*)take(sizeof(int32_t) * (size_t)(pool->cap + 1));
    w.slot_offset = (int32_t*)take(sizeof(int32_t) * (size_t)(pool->cap + 2));
    w.dA_ptrs = (float**)take(sizeof(float*) * (size_t)pool->cap);
    w.dB_ptrs = (float**)take(sizeof(float*) * (size_t)pool->cap);
    const size_t nblk = (Tn + 63) / 64;
    const bool grad_tc = grad_sm100_eligible(pool, (int64_t)Tn);
    w.HW = ((2 * pool->RP + 63) / 64) * 64;
    w.max_copies = grad_tc ? (int32_t)(3 * nblk + 2 * (size_t)pool->cap) : 0;
    const size_t gb = grad_tc ? nblk : 0, gc = grad_tc ? (size_t)pool->cap : 0;
    w.blk_np = (int32_t*)take(sizeof(int32_t) * gb);
    w.blk_base = (int32_t*)take(sizeof(int32_t) * (gb + 1));
    w.blk_rank = (int32_t*)take(sizeof(int32_t) * gb * gc);
    w.ten_nblk = (int32_t*)take(sizeof(int32_t) * gc);
    w.ten_blks = (int32_t*)take(sizeof(int32_t) * gb * gc);
    w.ten_pos = (int32_t*)take(sizeof(int32_t) * gb * gc);
    w.gflag = (int32_t*)take(16);
    // 2. What a forward call writes besides: a pool over P projections keeps one plane of h and hd per projection.
    const size_t P = (size_t)pool->P;
    w.h = (float*)take(sizeof(float) * P * Tn * pool->RP);
    w.hd = (bf16*)take(sizeof(bf16) * P * Tn * align_up((size_t)w.umax * 16, 64));   // decode path: pitch in whole 64-column panels
    w.fwd_min = o;
    w.xbuf = (float*)take(decode_wide_sm100_xbuf_bytes(pool, (int64_t)Tn));
    w.fwd_total = o;
    // 3. Backward only.
    w.g = (float*)take(sizeof(float) * P * Tn * pool->RP);
    w.hm = (bf16*)take(sizeof(bf16) * (size_t)w.max_copies * 64 * (size_t)w.HW);
    w.hm2 = (bf16*)take(sizeof(bf16) * (size_t)w.max_copies * 64 * (size_t)w.HW);
    w.total = o;
    return w;
}

static bool aligned16(const void* p) { return (((uintptr_t)p) & 15) == 0; }

static marlaas_status_t check_matrix(const char* fn, const char* name, const void* p, int64_t ld, int64_t cols) {
    if (!p) return fail(MARLAAS_ERR_INVALID_ARG, "%s: %s is NULL", fn, name);
    if (!aligned16(p)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: %s is not 16-byte aligned", fn, name);
    if (ld < cols || (ld % 8) != 0)
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: leading dimension of %s (%lld) must be >= %lld and a multiple of 8",
                    fn, name, (long long)ld, (long long)cols);
    return MARLAAS_OK;
}

// Validates the table argument; for host tables also validates the contents and expands them into
// host_tok_slot (so that nothing is launched for a malformed table).
static marlaas_status_t check_segments(const char* fn, const marlaas_pool* pool, int64_t T,
                                       const marlaas_segments_t* seg, uint32_t flags,
                                       std::vector<int32_t>* host_tok_slot) {
    if (!seg) return fail(MARLAAS_ERR_INVALID_ARG, "%s: segment table is NULL", fn);
    if (seg->num_segments < 0) return fail(MARLAAS_ERR_INVALID_ARG, "%s: negative segment count", fn);
    if (T > 0 && (seg->num_segments == 0 || !seg->seg_offsets || !seg->seg_slot))
        return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "%s: empty segment table for %lld tokens", fn, (long long)T);
    if (!(flags & MARLAAS_FLAG_HOST_TABLE)) return MARLAAS_OK;
    const int32_t S = seg->num_segments;
    if (S > 0 && (!seg->seg_offsets || !seg->seg_slot))
        return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "%s: segment arrays are NULL", fn);
    if (S > 0 && seg->seg_offsets[0] != 0)
        return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "%s: seg_offsets[0] = %d, expected 0", fn, seg->seg_offsets[0]);
    if (S > 0 && seg->seg_offsets[S] != T)
        return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "%s: seg_offsets[S] = %d, expected T = %lld", fn,
                    seg->seg_offsets[S], (long long)T);
    host_tok_slot->assign((size_t)T, -1);
    for (int32_t s = 0; s < S; ++s) {
        const int32_t a = seg->seg_offsets[s], b = seg->seg_offsets[s + 1];
        if (b < a) return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "%s: seg_offsets decreases at segment %d", fn, s);
        const int32_t t = seg->seg_slot[s];
        if (t < -1 || t >= pool->cap)
            return fail(MARLAAS_ERR_BAD_SEGMENT_TABLE, "%s: segment %d names slot %d outside [-1,%d)", fn, s, t,
                        pool->cap);
        if (t >= 0 && !pool->slots[t].used)
            return fail(MARLAAS_ERR_UNKNOWN_TENANT, "%s: segment %d names slot %d, which holds no adapter", fn, s, t);
        for (int32_t i = a; i < b; ++i) (*host_tok_slot)[i] = t;
    }
    return MARLAAS_OK;
}

static marlaas_status_t make_tok_slot(const marlaas_pool* pool, int64_t T, const marlaas_segments_t* seg,
                                      uint32_t flags, const std::vector<int32_t>& host_tok_slot, int32_t* tok_slot,
                                      cudaStream_t st) {
    if (T <= 0) return MARLAAS_OK;
    if (flags & MARLAAS_FLAG_HOST_TABLE) {
        // pageable source: the runtime stages it before returning, so the vector may die after this call
        MARLAAS_CUDA_TRY(cudaMemcpyAsync(tok_slot, host_tok_slot.data(), sizeof(int32_t) * (size_t)T,
                                         cudaMemcpyHostToDevice, st));
        return MARLAAS_OK;
    }
    return launch_tok_slot(pool, T, seg->num_segments, seg->seg_offsets, seg->seg_slot, tok_slot, st);
}

static marlaas_status_t make_plan(const marlaas_pool* pool, int64_t T, const marlaas_segments_t* seg, uint32_t flags,
                                  const std::vector<int32_t>& host_tok_slot, const Workspace& ws, cudaStream_t st) {
    if (T <= 0) return MARLAAS_OK;
    if (flags & MARLAAS_FLAG_HOST_TABLE) {
        MARLAAS_CUDA_TRY(cudaMemcpyAsync(ws.tok_slot, host_tok_slot.data(), sizeof(int32_t) * (size_t)T,
                                         cudaMemcpyHostToDevice, st));
        return launch_plan_tiles(pool, T, -1, nullptr, nullptr, ws, st);
    }
    return launch_plan_tiles(pool, T, seg->num_segments, seg->seg_offsets, seg->seg_slot, ws, st);
}

// Shrink for the tensor-core path: batches with several 128-token tiles go through the tcgen05 kernel, small
// (decode-shaped) batches through the per-token gather kernel, which spreads over more SMs.
static marlaas_status_t shrink(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                               const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st,
                               bool out_is_zero = false) {
    if (T >= 512 && shrink_split_sm100_eligible(pool, T, D))
        return launch_shrink_split_sm100(pool, T, src, ld, D, store, sld, ws, out, st, out_is_zero);
    if (T >= 512) return launch_shrink_sm100(pool, T, src, ld, D, store, sld, ws, out, st);
    return launch_shrink_hd(pool, T, src, ld, D, store, sld, ws, out, st);
}

// Projection p of a pool over several: the plan (per-token slots, unit lists, gradient block lists) is shared, h, g and hd
// are planes of T rows each.
static Workspace part_workspace(const marlaas_pool* pool, const Workspace& ws, int p, int64_t T) {
    Workspace w = ws;
    w.h = ws.h + (size_t)p * T * pool->RP;
    w.g = ws.g + (size_t)p * T * pool->RP;
    w.hd = ws.hd + (size_t)p * T * ((size_t)ws.umax * 16);
    return w;
}

static void set_parts(const marlaas_pool* pool, GemmOperands* o, bool all_parts) {
    o->parts = pool->P;
    o->all_parts = all_parts;
    for (int p = 0; p < pool->P; ++p) o->part_end[p] = pool->part_begin[p + 1];
}

// Host tables are copied from temporaries of the call: a stream capture would keep pointers into them for its replays.
static marlaas_status_t reject_host_table_in_capture(const char* fn, uint32_t flags, cudaStream_t st) {
    if (!(flags & MARLAAS_FLAG_HOST_TABLE)) return MARLAAS_OK;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    MARLAAS_CUDA_TRY(cudaStreamIsCapturing(st, &cs));
    if (cs != cudaStreamCaptureStatusNone)
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: MARLAAS_FLAG_HOST_TABLE cannot be used while the stream is being captured", fn);
    return MARLAAS_OK;
}

static marlaas_status_t finish(marlaas_pool* pool, uint32_t flags, cudaStream_t st) {
    if (flags & MARLAAS_FLAG_VALIDATE_SYNC) return marlaas_check_status(pool, (void*)st);
    return MARLAAS_OK;
}

}  // namespace marlaas

using namespace marlaas;

extern "C" {

size_t marlaas_lora_workspace_bytes(const marlaas_pool_t* pool, int64_t T) {
    if (!pool || T < 0) return 0;
    return carve_workspace(pool, T, nullptr).total;
}

size_t marlaas_lora_forward_workspace_bytes(const marlaas_pool_t* pool, int64_t T) {
    if (!pool || T < 0) return 0;
    return carve_workspace(pool, T, nullptr).fwd_total;
}

size_t marlaas_lora_forward_workspace_min_bytes(const marlaas_pool_t* pool, int64_t T) {
    if (!pool || T < 0) return 0;
    return carve_workspace(pool, T, nullptr).fwd_min;
}

marlaas_status_t marlaas_lora_build_index(marlaas_pool_t* pool, int64_t T, const marlaas_segments_t* seg,
                                          int32_t* tok_slot, int32_t* slot_count, int32_t* slot_offset,
                                          int32_t* perm, void* workspace, size_t workspace_bytes, uint32_t flags,
                                          void* cuda_stream) {
    const char* fn = "lora_build_index";
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: pool is NULL", fn);
    if (T < 0 || T >= (1ll << 31)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: T out of range", fn);
    std::vector<int32_t> host_ts;
    marlaas_status_t rc = check_segments(fn, pool, T, seg, flags, &host_ts);
    if (rc != MARLAAS_OK) return rc;
    if (!workspace || ((uintptr_t)workspace & 255)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: workspace NULL or misaligned", fn);
    const Workspace ws = carve_workspace(pool, T, workspace);
    if (workspace_bytes < ws.total)
        return fail(MARLAAS_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < required %zu", fn, workspace_bytes, ws.total);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    if ((rc = reject_host_table_in_capture(fn, flags, st)) != MARLAAS_OK) return rc;
    int32_t* ts = tok_slot ? tok_slot : ws.tok_slot;
    rc = make_tok_slot(pool, T, seg, flags, host_ts, ts, st);
    if (rc != MARLAAS_OK) return rc;
    if (slot_count || slot_offset || perm) {
        rc = launch_slot_sort(pool, T, ts, slot_count, slot_offset, perm, st);
        if (rc != MARLAAS_OK) return rc;
    }
    return finish(pool, flags, st);
}

// The forward call: validation first (launch = false stops after it), then the kernel sequence on the stream.
static marlaas_status_t forward_impl(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx, const void* W,
                                     int64_t ldw, void* y, int64_t ldy, const marlaas_segments_t* seg,
                                     float* h_save, void* workspace, size_t workspace_bytes, uint32_t flags,
                                     void* cuda_stream, bool launch, const char* fn) {
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: pool is NULL", fn);
    if (T < 0 || T >= (1ll << 31)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: T out of range", fn);
    if (T == 0) return MARLAAS_OK;
    marlaas_status_t rc;
    if ((rc = check_matrix(fn, "x", x, ldx, pool->K)) != MARLAAS_OK) return rc;
    if ((rc = check_matrix(fn, "W", W, ldw, pool->N)) != MARLAAS_OK) return rc;
    if ((rc = check_matrix(fn, "y", y, ldy, pool->N)) != MARLAAS_OK) return rc;
    if (h_save && !aligned16(h_save)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: h_save is not 16-byte aligned", fn);
    std::vector<int32_t> host_ts;
    if ((rc = check_segments(fn, pool, T, seg, flags, &host_ts)) != MARLAAS_OK) return rc;
    if (!workspace || ((uintptr_t)workspace & 255)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: workspace NULL or misaligned", fn);
    Workspace ws = carve_workspace(pool, T, workspace);
    ws.early_shrink = (flags & MARLAAS_FLAG_OVERLAP_PREVIOUS) && !(flags & MARLAAS_FLAG_HOST_TABLE);
    if (workspace_bytes < ws.fwd_min)
        return fail(MARLAAS_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < required %zu", fn, workspace_bytes, ws.fwd_min);
    // between the minimum and the full forward size the scratch for exchanged partial sums is missing: the decode kernels
    // that split a contraction over CTA pairs are then left out (same results up to the summation order of those kernels)
    const bool has_xbuf = workspace_bytes >= ws.fwd_total;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    if ((rc = reject_host_table_in_capture(fn, flags, st)) != MARLAAS_OK) return rc;
    if (!launch) return MARLAAS_OK;

    float* h = h_save ? h_save : ws.h;
    const bool stream_k = has_xbuf && decode_stream_sm100_eligible(pool, T);
    if (!(flags & MARLAAS_FLAG_CUDA_CORE_PATH) && (stream_k || decode_sm100_eligible(pool, T))) {
        int32_t S = seg->num_segments;
        if (flags & MARLAAS_FLAG_HOST_TABLE) {
            MARLAAS_CUDA_TRY(cudaMemcpyAsync(ws.tok_slot, host_ts.data(), sizeof(int32_t) * (size_t)T,
                                             cudaMemcpyHostToDevice, st));
            S = -1;
        }
        {
            TimedLaunch timed(pool, st);
            rc = stream_k
                     ? launch_decode_stream_sm100(pool, T, (const bf16*)x, ldx, (const bf16*)W, ldw, (bf16*)y, ldy, S,
                                                  seg->seg_offsets, seg->seg_slot, ws, h, st)
                 : (decode_wide_sm100_eligible(pool, T) && (has_xbuf || !decode_wide_sm100_splits(pool, T)))
                     ? launch_decode_wide_sm100(pool, T, (const bf16*)x, ldx, (const bf16*)W, ldw, (bf16*)y, ldy, S,
                                                seg->seg_offsets, seg->seg_slot, ws, h, st)
                     : launch_decode_sm100(pool, T, (const bf16*)x, ldx, (const bf16*)W, ldw, (bf16*)y, ldy, S,
                                           seg->seg_offsets, seg->seg_slot, ws, h, st);
            if (rc != MARLAAS_OK) return rc;
        }
        return finish(pool, flags, st);
    }
    const int NP = pool->P;
    if (!(flags & MARLAAS_FLAG_CUDA_CORE_PATH)) {
        // h is cleared before the plan so that plan -> shrink -> GEMM are consecutive kernels (each is launched as a
        // programmatic dependent of the one before and overlaps its tail)
        const bool pre_zero = T >= 512 && shrink_split_sm100_eligible(pool, T, pool->K);
        if (pre_zero) MARLAAS_CUDA_TRY(cudaMemsetAsync(h, 0, sizeof(float) * (size_t)NP * T * pool->RP, st));
        if (!(flags & MARLAAS_FLAG_REUSE_PLAN) && (rc = make_plan(pool, T, seg, flags, host_ts, ws, st)) != MARLAAS_OK) return rc;
        // ONE shrink over all projections' blocks of A rows where the cluster kernel applies (x is read once; planes of h
        // and hd per projection), else one shrink per projection; then ONE product over the side-by-side W
        if (NP > 1 && T >= 512 && shrink_split_sm100_parts_eligible(pool, T, pool->K, NP)) {
            if ((rc = launch_shrink_split_sm100(pool, T, (const bf16*)x, ldx, pool->K, pool->d_At, pool->K, ws, h, st, pre_zero,
                                                NP)) != MARLAAS_OK) return rc;
        } else {
            for (int p = 0; p < NP; ++p) {
                const Workspace wp = part_workspace(pool, ws, p, T);
                if ((rc = shrink(pool, T, (const bf16*)x, ldx, pool->K, pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K, pool->K, wp,
                                 h + (size_t)p * T * pool->RP, st, pre_zero)) != MARLAAS_OK) return rc;
            }
        }
        GemmOperands o;
        o.M = T; o.Nout = pool->N; o.Kc = pool->K;
        o.A = (const bf16*)x; o.lda = ldx;
        o.B = (const bf16*)W; o.ldb = ldw; o.b_mn = true;
        o.C = (bf16*)y; o.ldc = ldy;
        o.XA = ws.hd; o.xa_cols = (int64_t)ws.umax * 16;
        o.XB = pool->d_Bs; o.xb_rows = (int64_t)pool->cap * pool->RP; o.xb_ld = pool->ldB;
        o.tile_nunits = ws.tile_nunits; o.tile_units = ws.tile_units; o.umax = ws.umax;
        set_parts(pool, &o, false);
        {
            TimedLaunch timed(pool, st);
            rc = (NP > 1 || gemm2_sm100_eligible(pool, T)) ? launch_gemm2_sm100(pool, o, st) : launch_gemm_sm100(pool, o, st);
            if (rc != MARLAAS_OK) return rc;
        }
        return finish(pool, flags, st);
    }
    if ((rc = make_tok_slot(pool, T, seg, flags, host_ts, ws.tok_slot, st)) != MARLAAS_OK) return rc;
    for (int p = 0; p < NP; ++p) {      // the plain kernels take one projection at a time
        const int64_t c0 = pool->part_begin[p], Np = pool->part_begin[p + 1] - c0;
        float* hp = h + (size_t)p * T * pool->RP;
        if ((rc = launch_rowdot(pool, T, (const bf16*)x, ldx, pool->K, pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K, pool->K,
                                ws.tok_slot, hp, st)) != MARLAAS_OK) return rc;
        TimedLaunch timed(pool, st);
        if ((rc = launch_gemm_cuda_core(pool, T, Np, pool->K, (const bf16*)x, ldx, (const bf16*)W + c0, ldw, false,
                                        (bf16*)y + c0, ldy, hp, pool->d_Bs + c0, pool->ldB, ws.tok_slot, st)) != MARLAAS_OK) return rc;
    }
    return finish(pool, flags, st);
}

marlaas_status_t marlaas_lora_forward(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx, const void* W,
                                      int64_t ldw, void* y, int64_t ldy, const marlaas_segments_t* seg,
                                      float* h_save, void* workspace, size_t workspace_bytes, uint32_t flags,
                                      void* cuda_stream) {
    return forward_impl(pool, T, x, ldx, W, ldw, y, ldy, seg, h_save, workspace, workspace_bytes, flags, cuda_stream, true,
                        "lora_forward");
}

marlaas_status_t marlaas_lora_forward_multi(int32_t n, const marlaas_forward_call_t* calls, uint32_t flags, void* cuda_stream) {
    const char* fn = "lora_forward_multi";
    if (n < 0 || (n > 0 && !calls)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: bad call list", fn);
    if (n == 0) return MARLAAS_OK;
    if (flags & (MARLAAS_FLAG_VALIDATE_SYNC | MARLAAS_FLAG_REUSE_PLAN | MARLAAS_FLAG_OVERLAP_PREVIOUS))
        return fail(MARLAAS_ERR_INVALID_ARG, "%s: VALIDATE_SYNC, REUSE_PLAN and OVERLAP_PREVIOUS do not apply to a set of concurrent calls", fn);
    marlaas_status_t rc;
    // every call is validated before anything is launched
    for (int i = 0; i < n; ++i) {
        const marlaas_forward_call_t& c = calls[i];
        if (!c.pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: call %d has no pool", fn, i);
        if (c.pool->device != calls[0].pool->device) return fail(MARLAAS_ERR_INVALID_ARG, "%s: the calls' pools are on different devices", fn);
        if ((rc = forward_impl(c.pool, c.T, c.x, c.ldx, c.W, c.ldw, c.y, c.ldy, c.seg, c.h_save, c.workspace, c.workspace_bytes, flags,
                               cuda_stream, false, fn)) != MARLAAS_OK) return rc;
        for (int j = 0; j < i; ++j) {
            const marlaas_forward_call_t& d = calls[j];
            if (c.pool == d.pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: calls %d and %d use the same pool", fn, j, i);
            const char *a0 = (const char*)c.workspace, *b0 = (const char*)d.workspace;
            if (c.T > 0 && d.T > 0 && a0 < b0 + d.workspace_bytes && b0 < a0 + c.workspace_bytes)
                return fail(MARLAAS_ERR_INVALID_ARG, "%s: calls %d and %d share workspace memory", fn, j, i);
        }
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int dev = calls[0].pool->device;
    MARLAAS_CUDA_TRY(cudaSetDevice(dev));
    if (n == 1 || dev < 0 || dev >= 64) {
        for (int i = 0; i < n; ++i) {
            const marlaas_forward_call_t& c = calls[i];
            if ((rc = forward_impl(c.pool, c.T, c.x, c.ldx, c.W, c.ldw, c.y, c.ldy, c.seg, c.h_save, c.workspace, c.workspace_bytes, flags,
                                   cuda_stream, true, fn)) != MARLAAS_OK) return rc;
        }
        return MARLAAS_OK;
    }
    // Fork: call 0 stays on the caller's stream, the others go to side streams of the device (created on first use, never
    // destroyed), round robin; join: the caller's stream waits for every side stream.  Events only: legal inside a capture.
    constexpr int NSIDE = 3;
    static std::mutex mu;
    static cudaStream_t side[64][NSIDE] = {};
    static cudaEvent_t ev_fork[64] = {}, ev_join[64][NSIDE] = {};
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!ev_fork[dev]) {
            for (int k = 0; k < NSIDE; ++k) {
                MARLAAS_CUDA_TRY(cudaStreamCreateWithFlags(&side[dev][k], cudaStreamNonBlocking));
                MARLAAS_CUDA_TRY(cudaEventCreateWithFlags(&ev_join[dev][k], cudaEventDisableTiming));
            }
            MARLAAS_CUDA_TRY(cudaEventCreateWithFlags(&ev_fork[dev], cudaEventDisableTiming));
        }
    }
    const int used = n - 1 < NSIDE ? n - 1 : NSIDE;
    MARLAAS_CUDA_TRY(cudaEventRecord(ev_fork[dev], st));
    for (int k = 0; k < used; ++k) MARLAAS_CUDA_TRY(cudaStreamWaitEvent(side[dev][k], ev_fork[dev], 0));
    marlaas_status_t first_err = MARLAAS_OK;
    for (int i = 0; i < n && first_err == MARLAAS_OK; ++i) {
        const marlaas_forward_call_t& c = calls[i];
        cudaStream_t cs = i == 0 ? st : side[dev][(i - 1) % NSIDE];
        first_err = forward_impl(c.pool, c.T, c.x, c.ldx, c.W, c.ldw, c.y, c.ldy, c.seg, c.h_save, c.workspace, c.workspace_bytes, flags,
                                 (void*)cs, true, fn);
    }
    // whatever happened, the side streams are joined again
    for (int k = 0; k < used; ++k) {
        MARLAAS_CUDA_TRY(cudaEventRecord(ev_join[dev][k], side[dev][k]));
        MARLAAS_CUDA_TRY(cudaStreamWaitEvent(st, ev_join[dev][k], 0));
    }
    return first_err;
}

marlaas_status_t marlaas_lora_backward(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx, const void* W,
                                       int64_t ldw, const void* dy, int64_t lddy, void* dx, int64_t lddx,
                                       float* const* dA_slots, float* const* dB_slots,
                                       const marlaas_segments_t* seg, const float* h_saved, void* workspace,
                                       size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    const char* fn = "lora_backward";
    if (!pool) return fail(MARLAAS_ERR_INVALID_ARG, "%s: pool is NULL", fn);
    if (T < 0 || T >= (1ll << 31)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: T out of range", fn);
    marlaas_status_t rc;
    const bool want_dA = dA_slots != nullptr, want_dB = dB_slots != nullptr;
    if (T > 0) {
        if ((rc = check_matrix(fn, "W", W, ldw, pool->N)) != MARLAAS_OK) return rc;
        if ((rc = check_matrix(fn, "dy", dy, lddy, pool->N)) != MARLAAS_OK) return rc;
        if (dx && (rc = check_matrix(fn, "dx", dx, lddx, pool->K)) != MARLAAS_OK) return rc;
        if ((want_dA || (want_dB && !h_saved)) && (rc = check_matrix(fn, "x", x, ldx, pool->K)) != MARLAAS_OK) return rc;
    }
    if (h_saved && !aligned16(h_saved)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: h_saved is not 16-byte aligned", fn);
    for (int s = 0; s < pool->cap; ++s) {
        if (want_dA && dA_slots[s] && ((uintptr_t)dA_slots[s] & 3)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: dA_slots[%d] misaligned", fn, s);
        if (want_dB && dB_slots[s] && ((uintptr_t)dB_slots[s] & 3)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: dB_slots[%d] misaligned", fn, s);
    }
    std::vector<int32_t> host_ts;
    if ((rc = check_segments(fn, pool, T, seg, flags, &host_ts)) != MARLAAS_OK) return rc;
    if (!workspace || ((uintptr_t)workspace & 255)) return fail(MARLAAS_ERR_INVALID_ARG, "%s: workspace NULL or misaligned", fn);
    const Workspace ws = carve_workspace(pool, T, workspace);
    if (workspace_bytes < ws.total)
        return fail(MARLAAS_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < required %zu", fn, workspace_bytes, ws.total);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    MARLAAS_CUDA_TRY(cudaSetDevice(pool->device));
    if ((rc = reject_host_table_in_capture(fn, flags, st)) != MARLAAS_OK) return rc;
    if (pool->P > 1 && pool->cap > 64 && (want_dA || want_dB)) {
        // the per-projection pointer tables of such a pool are temporaries of this call, copied by memcpy nodes
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        MARLAAS_CUDA_TRY(cudaStreamIsCapturing(st, &cs));
        if (cs != cudaStreamCaptureStatusNone)
            return fail(MARLAAS_ERR_INVALID_ARG, "%s: adapter gradients of a pool over several projections with more than 64 slots "
                        "cannot be captured", fn);
    }
    const bool acc = (flags & MARLAAS_FLAG_ACCUMULATE) != 0;

    const bool tc_path = !(flags & MARLAAS_FLAG_CUDA_CORE_PATH);
    const int NP = pool->P;
    const size_t plane = (size_t)T * pool->RP;      // floats per projection in h, g (and h_saved)
    const bool pre_zero = tc_path && T >= 512 && (dx || want_dA) && shrink_split_sm100_eligible(pool, T, pool->N);
    if (tc_path && T > 0) {
        if (pre_zero) MARLAAS_CUDA_TRY(cudaMemsetAsync(ws.g, 0, sizeof(float) * NP * plane, st));   // see forward
        if (!(flags & MARLAAS_FLAG_REUSE_PLAN) && (rc = make_plan(pool, T, seg, flags, host_ts, ws, st)) != MARLAAS_OK) return rc;
    } else {
        if ((rc = make_tok_slot(pool, T, seg, flags, host_ts, ws.tok_slot, st)) != MARLAAS_OK) return rc;
    }
    // g_p = dy[:, columns of projection p] B_p^T: one pass over dy in all
    if (T > 0 && (dx || want_dA)) {
        for (int p = 0; p < NP; ++p) {
            const int64_t c0 = pool->part_begin[p], Np = pool->part_begin[p + 1] - c0;
            const Workspace wp = part_workspace(pool, ws, p, T);
            if (tc_path) {
                if ((rc = shrink(pool, T, (const bf16*)dy + c0, lddy, Np, pool->d_Bs + c0, pool->ldB, wp, wp.g, st, pre_zero)) != MARLAAS_OK) return rc;
            } else {
                if ((rc = launch_rowdot(pool, T, (const bf16*)dy + c0, lddy, Np, pool->d_Bs + c0, pool->ldB, ws.tok_slot, wp.g, st)) != MARLAAS_OK) return rc;
            }
        }
    }
    // per-projection views of the caller's gradient tables: block p of dA_t is [K][r_t], block p of dB_t is [r_t][N_p]
    std::vector<float*> dA_part, dB_part;
    auto part_tables = [&](int p) {
        if (NP == 1) return;
        dA_part.assign((size_t)pool->cap, nullptr);
        dB_part.assign((size_t)pool->cap, nullptr);
        for (int s = 0; s < pool->cap; ++s) {
            const size_t r = (size_t)pool->slots[s].rank;
            if (want_dA && dA_slots[s]) dA_part[s] = dA_slots[s] + (size_t)p * pool->K * r;
            if (want_dB && dB_slots[s]) dB_part[s] = dB_slots[s] + r * (size_t)pool->part_begin[p];
        }
    };
    // The adapter-gradient kernels read none of the dx GEMM's output: when they need no further pass over the workspace
    // the GEMM uses (the saved h is given, the tensor-core reduction is certain to fit) they are issued on a side stream
    // of the pool, forked here and joined at the end, so that their small planning and copy kernels run beside the
    // GEMM instead of after it.
    const bool tc_grad0 = tc_path && (want_dA || want_dB) && grad_sm100_eligible(pool, T);
    const bool fits0 = tc_grad0 && cdiv(T, 64) + (int64_t)seg->num_segments <= (int64_t)ws.max_copies;
    const bool gemm2 = NP > 1 || gemm2_sm100_eligible(pool, T);
    const bool overlap = fits0 && T > 0 && dx && (!want_dB || h_saved) && gemm2_sm100_eligible(pool, T) && pool->cap <= 64;
    if (overlap) {
        if (!pool->side) {
            int lo = 0, hi = 0;
            MARLAAS_CUDA_TRY(cudaDeviceGetStreamPriorityRange(&lo, &hi));
            MARLAAS_CUDA_TRY(cudaStreamCreateWithPriority(&pool->side, cudaStreamNonBlocking, lo));   // lowest priority
            MARLAAS_CUDA_TRY(cudaEventCreateWithFlags(&pool->ev_fork, cudaEventDisableTiming));
            MARLAAS_CUDA_TRY(cudaEventCreateWithFlags(&pool->ev_join, cudaEventDisableTiming));
        }
        MARLAAS_CUDA_TRY(cudaEventRecord(pool->ev_fork, st));
    }
    if (T > 0 && dx && tc_path) {
        GemmOperands o;
        o.M = T; o.Nout = pool->K; o.Kc = pool->N;
        o.A = (const bf16*)dy; o.lda = lddy;
        o.B = (const bf16*)W; o.ldb = ldw; o.b_mn = false;
        o.C = (bf16*)dx; o.ldc = lddx;
        o.XA = ws.hd; o.xa_cols = (int64_t)ws.umax * 16;
        o.XB = pool->d_At; o.xb_rows = (int64_t)NP * pool->cap * pool->RP; o.xb_ld = pool->K;
        o.tile_nunits = ws.tile_nunits; o.tile_units = ws.tile_units; o.umax = ws.umax;
        set_parts(pool, &o, true);      // the low-rank term of dx sums over every projection
        TimedLaunch timed(pool, st);
        rc = gemm2 ? launch_gemm2_sm100(pool, o, st) : launch_gemm_sm100(pool, o, st);
        if (rc != MARLAAS_OK) return rc;
    } else if (T > 0 && dx) {
        TimedLaunch timed(pool, st);
        if ((rc = launch_gemm_cuda_core(pool, T, pool->K, pool->N, (const bf16*)dy, lddy, (const bf16*)W, ldw, true,
                                        (bf16*)dx, lddx, ws.g, pool->d_At, pool->K, ws.tok_slot, st, NP, (int64_t)plane)) != MARLAAS_OK) return rc;
    }
    if (want_dA || want_dB) {
        const bool tc_grad = tc_path && grad_sm100_eligible(pool, T);
        // The tensor-core reduction needs one copy of a 64-token block per tenant present in it; there are at most
        // (blocks + segments) of them, so when that bound fits the workspace the CUDA-core fallback cannot be needed
        // and neither it, nor the sort it consumes, nor the device copies of the pointer tables are issued.
        const int64_t nblk = cdiv(T, 64);
        const bool fits = tc_grad && nblk + (int64_t)seg->num_segments <= (int64_t)ws.max_copies;
        const bool inline_tables = fits && pool->cap <= 64;
        const int32_t* run_flag = tc_grad ? ws.gflag : nullptr;   // the CUDA-core kernels run only if the flag is set
        if (overlap) {
            cudaStream_t gs = pool->side;
            MARLAAS_CUDA_TRY(cudaStreamWaitEvent(gs, pool->ev_fork, 0));
            // whatever happens from here on, the side stream is joined again before the call returns: a forked stream left
            // unjoined would invalidate a capture the caller's stream may be part of
            auto side_work = [&]() -> marlaas_status_t {
                marlaas_status_t r;
                for (int p = 0; p < NP; ++p) {
                    if (p == 0 && !(flags & MARLAAS_FLAG_REUSE_PLAN)) {
                        if ((r = launch_grad_plan(pool, T, ws, gs)) != MARLAAS_OK) return r;
                    } else {
                        // the plan kernel also zeroes the reductions' work-item counters; a reused plan needs them zeroed again
                        MARLAAS_CUDA_TRY(cudaMemsetAsync(ws.gflag + 2, 0, 2 * sizeof(int32_t), gs));
                    }
                    part_tables(p);
                    float* const* dAp = NP == 1 ? dA_slots : dA_part.data();
                    float* const* dBp = NP == 1 ? dB_slots : dB_part.data();
                    const int64_t c0 = pool->part_begin[p], Np = pool->part_begin[p + 1] - c0;
                    const bf16* dyp = (const bf16*)dy + c0;
                    const float* hp = h_saved ? h_saved + p * plane : nullptr;
                    const float* gp = ws.g + p * plane;
                    // both sets of copies first (small kernels that fit beside the GEMM's CTAs), then the two reductions
                    if (want_dB && (r = launch_grad_sm100(pool, T, Np, dyp, lddy, hp, nullptr, dBp, false, acc, ws,
                                                          gs, ws.hm, GRAD_PHASE_COPIES)) != MARLAAS_OK) return r;
                    if (want_dA && (r = launch_grad_sm100(pool, T, pool->K, (const bf16*)x, ldx, gp, nullptr, dAp, true, acc, ws,
                                                          gs, ws.hm2, GRAD_PHASE_COPIES)) != MARLAAS_OK) return r;
                    if (want_dB && (r = launch_grad_sm100(pool, T, Np, dyp, lddy, hp, nullptr, dBp, false, acc, ws,
                                                          gs, ws.hm, GRAD_PHASE_REDUCE)) != MARLAAS_OK) return r;
                    // the dA reduction reads x and its own copies (made above), nothing of the dB reduction: started behind it
                    // as a programmatic dependent, its CTAs take the SMs that the dB reduction's CTAs leave one by one
                    if (want_dA && (r = launch_grad_sm100(pool, T, pool->K, (const bf16*)x, ldx, gp, nullptr, dAp, true, acc, ws,
                                                          gs, ws.hm2, GRAD_PHASE_REDUCE | (want_dB ? GRAD_PHASE_EARLY : 0))) != MARLAAS_OK) return r;
                }
                return MARLAAS_OK;
            };
            rc = side_work();
            MARLAAS_CUDA_TRY(cudaEventRecord(pool->ev_join, gs));
            MARLAAS_CUDA_TRY(cudaStreamWaitEvent(st, pool->ev_join, 0));
            if (rc != MARLAAS_OK) return rc;
            return finish(pool, flags, st);
        }
        if (tc_grad && !(flags & MARLAAS_FLAG_REUSE_PLAN) && (rc = launch_grad_plan(pool, T, ws, st)) != MARLAAS_OK) return rc;
        if (!fits && (rc = launch_slot_sort(pool, T, ws.tok_slot, ws.slot_count, ws.slot_offset, ws.perm, st, run_flag)) != MARLAAS_OK) return rc;
        // h was not kept: recomputed here, for all projections of the pool in one pass over x where the cluster kernel applies
        bool h_all = false;
        if (want_dB && !h_saved && tc_path && NP > 1 && T >= 512 && shrink_split_sm100_parts_eligible(pool, T, pool->K, NP)) {
            if ((rc = launch_shrink_split_sm100(pool, T, (const bf16*)x, ldx, pool->K, pool->d_At, pool->K, ws, ws.h, st, false,
                                                NP)) != MARLAAS_OK) return rc;
            h_all = true;
        }
        for (int p = 0; p < NP; ++p) {
            if (tc_grad && (p > 0 || (flags & MARLAAS_FLAG_REUSE_PLAN)))
                MARLAAS_CUDA_TRY(cudaMemsetAsync(ws.gflag + 2, 0, 2 * sizeof(int32_t), st));
            part_tables(p);
            float* const* dAp = NP == 1 ? dA_slots : dA_part.data();
            float* const* dBp = NP == 1 ? dB_slots : dB_part.data();
            const int64_t c0 = pool->part_begin[p], Np = pool->part_begin[p + 1] - c0;
            const bf16* dyp = (const bf16*)dy + c0;
            const Workspace wp = part_workspace(pool, ws, p, T);
            if (want_dB) {
                const float* h = h_saved ? h_saved + p * plane : nullptr;
                if (!h && h_all) h = wp.h;
                if (!h && T > 0) {
                    const bf16* Ap = pool->d_At + (size_t)p * pool->cap * pool->RP * pool->K;
                    if (tc_path) rc = shrink(pool, T, (const bf16*)x, ldx, pool->K, Ap, pool->K, wp, wp.h, st);
                    else rc = launch_rowdot(pool, T, (const bf16*)x, ldx, pool->K, Ap, pool->K, ws.tok_slot, wp.h, st);
                    if (rc != MARLAAS_OK) return rc;
                    h = wp.h;
                }
                if (!inline_tables)
                    MARLAAS_CUDA_TRY(cudaMemcpyAsync(ws.dB_ptrs, dBp, sizeof(float*) * (size_t)pool->cap, cudaMemcpyHostToDevice, st));
                if (tc_grad && (rc = launch_grad_sm100(pool, T, Np, dyp, lddy, h, ws.dB_ptrs, dBp, false, acc, ws, st, ws.hm)) != MARLAAS_OK) return rc;
                if (!fits && (rc = launch_grad_reduce(pool, Np, dyp, lddy, h, ws.perm, ws.slot_offset, ws.dB_ptrs,
                                                      false, acc, st, run_flag)) != MARLAAS_OK) return rc;
            }
            if (want_dA) {
                if (!inline_tables)
                    MARLAAS_CUDA_TRY(cudaMemcpyAsync(ws.dA_ptrs, dAp, sizeof(float*) * (size_t)pool->cap, cudaMemcpyHostToDevice, st));
                if (tc_grad && (rc = launch_grad_sm100(pool, T, pool->K, (const bf16*)x, ldx, wp.g, ws.dA_ptrs, dAp, true, acc, ws, st, ws.hm)) != MARLAAS_OK) return rc;
                if (!fits && (rc = launch_grad_reduce(pool, pool->K, (const bf16*)x, ldx, wp.g, ws.perm, ws.slot_offset, ws.dA_ptrs,
                                                      true, acc, st, run_flag)) != MARLAAS_OK) return rc;
            }
        }
    }
    return finish(pool, flags, st);
}

}  // extern "C"
