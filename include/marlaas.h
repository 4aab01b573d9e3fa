/* marlaas.h -- C ABI of the B200 multi-tenant LoRA linear layer.
 *
 * The layer is the one every adapted projection of the shared base model runs when many tenants
 * share one frozen base weight through lightweight LoRA adapters (paper: abstract; Introduction;
 * Methods, "Multi-Task Manager" -- per-task LoRA parameters theta_t^(v) with a version counter --
 * and "Multi-LoRA Rollout with Single-Task Training" -- rollouts batched across tasks by multi-LoRA
 * kernels; Algorithm 1 "Commit updated parameters").  For a token i routed to tenant slot t:
 *
 *     y_i  = x_i W + s_t (x_i A_t) B_t                              (forward: rollout decode and training)
 *     dx_i = dy_i W^T + s_t (dy_i B_t^T) A_t^T                      (backward)
 *     dA_t = s_t sum_{i:t(i)=t} x_i^T (dy_i B_t^T)      dB_t = s_t sum_{i:t(i)=t} (x_i A_t)^T dy_i
 *
 * W is d_in x d_out (K x N), A_t is K x r_t, B_t is r_t x N, s_t = alpha_t / r_t; everything is
 * row-major; x, W, A, B, y, dy, dx are bf16 (1-8-7, round-to-nearest-even on output), sums are
 * carried in fp32, dA_t and dB_t are fp32.  W is frozen: there is no dW.
 *
 * Conventions
 *  - All data pointers are DEVICE pointers on the pool's device unless a comment says HOST.
 *  - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the legacy default
 *    stream) and the calls return without synchronising unless MARLAAS_FLAG_VALIDATE_SYNC is given.
 *    The caller keeps every buffer alive and unmodified until the stream has passed the call.
 *  - The library never allocates or frees device memory: the adapter store and the per-call workspace
 *    are caller-provided (sizes from the *_bytes functions).
 *  - Every function returns MARLAAS_OK (0) or a negative marlaas_status_t; nothing throws or aborts.
 *    marlaas_last_error() gives a thread-local message for the last failure on this thread.
 *  - Arguments are validated on the host BEFORE anything is launched; a failing call launches nothing.
 *  - A pool may be used from one host thread at a time.
 *  - Required alignment: every bf16 pointer 16-byte aligned, every leading dimension a multiple of 8
 *    elements, d_in and d_out multiples of 8.
 */
#ifndef MARLAAS_H_
#define MARLAAS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct marlaas_pool marlaas_pool_t; /* opaque; one pool per adapted projection (d_in, d_out) */
typedef int32_t marlaas_status_t;

enum {
    MARLAAS_OK = 0,
    MARLAAS_ERR_INVALID_ARG = -1,        /* null / misaligned pointer, negative size, leading dim too small */
    MARLAAS_ERR_BAD_SEGMENT_TABLE = -2,  /* offsets not 0..T non-decreasing (host tables: before launch; device
                                            tables: reported by marlaas_check_status) */
    MARLAAS_ERR_UNKNOWN_TENANT = -3,
    MARLAAS_ERR_RANK_TOO_LARGE = -4,
    MARLAAS_ERR_POOL_FULL = -5,
    MARLAAS_ERR_UNSUPPORTED_DEVICE = -6, /* not an sm_100 device, or no CUDA device */
    MARLAAS_ERR_CUDA = -7,               /* a CUDA runtime / driver call failed */
    MARLAAS_ERR_DEVICE_TIMEOUT = -8,     /* a bounded wait inside a kernel ran out; results of that call are invalid */
    MARLAAS_ERR_DEVICE_BAD_INDEX = -9,   /* a device-side check met a slot outside [-1, capacity): that token was
                                            computed with the base weight only */
    MARLAAS_ERR_WORKSPACE_TOO_SMALL = -10
};

enum {
    MARLAAS_FLAG_ACCUMULATE = 1u,     /* backward: dA_t, dB_t += instead of overwrite */
    MARLAAS_FLAG_HOST_TABLE = 2u,     /* seg_offsets / seg_slot are HOST arrays: validated on the host, then copied
                                         into the workspace in stream order (not while the stream is being captured:
                                         refused with MARLAAS_ERR_INVALID_ARG) */
    MARLAAS_FLAG_VALIDATE_SYNC = 4u,  /* synchronise the stream after the call and return the device status word */
    MARLAAS_FLAG_CUDA_CORE_PATH = 8u, /* diagnostics: run the plain CUDA-core kernels instead of the tcgen05 path */
    MARLAAS_FLAG_REUSE_PLAN = 16u,    /* the workspace still holds the plan of the previous call of the same kind
                                         (forward after forward, backward after backward) and that call had the same T,
                                         the same segment table contents and a pool of the same capacity and max_rank:
                                         the per-token slots and per-tile unit lists are not rebuilt.  For the
                                         projections of one decoder layer, which all see the same mixed batch.  The
                                         caller vouches for the condition; batches of at most 1024 tokens ignore the
                                         flag (their plan is built inside the first kernel anyway). */
    MARLAAS_FLAG_OVERLAP_PREVIOUS = 32u /* forward, decode-shaped batches (at most 1024 tokens): the caller states that the
                                         work submitted to the stream immediately before this call -- typically the same
                                         layer's call for another micro-batch of a serving loop that interleaves two --
                                         is independent of it: it does not produce this call's x, W or segment table,
                                         and it touches neither this call's workspace, y, h_save nor its pool.  The
                                         call's first kernel (the shrink) is then launched behind that work as a
                                         programmatic dependent that does not wait for it, and runs beside the end of
                                         it; a preceding marlaas_lora_forward lets it start once its own shrink has
                                         completed, so at most two consecutive calls are in flight together (two
                                         workspaces and two pools, used in turn, satisfy the condition).  Stream order
                                         holds for everything submitted after the call: it never completes before its
                                         predecessor.  Results are bit-identical with and without the flag.  Ignored
                                         for larger batches and with MARLAAS_FLAG_HOST_TABLE; refused by
                                         marlaas_lora_forward_multi and marlaas_lora_forward_static_ws.  If the
                                         condition does not hold the call races with its predecessor. */
};

/* Token-to-adapter segment table of one mixed batch: segment s covers tokens
 * [seg_offsets[s], seg_offsets[s+1]) and routes them to pool slot seg_slot[s] (-1 = base weight only).
 * seg_offsets[0] = 0, non-decreasing, seg_offsets[S] = T; zero-length segments are allowed; a slot may
 * recur in any number of non-adjacent segments.  An unsorted decode batch is T segments of one token.
 * The arrays are device memory unless MARLAAS_FLAG_HOST_TABLE is set. */
typedef struct {
    int32_t num_segments;       /* S >= 0 */
    const int32_t* seg_offsets; /* [S+1] */
    const int32_t* seg_slot;    /* [S]   */
} marlaas_segments_t;

/* ---- pooled adapter store (the manager's per-task parameters theta_t^(v), "Multi-Task Manager") ---- */

/* Bytes of device memory a pool of `capacity` slots needs (0 if the arguments are invalid).
 * max_rank in [1,128]; ranks are stored padded to a multiple of 16 with zero rows (exact). */
size_t marlaas_adapter_pool_storage_bytes(int64_t d_in, int64_t d_out, int32_t max_rank, int32_t capacity);

/* Create a pool over caller-owned device memory `storage` (256-byte aligned, >= storage_bytes, on
 * `device`); clears it in stream order.  The pool object itself is host memory freed by _destroy; the
 * storage stays the caller's.  Fails with UNSUPPORTED_DEVICE unless `device` has compute capability 10.x. */
marlaas_status_t marlaas_adapter_pool_create(marlaas_pool_t** out, int device, int64_t d_in, int64_t d_out,
                                             int32_t max_rank, int32_t capacity, void* storage,
                                             size_t storage_bytes, void* cuda_stream);
marlaas_status_t marlaas_adapter_pool_destroy(marlaas_pool_t* pool);

/* One pool for several projections that read the same activations (q, k, v; gate, up), served as ONE layer of width
 * d_out = part_d_out[0] + ... + part_d_out[n_parts-1] whose weight is the projections' weights side by side,
 * W = [W_1 | ... | W_P] (paper: Methods, "Multi-LoRA Rollout with Single-Task Training" -- every adapted projection of
 * the shared base model serves all tenants' tokens at once; Introduction -- rollout dominates the run time, so the
 * decode-shaped pass over the projections of a decoder layer is what one such call shortens).  Tenant t holds one
 * adapter pair per projection, all of the tenant's rank r_t and scale s_t:
 *
 *     y_i[:, columns of projection p] = x_i W_p + s_t (x_i A_t,p) B_t,p
 *
 * The store keeps one block of A rows per projection and the B matrices side by side ([r_t][d_out]): nothing is stored
 * or streamed for the zero blocks that the projections' adapters would have as one block-diagonal adapter of rank P r_t.
 * 1 <= n_parts <= 4; every part_d_out[p] is a positive multiple of 256.  On such a pool
 *  - register / export / adamw_commit take A as n_parts blocks [d_in][rank] one after another and B as n_parts blocks
 *    [rank][part_d_out[p]] one after another (the projections' own matrices, concatenated in memory); the fp32 masters,
 *    moments and gradients of adamw_commit and the dA_t / dB_t of backward have the same block layout;
 *  - forward / backward take W with d_out columns (the projections' weights side by side, leading dimension ldw),
 *    y / dy with d_out columns, and dx sums over the projections;
 *  - h_save / h_saved are [n_parts][T][rank_stride] (one plane per projection);
 *  - marlaas_lora_forward_static_ws and MARLAAS_FLAG_REUSE_PLAN work as on any pool.
 * With n_parts = 1 the pool is an ordinary one (but for the multiple-of-256 rule). */
size_t marlaas_adapter_pool_storage_bytes_segmented(int64_t d_in, int32_t n_parts, const int64_t* part_d_out,
                                                    int32_t max_rank, int32_t capacity);
marlaas_status_t marlaas_adapter_pool_create_segmented(marlaas_pool_t** out, int device, int64_t d_in, int32_t n_parts,
                                                       const int64_t* part_d_out /* HOST */, int32_t max_rank,
                                                       int32_t capacity, void* storage, size_t storage_bytes,
                                                       void* cuda_stream);
/* Number of projections the pool holds (1 for a pool made by marlaas_adapter_pool_create). */
int32_t marlaas_adapter_pool_parts(const marlaas_pool_t* pool);

/* Commit adapter version `version` of tenant `tenant_id` into the pool ("Commit updated parameters to M",
 * Algorithm 1; Asynchronous Execution, training step).  A: bf16 [d_in][rank], B: bf16 [rank][d_out],
 * both row-major device memory, copied and re-laid-out in stream order (the caller may reuse them once the
 * stream has passed the call).  The layer uses s = alpha / rank formed in fp32.  A tenant that is already
 * registered keeps its slot and is overwritten in stream order; a new tenant takes the lowest free slot.
 * rank = 0 (A, B may be NULL) makes the slot behave as "no adapter".  *slot_out (HOST) receives the slot. */
marlaas_status_t marlaas_adapter_pool_register(marlaas_pool_t* pool, uint64_t tenant_id, uint64_t version,
                                               int32_t rank, float alpha, const void* A, const void* B,
                                               int32_t* slot_out, void* cuda_stream);
/* Free the tenant's slot (its rank becomes 0 in stream order). */
marlaas_status_t marlaas_adapter_pool_unregister(marlaas_pool_t* pool, uint64_t tenant_id, void* cuda_stream);
/* Host-side lookup: slot / rank / scale / version of a tenant (any out pointer may be NULL). */
marlaas_status_t marlaas_adapter_pool_lookup(const marlaas_pool_t* pool, uint64_t tenant_id, int32_t* slot_out,
                                             int32_t* rank_out, float* scale_out, uint64_t* version_out);
/* Copy a slot's adapter back out in the caller's layout (A_out bf16 [d_in][rank], B_out bf16 [rank][d_out],
 * device memory; either may be NULL).  Used to check the store's re-layout bit for bit. */
marlaas_status_t marlaas_adapter_pool_export(marlaas_pool_t* pool, int32_t slot, void* A_out, void* B_out,
                                             void* cuda_stream);
/* Policy update and commit of the updated parameters for n tenants in one launch (Algorithm 1: "PolicyUpdate",
 * then the commit of the new adapter version; Methods, Multi-Task Manager: per-task optimizer state and version
 * counter).  The paper names no optimizer; this is AdamW with decoupled weight decay, in fp32:
 *     g = grad_scale * grad;  m = beta1 m + (1 - beta1) g;  v = beta2 v + (1 - beta2) g^2
 *     theta = theta - lr * ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay * theta )
 * applied to the fp32 master copies A [d_in][rank] and B [rank][d_out] of every listed tenant (moments m*, v* of the
 * same shapes, all updated in place), after which the bf16 rounding (round to nearest even) of the new masters
 * replaces the tenant's rows of the pooled store, as marlaas_adapter_pool_register would write them, and the
 * tenant's version becomes new_versions[i] (or its old version + 1 when new_versions is NULL).
 * tenant_ids / new_versions and the eight pointer tables are HOST arrays of n entries; the pointers in the tables are
 * device memory (4-byte aligned, caller-owned, gradients as marlaas_lora_backward wrote them: true rank, dense).
 * Stream-ordered like register.  Errors, before anything is launched: unknown tenant (MARLAAS_ERR_UNKNOWN_TENANT),
 * a tenant of rank 0 or listed twice, a NULL pointer, step < 1 (MARLAAS_ERR_INVALID_ARG). */
typedef struct marlaas_adamw {
    float lr, beta1, beta2, eps, weight_decay, grad_scale;
    int64_t step; /* >= 1: the step being taken */
} marlaas_adamw_t;
marlaas_status_t marlaas_adapter_pool_adamw_commit(marlaas_pool_t* pool, int32_t n, const uint64_t* tenant_ids,
                                                   const uint64_t* new_versions, const float* const* dA,
                                                   const float* const* dB, float* const* A, float* const* B,
                                                   float* const* m_A, float* const* v_A, float* const* m_B,
                                                   float* const* v_B, const marlaas_adamw_t* hp, void* cuda_stream);
/* Row stride (in floats) of the h_save / h_saved arrays: max_rank rounded up to a multiple of 16. */
int32_t marlaas_adapter_pool_rank_stride(const marlaas_pool_t* pool);

/* ---- the layer ---- */

/* Bytes of workspace forward/backward need for a batch of T tokens on this pool (device memory, 256-byte
 * aligned, contents need not be preserved between calls; two calls in flight need two workspaces).  The size does not
 * grow monotonically with T: the decode-shaped kernels chosen for small batches over large weights may use more exchange
 * scratch than those chosen for larger batches, so a workspace shared by calls of several batch sizes takes the largest
 * of their sizes (a call given less than its own full size still runs, see marlaas_lora_forward_workspace_min_bytes). */
size_t marlaas_lora_workspace_bytes(const marlaas_pool_t* pool, int64_t T);
/* The part of that workspace a forward call uses (its leading bytes): enough for marlaas_lora_forward alone. */
size_t marlaas_lora_forward_workspace_bytes(const marlaas_pool_t* pool, int64_t T);
/* The least a forward call accepts (also leading bytes).  The difference to the size above is scratch through which the
 * decode-shaped kernels for large weights pass partial sums between CTA pairs (up to about 20 MB); a call given less than
 * the full size runs the kernels that need no such scratch (slower on those shapes; every result still within the
 * layer's tolerance of the definition). */
size_t marlaas_lora_forward_workspace_min_bytes(const marlaas_pool_t* pool, int64_t T);

/* Forward: y[T][d_out] = x[T][d_in] W + s_t (x A_t) B_t with t from the segment table.
 * x (ldx >= d_in), W (ldw >= d_out), y (ldy >= d_out): bf16 row-major.  h_save: optional fp32
 * [T][rank_stride] that receives h_i = x_i A_t (zero beyond r_t) for reuse by backward; NULL = not kept.
 * T = 0 is a no-op. */
marlaas_status_t marlaas_lora_forward(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx,
                                      const void* W, int64_t ldw, void* y, int64_t ldy,
                                      const marlaas_segments_t* seg, float* h_save, void* workspace,
                                      size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/* Several forward calls that do not depend on one another, as one call: the projections of a decoder layer that read
 * the same activations (q, k, v; gate, up) during rollout, when every adapted projection of the shared base model serves
 * all tenants' decode tokens at once (paper: Methods, "Multi-LoRA Rollout with Single-Task Training"; Introduction:
 * rollouts dominate the run time).  Each entry holds the arguments of one marlaas_lora_forward.  The caller states that
 * no call's output is another's input and that pools, outputs, h_save arrays and workspaces are pairwise distinct; the
 * library may then run the calls side by side (on streams it owns, forked from cuda_stream and joined to it before the
 * call returns; events only, so legal inside a stream capture), which lets one projection's epilogue overlap the next
 * one's pass over its weight.  Everything the call writes is ordered on cuda_stream as if issued there.  All entries are
 * validated before anything is launched.  MARLAAS_FLAG_VALIDATE_SYNC and MARLAAS_FLAG_REUSE_PLAN are refused. */
typedef struct {
    marlaas_pool_t* pool;
    int64_t T;
    const void* x; int64_t ldx;
    const void* W; int64_t ldw;
    void* y; int64_t ldy;
    const marlaas_segments_t* seg;
    float* h_save;
    void* workspace; size_t workspace_bytes;
} marlaas_forward_call_t;
marlaas_status_t marlaas_lora_forward_multi(int32_t n, const marlaas_forward_call_t* calls, uint32_t flags, void* cuda_stream);

/* The same forward pass for callers that cannot allocate device memory (no counterpart in the paper: an
 * addition for deployments, not part of the method).  Some hosts of this layer may not call cudaMalloc at all:
 * a serving loop whose memory pool was sized and frozen at start-up, a plug-in that is handed nothing but its
 * input and output buffers, a latency-critical path that cannot afford the device-wide synchronisation an
 * allocation implies or its failure under a full memory budget.  For them the per-call scratch comes from an
 * array built into the library (marlaas_lora_static_workspace_limit() bytes, 8 MiB, resident on every GPU that
 * loads the library until the process exits) instead of a caller workspace; x, W, y, the pool storage and h_save
 * are still the caller's.  The call itself allocates and frees nothing on the device.
 *  - Batches whose forward scratch (marlaas_lora_forward_workspace_min_bytes) exceeds the limit are rejected with
 *    MARLAAS_ERR_WORKSPACE_TOO_SMALL before anything is launched: 256 tokens on a pool of 32 slots of rank
 *    up to 64 fit.
 *  - The first call on each device looks up the array's device address.  That lookup is also the moment the CUDA
 *    runtime loads this part of the library onto the device and the device's copy of the array comes into being
 *    (8 MiB of device memory, taken once, which can fail if the device is full): make that first call at start-up,
 *    while memory may still be taken, and before starting any stream capture on that device.  Later calls on the
 *    device leave its free memory unchanged.
 *  - All calls on a device share the one array and it keeps the previous call's contents (nothing in it has to
 *    start at zero: each call writes what it later reads).  Two calls whose kernels overlap on the GPU -- different
 *    streams, or different pools on different streams -- race on it; keep such calls on one stream. */
size_t marlaas_lora_static_workspace_limit(void);
marlaas_status_t marlaas_lora_forward_static_ws(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx,
                                                const void* W, int64_t ldw, void* y, int64_t ldy,
                                                const marlaas_segments_t* seg, float* h_save, uint32_t flags,
                                                void* cuda_stream);

/* Backward for the policy-training stage: dx[T][d_in] bf16 (NULL = skip) and per-slot fp32 adapter gradients.
 * dA_slots / dB_slots: HOST arrays of `capacity` device pointers (either table, or any entry, may be NULL =
 * skip); dA_t is [d_in][r_t], dB_t is [r_t][d_out], row-major, at the slot's true rank.  Without
 * MARLAAS_FLAG_ACCUMULATE every non-NULL slot is overwritten (tenants with no token in the batch get exact
 * zeros); with it the batch's contribution is added.  The sums over a tenant's tokens run over all of its
 * segments.  h_saved: what forward wrote to h_save for the same batch and adapters, or NULL = recompute.
 * Part of the work (the adapter-gradient kernels, when h_saved is given) may be issued on a stream that the pool
 * owns, forked from cuda_stream after the call's first kernels and joined to it before the call returns (events;
 * legal inside a stream capture): everything the call writes is ordered on cuda_stream as if issued there.  Inside a
 * stream capture, pools of more than 64 slots copy dA_slots / dB_slots with a memcpy node that keeps the HOST pointers:
 * the caller's tables must then stay alive and unchanged for every replay.  Calls on one pool are not to be issued from
 * several host threads at once. */
marlaas_status_t marlaas_lora_backward(marlaas_pool_t* pool, int64_t T, const void* x, int64_t ldx,
                                       const void* W, int64_t ldw, const void* dy, int64_t lddy,
                                       void* dx, int64_t lddx, float* const* dA_slots, float* const* dB_slots,
                                       const marlaas_segments_t* seg, const float* h_saved, void* workspace,
                                       size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/* The indexing contract, bit-exact: tok_slot[T] (slot of the segment containing each token),
 * slot_count[capacity+1] (tokens per slot; the last entry counts slot -1), slot_offset[capacity+2]
 * (exclusive prefix sum in the order 0..capacity-1, then -1; last entry = T) and perm[T] (token indices
 * stably sorted by that key).  All four are device int32 arrays; any may be NULL. */
marlaas_status_t marlaas_lora_build_index(marlaas_pool_t* pool, int64_t T, const marlaas_segments_t* seg,
                                          int32_t* tok_slot, int32_t* slot_count, int32_t* slot_offset,
                                          int32_t* perm, void* workspace, size_t workspace_bytes,
                                          uint32_t flags, void* cuda_stream);

/* Synchronise `cuda_stream`, read and clear the pool's device status word: MARLAAS_OK, or the first
 * device-side finding since the last check (BAD_SEGMENT_TABLE, DEVICE_BAD_INDEX, DEVICE_TIMEOUT). */
marlaas_status_t marlaas_check_status(marlaas_pool_t* pool, void* cuda_stream);

/* Diagnostic (no counterpart in the paper): every wait inside the tensor-core kernels is bounded, and a wait that runs
 * out makes its kernel drain and return with MARLAAS_ERR_DEVICE_TIMEOUT recorded in the pool's status word.  This call
 * exercises exactly that path without starving a real kernel: one small CTA waits, with the kernels' own wait routine,
 * on a barrier that nobody arrives on, gives up after limit_ns (at most 100 ms) and returns normally.  The next
 * marlaas_check_status on the pool then returns MARLAAS_ERR_DEVICE_TIMEOUT (and clears it); the pool stays usable. */
marlaas_status_t marlaas_debug_wait_runs_out(marlaas_pool_t* pool, uint64_t limit_ns, void* cuda_stream);

/* Message for the last non-OK status returned on the calling thread ("" if none). */
const char* marlaas_last_error(void);

/* Measurement aid (no counterpart in the paper): between _begin and _end the library brackets every launch of
 * the layer's dominant kernel (the base GEMM with the fused low-rank term, forward and dx) with CUDA events on
 * the launching stream.  _end synchronises those events and returns the summed device time in milliseconds
 * and the number of bracketed launches (either out pointer may be NULL). */
marlaas_status_t marlaas_kernel_timing_begin(marlaas_pool_t* pool);
marlaas_status_t marlaas_kernel_timing_end(marlaas_pool_t* pool, float* gemm_ms, int32_t* gemm_launches);

/* Number of kernels the library has launched in this process (all pools, all threads). */
uint64_t marlaas_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MARLAAS_H_ */
