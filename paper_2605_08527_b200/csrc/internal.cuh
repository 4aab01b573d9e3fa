// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <string>
#include <vector>

#include "marlaas.h"

namespace marlaas {

typedef __nv_bfloat16 bf16;

// ---- error plumbing -------------------------------------------------------------------------------
marlaas_status_t fail(marlaas_status_t code, const char* fmt, ...);
void count_launch(int n = 1);

#define MARLAAS_CUDA_TRY(expr)                                                                       \
    do {                                                                                             \
        cudaError_t e__ = (expr);                                                                    \
        if (e__ != cudaSuccess)                                                                      \
            return ::marlaas::fail(MARLAAS_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

#define MARLAAS_LAUNCH_CHECK(name)                                                                   \
    do {                                                                                             \
        cudaError_t e__ = cudaGetLastError();                                                        \
        if (e__ != cudaSuccess)                                                                      \
            return ::marlaas::fail(MARLAAS_ERR_CUDA, "launch of %s failed: %s", name, cudaGetErrorString(e__)); \
        ::marlaas::count_launch();                                                                   \
    } while (0)

// Brackets one launch of the dominant kernel with events while the pool's timing mode is on.
struct TimedLaunch {
    marlaas_pool* pool;
    cudaStream_t st;
    bool on;
    TimedLaunch(marlaas_pool* p, cudaStream_t s);
    ~TimedLaunch();
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

// device status word values (written with atomicCAS from 0, so the first finding wins)
enum { DEV_OK = 0, DEV_BAD_TABLE = 1, DEV_BAD_INDEX = 2, DEV_TIMEOUT = 3 };

struct SlotMeta {
    bool used = false;
    uint64_t tenant_id = 0;
    uint64_t version = 0;
    int32_t rank = 0;
    float alpha = 0.f;
    float scale = 0.f;
};

}  // namespace marlaas

// The pool: host bookkeeping plus pointers into the caller-provided device storage.
//   At : bf16 [P][capacity*RP][K]   row (slot*RP + j) of block p = column j of A_t,p   (zero rows for j >= r_t)
//   Bs : bf16 [capacity*RP][N]      row (slot*RP + j) = row j of [B_t,1 | ... | B_t,P]  (zero rows for j >= r_t)
// Both serve as gather sources for the shrink (dot products along a contiguous row) and as tensor-core
// operands for the extra k-steps of the fused expand (rows = rank index).  P = 1 for an ordinary pool; a pool over
// P projections that read the same activations keeps one A block per projection and the B matrices side by side,
// so that output range p of the layer pairs with A block p and columns [part_begin[p], part_begin[p+1]) of Bs.
constexpr int MARLAAS_MAX_PARTS = 4;
struct marlaas_pool {
    int device = 0;
    int64_t K = 0, N = 0;
    int32_t max_rank = 0, RP = 0, cap = 0;
    int32_t P = 1;
    int64_t part_begin[MARLAAS_MAX_PARTS + 1] = {0, 0, 0, 0, 0};
    int64_t ldB = 0;                // elements between rows of Bs (= N of the whole pool, also in a part's view)
    char* storage = nullptr;
    size_t storage_bytes = 0;
    int32_t* d_status = nullptr;
    int32_t* d_sync = nullptr;      // counters and flags of the decode-shaped forward (zero between calls)
    int32_t* d_rank = nullptr;
    float* d_scale = nullptr;
    marlaas::bf16* d_At = nullptr;
    marlaas::bf16* d_Bs = nullptr;
    std::vector<marlaas::SlotMeta> slots;
    int sm_count = 0;
    // kernel timing (marlaas_kernel_timing_begin/_end): event pairs around the dominant kernel
    bool timing = false;
    std::vector<cudaEvent_t> timing_events;
    size_t timing_used = 0;
    // backward: the adapter-gradient kernels run on a side stream beside the dx GEMM (created on first use)
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
};

namespace marlaas {

struct StorageLayout {
    size_t off_status, off_sync, off_rank, off_scale, off_At, off_Bs, total;
};
StorageLayout storage_layout(int64_t K, int64_t N, int32_t RP, int32_t cap, int32_t parts = 1);

// Part p of a pool over several projections, as a pool of its own (no slot table, no streams: for the kernel launchers
// only): its A block, its columns of Bs (row pitch ldB unchanged), the shared rank / scale / status arrays.
void part_view(const marlaas_pool* pool, int p, marlaas_pool* view);

// Per-call workspace (device), carved from the caller's buffer.
struct Workspace {
    int32_t* tok_slot;     // [T]
    int32_t* perm;         // [T]
    int32_t* slot_count;   // [cap+1]
    int32_t* slot_offset;  // [cap+2]
    float* h;              // [T][RP]
    float* g;              // [T][RP]
    float** dA_ptrs;       // [cap]
    float** dB_ptrs;       // [cap]
    // tensor-core path: per 256-token plan tile, the list of 16-deep rank units of the tenants present in it
    int32_t* tok_uoff;     // [T]  first unit of the token's tenant within its tile's list, -1 = none
    int32_t* tile_nunits;  // [ceil(T/256)]
    int32_t* tile_units;   // [ceil(T/256)][umax]  first store row (slot*RP + 16j) of each unit
    bf16* hd;              // [T][umax*16]  bf16(s_t h_i) (forward) or bf16(s_t g_i) (backward) in the tenant's unit
                           //               columns, zeros in the other units of the tile
    int32_t umax;
    float* xbuf;           // decode path with a split contraction: partial sums passed between the slices of a tile
    size_t fwd_min;        // bytes a forward call cannot do without (the fields above but xbuf: without it the decode
                           // kernels that exchange partial sums are not used)
    size_t fwd_total;      // bytes a forward call uses (the fields above); the rest serves backward only
    // tensor-core gradient reductions: 64-token blocks, one masked copy of the block's r-vectors per tenant present
    int32_t* blk_np;       // [nblk]        tenants present in the block
    int32_t* blk_base;     // [nblk+1]      exclusive scan of blk_np (= first copy of the block)
    int32_t* blk_rank;     // [nblk][cap]   rank of the tenant among the block's present tenants, -1 = absent
    int32_t* ten_nblk;     // [cap]         copies of the tenant
    int32_t* ten_blks;     // [cap][nblk]   the tenant's blocks, ascending
    int32_t* ten_pos;      // [cap][nblk]   the matching copy positions
    int32_t* gflag;        // [4]           [0] = 1 when the copies do not fit (CUDA-core reduction runs instead)
    bf16* hm;              // [max_copies*64][HW]  hi | lo split r-vectors
    bf16* hm2;             // a second set of copies, so that the dB and dA reductions need not share one
    int32_t max_copies, HW;
    size_t total;
    bool early_shrink = false;   // this call: the decode shrink is launched behind the stream's previous kernel without
                                 // waiting for it (MARLAAS_FLAG_OVERLAP_PREVIOUS)
};
Workspace carve_workspace(const marlaas_pool* pool, int64_t T, void* base);

// ---- kernels launched by api.cu ---------------------------------------------------------------------
// plan.cu
marlaas_status_t launch_tok_slot(const marlaas_pool* pool, int64_t T, int32_t S, const int32_t* seg_offsets,
                                 const int32_t* seg_slot, int32_t* tok_slot, cudaStream_t st);
// run_flag (optional, device): the kernel returns at once unless run_flag[0] != 0
marlaas_status_t launch_slot_sort(const marlaas_pool* pool, int64_t T, const int32_t* tok_slot,
                                  int32_t* slot_count, int32_t* slot_offset, int32_t* perm, cudaStream_t st,
                                  const int32_t* run_flag = nullptr);

// One CTA per 256-token plan tile: per-token slot (from the table, or already in tok_slot when S < 0), the tile's unit
// list and each token's unit offset.
marlaas_status_t launch_plan_tiles(const marlaas_pool* pool, int64_t T, int32_t S, const int32_t* seg_offsets,
                                   const int32_t* seg_slot, const Workspace& ws, cudaStream_t st);

// gemm_sm100.cu
struct GemmOperands {
    int64_t M, Nout, Kc;
    const bf16* A; int64_t lda;        // [M][Kc]
    const bf16* B; int64_t ldb;        // b_mn: [Kc][Nout]; else [Nout][Kc]
    bool b_mn;
    bf16* C; int64_t ldc;              // [M][Nout]
    const bf16* XA; int64_t xa_cols;   // [M][xa_cols] (pitch xa_cols)
    const bf16* XB; int64_t xb_rows;   // [xb_rows][Nout], rows xb_ld elements apart
    int64_t xb_ld;
    const int32_t* tile_nunits;        // nullptr = no low-rank term
    const int32_t* tile_units;
    int32_t umax;
    // pools over several projections (the 2-CTA kernel only): XA is [parts][M][xa_cols]; see Gemm2Args
    int32_t parts = 1;
    bool all_parts = false;
    int64_t part_end[4] = {0, 0, 0, 0};
};
marlaas_status_t launch_gemm_sm100(const marlaas_pool* pool, const GemmOperands& o, cudaStream_t st);
// gemm2_sm100.cu: the same product with 2-CTA clusters (256 x 256 tiles), for batches of at least 1024 rows
bool gemm2_sm100_eligible(const marlaas_pool* pool, int64_t M);
marlaas_status_t launch_gemm2_sm100(const marlaas_pool* pool, const GemmOperands& o, cudaStream_t st);

// decode_sm100.cu: the whole forward for batches of at most 1024 tokens (two overlapping kernels).
// S < 0: ws.tok_slot already holds the per-token slots.
bool decode_sm100_eligible(const marlaas_pool* pool, int64_t T);
// the shrink kernel of that path alone (writes tok_slot, h and hd)
marlaas_status_t launch_decode_shrink(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, int32_t S,
                                      const int32_t* seg_offsets, const int32_t* seg_slot, const Workspace& ws, float* h_out,
                                      cudaStream_t st);
size_t decode_shrink_smem_bytes(int64_t T, int32_t S);
// decode_wide_sm100.cu: the same forward for large weights (W columns on the MMA's M side; see the file)
bool decode_wide_sm100_eligible(const marlaas_pool* pool, int64_t T);
size_t decode_wide_sm100_xbuf_bytes(const marlaas_pool* pool, int64_t T);    // its exchange scratch (0 if unused)
bool decode_wide_sm100_splits(const marlaas_pool* pool, int64_t T);        // true if that kernel would cut the contraction in slices
marlaas_status_t launch_decode_wide_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                          int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                          const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st);
// the same forward when there are more tiles than CTA pairs: the tiles' steps spread evenly over all pairs
bool decode_stream_sm100_eligible(const marlaas_pool* pool, int64_t T);
marlaas_status_t launch_decode_stream_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                            int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                            const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st);
constexpr size_t DECODE_SYNC_BYTES = 16384;

marlaas_status_t launch_decode_sm100(const marlaas_pool* pool, int64_t T, const bf16* x, int64_t ldx, const bf16* W,
                                     int64_t ldw, bf16* y, int64_t ldy, int32_t S, const int32_t* seg_offsets,
                                     const int32_t* seg_slot, const Workspace& ws, float* h_out, cudaStream_t st);

// shrink_sm100.cu: the same outputs as launch_shrink_hd, computed on the tensor cores tile by tile
// store: the rows of the pooled store to contract with ([cap*RP] rows of D elements, sld elements apart)
marlaas_status_t launch_shrink_sm100(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                                     const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st);

// shrink_split_sm100.cu: the same outputs with one tile per cluster and the contraction split over the cluster's
// CTAs; applies when all tiles fit one wave
bool shrink_split_sm100_eligible(const marlaas_pool* pool, int64_t T, int64_t D);
marlaas_status_t launch_shrink_split_sm100(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                                           const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st,
                                           bool out_is_zero = false, int P = 1);
// whether ONE launch can serve all P blocks of adapter rows of a pool over several projections (planes of out and hd)
bool shrink_split_sm100_parts_eligible(const marlaas_pool* pool, int64_t T, int64_t D, int P);

// cuda_core_kernels.cu
// h/g (fp32, [T][RP]) as launch_rowdot, plus the bf16 block-diagonal operand rows hd for the tensor-core path
marlaas_status_t launch_shrink_hd(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                                  const bf16* store, int64_t sld, const Workspace& ws, float* out, cudaStream_t st);
// out[i][j] = sum_d src[i][d] * store[(slot_i*RP + j)][d] for j < RP (zeros for inactive tokens / padded rows)
marlaas_status_t launch_rowdot(const marlaas_pool* pool, int64_t T, const bf16* src, int64_t ld, int64_t D,
                               const bf16* store, int64_t sld, const int32_t* tok_slot, float* out, cudaStream_t st);
// C[T][Nout] = bf16( A[T][Kc] * op(W) + s_t * sum_j hg[i][j] * store[(slot*RP+j)][c] );
// trans_w = false: op(W) = W[Kc][Nout] (ldw);  true: op(W) = W^T with W stored [Nout][Kc] (ldw)
marlaas_status_t launch_gemm_cuda_core(const marlaas_pool* pool, int64_t T, int64_t Nout, int64_t Kc,
                                       const bf16* A, int64_t lda, const bf16* W, int64_t ldw, bool trans_w,
                                       bf16* C, int64_t ldc, const float* hg, const bf16* store, int64_t sld,
                                       const int32_t* tok_slot, cudaStream_t st, int nparts = 1, int64_t hg_plane = 0);
// out_t[j][c] (transpose_out = false, ld = C) or out_t[c][j] (true, ld = r_t) (+)= s_t * sum_{i in t} hg[i][j] * src[i][c]
marlaas_status_t launch_grad_reduce(const marlaas_pool* pool, int64_t C, const bf16* src, int64_t ld,
                                    const float* hg, const int32_t* perm, const int32_t* slot_offset,
                                    float* const* out_ptrs, bool transpose_out, bool accumulate, cudaStream_t st,
                                    const int32_t* run_flag = nullptr);

// grad_sm100.cu: the same reductions on the tensor cores
bool grad_sm100_eligible(const marlaas_pool* pool, int64_t T);
marlaas_status_t launch_grad_plan(const marlaas_pool* pool, int64_t T, const Workspace& ws, cudaStream_t st);
// phases: build the masked hi/lo copies of the r-vectors into hm, reduce from hm, or both
// GRAD_PHASE_EARLY: the reduction reads nothing the kernel before it in the stream writes and may start while that one ends
enum { GRAD_PHASE_COPIES = 1, GRAD_PHASE_REDUCE = 2, GRAD_PHASE_EARLY = 4 };
marlaas_status_t launch_grad_sm100(const marlaas_pool* pool, int64_t T, int64_t C, const bf16* src, int64_t ld,
                                   const float* hg, float* const* out_ptrs, float* const* host_ptrs, bool transpose_out,
                                   bool accumulate, const Workspace& ws, cudaStream_t st, bf16* hm, int phases = GRAD_PHASE_COPIES | GRAD_PHASE_REDUCE);
// host_ptrs: the same table in host memory; pools of at most 64 slots pass it with the launch and never read out_ptrs

}  // namespace marlaas
