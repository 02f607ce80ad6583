// Host side of the C ABI declared in cadd.h: argument validation, workspace carve-up, kernel launches.
// No allocation, no synchronisation, no state kept between calls.
#include <cuda_runtime.h>
#include <stdint.h>

#include "cadd.h"
#include "common.cuh"
#include "expand_emit.cuh"
#include "softmax_topk.cuh"
#include "verify.cuh"
#include "head_argmax.cuh"
#include "fit_cost.cuh"
#include "head_softmax_topk.cuh"
#include "sample_verify.cuh"

namespace cadd {

constexpr int kPreciseMin = 8;    // KP = max(K, 8): candidates per position singled out by the softmax/top-K kernel, exponentials in fp64

static inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

struct BuildPlan {
    int KP;          // candidates kept per (row, segment)
    int S;           // segments per row
    size_t partial_bytes;
    ExpandLayout lay;
};

static int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 148;
    return n;
}

static int check_build_shape(const cadd_build_args* a) {
    if (!a) return CADD_ERR_NULL;
    if (a->struct_size != sizeof(cadd_build_args)) return CADD_ERR_STRUCT_SIZE;
    if (a->batch < 1 || a->L < 1 || a->L > 64 || a->K < 1 || a->K > 64 || a->V < 1 || a->V >= ((int64_t)1 << 31) ||
        a->B_max < 0 || a->B_max > 2048 || a->R < a->B_max + 1)
        return CADD_ERR_SHAPE;
    if ((int64_t)a->batch * a->L * 8 >= ((int64_t)1 << 31) || (int64_t)a->batch * a->R >= ((int64_t)1 << 31)) return CADD_ERR_SHAPE;
    if (a->logits_dtype != CADD_DTYPE_BF16 && a->logits_dtype != CADD_DTYPE_FP32) return CADD_ERR_DTYPE;
    if (a->cost_kind != CADD_COST_QUADRATIC && a->cost_kind != CADD_COST_TABLE && a->cost_kind != CADD_COST_TABLE_INTERP) return CADD_ERR_DTYPE;
    if ((a->flags & CADD_FLAG_ONLY_TOPK) && (a->flags & CADD_FLAG_ONLY_EXPAND)) return CADD_ERR_DTYPE;
    return CADD_OK;
}

// Segments per row.  Whole rows are cheapest per element (one threshold warm-up per CTA), but the
// grid must fill the resident-CTA slots of the machine evenly: take the smallest cut whose last wave
// is at least 85 % full (else the fullest), never making a segment shorter than 4 iterations.
constexpr int kMaxSegments = 8;
// Rows are cut only while the grid stays within kSlotsCap CTAs (more than any device has resident slots for), so that the
// workspace -- sized for the largest cut whatever the device -- stays small for large batches.
constexpr int64_t kSlotsCap = 1024;
static int max_segments(int64_t rows) {
    const int64_t s = (kSlotsCap + rows - 1) / rows;
    return (int)(s < 1 ? 1 : (s > kMaxSegments ? kMaxSegments : s));
}
static BuildPlan plan_build(const cadd_build_args* a, int slots) {
    BuildPlan pl;
    pl.KP = a->K > kPreciseMin ? a->K : kPreciseMin;
    const int epc = a->logits_dtype == CADD_DTYPE_BF16 ? 8 : 4;
    const int64_t rows = (int64_t)a->batch * a->L;
    const int64_t chunks = a->V / epc;
    int64_t cap = chunks / (4 * kTkTileChunks);
    if (cap > max_segments(rows)) cap = max_segments(rows);
    if (cap > 512 / seg_key_cap(pl.KP)) cap = 512 / seg_key_cap(pl.KP);   // the expansion kernel holds every key of a row's records per warp
    if (cap < 1) cap = 1;
    int best = 1;
    double best_eff = 0.0;
    for (int S = 1; S <= (int)cap; ++S) {
        const int64_t items = rows * S;
        const int64_t waves = (items + slots - 1) / slots;
        const double eff = (double)items / (double)(waves * slots);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = S; }
        if (eff >= 0.85) { best = S; break; }
    }
    pl.S = best;
    pl.partial_bytes = (size_t)rows * pl.S * seg_record_stride(pl.KP);
    pl.lay = expand_layout(a->L, a->K, seg_key_cap(pl.KP), pl.S, a->B_max, 0);
    return pl;
}

// Resident CTAs of the softmax/top-K kernel on the current device (occupancy x SM count).
static int topk_slots(int dtype) {
    int per_sm = 0;
    if (cudaFuncSetAttribute(dtype == CADD_DTYPE_BF16 ? (const void*)softmax_topk_partial_kernel<CADD_DTYPE_BF16>
                                                       : (const void*)softmax_topk_partial_kernel<CADD_DTYPE_FP32>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)topk_smem_bytes()) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    cudaError_t e = dtype == CADD_DTYPE_BF16
        ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, softmax_topk_partial_kernel<CADD_DTYPE_BF16>, kTkThreads, topk_smem_bytes())
        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, softmax_topk_partial_kernel<CADD_DTYPE_FP32>, kTkThreads, topk_smem_bytes());
    if (e != cudaSuccess || per_sm < 1) { cudaGetLastError(); per_sm = 4; }
    return per_sm * sm_count();
}

static size_t build_workspace_bytes(const BuildPlan& pl) { return (pl.partial_bytes + 255) & ~(size_t)255; }

}  // namespace cadd

using namespace cadd;

// Problems that stream at least this many bytes of logits are launched with programmatic stream serialization.
constexpr int64_t kOverlapMinBytes = 16ll << 20;
// LIVE verification shares a CTA between eight rows up to this row capacity (node cap 512).
constexpr int kLiveSharedRowsMaxR = 513;

// Launch with programmatic stream serialization: the grid may be set up and its CTAs dispatched while the previous
// kernel of the stream drains; every kernel launched this way starts with griddepcontrol.wait, which returns once the
// previous kernel has completed and its writes are visible (and at once when there is no such dependency).
// Costs a few microseconds more on the host than a plain launch, so launch-bound (small) problems ask for `overlap` = false.
template <typename... KArgs, typename... Args>
static cudaError_t launch_dependent(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    if (!overlap) {
        kernel<<<grid, block, smem, st>>>(args...);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// Small problems are launch-bound: below these sizes tree construction is ONE kernel (the expansion kernel reads the
// short rows itself, one warp per row) and verification is ONE kernel (one CTA per request: arg-max of its rows, then
// the walk).  The single-kernel measurement flags and the test hook always take the regular path.
constexpr int64_t kSmallMaxV = 8192;                 // elements per row (verification)
constexpr int64_t kSmallBuildMaxV = 2048;            // elements per row (construction: eight staged rows fit in shared memory)
constexpr int64_t kSmallBuildBytes = 2ll << 20;      // draft logits of the whole call
constexpr int64_t kSmallVerifyBytes = 4ll << 20;     // target logits the call reads at most
static bool build_is_small(const cadd_build_args* a) {
    if (a->flags & (CADD_FLAG_ONLY_TOPK | CADD_FLAG_ONLY_EXPAND | CADD_FLAG_TEST_DROP_TILE | CADD_FLAG_REGULAR_PATH)) return false;
    const int64_t es = a->logits_dtype == CADD_DTYPE_BF16 ? 2 : 4;
    return a->V <= kSmallBuildMaxV && (int64_t)a->batch * a->L * a->V * es <= kSmallBuildBytes;
}
static bool verify_is_small(const cadd_verify_args* a) {
    if (a->flags & (CADD_VERIFY_ONLY_ARGMAX | CADD_VERIFY_ONLY_WALK | CADD_FLAG_TEST_DROP_TILE | CADD_VERIFY_REGULAR_PATH)) return false;
    const int64_t es = a->logits_dtype == CADD_DTYPE_BF16 ? 2 : 4;
    return a->V <= kSmallMaxV && (int64_t)a->batch * a->R * a->V * es <= kSmallVerifyBytes;
}

// Launches the expansion + emission kernel on the per-row partial records at `partials` (S records per row).
static int launch_expand(const cadd_build_args* a, int KP, int S, int rec_fmt, const unsigned char* partials, cudaStream_t st, bool overlap) {
    const ExpandLayout lay = expand_layout(a->L, a->K, rec_key_cap(rec_fmt, KP), S, a->B_max, rec_fmt == kRecDirect ? direct_stage_bytes(a->V, a->logits_dtype) : 0);
    ExpandParams ep;
    ep.batch = a->batch; ep.L = a->L; ep.K = a->K; ep.KP = KP; ep.S = S; ep.B_max = a->B_max; ep.R = a->R;
    ep.rec_fmt = rec_fmt;
    ep.logits = a->draft_logits; ep.V = a->V; ep.stride_b = a->stride_b; ep.stride_l = a->stride_l; ep.logits_dtype = a->logits_dtype;
    ep.flags = a->flags; ep.partials = partials;
    ep.l_eff = a->l_eff; ep.bonus_token = a->bonus_token; ep.ctx_len = a->ctx_len;
    ep.cost_kind = a->cost_kind; ep.cost_coef = a->cost_coef; ep.cost_table = a->cost_table;
    ep.table_idx = a->table_idx; ep.t_draft = a->t_draft; ep.ctx_grid = a->ctx_grid; ep.n_tables = a->n_tables;
    ep.n_nodes = a->n_nodes; ep.token_ids = a->token_ids; ep.parent_idx = a->parent_idx; ep.depth = a->depth;
    ep.position_ids = a->position_ids; ep.node_logprob = a->node_logprob; ep.phi = a->phi; ep.theta = a->theta; ep.theta_curve = a->theta_curve;
    ep.mask_bits = a->mask_bits; ep.mask_dense = a->mask_dense; ep.topk_token = a->topk_token;
    ep.topk_logprob = a->topk_logprob; ep.status = a->status;
    void (*kernel)(ExpandParams) = rec_fmt == kRecDirect ? expand_emit_kernel<true> : expand_emit_kernel<false>;
    if (lay.total > 48 * 1024) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lay.total) != cudaSuccess) {
            cudaGetLastError();
            return CADD_ERR_LAUNCH;
        }
    }
    if (launch_dependent(overlap, kernel, dim3((unsigned)a->batch), dim3(kExpandThreads), lay.total, st, ep) != cudaSuccess) { cudaGetLastError(); return CADD_ERR_LAUNCH; }
    return CADD_OK;
}

extern "C" {

int cadd_version(void) { return CADD_ABI_VERSION; }

const char* cadd_status_string(int code) {
    switch (code) {
        case CADD_OK: return "ok";
        case CADD_ERR_NULL: return "a required pointer is NULL";
        case CADD_ERR_STRUCT_SIZE: return "struct_size does not match this library";
        case CADD_ERR_SHAPE: return "shape out of range";
        case CADD_ERR_DTYPE: return "unknown dtype, cost kind or rows mode";
        case CADD_ERR_ALIGN: return "pointer or stride misaligned";
        case CADD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CADD_ERR_LAUNCH: return "CUDA launch failed";
        case CADD_ERR_STATIC_SCRATCH: return "problem needs more scratch than the built-in static array holds";
        default: return "unknown code";
    }
}

int cadd_build_workspace_bytes(const cadd_build_args* a, size_t* out) {
    int rc = check_build_shape(a);
    if (rc != CADD_OK) return rc;
    if (!out) return CADD_ERR_NULL;
    // the SM count only steers how rows are cut; size for the largest cut so the answer is device independent
    BuildPlan pl = plan_build(a, 148 * 3);
    BuildPlan worst = pl;
    worst.S = kMaxSegments;
    worst.partial_bytes = (size_t)a->batch * a->L * max_segments((int64_t)a->batch * a->L) * seg_record_stride(pl.KP);
    *out = build_workspace_bytes(worst);
    return CADD_OK;
}

int cadd_build_tree(const cadd_build_args* a, void* cuda_stream) {
    int rc = check_build_shape(a);
    if (rc != CADD_OK) return rc;
    if (!a->draft_logits || !a->n_nodes || !a->token_ids || !a->parent_idx || !a->depth) return CADD_ERR_NULL;
    if (a->cost_kind == CADD_COST_QUADRATIC && !a->cost_coef) return CADD_ERR_NULL;
    if (a->cost_kind == CADD_COST_TABLE && (!a->cost_table || !a->table_idx || !a->t_draft || a->n_tables < 1)) return CADD_ERR_NULL;
    if (a->cost_kind == CADD_COST_TABLE_INTERP && (!a->cost_table || !a->ctx_grid || !a->t_draft || a->n_tables < 1)) return CADD_ERR_NULL;
    if ((a->flags & CADD_FLAG_EMIT_DENSE_MASK) && !a->mask_dense) return CADD_ERR_NULL;
    if ((a->flags & CADD_FLAG_EMIT_TOPK) && !a->topk_token && !a->topk_logprob) return CADD_ERR_NULL;
    const size_t es = a->logits_dtype == CADD_DTYPE_BF16 ? 2 : 4;
    if (!aligned(a->draft_logits, es)) return CADD_ERR_ALIGN;
    if (!aligned(a->cost_coef, 8) || !aligned(a->cost_table, 8) || !aligned(a->t_draft, 8) || !aligned(a->node_logprob, 8) ||
        !aligned(a->phi, 8) || !aligned(a->theta, 8) || !aligned(a->theta_curve, 8) || !aligned(a->topk_logprob, 8))
        return CADD_ERR_ALIGN;
    if (!aligned(a->n_nodes, 4) || !aligned(a->token_ids, 4) || !aligned(a->parent_idx, 4) || !aligned(a->depth, 4) ||
        !aligned(a->position_ids, 4) || !aligned(a->mask_bits, 4) || !aligned(a->topk_token, 4) || !aligned(a->status, 4) ||
        !aligned(a->l_eff, 4) || !aligned(a->bonus_token, 4) || !aligned(a->ctx_len, 4) || !aligned(a->table_idx, 4) ||
        !aligned(a->ctx_grid, 4))
        return CADD_ERR_ALIGN;
    if (a->stride_l < a->V || a->stride_b < 0) return CADD_ERR_SHAPE;

    const int slots = topk_slots(a->logits_dtype);
    if (slots < 1) return CADD_ERR_LAUNCH;
    const BuildPlan pl = plan_build(a, slots);
    if (!a->workspace || !aligned(a->workspace, 256) || a->workspace_bytes < build_workspace_bytes(pl)) return CADD_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (build_is_small(a)) return launch_expand(a, pl.KP, 1, kRecDirect, nullptr, st, false);

    TopkParams tp;
    tp.logits = a->draft_logits; tp.V = a->V; tp.stride_b = a->stride_b; tp.stride_l = a->stride_l;
    tp.L = a->L; tp.S = pl.S; tp.KP = pl.KP; tp.l_eff = a->l_eff; tp.partials = (unsigned char*)a->workspace;
    tp.fault_tile = (a->flags & CADD_FLAG_TEST_DROP_TILE) ? 1 : -1;
    const unsigned items = (unsigned)((int64_t)a->batch * a->L * pl.S);
    const bool overlap = (int64_t)a->batch * a->L * a->V * (int64_t)es >= kOverlapMinBytes;
    if (!(a->flags & CADD_FLAG_ONLY_EXPAND)) {
        const cudaError_t le = a->logits_dtype == CADD_DTYPE_BF16
            ? launch_dependent(overlap, softmax_topk_partial_kernel<CADD_DTYPE_BF16>, dim3(items), dim3(kTkThreads), topk_smem_bytes(), st, tp)
            : launch_dependent(overlap, softmax_topk_partial_kernel<CADD_DTYPE_FP32>, dim3(items), dim3(kTkThreads), topk_smem_bytes(), st, tp);
        if (le != cudaSuccess) { cudaGetLastError(); return CADD_ERR_LAUNCH; }
    }
    if (a->flags & CADD_FLAG_ONLY_TOPK) return CADD_OK;
    return launch_expand(a, pl.KP, pl.S, kRecSegRecord, (const unsigned char*)a->workspace, st, overlap);
}

static int check_verify_shape(const cadd_verify_args* a) {
    if (!a) return CADD_ERR_NULL;
    if (a->struct_size != sizeof(cadd_verify_args)) return CADD_ERR_STRUCT_SIZE;
    if (a->batch < 1 || a->L < 1 || a->L > 64 || a->R < 1 || a->V < 1 || a->V >= ((int64_t)1 << 31) ||
        (int64_t)a->batch * a->R >= ((int64_t)1 << 31))
        return CADD_ERR_SHAPE;
    if (a->logits_dtype != CADD_DTYPE_BF16 && a->logits_dtype != CADD_DTYPE_FP32) return CADD_ERR_DTYPE;
    if (a->rows_mode != CADD_ROWS_LIVE && a->rows_mode != CADD_ROWS_DENSE) return CADD_ERR_DTYPE;
    if ((a->flags & CADD_VERIFY_ONLY_ARGMAX) && (a->flags & CADD_VERIFY_ONLY_WALK)) return CADD_ERR_DTYPE;
    return CADD_OK;
}

int cadd_build_launches(const cadd_build_args* a) {
    int rc = check_build_shape(a);
    if (rc != CADD_OK) return rc;
    if (a->flags & (CADD_FLAG_ONLY_TOPK | CADD_FLAG_ONLY_EXPAND)) return 1;
    return build_is_small(a) ? 1 : 2;
}

int cadd_verify_workspace_bytes(const cadd_verify_args* a, size_t* out) {
    int rc = check_verify_shape(a);
    if (rc != CADD_OK) return rc;
    if (!out) return CADD_ERR_NULL;
    *out = 0;
    return CADD_OK;
}

int cadd_verify_launches(const cadd_verify_args* a) {
    int rc = check_verify_shape(a);
    if (rc != CADD_OK) return rc;
    if (a->flags & (CADD_VERIFY_ONLY_ARGMAX | CADD_VERIFY_ONLY_WALK)) return 1;
    return verify_is_small(a) ? 1 : 2;
}

int cadd_verify_tree(const cadd_verify_args* a, void* cuda_stream) {
    int rc = check_verify_shape(a);
    if (rc != CADD_OK) return rc;
    if (!a->target_logits || !a->n_nodes || !a->token_ids || !a->parent_idx || !a->node_argmax || !a->accepted_len ||
        !a->accepted_nodes || !a->next_bonus)
        return CADD_ERR_NULL;
    const size_t es = a->logits_dtype == CADD_DTYPE_BF16 ? 2 : 4;
    if (!aligned(a->target_logits, es)) return CADD_ERR_ALIGN;
    if (!aligned(a->n_nodes, 4) || !aligned(a->token_ids, 4) || !aligned(a->parent_idx, 4) || !aligned(a->node_argmax, 4) ||
        !aligned(a->accepted_len, 4) || !aligned(a->accepted_nodes, 4) || !aligned(a->next_bonus, 4) || !aligned(a->status, 4))
        return CADD_ERR_ALIGN;
    if (a->stride_row < a->V || a->stride_b < 0) return CADD_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    ArgmaxParams ap;
    ap.logits = a->target_logits; ap.V = a->V; ap.stride_b = a->stride_b; ap.stride_row = a->stride_row;
    ap.R = a->R; ap.rows_mode = a->rows_mode; ap.n_nodes = a->n_nodes; ap.node_argmax = a->node_argmax;
    ap.fault_tile = (a->flags & CADD_FLAG_TEST_DROP_TILE) ? 1 : -1;
    if (verify_is_small(a)) {
        WalkParams wp;
        wp.batch = a->batch; wp.L = a->L; wp.R = a->R; wp.n_nodes = a->n_nodes; wp.token_ids = a->token_ids;
        wp.parent_idx = a->parent_idx; wp.node_argmax = a->node_argmax; wp.accepted_len = a->accepted_len;
        wp.accepted_nodes = a->accepted_nodes; wp.next_bonus = a->next_bonus; wp.status = a->status;
        ap.ctas_per_request = 1;
        if (a->logits_dtype == CADD_DTYPE_BF16) verify_small_kernel<CADD_DTYPE_BF16><<<(unsigned)a->batch, kVerifySmallThreads, 0, st>>>(ap, wp);
        else verify_small_kernel<CADD_DTYPE_FP32><<<(unsigned)a->batch, kVerifySmallThreads, 0, st>>>(ap, wp);
        if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
        return CADD_OK;
    }
    // LIVE with a small node cap: most rows are padding on typical trees, so eight rows share a CTA (interleaved, so
    // that a request's live rows, which come first, still spread over its CTAs) and few CTAs are launched only to exit.
    // Large caps and DENSE keep one row per CTA: every row is work there and short CTAs keep the last wave short.
    ap.ctas_per_request = (a->rows_mode == CADD_ROWS_LIVE && a->R <= kLiveSharedRowsMaxR) ? (a->R + 7) / 8 : a->R;
    const unsigned rows = (unsigned)((int64_t)a->batch * ap.ctas_per_request);
    const bool overlap = (int64_t)a->batch * a->R * a->V * (a->logits_dtype == CADD_DTYPE_BF16 ? 2 : 4) >= kOverlapMinBytes;
    const void* kfn = a->logits_dtype == CADD_DTYPE_BF16 ? (const void*)row_argmax_kernel<CADD_DTYPE_BF16>
                                                          : (const void*)row_argmax_kernel<CADD_DTYPE_FP32>;
    if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)argmax_smem_bytes()) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    if (!(a->flags & CADD_VERIFY_ONLY_WALK)) {
        const cudaError_t le = a->logits_dtype == CADD_DTYPE_BF16
            ? launch_dependent(overlap, row_argmax_kernel<CADD_DTYPE_BF16>, dim3(rows), dim3(kThreads), argmax_smem_bytes(), st, ap)
            : launch_dependent(overlap, row_argmax_kernel<CADD_DTYPE_FP32>, dim3(rows), dim3(kThreads), argmax_smem_bytes(), st, ap);
        if (le != cudaSuccess) { cudaGetLastError(); return CADD_ERR_LAUNCH; }
    }
    if (a->flags & CADD_VERIFY_ONLY_ARGMAX) return CADD_OK;

    WalkParams wp;
    wp.batch = a->batch; wp.L = a->L; wp.R = a->R; wp.n_nodes = a->n_nodes; wp.token_ids = a->token_ids;
    wp.parent_idx = a->parent_idx; wp.node_argmax = a->node_argmax; wp.accepted_len = a->accepted_len;
    wp.accepted_nodes = a->accepted_nodes; wp.next_bonus = a->next_bonus; wp.status = a->status;
    const int wpb = 4;
    if (launch_dependent(overlap, accept_walk_kernel, dim3((unsigned)((a->batch + wpb - 1) / wpb)), dim3(wpb * 32), 0, st, wp) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    return CADD_OK;
}

// ---------------- verification fused into the output projection ----------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// The driver's tensor-map encoder, looked up through the runtime (the library does not link the driver directly).
static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return (EncodeTiledFn) nullptr;
        }
        return (EncodeTiledFn)f;
    }();
    return fn;
}
// 2-D map of a row-major bf16 matrix [rows, cols] (row stride in elements); boxes of box_rows x 64 columns, 128-byte
// swizzle, out-of-range elements read as zero (ragged rows, columns and hidden sizes need no special casing).
static bool make_map_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t stride, int box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)stride * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kHeadBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int check_head_shape(const cadd_head_args* a) {
    if (!a) return CADD_ERR_NULL;
    if (a->struct_size != sizeof(cadd_head_args)) return CADD_ERR_STRUCT_SIZE;
    if (a->batch < 1 || a->L < 1 || a->L > 64 || a->R < 1 || a->V < 1 || a->V >= ((int64_t)1 << 31) || a->hidden < 1 ||
        a->hidden > (1 << 20) || (int64_t)a->batch * a->R >= ((int64_t)1 << 31))
        return CADD_ERR_SHAPE;
    if (a->rows_mode != CADD_ROWS_LIVE && a->rows_mode != CADD_ROWS_DENSE) return CADD_ERR_DTYPE;
    return CADD_OK;
}

// Workspace of the fused verification: packed row maxima [M] u64 | error word (256 B) | LIVE mode only: row offsets
// [batch + 1] int32 and the packed copy of the live hidden states [M, hidden] bf16 (sized for every row live).
struct HeadLayout { size_t best_bytes, off_bytes, pack_bytes, total; };
static HeadLayout head_layout(const cadd_head_args* a) {
    HeadLayout l;
    const size_t M = (size_t)a->batch * a->R;
    l.best_bytes = (M * 8 + 255) & ~(size_t)255;
    l.off_bytes = a->rows_mode == CADD_ROWS_LIVE ? ((((size_t)a->batch + 1) * 4 + 255) & ~(size_t)255) : 0;
    l.pack_bytes = a->rows_mode == CADD_ROWS_LIVE ? ((M * (size_t)a->hidden * 2 + 255) & ~(size_t)255) : 0;
    l.total = l.best_bytes + 256 + l.off_bytes + l.pack_bytes;
    return l;
}

int cadd_head_workspace_bytes(const cadd_head_args* a, size_t* out) {
    int rc = check_head_shape(a);
    if (rc != CADD_OK) return rc;
    if (!out) return CADD_ERR_NULL;
    *out = head_layout(a).total;
    return CADD_OK;
}

int cadd_verify_tree_fused_head(const cadd_head_args* a, void* cuda_stream) {
    int rc = check_head_shape(a);
    if (rc != CADD_OK) return rc;
    if (!a->hidden_states || !a->weight || !a->n_nodes || !a->token_ids || !a->parent_idx || !a->node_argmax || !a->accepted_len ||
        !a->accepted_nodes || !a->next_bonus)
        return CADD_ERR_NULL;
    // the tiled bulk copies need 16-byte aligned bases and row strides
    if (!aligned(a->hidden_states, 16) || !aligned(a->weight, 16) || a->stride_row % 8 != 0 || a->stride_w % 8 != 0) return CADD_ERR_ALIGN;
    if (!aligned(a->n_nodes, 4) || !aligned(a->token_ids, 4) || !aligned(a->parent_idx, 4) || !aligned(a->node_argmax, 4) ||
        !aligned(a->accepted_len, 4) || !aligned(a->accepted_nodes, 4) || !aligned(a->next_bonus, 4) || !aligned(a->status, 4))
        return CADD_ERR_ALIGN;
    if (a->stride_row < a->hidden || a->stride_w < a->hidden) return CADD_ERR_SHAPE;
    const bool live = a->rows_mode == CADD_ROWS_LIVE;
    if (live && a->hidden % 8 != 0) return CADD_ERR_ALIGN;        // packed rows must keep 16-byte alignment
    const HeadLayout lay = head_layout(a);
    if (!a->workspace || !aligned(a->workspace, 256) || a->workspace_bytes < lay.total) return CADD_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    const int64_t M = (int64_t)a->batch * a->R;
    unsigned char* ws = (unsigned char*)a->workspace;
    int32_t* err = (int32_t*)(ws + lay.best_bytes);
    int32_t* row_off = live ? (int32_t*)(ws + lay.best_bytes + 256) : nullptr;
    __nv_bfloat16* packed = live ? (__nv_bfloat16*)(ws + lay.best_bytes + 256 + lay.off_bytes) : nullptr;
    if (cudaMemsetAsync(ws, 0, lay.best_bytes + 256, st) != cudaSuccess) { cudaGetLastError(); return CADD_ERR_LAUNCH; }
    if (live) {
        // LIVE mode: the GEMM runs on the live rows only, copied next to one another first (a few MB at most for trees
        // of tens of nodes); the row count stays on the device
        head_live_offsets_kernel<<<1, 1024, 0, st>>>(a->n_nodes, a->batch, a->R, row_off);
        head_pack_rows_kernel<<<dim3((unsigned)a->R, (unsigned)a->batch), 128, 0, st>>>((const __nv_bfloat16*)a->hidden_states, a->stride_row,
                                                                                           a->hidden, a->R, a->n_nodes, row_off, packed);
        if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
    }
    CUtensorMap map_h, map_w;
    if (!(live ? make_map_bf16(&map_h, packed, M, a->hidden, a->hidden, kHeadBM)
               : make_map_bf16(&map_h, a->hidden_states, M, a->hidden, a->stride_row, kHeadBM)) ||
        !make_map_bf16(&map_w, a->weight, a->V, a->hidden, a->stride_w, kHeadBN))
        return CADD_ERR_LAUNCH;

    HeadParams hp;
    hp.M = M; hp.V = a->V; hp.Kdim = a->hidden;
    hp.m_tiles = (int)((M + kHeadBM - 1) / kHeadBM);
    hp.n_tiles = (int)((a->V + kHeadBN - 1) / kHeadBN);
    {
        // row tiles per group: about 24 MB of hidden states, so that they stay L2-resident while W streams by
        int64_t g = ((int64_t)24 << 20) / ((int64_t)kHeadBM * a->hidden * 2);
        hp.group_m = (int)(g < 1 ? 1 : (g > hp.m_tiles ? hp.m_tiles : g));
    }
    hp.R = a->R; hp.rows_mode = a->rows_mode; hp.n_nodes = a->n_nodes;
    hp.m_live = live ? row_off + a->batch : nullptr;
    hp.row_best = (unsigned long long*)ws;
    hp.error = err;
    if (cudaFuncSetAttribute(head_argmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)head_smem_bytes()) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    const int64_t work = (int64_t)hp.m_tiles * hp.n_tiles;
    const int sms = sm_count();
    const unsigned grid = (unsigned)(work < sms ? work : sms);
    head_argmax_kernel<<<grid, kHeadThreads, head_smem_bytes(), st>>>(map_h, map_w, hp);
    if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
    head_decode_kernel<<<(unsigned)((M + 255) / 256), 256, 0, st>>>(hp.row_best, a->n_nodes, row_off, hp.error, M, a->R, a->rows_mode, a->node_argmax);
    if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;

    WalkParams wp;
    wp.batch = a->batch; wp.L = a->L; wp.R = a->R; wp.n_nodes = a->n_nodes; wp.token_ids = a->token_ids;
    wp.parent_idx = a->parent_idx; wp.node_argmax = a->node_argmax; wp.accepted_len = a->accepted_len;
    wp.accepted_nodes = a->accepted_nodes; wp.next_bonus = a->next_bonus; wp.status = a->status;
    const int wpb = 4;
    accept_walk_kernel<<<(a->batch + wpb - 1) / wpb, wpb * 32, 0, st>>>(wp);
    if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
    return CADD_OK;
}

// ---------------- offline cost fitting (Eq. 12) ----------------

int cadd_fit_cost_tables(const cadd_fit_args* a, void* cuda_stream) {
    if (!a) return CADD_ERR_NULL;
    if (a->struct_size != sizeof(cadd_fit_args)) return CADD_ERR_STRUCT_SIZE;
    if (a->n_tables < 1 || a->n_tables > 65535 || a->N < 1 || a->N > kFitMaxN) return CADD_ERR_SHAPE;
    if (!a->y || !a->fit) return CADD_ERR_NULL;
    if (!aligned(a->y, 8) || !aligned(a->fit, 8) || !aligned(a->n_breaks, 4) || !aligned(a->status, 4)) return CADD_ERR_ALIGN;
    if (cudaFuncSetAttribute(fit_cost_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fit_smem_bytes()) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    FitParams fp;
    fp.n_tables = a->n_tables; fp.N = a->N; fp.y = a->y; fp.fit = a->fit; fp.n_breaks = a->n_breaks; fp.status = a->status;
    fit_cost_kernel<<<a->n_tables, kFitThreads, fit_smem_bytes(), (cudaStream_t)cuda_stream>>>(fp);
    if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
    return CADD_OK;
}

// ---------------- tree construction fused into the drafter's output projection ----------------

constexpr int kDraftMaxCtas = 256;        // CTAs of the fused draft kernel (one per SM); sizes its list scratch
struct DraftPlan {
    int KP, m_tiles, n_tiles, chunk_tiles, n_chunks, halves;
    size_t chunk_bytes, merged_bytes, list_bytes, total_bytes;
};
// Chunks of column tiles per row: at most kDraftMaxRecords records per row (one or two per chunk), chosen so that the number
// of work items (row tiles x chunks) fills whole waves of one CTA per SM without making chunks needlessly short.
static DraftPlan plan_draft_head(const cadd_build_args* a, int sms) {
    DraftPlan pl;
    pl.KP = a->K > kPreciseMin ? a->K : kPreciseMin;
    const int64_t M = (int64_t)a->batch * a->L;
    pl.m_tiles = (int)((M + kHeadBM - 1) / kHeadBM);
    pl.n_tiles = (int)((a->V + kHeadBN - 1) / kHeadBN);
    // estimated duration in tile times: waves x (tiles per chunk + about three tiles' worth of threshold warm-up and
    // pipeline fill per chunk); the smallest wins, ties go to fewer chunks
    pl.halves = pl.KP <= 16 ? 2 : 1;                                  // epilogue warps per group of 32 rows (see DraftHeadShared)
    const int max_chunks = kDraftMaxRecords / pl.halves;              // what the merge kernel folds per row
    const int cap = pl.n_tiles < max_chunks ? pl.n_tiles : max_chunks;
    int best = 1;
    int64_t best_cost = -1;
    for (int nc = 1; nc <= cap; ++nc) {
        const int ct = (pl.n_tiles + nc - 1) / nc;
        const int real = (pl.n_tiles + ct - 1) / ct;                       // chunks that actually exist with this size
        const int64_t items = (int64_t)pl.m_tiles * real;
        const int64_t waves = (items + sms - 1) / sms;
        const int64_t cost = waves * (ct + 3);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = real; }
    }
    pl.chunk_tiles = (pl.n_tiles + best - 1) / best;
    pl.n_chunks = (pl.n_tiles + pl.chunk_tiles - 1) / pl.chunk_tiles;
    const size_t stride = seg_partial_stride(pl.KP);
    pl.chunk_bytes = (((size_t)M * pl.n_chunks * pl.halves * stride) + 255) & ~(size_t)255;
    pl.merged_bytes = (((size_t)M * stride) + 255) & ~(size_t)255;
    pl.list_bytes = (size_t)kDraftMaxCtas * 2 * kDraftPending * kHeadBM * 8;   // the queues' scratch
    pl.total_bytes = pl.chunk_bytes + pl.merged_bytes + pl.list_bytes + 256;
    return pl;
}

static int check_build_head(const cadd_build_head_args* h) {
    if (!h) return CADD_ERR_NULL;
    if (h->struct_size != sizeof(cadd_build_head_args)) return CADD_ERR_STRUCT_SIZE;
    int rc = check_build_shape(&h->build);
    if (rc != CADD_OK) return rc;
    if (h->hidden < 1 || h->hidden > (1 << 20) || h->build.K > kDraftMaxKP) return CADD_ERR_SHAPE;
    return CADD_OK;
}

int cadd_build_head_workspace_bytes(const cadd_build_head_args* h, size_t* out) {
    int rc = check_build_head(h);
    if (rc != CADD_OK) return rc;
    if (!out) return CADD_ERR_NULL;
    // sized for the largest cut (kDraftMaxRecords records per row), so the answer does not depend on the device
    const size_t stride = seg_partial_stride(h->build.K > kPreciseMin ? h->build.K : kPreciseMin);
    const size_t M = (size_t)h->build.batch * h->build.L;
    *out = ((M * kDraftMaxRecords * stride + 255) & ~(size_t)255) + ((M * stride + 255) & ~(size_t)255) + (size_t)kDraftMaxCtas * 2 * kDraftPending * kHeadBM * 8 + 256;
    return CADD_OK;
}

int cadd_build_tree_fused_head(const cadd_build_head_args* h, void* cuda_stream) {
    int rc = check_build_head(h);
    if (rc != CADD_OK) return rc;
    const cadd_build_args* a = &h->build;
    if (!h->hidden_states || !h->weight || !a->n_nodes || !a->token_ids || !a->parent_idx || !a->depth) return CADD_ERR_NULL;
    if (a->cost_kind == CADD_COST_QUADRATIC && !a->cost_coef) return CADD_ERR_NULL;
    if (a->cost_kind == CADD_COST_TABLE && (!a->cost_table || !a->table_idx || !a->t_draft || a->n_tables < 1)) return CADD_ERR_NULL;
    if (a->cost_kind == CADD_COST_TABLE_INTERP && (!a->cost_table || !a->ctx_grid || !a->t_draft || a->n_tables < 1)) return CADD_ERR_NULL;
    if ((a->flags & CADD_FLAG_EMIT_DENSE_MASK) && !a->mask_dense) return CADD_ERR_NULL;
    if ((a->flags & CADD_FLAG_EMIT_TOPK) && !a->topk_token && !a->topk_logprob) return CADD_ERR_NULL;
    if (!aligned(h->hidden_states, 16) || !aligned(h->weight, 16) || h->stride_row % 8 != 0 || h->stride_w % 8 != 0) return CADD_ERR_ALIGN;
    if (h->stride_row < h->hidden || h->stride_w < h->hidden) return CADD_ERR_SHAPE;
    if (!aligned(a->cost_coef, 8) || !aligned(a->cost_table, 8) || !aligned(a->t_draft, 8) || !aligned(a->node_logprob, 8) ||
        !aligned(a->phi, 8) || !aligned(a->theta, 8) || !aligned(a->theta_curve, 8) || !aligned(a->topk_logprob, 8))
        return CADD_ERR_ALIGN;
    if (!aligned(a->n_nodes, 4) || !aligned(a->token_ids, 4) || !aligned(a->parent_idx, 4) || !aligned(a->depth, 4) ||
        !aligned(a->position_ids, 4) || !aligned(a->mask_bits, 4) || !aligned(a->topk_token, 4) || !aligned(a->status, 4) ||
        !aligned(a->l_eff, 4) || !aligned(a->bonus_token, 4) || !aligned(a->ctx_len, 4) || !aligned(a->table_idx, 4) ||
        !aligned(a->ctx_grid, 4))
        return CADD_ERR_ALIGN;
    const int sms = sm_count();
    const DraftPlan pl = plan_draft_head(a, sms);
    size_t need = 0;
    cadd_build_head_workspace_bytes(h, &need);
    if (!a->workspace || !aligned(a->workspace, 256) || a->workspace_bytes < need) return CADD_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    const int64_t M = (int64_t)a->batch * a->L;
    CUtensorMap map_h, map_w;
    if (!make_map_bf16(&map_h, h->hidden_states, M, h->hidden, h->stride_row, kHeadBM) ||
        !make_map_bf16(&map_w, h->weight, a->V, h->hidden, h->stride_w, kHeadBN))
        return CADD_ERR_LAUNCH;
    unsigned char* ws = (unsigned char*)a->workspace;
    unsigned char* merged = ws + pl.chunk_bytes;
    uint64_t* pend = (uint64_t*)(ws + pl.chunk_bytes + pl.merged_bytes);
    int32_t* err = (int32_t*)(ws + pl.chunk_bytes + pl.merged_bytes + pl.list_bytes);
    if (cudaMemsetAsync(err, 0, 256, st) != cudaSuccess) { cudaGetLastError(); return CADD_ERR_LAUNCH; }

    DraftHeadParams dp;
    dp.M = M; dp.V = a->V; dp.Kdim = h->hidden; dp.m_tiles = pl.m_tiles; dp.n_tiles = pl.n_tiles;
    dp.chunk_tiles = pl.chunk_tiles; dp.n_chunks = pl.n_chunks; dp.L = a->L; dp.KP = pl.KP; dp.l_eff = a->l_eff;
    dp.chunk_partials = ws; dp.pend = pend; dp.halves = pl.halves; dp.error = err;
    if (cudaFuncSetAttribute(head_softmax_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)draft_head_smem_bytes()) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    const int64_t items = (int64_t)pl.m_tiles * pl.n_chunks;
    const int ctas = sms < kDraftMaxCtas ? sms : kDraftMaxCtas;
    head_softmax_topk_kernel<<<(unsigned)(items < ctas ? items : ctas), kDraftThreads, draft_head_smem_bytes(), st>>>(map_h, map_w, dp);
    if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
    draft_merge_kernel<<<(unsigned)((M + 3) / 4), 128, 0, st>>>(dp, merged);
    if (cudaGetLastError() != cudaSuccess) return CADD_ERR_LAUNCH;
    return launch_expand(a, pl.KP, 1, kRecSegPartial, merged, st, false);
}

// ---------------- tree verification under sampling ----------------

int cadd_verify_tree_sampled(const cadd_sample_args* a, void* cuda_stream) {
    if (!a) return CADD_ERR_NULL;
    if (a->struct_size != sizeof(cadd_sample_args)) return CADD_ERR_STRUCT_SIZE;
    if (a->batch < 1 || a->L < 1 || a->L > 64 || a->R < 1 || a->V < 1 || a->V >= ((int64_t)1 << 31) ||
        (int64_t)a->batch * a->R >= ((int64_t)1 << 31) || !(a->temperature > 0.0) || !(a->temperature < 1e30))
        return CADD_ERR_SHAPE;
    if (a->logits_dtype != CADD_DTYPE_BF16 && a->logits_dtype != CADD_DTYPE_FP32) return CADD_ERR_DTYPE;
    if (a->rows_mode != CADD_ROWS_LIVE && a->rows_mode != CADD_ROWS_DENSE) return CADD_ERR_DTYPE;
    const int epc = a->logits_dtype == CADD_DTYPE_BF16 ? 8 : 4;
    if (a->V / epc / kRunChunks + 3 > kMaxRuns) return CADD_ERR_SHAPE;     // rows longer than the run table
    if (!a->target_logits || !a->uniforms || !a->n_nodes || !a->token_ids || !a->parent_idx || !a->node_token || !a->accepted_len ||
        !a->accepted_nodes || !a->next_bonus)
        return CADD_ERR_NULL;
    const size_t es = a->logits_dtype == CADD_DTYPE_BF16 ? 2 : 4;
    if (!aligned(a->target_logits, es) || !aligned(a->uniforms, 8)) return CADD_ERR_ALIGN;
    if (!aligned(a->n_nodes, 4) || !aligned(a->token_ids, 4) || !aligned(a->parent_idx, 4) || !aligned(a->node_token, 4) ||
        !aligned(a->accepted_len, 4) || !aligned(a->accepted_nodes, 4) || !aligned(a->next_bonus, 4) || !aligned(a->status, 4))
        return CADD_ERR_ALIGN;
    if (a->stride_row < a->V || a->stride_b < 0) return CADD_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    SampleParams sp;
    sp.logits = a->target_logits; sp.V = a->V; sp.stride_b = a->stride_b; sp.stride_row = a->stride_row;
    sp.R = a->R; sp.rows_mode = a->rows_mode; sp.c = (float)(1.4426950408889634 / a->temperature);
    sp.n_nodes = a->n_nodes; sp.uniforms = a->uniforms; sp.node_token = a->node_token;
    sp.fault_tile = (a->flags & CADD_FLAG_TEST_DROP_TILE) ? 1 : -1;
    // LIVE with a small node cap: eight rows of a request share a CTA (as in cadd_verify_tree)
    const bool shared_rows = a->rows_mode == CADD_ROWS_LIVE && a->R <= kLiveSharedRowsMaxR;
    sp.ctas_per_request = shared_rows ? (a->R + 7) / 8 : a->R;
    const unsigned rows = (unsigned)((int64_t)a->batch * sp.ctas_per_request);
    const bool bf16 = a->logits_dtype == CADD_DTYPE_BF16;
    auto kfn = bf16 ? (shared_rows ? row_sample_shared_rows_kernel<CADD_DTYPE_BF16> : row_sample_kernel<CADD_DTYPE_BF16>)
                    : (shared_rows ? row_sample_shared_rows_kernel<CADD_DTYPE_FP32> : row_sample_kernel<CADD_DTYPE_FP32>);
    if (cudaFuncSetAttribute((const void*)kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sample_smem_bytes()) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    const bool overlap = (int64_t)a->batch * a->R * a->V * (int64_t)es >= kOverlapMinBytes;
    if (launch_dependent(overlap, kfn, dim3(rows), dim3(kThreads), sample_smem_bytes(), st, sp) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }

    WalkParams wp;                                           // the walk is the greedy one with the drawn tokens in place of the arg-max
    wp.batch = a->batch; wp.L = a->L; wp.R = a->R; wp.n_nodes = a->n_nodes; wp.token_ids = a->token_ids;
    wp.parent_idx = a->parent_idx; wp.node_argmax = a->node_token; wp.accepted_len = a->accepted_len;
    wp.accepted_nodes = a->accepted_nodes; wp.next_bonus = a->next_bonus; wp.status = a->status;
    const int wpb = 4;
    if (launch_dependent(overlap, accept_walk_kernel, dim3((unsigned)((a->batch + wpb - 1) / wpb)), dim3(wpb * 32), 0, st, wp) != cudaSuccess) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    return CADD_OK;
}

}  // extern "C"
