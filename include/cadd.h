/*
 * cadd.h — C ABI of the B200 (sm_100a) implementation of the per-round hot path of CaDDTree
 * ("Cost-Aware Diffusion Draft Trees for Speculative Decoding"): batched cost-aware draft-tree
 * construction and tree verification.
 *
 * Conventions that hold for every call below
 *   - Every data pointer is a DEVICE pointer owned by the caller, unless a comment says HOST.
 *     The argument structs themselves live in HOST memory and are read during the call only.
 *   - The library allocates nothing, frees nothing, never synchronises the device and never
 *     touches a stream other than the one passed in.  Work is enqueued on `cuda_stream`
 *     (a cudaStream_t cast to void*; NULL = the legacy default stream) and the call returns
 *     immediately.  Results are valid once that stream reaches the end of the enqueued work.
 *   - Scratch memory is passed in (`workspace`, `workspace_bytes`); its size comes from the
 *     *_workspace_bytes query.  Its contents need no initialisation and are undefined after
 *     the call.  Two calls that may overlap on the device need distinct workspaces.
 *   - Return value: CADD_OK, or a negative code for an error detected on the host before any
 *     kernel was launched (nothing is written in that case).  Conditions found on the device
 *     are reported per request in the `status` output as CADD_STATUS_* bit flags.
 *   - Index arithmetic is 64-bit; strides are counted in ELEMENTS of the logits dtype; the
 *     vocabulary axis is contiguous.
 *   - There is no CPU fallback: a machine without a CUDA device gets CADD_ERR_LAUNCH.
 *   - Finite logits are expected to satisfy |x| <= 1e6 (real logits are far smaller).  Larger finite values are
 *     processed without fault, rankings stay exact, but the reported log-probabilities lose accuracy.
 *
 * Notation follows the paper: V vocabulary size, L draft block length (= maximum depth),
 * K candidates kept per position, n the number of DRAFT nodes of the tree (the root, i.e. the
 * bonus token, is row 0 and is not counted), B_max the cap on n, R >= B_max + 1 the row
 * capacity of the per-request node arrays, C_d the drafting cost, C_v(n) the verification cost.
 */
#ifndef CADD_H_
#define CADD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CADD_ABI_VERSION 4

/* ---- return codes (host side, synchronous) ---- */
#define CADD_OK              0
#define CADD_ERR_NULL       -1   /* a required pointer is NULL */
#define CADD_ERR_STRUCT_SIZE -2  /* struct_size does not match this library */
#define CADD_ERR_SHAPE      -3   /* batch<1, L not in [1,64], K not in [1,64], V<1 or V>=2^31, B_max not in [0,2048], R<B_max+1 */
#define CADD_ERR_DTYPE      -4   /* logits_dtype / cost_kind / rows_mode out of range */
#define CADD_ERR_ALIGN      -5   /* logits base pointer not aligned to its element size, or a double/int array misaligned */
#define CADD_ERR_WORKSPACE  -6   /* workspace NULL, misaligned (256 B) or smaller than the query says */
#define CADD_ERR_LAUNCH     -7   /* a CUDA runtime call failed (wraps cudaGetLastError) */
#define CADD_ERR_STATIC_SCRATCH -8  /* cadd_build_tree_static_scratch: the problem needs more scratch than CADD_STATIC_SCRATCH_BYTES */

/* ---- per-request status bits (device side, written to `status`) ---- */
#define CADD_STATUS_NONFINITE_INPUT      1   /* a NaN or +Inf draft logit was seen (NaN orders as -Inf; +Inf => empty tree) */
#define CADD_STATUS_FEWER_THAN_K_FINITE  2   /* some live position has fewer than K finite logits */
#define CADD_STATUS_CAP_HIT              4   /* expansion ended because n reached B_max */
#define CADD_STATUS_FRONTIER_EXHAUSTED   8   /* expansion ended because no candidate was left */
#define CADD_STATUS_L_EFF_CLAMPED       16   /* l_eff[b] was outside [0, L] */
#define CADD_STATUS_COST_NONPOSITIVE    32   /* C_d + C_v(n) <= 0 (or not finite) was met; expansion stopped there */
#define CADD_STATUS_BAD_N_NODES         64   /* verify: n_nodes[b] was outside [0, R-1] and was clamped */
#define CADD_STATUS_BAD_TABLE_IDX      256   /* build, CADD_COST_TABLE: table_idx[b] was outside [0, n_tables); the request returns the empty tree */
#define CADD_STATUS_INTERNAL_TIMEOUT   128   /* a bounded wait on an asynchronous copy ran out; build returns the empty tree, verify leaves -2 in node_argmax */

#define CADD_DTYPE_BF16 0
#define CADD_DTYPE_FP32 1

#define CADD_COST_QUADRATIC 0    /* C_v(n) = a + b n + c n^2, per request */
#define CADD_COST_TABLE     1    /* C_v(n) = cost_table[table_idx[b]][n], n = 0..B_max */
#define CADD_COST_TABLE_INTERP 2 /* context interpolation at inference (Eq. 13): cost_table row j is the fitted cost at
                                    context length ctx_grid[j]; with L_j <= ctx_len[b] < L_{j+1} and
                                    alpha = (ctx_len[b] - L_j) / (L_{j+1} - L_j),
                                    C_v(n) = (1 - alpha) cost_table[j][n] + alpha cost_table[j+1][n];
                                    outside the grid the nearest table is used */

#define CADD_FLAG_EMIT_DENSE_MASK 1u   /* also write mask_dense */
#define CADD_FLAG_EMIT_TOPK       2u   /* also write topk_token / topk_logprob */
#define CADD_FLAG_FIXED_BUDGET    4u   /* ignore the stopping rule: expand to B_max (DDTree; the paper's constant-cost ablation, Table 2) */

/* Measurement aids: a call with one of these enqueues only one of the two kernels of cadd_build_tree, so that each can
   be timed alone with events on the caller's stream.  ONLY_TOPK runs the softmax/top-K pass (Eq. 1; Algorithm 1,
   Require) and leaves its per-position records in the workspace, writing no output; ONLY_EXPAND runs Algorithm 1 and
   the emission on the records an earlier call left in the SAME workspace for the same shape.  Both together:
   CADD_ERR_DTYPE.  ONLY_TOPK followed by ONLY_EXPAND gives exactly the outputs of one plain call. */
#define CADD_FLAG_ONLY_TOPK       8u
#define CADD_FLAG_ONLY_EXPAND    16u
/* The same for cadd_verify_tree (its `flags` field): only the per-node argmax, or only the walk on a node_argmax
   array that an earlier call filled. */
#define CADD_VERIFY_ONLY_ARGMAX   1u
#define CADD_VERIFY_ONLY_WALK     2u
/* Small problems are served by one kernel per call (see cadd_build_tree / cadd_verify_tree); these flags make a call
   take the regular two-kernel path whatever its size (results are the same; for measurements and tests). */
#define CADD_FLAG_REGULAR_PATH   32u   /* cadd_build_tree */
#define CADD_VERIFY_REGULAR_PATH  4u   /* cadd_verify_tree */
/* Test hook, accepted in the `flags` of cadd_build_tree, cadd_verify_tree and cadd_verify_tree_sampled: the streaming
   kernel never issues the asynchronous copy of the second tile (16 KB) of each row it reads (the first, if the row has
   only one), and its wait for that one tile gives up after a few tries.  Nothing hangs and nothing faults: the call
   exercises the library's bounded-wait exit (copies already in flight are waited for, then the CTA leaves) and every
   request reports CADD_STATUS_INTERNAL_TIMEOUT with the empty tree (build) or accepted_len 0 (verify).  For tests only. */
#define CADD_FLAG_TEST_DROP_TILE  0x80000000u

#define CADD_ROWS_LIVE  0        /* verify reads target rows 0..n_nodes[b] only */
#define CADD_ROWS_DENSE 1        /* verify takes the argmax of all R rows */

/*
 * Arguments of cadd_build_tree: one decoding round's tree construction for `batch` requests.
 * Implements Eq. 1 (per-position marginals q_i = softmax(l_i)), the top-K lists Algorithm 1
 * requires, Algorithm 1 itself (best-first expansion over log prefix probabilities, Eq. 5, with
 * the greedy stopping rule of Eq. 11 / Corollary 1 on the surrogate throughput of Eq. 7), and the
 * draft-tree data structure with its ancestor mask (Section 3.3).
 *
 * Ordering rules (the paper is silent on ties): candidates of a position are ranked by
 * (logit descending, token id ascending); nodes are popped by (score descending, depth ascending,
 * token id ascending, parent row ascending).  Row 0 of every per-request array is the root.
 * Row j >= 1 is the j-th popped node.  Rows above n_nodes[b] are padding: token -1, parent -1,
 * depth 0, position 0, log-prob 0, empty mask row.
 */
typedef struct cadd_build_args {
    uint32_t struct_size;          /* = sizeof(cadd_build_args) */
    uint32_t flags;                /* CADD_FLAG_* */
    int32_t  batch, L, K, B_max, R;
    int32_t  logits_dtype;         /* CADD_DTYPE_* */
    int64_t  V;
    const void* draft_logits;      /* [batch, L, V]; element (b,i,v) at b*stride_b + i*stride_l + v */
    int64_t  stride_b, stride_l;   /* in elements */
    const int32_t* l_eff;          /* [batch] live positions per request, NULL => L (rows i >= l_eff[b] are never read) */
    const int32_t* bonus_token;    /* [batch] token of the root, NULL => -1 */
    const int32_t* ctx_len;        /* [batch] context length, NULL => 0; position_ids = ctx_len + depth */
    int32_t  cost_kind;            /* CADD_COST_* */
    int32_t  n_tables;             /* TABLE, TABLE_INTERP: number of rows of cost_table */
    const double*  cost_coef;      /* QUADRATIC: [batch,4] = (C_d, a, b, c) */
    const double*  cost_table;     /* TABLE: [n_tables, B_max+1] */
    const int32_t* table_idx;      /* TABLE: [batch], each in [0, n_tables); a value outside is never dereferenced: CADD_STATUS_BAD_TABLE_IDX, empty tree */
    const double*  t_draft;        /* TABLE, TABLE_INTERP: [batch] C_d */
    const int32_t* ctx_grid;       /* TABLE_INTERP: [n_tables] strictly ascending context lengths of the tables */
    /* outputs; n_nodes, token_ids, parent_idx, depth are required, the rest may be NULL */
    int32_t* n_nodes;              /* [batch] n* */
    int32_t* token_ids;            /* [batch,R] */
    int32_t* parent_idx;           /* [batch,R] row of the parent, -1 for the root and padding */
    int32_t* depth;                /* [batch,R] */
    int32_t* position_ids;         /* [batch,R] */
    double*  node_logprob;         /* [batch,R] log prefix probability sigma of each node (root 0) */
    double*  phi;                  /* [batch] expected accepted draft tokens Phi*(n*) (Eq. 6) */
    double*  theta;                /* [batch] surrogate throughput (1+Phi)/(C_d+C_v(n*)) (Eq. 7) */
    double*  theta_curve;          /* [batch,R] optional: theta*(n) for n = 0..n_nodes[b] (Prop. 1), 0 above; with
                                      CADD_FLAG_FIXED_BUDGET this is the whole budget sweep of one expansion */
    uint32_t* mask_bits;           /* [batch,R,ceil(R/32)] bit c of row j set iff c == j or c is an ancestor of j */
    uint8_t*  mask_dense;          /* [batch,R,R] same as bytes, written only with CADD_FLAG_EMIT_DENSE_MASK */
    int32_t* topk_token;           /* [batch,L,K] written only with CADD_FLAG_EMIT_TOPK; -1 where absent */
    double*  topk_logprob;         /* [batch,L,K] log q_i^(k); -Inf where absent */
    int32_t* status;               /* [batch] CADD_STATUS_* bits */
    void*    workspace;            /* >= cadd_build_workspace_bytes, 256-byte aligned */
    size_t   workspace_bytes;
} cadd_build_args;

/*
 * Arguments of cadd_verify_tree: greedy verification of the built trees (Section 3.1: a draft token
 * is accepted iff it equals the argmax of the target distribution given its prefix; Section 3.3: the
 * path with the longest accepted prefix is kept and the next bonus token follows it).
 * Step 1: node_argmax[b,j] = argmax_v target_logits[b,j,v], ties to the lowest v, NaN ordered as -Inf.
 * Step 2: walk from the root, at each node moving to the child whose token equals that node's argmax.
 * next_bonus[b] is the argmax at the last accepted node.
 */
typedef struct cadd_verify_args {
    uint32_t struct_size;          /* = sizeof(cadd_verify_args) */
    uint32_t flags;                /* 0, or one of CADD_VERIFY_ONLY_* */
    int32_t  batch, L, R;
    int32_t  logits_dtype;         /* CADD_DTYPE_* */
    int32_t  rows_mode;            /* CADD_ROWS_* */
    int32_t  reserved0;
    int64_t  V;
    const void* target_logits;     /* [batch, R, V]; element (b,j,v) at b*stride_b + j*stride_row + v */
    int64_t  stride_b, stride_row; /* in elements */
    const int32_t* n_nodes;        /* [batch]   from cadd_build_tree */
    const int32_t* token_ids;      /* [batch,R] from cadd_build_tree */
    const int32_t* parent_idx;     /* [batch,R] from cadd_build_tree */
    /* outputs, all required except status */
    int32_t* node_argmax;          /* [batch,R]; -1 for rows not read in LIVE mode */
    int32_t* accepted_len;         /* [batch] alpha >= 0 */
    int32_t* accepted_nodes;       /* [batch,L] rows of the accepted path in order, -1 padded */
    int32_t* next_bonus;           /* [batch] */
    int32_t* status;               /* [batch] CADD_STATUS_* bits, may be NULL */
    void*    workspace;            /* >= cadd_verify_workspace_bytes (may be 0 => NULL allowed) */
    size_t   workspace_bytes;
} cadd_verify_args;

/*
 * Tree verification fused into the target's output projection (Section 3.1: "the target's prediction at every
 * tree node" is argmax_v of h_j . W_v, with h_j the target's last hidden state at node j and W the output
 * embedding; Section 3.3 for the walk).  cadd_verify_tree reads materialised logits [batch, R, V]; this entry
 * point takes the hidden states and the weight instead and never writes the logits: the product is formed tile
 * by tile on the tensor cores (bf16 inputs, fp32 accumulation) and reduced to one token per row on the fly.
 * Outputs, tie rule (lowest token id), rows_mode and the walk are those of cadd_verify_tree.  A logit is the
 * fp32-accumulated dot product; two tokens whose exact dot products differ by less than that accumulation's
 * rounding error may be ranked either way.
 * All pointers are DEVICE pointers owned by the caller.
 */
typedef struct cadd_head_args {
    uint32_t struct_size;          /* = sizeof(cadd_head_args) */
    uint32_t flags;                /* reserved, 0 */
    int32_t  batch, L, R;
    int32_t  hidden;               /* hidden size (the contraction length), >= 1 */
    int32_t  rows_mode;            /* CADD_ROWS_*; in LIVE mode rows j > n_nodes[b] get node_argmax -1, and the product is
                                      formed for the live rows only (they are copied next to one another first) */
    int32_t  reserved0;
    int64_t  V;
    const void* hidden_states;     /* bf16 [batch, R, hidden]; element (b,j,k) at (b*R + j)*stride_row + k; 16-byte aligned */
    int64_t  stride_row;           /* in elements, >= hidden, multiple of 8 */
    const void* weight;            /* bf16 [V, hidden]; element (v,k) at v*stride_w + k; 16-byte aligned */
    int64_t  stride_w;             /* in elements, >= hidden, multiple of 8 */
    const int32_t* n_nodes;        /* [batch]   from cadd_build_tree */
    const int32_t* token_ids;      /* [batch,R] from cadd_build_tree */
    const int32_t* parent_idx;     /* [batch,R] from cadd_build_tree */
    /* outputs, all required except status */
    int32_t* node_argmax;          /* [batch,R] */
    int32_t* accepted_len;         /* [batch] */
    int32_t* accepted_nodes;       /* [batch,L], -1 padded */
    int32_t* next_bonus;           /* [batch] */
    int32_t* status;               /* [batch] CADD_STATUS_* bits, may be NULL */
    void*    workspace;            /* >= cadd_head_workspace_bytes, 256-byte aligned; needs no initialisation */
    size_t   workspace_bytes;
} cadd_head_args;

/*
 * Tree construction fused into the drafter's output projection (Eq. 1 with l_i = h_i . W^T; Algorithm 1).
 * cadd_build_tree reads materialised draft logits [batch, L, V]; this entry point takes the drafter's last hidden
 * states and the output-projection weight instead and never writes the logits: they are formed tile by tile on the
 * tensor cores (bf16 inputs, fp32 accumulation) and consumed at once by the softmax statistics and the top-K
 * selection.  Everything after that (expansion, stopping rule, emission, outputs, status bits) is cadd_build_tree's.
 * A logit is the fp32-accumulated dot product.  `build` carries all other arguments: its draft_logits, stride_b,
 * stride_l and logits_dtype are ignored, its V is the number of tokens, its workspace must hold
 * cadd_build_head_workspace_bytes.  K <= 32 on this path.
 */
typedef struct cadd_build_head_args {
    uint32_t struct_size;          /* = sizeof(cadd_build_head_args) */
    uint32_t flags;                /* reserved, 0 */
    int32_t  hidden;               /* hidden size (the contraction length) */
    int32_t  reserved0;
    const void* hidden_states;     /* bf16 [batch, L, hidden]; element (b,i,k) at (b*L + i)*stride_row + k; 16-byte aligned */
    int64_t  stride_row;           /* in elements, >= hidden, multiple of 8 */
    const void* weight;            /* bf16 [V, hidden]; element (v,k) at v*stride_w + k; 16-byte aligned */
    int64_t  stride_w;             /* in elements, >= hidden, multiple of 8 */
    cadd_build_args build;         /* struct_size = sizeof(cadd_build_args) */
} cadd_build_head_args;

/*
 * Tree verification under sampling (temperature T > 0; the paper's T = 1 tables use it but the text does not
 * define the tree variant).  The reading built here is lossless for a tree of deterministic candidates: at the
 * current node one token x is drawn from the target's distribution softmax(y / T); if a child of the node carries x
 * the walk moves there and repeats, otherwise it stops; x is the next bonus token either way.  Replace the draw by
 * the arg-max and this is cadd_verify_tree.  The random numbers are inputs: one uniform u in [0, 1) per (request,
 * row); the draw is the inverse CDF in token order, the smallest v with
 * sum_{w <= v} exp(y_w / T) > u * sum_w exp(y_w / T).  NaN and infinite logits carry no mass; a row without a finite
 * logit gives token 0.
 * All pointers are DEVICE pointers owned by the caller; no workspace is needed.
 */
typedef struct cadd_sample_args {
    uint32_t struct_size;          /* = sizeof(cadd_sample_args) */
    uint32_t flags;                /* reserved, 0 */
    int32_t  batch, L, R;
    int32_t  logits_dtype;         /* CADD_DTYPE_* */
    int32_t  rows_mode;            /* CADD_ROWS_*: LIVE draws for rows 0..n_nodes[b] only (others -1), DENSE for all R rows */
    int32_t  reserved0;
    int64_t  V;                    /* at most 650,000 (bf16) / 325,000 (fp32) elements per row */
    double   temperature;          /* T > 0 */
    const void* target_logits;     /* [batch, R, V]; element (b,j,v) at b*stride_b + j*stride_row + v */
    int64_t  stride_b, stride_row; /* in elements */
    const double* uniforms;        /* [batch, R] in [0, 1) */
    const int32_t* n_nodes;        /* [batch]   from cadd_build_tree */
    const int32_t* token_ids;      /* [batch,R] from cadd_build_tree */
    const int32_t* parent_idx;     /* [batch,R] from cadd_build_tree */
    /* outputs, all required except status */
    int32_t* node_token;           /* [batch,R] the token drawn at every row read; -1 for rows not read */
    int32_t* accepted_len;         /* [batch] */
    int32_t* accepted_nodes;       /* [batch,L], -1 padded */
    int32_t* next_bonus;           /* [batch] the token drawn at the last accepted node */
    int32_t* status;               /* [batch] CADD_STATUS_* bits, may be NULL */
} cadd_sample_args;

/*
 * Offline cost fitting (Section "Offline Cost Profiling", Eq. 12): for each of n_tables profiled context lengths,
 * the least-squares fit to N measured verification latencies (node counts equally spaced, e.g. n = 1..N) among
 * all convex, non-decreasing sequences.  The fitted rows can be passed to cadd_build_tree as cost_table (with
 * CADD_COST_TABLE or CADD_COST_TABLE_INTERP); the caller decides what C_v(0) is.
 * All pointers are DEVICE pointers owned by the caller; the call needs no workspace.
 */
#define CADD_FIT_MAX_N 2048
#define CADD_FIT_STATUS_ITERATION_CAP 1   /* the active-set iteration was cut off; the row is its last iterate */
#define CADD_FIT_STATUS_KNOT_CAP      2   /* reserved (the slope-change capacity equals CADD_FIT_MAX_N) */
typedef struct cadd_fit_args {
    uint32_t struct_size;          /* = sizeof(cadd_fit_args) */
    uint32_t flags;                /* reserved, 0 */
    int32_t  n_tables;             /* independent problems, >= 1 */
    int32_t  N;                    /* points per problem, 1 .. CADD_FIT_MAX_N */
    const double* y;               /* [n_tables, N] measurements */
    double*  fit;                  /* [n_tables, N] out: fitted values (convex, non-decreasing along N) */
    int32_t* n_breaks;             /* [n_tables] out: number of slope changes of the fit (first slope included), may be NULL */
    int32_t* status;               /* [n_tables] out: CADD_FIT_STATUS_* bits, 0 = optimal; may be NULL */
} cadd_fit_args;

/* ABI version of the loaded library (CADD_ABI_VERSION it was built with). */
int cadd_version(void);

/* Static, NUL-terminated description of a return code; never NULL, never freed. */
const char* cadd_status_string(int code);

/* Scratch sizes: pure host arithmetic on the shape fields (batch, L, K, B_max, R, V, dtype);
 * pointers in the struct are ignored.  *out (HOST) receives the byte count. */
int cadd_build_workspace_bytes(const cadd_build_args* a, size_t* out);
int cadd_verify_workspace_bytes(const cadd_verify_args* a, size_t* out);

/* Tree construction (Eq. 1, Algorithm 1, Section 3.3).  Asynchronous on `cuda_stream`: two kernels (softmax/top-K
 * over the rows, then expansion + emission), or ONE for small problems (rows of at most 2048 logits, 2 MiB of draft
 * logits in all), where the expansion kernel reads the rows itself. */
int cadd_build_tree(const cadd_build_args* a, void* cuda_stream);

/* Tree verification (Sections 3.1 and 3.3).  Asynchronous on `cuda_stream`: two kernels (arg-max of the rows, then the
 * walk), or ONE for small problems (rows of at most 8192 logits, 4 MiB of target logits in all). */
int cadd_verify_tree(const cadd_verify_args* a, void* cuda_stream);

/* Kernels the call with these arguments enqueues (pure host arithmetic on the shape fields and flags; pointers are
 * ignored): 1 or 2, or a negative CADD_ERR_* code for arguments the call itself would reject. */
int cadd_build_launches(const cadd_build_args* a);
int cadd_verify_launches(const cadd_verify_args* a);

/* Scratch size of cadd_verify_tree_fused_head: pure host arithmetic on batch, R, hidden and rows_mode (LIVE mode
 * needs room for a packed copy of the hidden states). */
int cadd_head_workspace_bytes(const cadd_head_args* a, size_t* out);

/* Tree verification from hidden states and the output-projection weight (see cadd_head_args).  Asynchronous on
 * `cuda_stream`: one memset of the workspace and three kernels.  Errors as for cadd_verify_tree; CADD_ERR_ALIGN
 * if a base pointer is not 16-byte aligned or a stride is not a multiple of 8 elements; CADD_ERR_LAUNCH if the
 * driver's tensor-map encoder is unavailable.  If an internal bounded wait runs out, every request reports
 * CADD_STATUS_INTERNAL_TIMEOUT. */
int cadd_verify_tree_fused_head(const cadd_head_args* a, void* cuda_stream);

/* Scratch size of cadd_build_tree_fused_head: pure host arithmetic on batch, L and K. */
int cadd_build_head_workspace_bytes(const cadd_build_head_args* a, size_t* out);

/* Tree construction from hidden states and the output-projection weight (see cadd_build_head_args).  Asynchronous on
 * `cuda_stream`: one small memset and three kernels.  Errors as for cadd_build_tree, plus CADD_ERR_SHAPE for K > 32,
 * CADD_ERR_ALIGN for a base pointer that is not 16-byte aligned or a stride that is not a multiple of 8 elements. */
int cadd_build_tree_fused_head(const cadd_build_head_args* a, void* cuda_stream);

/* Tree verification with one draw per node from softmax(target logits / T) (see cadd_sample_args).  Asynchronous on
 * `cuda_stream`: two kernels.  Errors as for cadd_verify_tree; CADD_ERR_SHAPE also for T <= 0 and for rows longer than
 * the stated limit. */
int cadd_verify_tree_sampled(const cadd_sample_args* a, void* cuda_stream);

/* Convex, non-decreasing least-squares fit of every row (see cadd_fit_args).  Asynchronous on `cuda_stream`: one
 * kernel, one CTA per row, fp64.  CADD_ERR_SHAPE if N > CADD_FIT_MAX_N. */
int cadd_fit_cost_tables(const cadd_fit_args* a, void* cuda_stream);

/*
 * cadd_build_tree for callers that cannot provide scratch memory.  (The paper has no counterpart to
 * this entry point; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where device allocation is off limits, for example a plugin inside a
 * serving engine that owns the whole memory pool and forbids cudaMalloc after start-up, a real-time
 * loop that must not take the allocator's locks, or a host language binding that can pass input and
 * output tensors but has no allocator of its own to size a workspace with.  Such a caller still passes
 * every input and output of cadd_build_args; the fields `workspace` and `workspace_bytes` are ignored.
 *
 * Where the scratch comes from: a fixed array of CADD_STATIC_SCRATCH_BYTES bytes that is part of the
 * library's device image.  Every GPU on which the library is used holds those bytes from first use
 * until the process ends.  The call itself allocates and frees nothing.
 *
 * Limits and rules
 *   - Problems whose cadd_build_workspace_bytes() exceeds CADD_STATIC_SCRATCH_BYTES are refused with
 *     CADD_ERR_STATIC_SCRATCH before anything is launched (8 MiB covers all five benchmark shapes,
 *     e.g. batch 256 x L 16 x K 8, or batch 64 x L 32 x K 32).
 *   - The first call on each device looks up the array's device address (a one-time, synchronous
 *     runtime query made with that device current).  Make that first call outside any CUDA stream
 *     capture; later calls only enqueue kernels.
 *   - All calls on one device share the one array.  It needs no clearing between calls (every byte a
 *     call reads was written earlier in the same call), but two calls that may run on the GPU at the
 *     same time -- different streams, or different host threads -- would overwrite each other's
 *     scratch: keep such calls on one stream or otherwise ordered.  Results are the same as those of
 *     cadd_build_tree given a private workspace.
 *   - Return codes and `status` bits otherwise as for cadd_build_tree.
 */
#define CADD_STATIC_SCRATCH_BYTES (8u << 20)
int cadd_build_tree_static_scratch(const cadd_build_args* a, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* CADD_H_ */
