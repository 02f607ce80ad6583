// Best-first expansion of the candidate tree with the greedy throughput stopping rule, and emission
// of the tree arrays and the ancestor mask (Algorithm 1; Eq. 5-7, Eq. 11, Corollary 1; Section 3.3).
//
// One CTA of ten warps per request: eight prepare the lists, one pops, one evaluates.
//   phase 0  eight warps, one half-warp per position: merge the softmax/top-K records of each live position (candidate
//            keys in no order, plus the mass of everything else as pairs W * 2^C) into the sorted top-K list (token,
//            a = logit - row max) and log Z, all in fp64.  (Small problems: there are no records, one warp per position
//            reads the short row itself.)  Meanwhile the evaluating warp turns the cost model into a table C_v(0..B_max),
//            and both it and the popping warp go once through their loops on a made-up node, so that the loops' code is
//            in the SM's caches when the lists are ready.
//   phase 1  popping warp: running log-partition sums S_d and the reachable depth
//   phase 2  popping warp: the best 32 entries of the frontier (Algorithm 1's heap) sit in the warp's registers, sorted
//            over the lanes on a 96-bit key (score, then depth / token / parent packed in 32 bits); what does not fit
//            waits, unsorted, in a shared-memory pool whose best key is tracked.  A pop takes lane 0's entry; the popped
//            node's next sibling and first child enter by two ballots (how many entries stay ahead of each) and one
//            gathering shuffle.
//            evaluating warp: follows through the node table; exp(sigma), Phi and the throughput test of one node after
//            the other (past the first 64: of up to 32 nodes at a time, one per lane); the first failing test fixes n*
//            and stops the popping warp.  The pop order does not depend on the cost model, so this yields exactly
//            Algorithm 1's tree.
//   phase 3  all threads: write token / parent / depth / position / log-prob rows and padding; zero
//            the mask rows with coalesced stores, then one thread per node walks its ancestors and
//            writes the few non-zero words (bytes for the dense form).
#pragma once
#include "common.cuh"
#include "softmax_topk.cuh"

namespace cadd {

struct ExpandParams {
    int batch, L, K, KP, S, B_max, R;
    int rec_fmt;               // records at `partials`: kRecSegRecord (softmax_topk_partial_kernel) or kRecSegPartial (draft_merge_kernel);
                               // kRecDirect: no records, the kernel reads the (short) rows of logits itself
    const void* logits;        // kRecDirect: [batch, L, V]
    int64_t V, stride_b, stride_l;
    int logits_dtype;
    uint32_t flags;
    const unsigned char* partials;
    const int32_t* l_eff;
    const int32_t* bonus_token;
    const int32_t* ctx_len;
    int cost_kind;
    const double* cost_coef;
    const double* cost_table;
    const int32_t* table_idx;
    const double* t_draft;
    const int32_t* ctx_grid;
    int n_tables;
    int32_t* n_nodes;
    int32_t* token_ids;
    int32_t* parent_idx;
    int32_t* depth;
    int32_t* position_ids;
    double* node_logprob;
    double* phi;
    double* theta;
    double* theta_curve;
    uint32_t* mask_bits;
    uint8_t* mask_dense;
    int32_t* topk_token;
    double* topk_logprob;
    int32_t* status;
};

constexpr int kRecSegPartial = 0, kRecSegRecord = 1, kRecDirect = 2;
// candidate keys a record of the given format holds at most
__host__ __device__ inline int rec_key_cap(int rec_fmt, int KP) { return rec_fmt == kRecSegRecord ? seg_key_cap(KP) : (rec_fmt == kRecDirect ? 0 : KP); }

constexpr int kEvalOneByOne = 64;          // nodes the evaluating warp takes one at a time before it turns to batches
constexpr int kLateStopPops = 24;          // pops that look at the stop flag a second time, at their end
constexpr int kEvalPollLimit = 1 << 20;    // polls of one node's score word before the evaluating warp gives up (tens of milliseconds)
constexpr int kMergeWarps = 8;             // sixteen half-warps: one per draft position in the merge phase for L <= 16
constexpr int kExpandWarps = kMergeWarps + 2;      // and the two warps of the expansion proper
constexpr int kExpandThreads = kExpandWarps * 32;

// A frontier entry / node besides its score, in 30 bits, most significant first: depth - 1 (6 bits), the token's place
// among the tokens of its position's top-K list in token-id order (6 bits), parent row (12 bits), rank - 1 in the
// list (6 bits).  Between entries of equal score a SMALLER word comes first: that is (depth, token id, parent row) in this
// order, because two entries of one depth compare their tokens like the tokens' places; the rank never decides (depth,
// token and parent already identify a node).
__device__ __forceinline__ uint32_t pack_meta(int depth, int place, int parent, int rank) {
    return ((uint32_t)(depth - 1) << 24) | ((uint32_t)place << 18) | ((uint32_t)parent << 6) | (uint32_t)(rank - 1);
}
__device__ __forceinline__ int me_depth(uint32_t me) { return (int)(me >> 24) + 1; }
__device__ __forceinline__ int me_parent(uint32_t me) { return (int)((me >> 6) & 0xfffu); }
__device__ __forceinline__ int me_rank(uint32_t me) { return (int)(me & 0x3fu) + 1; }

// Dynamic shared memory layout of the expansion kernel (byte offsets), same arithmetic on host and device.
struct ExpandLayout {
    size_t a_list, lz, S, nHi, nMe, nA, cv, region, tok_list, keff, place, total;
    int pool_cap;      // entries of the frontier's pool
};
// kRecDirect: bytes of shared memory for one staged row (the row, the up to 15 bytes before it back to a 16-byte boundary,
// rounded up to whole 16-byte pieces)
__host__ __device__ inline size_t direct_row_bytes(int64_t V, int dtype) { return (((size_t)V * (dtype == CADD_DTYPE_BF16 ? 2 : 4)) + 31) & ~(size_t)15; }
__host__ __device__ inline ExpandLayout expand_layout(int L, int K, int key_cap, int S, int B_max, size_t row_bytes) {
    ExpandLayout o;
    const size_t NR = (size_t)B_max + 2;                         // rows 0..B_max, and one that the trial pass writes
    // every pop takes one entry out of the frontier and puts at most two in
    o.pool_cap = B_max + 2;
    size_t frontier = (size_t)o.pool_cap * (8 + 4);
    size_t scratch = (size_t)kMergeWarps * 2 * S * key_cap * 8;     // phase 0: every key of a row's records, per warp
    size_t region = frontier > scratch ? frontier : scratch;
    if ((size_t)kMergeWarps * row_bytes > region) region = (size_t)kMergeWarps * row_bytes;   // kRecDirect: a staged row per warp
    region = (region + 15) & ~(size_t)15;
    size_t p = 0;
    o.a_list = p;   p += ((size_t)L + 1) * K * 8;                 // one row more than there are positions: indices one past
                                                                 // a list's or the tree's end stay inside (what they read is never used)
    o.lz = p;       p += (size_t)L * 8;
    o.S = p;        p += ((size_t)L + 2) * 8;
    o.nHi = p;      p += NR * 8;
    o.nMe = p;      p += ((NR * 4) + 7) & ~(size_t)7;
    o.nA = p;       p += NR * 8;
    o.cv = p;       p += NR * 8;
    p = (p + 15) & ~(size_t)15;
    o.region = p;   p += region;
    o.tok_list = p; p += ((size_t)L + 1) * K * 4;
    o.keff = p;     p += ((size_t)L + 2) * 4;
    o.place = p;    p += ((size_t)L + 2) * K + 8;               // (the last array: room for the reads one past a list's end and
                                                                 // for the rank the trial pass may make up)
    o.total = (p + 15) & ~(size_t)15;
    return o;
}

// The verification cost C_v(n) of one request: quadratic, one table row, or two table rows blended by
// context length (Eq. 13).
struct CostModel {
    int kind;
    double q[4];            // QUADRATIC: (C_d, a, b, c)
    const double* row0;     // TABLE: the row; TABLE_INTERP: the row of L_j
    const double* row1;     // TABLE_INTERP: the row of L_{j+1}
    double alpha;           // TABLE_INTERP
};
__device__ __forceinline__ double cost_verify(const CostModel& cm, int n) {
    if (cm.kind == CADD_COST_TABLE) return cm.row0[n];
    if (cm.kind == CADD_COST_TABLE_INTERP) return (1.0 - cm.alpha) * cm.row0[n] + cm.alpha * cm.row1[n];
    const double x = (double)n;
    return cm.q[1] + cm.q[2] * x + cm.q[3] * (x * x);
}

__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// Small problems (a few thousand logits per row): one warp turns one row into the sorted top-K list and log Z by itself
// (Eq. 1; Algorithm 1, Require).  The row comes to shared memory in one round trip and is read there twice:
//   first pass   every lane's largest finite key (and with it the row maximum m), the number of finite logits, flags
//   bound        the K-th largest of the 32 lanes' maxima: at least K keys are at or above it, so the K best are
//   second pass  every key at or above the bound goes to a candidate list (a handful for most rows); the mass of all
//                others is summed as fp32 exponentials against the reference exponent ceil(m * log2e) + 1, in fp64
//   selection    the candidates are ranked by counting (keys are unique); the K best go through the fp64 exponential, as
//                on the large path, the others join the mass
// For K above 32, or if the candidates do not fit, the K best are taken one after the other instead (each the largest
// key below the one before: K more passes).  NaN and infinities carry no mass and are flagged.
constexpr int kDirectCandCap = 256;
__host__ __device__ inline size_t direct_stage_bytes(int64_t V, int dtype) { return direct_row_bytes(V, dtype) + (size_t)kDirectCandCap * 8; }

template <int DT>
__device__ __forceinline__ void row_lists_warp(const void* grow, unsigned char* buf, int64_t V, int K, int32_t* tok_out, double* a_out,
                                               double* logZ_out, int32_t* keff_out, uint32_t* flags_out) {
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    // whole 16-byte pieces from the boundary at or below the row's start
    const size_t lead = (size_t)((uintptr_t)grow & 15);
    const char* g0 = (const char*)grow - lead;
    const int pieces = (int)((lead + (size_t)V * (DT == CADD_DTYPE_BF16 ? 2 : 4) + 15) >> 4);
    for (int c = lane; c < pieces; c += 32) cp_async16(buf + 16 * c, g0 + 16 * (size_t)c);
    cp_async_wait_all();
    __syncwarp();
    const void* row = buf + lead;
    uint64_t* cand = (uint64_t*)(buf + direct_row_bytes(V, DT));

    // (four elements per turn in both passes, each with its own running values: one warp is alone with this row, and
    // what it waits for is its own previous instruction)
    uint64_t mine = 0;                                       // this lane's largest finite key (0: none)
    uint32_t fl = 0;
    int nfin = 0;
    {
        uint64_t best[4] = {0ull, 0ull, 0ull, 0ull};
        for (int64_t i0 = lane; i0 < V; i0 += 128) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t i = i0 + 32 * u;
                const float x = i < V ? E::load(row, i) : -INFINITY;
                const uint32_t b = __float_as_uint(x);
                const bool fin = (b & 0x7f800000u) != 0x7f800000u;
                if (!fin && i < V) {
                    if (b != 0xff800000u) fl |= kPartNonfinite;
                    if (b == 0x7f800000u) fl |= kPartPosInf;
                }
                const uint64_t key = fin ? make_key(x, (uint32_t)i) : 0ull;
                best[u] = max(best[u], key);
                nfin += fin ? 1 : 0;
            }
        }
        mine = max(max(best[0], best[1]), max(best[2], best[3]));
    }
    nfin = __reduce_add_sync(kFullMask, nfin);
    fl = __reduce_or_sync(kFullMask, fl);
    const int ke = nfin < K ? nfin : K;
    uint64_t top = mine;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) top = max(top, __shfl_xor_sync(kFullMask, top, o));
    const float m = nfin > 0 ? key_value(top) : -INFINITY;
    const float negc = m > -INFINITY ? -(ceilf(fminf(m, 2.0e38f) * kLog2eHi) + 1.0f) : 0.0f;
    double acc = 0.0;
    bool listed = false;
    if (K <= 32) {
        // the K-th largest of the lanes' maxima (0 if fewer lanes than that hold a finite logit: then everything is listed)
        uint64_t bound = top, left = mine == top ? 0ull : mine;
        for (int r = 1; r < K; ++r) {
            uint64_t nx = left;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) nx = max(nx, __shfl_xor_sync(kFullMask, nx, o));
            bound = nx;
            if (left == nx) left = 0ull;
        }
        int nc = 0;
        for (int64_t i0 = 0; i0 < V; i0 += 128) {
            float part[4];
            bool is_cand[4];
            uint64_t key[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t i = i0 + 32 * u + lane;
                const float x = i < V ? E::load(row, i) : INFINITY;
                const bool fin = fabsf(x) < INFINITY;
                key[u] = fin ? make_key(x, (uint32_t)i) : 0ull;
                is_cand[u] = fin && key[u] >= bound;
                part[u] = exp2_term((fin && !is_cand[u]) ? x : -INFINITY, negc);      // 2^-inf = 0
            }
            acc += (double)((part[0] + part[1]) + (part[2] + part[3]));
            if (__any_sync(kFullMask, is_cand[0] || is_cand[1] || is_cand[2] || is_cand[3])) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const unsigned cm = __ballot_sync(kFullMask, is_cand[u]);
                    if (is_cand[u]) {
                        const int at = nc + __popc(cm & ((1u << lane) - 1u));
                        if (at < kDirectCandCap) cand[at] = key[u];
                    }
                    nc += __popc(cm);
                }
            }
        }
        __syncwarp();
        if (nc <= kDirectCandCap) {
            listed = true;
            for (int q = lane; q < nc; q += 32) {
                const uint64_t k = cand[q];
                int rank = 0;
                for (int r = 0; r < nc; ++r) rank += cand[r] > k;
                if (rank < K) { tok_out[rank] = (int32_t)key_id(k); a_out[rank] = (double)key_value(k) - (double)m; }
                else acc += (double)exp2_term(key_value(k), negc);
            }
        }
    }
    if (!listed) {
        acc = 0.0;
        uint64_t prev = ~0ull;                               // above every key
        for (int r = 0; r < ke; ++r) {
            uint64_t best = 0;
            for (int64_t i = lane; i < V; i += 32) {
                const float x = E::load(row, i);
                if (fabsf(x) < INFINITY) {
                    const uint64_t key = make_key(x, (uint32_t)i);
                    if (key < prev && key > best) best = key;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(kFullMask, best, o));
            if (lane == 0) { tok_out[r] = (int32_t)key_id(best); a_out[r] = (double)key_value(best) - (double)m; }
            prev = best;
        }
        for (int64_t i = lane; i < V; i += 32) {
            const float x = E::load(row, i);
            if (fabsf(x) < INFINITY && (ke == 0 || make_key(x, (uint32_t)i) < prev)) acc += (double)exp2_term(x, negc);
        }
    }
    __syncwarp();
    double zsum = lane < ke ? exp(a_out[lane]) : 0.0;
    for (int r = lane + 32; r < ke; r += 32) zsum += exp(a_out[r]);
    if (acc != 0.0) zsum += acc * kEx2BiasFix * exp((double)(-negc) * 0.6931471805599453094 - (double)m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) zsum += __shfl_xor_sync(kFullMask, zsum, o);
    if (lane == 0) { *logZ_out = log(zsum); *keff_out = ke; *flags_out = fl; }
    __syncwarp();
}

// Barrier 1 of the CTA: every warp arrives once, the merging warps when their lists are complete, the popping and the
// evaluating warp before their real pass.
__device__ __forceinline__ void lists_ready_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kExpandThreads) : "memory"); }

// The evaluating warp on a large tree: whatever has been popped since the last look, up to 32 nodes at a time, one per
// lane: the exponentials and the divisions side by side, so that this warp keeps ahead of the popping warp whatever that
// one's pace; Phi is still summed in node order (every lane adds up its own prefix).  Takes over at node es.j with es.n
// nodes accepted; returns when the stopping rule fires (end & 1), the popping warp is through, or a wait ran out (end & 2).
struct EvalState { double Phi, theta_prev; int j, n, st, end; };
__device__ __noinline__ EvalState evaluate_in_batches(EvalState es, const uint64_t* nHi, const double* cv, double* theta_curve_row,
                                                      int B_max, double C_d, bool fixed, int* s_stop, int* s_pop_done) {
    const int lane = threadIdx.x & 31;
    int polls = 0;
    while (es.j <= B_max) {
        const int jj = es.j + lane;
        uint64_t sw = jj <= B_max ? *(volatile const uint64_t*)&nHi[jj] : 0ull;
        unsigned have = __ballot_sync(kFullMask, sw != 0ull);
        if ((have & 1u) == 0u) {
            if (!*(volatile int*)s_pop_done) {
                if (++polls > kEvalPollLimit) { es.end |= 2; break; }
                continue;
            }
            __threadfence_block();
            sw = jj <= B_max ? *(volatile const uint64_t*)&nHi[jj] : 0ull;   // the popping warp is through: what is there now is final
            have = __ballot_sync(kFullMask, sw != 0ull);
            if ((have & 1u) == 0u) break;
        }
        polls = 0;
        const int g = have == 0xffffffffu ? 32 : __ffs(~have) - 1;      // the nodes that are there form a prefix
        const bool act = lane < g;
        const double delta = act ? exp(unord64(sw)) : 0.0;
        double Phi_l = es.Phi;
        for (int i = 0; i < g; ++i) {
            const double di = __shfl_sync(kFullMask, delta, i);
            if (i <= lane) Phi_l += di;
        }
        const double den = act ? C_d + cv[jj] : 1.0;
        const bool bad = !(den > 0.0);
        const double theta_l = (1.0 + Phi_l) / den;
        double theta_before = __shfl_up_sync(kFullMask, theta_l, 1);
        if (lane == 0) theta_before = es.theta_prev;
        const unsigned sm = __ballot_sync(kFullMask, act && (bad || (!fixed && theta_l <= theta_before)));
        const int f = sm ? __ffs(sm) - 1 : g;                           // nodes j .. j + f - 1 are accepted
        if (sm && lane == 0) *(volatile int*)s_stop = 1;
        if (theta_curve_row && lane < f) theta_curve_row[jj] = theta_l;
        if (f > 0) {
            es.Phi = __shfl_sync(kFullMask, Phi_l, f - 1);
            es.theta_prev = __shfl_sync(kFullMask, theta_l, f - 1);
        }
        es.n += f; es.j += f;
        if (sm) {
            if (__shfl_sync(kFullMask, (int)bad, f)) es.st |= CADD_STATUS_COST_NONPOSITIVE;
            es.end |= 1;
            break;
        }
    }
    return es;
}

// The pool's turn (rare): finds the pool's best entry under the order of the frontier (lanes scan stripes of the pool, then
// a butterfly), takes it out (the last entry fills its slot) and finds the new best.  Out of line: the usual pop should
// not carry this code.
struct PoolTake { uint64_t qhi, pmax_hi; uint32_t qme, pmax_me; };   // the entry taken, and the pool's best after it
__device__ __noinline__ PoolTake pool_take_best(uint64_t* pHi, uint32_t* pMe, int pn) {   // pn: entries before the call (one fewer after)
    const int lane = threadIdx.x & 31;
    auto before = [](uint64_t ahi, uint32_t ame, uint64_t bhi, uint32_t bme) { return (bool)((int)(ahi > bhi) | ((int)(ahi == bhi) & (int)(ame < bme))); };
    __syncwarp();
    uint64_t bhi = 0;
    uint32_t bme = 0;
    int bi = -1;
    for (int q = lane; q < pn; q += 32) {
        const uint64_t hi = pHi[q];
        const uint32_t me = pMe[q];
        if (before(hi, me, bhi, bme)) { bhi = hi; bme = me; bi = q; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t ohi = __shfl_xor_sync(kFullMask, bhi, o);
        const uint32_t ome = __shfl_xor_sync(kFullMask, bme, o);
        const int oi = __shfl_xor_sync(kFullMask, bi, o);
        if (before(ohi, ome, bhi, bme)) { bhi = ohi; bme = ome; bi = oi; }
    }
    PoolTake out;
    out.qhi = bhi;
    out.qme = bme;
    --pn;
    __syncwarp();
    if (bi != pn) { const uint64_t lhi = pHi[pn]; const uint32_t lme = pMe[pn]; __syncwarp(); pHi[bi] = lhi; pMe[bi] = lme; }
    __syncwarp();
    bhi = 0; bme = 0;
    for (int q = lane; q < pn; q += 32) {
        const uint64_t hi = pHi[q];
        const uint32_t me = pMe[q];
        if (before(hi, me, bhi, bme)) { bhi = hi; bme = me; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t ohi = __shfl_xor_sync(kFullMask, bhi, o);
        const uint32_t ome = __shfl_xor_sync(kFullMask, bme, o);
        if (before(ohi, ome, bhi, bme)) { bhi = ohi; bme = ome; }
    }
    out.pmax_hi = bhi; out.pmax_me = bme;
    return out;
}

// kDirect: the kernel for p.rec_fmt == kRecDirect (its own instantiation, so that neither carries the other's phase 0)
template <bool kDirect>
__global__ void __launch_bounds__(kExpandThreads, 2) expand_emit_kernel(ExpandParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int key_cap = rec_key_cap(p.rec_fmt, p.KP);
    const ExpandLayout lay = expand_layout(p.L, p.K, key_cap, p.S, p.B_max, kDirect ? direct_stage_bytes(p.V, p.logits_dtype) : 0);
    double* a_list = (double*)(smem + lay.a_list);
    double* lz = (double*)(smem + lay.lz);
    double* Sd = (double*)(smem + lay.S);
    uint64_t* nHi = (uint64_t*)(smem + lay.nHi);          // ordered image of the node's score sigma
    uint32_t* nMe = (uint32_t*)(smem + lay.nMe);          // pack_meta(depth, parent row, rank)
    int32_t* tok_list = (int32_t*)(smem + lay.tok_list);
    int32_t* keff = (int32_t*)(smem + lay.keff);          // keff[d], d = 1..L
    uint8_t* place = smem + lay.place;                    // of each listed token among its list's tokens, by token id
    double* nA = (double*)(smem + lay.nA);                // the node's sum of (logit - row max) along its path
    double* cv = (double*)(smem + lay.cv);                // C_v(n), n = 0..B_max
    uint64_t* pHi = (uint64_t*)(smem + lay.region);       // the frontier's pool (see phase 2), in no order
    uint32_t* pMe = (uint32_t*)(pHi + lay.pool_cap);

    __shared__ int s_status, s_pinf, s_n;
    __shared__ int s_cost_ok, s_pop_done, s_stop, s_fsize_end;   // between the popping warp and the evaluating warp
    __shared__ double s_phi, s_theta, s_theta0;

    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = p.L, K = p.K, R = p.R, B_max = p.B_max;
    int clamped;
    int Le = clamp_l_eff(p.l_eff, b, L, &clamped);         // (not written by the kernel before this one: read at once)
    asm volatile("" : "+r"(Le));                          // a register from here on: never read from memory again
    if (tid == 0) { s_status = 0; s_pinf = 0; s_pop_done = 0; s_stop = 0; s_fsize_end = 0; s_cost_ok = 0; }
    for (int d = tid; d < L + 2; d += kExpandThreads) keff[d] = 0;
    for (int j = tid; j <= B_max + 1; j += kExpandThreads) nHi[j] = 0;   // "not popped yet" (see phase 2)
    __syncthreads();
    if (tid == 0 && clamped) atomicOr(&s_status, CADD_STATUS_L_EFF_CLAMPED);
    // (used by the emission only; read here so that the emission does not start with a trip to DRAM)
    const int ctx = p.ctx_len ? p.ctx_len[b] : 0;
    const int bonus = p.bonus_token ? p.bonus_token[b] : -1;

    const int kPopWarp = kMergeWarps;                       // the last warp evaluates
    if (warp < kMergeWarps) {
    // ---------------- phase 0: the sorted top-K list and log Z of every live position ----------------
    grid_dependency_wait();                                 // the records are the previous kernel's
    const bool emit = (p.flags & CADD_FLAG_EMIT_TOPK) != 0;
    if constexpr (kDirect) {
        // small problem: there are no records, one warp per position reads the (short) row itself
        for (int i = warp; i < L; i += kMergeWarps) {
            int32_t* out_tok = p.topk_token ? p.topk_token + ((int64_t)b * L + i) * K : nullptr;
            double* out_lp = p.topk_logprob ? p.topk_logprob + ((int64_t)b * L + i) * K : nullptr;
            if (i >= Le) {
                if (emit) for (int k = lane; k < K; k += 32) {
                    if (out_tok) out_tok[k] = -1;
                    if (out_lp) out_lp[k] = -INFINITY;
                }
                continue;
            }
            const size_t es = p.logits_dtype == CADD_DTYPE_BF16 ? 2 : 4;
            const char* row = (const char*)p.logits + ((int64_t)b * p.stride_b + (int64_t)i * p.stride_l) * (int64_t)es;
            unsigned char* stage = smem + lay.region + (size_t)warp * direct_stage_bytes(p.V, p.logits_dtype);
            uint32_t fl;
            if (p.logits_dtype == CADD_DTYPE_BF16) row_lists_warp<CADD_DTYPE_BF16>(row, stage, p.V, K, tok_list + i * K, a_list + i * K, &lz[i], &keff[i + 1], &fl);
            else row_lists_warp<CADD_DTYPE_FP32>(row, stage, p.V, K, tok_list + i * K, a_list + i * K, &lz[i], &keff[i + 1], &fl);
            fl = __shfl_sync(kFullMask, fl, 0);
            const int ke = keff[i + 1];
            for (int k = lane; k < ke; k += 32) {
                const int t = tok_list[i * K + k];
                int c = 0;
                for (int q = 0; q < ke; ++q) c += tok_list[i * K + q] < t;
                place[i * K + k] = (uint8_t)c;
            }
            if (lane == 0) {
                int st = 0;
                if (fl & kPartNonfinite) st |= CADD_STATUS_NONFINITE_INPUT;
                if (ke < K) st |= CADD_STATUS_FEWER_THAN_K_FINITE;
                if (st) atomicOr(&s_status, st);
                if (fl & kPartPosInf) s_pinf = 1;
            }
            if (emit) for (int k = lane; k < K; k += 32) {
                if (out_tok) out_tok[k] = k < ke ? tok_list[i * K + k] : -1;
                if (out_lp) out_lp[k] = k < ke ? a_list[i * K + k] - lz[i] : -INFINITY;
            }
        }
    } else {
    // Merge of the softmax/top-K records, one HALF-warp per position (a row's records hold a few dozen keys and at most
    // sixteen headers).  A record lists candidate keys (a superset of the K best of its part of the row) and one or more
    // pairs (W, C) with the mass of everything else as W * 2^C.  All keys of the row are ranked by counting (they are
    // unique); every listed key's exponential is taken in fp64.  Every key slot of the row's records is copied to shared
    // memory asynchronously and the headers and first sums are read in the same round trip; what a record does not use
    // is dropped afterwards.  Shuffles below move data within a half only (offsets below 16, or an explicit lane).
    const bool seg_records = p.rec_fmt == kRecSegRecord;
    const size_t pstride = seg_records ? seg_record_stride(p.KP) : seg_partial_stride(p.KP);
    const size_t keys_at = seg_records ? sizeof(SegRecord) + (size_t)kSegSums * 16 : sizeof(SegPartial);
    const int slots = p.S * key_cap;                        // at most 512, and at most 16 records
    const int n_pairs = seg_records ? p.S * kSegSums : p.S; // (W, C) pairs of a row
    const int hl = lane & 15, half = lane >> 4, lane0 = half << 4;
    for (int i0 = 2 * warp; i0 < L; i0 += 2 * kMergeWarps) {
        const int i = i0 + half;                            // this half-warp's position
        const bool has_row = i < L;
        const int ii = has_row ? i : L - 1;                 // (addresses stay inside the arrays; nothing of it is kept)
        int32_t* out_tok = p.topk_token ? p.topk_token + ((int64_t)b * L + ii) * K : nullptr;
        double* out_lp = p.topk_logprob ? p.topk_logprob + ((int64_t)b * L + ii) * K : nullptr;
        uint64_t* scr = (uint64_t*)(smem + lay.region) + (size_t)(2 * warp + half) * slots;
        const unsigned char* rec0 = p.partials + ((size_t)((int64_t)b * L + ii) * p.S) * pstride;
        for (int s = 0; s < p.S; ++s) {
            const uint64_t* keys = (const uint64_t*)(rec0 + (size_t)s * pstride + keys_at);
            for (int q = hl; q < key_cap; q += 16) cp_async8(&scr[s * key_cap + q], keys + q);
        }
        // lane s of the half reads the header of record s, lane t the row's pair t (pair t % 8 of record t / 8)
        int my_cnt = 0, my_ns = 0;
        uint32_t my_fl = 0;
        double W0 = 0.0, C0 = 0.0;
        if (seg_records) {
            if (hl < p.S) {
                const int4 h = *(const int4*)(rec0 + (size_t)hl * pstride);
                my_cnt = h.x; my_fl = (uint32_t)h.y; my_ns = h.z;
            }
            if (hl < n_pairs) {
                const double2 wc = *(const double2*)(rec0 + (size_t)(hl / kSegSums) * pstride + sizeof(SegRecord) + (size_t)(hl % kSegSums) * 16);
                W0 = wc.x; C0 = wc.y;
            }
        } else if (hl < p.S) {
            const SegPartial* h = (const SegPartial*)(rec0 + (size_t)hl * pstride);
            my_cnt = h->cnt; my_fl = h->flags; my_ns = 1;
            W0 = h->W; C0 = h->C;
        }
        cp_async_wait_all();
        __syncwarp();
        const bool live = has_row && i < Le;                // a masked position: whatever its records hold is not looked at
        my_cnt = live ? min(max(my_cnt, 0), key_cap) : 0;
        uint32_t fl = live ? my_fl : 0u;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) fl |= __shfl_xor_sync(kFullMask, fl, o);
        // keep the slots that are in use, in place (a batch of 16 is read before its survivors are written below it)
        int n = 0;
        for (int s = 0; s < p.S; ++s) {
            const int cnt_s = __shfl_sync(kFullMask, my_cnt, lane0 + s);
            for (int q0 = 0; q0 < key_cap; q0 += 16) {
                const int q = q0 + hl;
                const bool valid = q < cnt_s;                   // (cnt_s <= key_cap)
                const uint64_t key = valid ? scr[s * key_cap + q] : 0ull;
                const unsigned m = (__ballot_sync(kFullMask, valid) >> lane0) & 0xffffu;
                __syncwarp();
                if (valid) scr[n + __popc(m & ((1u << hl) - 1u))] = key;
                n += __popc(m);
            }
        }
        __syncwarp();
        uint64_t mk = 0;
        for (int q = hl; q < n; q += 16) mk = max(mk, scr[q]);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) mk = max(mk, __shfl_xor_sync(kFullMask, mk, o));
        const double m = (double)key_value(mk);
        // This lane's terms of Z: its keys (ranked by counting on the way), then its pair of the mass outside the lists,
        // one (W, C) per record or per warp of the CTA that wrote it -- all through one exponential, so that its code is
        // there once.  (A warp's W can be negative: the warp that takes a candidate's term out of the sums need not be the
        // one that added it; only the total over a record's warps is a sum of terms.)
        const int ns0 = __shfl_sync(kFullMask, my_ns, lane0 + ((seg_records ? hl / kSegSums : hl) & 15));
        const bool used0 = live && hl < n_pairs && (seg_records ? hl % kSegSums < ns0 : true);
        // ranks by counting, four of this lane's keys against each key of the row at a time (one load serves four compares)
        for (int q0 = hl; q0 < n; q0 += 64) {
            uint64_t key[4];
            int rank[4] = {0, 0, 0, 0};
#pragma unroll
            for (int u = 0; u < 4; ++u) key[u] = q0 + 16 * u < n ? scr[q0 + 16 * u] : ~0ull;   // (nothing is above ~0: no rank, no store)
            for (int r = 0; r < n; ++r) {
                const uint64_t v = scr[r];
#pragma unroll
                for (int u = 0; u < 4; ++u) rank[u] += v > key[u] ? 1 : 0;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (q0 + 16 * u < n && rank[u] < K) {
                    tok_list[i * K + rank[u]] = (int32_t)key_id(key[u]);
                    a_list[i * K + rank[u]] = (double)key_value(key[u]) - m;
                }
        }
        const int nk = n > hl ? (n - hl + 15) >> 4 : 0;        // keys of this lane
        double zsum = 0.0;
        for (int k = 0; k <= nk; ++k) {
            double arg, w;
            if (k < nk) {
                arg = (double)key_value(scr[hl + 16 * k]) - m; w = 1.0;
            } else {
                arg = C0 * 0.6931471805599453094 - m; w = used0 ? W0 : 0.0;
            }
            if (w != 0.0) zsum += w * exp(arg);
        }
        for (int t0 = 16; t0 < n_pairs; t0 += 16) {             // (more than two records to a row: rare)
            const int t = t0 + hl;
            const int rec = seg_records ? t / kSegSums : t;
            const int ns = __shfl_sync(kFullMask, my_ns, lane0 + (rec & 15));
            double W = 0.0, C = 0.0;
            if (seg_records && t < n_pairs) {
                const double2 wc = *(const double2*)(rec0 + (size_t)rec * pstride + sizeof(SegRecord) + (size_t)(t % kSegSums) * 16);
                W = wc.x; C = wc.y;
            }
            const bool used = live && t < n_pairs && (seg_records ? t % kSegSums < ns : false);
            if (used && W != 0.0) zsum += W * exp(C * 0.6931471805599453094 - m);
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) zsum += __shfl_xor_sync(kFullMask, zsum, o);
        const double logZ = log(zsum);
        const int ke = n < K ? n : K;
        __syncwarp();
        for (int k = hl; k < ke; k += 16) {
            const int t = tok_list[i * K + k];
            int c = 0;
            for (int q = 0; q < ke; ++q) c += tok_list[i * K + q] < t;
            place[i * K + k] = (uint8_t)c;
        }
        if (hl == 0 && live) {
            keff[i + 1] = ke;
            lz[i] = logZ;
            int st = 0;
            if (fl & kPartNonfinite) st |= CADD_STATUS_NONFINITE_INPUT;
            if (fl & kPartTimeout) { st |= CADD_STATUS_INTERNAL_TIMEOUT; s_pinf = 1; }   // nothing is known of the row: empty tree
            else if (ke < K) st |= CADD_STATUS_FEWER_THAN_K_FINITE;
            if (st) atomicOr(&s_status, st);
            if (fl & kPartPosInf) s_pinf = 1;
        }
        if (emit && has_row) for (int k = hl; k < K; k += 16) {
            if (out_tok) out_tok[k] = (live && k < ke) ? tok_list[i * K + k] : -1;
            if (out_lp) out_lp[k] = (live && k < ke) ? a_list[i * K + k] - logZ : -INFINITY;
        }
    }
    }
    lists_ready_barrier();
    }
    // ---------------- phase 2: the pop loop (one warp) and the throughput tests (another) ----------------
    // The popping warp pops; the evaluating warp follows it through the node table, taking exp(sigma), the prefix sums
    // Phi and the throughput tests of whatever has been popped since it last looked, up to 32 nodes at a time, one per
    // lane.  The first failing test fixes n* and tells the popping warp to stop.  The pop order does not depend on the
    // cost model, so what is popped beyond n* (as many nodes as fit into one evaluation's latency) is simply left unused.
    // While the lists are being merged both warps go once through their loops on a made-up node (row B_max + 1 of the
    // node table, nothing of it is kept): a trial pass that brings the loops' instructions into the SM's caches, since a
    // CTA of this kernel lives for some tens of microseconds and its first pops would otherwise wait for their code.
    else if (warp == kPopWarp) {
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            const bool trial = pass == 0;
            if (!trial) lists_ready_barrier();
            // phase 1: running log-partition sums S_d (each lane adds up its own prefix, in position order) and the
            // reachable depth (the trial pass does the same on whatever the arrays hold)
            int Lr = Le;
            for (int d0 = 0; d0 < Le; d0 += 32) {
                const int d = d0 + lane + 1;
                double acc = 0.0;
                for (int i = 0; i < Le; ++i) {                     // (the same trip count for every lane)
                    const double v = lz[i];
                    if (i < d) acc += v;
                }
                if (d <= Le) Sd[d] = acc;
                const unsigned z = __ballot_sync(kFullMask, d <= Le && keff[d] == 0);   // positions without a finite logit
                if (z != 0 && Lr == Le) Lr = d0 + __ffs(z) - 1;
            }
            if (lane == 0) Sd[0] = 0.0;
            bool ok = *(volatile int*)&s_cost_ok != 0 && *(volatile int*)&s_pinf == 0;
            if (trial) { ok = true; Lr = 1; }
            nA[0] = 0.0;
            nHi[0] = ord64(0.0); nMe[0] = 0u;
            __syncwarp();
            // The frontier (Algorithm 1's heap) in two parts.  The WINDOW is its best entries, at most 32, sorted best
            // first over the lanes of the warp: lane i holds the i-th best as the ordered image of its score and a 32-bit
            // word (depth, place of its token, parent row, rank: see pack_meta); a score word of 0 is an empty lane (no
            // score's image is 0).  Entry A comes before entry B if its score word is larger or, at equal scores, its second
            // word is smaller: the total order (score, depth, token id, parent row).  The POOL, in shared memory and in no
            // order, holds what did not fit: an entry goes there only if the window is full and all of its entries are
            // better, or by falling off the window's end; (pmax_hi, pmax_me) is the pool's best.  A pop takes the window's
            // head unless the pool's best comes before it.  In the usual case (the head is popped) the window changes once
            // per pop: the head leaves and the node's next sibling and first child enter, each lane taking its new entry
            // from its old one or a neighbour's according to two ballots on the old window.  The parent's sum A is read
            // from the node table instead of travelling with the entry.  All lanes hold the same scalars and write the same
            // values to the node table and the pool, so a lane only ever reads back what it has written itself.
            uint64_t whi = 0;                                   // this lane's window entry
            uint32_t wme = 0;
            int pn = 0;                                         // entries in the pool
            uint64_t pmax_hi = 0;
            uint32_t pmax_me = 0;
            // (bitwise on purpose: three comparisons and two logic operations, no branch)
            auto before = [](uint64_t ahi, uint32_t ame, uint64_t bhi, uint32_t bme) { return (bool)((int)(ahi > bhi) | ((int)(ahi == bhi) & (int)(ame < bme))); };
            auto to_pool = [&](uint64_t khi, uint32_t kme) {
                pHi[pn] = khi; pMe[pn] = kme;
                if (before(khi, kme, pmax_hi, pmax_me)) { pmax_hi = khi; pmax_me = kme; }
                ++pn;
            };
            // a new entry joins the frontier (the general form: any state of the window, full comparisons)
            auto push = [&](uint64_t khi, uint32_t kme) {
                const int pos = __popc(__ballot_sync(kFullMask, before(whi, wme, khi, kme)));   // window entries that stay ahead of it
                if (pos >= 32) {                                // a full window of better entries: to the pool
                    to_pool(khi, kme);
                    return;
                }
                const uint64_t lhi = __shfl_sync(kFullMask, whi, 31);     // a full window: its last entry makes room
                const uint32_t lme = __shfl_sync(kFullMask, wme, 31);
                if (lhi != 0ull) to_pool(lhi, lme);
                const uint64_t uhi = __shfl_up_sync(kFullMask, whi, 1);
                const uint32_t ume = __shfl_up_sync(kFullMask, wme, 1);
                if (lane > pos) { whi = uhi; wme = ume; }
                else if (lane == pos) { whi = khi; wme = kme; }
            };
            if (trial) push(ord64(-1.0), pack_meta(1, 0, 0, 1));
            else if (ok && Lr >= 1)                             // Algorithm 1, line 3: the heap starts with node (1)
                push(ord64(a_list[0] - Sd[1]), pack_meta(1, place[0], 0, 1));
            const int limit = !ok ? 0 : (trial ? 1 : B_max);
            const int jbase = trial ? B_max + 1 : 1;               // row of the first popped node

            int popped = 0;
            int stop_now = 0;
            // What a pop reads about its node: fetched as soon as the node is known, which for the usual pop is before the
            // previous pop has finished with the window (the next head is the window's second entry or the better
            // successor), so that the loads are under way while the window is put in order.
            struct NodeIn { double Apar, a_cur, a_sib, a_chi, S_d, S_c; int keff_d; uint32_t pl_sib, pl_chi; };
            auto load_node = [&](uint32_t kme) {
                const int d = me_depth(kme), par = me_parent(kme), r = me_rank(kme);
                const double* arow = a_list + (d - 1) * K;
                NodeIn in;
                in.Apar = nA[par];
                in.a_cur = arow[r - 1];
                // (the next sibling and the first child are read whether they exist or not: the arrays have room)
                in.a_sib = arow[r]; in.a_chi = a_list[d * K];
                in.S_d = Sd[d]; in.S_c = Sd[d + 1];
                in.keff_d = keff[d];
                // (six bits each: what the trial pass reads here is whatever the memory holds, and must stay in its field)
                in.pl_sib = place[(d - 1) * K + r] & 63u; in.pl_chi = place[d * K] & 63u;
                return in;
            };
            // The popped node (khi, kme) becomes row j: its score word at once (the evaluating warp waits for it), then
            // its two successors (Algorithm 1, lines 12-19): a is the better one (equal scores: the sibling, which is
            // less deep), b the other; a missing one is all zero.
            auto node_and_successors = [&](uint64_t khi, uint32_t kme, const NodeIn& in, int j, uint64_t& ahi, uint32_t& ame, uint64_t& bhi, uint32_t& bme) {
                const int d = me_depth(kme), r = me_rank(kme);
                *(volatile uint64_t*)&nHi[j] = khi;
                const bool has_sib = r < in.keff_d;
                const bool has_child = d < Lr;
                const double A = in.Apar + in.a_cur;
                nA[j] = A;
                nMe[j] = kme;
                // (both are computed whether they exist or not and masked afterwards: no branch)
                const uint64_t ms = 0ull - (uint64_t)has_sib, mc = 0ull - (uint64_t)has_child;
                const uint64_t shi = ord64((in.Apar + in.a_sib) - in.S_d) & ms;
                const uint32_t sme = ((kme & 0x3f03ffc0u) | (in.pl_sib << 18) | (uint32_t)r) & (uint32_t)ms;   // same depth and parent, next rank
                const uint64_t chi = ord64((A + in.a_chi) - in.S_c) & mc;
                const uint32_t cme = (((uint32_t)d << 24) | (in.pl_chi << 18) | ((uint32_t)j << 6)) & (uint32_t)mc;   // pack_meta(d + 1, place, j, 1)
                const bool sib_first = shi >= chi;
                ahi = sib_first ? shi : chi; bhi = sib_first ? chi : shi;
                ame = sib_first ? sme : cme; bme = sib_first ? cme : sme;
            };
            uint64_t khi = __shfl_sync(kFullMask, whi, 0);          // the window's head, and what its pop will read
            uint32_t kme = __shfl_sync(kFullMask, wme, 0);
            NodeIn in = load_node(kme);
            // (the frontier is empty when the window's head is and the pool holds nothing)
            while (popped < limit && (khi != 0ull || pn != 0) && !stop_now) {
                const int j = popped + jbase;
                ++popped;
                if (before(pmax_hi, pmax_me, khi, kme)) {
                    // Rare: the pool holds the best entry (always, if the window is empty).  Find it (lanes scan stripes
                    // of the pool, then a butterfly), take it out, find the pool's new best; the node's successors enter
                    // one after the other.
                    const PoolTake took = pool_take_best(pHi, pMe, pn);
                    --pn;
                    pmax_hi = took.pmax_hi; pmax_me = took.pmax_me;
                    const uint64_t qhi = took.qhi;
                    const uint32_t qme = took.qme;
                    uint64_t ahi, b2hi;
                    uint32_t ame, b2me;
                    node_and_successors(qhi, qme, load_node(qme), j, ahi, ame, b2hi, b2me);
                    if (ahi != 0ull) push(ahi, ame);
                    if (b2hi != 0ull) push(b2hi, b2me);
                    stop_now = *(volatile int*)&s_stop;
                    khi = __shfl_sync(kFullMask, whi, 0);
                    kme = __shfl_sync(kFullMask, wme, 0);
                    in = load_node(kme);
                    continue;
                }
                const uint64_t o1hi = __shfl_sync(kFullMask, whi, 1);      // the window's second entry: the next head unless a is
                const uint32_t o1me = __shfl_sync(kFullMask, wme, 1);
                uint64_t ahi, bhi;
                uint32_t ame, bme;
                node_and_successors(khi, kme, in, j, ahi, ame, bhi, bme);
                stop_now = *(volatile int*)&s_stop;                     // looked at when this pop is over
                // The head leaves, a and b enter; a missing one lands on the first empty lane.  Old entries ahead of a move up
                // one lane, those between a and b stay, those behind b move down one: one gathering shuffle.  Every successor
                // is behind its node in the order, so the head counts in both ballots.
                // the new head is the window's second entry unless a comes before it (known without the ballots); its
                // loads go out now
                const bool second_stays = before(o1hi, o1me, ahi, ame);
                khi = second_stays ? o1hi : ahi;
                kme = second_stays ? o1me : ame;
                in = load_node(kme);
                const int pa = __popc(__ballot_sync(kFullMask, before(whi, wme, ahi, ame))) - 1;
                const int pb = __popc(__ballot_sync(kFullMask, before(whi, wme, bhi, bme)));
                const int src = lane + (lane < pa ? 1 : 0) - (lane > pb ? 1 : 0);      // whose old entry this lane takes
                const uint64_t ghi = __shfl_sync(kFullMask, whi, src);
                const uint32_t gme = __shfl_sync(kFullMask, wme, src);
                // 33 entries: the one that does not fit (b, if all 32 old entries come before it, else the window's last)
                // goes to the pool; written without a branch, the stress regime spills on every pop
                const uint64_t lhi = __shfl_sync(kFullMask, whi, 31);
                const uint32_t lme = __shfl_sync(kFullMask, wme, 31);
                const bool spill = lhi != 0ull && bhi != 0ull;          // a full window and two new entries
                const uint64_t xhi = pb == 32 ? bhi : lhi;
                const uint32_t xme = pb == 32 ? bme : lme;
                if (spill) { pHi[pn] = xhi; pMe[pn] = xme; }
                const bool new_best = (bool)((int)spill & (int)before(xhi, xme, pmax_hi, pmax_me));
                pmax_hi = new_best ? xhi : pmax_hi;
                pmax_me = new_best ? xme : pmax_me;
                pn += spill ? 1 : 0;
                whi = lane == pa ? ahi : (lane == pb ? bhi : ghi);
                wme = lane == pa ? ame : (lane == pb ? bme : gme);
                // On the first pops the flag is read once more at the very end: the verdict on this pop's node arrives about
                // now, and a small tree should not pay for a pop it does not need.  (Later the wait for this load would
                // cost more than the occasional extra pop.)
                if (popped <= kLateStopPops) stop_now |= *(volatile int*)&s_stop;
            }
            __syncwarp();
            if (!trial && lane == 0) { s_fsize_end = (khi != 0ull ? 1 : 0) + pn; __threadfence_block(); *(volatile int*)&s_pop_done = 1; }
        }
    } else {
        // the cost model of this request as a table: C_v(n) for every n the tree can reach, and the draft cost C_d
        CostModel cm;
        cm.kind = p.cost_kind; cm.row0 = cm.row1 = nullptr; cm.alpha = 0.0;
        cm.q[0] = cm.q[1] = cm.q[2] = cm.q[3] = 0.0;
        double C_d;
        int st = 0;
        bool ok = true;
        if (p.cost_kind == CADD_COST_QUADRATIC) {
            for (int c = 0; c < 4; ++c) cm.q[c] = p.cost_coef[(int64_t)b * 4 + c];
            C_d = cm.q[0];
        } else if (p.cost_kind == CADD_COST_TABLE) {
            int ti = p.table_idx[b];
            if (ti < 0 || ti >= p.n_tables) {               // no such table: flagged, empty tree, nothing of it is read
                st |= CADD_STATUS_BAD_TABLE_IDX;
                ok = false;
                ti = 0;
            }
            cm.row0 = p.cost_table + (int64_t)ti * (B_max + 1);
            C_d = p.t_draft[b];
        } else {                                            // Eq. 13: the two profiled context lengths around l
            const int l = p.ctx_len ? p.ctx_len[b] : 0;
            int jlo = 0;
            while (jlo + 1 < p.n_tables && p.ctx_grid[jlo + 1] <= l) ++jlo;
            int jhi = jlo + 1 < p.n_tables ? jlo + 1 : jlo;
            if (l <= p.ctx_grid[0]) jlo = jhi = 0;
            cm.row0 = p.cost_table + (int64_t)jlo * (B_max + 1);
            cm.row1 = p.cost_table + (int64_t)jhi * (B_max + 1);
            cm.alpha = jhi == jlo ? 0.0 : ((double)l - (double)p.ctx_grid[jlo]) / ((double)p.ctx_grid[jhi] - (double)p.ctx_grid[jlo]);
            C_d = p.t_draft[b];
        }
        for (int n0 = lane; n0 <= B_max; n0 += 32 * 16) {       // (sixteen loads in flight: the rows may come from DRAM)
            double v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = n0 + 32 * u <= B_max ? cost_verify(cm, n0 + 32 * u) : 0.0;
#pragma unroll
            for (int u = 0; u < 16; ++u) if (n0 + 32 * u <= B_max) cv[n0 + 32 * u] = v[u];
        }
        if (lane == 0) cv[B_max + 1] = 1.0;
        __syncwarp();
        const double den0 = C_d + cv[0];
        double theta_first = 0.0;                               // theta*(0) as the stopping rule sees it
        if (ok && !(den0 > 0.0)) { st |= CADD_STATUS_COST_NONPOSITIVE; ok = false; }
        else theta_first = 1.0 / den0;
        const double theta0 = (den0 > 0.0) ? 1.0 / den0 : 0.0;
        const bool fixed = (p.flags & CADD_FLAG_FIXED_BUDGET) != 0;
        if (lane == 0) *(volatile int*)&s_cost_ok = ok ? 1 : 0;          // (ahead of the barrier the popping warp waits at)

        int n = 0;
        double Phi = 0.0, theta_prev = theta_first;
        bool stopped = false, gave_up = false;
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
            const bool trial = pass == 0;
            if (!trial) {
                lists_ready_barrier();
                if (*(volatile int*)&s_pinf) ok = false;
            }
            n = 0; Phi = 0.0; theta_prev = theta_first; stopped = false;
            // The first nodes one after the other, as soon as a node's score word is there (no score's ordered image is
            // zero); every lane does the same arithmetic, so nothing has to be exchanged and the verdict on a node is out
            // within a pop.  (Small trees end here.)
            int j = trial ? B_max + 1 : 1;
            int polls = 0;                                          // looks at a score word that was not there yet
            while ((ok || trial) && !stopped) {
                uint64_t sw;
                if (trial) sw = ord64(-1.0);
                else {
                    if (j > B_max || j > kEvalOneByOne) break;          // the cap (every node was worth its cost), or the batches' turn
                    sw = *(volatile uint64_t*)&nHi[j];
                    if (sw == 0ull) {
                        if (!*(volatile int*)&s_pop_done) {             // not popped yet
                            // (the popping warp waits for nobody and a pop is some hundred cycles; the limit is there so
                            // that no wait in this library is without one)
                            if (++polls > kEvalPollLimit) { gave_up = true; break; }
                            continue;
                        }
                        __threadfence_block();
                        sw = *(volatile uint64_t*)&nHi[j];              // the popping warp is through: what is there now is final
                        if (sw == 0ull) break;
                    }
                }
                polls = 0;
                const double Phi_j = Phi + exp(unord64(sw));
                const double den = C_d + cv[j];
                const bool bad = !(den > 0.0);
                const double theta_j = (1.0 + Phi_j) / den;
                const bool stop = bad || (!fixed && theta_j <= theta_prev);
                if (trial) break;
                if (stop) {
                    if (lane == 0) *(volatile int*)&s_stop = 1;         // the popping warp need not go on
                    if (bad) st |= CADD_STATUS_COST_NONPOSITIVE;
                    stopped = true;
                } else {
                    if (p.theta_curve && lane == 0) p.theta_curve[(int64_t)b * R + j] = theta_j;   // theta*(n) of every accepted n (Prop. 1)
                    Phi = Phi_j; theta_prev = theta_j;
                    n = j;
                    ++j;
                }
            }
            // A large tree goes on in batches (out of line: small trees never get there).
            if (!trial && ok && !stopped && !gave_up && j <= B_max) {
                const EvalState es = evaluate_in_batches(EvalState{Phi, theta_prev, j, n, st, 0}, nHi, cv, p.theta_curve ? p.theta_curve + (int64_t)b * R : nullptr,
                                                         B_max, C_d, fixed, &s_stop, &s_pop_done);
                Phi = es.Phi; theta_prev = es.theta_prev; j = es.j; n = es.n; st = es.st;
                stopped = (es.end & 1) != 0; gave_up = (es.end & 2) != 0;
            }
        }
        if (gave_up) {                                              // flagged, empty tree; the popping warp is told to stop
            if (lane == 0) *(volatile int*)&s_stop = 1;
            st = CADD_STATUS_INTERNAL_TIMEOUT;
            n = 0; Phi = 0.0; theta_prev = theta_first;
        } else if (ok && !stopped) {
            // the loop above only ends this way after it has seen the flag set (or at the cap, a pop or two before it is)
            for (int q = 0; !*(volatile int*)&s_pop_done && q < kEvalPollLimit; ++q) __nanosleep(40);
            st |= (*(volatile int*)&s_fsize_end == 0) ? CADD_STATUS_FRONTIER_EXHAUSTED : CADD_STATUS_CAP_HIT;
        }
        if (lane == 0) {
            s_n = n; s_phi = Phi; s_theta = theta_prev; s_theta0 = theta0;
            if (st) atomicOr(&s_status, st);
        }
    }
    __syncthreads();
    // ---------------- phase 3: emission ----------------
    const int n = s_n;
    if (tid == 0) {
        p.n_nodes[b] = n;
        if (p.phi) p.phi[b] = s_phi;
        if (p.theta) p.theta[b] = s_theta;
        if (p.status) p.status[b] = s_status;
        if (p.theta_curve) p.theta_curve[(int64_t)b * R] = s_theta0;
    }
    if (p.theta_curve)
        for (int j = n + 1 + tid; j < R; j += kExpandThreads) p.theta_curve[(int64_t)b * R + j] = 0.0;
    for (int j = tid; j < R; j += kExpandThreads) {
        const int64_t o = (int64_t)b * R + j;
        int t = -1, par = -1, d = 0, pos = 0;
        double lp = 0.0;
        if (j == 0) { t = bonus; pos = ctx; }
        else if (j <= n) {
            const uint32_t me = nMe[j];
            d = me_depth(me); par = me_parent(me); t = tok_list[(d - 1) * K + me_rank(me) - 1]; pos = ctx + d; lp = unord64(nHi[j]);
        }
        p.token_ids[o] = t;
        p.parent_idx[o] = par;
        p.depth[o] = d;
        if (p.position_ids) p.position_ids[o] = pos;
        if (p.node_logprob) p.node_logprob[o] = lp;
    }
    const bool dense = (p.flags & CADD_FLAG_EMIT_DENSE_MASK) && p.mask_dense;
    const int W = (R + 31) >> 5;
    // all rows zero first (16 bytes per store between the ragged ends), then the few non-zero words / bytes of the live rows
    auto zero_bytes = [&](unsigned char* base, int64_t total) {
        int64_t head = (16 - (int64_t)((uintptr_t)base & 15)) & 15;
        if (head > total) head = total;
        const int64_t chunks = (total - head) >> 4;
        if (tid < head) base[tid] = 0;
        uint4* mid = (uint4*)(base + head);
        for (int64_t q = tid; q < chunks; q += kExpandThreads) mid[q] = make_uint4(0u, 0u, 0u, 0u);
        for (int64_t q = head + chunks * 16 + tid; q < total; q += kExpandThreads) base[q] = 0;
    };
    if (p.mask_bits) zero_bytes((unsigned char*)(p.mask_bits + (int64_t)b * R * W), (int64_t)R * W * 4);
    if (dense) zero_bytes(p.mask_dense + (int64_t)b * R * R, (int64_t)R * R);
    __syncthreads();
    for (int j = tid; j <= n; j += kExpandThreads) {              // self and ancestors: at most L+1 bits, rows descending
        uint32_t* wrow = p.mask_bits ? p.mask_bits + ((int64_t)b * R + j) * W : nullptr;
        uint8_t* brow = dense ? p.mask_dense + ((int64_t)b * R + j) * R : nullptr;
        int cur = j, word = j >> 5;
        uint32_t acc = 0;
        for (;;) {
            acc |= 1u << (cur & 31);
            if (brow) brow[cur] = 1;
            if (cur == 0) break;
            const int next = me_parent(nMe[cur]);
            if ((next >> 5) != word) {
                if (wrow) wrow[word] = acc;
                acc = 0;
                word = next >> 5;
            }
            cur = next;
        }
        if (wrow) wrow[word] = acc;
    }
}

}  // namespace cadd
