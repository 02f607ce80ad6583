// Tree verification kernels: per-node argmax of the target logits and the accepted-path walk
// (greedy acceptance, Section 3.1; longest accepted prefix and next bonus token, Section 3.3).
#pragma once
#include "common.cuh"
#include "tile_ring.cuh"

namespace cadd {

struct ArgmaxParams {
    const void* logits;        // [batch, R, V]
    int64_t V, stride_b, stride_row;
    int R, rows_mode;
    int ctas_per_request;      // CTA g of a request reads rows g, g + ctas_per_request, ... (= R: one row per CTA)
    const int32_t* n_nodes;    // [batch]
    int32_t* node_argmax;      // [batch, R]
    int fault_tile;            // test hook: this tile of every row is never copied (-1: none)
};

// Shared memory of row_argmax_kernel.
struct ArgmaxRing {
    alignas(8) uint64_t full[kStages];                 // mbarriers: tile landed
    unsigned released[kStages];                        // warps done with the stage's current tile
    unsigned last_seq[kStages];                        // last tile issued into the stage (see ring_drain)
    unsigned timeout;
    float red_m[kThreads / 32];
    int64_t red_p[kThreads / 32];
    alignas(128) uint4 ring[kStages][kTileChunks];
};
inline size_t argmax_smem_bytes() { return sizeof(ArgmaxRing) + 128; }

// One CTA per (request, row) (or per few rows of a request, see ctas_per_request).  One thread streams the row's 16-byte chunks into a ring of 16 KB
// shared-memory tiles with cp.async.bulk + mbarrier (own shared memory only); the last warp to finish a tile refills
// its stage, so (kStages - 1) x 16 KB stay in flight per CTA (4 CTAs per SM) without living in registers.
// Each thread keeps the running maximum (packed bf16 max, NaN ignored) and the first position (chunk start or
// scalar element) where it was reached; the CTA reduces (value descending, position ascending) and one warp
// finds the first maximal element inside that one chunk.  HBM-bound: ~9 instructions per 16 bytes.
template <int DT>
__global__ void __launch_bounds__(kThreads, 4) row_argmax_kernel(ArgmaxParams p) {
    using E = Elem<DT>;
    grid_dependency_wait();
    grid_launch_dependents();                            // the walk kernel that follows is a handful of warps
    extern __shared__ __align__(16) unsigned char argmax_smem_raw[];
    // aligned by pointer arithmetic on the shared array itself: accesses stay shared-memory instructions
    ArgmaxRing& sh = *reinterpret_cast<ArgmaxRing*>(argmax_smem_raw + ((128u - (smem_u32(argmax_smem_raw) & 127u)) & 127u));
    // CTA g of request b takes rows g, g + ctas_per_request, ...: one row each when every row is read (DENSE), several
    // when most rows are expected to be padding (LIVE with a small node cap), so that few CTAs are launched only to exit.
    const int b = blockIdx.x / p.ctas_per_request;
    const int g = blockIdx.x - b * p.ctas_per_request;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int n = p.R - 1;
    if (p.rows_mode == CADD_ROWS_LIVE) {
        n = p.n_nodes[b];
        n = n < 0 ? 0 : (n > p.R - 1 ? p.R - 1 : n);
        if (g > n) {                                     // nothing to read for this CTA: mark its rows and leave
            for (int j = g + tid * p.ctas_per_request; j < p.R; j += kThreads * p.ctas_per_request)
                p.node_argmax[(int64_t)b * p.R + j] = -1;
            return;
        }
    }
    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) { mbar_init(&sh.full[q], 1); sh.released[q] = 0; sh.last_seq[q] = kNoTile; }
        sh.timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned st = 0, phase = 0;                          // ring position: carries on from row to row
    unsigned issued = 0;                                 // tiles issued so far (thread-uniform by construction)
    for (int j = g; j < p.R; j += p.ctas_per_request) {
        int32_t* out = p.node_argmax + (int64_t)b * p.R + j;
        if (j > n) {
            if (tid == 0) *out = -1;
            continue;
        }
        const char* row = (const char*)p.logits + ((int64_t)b * p.stride_b + (int64_t)j * p.stride_row) * E::ES;
        const RowSplit sp = split_row<DT>(row, p.V);
        const uint4* body = (const uint4*)(row + (int64_t)sp.head * E::ES);
        const int nc = sp.n_chunks;
        const int n_tiles = (nc + kTileChunks - 1) / kTileChunks;
        const unsigned base = issued;                    // stage of tile t of this row: (base + t) % kStages
        const int fault_tile = p.fault_tile < 0 ? -1 : min(p.fault_tile, n_tiles - 1);
        auto issue_tile = [&](int t) {
            if (t == fault_tile) return;                 // test hook: this copy is never made
            const int c0 = t * kTileChunks;
            const unsigned bytes = (unsigned)min(kTileChunks, nc - c0) * 16u;
            const unsigned stg = (base + (unsigned)t) % kStages;
            *(volatile unsigned*)&sh.last_seq[stg] = base + (unsigned)t;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive_expect_tx(&sh.full[stg], bytes);
            bulk_load(&sh.ring[stg][0], body + c0, bytes, &sh.full[stg]);
        };
        if (tid == 0)
            for (int t = 0; t < kStages && t < n_tiles; ++t) issue_tile(t);
        issued += (unsigned)n_tiles;

        float rm = -INFINITY;            // running maximum (NaN never enters: only strict '>' updates it)
        int64_t rpos = INT64_MAX;        // first position where rm was reached
        if (tid < sp.head) {
            float x = E::load(row, tid);
            if (x > rm) { rm = x; rpos = tid; }
        }
        for (int t = 0; t < n_tiles; ++t) {
            if (!__all_sync(kFullMask, mbar_wait_limited(&sh.full[st], phase, tile_wait_limit(t, fault_tile)))) { sh.timeout = 1; break; }
            const uint4* tile = &sh.ring[st][tid];
            const int cbase = t * kTileChunks + tid;
#pragma unroll
            for (int u = 0; u < kTopkUnroll; ++u) {
                const int c = cbase + u * kThreads;
                if (c < nc) {
                    const float cm = E::chunk_max(tile[u * kThreads]);
                    if (cm > rm) { rm = cm; rpos = sp.head + (int64_t)c * E::EPC; }
                }
            }
            __syncwarp();
            if (lane == 0 && atomicAdd(&sh.released[st], 1u) == kThreads / 32 - 1) {   // last warp refills the stage
                atomicExch(&sh.released[st], 0u);
                if (t + kStages < n_tiles) issue_tile(t + kStages);
            }
            if (++st == kStages) { st = 0; phase ^= 1u; }
        }
        if (tid < sp.tail) {
            int64_t i = p.V - sp.tail + tid;
            float x = E::load(row, i);
            if (x > rm) { rm = x; rpos = i; }
        }

        // CTA reduction of (value descending, position ascending)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float om = __shfl_xor_sync(kFullMask, rm, o);
            int64_t op = __shfl_xor_sync(kFullMask, rpos, o);
            if (om > rm || (om == rm && op < rpos)) { rm = om; rpos = op; }
        }
        if (lane == 0) { sh.red_m[warp] = rm; sh.red_p[warp] = rpos; }
        __syncthreads();
        const bool timed_out = sh.timeout != 0;
        if (tid < 32) {
            rm = tid < kThreads / 32 ? sh.red_m[tid] : -INFINITY;
            rpos = tid < kThreads / 32 ? sh.red_p[tid] : INT64_MAX;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                float om = __shfl_xor_sync(kFullMask, rm, o);
                int64_t op = __shfl_xor_sync(kFullMask, rpos, o);
                if (om > rm || (om == rm && op < rpos)) { rm = om; rpos = op; }
            }
            rm = __shfl_sync(kFullMask, rm, 0);
            rpos = __shfl_sync(kFullMask, rpos, 0);
            int32_t ans = 0;                                  // every logit is -Inf or NaN: lowest id
            if (rpos != INT64_MAX) {
                int64_t i = rpos + tid;
                bool hit = tid < E::EPC && i < p.V && E::load(row, i) == rm;
                unsigned m = __ballot_sync(kFullMask, hit);
                ans = (int32_t)(rpos + (__ffs(m) - 1));
            }
            if (timed_out) ans = -2;                          // a bulk copy never landed: the walk kernel flags the request
            if (tid == 0) *out = ans;
        }
        if (timed_out) {                                      // the ring's state is unknown: give up on this CTA's other rows too
            for (int jj = j + p.ctas_per_request + tid * p.ctas_per_request; jj < p.R; jj += kThreads * p.ctas_per_request)
                p.node_argmax[(int64_t)b * p.R + jj] = jj > n ? -1 : -2;
            if (tid == 0) ring_drain(sh.full, sh.last_seq);   // every warp is past the barrier above: let the copies in flight land
            return;
        }
        __syncthreads();                                      // red_m / red_p and the ring are free for the next row
    }
}

struct WalkParams {
    int batch, L, R;
    const int32_t* n_nodes;
    const int32_t* token_ids;
    const int32_t* parent_idx;
    const int32_t* node_argmax;
    int32_t* accepted_len;
    int32_t* accepted_nodes;   // [batch, L]
    int32_t* next_bonus;
    int32_t* status;           // may be NULL
};

// The walk of one request by one warp: from the root, move to the child whose token equals the target's argmax at
// the current node (children always have a larger row index than their parent); stop at the first miss.
__device__ __forceinline__ void accept_walk_warp(const WalkParams& p, int b) {
    const int lane = threadIdx.x & 31;
    int st = 0;
    int n = p.n_nodes[b];
    if (n < 0) { n = 0; st |= CADD_STATUS_BAD_N_NODES; }
    if (n > p.R - 1) { n = p.R - 1; st |= CADD_STATUS_BAD_N_NODES; }
    const int32_t* tok = p.token_ids + (int64_t)b * p.R;
    const int32_t* par = p.parent_idx + (int64_t)b * p.R;
    const int32_t* gmx = p.node_argmax + (int64_t)b * p.R;
    int32_t* acc = p.accepted_nodes + (int64_t)b * p.L;
    for (int i = lane; i < p.L; i += 32) acc[i] = -1;
    __syncwarp();
    for (int c = lane; c <= n; c += 32)                    // -2 marks a row whose bulk copy never landed
        if (gmx[c] == -2) st |= CADD_STATUS_INTERNAL_TIMEOUT;
    st |= __shfl_xor_sync(kFullMask, st, 16); st |= __shfl_xor_sync(kFullMask, st, 8); st |= __shfl_xor_sync(kFullMask, st, 4);
    st |= __shfl_xor_sync(kFullMask, st, 2); st |= __shfl_xor_sync(kFullMask, st, 1);
    int cur = 0, alpha = 0;
    while (alpha < p.L) {
        const int32_t g = gmx[cur];
        int child = -1;
        for (int base = cur + 1; base <= n && child < 0; base += 32) {
            int c = base + lane;
            bool hit = c <= n && par[c] == cur && tok[c] == g;
            unsigned m = __ballot_sync(kFullMask, hit);
            if (m) child = base + __ffs(m) - 1;
        }
        if (child < 0) break;
        if (lane == 0) acc[alpha] = child;
        alpha += 1;
        cur = child;
    }
    if (lane == 0) {
        p.accepted_len[b] = alpha;
        p.next_bonus[b] = gmx[cur];
        if (p.status) p.status[b] = st;
    }
}

// One warp per request.
__global__ void __launch_bounds__(128) accept_walk_kernel(WalkParams p) {
    grid_dependency_wait();
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= p.batch) return;
    accept_walk_warp(p, b);
}

// Small problems (short rows, few of them): the whole verification of a request in one CTA and one launch.  Every warp
// takes rows of the request in turn and finds the row's first maximal element by itself (lanes read elements
// lane, lane + 32, ... in ascending order, so a lane's first maximum is its lowest index; the warp reduces on
// (value descending, index ascending)); after a CTA barrier warp 0 walks the accepted path.
constexpr int kVerifySmallThreads = 512;
template <int DT>
__global__ void __launch_bounds__(kVerifySmallThreads) verify_small_kernel(ArgmaxParams p, WalkParams wp) {
    using E = Elem<DT>;
    grid_dependency_wait();
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int n = p.R - 1;
    if (p.rows_mode == CADD_ROWS_LIVE) {
        n = p.n_nodes[b];
        n = n < 0 ? 0 : (n > p.R - 1 ? p.R - 1 : n);
    }
    for (int j = warp; j < p.R; j += kVerifySmallThreads / 32) {
        int32_t* out = p.node_argmax + (int64_t)b * p.R + j;
        if (j > n) {
            if (lane == 0) *out = -1;
            continue;
        }
        const char* row = (const char*)p.logits + ((int64_t)b * p.stride_b + (int64_t)j * p.stride_row) * E::ES;
        float rm = -INFINITY;            // running maximum (NaN never enters: only strict '>' updates it)
        int64_t rpos = INT64_MAX;        // first position where rm was reached
        for (int64_t i = lane; i < p.V; i += 32) {
            const float x = E::load(row, i);
            if (x > rm) { rm = x; rpos = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(kFullMask, rm, o);
            const int64_t op = __shfl_xor_sync(kFullMask, rpos, o);
            if (om > rm || (om == rm && op < rpos)) { rm = om; rpos = op; }
        }
        if (lane == 0) *out = rpos == INT64_MAX ? 0 : (int32_t)rpos;      // every logit is -Inf or NaN: lowest id
    }
    __syncthreads();
    if (warp == 0) accept_walk_warp(wp, b);
}

}  // namespace cadd
