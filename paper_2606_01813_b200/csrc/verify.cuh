// Tree verification kernels: per-node argmax of the target logits and the accepted-path walk
// (greedy acceptance, Section 3.1; longest accepted prefix and next bonus token, Section 3.3).
#pragma once
#include "common.cuh"

namespace cadd {

struct ArgmaxParams {
    const void* logits;        // [batch, R, V]
    int64_t V, stride_b, stride_row;
    int R, rows_mode;
    const int32_t* n_nodes;    // [batch]
    int32_t* node_argmax;      // [batch, R]
};

constexpr int kArgmaxUnroll = 4;   // 16-byte loads in flight per thread

// One CTA per (request, row): stream the row once, keep per thread the running maximum and the
// first position (chunk start or scalar element) where it was reached, reduce over the CTA, then
// find the first maximal element inside that one chunk.  HBM-bound: 9 instructions per 16 bytes.
template <int DT>
__global__ void __launch_bounds__(kThreads) row_argmax_kernel(ArgmaxParams p) {
    using E = Elem<DT>;
    const int b = blockIdx.x / p.R;
    const int j = blockIdx.x - b * p.R;
    const int tid = threadIdx.x;
    int32_t* out = p.node_argmax + (int64_t)b * p.R + j;
    if (p.rows_mode == CADD_ROWS_LIVE) {
        int n = p.n_nodes[b];
        n = n < 0 ? 0 : (n > p.R - 1 ? p.R - 1 : n);
        if (j > n) {
            if (tid == 0) *out = -1;
            return;
        }
    }
    const char* row = (const char*)p.logits + ((int64_t)b * p.stride_b + (int64_t)j * p.stride_row) * E::ES;
    const RowSplit sp = split_row<DT>(row, p.V);

    float rm = -INFINITY;            // running maximum (NaN never enters: only strict '>' updates it)
    int64_t rpos = INT64_MAX;        // first position where rm was reached
    if (tid < sp.head) {
        float x = E::load(row, tid);
        if (x > rm) { rm = x; rpos = tid; }
    }
    const uint4* body = (const uint4*)(row + (int64_t)sp.head * E::ES);
    const int nc = sp.n_chunks;
    int c = tid;
    for (; c + (kArgmaxUnroll - 1) * kThreads < nc; c += kArgmaxUnroll * kThreads) {
        uint4 w[kArgmaxUnroll];
#pragma unroll
        for (int u = 0; u < kArgmaxUnroll; ++u) w[u] = ld_stream16(body + c + u * kThreads);
#pragma unroll
        for (int u = 0; u < kArgmaxUnroll; ++u) {
            float cm = E::chunk_max(w[u]);
            if (cm > rm) { rm = cm; rpos = sp.head + (int64_t)(c + u * kThreads) * E::EPC; }
        }
    }
    for (; c < nc; c += kThreads) {
        float cm = E::chunk_max(ld_stream16(body + c));
        if (cm > rm) { rm = cm; rpos = sp.head + (int64_t)c * E::EPC; }
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
    __shared__ float s_m[kThreads / 32];
    __shared__ int64_t s_p[kThreads / 32];
    if ((tid & 31) == 0) { s_m[tid >> 5] = rm; s_p[tid >> 5] = rpos; }
    __syncthreads();
    if (tid < 32) {
        rm = tid < kThreads / 32 ? s_m[tid] : -INFINITY;
        rpos = tid < kThreads / 32 ? s_p[tid] : INT64_MAX;
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
            float om = __shfl_xor_sync(kFullMask, rm, o);
            int64_t op = __shfl_xor_sync(kFullMask, rpos, o);
            if (om > rm || (om == rm && op < rpos)) { rm = om; rpos = op; }
        }
        rm = __shfl_sync(kFullMask, rm, 0);
        rpos = __shfl_sync(kFullMask, rpos, 0);
        // first element equal to the maximum within the EPC elements starting at rpos
        int32_t ans = 0;                                  // every logit is -Inf or NaN: lowest id
        if (rpos != INT64_MAX) {
            int64_t i = rpos + tid;
            bool hit = tid < E::EPC && i < p.V && E::load(row, i) == rm;
            unsigned m = __ballot_sync(kFullMask, hit);
            ans = (int32_t)(rpos + (__ffs(m) - 1));
        }
        if (tid == 0) *out = ans;
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

// One warp per request: from the root, move to the child whose token equals the target's argmax at
// the current node (children always have a larger row index than their parent); stop at the first miss.
__global__ void __launch_bounds__(128) accept_walk_kernel(WalkParams p) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= p.batch) return;
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

}  // namespace cadd
