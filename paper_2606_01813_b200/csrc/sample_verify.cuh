// Tree verification under sampling (temperature T > 0).  The paper reports T = 1 results (its Section 5 tables) but
// does not spell the tree variant out; the reading built here is the lossless scheme for a tree of deterministic
// candidates (the drafter's top-K tokens are not samples): at the current node, draw ONE token x from the target's
// distribution softmax(y / T); if a child of the node carries x, move there and repeat, otherwise stop; x is the
// next token either way.  The emitted sequence is distributed exactly as the target's own sampling, whatever the
// tree.  With the draws replaced by the arg-max this is Section 3.1's greedy verification.
//
// The random numbers are inputs: one uniform u in [0, 1) per (request, row).  The draw is the inverse CDF in token
// order: the smallest v with  sum_{w <= v} exp(y_w / T)  >  u * sum_w exp(y_w / T)  (a token without mass is never drawn).
//
// One streaming pass per row (same bulk-copy ring as row_argmax_kernel).  A row is cut into runs of kRunElems
// consecutive elements; each warp owns the runs at its offset in every tile and leaves, per run, the run's maximum m
// and the sum of exp((y - m) / T) (fp32 ex2.approx terms, fp64 sums).  After the pass one warp combines the runs
// (global maximum, total, prefix in token order), finds the run that holds the crossing and scans that run's
// elements once more (2 KB, still in L2).
#pragma once
#include "common.cuh"
#include "tile_ring.cuh"
#include "verify.cuh"
#include "softmax_topk.cuh"     // packed fp32x2 helpers, ex2_approx

namespace cadd {

constexpr int kMaxRuns = 640;                                 // runs per row kept in shared memory (V up to 650k bf16 / 325k fp32 elements);
                                                              // sized so that four CTAs fit in an SM's shared memory

struct SampleParams {
    const void* logits;        // [batch, R, V]
    int64_t V, stride_b, stride_row;
    int R, rows_mode;
    int ctas_per_request;      // row_sample_shared_rows_kernel: CTA g of a request reads rows g, g + ctas_per_request, ...
    float c;                   // log2(e) / T
    const int32_t* n_nodes;    // [batch]
    const double* uniforms;    // [batch, R]
    int32_t* node_token;       // [batch, R]
    int fault_tile;            // test hook: this tile of every row is never copied (-1: none)
};

struct SampleShared {
    alignas(8) uint64_t full[kStages];
    unsigned released[kStages];
    unsigned last_seq[kStages];           // last tile issued into the stage (see ring_drain)
    unsigned timeout;
    int n_runs;
    float run_ref[kMaxRuns];              // per run: reference exponent = fp32(max * log2(e) / T) over its finite elements; -Inf if none
    double run_s[kMaxRuns];               // per run: sum of 2^(y * log2(e) / T - reference)
    alignas(128) uint4 ring[kStages][kTileChunks];
};
inline size_t sample_smem_bytes() { return sizeof(SampleShared) + 128; }

// Combine step of row_sample_kernel, run by one warp once the row's runs are in shared memory.  Kept out of line so
// that its registers (a lane's 32 terms of the crossing run) do not weigh on the streaming loop.
// Everything is in "run units": an element's mass inside run r is the very term the streaming pass summed,
// ex2(y * c - ref_r), and the run's weight in the row is s_r * 2^(ref_r - M) with M the largest reference.
template <int DT>
__device__ __noinline__ int32_t sample_combine(SampleShared& sh, int n_runs, float c, double u, const char* row, RowSplit sp,
                                               const uint4* body, int64_t V) {
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const int nc = sp.n_chunks;
    const int nr = min(n_runs, kMaxRuns);
    float M = -INFINITY;
    for (int r = lane; r < nr; r += 32) M = fmaxf(M, sh.run_ref[r]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFullMask, M, o));
    int32_t ans = 0;                                           // no finite logit at all: token 0, as the arg-max does
    if (M > -INFINITY) {
        // weights of the runs relative to M (kept in place of the sums); prefix in token order, 32 runs per step
        double Z = 0.0;
        for (int r = lane; r < nr; r += 32) {
            const float ref = sh.run_ref[r];
            const double wgt = ref > -INFINITY ? sh.run_s[r] * (double)ex2_approx((float)((double)ref - (double)M)) : 0.0;
            sh.run_s[r] = wgt;
            Z += wgt;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(kFullMask, Z, o);
        __syncwarp();
        const double target = u * Z;
        double before = 0.0;                                   // mass of the runs before the current block of 32
        int hit_run = -1;
        double hit_before = 0.0;
        for (int r0 = 0; r0 < nr && hit_run < 0; r0 += 32) {
            const int r = r0 + lane;
            const double wgt = r < nr ? sh.run_s[r] : 0.0;
            double incl = wgt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(kFullMask, incl, o);
                if (lane >= o) incl += up;
            }
            const unsigned cross = __ballot_sync(kFullMask, wgt > 0.0 && before + incl > target);
            if (cross) {
                const int l = __ffs(cross) - 1;
                hit_run = r0 + l;
                hit_before = before + __shfl_sync(kFullMask, incl - wgt, l);
            }
            before += __shfl_sync(kFullMask, incl, 31);
        }
        bool take_last = false;                                // rounding left the target a hair above the total:
        if (hit_run < 0) {                                     // the last element with mass of the last run with mass
            for (int r = nr - 1; r >= 0 && hit_run < 0; --r)
                if (sh.run_s[r] > 0.0) hit_run = r;
            take_last = true;
        }
        const float ref = sh.run_ref[hit_run];
        // mass wanted inside the run, in the run's own units
        const double need = take_last ? 1e300 : (target - hit_before) / (double)ex2_approx((float)((double)ref - (double)M));
        // ---- the elements of that run in token order: consecutive elements per lane, the streaming pass's terms ----
        constexpr int EPL = (kRunChunks / 32) * E::EPC;        // elements per lane in a body run: 32 (bf16) / 16 (fp32)
        float tm[EPL];
        int64_t e0;                                            // token of this lane's first element
        if (hit_run == 0 || hit_run == n_runs - 1) {           // scalar head / tail: one element per lane
            const int cnt = hit_run == 0 ? sp.head : sp.tail;
            e0 = (hit_run == 0 ? 0 : V - sp.tail) + lane;
#pragma unroll
            for (int q = 0; q < EPL; ++q) tm[q] = 0.0f;
            if (lane < cnt) {
                const float x = E::load(row, e0);
                if (fabsf(x) < INFINITY) tm[0] = ex2_approx(fmaf(x, c, -ref));
            }
        } else {
            const int rc0 = (hit_run - 1) * kRunChunks;        // first chunk of the run
            e0 = sp.head + ((int64_t)rc0 + lane * (kRunChunks / 32)) * E::EPC;
#pragma unroll
            for (int u = 0; u < kRunChunks / 32; ++u) {
                const int cidx = rc0 + lane * (kRunChunks / 32) + u;
                float f[E::EPC];
                if (cidx < nc) E::unpack(body[cidx], f);
#pragma unroll
                for (int q = 0; q < E::EPC; ++q)
                    tm[u * E::EPC + q] = (cidx < nc && fabsf(f[q]) < INFINITY) ? ex2_approx(fmaf(f[q], c, -ref)) : 0.0f;
            }
        }
        double mine = 0.0;
#pragma unroll
        for (int q = 0; q < EPL; ++q) mine += (double)tm[q];
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(kFullMask, incl, o);
            if (lane >= o) incl += up;
        }
        unsigned cross = __ballot_sync(kFullMask, mine > 0.0 && incl > need);
        if (!cross) cross = 0x80000000u >> __clz(__ballot_sync(kFullMask, mine > 0.0) | 1u);   // the last lane with mass
        const int l = __ffs(cross) - 1;
        double acc = incl - mine;                              // mass before this lane's elements
        int pick = -1, last = 0;
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            acc += (double)tm[q];
            if (tm[q] > 0.0f) {
                last = q;
                if (pick < 0 && acc > need) pick = q;
            }
        }
        ans = (int32_t)(e0 + (pick >= 0 ? pick : last));
        ans = __shfl_sync(kFullMask, ans, l);
    }
    return ans;
}

// One row of row_sample_kernel: streams the row through the ring (whose position st / phase and tile count `issued`
// carry on from the caller's previous row), leaves the runs in shared memory and lets warp 0 draw the token.
// Returns false if a wait ran out (the row then reads -2 and the ring must not be used again).
template <int DT>
__device__ __forceinline__ bool sample_one_row(SampleShared& sh, const SampleParams& p, int b, int j, unsigned& st, unsigned& phase,
                                               unsigned& issued) {
    using E = Elem<DT>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* out = p.node_token + (int64_t)b * p.R + j;
    const char* row = (const char*)p.logits + ((int64_t)b * p.stride_b + (int64_t)j * p.stride_row) * E::ES;
    const RowSplit sp = split_row<DT>(row, p.V);
    const uint4* body = (const uint4*)(row + (int64_t)sp.head * E::ES);
    const int nc = sp.n_chunks;
    const int n_tiles = (nc + kTileChunks - 1) / kTileChunks;
    // runs in token order: run 0 = the scalar head (if any), then the 2 KB runs of the body, then the scalar tail
    const int body_runs = (nc + kRunChunks - 1) / kRunChunks;
    const int n_runs = 1 + body_runs + 1;

    const unsigned base = issued;                        // stage of tile t of this row: (base + t) % kStages
    issued += (unsigned)n_tiles;
    const int fault_tile = p.fault_tile < 0 ? -1 : min(p.fault_tile, n_tiles - 1);
    auto issue_tile = [&](int t) {
        if (t == fault_tile) return;                     // test hook: this copy is never made
        const int c0 = t * kTileChunks;
        const unsigned bytes = (unsigned)min(kTileChunks, nc - c0) * 16u;
        const unsigned st = (base + (unsigned)t) % kStages;
        *(volatile unsigned*)&sh.last_seq[st] = base + (unsigned)t;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive_expect_tx(&sh.full[st], bytes);
        bulk_load(&sh.ring[st][0], body + c0, bytes, &sh.full[st]);
    };
    if (tid == 0)
        for (int t = 0; t < kStages && t < n_tiles; ++t) issue_tile(t);

    // head and tail runs: warp 0 / warp 1, one element per lane (at most 7 elements each)
    if (warp < 2) {
        const int cnt = warp == 0 ? sp.head : sp.tail;
        const int64_t e0 = warp == 0 ? 0 : p.V - sp.tail;
        float x = -INFINITY;
        if (lane < cnt) { x = E::load(row, e0 + lane); if (!(fabsf(x) < INFINITY)) x = -INFINITY; }
        float m = x;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFullMask, m, o));
        const float ref = m * p.c;
        double s = (lane < cnt && x > -INFINITY) ? (double)ex2_approx(fmaf(x, p.c, -ref)) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
        if (lane == 0) { const int r = warp == 0 ? 0 : n_runs - 1; sh.run_ref[r] = ref; sh.run_s[r] = s; }
    }

    const uint64_t c2 = pack2(p.c, p.c);
    for (int t = 0; t < n_tiles; ++t) {
        if (!__all_sync(kFullMask, mbar_wait_limited(&sh.full[st], phase, tile_wait_limit(t, fault_tile)))) { sh.timeout = 1; break; }
        // this warp's run of the tile: chunks [c0, c0 + kRunChunks), four per lane
        const int c0 = t * kTileChunks + warp * kRunChunks;
        const int nvw = max(0, min(kRunChunks, nc - c0));
        if (nvw > 0) {
            const uint4* run = &sh.ring[st][warp * kRunChunks];
            const uint32_t ninf = E::ES == 2 ? 0xff80ff80u : 0xff800000u;      // -Inf in every element of a word
            uint4 w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) w[u] = u * 32 + lane < nvw ? run[u * 32 + lane] : make_uint4(ninf, ninf, ninf, ninf);
            // fast path: packed maximum (NaN ignored), one packed FMA per two elements, one ex2 per element.
            // A +Inf or a NaN in the run shows as an infinite maximum or a NaN sum and sends the warp to the
            // element-by-element path below.
            float m = E::max4(w[0], w[1], w[2], w[3]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFullMask, m, o));
            float ref = m * p.c;                                                // reference exponent of the run
            double s = 0.0;
            bool careful = !(m < INFINITY);                                     // +Inf, or nothing but NaN
            if (!careful && m > -INFINITY) {
                const uint64_t nref2 = pack2(-ref, -ref);
                uint64_t acc2 = 0ull;                                           // {0.0f, 0.0f}
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float f[E::EPC];
                    E::unpack(w[u], f);
                    uint64_t pr[E::EPC / 2];
#pragma unroll
                    for (int q = 0; q < E::EPC; q += 2) {
                        float t0, t1;
                        unpack2(fma2(pack2(f[q], f[q + 1]), c2, nref2), t0, t1);
                        pr[q / 2] = pack2(ex2_approx(t0), ex2_approx(t1));     // exp2(-Inf) = 0
                    }
                    uint64_t r2 = add2(pr[0], pr[1]);
                    if constexpr (E::EPC == 8) r2 = add2(r2, add2(pr[2], pr[3]));
                    acc2 = add2(acc2, r2);
                }
                float a0, a1;
                unpack2(acc2, a0, a1);
                s = (double)(a0 + a1);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
                careful = !(s == s);                                            // a NaN among the elements
            }
            if (careful) {                                                      // warp-uniform, rare
                float f[4 * E::EPC];
                m = -INFINITY;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    E::unpack(w[u], &f[u * E::EPC]);
#pragma unroll
                    for (int q = 0; q < E::EPC; ++q) {
                        float& x = f[u * E::EPC + q];
                        if (!(fabsf(x) < INFINITY)) x = -INFINITY;              // NaN and infinities carry no mass
                        m = fmaxf(m, x);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFullMask, m, o));
                ref = m * p.c;
                float part = 0.0f;
                if (m > -INFINITY) {
#pragma unroll
                    for (int q = 0; q < 4 * E::EPC; ++q) part += ex2_approx(fmaf(f[q], p.c, -ref));
                }
                s = (double)part;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
            }
            const int r = 1 + c0 / kRunChunks;
            if (lane == 0 && r < kMaxRuns) { sh.run_ref[r] = ref; sh.run_s[r] = s; }
        }
        __syncwarp();
        if (lane == 0 && atomicAdd(&sh.released[st], 1u) == kThreads / 32 - 1) {
            atomicExch(&sh.released[st], 0u);
            if (t + kStages < n_tiles) issue_tile(t + kStages);
        }
        if (++st == kStages) { st = 0; phase ^= 1u; }
    }
    __syncthreads();

    // ---- combine the runs (warp 0): total, the run that holds the crossing, the token inside it ----
    const bool ok = sh.timeout == 0;
    if (!ok && tid == 32) ring_drain(sh.full, sh.last_seq);        // every warp has left the tile loop: let the copies in flight land
    if (warp == 0) {
        int32_t ans = -2;                                          // a wait ran out: no draw
        if (ok) ans = sample_combine<DT>(sh, n_runs, p.c, p.uniforms[(int64_t)b * p.R + j], row, sp, body, p.V);
        if (lane == 0) *out = ans;
    }
    return ok;
}

// One CTA per (request, row).
template <int DT>
__global__ void __launch_bounds__(kThreads, 4) row_sample_kernel(SampleParams p) {
    grid_dependency_wait();
    grid_launch_dependents();                            // the walk kernel that follows is a handful of warps
    extern __shared__ __align__(16) unsigned char sample_smem_raw[];
    SampleShared& sh = *reinterpret_cast<SampleShared*>(sample_smem_raw + ((128u - (smem_u32(sample_smem_raw) & 127u)) & 127u));
    const int b = blockIdx.x / p.R;
    const int j = blockIdx.x - b * p.R;
    const int tid = threadIdx.x;
    if (p.rows_mode == CADD_ROWS_LIVE) {
        int n = p.n_nodes[b];
        n = n < 0 ? 0 : (n > p.R - 1 ? p.R - 1 : n);
        if (j > n) {
            if (tid == 0) p.node_token[(int64_t)b * p.R + j] = -1;
            return;
        }
    }
    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) { mbar_init(&sh.full[q], 1); sh.released[q] = 0; sh.last_seq[q] = kNoTile; }
        sh.timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned st = 0, phase = 0, issued = 0;
    sample_one_row<DT>(sh, p, b, j, st, phase, issued);
}

// LIVE with a small node cap: CTA g of request b takes rows g, g + ctas_per_request, ... one after the other (see
// row_argmax_kernel), so that few CTAs are launched only to exit.
template <int DT>
__global__ void __launch_bounds__(kThreads, 4) row_sample_shared_rows_kernel(SampleParams p) {
    grid_dependency_wait();
    grid_launch_dependents();
    extern __shared__ __align__(16) unsigned char sample_smem_raw[];
    SampleShared& sh = *reinterpret_cast<SampleShared*>(sample_smem_raw + ((128u - (smem_u32(sample_smem_raw) & 127u)) & 127u));
    const int b = blockIdx.x / p.ctas_per_request;
    const int g = blockIdx.x - b * p.ctas_per_request;
    const int tid = threadIdx.x;
    int n = p.n_nodes[b];
    n = n < 0 ? 0 : (n > p.R - 1 ? p.R - 1 : n);
    if (g > n) {                                         // nothing to read for this CTA: mark its rows and leave
        for (int j = g + tid * p.ctas_per_request; j < p.R; j += kThreads * p.ctas_per_request)
            p.node_token[(int64_t)b * p.R + j] = -1;
        return;
    }
    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) { mbar_init(&sh.full[q], 1); sh.released[q] = 0; sh.last_seq[q] = kNoTile; }
        sh.timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned st = 0, phase = 0, issued = 0;
    for (int j = g; j < p.R; j += p.ctas_per_request) {
        if (j > n) {
            if (tid == 0) p.node_token[(int64_t)b * p.R + j] = -1;
            continue;
        }
        if (!sample_one_row<DT>(sh, p, b, j, st, phase, issued)) {   // give up on this CTA's other rows too
            for (int jj = j + p.ctas_per_request + tid * p.ctas_per_request; jj < p.R; jj += kThreads * p.ctas_per_request)
                p.node_token[(int64_t)b * p.R + jj] = jj > n ? -1 : -2;
            return;
        }
        __syncthreads();                                 // the run table and the ring are free for the next row
    }
}

}  // namespace cadd
