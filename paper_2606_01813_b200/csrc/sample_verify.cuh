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

namespace cadd {

constexpr int kRunChunks = kTileChunks / (kThreads / 32);     // 128 chunks = 2 KB per warp and tile
constexpr int kMaxRuns = 1024;                                // runs per row kept in shared memory (V up to ~1M bf16 / 0.5M fp32 elements)

struct SampleParams {
    const void* logits;        // [batch, R, V]
    int64_t V, stride_b, stride_row;
    int R, rows_mode;
    float c;                   // log2(e) / T
    const int32_t* n_nodes;    // [batch]
    const double* uniforms;    // [batch, R]
    int32_t* node_token;       // [batch, R]
};

struct SampleShared {
    alignas(8) uint64_t full[kStages];
    unsigned released[kStages];
    unsigned timeout;
    int n_runs;
    float run_m[kMaxRuns];                // per run: maximum (finite elements; -Inf if none)
    double run_s[kMaxRuns];               // per run: sum of exp((y - m) / T)
    alignas(128) uint4 ring[kStages][kTileChunks];
};
inline size_t sample_smem_bytes() { return sizeof(SampleShared) + 128; }

__device__ __forceinline__ float ex2f(float t) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 3) row_sample_kernel(SampleParams p) {
    using E = Elem<DT>;
    extern __shared__ __align__(16) unsigned char sample_smem_raw[];
    SampleShared& sh = *reinterpret_cast<SampleShared*>(sample_smem_raw + ((128u - (smem_u32(sample_smem_raw) & 127u)) & 127u));
    const int b = blockIdx.x / p.R;
    const int j = blockIdx.x - b * p.R;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* out = p.node_token + (int64_t)b * p.R + j;
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
    const uint4* body = (const uint4*)(row + (int64_t)sp.head * E::ES);
    const int nc = sp.n_chunks;
    const int n_tiles = (nc + kTileChunks - 1) / kTileChunks;
    // runs in token order: run 0 = the scalar head (if any), then the 2 KB runs of the body, then the scalar tail
    const int body_runs = (nc + kRunChunks - 1) / kRunChunks;
    const int n_runs = 1 + body_runs + 1;

    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) { mbar_init(&sh.full[q], 1); sh.released[q] = 0; }
        sh.timeout = 0;
        sh.n_runs = n_runs;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue_tile = [&](int t) {
        const int c0 = t * kTileChunks;
        const unsigned bytes = (unsigned)min(kTileChunks, nc - c0) * 16u;
        const unsigned st = (unsigned)t % kStages;
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
        double s = (lane < cnt && x > -INFINITY) ? (double)ex2f((x - m) * p.c) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
        if (lane == 0) { const int r = warp == 0 ? 0 : n_runs - 1; sh.run_m[r] = m; sh.run_s[r] = s; }
    }

    unsigned st = 0, phase = 0;
    for (int t = 0; t < n_tiles; ++t) {
        if (!__all_sync(kFullMask, mbar_wait_bounded(&sh.full[st], phase))) { sh.timeout = 1; break; }
        // this warp's run of the tile: chunks [c0, c0 + kRunChunks), four per lane
        const int c0 = t * kTileChunks + warp * kRunChunks;
        const int nvw = max(0, min(kRunChunks, nc - c0));
        if (nvw > 0) {
            const uint4* run = &sh.ring[st][warp * kRunChunks];
            float f[4 * E::EPC];
            float m = -INFINITY;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (u * 32 + lane < nvw) {
                    E::unpack(run[u * 32 + lane], &f[u * E::EPC]);
#pragma unroll
                    for (int q = 0; q < E::EPC; ++q) {
                        float& x = f[u * E::EPC + q];
                        if (!(fabsf(x) < INFINITY)) x = -INFINITY;          // NaN and infinities carry no mass
                        m = fmaxf(m, x);
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < E::EPC; ++q) f[u * E::EPC + q] = -INFINITY;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFullMask, m, o));
            float part = 0.0f;
            if (m > -INFINITY) {
#pragma unroll
                for (int q = 0; q < 4 * E::EPC; ++q) part += ex2f((f[q] - m) * p.c);   // exp2(-inf) = 0
            }
            double s = (double)part;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
            const int r = 1 + c0 / kRunChunks;
            if (lane == 0 && r < kMaxRuns) { sh.run_m[r] = m; sh.run_s[r] = s; }
        }
        __syncwarp();
        if (lane == 0 && atomicAdd(&sh.released[st], 1u) == kThreads / 32 - 1) {
            atomicExch(&sh.released[st], 0u);
            if (t + kStages < n_tiles) issue_tile(t + kStages);
        }
        if (++st == kStages) { st = 0; phase ^= 1u; }
    }
    __syncthreads();

    // ---- combine the runs (warp 0): global maximum, total, the run that holds the crossing ----
    if (warp == 0) {
        const int nr = min(n_runs, kMaxRuns);
        float M = -INFINITY;
        for (int r = lane; r < nr; r += 32) M = fmaxf(M, sh.run_m[r]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFullMask, M, o));
        int32_t ans = 0;                                           // no finite logit at all: token 0, as the arg-max does
        if (M > -INFINITY && !sh.timeout) {
            // weights of the runs relative to M, in fp64; prefix over the runs in token order, 32 runs per step
            double Z = 0.0;
            for (int r = lane; r < nr; r += 32)
                if (sh.run_m[r] > -INFINITY) Z += sh.run_s[r] * exp2((double)(sh.run_m[r] - M) * (double)p.c);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) Z += __shfl_xor_sync(kFullMask, Z, o);
            const double target = p.uniforms[(int64_t)b * p.R + j] * Z;
            double before = 0.0;                                   // mass of the runs before the current block of 32
            int hit_run = -1;
            double hit_before = 0.0;
            for (int r0 = 0; r0 < nr && hit_run < 0; r0 += 32) {
                const int r = r0 + lane;
                const double wgt = (r < nr && sh.run_m[r] > -INFINITY) ? sh.run_s[r] * exp2((double)(sh.run_m[r] - M) * (double)p.c) : 0.0;
                double incl = wgt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double up = __shfl_up_sync(kFullMask, incl, o);
                    if (lane >= o) incl += up;
                }
                const unsigned cross = __ballot_sync(kFullMask, r < nr && wgt > 0.0 && before + incl > target);
                if (cross) {
                    const int l = __ffs(cross) - 1;
                    hit_run = r0 + l;
                    hit_before = before + __shfl_sync(kFullMask, incl - wgt, l);
                }
                before += __shfl_sync(kFullMask, incl, 31);
            }
            if (hit_run < 0) {                                     // rounding left the target a hair above the total: last run with mass
                for (int r = nr - 1; r >= 0 && hit_run < 0; --r)
                    if (sh.run_m[r] > -INFINITY && sh.run_s[r] > 0.0) hit_run = r;
                hit_before = -1.0;                                 // marks "take the run's last element with mass"
            }
            // ---- scan the elements of that run in token order: 32 consecutive elements per lane ----
            int64_t e0;
            int ne;
            if (hit_run == 0) { e0 = 0; ne = sp.head; }
            else if (hit_run == n_runs - 1) { e0 = p.V - sp.tail; ne = sp.tail; }
            else { e0 = sp.head + (int64_t)(hit_run - 1) * kRunChunks * E::EPC; ne = (int)min((int64_t)kRunChunks * E::EPC, sp.head + (int64_t)nc * E::EPC - e0); }
            const int per = (ne + 31) / 32;
            const int lo = lane * per, hi = min(ne, lo + per);
            double mine = 0.0;
            for (int q = lo; q < hi; ++q) {
                const float x = E::load(row, e0 + q);
                if (fabsf(x) < INFINITY) mine += exp2((double)(x - M) * (double)p.c);
            }
            double incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(kFullMask, incl, o);
                if (lane >= o) incl += up;
            }
            const double need = hit_before < 0.0 ? 1e300 : target - hit_before;      // mass wanted inside the run
            unsigned cross = __ballot_sync(kFullMask, mine > 0.0 && incl > need);
            if (!cross) cross = 0x80000000u >> __clz(__ballot_sync(kFullMask, mine > 0.0) | 1u);   // the last lane with mass
            const int l = __ffs(cross) - 1;
            const double base = __shfl_sync(kFullMask, incl - mine, l);
            if (lane == l) {
                double acc = base;
                int64_t pick = -1, last = -1;
                for (int q = lo; q < hi; ++q) {
                    const float x = E::load(row, e0 + q);
                    if (!(fabsf(x) < INFINITY)) continue;
                    acc += exp2((double)(x - M) * (double)p.c);
                    last = e0 + q;
                    if (acc > need) { pick = e0 + q; break; }
                }
                ans = (int32_t)(pick >= 0 ? pick : last);
            }
            ans = __shfl_sync(kFullMask, ans, l);
        }
        if (sh.timeout) ans = -2;
        if (lane == 0) *out = ans;
    }
}

}  // namespace cadd
