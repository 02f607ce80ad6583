// Fused softmax statistics + top-K over the vocabulary of every live (request, position) row
// (Eq. 1: q_i = softmax(l_i); Algorithm 1, Require: top-K tokens and log-probs per position).
//
// One pass over the logits.  A row is cut into S segments; one CTA handles one (row, segment) and
// leaves a partial result in the workspace:
//   - the KP best candidates of the segment as 64-bit keys (logit descending, token id ascending),
//   - W and C with  sum over all OTHER finite elements of 2^(x*log2(e) - C) = W   (fp64 W, integer C).
// The expansion kernel merges the S partials of a row.  The best candidates are kept out of W on
// purpose: their exponentials are taken in fp64 at merge time, so the fp32 exponentials used here
// only ever cover the part of the mass that is spread over many small terms.
//
// Data path: one elected thread streams the segment into a ring of shared-memory tiles with bulk
// asynchronous copies (cp.async.bulk into this CTA's own shared memory, completion on an mbarrier); a per-stage counter tells when
// all eight warps are done with a stage, and the last of them refills it.  Warps advance through the tiles on their own:
// there is no CTA-wide barrier in the steady state.
//
// Hot loop per thread and tile (four 16-byte chunks = 32 bf16 / 16 fp32): one packed max over all
// elements and one compare against the CTA's running threshold, voted across the warp; per element two FMAs
// (x*log2e split in hi+lo, minus an integer reference exponent; issued as packed fma.rn.f32x2), one
// ex2.approx, packed adds; the fp32 sum of the tile goes to an fp64 accumulator.  When some lane holds an
// element that reaches the threshold, the whole warp examines that lane's elements together, one element per
// lane, straight from the tile in shared memory: candidates are appended to a shared buffer of keys (one atomic
// per lane examined) and overwritten by -Inf in the tile, and the owner reloads its chunks, so that candidates
// are left out of the sum exactly.  The buffer is append-only while the segment streams.  The append that
// completes a block of 2*KP candidates makes its warp sort that block in registers (bitonic network over the
// lanes) and raise the threshold to the block's KP-th best key: every candidate already beat the old
// threshold, so this is a valid lower bound on the segment's KP-th best, with no lock and no list to maintain.
// At the end of the segment the CTA selects the KP best of the buffer and folds the rest back into the sums.
//
// If the buffer overflows (pathological inputs such as an ascending row) or a non-finite value poisons the
// sums, the segment is redone by the careful path: element by element from global memory, with a CTA-wide
// barrier protocol that compacts the buffer as it goes.  Slow, but correct for every input.
#pragma once
#include "common.cuh"
#include "tile_ring.cuh"

namespace cadd {

constexpr int kCandCap = 768;             // candidate buffer entries per CTA
constexpr int kMaxKP = 64;

constexpr uint32_t kPartNonfinite = 1u;   // NaN or +Inf seen
constexpr uint32_t kPartPosInf = 2u;      // +Inf seen
constexpr uint32_t kPartTimeout = 4u;     // a bulk copy did not complete within the spin limit

// Partial result of one (row, segment); followed in memory by KP keys (sorted, best first).
struct SegPartial {
    double W;          // sum of 2^(x*log2e - C) over finite elements that are not in the key list
    double C;          // integer-valued reference exponent
    int32_t cnt;       // number of keys (= min(KP, finite elements in the segment))
    uint32_t flags;
    uint32_t pad[2];
};
static_assert(sizeof(SegPartial) == 32, "SegPartial layout");

__host__ __device__ inline size_t seg_partial_stride(int KP) { return sizeof(SegPartial) + (size_t)KP * 8; }

struct TopkParams {
    const void* logits;          // [batch, L, V]
    int64_t V, stride_b, stride_l;
    int L, S, KP;
    const int32_t* l_eff;
    unsigned char* partials;     // [batch*L*S] records of seg_partial_stride(KP) bytes
    int fault_tile;              // test hook: this tile of every segment is never copied (-1: none)
};

constexpr float kLog2eHi = 1.44269502162933349609375f;     // float(log2 e)
constexpr float kLog2eLo = 1.92596299112661746e-8f;        // log2 e - kLog2eHi

__device__ __forceinline__ float ex2_approx(float t) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

// Per-thread running sum: acc = sum of 2^(x*log2e - c) over the elements this thread has folded in.
struct ThreadSum {
    double acc;
    float tmax;      // largest element folded in so far
    float negc;      // -c, c integer-valued, c >= tmax*log2e + 1
};

__device__ __forceinline__ void raise_reference(ThreadSum& s, float x) {
    float cnew = ceilf(fminf(x, 2.0e38f) * kLog2eHi) + 1.0f;
    float cold = -s.negc;
    if (s.acc != 0.0) s.acc = scalbn(s.acc, (int)fmaxf(cold - cnew, -4000.0f));
    s.negc = -cnew;
    s.tmax = x;
}

__device__ __forceinline__ float exp2_term(float x, float negc) {
    return ex2_approx(fmaf(x, kLog2eLo, fmaf(x, kLog2eHi, negc)));
}

__device__ __forceinline__ void fold_scalar(ThreadSum& s, float x) {   // x finite
    if (x > s.tmax) raise_reference(s, x);
    s.acc += (double)exp2_term(x, s.negc);
}

// Shared state of one CTA.
struct TopkShared {
    uint64_t keys[kCandCap]; // candidate keys; fast path: append-only, 0 = not written yet
    uint64_t win[kMaxKP];    // the KP best candidates so far, sorted, best first
    unsigned hist[256];
    unsigned count;          // careful path: entries in keys[]
    unsigned nwin;           // entries in win[]
    uint64_t thr_key;        // candidates must beat this key (0 = none yet); only ever rises
    float thr_val;           // careful path: its logit value
    uint64_t sel_prefix;
    unsigned sel_need;
    unsigned pushed;         // fast path: candidates appended so far
    unsigned overflow;       // fast path: the candidate buffer was full at some push
    unsigned timeout;        // a bounded wait ran out
    double red_d[kThreads / 32];
    float red_f[kThreads / 32];
    unsigned red_u[kThreads / 32];
    alignas(8) uint64_t full[kStages];                 // mbarriers: tile landed
    unsigned released[kStages];                        // warps done with the stage's current tile
    unsigned last_seq[kStages];                        // last tile issued into the stage (see ring_drain)
    alignas(128) uint4 ring[kStages][kTileChunks];     // tiles of logits
};

// ---- packed fp32x2 arithmetic (one instruction for two lanes of a register pair) ----
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Examine one element on the careful path (ragged row ends, retries, poisoned segments).  Returns
// true when the element had to be dropped because the candidate buffer was full (the caller retries
// it after the next refresh).
__device__ __forceinline__ bool slow_element(TopkShared& sh, ThreadSum& s, uint32_t& flags, bool& want_refresh,
                                             float x, uint32_t id) {
    uint32_t b = __float_as_uint(x);
    if ((b & 0x7f800000u) == 0x7f800000u) {               // Inf or NaN: no mass, never a candidate
        if (b != 0xff800000u) flags |= kPartNonfinite;    // anything but -Inf
        if (b == 0x7f800000u) flags |= kPartPosInf;
        return false;
    }
    uint64_t key = make_key(x, id);
    if (key > *(volatile uint64_t*)&sh.thr_key) {
        unsigned pos = atomicAdd(&sh.count, 1u);
        if (pos >= (unsigned)kCandCap) return true;
        sh.keys[pos] = key;
        want_refresh = true;
        return false;
    }
    fold_scalar(s, x);
    return false;
}

// Candidates per threshold update: at least twice KP, so that the block's KP-th best is a sharp bound.
__device__ __forceinline__ unsigned threshold_block(int KP) { return KP <= 16 ? 32u : (KP <= 32 ? 64u : 128u); }

// One warp turns a block of freshly appended candidates, starting at entry c0, into a new threshold: the
// block's KP-th best key.  Any KP distinct elements of the segment bound its KP-th best from below, so the
// result is always valid.  Nothing is removed from the buffer.
// Returns false if an announced entry never showed up within the spin limit.
__device__ __noinline__ bool warp_block_threshold(TopkShared& sh, unsigned c0, int KP) {
    const int lane = threadIdx.x & 31;
    const int per_lane = (int)threshold_block(KP) / 32;    // 1, 2 or 4
    uint64_t k[4] = {0ull, 0ull, 0ull, 0ull};
    bool ok = true;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (q < per_lane) {
            volatile uint64_t* slot = &sh.keys[c0 + q * 32 + lane];
            int spins = 0;
            while ((k[q] = *slot) == 0ull && spins < kSpinLimit && !*(volatile unsigned*)&sh.overflow) ++spins;   // its writer is about to store it
            if (k[q] == 0ull) ok = false;
        }
    }
    if (!__all_sync(kFullMask, ok)) return false;
    uint64_t kth;
    if (per_lane == 1) {
        uint64_t key = k[0];                               // bitonic sort over the lanes, best first
#pragma unroll
        for (int blk = 2; blk <= 32; blk <<= 1) {
#pragma unroll
            for (int j = blk >> 1; j > 0; j >>= 1) {
                const uint64_t other = __shfl_xor_sync(kFullMask, key, j);
                const bool take_max = ((lane & j) != 0) == ((lane & blk) != 0);
                key = take_max ? max(key, other) : min(key, other);
            }
        }
        kth = __shfl_sync(kFullMask, key, KP - 1);
    } else {                                               // rank the keys by counting (they are unique)
        int r[4] = {0, 0, 0, 0};
        for (int j = 0; j < 32; ++j) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (q < per_lane) {
                    const uint64_t bq = __shfl_sync(kFullMask, k[q], j);
#pragma unroll
                    for (int t = 0; t < 4; ++t) r[t] += (t < per_lane) && bq > k[t];
                }
            }
        }
        kth = 0ull;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const unsigned m = __ballot_sync(kFullMask, q < per_lane && r[q] == KP - 1);
            if (m) kth = __shfl_sync(kFullMask, k[q], __ffs(m) - 1);
        }
    }
    if (lane == 0) atomicMax((unsigned long long*)&sh.thr_key, (unsigned long long)kth);
    return true;
}

// The thread's sum is passed and returned by value so that it stays in registers in the hot loop.
// CTA-wide: keep the KP best candidates of the buffer, fold the rest into the callers' sums and raise
// the threshold to the KP-th best key.  Entries below the current threshold are dropped first; what is left is
// ranked by counting, or goes through an MSB-first radix select if it is still large.  Leaves the survivors sorted, best first.
__device__ __noinline__ ThreadSum refresh_candidates(TopkShared& sh, ThreadSum s, int KP) {
    const int tid = threadIdx.x;
    __syncthreads();
    int n = min(sh.count, (unsigned)kCandCap);
    if (n <= KP) {
        if (tid == 0) sh.count = n;
        __syncthreads();
        return s;
    }
    if (n > 64) {
        // The current threshold is the KP-th best of some subset of the buffer (or zero), so at least KP entries
        // reach it: everything below it is folded into the sums right away and only the rest is ranked.
        const uint64_t thr = sh.thr_key;
        uint64_t mine[kCandCap / kThreads];
#pragma unroll
        for (int q = 0; q < kCandCap / kThreads; ++q) mine[q] = tid + q * kThreads < n ? sh.keys[tid + q * kThreads] : 0ull;
        if (tid == 0) sh.nwin = 0;
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kCandCap / kThreads; ++q) {
            if (mine[q] == 0ull) continue;
            if (mine[q] >= thr) sh.keys[atomicAdd(&sh.nwin, 1u)] = mine[q];
            else fold_scalar(s, key_value(mine[q]));
        }
        __syncthreads();
        n = (int)sh.nwin;
        __syncthreads();
    }
    uint64_t kth;
    if (n <= kThreads) {
        // rank by counting, one thread per entry (keys are unique); every entry is read as a broadcast
        if (tid < n) {
            const uint64_t k = sh.keys[tid];
            int rank = 0;
            for (int j = 0; j < n; ++j) rank += sh.keys[j] > k;
            if (rank < KP) sh.win[rank] = k;
            else fold_scalar(s, key_value(k));
        }
        __syncthreads();
        kth = sh.win[KP - 1];
    } else {
        if (tid == 0) { sh.sel_prefix = 0; sh.sel_need = KP; sh.nwin = 0; }
        uint64_t mask = 0;
        for (int shift = 56; shift >= 0; shift -= 8) {
            sh.hist[tid] = 0;                                  // kThreads == 256 bins
            __syncthreads();
            const uint64_t prefix = sh.sel_prefix;
            for (int i = tid; i < n; i += kThreads) {
                uint64_t k = sh.keys[i];
                if ((k & mask) == prefix) atomicAdd(&sh.hist[(unsigned)(k >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (tid < 32) {
                // lane l owns digits 8l..8l+7; find the largest digit d with (count of digits > d) < need
                unsigned h[8], tot = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { h[q] = sh.hist[tid * 8 + q]; tot += h[q]; }
                unsigned incl = tot;                           // inclusive suffix sum over lanes
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    unsigned t = __shfl_down_sync(kFullMask, incl, o);
                    if (tid + o < 32) incl += t;
                }
                const unsigned above = incl - tot;             // entries in lanes above this one
                const unsigned need = sh.sel_need;
                __syncwarp();                                  // every lane has read sel_need before one rewrites it
                if (above < need && need <= incl) {            // the wanted digit lies in this lane's bins
                    unsigned run = above;
                    int d = 7;
#pragma unroll
                    for (int q = 7; q >= 0; --q) {
                        if (d == q && run + h[q] < need) { run += h[q]; d = q - 1; }
                    }
                    sh.sel_need = need - run;
                    sh.sel_prefix = prefix | ((uint64_t)(tid * 8 + d) << shift);
                }
            }
            mask |= (uint64_t)255u << shift;
            __syncthreads();
        }
        kth = sh.sel_prefix;                                   // keys are unique: exactly KP keys are >= kth
        for (int i = tid; i < n; i += kThreads) {
            uint64_t k = sh.keys[i];
            if (k >= kth) sh.win[atomicAdd(&sh.nwin, 1u)] = k;
            else fold_scalar(s, key_value(k));
        }
        __syncthreads();
        if (tid < KP) {                                        // sort the KP survivors by counting
            const uint64_t k = sh.win[tid];
            int rank = 0;
            for (int q = 0; q < KP; ++q) rank += sh.win[q] > k;
            sh.keys[kCandCap - kMaxKP + rank] = k;             // park them at the end of the buffer
        }
        __syncthreads();
        if (tid < KP) sh.win[tid] = sh.keys[kCandCap - kMaxKP + tid];
        __syncthreads();
    }
    if (tid < KP) sh.keys[tid] = sh.win[tid];
    if (tid == 0) {
        sh.count = KP;
        sh.thr_key = kth;
        sh.thr_val = key_value(kth);
    }
    __syncthreads();
    return s;
}

// ex2.approx on sm_100 returns the exponential truncated toward zero: measured mean relative error
// -5.05e-8 (arguments -32..-1, spread +-0.1e-8 over unit intervals).  The fast sums are scaled by this
// factor; the remaining per-term error is zero-mean.
constexpr double kEx2BiasFix = 1.0 + 5.05e-8;

// Dynamic shared memory of the kernel.
inline size_t topk_smem_bytes() { return sizeof(TopkShared) + 128; }

// Packed sum of 2^(x*log2e - c) over one chunk: lane 0 holds the even elements' sum, lane 1 the odd ones'.
template <int DT>
__device__ __forceinline__ uint64_t chunk_exp_sum2(const uint4& w, uint64_t l2e_hi2, uint64_t l2e_lo2, uint64_t negc2) {
    using E = Elem<DT>;
    float f[E::EPC];
    E::unpack(w, f);
    uint64_t pr[E::EPC / 2];
#pragma unroll
    for (int q = 0; q < E::EPC; q += 2) {
        const uint64_t x2 = pack2(f[q], f[q + 1]);
        float t0, t1;
        unpack2(fma2(x2, l2e_lo2, fma2(x2, l2e_hi2, negc2)), t0, t1);
        pr[q / 2] = pack2(ex2_approx(t0), ex2_approx(t1));
    }
    uint64_t r = add2(pr[0], pr[1]);
    if constexpr (E::EPC == 8) r = add2(r, add2(pr[2], pr[3]));
    return r;
}

// Careful path of softmax_topk_partial_kernel: the segment element by element from global memory under a CTA-wide
// protocol (taken when the candidate buffer overflowed or the sum came out non-finite).  Out of line: it is rare and
// large, and the streaming loop's code should not carry it.  Leaves the winners sorted in win[].
template <int DT>
__device__ __noinline__ ThreadSum careful_segment(TopkShared& sh, const char* row, RowSplit sp, int64_t V, int seg, int S,
                                                  int c_begin, int c_end, int KP, uint32_t* flags_out) {
    using E = Elem<DT>;
    const int tid = threadIdx.x;
    ThreadSum s;
    uint32_t flags;
    __syncthreads();
    if (tid == 0) { sh.count = 0; sh.nwin = 0; sh.thr_key = 0; sh.thr_val = -INFINITY; }
    __syncthreads();
    s = ThreadSum{0.0, -INFINITY, 0.0f};
    flags = 0;
    bool want_refresh = false;
    if (seg == 0 && tid < sp.head) slow_element(sh, s, flags, want_refresh, E::load(row, tid), (uint32_t)tid);
    if (seg == S - 1 && tid < sp.tail) {
        const int64_t e = V - sp.tail + tid;
        slow_element(sh, s, flags, want_refresh, E::load(row, e), (uint32_t)e);
    }
    for (int cbase = c_begin; cbase < c_end; cbase += kThreads) {
        const int c = cbase + tid;
        uint32_t dropped = 0;
        if (c < c_end) {
            const int64_t e0 = sp.head + (int64_t)c * E::EPC;
#pragma unroll 1
            for (int q = 0; q < E::EPC; ++q)
                if (slow_element(sh, s, flags, want_refresh, E::load(row, e0 + q), (uint32_t)(e0 + q))) dropped |= 1u << q;
        }
        if (__syncthreads_or(want_refresh || dropped != 0)) {
            want_refresh = false;
            for (;;) {
                s = refresh_candidates(sh, s, KP);
                uint32_t again = 0;
                while (dropped) {                               // retry what did not fit
                    const int q = __ffs(dropped) - 1;
                    dropped &= dropped - 1;
                    const int64_t e = sp.head + (int64_t)c * E::EPC + q;
                    if (slow_element(sh, s, flags, want_refresh, E::load(row, e), (uint32_t)e)) again |= 1u << q;
                }
                dropped = again;
                if (!__syncthreads_or(dropped != 0 || want_refresh)) break;
                want_refresh = false;
            }
        }
    }
    s = refresh_candidates(sh, s, KP);                          // leaves min(KP, candidates) keys in keys[]
    __syncthreads();
    // sort them into win[] by counting
    const int cnt = (int)sh.count;
    if (tid < cnt) {
        const uint64_t k = sh.keys[tid];
        int rank = 0;
        for (int q = 0; q < cnt; ++q) rank += sh.keys[q] > k;
        sh.win[rank] = k;
    }
    if (tid == 0) sh.nwin = cnt;
    __syncthreads();
    *flags_out = flags;
    return s;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 4) softmax_topk_partial_kernel(TopkParams p) {
    using E = Elem<DT>;
    static_assert(kTopkUnroll == 4, "the tile loop below is written for four chunks per thread");
    grid_dependency_wait();
    extern __shared__ __align__(16) unsigned char topk_smem_raw[];
    // aligned by pointer arithmetic on the shared array itself, so that every access below compiles to a
    // shared-memory instruction rather than a generic one
    TopkShared& sh = *reinterpret_cast<TopkShared*>(topk_smem_raw + ((128u - (smem_u32(topk_smem_raw) & 127u)) & 127u));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int item = blockIdx.x;
    const int rowi = item / p.S;
    const int seg = item - rowi * p.S;
    const int b = rowi / p.L;
    const int i = rowi - b * p.L;
    int clamped;
    if (i >= clamp_l_eff(p.l_eff, b, p.L, &clamped)) return;      // masked position: never read

    const char* row = (const char*)p.logits + ((int64_t)b * p.stride_b + (int64_t)i * p.stride_l) * E::ES;
    const RowSplit sp = split_row<DT>(row, p.V);
    const int cps = (sp.n_chunks + p.S - 1) / p.S;                 // chunks per segment
    const int c_begin = min(seg * cps, sp.n_chunks);
    const int c_end = min(c_begin + cps, sp.n_chunks);
    const uint4* body = (const uint4*)(row + (int64_t)sp.head * E::ES);
    const int KP = p.KP;
    const int n_tiles = (c_end - c_begin + kTileChunks - 1) / kTileChunks;

    for (int q = tid; q < kCandCap; q += kThreads) sh.keys[q] = 0ull;
    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) { mbar_init(&sh.full[q], 1); sh.released[q] = 0; sh.last_seq[q] = kNoTile; }
        sh.timeout = 0; sh.overflow = 0; sh.pushed = 0; sh.nwin = 0;
        sh.count = 0; sh.thr_key = 0; sh.thr_val = -INFINITY;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // one thread issues tile t into stage t % kStages: thread 0 for the first kStages tiles, afterwards
    // lane 0 of whichever warp is the last to finish with the tile that occupied the stage
    const int fault_tile = p.fault_tile < 0 ? -1 : min(p.fault_tile, n_tiles - 1);
    auto issue_tile = [&](int t) {
        if (t == fault_tile) return;                                   // test hook: this copy is never made
        const int c0 = c_begin + t * kTileChunks;
        const unsigned bytes = (unsigned)min(kTileChunks, c_end - c0) * 16u;
        const unsigned st = (unsigned)t % kStages;
        *(volatile unsigned*)&sh.last_seq[st] = (unsigned)t;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic reads of the stage are done
        mbar_arrive_expect_tx(&sh.full[st], bytes);
        bulk_load(&sh.ring[st][0], body + c0, bytes, &sh.full[st]);
    };
    if (tid == 0)
        for (int t = 0; t < kStages && t < n_tiles; ++t) issue_tile(t);

    const uint64_t l2e_hi2 = pack2(kLog2eHi, kLog2eHi), l2e_lo2 = pack2(kLog2eLo, kLog2eLo);
    ThreadSum s{0.0, -INFINITY, 0.0f};
    uint32_t flags = 0;

    // ================= fast path: warps advance on their own =================
    {
        // ragged ends of the row, one element per thread (segment 0 takes the head, the last one the tail)
        bool dummy = false;
        if (seg == 0 && tid < sp.head) slow_element(sh, s, flags, dummy, E::load(row, tid), (uint32_t)tid);
        if (seg == p.S - 1 && tid < sp.tail) {
            const int64_t e = p.V - sp.tail + tid;
            slow_element(sh, s, flags, dummy, E::load(row, e), (uint32_t)e);
        }
        // (slow_element appends to keys[0..count): at most 14 entries; they become the first candidates)
        __syncthreads();
        if (tid == 0) { sh.pushed = sh.count; sh.count = 0; }

        // Seed the threshold from tile 0.  Every thread takes the maximum of its chunks of the tile: 256 distinct
        // elements.  For KP <= 32 the seed is the exact KP-th largest of them: each warp sorts its 32 maxima over
        // the lanes (bitonic network), then warp 0 folds the eight sorted lists together, keeping the 32 largest
        // (elementwise max of one list with the other reversed, then one bitonic merge).  For larger KP it is the
        // smallest of 64 group maxima.  At least KP finite elements are >= the seed either way; elements equal
        // to it stay candidates.
        bool landed = true;
        float* seeds = (float*)sh.hist;
        float gm = -INFINITY;
        if (n_tiles > 0) {
            landed = mbar_wait_limited(&sh.full[0], 0, tile_wait_limit(0, fault_tile));
            if (landed) {
#pragma unroll
                for (int u = 0; u < kTopkUnroll; ++u)
                    if (c_begin + u * kThreads + tid < c_end) gm = fmaxf(gm, E::chunk_max(sh.ring[0][u * kThreads + tid]));
            }
            if (!(fabsf(gm) < INFINITY)) gm = -INFINITY;           // NaN or Inf: no help from this thread
            if (KP <= 32) {
#pragma unroll
                for (int blk = 2; blk <= 32; blk <<= 1) {
#pragma unroll
                    for (int j = blk >> 1; j > 0; j >>= 1) {
                        const float other = __shfl_xor_sync(kFullMask, gm, j);
                        const bool take_max = ((lane & j) != 0) == ((lane & blk) != 0);
                        gm = take_max ? fmaxf(gm, other) : fminf(gm, other);
                    }
                }
                seeds[tid] = gm;                                   // lane q of a warp: its q-th largest
            } else {
                for (int o = 2; o > 0; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(kFullMask, gm, o));
                if ((tid & 3) == 0) seeds[tid >> 2] = gm;
            }
            if (!landed) sh.timeout = 1;
        }
        __syncthreads();
        if (tid < 32 && n_tiles > 0) {
            float v;
            if (KP <= 32) {
                v = gm;
                for (int w = 1; w < kThreads / 32; ++w) {
                    v = fmaxf(v, seeds[w * 32 + 31 - lane]);       // the 32 largest of both lists, as a bitonic sequence
#pragma unroll
                    for (int j = 16; j > 0; j >>= 1) {
                        const float other = __shfl_xor_sync(kFullMask, v, j);
                        v = (lane & j) == 0 ? fmaxf(v, other) : fminf(v, other);
                    }
                }
                v = __shfl_sync(kFullMask, v, KP - 1);
            } else {
                v = fminf(seeds[tid], seeds[tid + 32]);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(kFullMask, v, o));
            }
            if (tid == 0 && v > -INFINITY) sh.thr_key = make_key(v, 0xffffffffu);   // the lowest key carrying this value
        }
        __syncthreads();

        const bool timed_out = sh.timeout != 0;
        unsigned st = 0, phase = 0;
        for (int t = 0; t < n_tiles && !timed_out; ++t, st = (st + 1 == kStages ? 0u : st + 1), phase ^= (st == 0 ? 1u : 0u)) {
            const bool here = __all_sync(kFullMask, mbar_wait_limited(&sh.full[st], phase, tile_wait_limit(t, fault_tile)));
            if (!here) { sh.timeout = 1; break; }
            const uint64_t thrk = *(volatile uint64_t*)&sh.thr_key;          // only ever rises; stale is safe
            const float thrv = thrk ? key_value(thrk) : -INFINITY;
            if (thrv > s.tmax + 60.0f) raise_reference(s, thrv);             // keeps 2^(x*log2e - c) in range for x < thrv
            const uint64_t negc2 = pack2(s.negc, s.negc);
            const int cbase = c_begin + t * kTileChunks;
            const uint4* tile = &sh.ring[st][tid];
            // this thread's chunks of the tile; chunks past the end of the segment read as -Inf (no mass, never
            // a candidate), so that one code path serves whole and ragged tiles
            const uint4 kNone = DT == CADD_DTYPE_BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                                                      : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
            const int nv = c_end - (cbase + tid);                        // > u * kThreads  <=>  chunk u is valid
            const bool whole = cbase + kTileChunks <= c_end;             // CTA-uniform: every chunk of the tile is valid
            uint4 w0, w1, w2, w3;
            if (whole) {
                w0 = tile[0]; w1 = tile[kThreads]; w2 = tile[2 * kThreads]; w3 = tile[3 * kThreads];
            } else {
                w0 = nv > 0 ? tile[0] : kNone;
                w1 = nv > kThreads ? tile[kThreads] : kNone;
                w2 = nv > 2 * kThreads ? tile[2 * kThreads] : kNone;
                w3 = nv > 3 * kThreads ? tile[3 * kThreads] : kNone;
            }
            const float mx = E::max4(w0, w1, w2, w3);
            unsigned hits = __ballot_sync(kFullMask, mx >= thrv && mx > -INFINITY);
            if (hits) {
                // Some lane holds an element that reaches the threshold (about every second warp-tile, one or two
                // lanes).  The whole warp looks at that lane's elements together, one element per lane, straight
                // from the tile in shared memory: candidates are appended with one atomic per lane examined, and
                // overwritten by -Inf in the tile so that the owner's reload leaves them out of the sum exactly.
                constexpr int NE = kTopkUnroll * E::EPC;                 // elements per thread and tile: 32 or 16
                const int u = lane / E::EPC, q = lane % E::EPC;
                do {
                    const int src = __ffs(hits) - 1;
                    hits &= hits - 1;
                    const int slot = u * kThreads + warp * 32 + src;     // chunk slot inside the tile
                    const int c = cbase + slot;
                    const bool valid = lane < NE && c < c_end;
                    char* ep = (char*)&sh.ring[st][0] + (size_t)slot * 16 + q * E::ES;
                    float x = -INFINITY;
                    if (valid) x = E::load(ep, 0);
                    const uint32_t bits = __float_as_uint(x);
                    const bool ge = valid && x >= thrv;                  // false for NaN
                    const bool inf = (bits & 0x7f800000u) == 0x7f800000u;
                    const uint32_t id = (uint32_t)(sp.head + (int64_t)c * E::EPC + q);
                    const uint64_t key = make_key(x, id);
                    const bool cand = ge && !inf && key > thrk;          // equal value, higher id than the threshold key: stays in the sum
                    if (ge && bits == 0x7f800000u) flags |= kPartNonfinite | kPartPosInf;
                    const unsigned m = __ballot_sync(kFullMask, cand);
                    if (m) {
                        const unsigned cnt = __popc(m);
                        unsigned base = 0;
                        if (lane == 0) base = atomicAdd(&sh.pushed, cnt);
                        base = __shfl_sync(kFullMask, base, 0);
                        if (cand) {
                            const unsigned pos = base + __popc(m & ((1u << lane) - 1u));
                            if (pos < (unsigned)kCandCap) *(volatile uint64_t*)&sh.keys[pos] = key;
                            else sh.overflow = 1;                        // no room: the segment will be redone carefully
                        }
                        // the append that completes a block of candidates turns that block into a new threshold
                        const unsigned blk = threshold_block(KP), end = base + cnt;
                        if (end / blk != base / blk && end <= (unsigned)kCandCap) {
                            __syncwarp();
                            if (!warp_block_threshold(sh, (end / blk - 1u) * blk, KP) && !*(volatile unsigned*)&sh.overflow) sh.timeout = 1;
                        }
                    }
                    if (cand || (ge && inf)) {
                        if constexpr (DT == CADD_DTYPE_BF16) *(volatile uint16_t*)ep = 0xff80u;
                        else *(volatile uint32_t*)ep = 0xff800000u;
                    }
                } while (hits);
                __syncwarp();
                w0 = nv > 0 ? tile[0] : kNone;
                w1 = nv > kThreads ? tile[kThreads] : kNone;
                w2 = nv > 2 * kThreads ? tile[2 * kThreads] : kNone;
                w3 = nv > 3 * kThreads ? tile[3 * kThreads] : kNone;
            }
            {
                const uint64_t a = add2(chunk_exp_sum2<DT>(w0, l2e_hi2, l2e_lo2, negc2),
                                        chunk_exp_sum2<DT>(w1, l2e_hi2, l2e_lo2, negc2));
                const uint64_t c2 = add2(chunk_exp_sum2<DT>(w2, l2e_hi2, l2e_lo2, negc2),
                                         chunk_exp_sum2<DT>(w3, l2e_hi2, l2e_lo2, negc2));
                float lo, hi;
                unpack2(add2(a, c2), lo, hi);
                s.acc += (double)(lo + hi);
            }
            __syncwarp();
            // This warp is done with the stage: its loads from it have returned (their values were consumed above)
            // and its stores to it are ordered before the release.  The last warp to say so refills the stage.
            if (lane == 0) {
                __threadfence_block();
                if (atomicAdd(&sh.released[st], 1u) == kThreads / 32 - 1) {
                    atomicExch(&sh.released[st], 0u);
                    __threadfence_block();
                    if (t + kStages < n_tiles) issue_tile(t + kStages);
                }
            }
        }
        __syncthreads();
        // keep the KP best of the buffer, fold the rest into the sums (CTA-wide), sort the survivors into win[]
        if (tid == 0) {
            sh.count = min(sh.pushed, (unsigned)kCandCap);
            if (sh.timeout) ring_drain(sh.full, sh.last_seq);          // a wait ran out: let the copies still in flight land
        }
        __syncthreads();
        if (!sh.overflow && !sh.timeout) {
            s = refresh_candidates(sh, s, KP);
            const int cnt = (int)sh.count;
            if (tid < cnt) {
                const uint64_t k = sh.keys[tid];
                int rank = 0;
                for (int q = 0; q < cnt; ++q) rank += sh.keys[q] > k;
                sh.win[rank] = k;
            }
            if (tid == 0) sh.nwin = cnt;
        }
        __syncthreads();
    }

    // CTA combine: common reference C = max c_t, W = sum acc_t * 2^(c_t - C)
    double W, Cmax;
    auto combine = [&]() {
        float c_t = (s.acc != 0.0) ? -s.negc : -INFINITY;
        float cm = c_t;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(kFullMask, cm, o));
        if (lane == 0) sh.red_f[warp] = cm;
        __syncthreads();
        cm = sh.red_f[0];
#pragma unroll
        for (int q = 1; q < kThreads / 32; ++q) cm = fmaxf(cm, sh.red_f[q]);
        double part = (s.acc != 0.0) ? scalbn(s.acc, (int)fmaxf(c_t - cm, -4000.0f)) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFullMask, part, o);
        uint32_t fl = flags;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fl |= __shfl_xor_sync(kFullMask, fl, o);
        if (lane == 0) { sh.red_d[warp] = part; sh.red_u[warp] = fl; }
        __syncthreads();
        W = 0.0; flags = 0;
#pragma unroll
        for (int q = 0; q < kThreads / 32; ++q) { W += sh.red_d[q]; flags |= sh.red_u[q]; }
        Cmax = (cm == -INFINITY) ? 0.0 : (double)cm;
        __syncthreads();
    };
    combine();
    const bool timed_out = sh.timeout != 0;
    const bool redo = !timed_out && (sh.overflow != 0 || !(W == W && W < INFINITY));

    // ================= careful path: element by element from global memory, CTA-wide protocol =================
    if (redo) {
        s = careful_segment<DT>(sh, row, sp, p.V, seg, p.S, c_begin, c_end, KP, &flags);
        combine();
    }

    // write the record: win[] is sorted, best first
    unsigned char* rec = p.partials + (size_t)item * seg_partial_stride(KP);
    uint64_t* out_keys = (uint64_t*)(rec + sizeof(SegPartial));
    const int cnt = timed_out ? 0 : (int)sh.nwin;
    if (tid < cnt) out_keys[tid] = sh.win[tid];
    if (tid == 0) {
        SegPartial h;
        h.W = timed_out ? 0.0 : W * kEx2BiasFix; h.C = timed_out ? 0.0 : Cmax; h.cnt = cnt;
        h.flags = flags | (timed_out ? kPartTimeout : 0u); h.pad[0] = h.pad[1] = 0;
        *(SegPartial*)rec = h;
    }
}

}  // namespace cadd
