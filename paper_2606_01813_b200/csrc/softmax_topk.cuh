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
// asynchronous copies (cp.async.bulk, completion on an mbarrier; no multicast), so several tiles are
// always in flight per CTA while the other threads compute from shared memory.
//
// Hot loop per 16-byte chunk (8 bf16 / 4 fp32): chunk max (packed), one compare against the CTA's
// running KP-th best value; per element two FMAs (x*log2e split in hi+lo, minus an integer reference
// exponent; issued as packed fma.rn.f32x2), one ex2.approx, and packed adds; the fp32 sum of one chunk
// goes to an fp64 accumulator.  A chunk whose maximum reaches the threshold value pushes its
// candidates into a shared buffer and keeps them out of the sum; when the buffer holds 2*KP entries
// the CTA ranks them, keeps the KP best, raises the threshold and folds the evicted ones into the sums.
#pragma once
#include "common.cuh"

namespace cadd {

constexpr int kTopkUnroll = 4;            // chunks per thread per tile
constexpr int kTileChunks = kTopkUnroll * kThreads;   // 16-byte chunks per tile (16 KB)
constexpr int kStages = 3;                // tiles in flight per CTA
constexpr int kSpinLimit = 1 << 18;       // bounded mbarrier wait (each try may itself block for a while)
constexpr int kCandCap = 512;             // candidate buffer entries per CTA
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
    uint64_t keys[kCandCap];
    uint64_t win[kMaxKP];
    unsigned hist[256];
    unsigned count;          // pushes so far (may exceed kCandCap: the excess was not stored)
    unsigned nwin;
    uint64_t thr_key;        // candidates must beat this key (0 = none yet)
    float thr_val;           // its logit value (-Inf = none yet)
    uint64_t sel_prefix;
    unsigned sel_need;
    double red_d[kThreads / 32];
    float red_f[kThreads / 32];
    unsigned red_u[kThreads / 32];
    unsigned timeout;        // set when a bounded wait ran out
    alignas(8) uint64_t full[kStages];                 // mbarriers: tile landed
    alignas(128) uint4 ring[kStages][kTileChunks];     // tiles of logits
};

// ---- mbarrier / bulk-copy primitives (shared::cta addresses, no cluster, no multicast) ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Wait for a phase with an iteration limit; false = gave up (the caller flags an error and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, unsigned parity) {
    for (int it = 0; it < kSpinLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// 1-D bulk copy global -> this CTA's shared memory; both addresses 16-byte aligned, bytes % 16 == 0.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

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

// Hot-loop handling of one element whose value reached the threshold value.  Kept out of line so that
// the chunk loop stays small.  Returns a bit set: kTakeExclude = keep it out of the fast sum,
// kTakeDropped = buffer full, retry after the next refresh, kTakeRefresh = the buffer now holds 2*KP
// entries or more, plus partial flags shifted left by 8.
constexpr uint32_t kTakeExclude = 1u, kTakeDropped = 2u, kTakeRefresh = 4u;
__device__ __noinline__ uint32_t take_candidate(TopkShared& sh, float x, uint32_t id, uint64_t thrk, int KP) {
    const uint32_t bits = __float_as_uint(x);
    if ((bits & 0x7f800000u) == 0x7f800000u)               // +Inf (-Inf only while no threshold is set)
        return kTakeExclude | (bits == 0x7f800000u ? (kPartNonfinite | kPartPosInf) << 8 : 0u);
    const uint64_t key = make_key(x, id);
    if (key <= thrk) return 0u;                            // equal value, higher id than the threshold key
    const unsigned pos = atomicAdd(&sh.count, 1u);
    if (pos >= (unsigned)kCandCap) return kTakeExclude | kTakeDropped | kTakeRefresh;
    sh.keys[pos] = key;
    return kTakeExclude | (pos + 1 >= 2u * (unsigned)KP ? kTakeRefresh : 0u);
}

// The thread's sum is passed and returned by value so that it stays in registers in the hot loop.
// CTA-wide: keep the KP best candidates of the buffer, fold the rest into the callers' sums and raise
// the threshold to the KP-th best key.  Small buffers are ranked by counting; larger ones go through
// an MSB-first radix select.  Leaves the survivors sorted, best first.
__device__ __noinline__ ThreadSum refresh_candidates(TopkShared& sh, ThreadSum s, int KP) {
    const int tid = threadIdx.x;
    __syncthreads();
    const int n = min(sh.count, (unsigned)kCandCap);
    if (n <= KP) {
        if (tid == 0) sh.count = n;
        __syncthreads();
        return s;
    }
    uint64_t kth;
    if (n <= 64) {
        // the common case: warp 0 ranks all entries in registers (two per lane), every entry is
        // broadcast once and compared against both
        if (tid < 32) {
            const uint64_t k0 = tid < n ? sh.keys[tid] : 0ull;
            const uint64_t k1 = tid + 32 < n ? sh.keys[tid + 32] : 0ull;
            int r0 = 0, r1 = 0;
            for (int j = 0; j < n; ++j) {
                const uint64_t kj = __shfl_sync(kFullMask, j < 32 ? k0 : k1, j & 31);
                r0 += kj > k0;
                r1 += kj > k1;
            }
            if (tid < n) { if (r0 < KP) sh.win[r0] = k0; else fold_scalar(s, key_value(k0)); }
            if (tid + 32 < n) { if (r1 < KP) sh.win[r1] = k1; else fold_scalar(s, key_value(k1)); }
        }
        __syncthreads();
        kth = sh.win[KP - 1];
    } else if (n <= kThreads) {
        // rank by counting, one warp per entry: 32 comparisons per step, counted with a ballot
        const int lane = tid & 31;
        for (int i = tid >> 5; i < n; i += kThreads / 32) {
            const uint64_t k = sh.keys[i];
            int rank = 0;
            for (int q0 = 0; q0 < n; q0 += 32) {
                const uint64_t kk = (q0 + lane < n) ? sh.keys[q0 + lane] : 0ull;
                rank += __popc(__ballot_sync(kFullMask, kk > k));
            }
            if (lane == 0) {
                if (rank < KP) sh.win[rank] = k;
                else fold_scalar(s, key_value(k));
            }
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

// Replace element q of a chunk by -Inf (its exponential is exactly zero afterwards).
template <int DT>
__device__ __forceinline__ void mask_out(uint4& w, int q) {
    uint32_t* words = reinterpret_cast<uint32_t*>(&w);
    if constexpr (DT == CADD_DTYPE_BF16) {
        uint32_t& x = words[q >> 1];
        x = (q & 1) ? ((x & 0x0000ffffu) | 0xff800000u) : ((x & 0xffff0000u) | 0x0000ff80u);
    } else {
        words[q] = 0xff800000u;
    }
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 4) softmax_topk_partial_kernel(TopkParams p) {
    using E = Elem<DT>;
    static_assert(kTopkUnroll == 4, "the tile loop below is written for four chunks per thread");
    extern __shared__ unsigned char topk_smem_raw[];
    TopkShared& sh = *reinterpret_cast<TopkShared*>(((uintptr_t)topk_smem_raw + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x;
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

    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) mbar_init(&sh.full[q], 1);
        sh.timeout = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // the elected thread issues tile t of this attempt into stage (seq % kStages)
    auto issue_tile = [&](int t, unsigned seq) {
        const int c0 = c_begin + t * kTileChunks;
        const unsigned bytes = (unsigned)min(kTileChunks, c_end - c0) * 16u;
        const unsigned st = seq % kStages;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic reads of the stage are done
        mbar_arrive_expect_tx(&sh.full[st], bytes);
        bulk_load(&sh.ring[st][0], body + c0, bytes, &sh.full[st]);
    };

    const uint64_t l2e_hi2 = pack2(kLog2eHi, kLog2eHi), l2e_lo2 = pack2(kLog2eLo, kLog2eLo);
    unsigned seq0 = 0;             // sequence number of tile 0 of the current attempt
    bool careful = false;          // second attempt: every element goes through slow_element
    double W = 0.0, Cmax = 0.0;
    uint32_t flags = 0;
    for (;;) {
        if (tid == 0) {
            sh.count = 0; sh.thr_key = 0; sh.thr_val = -INFINITY;
            for (int t = 0; t < kStages && t < n_tiles; ++t) issue_tile(t, seq0 + t);
        }
        __syncthreads();
        ThreadSum s{0.0, -INFINITY, 0.0f};
        flags = 0;
        bool want_refresh = false;
        uint32_t dropped = 0;
        // ragged ends of the row, one element per thread
        if (seg == 0 && tid < sp.head)
            slow_element(sh, s, flags, want_refresh, E::load(row, tid), (uint32_t)tid);
        if (seg == p.S - 1 && tid < sp.tail) {
            int64_t e = p.V - sp.tail + tid;
            slow_element(sh, s, flags, want_refresh, E::load(row, e), (uint32_t)e);
        }

        float thrv = -INFINITY;
        uint64_t thrk = 0, negc2 = 0;
        auto reload_threshold = [&]() {                             // both only change inside a refresh
            thrv = sh.thr_val;
            thrk = sh.thr_key;
            if (thrv > s.tmax + 60.0f) raise_reference(s, thrv);    // keeps 2^(x*log2e - c) in range for x < thrv
            negc2 = pack2(s.negc, s.negc);
        };
        // Push the candidates of a chunk (value >= threshold value, key above the threshold key) and replace
        // them by -Inf in the register copy, so that the common arithmetic leaves them out of the sum exactly.
        auto extract_candidates = [&](uint4& w, int c, int bit0) {
            const uint32_t id0 = (uint32_t)(sp.head + (int64_t)c * E::EPC);
            float f[E::EPC];
            E::unpack(w, f);
#pragma unroll
            for (int q = 0; q < E::EPC; ++q) {
                if (f[q] >= thrv) {
                    const uint32_t r = take_candidate(sh, f[q], id0 + q, thrk, KP);
                    if (r & kTakeExclude) mask_out<DT>(w, q);
                    if (r & kTakeDropped) dropped |= 1u << (bit0 + q);
                    if (r & kTakeRefresh) want_refresh = true;
                    flags |= r >> 8;
                }
            }
        };
        // one chunk with all checks (tile 0, ragged tiles, the careful attempt)
        auto checked_chunk = [&](uint4 w, int c, int bit0) {
            if (careful) {                                          // rare: re-read element by element
                const uint32_t id0 = (uint32_t)(sp.head + (int64_t)c * E::EPC);
#pragma unroll 1
                for (int q = 0; q < E::EPC; ++q)
                    if (slow_element(sh, s, flags, want_refresh, E::load(row, id0 + q), id0 + q)) dropped |= 1u << (bit0 + q);
                return;
            }
            if (E::chunk_max(w) >= thrv) extract_candidates(w, c, bit0);
            float lo, hi;
            unpack2(chunk_exp_sum2<DT>(w, l2e_hi2, l2e_lo2, negc2), lo, hi);
            s.acc += (double)(lo + hi);
        };
        // end of a step: refresh the candidate buffer when asked to, retry dropped elements
        auto settle = [&](bool force, int cbase) {
            if (!__syncthreads_or(want_refresh || dropped != 0 || force)) return;
            want_refresh = false;
            for (;;) {
                s = refresh_candidates(sh, s, KP);
                uint32_t again = 0;
                while (dropped) {                                   // retry what did not fit
                    int bit = __ffs(dropped) - 1;
                    dropped &= dropped - 1;
                    int u = bit / E::EPC, q = bit - u * E::EPC;
                    int64_t el = sp.head + (int64_t)(cbase + u * kThreads + tid) * E::EPC + q;
                    if (slow_element(sh, s, flags, want_refresh, E::load(row, el), (uint32_t)el)) again |= 1u << bit;
                }
                dropped = again;
                if (!__syncthreads_or(dropped != 0 || want_refresh)) break;
                want_refresh = false;
            }
            reload_threshold();
        };

        bool failed = false;
        for (int t = 0; t < n_tiles; ++t) {
            const unsigned seq = seq0 + t;
            const unsigned st = seq % kStages;
            // every thread waits for the tile; a thread that gives up raises a flag which all threads read
            // after the next barrier, so that the decision to leave is uniform
            bool landed = mbar_wait_bounded(&sh.full[st], (seq / kStages) & 1u);
            if (!landed) sh.timeout = 1;
            const int cbase = c_begin + t * kTileChunks;
            const uint4* tile = &sh.ring[st][tid];
            const int c3 = cbase + 3 * kThreads + tid;

            if (t == 0) {
                landed = __syncthreads_and(landed) != 0;            // the steps below have barriers of their own
                if (!landed) { failed = true; break; }
                if (!careful && c_end - c_begin >= kThreads) {
                    // Seed the threshold: at least KP finite elements are >= the smallest of KP' group maxima
                    // (groups of 256/KP' consecutive threads, KP' = KP rounded up to a power of two), each
                    // thread contributing the maximum of its chunks of this tile.  Elements equal to the
                    // seed value stay candidates.
                    float gm = -INFINITY;
#pragma unroll
                    for (int u = 0; u < kTopkUnroll; ++u)
                        if (cbase + u * kThreads + tid < c_end) gm = fmaxf(gm, E::chunk_max(tile[u * kThreads]));
                    if (!(fabsf(gm) < INFINITY)) gm = -INFINITY;   // NaN or Inf: no help from this thread
                    const int gs = KP <= 16 ? 16 : (KP <= 32 ? 8 : 4);
                    for (int o = gs >> 1; o > 0; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(kFullMask, gm, o));
                    float* seeds = (float*)sh.hist;
                    if ((tid & (gs - 1)) == 0) seeds[tid / gs] = gm;
                    __syncthreads();
                    if (tid < 32) {
                        const int ng = kThreads / gs;
                        float v = INFINITY;
                        for (int q = tid; q < ng; q += 32) v = fminf(v, seeds[q]);
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(kFullMask, v, o));
                        if (tid == 0 && v > -INFINITY) {
                            sh.thr_val = v;
                            sh.thr_key = make_key(v, 0xffffffffu); // the lowest key carrying this value
                        }
                    }
                    __syncthreads();
                }
                reload_threshold();
#pragma unroll 1
                for (int u = 0; u < kTopkUnroll; ++u) {
                    const int c = cbase + u * kThreads + tid;
                    if (c < c_end) checked_chunk(tile[u * kThreads], c, u * E::EPC);
                }
            } else if (landed && !careful && c3 < c_end) {
                // lean path: four whole chunks per thread, one test for all 32 (16) elements
                uint4 w0 = tile[0], w1 = tile[kThreads], w2 = tile[2 * kThreads], w3 = tile[3 * kThreads];
                if (E::max4(w0, w1, w2, w3) >= thrv) {              // rare: some element is a candidate
                    extract_candidates(w0, cbase + tid, 0);
                    extract_candidates(w1, cbase + kThreads + tid, E::EPC);
                    extract_candidates(w2, cbase + 2 * kThreads + tid, 2 * E::EPC);
                    extract_candidates(w3, c3, 3 * E::EPC);
                }
                const uint64_t a = add2(chunk_exp_sum2<DT>(w0, l2e_hi2, l2e_lo2, negc2),
                                        chunk_exp_sum2<DT>(w1, l2e_hi2, l2e_lo2, negc2));
                const uint64_t c2 = add2(chunk_exp_sum2<DT>(w2, l2e_hi2, l2e_lo2, negc2),
                                         chunk_exp_sum2<DT>(w3, l2e_hi2, l2e_lo2, negc2));
                float lo, hi;
                unpack2(add2(a, c2), lo, hi);
                s.acc += (double)(lo + hi);
            } else if (landed) {                                    // ragged last tile, or the careful attempt
#pragma unroll 1
                for (int u = 0; u < kTopkUnroll; ++u) {
                    const int c = cbase + u * kThreads + tid;
                    if (c < c_end) checked_chunk(tile[u * kThreads], c, u * E::EPC);
                }
            }
            settle(t == 0, cbase);                                  // always sharpen the threshold after tile 0
            if (sh.timeout) { failed = true; break; }               // written before the barrier in settle(): uniform
            if (tid == 0 && t + kStages < n_tiles) issue_tile(t + kStages, seq + kStages);   // the stage is free again
        }
        if (failed) {
            // give copies still in flight a bounded chance to land before this CTA's shared memory is released
            if (tid == 0)
                for (int q = 0; q < kStages; ++q) mbar_wait_bounded(&sh.full[q], 0);
            flags |= kPartTimeout;
            __syncthreads();
            if (tid == 0) sh.count = 0;
            __syncthreads();
            W = 0.0; Cmax = 0.0;
            break;
        }
        seq0 += n_tiles;
        s = refresh_candidates(sh, s, KP);                          // leaves min(KP, candidates) keys, sorted

        // CTA combine: common reference C = max c_t, W = sum acc_t * 2^(c_t - C)
        float c_t = (s.acc != 0.0) ? -s.negc : -INFINITY;
        float cm = c_t;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(kFullMask, cm, o));
        if ((tid & 31) == 0) sh.red_f[tid >> 5] = cm;
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
        if ((tid & 31) == 0) { sh.red_d[tid >> 5] = part; sh.red_u[tid >> 5] = fl; }
        __syncthreads();
        W = 0.0; flags = 0;
#pragma unroll
        for (int q = 0; q < kThreads / 32; ++q) { W += sh.red_d[q]; flags |= sh.red_u[q]; }
        Cmax = (cm == -INFINITY) ? 0.0 : (double)cm;
        // A NaN that slipped through the fast path poisons W: redo the segment element by element.
        if (careful || (W == W && W < INFINITY)) break;
        careful = true;
        __syncthreads();
    }

    // write the record: the surviving keys are already sorted, best first
    unsigned char* rec = p.partials + (size_t)item * seg_partial_stride(KP);
    uint64_t* out_keys = (uint64_t*)(rec + sizeof(SegPartial));
    const int cnt = (int)sh.count;
    if (tid < cnt) {
        const uint64_t k = sh.keys[tid];
        int rank = 0;
        for (int q = 0; q < cnt; ++q) rank += sh.keys[q] > k;      // (also sorts the cnt <= KP early-out case)
        out_keys[rank] = k;
    }
    if (tid == 0) {
        SegPartial h;
        h.W = W * kEx2BiasFix; h.C = Cmax; h.cnt = cnt; h.flags = flags; h.pad[0] = h.pad[1] = 0;
        *(SegPartial*)rec = h;
    }
}

}  // namespace cadd
