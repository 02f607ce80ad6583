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
// Hot loop per 16-byte chunk (8 bf16 / 4 fp32): chunk max (packed), one compare against the CTA's
// running K-th best value; below it, the fast path: per element two FMAs (x*log2e split in hi+lo,
// minus the thread's integer reference C_t), one ex2.approx, one add; fp32 sums of one chunk go to an
// fp64 accumulator.  At or above it, the slow path pushes candidates into a shared buffer; when the
// buffer passes its high-water mark the CTA radix-selects the KP-th best key, raises the threshold
// and folds the evicted candidates into the sums.
#pragma once
#include "common.cuh"

namespace cadd {

constexpr int kTopkUnroll = 4;            // chunks per thread per iteration
constexpr int kCandCap = 2048;            // candidate buffer entries per CTA
constexpr int kMaxKP = 64;

constexpr uint32_t kPartNonfinite = 1u;   // NaN or +Inf seen
constexpr uint32_t kPartPosInf = 2u;      // +Inf seen

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
};

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
    if (n <= kThreads) {
        uint64_t k = 0;
        int rank = 0;
        if (tid < n) {
            k = sh.keys[tid];
            for (int q = 0; q < n; ++q) rank += sh.keys[q] > k;
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

template <int DT>
__global__ void __launch_bounds__(kThreads, 3) softmax_topk_partial_kernel(TopkParams p) {
    using E = Elem<DT>;
    __shared__ TopkShared sh;
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
    constexpr int kIter = kTopkUnroll * kThreads;                  // chunks per CTA iteration

    bool careful = false;          // second attempt: every element goes through slow_element
    double W, Cmax;
    uint32_t flags;
    for (;;) {
        if (tid == 0) { sh.count = 0; sh.thr_key = 0; sh.thr_val = -INFINITY; }
        __syncthreads();
        ThreadSum s{0.0, -INFINITY, 0.0f};
        flags = 0;
        bool want_refresh = false;
        // ragged ends of the row, one element per thread
        if (seg == 0 && tid < sp.head)
            slow_element(sh, s, flags, want_refresh, E::load(row, tid), (uint32_t)tid);
        if (seg == p.S - 1 && tid < sp.tail) {
            int64_t e = p.V - sp.tail + tid;
            slow_element(sh, s, flags, want_refresh, E::load(row, e), (uint32_t)e);
        }

        uint4 w[kTopkUnroll], wn[kTopkUnroll];
#pragma unroll
        for (int u = 0; u < kTopkUnroll; ++u) {
            int c = c_begin + u * kThreads + tid;
            if (c < c_end) w[u] = ld_stream16(body + c);
        }
        // Seed the threshold: at least KP finite elements are >= the smallest of KP' group maxima
        // (groups of 256/KP' consecutive threads, KP' = KP rounded up to a power of two), taken over the
        // first chunk of every thread.  All elements equal to the seed value stay candidates.
        if (!careful && c_end - c_begin >= kThreads) {
            float gm = E::chunk_max(w[0]);
            if (!(fabsf(gm) < INFINITY)) gm = -INFINITY;           // NaN or Inf: no help from this chunk
            const int gs = KP <= 16 ? 16 : (KP <= 32 ? 8 : 4);     // threads per group
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
                    sh.thr_key = make_key(v, 0xffffffffu);         // the lowest key carrying this value
                }
            }
            __syncthreads();
        }

        for (int cbase = c_begin; cbase < c_end; cbase += kIter) {
#pragma unroll
            for (int u = 0; u < kTopkUnroll; ++u) {                 // prefetch the next iteration
                int c = cbase + kIter + u * kThreads + tid;
                if (c < c_end) wn[u] = ld_stream16(body + c);
            }
            const float thrv = sh.thr_val;                          // both only change inside a refresh
            const uint64_t thrk = sh.thr_key;
            uint32_t dropped = 0;
#pragma unroll
            for (int u = 0; u < kTopkUnroll; ++u) {
                const int c = cbase + u * kThreads + tid;
                if (c >= c_end) continue;
                const uint32_t id0 = (uint32_t)(sp.head + (int64_t)c * E::EPC);
                if (careful) {                                      // rare: re-read element by element
#pragma unroll 1
                    for (int q = 0; q < E::EPC; ++q)
                        if (slow_element(sh, s, flags, want_refresh, E::load(row, id0 + q), id0 + q)) dropped |= 1u << (u * E::EPC + q);
                    continue;
                }
                float f[E::EPC];
                E::unpack(w[u], f);
                const float cm = E::chunk_max(w[u]);
                if (cm > s.tmax && cm < INFINITY) raise_reference(s, cm);
                float e[E::EPC];
#pragma unroll
                for (int q = 0; q < E::EPC; ++q) e[q] = exp2_term(f[q], s.negc);
                if (cm >= thrv) {                                   // some element may be a candidate
#pragma unroll
                    for (int q = 0; q < E::EPC; ++q) {
                        if (f[q] >= thrv) {
                            const uint32_t r = take_candidate(sh, f[q], id0 + q, thrk, KP);
                            if (r & kTakeExclude) e[q] = 0.0f;      // candidates stay out of the fast sum
                            if (r & kTakeDropped) dropped |= 1u << (u * E::EPC + q);
                            if (r & kTakeRefresh) want_refresh = true;
                            flags |= r >> 8;
                        }
                    }
                }
                float sum = (e[0] + e[1]) + (e[2] + e[3]);
                if constexpr (E::EPC == 8) sum += (e[4] + e[5]) + (e[6] + e[7]);
                s.acc += (double)sum;
            }
            if (__syncthreads_or(want_refresh || dropped != 0)) {
                want_refresh = false;
                for (;;) {
                    s = refresh_candidates(sh, s, KP);
                    uint32_t again = 0;
                    while (dropped) {                               // retry what did not fit
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
            }
#pragma unroll
            for (int u = 0; u < kTopkUnroll; ++u) w[u] = wn[u];
        }
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
