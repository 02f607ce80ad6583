// Fused softmax statistics + top-K over the vocabulary of every live (request, position) row
// (Eq. 1: q_i = softmax(l_i); Algorithm 1, Require: top-K tokens and log-probs per position).
//
// One pass over the logits.  A row is cut into S segments; one CTA handles one (row, segment) and
// leaves a record in the workspace (SegRecord below):
//   - a short, unsorted list of candidate keys (logit descending, token id ascending as one 64-bit integer) that is
//     guaranteed to contain the KP best elements of the segment,
//   - per warp, W and C with  sum over the warp's share of all OTHER finite elements of 2^(x*log2(e) - C) = W
//     (fp64 W, integer C).
// The expansion kernel merges the records of a row: it ranks the candidates, takes the exponential of every listed
// candidate in fp64 and adds the warps' sums.  The candidates are kept out of W on purpose, so that the fp32
// exponentials used here only ever cover the part of the mass that is spread over many small terms.
//
// Data path: one elected thread streams the segment into a ring of shared-memory tiles with bulk asynchronous copies
// (cp.async.bulk into this CTA's own shared memory, completion on an mbarrier); a per-stage counter tells when all
// warps are done with a stage, and the last of them refills it.  Warps advance through the tiles on their own.  A CTA
// is four warps with a ring of three 8 KB tiles, eight CTAs to an SM: while one CTA finishes its segment (the serial
// part below), seven others stream.
//
// The streaming loop does no selection at all.  Per thread and tile (four 16-byte chunks = 32 bf16 / 16 fp32): one
// packed max over all elements, folded into the thread's running maximum and, across the warp, into a table with one
// entry per (tile, warp); per element two FMAs (x*log2e split in hi+lo, minus ONE reference exponent fixed for the
// whole segment after its first tile; issued as packed fma.rn.f32x2), one ex2.approx, packed adds; the fp32 sum of
// the tile goes to an fp64 accumulator.
// When the segment has gone by, the KP-th largest of the threads' maxima -- maxima of disjoint parts of the segment,
// hence values of distinct elements -- is a lower bound T of the segment's KP-th best element.  Only the (tile, warp)
// parts whose table entry reaches T can hold an element at or above T: there are about as many as such elements
// (16 or 17 of the 152 parts of a 150k-element row at KP = 16).  They are read once more (2 KB each, from L2), every
// element at or above T becomes a candidate, and its term -- recomputed with the same reference exponent, hence
// bit-identical to the one that was added -- is taken out of the sums again.
//
// If a sum comes out non-finite (NaN or +Inf in the input, or logits so far above the first tile's that 2^t
// overflows), or there are more candidates or hot parts than the buffers hold, the segment is redone by the careful
// path: element by element from global memory, with a CTA-wide barrier protocol that compacts a candidate buffer as
// it goes.  Slow, but correct for every input.
#pragma once
#include "common.cuh"
#include "tile_ring.cuh"

namespace cadd {

constexpr int kTkThreads = 128;                           // threads per CTA of the softmax/top-K kernel
constexpr int kTkTileChunks = kTopkUnroll * kTkThreads;   // 16-byte chunks per tile of its ring
constexpr int kCandCap = 512;             // careful path: candidate buffer entries per CTA
constexpr int kTkWarps = kTkThreads / 32;
constexpr int kPartCap = 64 * kTkWarps;   // fast path: entries of the table of per-(tile group, warp) maxima
constexpr int kHotCap = 128;              // fast path: parts read again at the end of a segment
constexpr int kMaxKP = 64;
constexpr int kWinCap = 4 * kMaxKP;       // entries handed over per segment at most (seg_key_cap(kMaxKP))

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

// Record of one (row, segment) as softmax_topk_partial_kernel leaves it: header, kSegSums pairs (W, C) -- one per warp;
// only the first n_sums are meaningful -- then up to seg_key_cap(KP) candidate keys in no particular order.
struct SegRecord {
    int32_t cnt;       // candidate keys that follow the sums
    uint32_t flags;    // kPart*
    int32_t n_sums;    // (W, C) pairs in use
    int32_t pad;
};
static_assert(sizeof(SegRecord) == 16, "SegRecord layout");
constexpr int kSegSums = 8;               // room for one pair per warp of the writing CTA
__host__ __device__ inline int seg_key_cap(int KP) { return 4 * KP; }
__host__ __device__ inline size_t seg_record_stride(int KP) { return sizeof(SegRecord) + (size_t)kSegSums * 16 + (size_t)seg_key_cap(KP) * 8; }

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

// What the end of a segment and the careful path keep in shared memory.  It lives in the tile ring, which is free by
// then: every tile has been consumed and no copy is in flight.
struct EndArea {
    uint64_t keys[kCandCap]; // careful path: candidate keys
    uint64_t win[kWinCap];   // what the segment hands over (careful path: the KP best, sorted, best first)
    unsigned hist[256];      // careful path: radix-select histogram
};

// Shared state of one CTA.
struct TopkShared {
    unsigned part_max[kPartCap];   // fast path: ord32 image of the largest value of every (tile group, warp) part; 0 = none
    unsigned short hot[kHotCap];   // fast path: parts that may hold an element at or above the bound T
    unsigned n_hot;
    alignas(16) float seeds[kTkThreads];   // the warps' sorted maxima while T is formed; afterwards eight 64-byte slots for the second look
    float bound;                   // T
    float tile0_max;
    unsigned count;          // careful path: entries in keys[]
    unsigned nwin;           // entries in win[]
    uint64_t thr_key;        // careful path: candidates must beat this key (0 = none yet)
    float thr_val;           // careful path: its logit value
    uint64_t sel_prefix;
    unsigned sel_need;
    unsigned timeout;        // a bounded wait ran out
    unsigned redo;           // fast path: too many hot parts or candidates, or a sum came out non-finite
    unsigned flags_all;      // OR of the threads' kPart* flags
    double red_d[kTkWarps];
    float red_f[kTkWarps];
    unsigned red_u[kTkWarps];
    alignas(8) uint64_t full[kStages];                 // mbarriers: tile landed
    unsigned released[kStages];                        // warps done with the stage's current tile
    unsigned last_seq[kStages];                        // last tile issued into the stage (see ring_drain)
    alignas(128) uint4 ring[kStages][kTkTileChunks];     // tiles of logits
    __device__ __forceinline__ EndArea& end() { return *reinterpret_cast<EndArea*>(&ring[0][0]); }
};
static_assert(sizeof(EndArea) <= sizeof(uint4) * kStages * kTkTileChunks, "the end-of-segment area must fit in the ring");


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
        sh.end().keys[pos] = key;
        want_refresh = true;
        return false;
    }
    fold_scalar(s, x);
    return false;
}

// Order-preserving image of a logit's value alone (-0 and +0 are the same value).
__device__ __forceinline__ uint32_t ord_value(float x) {
    uint32_t b = __float_as_uint(x);
    if (b == 0x80000000u) b = 0;
    return ord32(b);
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
        uint64_t mine[kCandCap / kTkThreads];
#pragma unroll
        for (int q = 0; q < kCandCap / kTkThreads; ++q) mine[q] = tid + q * kTkThreads < n ? sh.end().keys[tid + q * kTkThreads] : 0ull;
        if (tid == 0) sh.nwin = 0;
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kCandCap / kTkThreads; ++q) {
            if (mine[q] == 0ull) continue;
            if (mine[q] >= thr) sh.end().keys[atomicAdd(&sh.nwin, 1u)] = mine[q];
            else fold_scalar(s, key_value(mine[q]));
        }
        __syncthreads();
        n = (int)sh.nwin;
        __syncthreads();
    }
    uint64_t kth;
    if (n <= kTkThreads) {
        // rank by counting, one thread per entry (keys are unique); every entry is read as a broadcast
        if (tid < n) {
            const uint64_t k = sh.end().keys[tid];
            int rank = 0;
            for (int j = 0; j < n; ++j) rank += sh.end().keys[j] > k;
            if (rank < KP) sh.end().win[rank] = k;
            else fold_scalar(s, key_value(k));
        }
        __syncthreads();
        kth = sh.end().win[KP - 1];
    } else {
        if (tid == 0) { sh.sel_prefix = 0; sh.sel_need = KP; sh.nwin = 0; }
        uint64_t mask = 0;
        for (int shift = 56; shift >= 0; shift -= 8) {
            for (int q = tid; q < 256; q += kTkThreads) sh.end().hist[q] = 0;
            __syncthreads();
            const uint64_t prefix = sh.sel_prefix;
            for (int i = tid; i < n; i += kTkThreads) {
                uint64_t k = sh.end().keys[i];
                if ((k & mask) == prefix) atomicAdd(&sh.end().hist[(unsigned)(k >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (tid < 32) {
                // lane l owns digits 8l..8l+7; find the largest digit d with (count of digits > d) < need
                unsigned h[8], tot = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { h[q] = sh.end().hist[tid * 8 + q]; tot += h[q]; }
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
        for (int i = tid; i < n; i += kTkThreads) {
            uint64_t k = sh.end().keys[i];
            if (k >= kth) sh.end().win[atomicAdd(&sh.nwin, 1u)] = k;
            else fold_scalar(s, key_value(k));
        }
        __syncthreads();
        if (tid < KP) {                                        // sort the KP survivors by counting
            const uint64_t k = sh.end().win[tid];
            int rank = 0;
            for (int q = 0; q < KP; ++q) rank += sh.end().win[q] > k;
            sh.end().keys[kCandCap - kMaxKP + rank] = k;             // park them at the end of the buffer
        }
        __syncthreads();
        if (tid < KP) sh.end().win[tid] = sh.end().keys[kCandCap - kMaxKP + tid];
        __syncthreads();
    }
    if (tid < KP) sh.end().keys[tid] = sh.end().win[tid];
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
    for (int cbase = c_begin; cbase < c_end; cbase += kTkThreads) {
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
        const uint64_t k = sh.end().keys[tid];
        int rank = 0;
        for (int q = 0; q < cnt; ++q) rank += sh.end().keys[q] > k;
        sh.end().win[rank] = k;
    }
    if (tid == 0) sh.nwin = cnt;
    __syncthreads();
    *flags_out = flags;
    return s;
}

// End of a segment, one element that did not go through the tile stream (the ragged ends of a row): at or above the
// bound it becomes a candidate, below it its term joins the caller's sum; infinities and NaN carry no mass and are
// flagged.
__device__ __forceinline__ void settle_scalar(TopkShared& sh, double& acc, uint32_t& flags, float x, uint32_t id, float bound, float negc) {
    const uint32_t b = __float_as_uint(x);
    if ((b & 0x7f800000u) == 0x7f800000u) {
        if (b != 0xff800000u) flags |= kPartNonfinite;    // anything but -Inf
        if (b == 0x7f800000u) flags |= kPartPosInf;
        return;
    }
    if (x >= bound) {
        const unsigned pos = atomicAdd(&sh.nwin, 1u);
        if (pos < (unsigned)kWinCap) sh.end().win[pos] = make_key(x, id);
        else sh.redo = 1;
    } else {
        acc += (double)exp2_term(x, negc);
    }
}

template <int DT>
__global__ void __launch_bounds__(kTkThreads, 1024 / kTkThreads) softmax_topk_partial_kernel(TopkParams p) {
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
    const int n_tiles = (c_end - c_begin + kTkTileChunks - 1) / kTkTileChunks;
    const int group = (n_tiles * (kTkWarps) + kPartCap - 1) / kPartCap > 1 ? (n_tiles * (kTkWarps) + kPartCap - 1) / kPartCap : 1;   // tiles per table entry

    if (tid == 0) {
        for (int q = 0; q < kStages; ++q) { mbar_init(&sh.full[q], 1); sh.released[q] = 0; sh.last_seq[q] = kNoTile; }
        sh.timeout = 0; sh.n_hot = 0; sh.nwin = 0; sh.redo = 0; sh.flags_all = 0;
        sh.count = 0; sh.thr_key = 0; sh.thr_val = -INFINITY;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // one thread issues tile t into stage t % kStages: thread 0 for the first kStages tiles, afterwards
    // lane 0 of whichever warp is the last to finish with the tile that occupied the stage
    const int fault_tile = p.fault_tile < 0 ? -1 : min(p.fault_tile, n_tiles - 1);
    auto issue_tile = [&](int t) {
        if (t == fault_tile) return;                                   // test hook: this copy is never made
        const int c0 = c_begin + t * kTkTileChunks;
        const unsigned bytes = (unsigned)min(kTkTileChunks, c_end - c0) * 16u;
        const unsigned st = (unsigned)t % kStages;
        *(volatile unsigned*)&sh.last_seq[st] = (unsigned)t;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic reads of the stage are done
        mbar_arrive_expect_tx(&sh.full[st], bytes);
        bulk_load(&sh.ring[st][0], body + c0, bytes, &sh.full[st]);
    };
    if (tid == 0)
        for (int t = 0; t < kStages && t < n_tiles; ++t) issue_tile(t);

    const uint64_t l2e_hi2 = pack2(kLog2eHi, kLog2eHi), l2e_lo2 = pack2(kLog2eLo, kLog2eLo);
    double acc = 0.0;                 // this thread's sum of 2^(x*log2e - c) over the tiles
    float tmaxv = -INFINITY;          // this thread's largest element (NaN ignored)
    float negc = 0.0f;                // -c: the reference exponent, one for the whole segment
    uint32_t flags = 0;

    // ================= fast path: warps advance on their own =================
    {
        // The reference exponent comes from the first tile: c = ceil(max of tile 0 * log2e) + 1.  Later elements may
        // exceed it by almost 90 before 2^t overflows (which the end of the segment notices); elements more than 87
        // below it count as zero, as they should.  Fixed once, it makes every term reproducible bit for bit.
        bool landed = true;
        if (n_tiles > 0) {
            landed = __all_sync(kFullMask, mbar_wait_limited(&sh.full[0], 0, tile_wait_limit(0, fault_tile)));
            float v = -INFINITY;
            if (landed) {
#pragma unroll
                for (int u = 0; u < kTopkUnroll; ++u)
                    if (c_begin + u * kTkThreads + tid < c_end) v = fmaxf(v, E::chunk_max(sh.ring[0][u * kTkThreads + tid]));
                if (!(fabsf(v) < INFINITY)) v = -INFINITY;             // NaN or Inf: no help from this thread
            } else if (lane == 0) {
                sh.timeout = 1;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
            if (lane == 0) sh.red_f[warp] = v;
            __syncthreads();
            v = sh.red_f[lane % kTkWarps];
#pragma unroll
            for (int o = kTkWarps / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
            if (v > -INFINITY) negc = -(ceilf(fminf(v, 2.0e38f) * kLog2eHi) + 1.0f);
        }
        const uint64_t negc2 = pack2(negc, negc);

        unsigned st = 0, phase = 0;
        unsigned pm = 0;                                                     // running maximum of this warp's part (ord32 image)
        int pe = warp, in_group = 0;                                         // its table entry, and how many tiles of the entry's group have gone by
        for (int t = 0; t < n_tiles && landed; ++t, st = (st + 1 == kStages ? 0u : st + 1), phase ^= (st == 0 ? 1u : 0u)) {
            const bool here = __all_sync(kFullMask, mbar_wait_limited(&sh.full[st], phase, tile_wait_limit(t, fault_tile)));
            if (!here) { sh.timeout = 1; break; }
            const int cbase = c_begin + t * kTkTileChunks;
            const uint4* tile = &sh.ring[st][tid];
            // this thread's chunks of the tile; chunks past the end of the segment read as -Inf (no mass, never
            // a candidate), so that one code path serves whole and ragged tiles
            const uint4 kNone = DT == CADD_DTYPE_BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                                                      : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
            uint4 w0, w1, w2, w3;
            if (cbase + kTkTileChunks <= c_end) {                          // CTA-uniform: every chunk of the tile is valid
                w0 = tile[0]; w1 = tile[kTkThreads]; w2 = tile[2 * kTkThreads]; w3 = tile[3 * kTkThreads];
            } else {
                const int nv = c_end - (cbase + tid);                    // > u * kTkThreads  <=>  chunk u is valid
                w0 = nv > 0 ? tile[0] : kNone;
                w1 = nv > kTkThreads ? tile[kTkThreads] : kNone;
                w2 = nv > 2 * kTkThreads ? tile[2 * kTkThreads] : kNone;
                w3 = nv > 3 * kTkThreads ? tile[3 * kTkThreads] : kNone;
            }
            const float mx = E::max4(w0, w1, w2, w3);
            tmaxv = fmaxf(tmaxv, mx);
            // the largest value of this (tile, warp) part goes to the table (several tiles share an entry on very long rows)
            pm = max(pm, __reduce_max_sync(kFullMask, ord_value(mx)));
            if (lane == 0) sh.part_max[pe] = pm;
            if (++in_group == group) { in_group = 0; pe += kTkWarps; pm = 0; }
            {
                const uint64_t a = add2(chunk_exp_sum2<DT>(w0, l2e_hi2, l2e_lo2, negc2),
                                        chunk_exp_sum2<DT>(w1, l2e_hi2, l2e_lo2, negc2));
                const uint64_t c2 = add2(chunk_exp_sum2<DT>(w2, l2e_hi2, l2e_lo2, negc2),
                                         chunk_exp_sum2<DT>(w3, l2e_hi2, l2e_lo2, negc2));
                float lo, hi;
                unpack2(add2(a, c2), lo, hi);
                acc += (double)(lo + hi);
            }
            __syncwarp();
            // This warp is done with the stage: its loads from it have returned (their values were consumed above).
            // The last warp to say so refills the stage.
            if (lane == 0) {
                __threadfence_block();
                if (atomicAdd(&sh.released[st], 1u) == kTkWarps - 1) {
                    atomicExch(&sh.released[st], 0u);
                    __threadfence_block();
                    if (t + kStages < n_tiles) issue_tile(t + kStages);
                }
            }
        }
    }

    // ================= end of the segment =================
    // (1) every warp has left the tile loop: the table is complete, the ring is free
    __syncthreads();
    const bool timed_out = sh.timeout != 0;
    if (tid == 0 && timed_out) ring_drain(sh.full, sh.last_seq);   // a wait ran out: let the copies still in flight land
    // The bound T: the KP-th largest of the 256 threads' maxima.  Each warp sorts its 32 over the lanes (bitonic network);
    // for KP <= 32 warp 0 folds the eight sorted lists together, keeping the 32 largest (elementwise max of one list with
    // the other reversed, then one bitonic merge); for larger KP T is the smallest, over the warps, of a warp's
    // ceil(KP / warps)-th largest.  Either way at least KP distinct elements of the segment reach T.
    {
        float v = tmaxv;
        if (!(fabsf(v) < INFINITY)) v = -INFINITY;                 // NaN or Inf: no help from this thread
#pragma unroll
        for (int blk = 2; blk <= 32; blk <<= 1) {
#pragma unroll
            for (int j = blk >> 1; j > 0; j >>= 1) {
                const float other = __shfl_xor_sync(kFullMask, v, j);
                const bool take_max = ((lane & j) != 0) == ((lane & blk) != 0);
                v = take_max ? fmaxf(v, other) : fminf(v, other);
            }
        }
        sh.seeds[tid] = v;                                         // lane q of a warp: its q-th largest
        __syncthreads();                                           // (2)
        if (KP <= 32) {
            // three rounds of pairwise merges: warps 0,2,4,6 take in their right neighbour's list, then 0 and 4, then 0
#pragma unroll
            for (int step = 1; step < kTkWarps; step <<= 1) {
                if ((warp & (2 * step - 1)) == 0) {
                    v = fmaxf(v, sh.seeds[(warp + step) * 32 + 31 - lane]);    // the 32 largest of both lists, as a bitonic sequence
#pragma unroll
                    for (int j = 16; j > 0; j >>= 1) {
                        const float other = __shfl_xor_sync(kFullMask, v, j);
                        v = (lane & j) == 0 ? fmaxf(v, other) : fminf(v, other);
                    }
                    if (2 * step < kTkWarps) sh.seeds[tid] = v;
                }
                if (2 * step < kTkWarps) __syncthreads();
            }
            if (warp == 0) {
                v = __shfl_sync(kFullMask, v, KP - 1);
                if (lane == 0) sh.bound = v;
            }
        } else if (warp == 0) {
            v = sh.seeds[(lane % kTkWarps) * 32 + (KP + kTkWarps - 1) / kTkWarps - 1];
#pragma unroll
            for (int o = kTkWarps / 2; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(kFullMask, v, o));
            if (lane == 0) sh.bound = v;
        }
        __syncthreads();                                           // (3)
    }
    const float bound = sh.bound;
    const int cap = seg_key_cap(KP);
    double sub = 0.0;                                              // terms of candidates, to be taken out of the sums again
    if (!timed_out) {
        // the parts that can hold an element at or above the bound
        const unsigned bound_ord = bound > -INFINITY ? ord_value(bound) : 0u;
        const int n_parts = ((n_tiles + group - 1) / group) * (kTkWarps);
        for (int e = tid; e < n_parts; e += kTkThreads) {
            if (sh.part_max[e] >= bound_ord) {
                const unsigned pos = atomicAdd(&sh.n_hot, 1u);
                if (pos < (unsigned)kHotCap) sh.hot[pos] = (unsigned short)e;
                else sh.redo = 1;
            }
        }
        __syncthreads();                                           // (4)
        // Read them once more (from L2), two parts per warp at a time with all loads issued before any is used.  A lane
        // that holds an element at or above the bound hands its 32 elements to the whole warp, one element per lane
        // (through a small shared-memory slot).  A candidate's term is recomputed -- same instructions, same reference
        // exponent: the same bits as in the stream -- and taken out of the sums again.  (What stays behind is the
        // rounding of the one fp32 tile sum the term went through: at most 6e-8 of the term.)
        constexpr int NE = kTopkUnroll * E::EPC;                   // elements per thread and tile: 32 or 16
        const int nh = min((int)sh.n_hot, kHotCap);
        uint4* slot = reinterpret_cast<uint4*>(sh.seeds) + warp * kTopkUnroll;   // this warp's 64 bytes (the seeds are no longer needed)
        const int u_of = lane / E::EPC, q_of = lane % E::EPC;
        for (int h0 = warp; h0 < nh; h0 += 2 * (kTkWarps)) {
            uint4 wv[2][kTopkUnroll];
            int cbs[2], ngrp[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int h = h0 + k * (kTkWarps);
                const int e = h < nh ? sh.hot[h] : 0;
                const int g = e / (kTkWarps), w = e - g * (kTkWarps);
                ngrp[k] = h < nh ? min((g + 1) * group, n_tiles) - g * group : 0;     // tiles behind this table entry (1 unless the row is very long)
                cbs[k] = c_begin + g * group * kTkTileChunks + w * 32;
#pragma unroll
                for (int u = 0; u < kTopkUnroll; ++u) {
                    const int c = cbs[k] + u * kTkThreads + lane;
                    wv[k][u] = (ngrp[k] > 0 && c < c_end) ? __ldg(body + c) : (DT == CADD_DTYPE_BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                                                                                                          : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u));
                }
            }
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                for (int tt = 0; tt < ngrp[k]; ++tt) {
                    const int cb = cbs[k] + tt * kTkTileChunks;
                    if (tt > 0) {                                  // very long rows only: the further tiles of the group
#pragma unroll
                        for (int u = 0; u < kTopkUnroll; ++u) {
                            const int c = cb + u * kTkThreads + lane;
                            wv[k][u] = c < c_end ? __ldg(body + c) : (DT == CADD_DTYPE_BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                                                                                             : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u));
                        }
                    }
                    const float m = E::max4(wv[k][0], wv[k][1], wv[k][2], wv[k][3]);
                    unsigned hits = __ballot_sync(kFullMask, m >= bound);
                    while (hits) {
                        const int src = __ffs(hits) - 1;
                        hits &= hits - 1;
                        __syncwarp();
                        if (lane == src) { slot[0] = wv[k][0]; slot[1] = wv[k][1]; slot[2] = wv[k][2]; slot[3] = wv[k][3]; }
                        __syncwarp();
                        float x = -INFINITY;                       // lanes beyond the 16 elements of an fp32 thread-tile: no term
                        if (lane < NE) x = E::load(slot + u_of, q_of);
                        const int c = cb + u_of * kTkThreads + src;
                        const bool cand = lane < NE && c < c_end && x >= bound && fabsf(x) < INFINITY;
                        if (cand) {
                            const unsigned pos = atomicAdd(&sh.nwin, 1u);
                            if (pos < (unsigned)kWinCap) sh.end().win[pos] = make_key(x, (uint32_t)(sp.head + (int64_t)c * E::EPC + q_of));
                            else sh.redo = 1;
                        }
                        if (cand) sub += (double)exp2_term(x, negc);   // the very bits the stream added
                    }
                }
            }
        }
        // the ragged ends of the row, one element per thread (segment 0 takes the head, the last one the tail)
        if (seg == 0 && tid < sp.head) settle_scalar(sh, acc, flags, E::load(row, tid), (uint32_t)tid, bound, negc);
        if (seg == p.S - 1 && tid < sp.tail) {
            const int64_t e = p.V - sp.tail + tid;
            settle_scalar(sh, acc, flags, E::load(row, e), (uint32_t)e, bound, negc);
        }
    }
    flags = __reduce_or_sync(kFullMask, flags);
    if (lane == 0 && flags) atomicOr(&sh.flags_all, flags);
    __syncthreads();                                               // (5) the candidates are all in win[]
    const uint64_t* hand = sh.end().win;                           // what is handed over, and how many
    int cnt = min((int)sh.nwin, kWinCap);
    if (!timed_out && cnt > cap) {
        // more than a record holds (many equal values at the bound, very short rows): keep exactly the KP best, ranked
        // by counting (keys are unique); the terms of the others go back into the sums
        for (int e = tid; e < cnt; e += kTkThreads) {
            const uint64_t k = sh.end().win[e];
            int rank = 0;
            for (int j = 0; j < cnt; ++j) rank += sh.end().win[j] > k;
            if (rank < KP) sh.end().keys[rank] = k;
            else acc += (double)exp2_term(key_value(k), negc);
        }
        hand = sh.end().keys;
        cnt = KP;
    }
    // the warp's sum; the reference exponent is the same for all
    unsigned char* rec = p.partials + (size_t)item * seg_record_stride(KP);
    double* rec_sums = (double*)(rec + sizeof(SegRecord));
    uint64_t* rec_keys = (uint64_t*)(rec + sizeof(SegRecord) + (size_t)kSegSums * 16);
    {
        double part = acc - sub;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFullMask, part, o);
        if (lane == 0) {
            if (!(part == part && fabs(part) < INFINITY)) sh.redo = 1;   // NaN, +Inf or an overflowing term went through the fast path
            rec_sums[2 * warp] = part * kEx2BiasFix;
            rec_sums[2 * warp + 1] = (double)(-negc);
        }
    }
    __syncthreads();                                               // (6)
    flags = sh.flags_all;
    const bool redo = !timed_out && sh.redo != 0;

    if (!redo) {
        if (timed_out) cnt = 0;
        for (int e = tid; e < cnt; e += kTkThreads) rec_keys[e] = hand[e];
        if (tid == 0) {
            SegRecord h;
            h.cnt = cnt; h.flags = flags | (timed_out ? kPartTimeout : 0u); h.n_sums = timed_out ? 0 : kTkWarps; h.pad = 0;
            *(SegRecord*)rec = h;
        }
        return;
    }

    // ================= careful path: element by element from global memory, CTA-wide protocol =================
    ThreadSum s = careful_segment<DT>(sh, row, sp, p.V, seg, p.S, c_begin, c_end, KP, &flags);
    // CTA combine: common reference C = max c_t, W = sum acc_t * 2^(c_t - C)
    {
        float c_t = (s.acc != 0.0) ? -s.negc : -INFINITY;
        float cm = c_t;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(kFullMask, cm, o));
        if (lane == 0) sh.red_f[warp] = cm;
        __syncthreads();
        cm = sh.red_f[0];
#pragma unroll
        for (int q = 1; q < kTkWarps; ++q) cm = fmaxf(cm, sh.red_f[q]);
        double part = (s.acc != 0.0) ? scalbn(s.acc, (int)fmaxf(c_t - cm, -4000.0f)) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFullMask, part, o);
        uint32_t fl = __reduce_or_sync(kFullMask, flags);
        if (lane == 0) { sh.red_d[warp] = part; sh.red_u[warp] = fl; }
        __syncthreads();
        double W = 0.0;
        flags = 0;
#pragma unroll
        for (int q = 0; q < kTkWarps; ++q) { W += sh.red_d[q]; flags |= sh.red_u[q]; }
        const int ncare = (int)sh.nwin;
        if (tid < ncare) rec_keys[tid] = sh.end().win[tid];
        if (tid == 0) {
            rec_sums[0] = W * kEx2BiasFix;
            rec_sums[1] = (cm == -INFINITY) ? 0.0 : (double)cm;
            SegRecord h;
            h.cnt = ncare; h.flags = flags; h.n_sums = 1; h.pad = -1;
            *(SegRecord*)rec = h;
        }
    }
}

}  // namespace cadd
