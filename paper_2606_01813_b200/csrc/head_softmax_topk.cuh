// Softmax statistics and top-K of the draft positions fused into the drafter's output projection (Eq. 1 and
// Algorithm 1's "Require", computed from the drafter's last hidden states instead of materialised logits).
// The logits l_i = h_i . W^T are formed tile by tile on the tensor cores exactly as in head_argmax.cuh (same TMA
// ring, same tcgen05.mma issue, accumulators in tensor memory); the epilogue turns every row of a tile into running
// softmax / top-K state instead of a single maximum:
//   - the KP best (logit, token) pairs of the row so far, a small unsorted list per row in shared memory with its
//     smallest entry cached; elements that reach the threshold are queued per row and folded into the list by the
//     whole warp at once, so the rare list update does not split the warp element by element;
//   - W = sum over all other elements of 2^(x*log2e - C) with an integer reference exponent C, accumulated in fp64
//     from fp32 exponentials (ex2.approx), the same split as in softmax_topk.cuh: the KP best are never put through
//     the fp32 exponential.
// A work item is (row tile, chunk of consecutive column tiles): the row state lives across the chunk's tiles and is
// written as one partial record per (row, chunk) in the format of softmax_topk.cuh.  A second kernel folds a row's
// chunk records into one record, which the expansion kernel then reads with S = 1.
#pragma once
#include "head_argmax.cuh"
#include "softmax_topk.cuh"

namespace cadd {

constexpr int kDraftMaxRecords = 96;      // chunk records per row the merge kernel can fold (three lists per lane)
constexpr int kDraftMaxKP = 32;           // list capacity per row that fits beside the operand ring in shared memory

constexpr int kDraftStages = 4;           // operand ring as in head_argmax.cuh: about 190 KB in flight cover the TMA latency
constexpr int kDraftPending = 8;          // queued candidates per row and column half between two list updates
constexpr int kDraftThreads = 320;        // producer warp, MMA warp, eight epilogue warps

struct DraftHeadShared {
    alignas(1024) unsigned char a[kDraftStages][kHeadABytes];
    alignas(1024) unsigned char b[kDraftStages][kHeadBBytes];
    // The rows' lists of best keys, unsorted: list[(half * KP + k) * 128 + row of the tile].  32 KB is what is left
    // beside four operand stages: for KP <= 16 two epilogue warps share each group of 32 rows and split the tile's
    // columns in halves, each half with its own row state and its own record; for KP <= 32 one warp takes all columns.
    uint64_t list[2 * 16 * kHeadBM];
    alignas(8) uint64_t full[kDraftStages];
    uint64_t empty[kDraftStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t error;
};
inline size_t draft_head_smem_bytes() { return sizeof(DraftHeadShared) + 1024; }

struct DraftHeadParams {
    int64_t M;                 // rows = batch * L
    int64_t V;
    int Kdim;                  // hidden size
    int m_tiles, n_tiles;
    int chunk_tiles;           // column tiles per chunk
    int n_chunks;              // chunks per row = ceil(n_tiles / chunk_tiles)
    int L, KP;
    const int32_t* l_eff;      // [batch] or NULL
    uint64_t* pend;            // [gridDim][2][kDraftPending][128] scratch: candidates waiting for the next list update
                               // (global memory: written on a hit, read back once per tile; L1/L2-resident)
    int halves;                // column halves per tile handled by separate epilogue warps: 2 (KP <= 16) or 1
    unsigned char* chunk_partials;   // [M * n_chunks * halves] records of seg_partial_stride(KP) bytes
    int32_t* error;
};

// r[i] for a run-time i, without spilling the array: a binary tree of selects (31 of them).
__device__ __forceinline__ uint32_t pick32(const uint32_t (&r)[32], int i) {
    uint32_t a[16], b[8], c[4];
#pragma unroll
    for (int j = 0; j < 16; ++j) a[j] = (i & 1) ? r[2 * j + 1] : r[2 * j];
#pragma unroll
    for (int j = 0; j < 8; ++j) b[j] = (i & 2) ? a[2 * j + 1] : a[2 * j];
#pragma unroll
    for (int j = 0; j < 4; ++j) c[j] = (i & 4) ? b[2 * j + 1] : b[2 * j];
    const uint32_t d0 = (i & 8) ? c[1] : c[0], d1 = (i & 8) ? c[3] : c[2];
    return (i & 16) ? d1 : d0;
}

// Row r = b * L + i is read iff i < l_eff[b].
__device__ __forceinline__ bool draft_row_live(const DraftHeadParams& p, int64_t r) {
    if (r >= p.M) return false;
    if (!p.l_eff) return true;
    const int64_t b = r / p.L;
    int clamped;
    return (int)(r - b * p.L) < clamp_l_eff(p.l_eff, (int)b, p.L, &clamped);
}
__device__ __forceinline__ bool draft_tile_live(const DraftHeadParams& p, int mt) {
    if (!p.l_eff) return true;
    const int64_t r0 = (int64_t)mt * kHeadBM, r1 = min(r0 + kHeadBM, p.M);
    for (int64_t r = r0; r < r1; ++r)
        if (draft_row_live(p, r)) return true;
    return false;
}

__global__ void __launch_bounds__(kDraftThreads, 1)
head_softmax_topk_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, DraftHeadParams p) {
    extern __shared__ __align__(16) unsigned char head_smem_raw[];
    DraftHeadShared& sh = *reinterpret_cast<DraftHeadShared*>(head_smem_raw + ((1024u - (smem_u32(head_smem_raw) & 1023u)) & 1023u));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k_steps = (p.Kdim + kHeadBK - 1) / kHeadBK;
    const int64_t n_items = (int64_t)p.m_tiles * p.n_chunks;      // item w -> (chunk = w / m_tiles, row tile = w % m_tiles)
    const int KP = p.KP;

    if (tid == 0) {
        for (int s = 0; s < kDraftStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sh.acc_full[s], 1); mbar_init(&sh.acc_empty[s], 4 * p.halves); }
        sh.error = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&sh.tmem_base, kHeadTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *(volatile uint32_t*)&sh.tmem_base;

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            unsigned s = 0, ph = 0;
            for (int64_t w = blockIdx.x; w < n_items && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
                const int ch = (int)(w / p.m_tiles), mt = (int)(w - (int64_t)ch * p.m_tiles);
                if (!draft_tile_live(p, mt)) continue;
                const int nt1 = min((ch + 1) * p.chunk_tiles, p.n_tiles);
                for (int nt = ch * p.chunk_tiles; nt < nt1 && !*(volatile uint32_t*)&sh.error; ++nt)
                    if (!head_produce_tile<DraftHeadShared, kDraftStages>(sh, &map_h, &map_w, mt, nt, k_steps, s, ph)) { sh.error = 1; break; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            unsigned s = 0, ph = 0, buf = 0, aph = 0;
            for (int64_t w = blockIdx.x; w < n_items && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
                const int ch = (int)(w / p.m_tiles), mt = (int)(w - (int64_t)ch * p.m_tiles);
                if (!draft_tile_live(p, mt)) continue;
                const int nt1 = min((ch + 1) * p.chunk_tiles, p.n_tiles);
                for (int nt = ch * p.chunk_tiles; nt < nt1 && !*(volatile uint32_t*)&sh.error; ++nt) {
                    if (!head_wait(&sh.acc_empty[buf], aph ^ 1u)) { sh.error = 2; break; }
                    tc_fence_after();
                    if (!head_mma_tile<DraftHeadShared, kDraftStages>(sh, tmem_base + buf * kHeadBN, &sh.acc_full[buf], k_steps, s, ph)) { sh.error = 3; break; }
                    if (++buf == 2) { buf = 0; aph ^= 1u; }
                }
            }
        }
    } else {
        // ---------------- epilogue: warps 2..9; thread = one row of the tile, one half of its columns ----------------
        const int quarter = warp & 3;                            // tensor-memory lane quarter this warp may read
        const int half = (warp - 2) >> 2;                        // columns [half * 128, half * 128 + 128) of every tile
        const int trow = quarter * 32 + lane;                    // row inside the tile = tensor-memory lane
        uint64_t* list = &sh.list[(size_t)half * KP * kHeadBM + trow];                        // this thread's column of the list
        uint64_t* pend = p.pend + (((size_t)blockIdx.x * 2 + half) * kDraftPending) * kHeadBM + trow;
        const int width = kHeadBN / p.halves;                    // columns of a tile this warp handles
        unsigned buf = 0, aph = 0;
        for (int64_t w = blockIdx.x; w < n_items && half < p.halves && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
            const int ch = (int)(w / p.m_tiles), mt = (int)(w - (int64_t)ch * p.m_tiles);
            if (!draft_tile_live(p, mt)) continue;
            const int64_t row = (int64_t)mt * kHeadBM + trow;
            const bool live = draft_row_live(p, row);
            // row state over the chunk
            ThreadSum s{0.0, -INFINITY, 0.0f};
            uint32_t flags = 0;
            int cnt = 0;                                          // entries in the row's list
            float thr = -INFINITY;                                // hit test: value of the list's smallest entry at the last update
            uint64_t thr_key = 0;                                 // the smallest entry itself (list full), at slot min_pos
            int min_pos = 0;
            int np = 0;                                           // queued candidates
            // Folds the queue into the list.  It runs once per tile for all lanes together (lanes with fewer entries
            // idle), and otherwise only when a lane's queue is full, so the rare, expensive list update does not split
            // the warp element by element.  The list is unsorted with its smallest entry cached: a better key
            // overwrites that slot and one scan finds the next smallest; whatever drops out, or never makes it in,
            // joins the sum.
            auto drain = [&]() {
                for (int j = 0; j < np; ++j) {
                    const uint64_t key = pend[(size_t)j * kHeadBM];
                    if (cnt < KP) {
                        list[(size_t)cnt * kHeadBM] = key;
                        ++cnt;
                        if (cnt < KP) continue;
                    } else if (key > thr_key) {
                        s.acc += (double)exp2_term(key_value(thr_key), s.negc);
                        list[(size_t)min_pos * kHeadBM] = key;
                    } else {
                        s.acc += (double)exp2_term(key_value(key), s.negc);
                        continue;
                    }
                    uint64_t mk = ~0ull;
                    int mp = 0;
#pragma unroll 4
                    for (int k = 0; k < KP; ++k) {
                        const uint64_t v = list[(size_t)k * kHeadBM];
                        if (v < mk) { mk = v; mp = k; }
                    }
                    thr_key = mk; min_pos = mp;
                    const float tv = key_value(mk);
                    if (tv > s.tmax + 60.0f || s.tmax == -INFINITY) raise_reference(s, tv);   // keeps 2^(x*log2e - c) in range below tv
                }
                np = 0;
                if (cnt == KP) thr = key_value(thr_key);
            };
            const int nt1 = min((ch + 1) * p.chunk_tiles, p.n_tiles);
            bool ok = true;
            for (int nt = ch * p.chunk_tiles; nt < nt1 && ok; ++nt) {
                if (!__all_sync(kFullMask, head_wait(&sh.acc_full[buf], aph, 256))) { sh.error = 4; ok = false; break; }
                tc_fence_after();
                const int64_t col0 = (int64_t)nt * kHeadBN + half * width;
                const bool inside = col0 + width <= p.V;          // no column of this warp's share is past the vocabulary
                // 32 columns per tensor-memory load (narrow loads have the same latency, about 2 k cycles while the
                // tensor cores run the next tile), the next 32 already on their way.  Pass 1 is branch-free: every
                // element below the threshold adds its exponential, the others set a bit.  Pass 2 runs only while
                // some lane has bits left: each lane takes one of its marked elements per turn and queues it (or sums
                // it, if a list update has raised the threshold meanwhile); when a lane's queue is full the whole warp
                // folds its queues into the lists and pass 2 goes on.
                const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kHeadBN + half * width;
                uint32_t r[32], rn[32];
                tmem_ld32(tbase, r);
                tmem_ld_wait();
#pragma unroll 1
                for (int c = 0; c < width / 32; ++c) {
                    if (c + 1 < width / 32) tmem_ld32(tbase + (c + 1) * 32, rn);
                    const int64_t cb = col0 + c * 32;
                    float part = 0.0f;                            // fp32 sum of this run of 32 columns
                    unsigned hit = 0;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float x = __uint_as_float(r[i]);
                        const bool valid = live && (inside || cb + i < p.V);
                        const bool fast = valid && x < thr;
                        part += exp2_term(fast ? x : -INFINITY, s.negc);              // 2^-inf = 0
                        hit |= (valid && !fast) ? (1u << i) : 0u;
                    }
                    s.acc += (double)part;
                    while (__any_sync(kFullMask, hit != 0)) {
                        // one marked element per lane and turn, fetched from the register file by a select tree
                        bool blocked = false;
                        if (hit) {
                            const int i = __ffs(hit) - 1;
                            const float x = __uint_as_float(pick32(r, i));
                            const uint32_t bits = __float_as_uint(x);
                            if ((bits & 0x7f800000u) == 0x7f800000u) {                // Inf or NaN: no mass, never a candidate
                                if (bits != 0xff800000u) flags |= kPartNonfinite;
                                if (bits == 0x7f800000u) flags |= kPartPosInf;
                                hit &= hit - 1;
                            } else if (x < thr) {                                     // the threshold has risen since pass 1
                                s.acc += (double)exp2_term(x, s.negc);
                                hit &= hit - 1;
                            } else if (np < kDraftPending) {
                                pend[(size_t)np * kHeadBM] = make_key(x, (uint32_t)(cb + i));
                                ++np;
                                hit &= hit - 1;
                            } else {
                                blocked = true;
                            }
                        }
                        if (__any_sync(kFullMask, blocked)) drain();                  // a queue is full: fold, then go on
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = rn[i];
                }
                drain();                                          // the accumulator's last candidates, then release it
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.acc_empty[buf]);
                if (++buf == 2) { buf = 0; aph ^= 1u; }
            }
            if (!ok) break;
            if (live) {
                unsigned char* rec = p.chunk_partials + (((size_t)row * p.n_chunks + ch) * p.halves + half) * seg_partial_stride(KP);
                uint64_t* out_keys = (uint64_t*)(rec + sizeof(SegPartial));
                for (int k = 0; k < cnt; ++k) {                     // rank by counting (keys are unique): sorted, best first
                    const uint64_t v = list[(size_t)k * kHeadBM];
                    int rank = 0;
                    for (int j = 0; j < cnt; ++j) rank += list[(size_t)j * kHeadBM] > v;
                    out_keys[rank] = v;
                }
                SegPartial h;
                h.W = s.acc * kEx2BiasFix; h.C = s.acc != 0.0 ? (double)(-s.negc) : 0.0; h.cnt = cnt;
                h.flags = flags; h.pad[0] = h.pad[1] = 0;
                *(SegPartial*)rec = h;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kHeadTmemCols);
    }
    if (tid == 0 && sh.error) atomicExch(p.error, (int32_t)sh.error);
}

// Folds the chunk records of one row into a single record (the format the expansion kernel reads with S = 1).
// One warp per row: the KP best keys come from a KP-step selection over the chunks' sorted lists (each lane walks
// up to two lists); every key that is not selected joins the sum through an fp64 exponential; the chunks' sums are
// brought to a common reference exponent.
__global__ void __launch_bounds__(128) draft_merge_kernel(DraftHeadParams p, unsigned char* merged) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= p.M || !draft_row_live(p, row)) return;
    const int KP = p.KP;
    const size_t stride = seg_partial_stride(KP);
    const double kLog2e = 1.4426950408889634;
    // lane owns records lane, lane + 32 and lane + 64 (at most kDraftMaxRecords per row)
    constexpr int NL = kDraftMaxRecords / 32;
    const SegPartial* hdr[NL];
    const uint64_t* keys[NL];
    int cnt[NL], cur[NL];
    double Cmax = -1e300;
    uint32_t flags = 0;
    int total = 0;
    for (int q = 0; q < NL; ++q) {
        cur[q] = 0;
        const int ch = lane + 32 * q;                            // record index: chunk * halves + column half
        if (ch < p.halves * p.n_chunks) {
            const unsigned char* rec = p.chunk_partials + ((size_t)row * p.n_chunks * p.halves + ch) * stride;
            hdr[q] = (const SegPartial*)rec;
            keys[q] = (const uint64_t*)(rec + sizeof(SegPartial));
            cnt[q] = hdr[q]->cnt;
            flags |= hdr[q]->flags;
            if (hdr[q]->W != 0.0) Cmax = fmax(Cmax, hdr[q]->C);
            total += cnt[q];
        } else { hdr[q] = nullptr; keys[q] = nullptr; cnt[q] = 0; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        total += __shfl_xor_sync(kFullMask, total, o);
        flags |= __shfl_xor_sync(kFullMask, flags, o);
    }
    unsigned char* out = merged + (size_t)row * stride;
    uint64_t* out_keys = (uint64_t*)(out + sizeof(SegPartial));
    const int n_out = min(KP, total);
    for (int k = 0; k < n_out; ++k) {
        uint64_t mine = 0ull;
        int from = 0;
#pragma unroll
        for (int q = 0; q < NL; ++q) {
            const uint64_t hq = cur[q] < cnt[q] ? keys[q][cur[q]] : 0ull;
            if (hq > mine) { mine = hq; from = q; }
        }
        uint64_t best = mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(kFullMask, best, o));
        if (mine == best && best != 0ull) {                      // keys are unique across chunks (distinct tokens)
#pragma unroll
            for (int q = 0; q < NL; ++q) cur[q] += (q == from) ? 1 : 0;
            out_keys[k] = best;
        }
    }
    // what is left in the lists joins the sum; reference exponent: the largest of the chunks' and the leftovers' own
    double xmax = -1e300;
    for (int q = 0; q < NL; ++q)
        if (cur[q] < cnt[q]) xmax = fmax(xmax, (double)key_value(keys[q][cur[q]]));     // lists are sorted: the first is the largest
    double Cg = fmax(Cmax, xmax > -1e299 ? ceil(xmax * kLog2e) + 1.0 : -1e300);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Cg = fmax(Cg, __shfl_xor_sync(kFullMask, Cg, o));
    double W = 0.0;
    if (Cg > -1e299) {
        for (int q = 0; q < NL; ++q) {
            if (!hdr[q]) continue;
            if (hdr[q]->W != 0.0) W += hdr[q]->W * exp2(hdr[q]->C - Cg);
            for (int k = cur[q]; k < cnt[q]; ++k) W += exp2((double)key_value(keys[q][k]) * kLog2e - Cg);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) W += __shfl_xor_sync(kFullMask, W, o);
    if (lane == 0) {
        SegPartial h;
        h.W = W; h.C = (W != 0.0) ? Cg : 0.0; h.cnt = n_out; h.flags = flags | (*p.error ? kPartTimeout : 0u);
        h.pad[0] = h.pad[1] = 0;
        *(SegPartial*)out = h;
    }
}

}  // namespace cadd
