// Softmax statistics and top-K of the draft positions fused into the drafter's output projection (Eq. 1 and
// Algorithm 1's "Require", computed from the drafter's last hidden states instead of materialised logits).
// The logits l_i = h_i . W^T are formed tile by tile on the tensor cores exactly as in head_argmax.cuh (same TMA
// ring, same tcgen05.mma issue, accumulators in tensor memory); the epilogue turns every row of a tile into running
// softmax / top-K state instead of a single maximum:
//   - the KP best (logit, token) pairs of the row so far, a sorted list per row in shared memory;
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

constexpr int kDraftMaxKP = 32;           // list capacity per row that fits beside the operand ring in shared memory

struct DraftHeadShared {
    HeadShared g;                                          // operand ring, barriers (head_argmax.cuh)
    uint64_t list[kDraftMaxKP][kHeadBM];                   // list[k][row of the tile]: k-th best key of the row so far
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
    unsigned char* chunk_partials;   // [M * n_chunks] records of seg_partial_stride(KP) bytes
    int32_t* error;
};

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

__global__ void __launch_bounds__(kHeadThreads, 1)
head_softmax_topk_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, DraftHeadParams p) {
    extern __shared__ __align__(16) unsigned char head_smem_raw[];
    DraftHeadShared& dsh = *reinterpret_cast<DraftHeadShared*>(head_smem_raw + ((1024u - (smem_u32(head_smem_raw) & 1023u)) & 1023u));
    HeadShared& sh = dsh.g;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k_steps = (p.Kdim + kHeadBK - 1) / kHeadBK;
    const int64_t n_items = (int64_t)p.m_tiles * p.n_chunks;      // item w -> (chunk = w / m_tiles, row tile = w % m_tiles)
    const int KP = p.KP;

    if (tid == 0) {
        for (int s = 0; s < kHeadStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sh.acc_full[s], 1); mbar_init(&sh.acc_empty[s], 4); }
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
                    for (int k = 0; k < k_steps; ++k) {
                        if (!head_wait(&sh.empty[s], ph ^ 1u, 64)) { sh.error = 1; break; }
                        mbar_arrive_expect_tx(&sh.full[s], kHeadABytes + kHeadBBytes);
                        tma_load_2d(&sh.a[s][0], &map_h, k * kHeadBK, mt * kHeadBM, &sh.full[s]);
                        tma_load_2d(&sh.b[s][0], &map_w, k * kHeadBK, nt * kHeadBN, &sh.full[s]);
                        if (++s == kHeadStages) { s = 0; ph ^= 1u; }
                    }
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
                    const uint32_t d = tmem_base + buf * kHeadBN;
                    bool ok = true;
                    for (int k = 0; k < k_steps; ++k) {
                        if (!head_wait(&sh.full[s], ph)) { sh.error = 3; ok = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int kk = 0; kk < kHeadBK / 16; ++kk)
                            umma_bf16(d, umma_desc_k_sw128(&sh.a[s][0], kk), umma_desc_k_sw128(&sh.b[s][0], kk), kHeadIdesc,
                                      (k | kk) != 0 ? 1u : 0u);
                        umma_commit(&sh.empty[s]);
                        if (++s == kHeadStages) { s = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit(&sh.acc_full[buf]);
                    if (++buf == 2) { buf = 0; aph ^= 1u; }
                }
            }
        }
    } else {
        // ---------------- epilogue: warps 2..5; thread = one row of the tile ----------------
        const int quarter = warp & 3;
        const int trow = quarter * 32 + lane;                    // row inside the tile = tensor-memory lane
        unsigned buf = 0, aph = 0;
        for (int64_t w = blockIdx.x; w < n_items && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
            const int ch = (int)(w / p.m_tiles), mt = (int)(w - (int64_t)ch * p.m_tiles);
            if (!draft_tile_live(p, mt)) continue;
            const int64_t row = (int64_t)mt * kHeadBM + trow;
            const bool live = draft_row_live(p, row);
            // row state over the chunk
            ThreadSum s{0.0, -INFINITY, 0.0f};
            uint32_t flags = 0;
            int cnt = 0;                                          // entries in the row's list
            float thr = -INFINITY;                                // value of the list's last entry once it is full
            uint64_t thr_key = 0;
            const int nt1 = min((ch + 1) * p.chunk_tiles, p.n_tiles);
            bool ok = true;
            for (int nt = ch * p.chunk_tiles; nt < nt1 && ok; ++nt) {
                if (!__all_sync(kFullMask, head_wait(&sh.acc_full[buf], aph, 256))) { sh.error = 4; ok = false; break; }
                tc_fence_after();
                const int64_t col0 = (int64_t)nt * kHeadBN;
#pragma unroll 1
                for (int c = 0; c < kHeadBN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kHeadBN + c * 32, r);
                    tmem_ld_wait();
                    const int64_t cb = col0 + c * 32;
                    float part = 0.0f;                            // fp32 sum of this run of 32 columns
#pragma unroll
                    for (int i = 0; i < 32; ++i) {                 // fully unrolled: r[] must stay in registers
                        const float x = __uint_as_float(r[i]);
                        if (cb + i >= p.V || !live) continue;
                        if (x < thr) { part += exp2_term(x, s.negc); continue; }      // the common case
                        const uint32_t bits = __float_as_uint(x);
                        if ((bits & 0x7f800000u) == 0x7f800000u) {                    // Inf or NaN: no mass, never a candidate
                            if (bits != 0xff800000u) flags |= kPartNonfinite;
                            if (bits == 0x7f800000u) flags |= kPartPosInf;
                            continue;
                        }
                        const uint64_t key = make_key(x, (uint32_t)(cb + i));
                        if (cnt == KP && key < thr_key) { part += exp2_term(x, s.negc); continue; }   // ties with the last entry
                        // insert into the sorted list; when it is full the last entry drops out and joins the sum
                        if (cnt == KP) {
                            s.acc += (double)part; part = 0.0f;
                            fold_scalar(s, key_value(dsh.list[KP - 1][trow]));
                        } else {
                            ++cnt;
                        }
                        int k = cnt - 1;
                        while (k > 0 && dsh.list[k - 1][trow] < key) { dsh.list[k][trow] = dsh.list[k - 1][trow]; --k; }
                        dsh.list[k][trow] = key;
                        if (cnt == KP) {
                            thr_key = dsh.list[KP - 1][trow];
                            thr = key_value(thr_key);
                            if (thr > s.tmax + 60.0f || s.tmax == -INFINITY) {       // keep 2^(x*log2e - c) in range for x < thr
                                s.acc += (double)part; part = 0.0f;
                                raise_reference(s, thr);
                            }
                        }
                    }
                    s.acc += (double)part;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.acc_empty[buf]);
                if (++buf == 2) { buf = 0; aph ^= 1u; }
            }
            if (!ok) break;
            if (live) {
                unsigned char* rec = p.chunk_partials + ((size_t)row * p.n_chunks + ch) * seg_partial_stride(KP);
                uint64_t* out_keys = (uint64_t*)(rec + sizeof(SegPartial));
                for (int k = 0; k < cnt; ++k) out_keys[k] = dsh.list[k][trow];
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
    // lane owns chunks lane and lane + 32
    const SegPartial* hdr[2];
    const uint64_t* keys[2];
    int cnt[2], cur[2] = {0, 0};
    double Cmax = -1e300;
    uint32_t flags = 0;
    int total = 0;
    for (int q = 0; q < 2; ++q) {
        const int ch = lane + 32 * q;
        if (ch < p.n_chunks) {
            const unsigned char* rec = p.chunk_partials + ((size_t)row * p.n_chunks + ch) * stride;
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
        const uint64_t h0 = cur[0] < cnt[0] ? keys[0][cur[0]] : 0ull, h1 = cur[1] < cnt[1] ? keys[1][cur[1]] : 0ull;
        const uint64_t mine = max(h0, h1);
        uint64_t best = mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(kFullMask, best, o));
        if (mine == best && best != 0ull) {                      // keys are unique across chunks (distinct tokens)
            if (h0 == best) ++cur[0]; else ++cur[1];
            out_keys[k] = best;
        }
    }
    // what is left in the lists joins the sum; reference exponent: the largest of the chunks' and the leftovers' own
    double xmax = -1e300;
    for (int q = 0; q < 2; ++q)
        if (cur[q] < cnt[q]) xmax = fmax(xmax, (double)key_value(keys[q][cur[q]]));     // lists are sorted: the first is the largest
    double Cg = fmax(Cmax, xmax > -1e299 ? ceil(xmax * kLog2e) + 1.0 : -1e300);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Cg = fmax(Cg, __shfl_xor_sync(kFullMask, Cg, o));
    double W = 0.0;
    if (Cg > -1e299) {
        for (int q = 0; q < 2; ++q) {
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
