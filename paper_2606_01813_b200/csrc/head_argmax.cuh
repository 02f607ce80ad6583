// Verification argmax fused into the output projection (the step right before the path: Section 3.1 takes the
// target's prediction at every tree node, i.e. argmax over v of  h_j . W_v  with h the target's last hidden state at
// node j and W the output embedding).  The logits [rows, V] are never written to memory: a bf16 x bf16 -> fp32 GEMM
// on the 5th-generation tensor cores keeps each 128 x 256 tile of logits in tensor memory, and the epilogue reduces it
// to one (value, token) pair per row, merged across tiles by a 64-bit atomic max.
//
// One CTA per SM, 192 threads, three roles:
//   warp 0      producer: 2-D tiled bulk tensor copies (TMA, 128-byte swizzle, each into this CTA's own shared memory) of a 128 x 64 tile of
//               hidden states and a 256 x 64 tile of W into a 4-stage shared-memory ring, completion on mbarriers;
//   warp 1      one elected thread issues tcgen05.mma (M 128, N 256, K 16 per instruction, operands described by
//               shared-memory matrix descriptors, accumulator in tensor memory), tcgen05.commit frees the stage and,
//               after the last k-step, hands the accumulator to the epilogue; the warp also owns the tensor-memory
//               allocation (all 512 columns = two accumulators, so the epilogue of one tile overlaps the next);
//   warps 2-5   epilogue: each thread owns one row of the tile (one tensor-memory lane), reads it 32 columns at a time
//               with tcgen05.ld and keeps the running maximum and its first column.
// Tiles are walked in groups of row tiles whose hidden states fit in L2 (about 24 MB); inside a group the order is
// (column tile outer, row tile inner), CTA c taking tiles c, c + grid, ...: at any time the CTAs work on neighbouring
// column tiles of W, which come from L2 after their first use, the group's hidden states stay L2-resident, and W is
// streamed from HBM once per group.
//
// Every wait on an mbarrier has an iteration limit; a role that gives up sets an error word, all roles then leave
// their loops, the CTA meets at a barrier and the tensor memory is released before it exits.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "tile_ring.cuh"

namespace cadd {

constexpr int kHeadBM = 128;              // rows per tile (tensor-memory lanes)
constexpr int kHeadBN = 256;              // columns (tokens) per tile
constexpr int kHeadBK = 64;               // bf16 elements per k-step: one 128-byte swizzle row
constexpr int kHeadStages = 4;
constexpr int kHeadThreads = 192;
constexpr int kHeadTmemCols = 512;        // two fp32 accumulators of kHeadBN columns
constexpr uint32_t kHeadABytes = kHeadBM * kHeadBK * 2;   // 16 KB
constexpr uint32_t kHeadBBytes = kHeadBN * kHeadBK * 2;   // 32 KB

struct HeadShared {
    alignas(1024) unsigned char a[kHeadStages][kHeadABytes];
    alignas(1024) unsigned char b[kHeadStages][kHeadBBytes];
    alignas(8) uint64_t full[kHeadStages];     // tile pair landed (producer -> MMA)
    uint64_t empty[kHeadStages];               // MMAs that read the stage are done (MMA -> producer)
    uint64_t acc_full[2];                      // accumulator complete (MMA -> epilogue)
    uint64_t acc_empty[2];                     // accumulator read out (epilogue -> MMA)
    uint32_t tmem_base;
    uint32_t error;
};
inline size_t head_smem_bytes() { return sizeof(HeadShared) + 1024; }

struct HeadParams {
    int64_t M;                 // rows = batch * R
    int64_t V;                 // tokens
    int Kdim;                  // hidden size
    int m_tiles, n_tiles;
    int group_m;               // row tiles per group: a group's hidden states stay L2-resident while all of W streams by
    int R, rows_mode;
    const int32_t* n_nodes;    // [batch]
    const int32_t* m_live;     // LIVE mode: device word holding the number of packed rows (the GEMM runs on the packed copy
                               // of the live rows only); NULL in DENSE mode
    unsigned long long* row_best;   // [M] packed (ordered logit << 32 | ~token), zeroed before the launch
    int32_t* error;            // device word, set non-zero when a bounded wait ran out
};

// Bounded wait.  The MMA thread polls without a sleep between tries: a late wake-up would leave the tensor cores
// idle.
constexpr int kHeadSpinLimit = 1 << 20;
__device__ __forceinline__ bool head_wait(uint64_t* bar, unsigned parity, unsigned sleep_ns = 0) {
    for (int it = 0; it < kHeadSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (sleep_ns) __nanosleep(sleep_ns);      // roles off the critical path back off: spinning costs power the tensor cores need
    }
    return false;
}

// ---- tcgen05 / TMA wrappers ----
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t cols) {      // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {         // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate; one thread issues.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier gets one arrival when all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {         // whole warp: 32 lanes x 32 columns
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {           // whole warp: 32 lanes x 8 columns
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements) under the 128-byte
// swizzle, rows packed densely: 8-row groups are 1024 bytes apart (stride byte offset), the leading byte offset is
// unused for swizzled K-major operands (1), descriptor version 1 (sm_100), layout type 2 = 128-byte swizzle.
// A k-step of 16 elements inside the 128-byte row advances the start address by 32 bytes.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(const void* tile, int k16) {
    const uint32_t addr = smem_u32(tile) + (uint32_t)k16 * 32u;
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)1 << 16) | ((uint64_t)(1024u >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9 and 10-12 = 1), both K-major
// (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28.
constexpr uint32_t kHeadIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kHeadBN >> 3) << 17) | ((uint32_t)(kHeadBM >> 4) << 24);

// ---- the two single-thread roles' inner loops, shared by the kernels that run this GEMM pipeline ----
// Producer: streams the k_steps operand tile pairs of one output tile (row tile mt, column tile nt) into the ring.
// `s` / `ph` are the ring position and its phase parity, carried across tiles.  Returns false on a wait that ran out.
template <class Shared, int Stages>
__device__ __forceinline__ bool head_produce_tile(Shared& sh, const CUtensorMap* map_h, const CUtensorMap* map_w, int mt, int nt,
                                                  int k_steps, unsigned& s, unsigned& ph) {
    for (int k = 0; k < k_steps; ++k) {
        if (!head_wait(&sh.empty[s], ph ^ 1u, 64)) return false;             // first pass over the ring: free at once
        mbar_arrive_expect_tx(&sh.full[s], kHeadABytes + kHeadBBytes);
        tma_load_2d(&sh.a[s][0], map_h, k * kHeadBK, mt * kHeadBM, &sh.full[s]);
        tma_load_2d(&sh.b[s][0], map_w, k * kHeadBK, nt * kHeadBN, &sh.full[s]);
        if (++s == Stages) { s = 0; ph ^= 1u; }
    }
    return true;
}
// MMA issuer: accumulates one output tile into the tensor-memory accumulator at `d`; every stage is committed back to
// the producer once its MMAs have read it, the finished accumulator is committed to `acc_full`.
template <class Shared, int Stages>
__device__ __forceinline__ bool head_mma_tile(Shared& sh, uint32_t d, uint64_t* acc_full, int k_steps, unsigned& s, unsigned& ph) {
    for (int k = 0; k < k_steps; ++k) {
        if (!head_wait(&sh.full[s], ph)) return false;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kHeadBK / 16; ++kk)
            umma_bf16(d, umma_desc_k_sw128(&sh.a[s][0], kk), umma_desc_k_sw128(&sh.b[s][0], kk), kHeadIdesc, (k | kk) != 0 ? 1u : 0u);
        umma_commit(&sh.empty[s]);                                            // the stage is free once these MMAs have read it
        if (++s == Stages) { s = 0; ph ^= 1u; }
    }
    umma_commit(acc_full);                                                    // accumulator complete
    return true;
}

// Tile order: groups of group_m row tiles; inside a group the column tile is the outer index and the row tile the
// inner one.  Work item w (CTA c takes w = c, c + grid, ...) -> (row tile, column tile).
__device__ __forceinline__ void head_tile_of(const HeadParams& p, int64_t w, int& mt, int& nt) {
    const int64_t per_group = (int64_t)p.group_m * p.n_tiles;
    const int g = (int)(w / per_group);
    const int64_t rem = w - (int64_t)g * per_group;
    const int gsz = min(p.group_m, p.m_tiles - g * p.group_m);
    nt = (int)(rem / gsz);
    mt = g * p.group_m + (int)(rem - (int64_t)nt * gsz);
}

__global__ void __launch_bounds__(kHeadThreads, 1)
head_argmax_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, HeadParams p) {
    extern __shared__ __align__(16) unsigned char head_smem_raw[];
    HeadShared& sh = *reinterpret_cast<HeadShared*>(head_smem_raw + ((1024u - (smem_u32(head_smem_raw) & 1023u)) & 1023u));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k_steps = (p.Kdim + kHeadBK - 1) / kHeadBK;
    if (p.m_live) {                                               // LIVE mode: only the packed live rows exist
        p.M = *p.m_live;
        p.m_tiles = (int)((p.M + kHeadBM - 1) / kHeadBM);
        if (p.group_m > p.m_tiles) p.group_m = p.m_tiles > 0 ? p.m_tiles : 1;
    }
    const int64_t n_work = (int64_t)p.m_tiles * p.n_tiles;

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
            for (int64_t w = blockIdx.x; w < n_work && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
                int mt, nt;
                head_tile_of(p, w, mt, nt);
                if (!head_produce_tile<HeadShared, kHeadStages>(sh, &map_h, &map_w, mt, nt, k_steps, s, ph)) { sh.error = 1; break; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            unsigned s = 0, ph = 0, buf = 0, aph = 0;
            for (int64_t w = blockIdx.x; w < n_work && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
                int mt, nt;
                head_tile_of(p, w, mt, nt);
                if (!head_wait(&sh.acc_empty[buf], aph ^ 1u)) { sh.error = 2; break; }   // epilogue has drained it
                tc_fence_after();
                if (!head_mma_tile<HeadShared, kHeadStages>(sh, tmem_base + buf * kHeadBN, &sh.acc_full[buf], k_steps, s, ph)) { sh.error = 3; break; }
                if (++buf == 2) { buf = 0; aph ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue: warps 2..5, tensor-memory lane quarter = warp % 4 ----------------
        const int quarter = warp & 3;
        unsigned buf = 0, aph = 0;
        for (int64_t w = blockIdx.x; w < n_work && !*(volatile uint32_t*)&sh.error; w += gridDim.x) {
            int mt, nt;
            head_tile_of(p, w, mt, nt);
            if (!__all_sync(kFullMask, head_wait(&sh.acc_full[buf], aph, 256))) { sh.error = 4; break; }
            tc_fence_after();
            const int64_t row = (int64_t)mt * kHeadBM + quarter * 32 + lane;
            const int64_t col0 = (int64_t)nt * kHeadBN;
            float best = -INFINITY;
            int64_t best_col = -1;
#pragma unroll 1
            for (int c = 0; c < kHeadBN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * kHeadBN + c * 32, r);
                tmem_ld_wait();
                const int64_t cb = col0 + c * 32;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float v = __uint_as_float(r[i]);
                    if (v > best && cb + i < p.V) { best = v; best_col = cb + i; }     // strict: the first column wins ties
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.acc_empty[buf]);
            if (row < p.M && best_col >= 0)
                atomicMax(&p.row_best[row], (unsigned long long)make_key(best, (uint32_t)best_col));
            if (++buf == 2) { buf = 0; aph ^= 1u; }
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

// LIVE mode, step 1: row_off[b] = number of live rows (j <= n_nodes[b]) of the requests before b; row_off[batch] is
// the packed row count.  One CTA.
__global__ void __launch_bounds__(1024) head_live_offsets_kernel(const int32_t* n_nodes, int batch, int R, int32_t* row_off) {
    __shared__ int part[1024];
    const int tid = threadIdx.x;
    const int per = (batch + 1023) / 1024;
    int run = 0;
    for (int b = tid * per; b < min(batch, (tid + 1) * per); ++b) {
        int n = n_nodes[b];
        n = n < 0 ? 0 : (n > R - 1 ? R - 1 : n);
        run += n + 1;
    }
    part[tid] = run;
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int t = 0; t < 1024; ++t) { const int x = part[t]; part[t] = acc; acc += x; }
        row_off[batch] = acc;
    }
    __syncthreads();
    int acc = part[tid];
    for (int b = tid * per; b < min(batch, (tid + 1) * per); ++b) {
        row_off[b] = acc;
        int n = n_nodes[b];
        n = n < 0 ? 0 : (n > R - 1 ? R - 1 : n);
        acc += n + 1;
    }
}

// LIVE mode, step 2: copies the live rows of the hidden states next to one another (one CTA per (request, row)).
__global__ void __launch_bounds__(128) head_pack_rows_kernel(const __nv_bfloat16* hidden_states, int64_t stride_row, int hidden, int R,
                                                             const int32_t* n_nodes, const int32_t* row_off, __nv_bfloat16* packed) {
    const int b = blockIdx.y, j = blockIdx.x;
    int n = n_nodes[b];
    n = n < 0 ? 0 : (n > R - 1 ? R - 1 : n);
    if (j > n) return;
    const uint4* src = (const uint4*)(hidden_states + ((int64_t)b * R + j) * stride_row);      // 16-byte aligned rows
    uint4* dst = (uint4*)(packed + (int64_t)(row_off[b] + j) * hidden);
    for (int c = threadIdx.x; c < hidden / 8; c += blockDim.x) dst[c] = src[c];
    for (int k = (hidden / 8) * 8 + threadIdx.x; k < hidden; k += blockDim.x)                 // hidden % 8 != 0 cannot pass the
        packed[(int64_t)(row_off[b] + j) * hidden + k] = hidden_states[((int64_t)b * R + j) * stride_row + k];   // stride check
}

// Turns the packed per-row maxima into token ids.  Rows not read in LIVE mode get -1; a row whose logits were all
// -Inf or NaN gets 0, like the plain argmax kernel; -2 marks every row when the GEMM gave up on a wait.  In LIVE
// mode row (b, j) of the output is packed row row_off[b] + j of the GEMM.
__global__ void head_decode_kernel(const unsigned long long* row_best, const int32_t* n_nodes, const int32_t* row_off,
                                   const int32_t* error, int64_t M, int R, int rows_mode, int32_t* node_argmax) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= M) return;
    const int64_t b = r / R;
    const int j = (int)(r - b * R);
    int64_t src = r;
    if (rows_mode == CADD_ROWS_LIVE) {
        int n = n_nodes[b];
        n = n < 0 ? 0 : (n > R - 1 ? R - 1 : n);
        if (j > n) { node_argmax[r] = -1; return; }
        src = (int64_t)row_off[b] + j;
    }
    const unsigned long long k = row_best[src];
    int32_t ans = k ? (int32_t)key_id((uint64_t)k) : 0;
    if (*error) ans = -2;
    node_argmax[r] = ans;
}

}  // namespace cadd
