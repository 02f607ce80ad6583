// Best-first expansion of the candidate tree with the greedy throughput stopping rule, and emission
// of the tree arrays and the ancestor mask (Algorithm 1; Eq. 5-7, Eq. 11, Corollary 1; Section 3.3).
//
// One CTA per request.
//   phase 0  all warps: merge the per-segment softmax/top-K partials of each live position into the
//            sorted top-K list (token, a = logit - row max) and log Z, all in fp64
//   phase 1  one thread: running log-partition sums S_d and the reachable depth
//   phase 2  warp 0: the pop loop.  The frontier (Algorithm 1's heap) is striped over the 32 lanes;
//            each lane caches the best entry of its stripe, a pop is a 128-bit warp arg-max
//            (four redux.sync steps) followed by a rescan of the winner's stripe only.  Nodes are
//            popped speculatively in groups; the group's exp(sigma), prefix sums Phi and throughput
//            tests are then evaluated lane-parallel, and the first failing test fixes n*.  The pop
//            order does not depend on the cost model, so this yields exactly Algorithm 1's tree.
//   phase 3  all warps: write token / parent / depth / position / log-prob rows, padding, and the
//            packed (and optionally dense) ancestor mask.
#pragma once
#include "common.cuh"
#include "softmax_topk.cuh"

namespace cadd {

struct ExpandParams {
    int batch, L, K, KP, S, B_max, R;
    uint32_t flags;
    const unsigned char* partials;
    const int32_t* l_eff;
    const int32_t* bonus_token;
    const int32_t* ctx_len;
    int cost_kind;
    const double* cost_coef;
    const double* cost_table;
    const int32_t* table_idx;
    const double* t_draft;
    int32_t* n_nodes;
    int32_t* token_ids;
    int32_t* parent_idx;
    int32_t* depth;
    int32_t* position_ids;
    double* node_logprob;
    double* phi;
    double* theta;
    uint32_t* mask_bits;
    uint8_t* mask_dense;
    int32_t* topk_token;
    double* topk_logprob;
    int32_t* status;
};

constexpr int kExpandWarps = kThreads / 32;
constexpr int kMaskRowWords = 65;      // words that can hold a set bit: rows 0..2048

// Dynamic shared memory layout of the expansion kernel (byte offsets), same arithmetic on host and device.
struct ExpandLayout {
    size_t a_list, lz, S, nA, nSig, region, tok_list, nTok, keff, maskrow, nPar, nDep, nRank, total;
    int fr_slots;      // frontier slots per lane
};
__host__ __device__ inline ExpandLayout expand_layout(int L, int K, int KP, int S, int B_max) {
    ExpandLayout o;
    const size_t NR = (size_t)B_max + 1;
    o.fr_slots = (2 * B_max + 1 + 31) / 32 + 1;
    size_t frontier = (size_t)o.fr_slots * 32 * (8 + 8 + 4);
    size_t scratch = (size_t)kExpandWarps * S * KP * 8;
    size_t region = frontier > scratch ? frontier : scratch;
    region = (region + 7) & ~(size_t)7;
    size_t p = 0;
    o.a_list = p;   p += (size_t)L * K * 8;
    o.lz = p;       p += (size_t)L * 8;
    o.S = p;        p += ((size_t)L + 1) * 8;
    o.nA = p;       p += NR * 8;
    o.nSig = p;     p += NR * 8;
    o.region = p;   p += region;
    o.tok_list = p; p += (size_t)L * K * 4;
    o.nTok = p;     p += NR * 4;
    o.keff = p;     p += ((size_t)L + 2) * 4;
    o.maskrow = p;  p += (size_t)kExpandWarps * kMaskRowWords * 4;
    o.nPar = p;     p += NR * 2;  p = (p + 3) & ~(size_t)3;
    o.nDep = p;     p += NR;
    o.nRank = p;    p += NR;
    o.total = (p + 15) & ~(size_t)15;
    return o;
}

__device__ __forceinline__ double cost_verify(int kind, const double* q, const double* trow, int n) {
    if (kind == CADD_COST_TABLE) return trow[n];
    double x = (double)n;
    return q[1] + q[2] * x + q[3] * (x * x);
}

__global__ void __launch_bounds__(kThreads) expand_emit_kernel(ExpandParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const ExpandLayout lay = expand_layout(p.L, p.K, p.KP, p.S, p.B_max);
    double* a_list = (double*)(smem + lay.a_list);
    double* lz = (double*)(smem + lay.lz);
    double* Sd = (double*)(smem + lay.S);
    double* nA = (double*)(smem + lay.nA);
    double* nSig = (double*)(smem + lay.nSig);
    int32_t* tok_list = (int32_t*)(smem + lay.tok_list);
    int32_t* nTok = (int32_t*)(smem + lay.nTok);
    int32_t* keff = (int32_t*)(smem + lay.keff);          // keff[d], d = 1..L
    uint32_t* maskrow = (uint32_t*)(smem + lay.maskrow);
    uint16_t* nPar = (uint16_t*)(smem + lay.nPar);
    uint8_t* nDep = (uint8_t*)(smem + lay.nDep);
    uint8_t* nRank = (uint8_t*)(smem + lay.nRank);
    uint64_t* fHi = (uint64_t*)(smem + lay.region);
    uint64_t* fLo = fHi + (size_t)lay.fr_slots * 32;
    uint32_t* fPay = (uint32_t*)(fLo + (size_t)lay.fr_slots * 32);

    __shared__ int s_status, s_pinf, s_Lr, s_n;
    __shared__ double s_phi, s_theta;

    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = p.L, K = p.K, R = p.R;
    int clamped;
    const int Le = clamp_l_eff(p.l_eff, b, L, &clamped);
    if (tid == 0) { s_status = clamped ? CADD_STATUS_L_EFF_CLAMPED : 0; s_pinf = 0; }
    for (int d = tid; d < L + 2; d += kThreads) keff[d] = 0;
    __syncthreads();

    // ---------------- phase 0: merge partials, one warp per position ----------------
    const size_t pstride = seg_partial_stride(p.KP);
    for (int i = warp; i < L; i += kExpandWarps) {
        int32_t* out_tok = p.topk_token ? p.topk_token + ((int64_t)b * L + i) * K : nullptr;
        double* out_lp = p.topk_logprob ? p.topk_logprob + ((int64_t)b * L + i) * K : nullptr;
        const bool emit = (p.flags & CADD_FLAG_EMIT_TOPK) != 0;
        if (i >= Le) {
            if (emit) for (int k = lane; k < K; k += 32) {
                if (out_tok) out_tok[k] = -1;
                if (out_lp) out_lp[k] = -INFINITY;
            }
            continue;
        }
        uint64_t* scr = (uint64_t*)(smem + lay.region) + (size_t)warp * p.S * p.KP;
        const unsigned char* rec0 = p.partials + ((size_t)((int64_t)b * L + i) * p.S) * pstride;
        int n = 0;
        uint32_t fl = 0;
        for (int s = 0; s < p.S; ++s) {
            const SegPartial* h = (const SegPartial*)(rec0 + (size_t)s * pstride);
            const uint64_t* keys = (const uint64_t*)(h + 1);
            const int cnt = h->cnt;
            fl |= h->flags;
            for (int q = lane; q < cnt; q += 32) scr[n + q] = keys[q];
            n += cnt;
        }
        __syncwarp();
        uint64_t mk = 0;
        for (int q = lane; q < n; q += 32) mk = max(mk, scr[q]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mk = max(mk, __shfl_xor_sync(kFullMask, mk, o));
        const double m = (double)key_value(mk);
        double zsum = 0.0;
        for (int q = lane; q < n; q += 32) {
            const uint64_t k = scr[q];
            int rank = 0;
            for (int r = 0; r < n; ++r) rank += scr[r] > k;
            const double x = (double)key_value(k);
            zsum += exp(x - m);
            if (rank < K) { tok_list[i * K + rank] = (int32_t)key_id(k); a_list[i * K + rank] = x - m; }
        }
        for (int s = lane; s < p.S; s += 32) {
            const SegPartial* h = (const SegPartial*)(rec0 + (size_t)s * pstride);
            if (h->W > 0.0) zsum += h->W * exp(h->C * 0.6931471805599453094 - m);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zsum += __shfl_xor_sync(kFullMask, zsum, o);
        const double logZ = log(zsum);
        const int ke = n < K ? n : K;
        __syncwarp();
        if (lane == 0) {
            keff[i + 1] = ke;
            lz[i] = logZ;
            int st = 0;
            if (fl & kPartNonfinite) st |= CADD_STATUS_NONFINITE_INPUT;
            if (ke < K) st |= CADD_STATUS_FEWER_THAN_K_FINITE;
            if (st) atomicOr(&s_status, st);
            if (fl & kPartPosInf) s_pinf = 1;
        }
        if (emit) for (int k = lane; k < K; k += 32) {
            if (out_tok) out_tok[k] = k < ke ? tok_list[i * K + k] : -1;
            if (out_lp) out_lp[k] = k < ke ? a_list[i * K + k] - logZ : -INFINITY;
        }
    }
    __syncthreads();

    // ---------------- phase 1: S_d and the reachable depth ----------------
    if (tid == 0) {
        Sd[0] = 0.0;
        int Lr = Le;
        for (int d = 1; d <= Le; ++d) {
            Sd[d] = Sd[d - 1] + lz[d - 1];
            if (keff[d] == 0 && Lr == Le) Lr = d - 1;
        }
        s_Lr = Lr;
        nA[0] = 0.0; nSig[0] = 0.0; nTok[0] = -1; nPar[0] = 0; nDep[0] = 0; nRank[0] = 0;
    }
    __syncthreads();

    // ---------------- phase 2: the pop loop (warp 0) ----------------
    if (warp == 0) {
        const int Lr = s_Lr;
        const int B_max = p.B_max;
        const bool fixed = (p.flags & CADD_FLAG_FIXED_BUDGET) != 0;
        double q4[4] = {0, 0, 0, 0};
        const double* trow = nullptr;
        double C_d;
        if (p.cost_kind == CADD_COST_QUADRATIC) {
            for (int c = 0; c < 4; ++c) q4[c] = p.cost_coef[(int64_t)b * 4 + c];
            C_d = q4[0];
        } else {
            trow = p.cost_table + (int64_t)p.table_idx[b] * (B_max + 1);
            C_d = p.t_draft[b];
        }
        int st = 0;
        bool ok = true;
        double theta_prev = 0.0, Phi = 0.0;
        const double den0 = C_d + cost_verify(p.cost_kind, q4, trow, 0);
        if (!(den0 > 0.0)) { st |= CADD_STATUS_COST_NONPOSITIVE; ok = false; }
        else theta_prev = 1.0 / den0;
        if (s_pinf) ok = false;

        // lane-private view of the frontier
        int cnt = 0, bslot = -1;
        uint64_t bhi = 0, blo = 0;
        uint32_t brank = 0;
        int fsize = 0;
        unsigned pushctr = 0;
        auto push = [&](double sigma, int d, int token, int parent, int rank) {
            const uint64_t hi = ord64(sigma);
            const uint64_t lo = ~(((uint64_t)d << 43) | ((uint64_t)(uint32_t)token << 12) | (uint64_t)parent);
            const int t = pushctr & 31;
            ++pushctr;
            ++fsize;
            if (lane == t) {
                const int slot = cnt++;
                fHi[slot * 32 + lane] = hi; fLo[slot * 32 + lane] = lo; fPay[slot * 32 + lane] = (uint32_t)rank;
                if (bslot < 0 || hi > bhi || (hi == bhi && lo > blo)) { bhi = hi; blo = lo; bslot = slot; brank = rank; }
            }
        };
        if (ok && Lr >= 1) push(a_list[0] - Sd[1], 1, tok_list[0], 0, 1);

        int n = 0, popped = 0;
        bool stopped = false;
        while (ok && !stopped) {
            const int G = popped < 16 ? 8 : 32;
            int g = 0;
            while (g < G && popped < B_max && fsize > 0) {
                // 128-bit arg-max over the lanes' cached bests
                const bool has = cnt > 0;
                uint32_t v = has ? (uint32_t)(bhi >> 32) : 0u;
                uint32_t mx = __reduce_max_sync(kFullMask, v);
                bool alive = has && v == mx;
                v = alive ? (uint32_t)bhi : 0u;
                mx = __reduce_max_sync(kFullMask, v);
                alive = alive && v == mx;
                v = alive ? (uint32_t)(blo >> 32) : 0u;
                mx = __reduce_max_sync(kFullMask, v);
                alive = alive && v == mx;
                v = alive ? (uint32_t)blo : 0u;
                mx = __reduce_max_sync(kFullMask, v);
                alive = alive && v == mx;
                const int win = __ffs(__ballot_sync(kFullMask, alive)) - 1;
                const uint64_t whi = __shfl_sync(kFullMask, bhi, win);
                const uint64_t wlo = __shfl_sync(kFullMask, blo, win);
                const int r = (int)__shfl_sync(kFullMask, brank, win);
                if (lane == win) {                          // remove the entry, rescan this stripe
                    const int last = --cnt;
                    if (bslot != last) {
                        fHi[bslot * 32 + lane] = fHi[last * 32 + lane];
                        fLo[bslot * 32 + lane] = fLo[last * 32 + lane];
                        fPay[bslot * 32 + lane] = fPay[last * 32 + lane];
                    }
                    bslot = -1; bhi = 0; blo = 0;
                    for (int s = 0; s < cnt; ++s) {
                        const uint64_t hi = fHi[s * 32 + lane], lo = fLo[s * 32 + lane];
                        if (bslot < 0 || hi > bhi || (hi == bhi && lo > blo)) { bhi = hi; blo = lo; bslot = s; }
                    }
                    if (bslot >= 0) brank = fPay[bslot * 32 + lane];
                }
                --fsize;
                const uint64_t tb = ~wlo;
                const int d = (int)(tb >> 43);
                const int token = (int)((tb >> 12) & 0x7fffffffu);
                const int par = (int)(tb & 0xfffu);
                const double A = nA[par] + a_list[(d - 1) * K + (r - 1)];
                const int j = ++popped;
                if (lane == 0) {
                    nA[j] = A; nSig[j] = unord64(whi); nTok[j] = token;
                    nPar[j] = (uint16_t)par; nDep[j] = (uint8_t)d; nRank[j] = (uint8_t)r;
                }
                __syncwarp();
                if (r + 1 <= keff[d])                       // next sibling
                    push((nA[par] + a_list[(d - 1) * K + r]) - Sd[d], d, tok_list[(d - 1) * K + r], par, r + 1);
                if (d < Lr)                                 // first child
                    push((A + a_list[d * K]) - Sd[d + 1], d + 1, tok_list[d * K], j, 1);
                ++g;
            }
            if (g == 0) break;
            __syncwarp();
            // evaluate the group: rows n+1 .. n+g, one per lane
            const int j = n + 1 + lane;
            const bool act = lane < g;
            const double delta = act ? exp(nSig[j]) : 0.0;
            double cum = delta;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double t = __shfl_up_sync(kFullMask, cum, o);
                if (lane >= o) cum += t;
            }
            const double Phi_j = Phi + cum;
            const double den = act ? C_d + cost_verify(p.cost_kind, q4, trow, j) : 1.0;
            const bool bad = !(den > 0.0);
            const double theta_j = (1.0 + Phi_j) / den;
            double theta_jm1 = __shfl_up_sync(kFullMask, theta_j, 1);
            if (lane == 0) theta_jm1 = theta_prev;
            const bool stop = act && (bad || (!fixed && theta_j <= theta_jm1));
            const unsigned sm = __ballot_sync(kFullMask, stop);
            if (sm) {
                const int f = __ffs(sm) - 1;                // rows n+1 .. n+f are accepted
                if (__shfl_sync(kFullMask, (int)bad, f)) st |= CADD_STATUS_COST_NONPOSITIVE;
                const double ph = __shfl_sync(kFullMask, Phi_j, f > 0 ? f - 1 : 0);
                const double th = __shfl_sync(kFullMask, theta_j, f > 0 ? f - 1 : 0);
                if (f > 0) { Phi = ph; theta_prev = th; }
                n += f;
                stopped = true;
            } else {
                Phi = __shfl_sync(kFullMask, Phi_j, g - 1);
                theta_prev = __shfl_sync(kFullMask, theta_j, g - 1);
                n += g;
            }
        }
        if (ok && !stopped) st |= (fsize == 0) ? CADD_STATUS_FRONTIER_EXHAUSTED : CADD_STATUS_CAP_HIT;
        if (lane == 0) {
            s_n = n; s_phi = Phi; s_theta = theta_prev;
            if (st) atomicOr(&s_status, st);
        }
    }
    __syncthreads();

    // ---------------- phase 3: emission ----------------
    const int n = s_n;
    const int ctx = p.ctx_len ? p.ctx_len[b] : 0;
    const int bonus = p.bonus_token ? p.bonus_token[b] : -1;
    if (tid == 0) {
        p.n_nodes[b] = n;
        if (p.phi) p.phi[b] = s_phi;
        if (p.theta) p.theta[b] = s_theta;
        if (p.status) p.status[b] = s_status;
    }
    for (int j = tid; j < R; j += kThreads) {
        const int64_t o = (int64_t)b * R + j;
        int t = -1, par = -1, d = 0, pos = 0;
        double lp = 0.0;
        if (j == 0) { t = bonus; pos = ctx; }
        else if (j <= n) { t = nTok[j]; par = nPar[j]; d = nDep[j]; pos = ctx + d; lp = nSig[j]; }
        p.token_ids[o] = t;
        p.parent_idx[o] = par;
        p.depth[o] = d;
        if (p.position_ids) p.position_ids[o] = pos;
        if (p.node_logprob) p.node_logprob[o] = lp;
    }
    const bool dense = (p.flags & CADD_FLAG_EMIT_DENSE_MASK) && p.mask_dense;
    if (p.mask_bits || dense) {
        const int W = (R + 31) >> 5;
        uint32_t* mr = maskrow + warp * kMaskRowWords;
        for (int j = warp; j < R; j += kExpandWarps) {
            for (int w = lane; w < kMaskRowWords; w += 32) mr[w] = 0;
            __syncwarp();
            if (j <= n && lane == 0) {                      // self and ancestors: at most L+1 bits
                int cur = j;
                for (;;) {
                    mr[cur >> 5] |= 1u << (cur & 31);
                    if (cur == 0) break;
                    cur = nPar[cur];
                }
            }
            __syncwarp();
            if (p.mask_bits) {
                uint32_t* dst = p.mask_bits + ((int64_t)b * R + j) * W;
                for (int w = lane; w < W; w += 32) dst[w] = w < kMaskRowWords ? mr[w] : 0u;
            }
            if (dense) {
                uint8_t* dst = p.mask_dense + ((int64_t)b * R + j) * R;
                for (int c = lane; c < R; c += 32)
                    dst[c] = (c >> 5) < kMaskRowWords ? (uint8_t)((mr[c >> 5] >> (c & 31)) & 1u) : (uint8_t)0;
            }
            __syncwarp();
        }
    }
}

}  // namespace cadd
