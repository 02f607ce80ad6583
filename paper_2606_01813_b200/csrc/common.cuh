// Shared device helpers for the CaDDTree kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "cadd.h"

namespace cadd {

constexpr int kThreads = 256;              // threads per CTA in every streaming kernel
constexpr unsigned kFullMask = 0xffffffffu;

// ---- order-preserving integer images of IEEE values ----
// ord32(a) < ord32(b)  <=>  a < b as floats, for non-NaN a, b with -0 canonicalised to +0 by the caller.
__device__ __forceinline__ uint32_t ord32(uint32_t bits) {
    return bits ^ ((uint32_t)((int32_t)bits >> 31) | 0x80000000u);
}
__device__ __forceinline__ uint32_t unord32(uint32_t o) {
    return o ^ ((o & 0x80000000u) ? 0x80000000u : 0xffffffffu);
}
__device__ __forceinline__ uint64_t ord64(double x) {
    uint64_t b = (uint64_t)__double_as_longlong(x);
    return b ^ ((uint64_t)((int64_t)b >> 63) | 0x8000000000000000ull);
}
__device__ __forceinline__ double unord64(uint64_t o) {
    uint64_t b = o ^ ((o & 0x8000000000000000ull) ? 0x8000000000000000ull : 0xffffffffffffffffull);
    return __longlong_as_double((long long)b);
}

// A top-K candidate as one 64-bit key: larger key = better under (logit descending, token id ascending).
__device__ __forceinline__ uint64_t make_key(float x, uint32_t id) {
    uint32_t b = __float_as_uint(x);
    if (b == 0x80000000u) b = 0;                         // -0 and +0 are the same logit value
    return ((uint64_t)ord32(b) << 32) | (uint32_t)(~id);
}
__device__ __forceinline__ float key_value(uint64_t key) { return __uint_as_float(unord32((uint32_t)(key >> 32))); }
__device__ __forceinline__ uint32_t key_id(uint64_t key) { return ~(uint32_t)key; }

// ---- per-dtype access to a row of logits ----
template <int DT> struct Elem;
template <> struct Elem<CADD_DTYPE_BF16> {
    static constexpr int ES = 2;     // bytes per element
    static constexpr int EPC = 8;    // elements per 16-byte chunk
    static __device__ __forceinline__ float load(const void* row, int64_t i) {
        return __uint_as_float((uint32_t)((const uint16_t*)row)[i] << 16);
    }
    // the eight values of a chunk, widened exactly
    static __device__ __forceinline__ void unpack(const uint4& w, float* f) {
        f[0] = __uint_as_float(w.x << 16); f[1] = __uint_as_float(w.x & 0xffff0000u);
        f[2] = __uint_as_float(w.y << 16); f[3] = __uint_as_float(w.y & 0xffff0000u);
        f[4] = __uint_as_float(w.z << 16); f[5] = __uint_as_float(w.z & 0xffff0000u);
        f[6] = __uint_as_float(w.w << 16); f[7] = __uint_as_float(w.w & 0xffff0000u);
    }
    // maximum of a chunk, NaN ignored (NaN only if every element is NaN)
    static __device__ __forceinline__ float chunk_max(const uint4& w) {
        __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&w.x);
        __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&w.y);
        __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&w.z);
        __nv_bfloat162 d = *reinterpret_cast<const __nv_bfloat162*>(&w.w);
        __nv_bfloat162 m = __hmax2(__hmax2(a, b), __hmax2(c, d));
        uint32_t bits = *reinterpret_cast<uint32_t*>(&m);
        return fmaxf(__uint_as_float(bits << 16), __uint_as_float(bits & 0xffff0000u));
    }
    // maximum over four chunks (32 elements), NaN ignored
    static __device__ __forceinline__ float max4(const uint4& a, const uint4& b, const uint4& c, const uint4& d) {
        auto h = [](uint32_t x) { return *reinterpret_cast<const __nv_bfloat162*>(&x); };
        auto m4 = [&](const uint4& w) { return __hmax2(__hmax2(h(w.x), h(w.y)), __hmax2(h(w.z), h(w.w))); };
        __nv_bfloat162 m = __hmax2(__hmax2(m4(a), m4(b)), __hmax2(m4(c), m4(d)));
        uint32_t bits = *reinterpret_cast<uint32_t*>(&m);
        return fmaxf(__uint_as_float(bits << 16), __uint_as_float(bits & 0xffff0000u));
    }
};
template <> struct Elem<CADD_DTYPE_FP32> {
    static constexpr int ES = 4;
    static constexpr int EPC = 4;
    static __device__ __forceinline__ float load(const void* row, int64_t i) { return ((const float*)row)[i]; }
    static __device__ __forceinline__ void unpack(const uint4& w, float* f) {
        f[0] = __uint_as_float(w.x); f[1] = __uint_as_float(w.y);
        f[2] = __uint_as_float(w.z); f[3] = __uint_as_float(w.w);
    }
    static __device__ __forceinline__ float chunk_max(const uint4& w) {
        return fmaxf(fmaxf(__uint_as_float(w.x), __uint_as_float(w.y)),
                     fmaxf(__uint_as_float(w.z), __uint_as_float(w.w)));
    }
    static __device__ __forceinline__ float max4(const uint4& a, const uint4& b, const uint4& c, const uint4& d) {
        return fmaxf(fmaxf(chunk_max(a), chunk_max(b)), fmaxf(chunk_max(c), chunk_max(d)));
    }
};

// How a row of V elements starting at `row` splits into scalar head, 16-byte chunks and scalar tail.
struct RowSplit {
    int head;        // elements before the first 16-byte boundary
    int n_chunks;    // aligned chunks
    int tail;        // elements after the last whole chunk
};
template <int DT>
__device__ __forceinline__ RowSplit split_row(const void* row, int64_t V) {
    using E = Elem<DT>;
    RowSplit s;
    int mis = (int)(((uintptr_t)row & 15u) / E::ES);
    int64_t head = mis ? (E::EPC - mis) : 0;
    if (head > V) head = V;
    s.head = (int)head;
    s.n_chunks = (int)((V - head) / E::EPC);
    s.tail = (int)(V - head - (int64_t)s.n_chunks * E::EPC);
    return s;
}

__device__ __forceinline__ int clamp_l_eff(const int32_t* l_eff, int b, int L, int* clamped) {
    int le = l_eff ? l_eff[b] : L;
    *clamped = 0;
    if (le < 0) { le = 0; *clamped = 1; }
    if (le > L) { le = L; *clamped = 1; }
    return le;
}

}  // namespace cadd
