// Device-side building blocks shared by the spec_verify kernels: element access for
// fp32 / bf16 logits rows, the base-2 exponential, warp and block reductions, and the
// merge of running (reference, sum) pairs of the online softmax.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace specv {

constexpr int kF32 = 0;
constexpr int kBF16 = 1;
constexpr int kF16 = 2;

// Finite stand-in for "no maximum seen yet".  Finite so that (-inf logit) - reference
// is -inf, never NaN: masked logits (-inf) then contribute exactly 0.
constexpr float kNoMax = -3.0e38f;

// Debug build (-DSPECV_DEBUG): every row index and token id the streaming kernels compute is
// range-checked before it is used; a violation is recorded (the largest site code seen, readable
// through spec_verify_debug_violation) and the access is skipped -- nothing traps.  In the normal
// build the checks compile to nothing.
#ifdef SPECV_DEBUG
__device__ int g_debug_violation = 0;
__device__ __forceinline__ bool debug_in_range(bool ok, int site) {
    if (!ok) atomicMax(&g_debug_violation, site);
    return ok;
}
#else
__device__ __forceinline__ bool debug_in_range(bool, int) { return true; }
#endif
constexpr double kLog2e = 1.4426950408889634074;

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two fp32 values in one 64-bit register and the packed arithmetic of sm_100 on them: one
// instruction does two IEEE operations (same results as the scalar forms), which halves the
// instruction count of the multiply-add and of the accumulation in the streaming loops.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b,
                                                        unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// 16-byte read-only load that does not allocate in L1 (every logit is used once per pass).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <int DT>
struct Elt;

template <>
struct Elt<kF32> {
    static constexpr int kBytes = 4;
    static constexpr int kPerVec = 4;                // elements in 16 bytes
    static constexpr uint32_t kNegInfWord = 0xff800000u;
    __device__ static __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = __uint_as_float(v.x);
        x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z);
        x[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float load1(const char* row, int64_t j) {
        return reinterpret_cast<const float*>(row)[j];
    }
    // 16 bytes starting at element j0, element by element, -inf beyond V.
    __device__ static __forceinline__ uint4 gather(const char* row, int64_t j0, int64_t V) {
        const uint32_t* r = reinterpret_cast<const uint32_t*>(row);
        uint4 v;
        v.x = (j0 + 0 < V) ? r[j0 + 0] : kNegInfWord;
        v.y = (j0 + 1 < V) ? r[j0 + 1] : kNegInfWord;
        v.z = (j0 + 2 < V) ? r[j0 + 2] : kNegInfWord;
        v.w = (j0 + 3 < V) ? r[j0 + 3] : kNegInfWord;
        return v;
    }
};

template <>
struct Elt<kBF16> {
    static constexpr int kBytes = 2;
    static constexpr int kPerVec = 8;
    static constexpr uint32_t kNegInfWord = 0xff80ff80u;   // two bf16 -inf
    __device__ static __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
        x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
        x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    __device__ static __forceinline__ float load1(const char* row, int64_t j) {
        return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(row)[j]) << 16);
    }
    __device__ static __forceinline__ uint32_t pair(const uint16_t* r, int64_t j, int64_t V) {
        uint32_t lo = (j < V) ? r[j] : 0xff80u;
        uint32_t hi = (j + 1 < V) ? r[j + 1] : 0xff80u;
        return lo | (hi << 16);
    }
    __device__ static __forceinline__ uint4 gather(const char* row, int64_t j0, int64_t V) {
        const uint16_t* r = reinterpret_cast<const uint16_t*>(row);
        uint4 v;
        v.x = pair(r, j0 + 0, V);
        v.y = pair(r, j0 + 2, V);
        v.z = pair(r, j0 + 4, V);
        v.w = pair(r, j0 + 6, V);
        return v;
    }
};

template <>
struct Elt<kF16> {
    static constexpr int kBytes = 2;
    static constexpr int kPerVec = 8;
    static constexpr uint32_t kNegInfWord = 0xfc00fc00u;   // two fp16 -inf
    __device__ static __forceinline__ void unpack2(uint32_t w, float& lo, float& hi) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        lo = f.x; hi = f.y;
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float* x) {
        unpack2(v.x, x[0], x[1]); unpack2(v.y, x[2], x[3]);
        unpack2(v.z, x[4], x[5]); unpack2(v.w, x[6], x[7]);
    }
    __device__ static __forceinline__ float load1(const char* row, int64_t j) {
        return __half2float(reinterpret_cast<const __half*>(row)[j]);
    }
    __device__ static __forceinline__ uint32_t pair(const uint16_t* r, int64_t j, int64_t V) {
        uint32_t lo = (j < V) ? r[j] : 0xfc00u;
        uint32_t hi = (j + 1 < V) ? r[j + 1] : 0xfc00u;
        return lo | (hi << 16);
    }
    __device__ static __forceinline__ uint4 gather(const char* row, int64_t j0, int64_t V) {
        const uint16_t* r = reinterpret_cast<const uint16_t*>(row);
        uint4 v;
        v.x = pair(r, j0 + 0, V);
        v.y = pair(r, j0 + 2, V);
        v.z = pair(r, j0 + 4, V);
        v.w = pair(r, j0 + 6, V);
        return v;
    }
};

// Vector number `v` of a row (elements v*kPerVec ...): one 16-byte load when the row
// starts on a 16-byte boundary and the vector lies inside the row, else element loads.
template <int DT>
__device__ __forceinline__ uint4 load_vec(const char* row, bool row_aligned, int64_t v, int64_t V) {
    const int64_t j0 = v * Elt<DT>::kPerVec;
    if (row_aligned && j0 + Elt<DT>::kPerVec <= V) return ld_stream16(row + j0 * Elt<DT>::kBytes);
    return Elt<DT>::gather(row, j0, V);
}

__device__ __forceinline__ uint4 neg_inf_vec(uint32_t word) { return make_uint4(word, word, word, word); }

// (reference, sum) pairs: sum_j 2^(t_j - ref).  Merge two of them onto the larger reference.
__device__ __forceinline__ void merge_ref_sum(float& ref, float& sum, float oref, float osum) {
    const float nref = fmaxf(ref, oref);
    sum = sum * ex2_approx(ref - nref) + osum * ex2_approx(oref - nref);
    ref = nref;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double shfl_up_double(double v, int delta) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_up_sync(0xffffffffu, lo, delta);
    hi = __shfl_up_sync(0xffffffffu, hi, delta);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double shfl_double(double v, int src) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src);
    hi = __shfl_sync(0xffffffffu, hi, src);
    return __hiloint2double(hi, lo);
}

// Inclusive prefix sum across the 32 lanes of a warp.
__device__ __forceinline__ double warp_inclusive_scan(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = shfl_up_double(v, o);
        if (lane >= o) v += up;
    }
    return v;
}

}  // namespace specv
