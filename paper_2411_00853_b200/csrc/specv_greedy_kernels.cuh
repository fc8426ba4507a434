// Greedy verification (the temperature -> 0 limit of the verify-and-resample pass of the
// paper's section "Speculative Sampling Results"): a draft token is accepted iff it is the
// argmax of its target row; the token emitted after the accepted prefix is the argmax of the
// next target row.  Only target rows are read, each once.
//
//   specv_prologue        (shared) offsets, per-sequence checks, -1 fill
//   specv_ring_argmax     persistent CTAs, one per SM; rows stream through the shared-memory
//                         ring of the ring kernel set; sixteen warps keep (largest value, first
//                         16-byte vector that holds it) per lane; one warp merges and finds the
//                         element inside the winning vector
//   specv_row_argmax      the same result with plain loads, for any pitch and alignment
//   specv_greedy_resolve  one warp per sequence: first mismatch, emit
//
// Ties: the smallest token id among equal largest logits; NaN is never the largest; a row with
// nothing above -inf gives token 0.
#pragma once

#include "specv_ring_kernels.cuh"

namespace specv {

constexpr int32_t kNoVec = 0x7fffffff;

// Candidate order: larger value first, then smaller vector index.  A total order, so the result
// of any reduction tree is the same.
__device__ __forceinline__ void best_take(float& val, int32_t& vec, float oval, int32_t ovec) {
    if (oval > val || (oval == val && ovec < vec)) { val = oval; vec = ovec; }
}

// Largest element of one 16-byte vector (NaN elements are ignored).
template <int DT>
__device__ __forceinline__ float vec_max(const uint4& a) {
    if (DT == kBF16) {
        const uint32_t m2 = max_bf16x2(max_bf16x2(a.x, a.y), max_bf16x2(a.z, a.w));
        return fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
    } else if (DT == kF16) {
        const uint32_t m2 = max_f16x2(max_f16x2(a.x, a.y), max_f16x2(a.z, a.w));
        float lo, hi;
        Elt<kF16>::unpack2(m2, lo, hi);
        return fmaxf(lo, hi);
    } else {
        return fmaxf(fmaxf(__uint_as_float(a.x), __uint_as_float(a.y)),
                     fmaxf(__uint_as_float(a.z), __uint_as_float(a.w)));
    }
}

// Token id from the winning (value, vector): first element of that vector equal to the value.
template <int DT>
__device__ __forceinline__ int32_t token_in_vector(const uint4& raw, float val, int32_t vec) {
    constexpr int N = Elt<DT>::kPerVec;
    if (vec == kNoVec) return 0;
    float x[N];
    Elt<DT>::unpack(raw, x);
    int k_sel = 0;
#pragma unroll
    for (int k = N - 1; k >= 0; --k)
        if (x[k] == val) k_sel = k;
    return vec * N + k_sel;
}

__device__ __forceinline__ void warp_best(float& val, int32_t& vec) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float oval = __shfl_xor_sync(0xffffffffu, val, o);
        const int32_t ovec = __shfl_xor_sync(0xffffffffu, vec, o);
        best_take(val, vec, oval, ovec);
    }
}

// ---------------------------------------------------------------------------------
// specv_ring_argmax
// ---------------------------------------------------------------------------------
constexpr int kArgMergeWarp = kCWarps;          // [0,16) scanning warps, 16 merge, 17 bulk copies
constexpr int kArgCopyWarp = kCWarps + 1;
constexpr int kRingArgmaxThreads = (kArgCopyWarp + 1) * 32;

struct RingArgmaxShared {
    ChunkRing ring;
    unsigned long long item_done[kItemDepth], item_free[kItemDepth];
    float wval[kItemDepth][kCWarps];
    int32_t wvec[kItemDepth][kCWarps];
    int err;
};
static_assert(sizeof(RingArgmaxShared) <= 227 * 1024, "RingArgmaxShared exceeds the shared memory of one CTA");

template <int DT>
__global__ void __launch_bounds__(kRingArgmaxThreads, 1)
specv_ring_argmax(const char* __restrict__ target, int64_t pitch_t, int64_t V, int64_t n_rows,
                  int32_t* __restrict__ argmax_out, int32_t* __restrict__ ctrl) {
    using E = Elt<DT>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RingArgmaxShared& sh = *reinterpret_cast<RingArgmaxShared*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row_bytes = V * E::kBytes;
    const int nck = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);
    constexpr int kQuarterVecs = kChunkBytes / kWarpsPerChunk / 16;

    ring_init(sh.ring, tid);
    if (tid >= 32 && tid < 32 + kItemDepth) {
        mbar_init(smem_u32(&sh.item_done[tid - 32]), kCWarps);
        mbar_init(smem_u32(&sh.item_free[tid - 32]), 1);
    } else if (tid == 64) {
        sh.err = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    pdl_launch_dependents();
    // nothing the prologue writes is read here: the rows are the caller's; the wait for it sits
    // at the end, so that this grid never completes before the prologue has

    const int64_t cid = blockIdx.x, NC = gridDim.x;
    const int32_t J = n_rows > cid ? (int32_t)((n_rows - cid + NC - 1) / NC) : 0;
    volatile int* err = &sh.err;

    if (warp == kArgCopyWarp) {
        uint32_t g0 = 0;
        for (int32_t j = 0; j < J; ++j) {
            const char* src = target + (cid + (int64_t)j * NC) * pitch_t;
            if (!ring_issue_item(sh.ring, src, nullptr, 0, nck, row_bytes, g0, lane, err, 21)) break;
            g0 += nck;
        }
        if (*err) ring_drain(sh.ring, lane);
    } else if (warp < kCWarps) {
        const int group = warp / kWarpsPerChunk, sub = warp % kWarpsPerChunk;
        uint32_t g0 = 0;
        RingRun run;
        for (int32_t j = 0; j < J; ++j) {
            float best = __uint_as_float(0xff800000u);
            int32_t bvec = kNoVec;
            run.begin_item(g0, g0 % kChunkGroups);      // chunk ci of a row goes to warp group ci % 4
            for (int ci = group; ci < nck; ci += kChunkGroups) {
                const uint32_t gi = g0 + ci;
                const uint32_t s = gi % kRingSlots;
                ring_wait_chunk(sh.ring, gi, run.guard_until, err, 22);
                const int64_t rem = row_bytes - (int64_t)ci * kChunkBytes;
                const int nvec_q = (int)((rem < kChunkBytes ? rem : kChunkBytes) / 16) - sub * kQuarterVecs;
                const unsigned char* quarter = sh.ring.slot[s] + sub * (kChunkBytes / kWarpsPerChunk);
                uint4 a[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int v = lane + 32 * i;
                    a[i] = v < nvec_q ? *reinterpret_cast<const uint4*>(quarter + v * 16) : neg_inf_vec(E::kNegInfWord);
                }
                const int32_t vbase = ci * (kChunkBytes / 16) + sub * kQuarterVecs + lane;
#pragma unroll
                for (int i = 0; i < 4; ++i) {      // increasing vector index: ">" keeps the first
                    const float m = vec_max<DT>(a[i]);
                    if (m > best) { best = m; bvec = vbase + 32 * i; }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.ring.empty_bar[s]));   // quarter consumed
            }
            warp_best(best, bvec);
            const int is = j % kItemDepth;
            if (lane == 0) {
                mbar_wait(smem_u32(&sh.item_free[is]), ((j / kItemDepth) & 1) ^ 1, err, 23);
                sh.wval[is][warp] = best;
                sh.wvec[is][warp] = bvec;
                mbar_arrive(smem_u32(&sh.item_done[is]));
            }
            g0 += nck;
        }
    } else if (warp == kArgMergeWarp) {
        for (int32_t j = 0; j < J; ++j) {
            const int is = j % kItemDepth;
            mbar_wait(smem_u32(&sh.item_done[is]), (j / kItemDepth) & 1, err, 24);
            float val = lane < kCWarps ? sh.wval[is][lane] : __uint_as_float(0xff800000u);
            int32_t vec = lane < kCWarps ? sh.wvec[is][lane] : kNoVec;
            warp_best(val, vec);
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.item_free[is]));   // this warp is the only waiter
                if (!*err) {
                    const int64_t row = cid + (int64_t)j * NC;
                    uint4 raw = neg_inf_vec(E::kNegInfWord);
                    if (vec != kNoVec) raw = ld_stream16(target + row * pitch_t + (int64_t)vec * 16);
                    argmax_out[row] = token_in_vector<DT>(raw, val, vec);
                }
            }
            __syncwarp();
        }
    }
    __syncthreads();
    pdl_wait_for_predecessor();
    if (tid == 0 && sh.err) atomicExch(&ctrl[0], sh.err);
}

// ---------------------------------------------------------------------------------
// specv_row_argmax: a block per row, plain loads
// ---------------------------------------------------------------------------------
constexpr int kArgmaxThreads = 256;

template <int DT>
__global__ void __launch_bounds__(kArgmaxThreads)
specv_row_argmax(const char* __restrict__ target, int64_t pitch_t, int64_t V, int64_t n_rows,
                 int32_t* __restrict__ argmax_out) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    constexpr int U = 4;
    __shared__ float wval[kArgmaxThreads / 32];
    __shared__ int32_t wvec[kArgmaxThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    const int64_t nvec = (V + N - 1) / N;
    for (int64_t row = blockIdx.x; row < n_rows; row += gridDim.x) {
        const char* rp = target + row * pitch_t;
        const bool aligned = (reinterpret_cast<uintptr_t>(rp) & 15u) == 0;
        float best = __uint_as_float(0xff800000u);
        int32_t bvec = kNoVec;
        for (int64_t v = tid; v < nvec; v += kArgmaxThreads * U) {
            uint4 raw[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int64_t vv = v + (int64_t)k * kArgmaxThreads;
                raw[k] = vv < nvec ? load_vec<DT>(rp, aligned, vv, V) : neg_inf_vec(E::kNegInfWord);
            }
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const float m = vec_max<DT>(raw[k]);
                if (m > best) { best = m; bvec = (int32_t)(v + (int64_t)k * kArgmaxThreads); }
            }
        }
        warp_best(best, bvec);
        if (lane == 0) { wval[warp] = best; wvec[warp] = bvec; }
        __syncthreads();
        if (warp == 0) {
            float val = lane < kArgmaxThreads / 32 ? wval[lane] : __uint_as_float(0xff800000u);
            int32_t vec = lane < kArgmaxThreads / 32 ? wvec[lane] : kNoVec;
            warp_best(val, vec);
            if (lane == 0) {
                uint4 raw = neg_inf_vec(E::kNegInfWord);
                if (vec != kNoVec) raw = load_vec<DT>(rp, aligned, vec, V);
                argmax_out[row] = token_in_vector<DT>(raw, val, vec);
            }
        }
        __syncthreads();
    }
    pdl_wait_for_predecessor();   // never complete before the prologue has (see specv_ring_argmax)
}

// ---------------------------------------------------------------------------------
// specv_greedy_resolve: one warp per sequence
// ---------------------------------------------------------------------------------
constexpr int kGreedyResolveThreads = 128;

__global__ void __launch_bounds__(kGreedyResolveThreads)
specv_greedy_resolve(BatchView in, const int32_t* __restrict__ off_d, const int32_t* __restrict__ seq_status,
                     const int32_t* __restrict__ argmax, const int32_t* __restrict__ ctrl,
                     int32_t* __restrict__ accepted_len, int32_t* __restrict__ emitted,
                     int32_t* __restrict__ row_status) {
    const int lane = threadIdx.x & 31;
    const int32_t b = blockIdx.x * (kGreedyResolveThreads / 32) + (threadIdx.x >> 5);
    pdl_wait_for_predecessor();
    if (b >= in.B) return;
    const int error_word = ctrl ? ctrl[0] : 0;
    int status = seq_status[b] | (error_word ? (16 | (error_word << 8)) : 0);
    const int32_t k_raw = in.k_per_row ? in.k_per_row[b] : in.k_uniform;
    const int32_t K = k_raw > 0 ? k_raw : 0;
    const int64_t d0 = off_d[b], t0 = d0 + b;
    if (!(status & 1)) {
        bool bad = false;
        for (int32_t i = lane; i < K; i += 32) {
            const int32_t x = in.tokens[d0 + i];
            bad |= (x < 0 || (int64_t)x >= in.V);
        }
        if (__any_sync(0xffffffffu, bad)) status |= 4;   // SPECV_ROW_BAD_TOKEN
    }
    if (status) {
        if (lane == 0) {
            accepted_len[b] = 0;
            if (row_status) row_status[b] = status;
        }
        return;   // the prologue already wrote -1 into every slot
    }
    int32_t n = K;
    for (int32_t base = 0; base < K && n == K; base += 32) {
        const int32_t i = base + lane;
        const bool miss = i < K && in.tokens[d0 + i] != argmax[t0 + i];
        const unsigned m = __ballot_sync(0xffffffffu, miss);
        if (m) n = base + __ffs(m) - 1;
    }
    for (int32_t i = lane; i <= n; i += 32) emitted[t0 + i] = i < n ? in.tokens[d0 + i] : argmax[t0 + n];
    if (lane == 0) {
        accepted_len[b] = n;
        if (row_status) row_status[b] = 0;
    }
}

}  // namespace specv
