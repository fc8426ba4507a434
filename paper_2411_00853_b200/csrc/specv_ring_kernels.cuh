// The ring kernel set: the same steps as the streaming set (offsets, row statistics, resolve),
// in two kernels built around a shared-memory ring that bulk async copies keep full, so that the
// arithmetic never waits for anything but HBM.  There is no prologue kernel in the normal form:
// every CTA scans the lookahead lengths itself, the first CTA of the statistics kernel writes the
// per-sequence argument checks, the resolve kernel writes the -1 padding.  (The early-exit form at
// the end of this file, and the tree and greedy passes, still start with specv_prologue.)
//
//   specv_ring_stats    persistent CTAs, one per SM.  The batch is cut into equal byte ranges,
//                       one per CTA: all 16 KB units (chunk k of a target row with chunk k of the
//                       draft row of the same position, or two chunks of a last target row) are
//                       numbered in row order and CTA c takes units [c q, (c+1) q), so a row
//                       (pair) may be shared by up to kStatParts CTAs, each storing the statistics
//                       of its part.  Eight lanes of one warp issue 8 KB bulk copies into a
//                       24-slot ring, prefetching across items; sixteen warps turn chunks into
//                       online-softmax statistics and release them at once; one warp merges the
//                       sixteen partials of an item and stores them.
//   specv_ring_resolve  persistent CTAs.  The rows to draw from (one pair or one row per sequence)
//                       are again cut into equal ranges of chunk columns; one warp decides the
//                       sequences a CTA touches (acceptance tests of all draft positions in double,
//                       first rejection); the copy warp streams the CTA's parts through the same
//                       ring; sixteen warps turn chunks into segment sums of max(0, p - q) (or p)
//                       in a global table; the CTA that finishes a sequence's last part does the
//                       prefix / locate step of the inverse CDF and emits.
//
// Steps and formulas: the verify-and-resample pass of the paper's section "Speculative
// Sampling Results" with the accept / residual rule stated in include/spec_verify.h.
#pragma once

#include <cuda_runtime.h>

#include "specv_device.cuh"
#include "specv_stream_kernels.cuh"

namespace specv {

constexpr int kChunkBytes = 8192;
constexpr int kRingSlots = 24;
constexpr int kCWarps = 16;                     // consumer warps of both kernels
constexpr int kWarpsPerChunk = 4;               // resolve, argmax: a chunk is consumed by four warps, 2 KB each
constexpr int kChunkGroups = kCWarps / kWarpsPerChunk;
constexpr int kStatsWarpsPerChunk = 2;          // statistics: two warps, 4 KB each (fewer waits, arrivals and
constexpr int kStatsGroups = kCWarps / kStatsWarpsPerChunk;   // loop turns per logit)
static_assert(kRingSlots % kStatsGroups == 0 && kRingSlots % (2 * kChunkGroups) == 0,
              "within an item a ring slot must fall to the same warp group lap after lap");
constexpr int kCopyLanes = 8;                   // lanes of the copy warp that issue bulk copies
constexpr int kDescBatch = 32;                  // items described per batch (one per lane)
constexpr int kItemDepth = 8;                   // items the statistics warps may run ahead of the merge
constexpr int kPartDepth = 16;                  // part records in flight per CTA of the resolve kernel
constexpr int kMaxSegs = 2048;                  // segment table of the sampler
constexpr int kStatParts = 4;                   // statistics slots per logits row: CTAs that may share a row
constexpr int kMaxRingSeqs = 4095;              // the ring kernels keep B + 1 offsets in shared memory
constexpr long long kWaitLimitCycles = 2000000000LL;   // ~1 s: a wait that long is a failure

// warp roles
constexpr int kMergeWarp = kCWarps;             // specv_ring_stats: [0,16) statistics, 16 merge,
constexpr int kStatsCopyWarp = kCWarps + 1;     // 17 bulk copies, 18 descriptors
constexpr int kStatsDescWarp = kCWarps + 2;
constexpr int kRingStatsThreads = (kStatsDescWarp + 1) * 32;
constexpr int kResolveCopyWarp = kCWarps;       // specv_ring_resolve: [0,16) segment sums, 16 bulk
constexpr int kLocatorWarp = kCWarps + 1;       // copies, 17 prefix / locate / emit, 18 part records
constexpr int kFetchWarp = kCWarps + 2;
constexpr int kRingResolveThreads = (kFetchWarp + 1) * 32;

struct RingScratch {
    int32_t* off_d;         // [B+1]   (prologue kernel only; the ring kernels scan their own copy)
    int32_t* seq_status;    // [B]     argument checks (first CTA of specv_ring_stats, or the prologue)
    float2* stat_p;         // [(D+B) * kStatParts]  (ref, sum) of the parts of every target row
    float2* stat_q;         // [D * kStatParts]      same for every draft row; unused slots hold (kNoMax, 0)
    int32_t* done;          // [B]     chunk columns whose segment sums are in gseg (zeroed where seq_status is written)
    float* gseg;            // [B * nseg]  segment sums of the distribution the token is drawn from
    int32_t* ctrl;          // [0] error word of the ring kernels (0: none), [1] unused,
                            // [2] early-exit form: number of work items, [3] rows it did not read, [4] its work counter
    // early-exit form only
    int32_t* item_seq;      // [D+B]   work list, ordered by position first
    int32_t* item_pos;      // [D+B]
    int32_t* level_start;   // [D+2]
    int32_t* first_rej;     // [B]     smallest position known to be rejected with a clear margin
};

// ---------------------------------------------------------------------------------
// PTX helpers: mbarriers, bulk async copy
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  On expiry (or once another wait of this CTA has expired) raises *err and
// returns; the caller carries on with whatever is in memory -- every later access stays in
// bounds by construction -- so that all barriers are still reached and the kernel ends.
// `site` (non-zero) names the wait in the error word, for diagnosis.
//
// A parity wait is only sound while the barrier is at most one phase ahead of the waiter;
// every barrier below is used so that its next phase cannot complete before all waiters of
// the current one are through.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* err, int site,
                                          long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*err) return;
        if (clock64() - t0 > limit_cycles) { *err = site; return; }
    }
}

// Self-test of the bounded wait (spec_verify_selftest_bounded_wait): one warp waits on a barrier
// that nothing ever completes, with a short limit.  The wait must give up, name itself in the
// error word, and every later wait of the CTA must return at once; the kernel ends normally.
// out[0]: error word, out[1]: clock cycles the first wait took, out[2]: cycles of a second wait,
// out[3]: 1 once the end of the kernel is reached.
__global__ void specv_selftest_bounded_wait(long long limit_cycles, long long* out) {
    __shared__ unsigned long long never[2];
    __shared__ int err_word;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never[0]), 1);
        mbar_init(smem_u32(&never[1]), 1);
        err_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int* err = &err_word;
    const long long t0 = clock64();
    mbar_wait(smem_u32(&never[0]), 0, err, 77, limit_cycles);      // phase 0 never completes
    const long long t1 = clock64();
    __syncwarp();
    mbar_wait(smem_u32(&never[1]), 0, err, 78, limit_cycles);      // another barrier: returns because the CTA has failed
    const long long t2 = clock64();
    __syncthreads();
    if (threadIdx.x == 0) {
        out[0] = err_word;
        out[1] = t1 - t0;
        out[2] = t2 - t1;
        out[3] = 1;
    }
    (void)lane;
}
// Plain bulk copy global -> this CTA's shared memory, completion on this CTA's mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Programmatic dependent launch: the next kernel of the stream may be scheduled while this one
// still runs (its CTAs start as SMs free up and do their set-up), and waits here for this grid
// to have finished and flushed before it touches anything this grid wrote.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d; asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}
__device__ __forceinline__ uint32_t max_f16x2(uint32_t a, uint32_t b) {
    uint32_t d; asm("max.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}

// The chunk ring and its barriers; both kernels embed one.
struct ChunkRing {
    alignas(128) unsigned char slot[kRingSlots][kChunkBytes];
    unsigned long long full_bar[kRingSlots];    // armed by the copy warp, completed by the copy's bytes
    unsigned long long empty_bar[kRingSlots];   // one arrival per consuming warp
    signed char armed_parity[kRingSlots];       // parity of the last copy armed on a slot, -1: none
};

// Called by every thread of the CTA (one slot per thread; a fence and a CTA barrier must follow).
__device__ __forceinline__ void ring_init(ChunkRing& ring, int tid, int warps_per_chunk = kWarpsPerChunk) {
    if (tid < kRingSlots) {
        mbar_init(smem_u32(&ring.full_bar[tid]), 1);
        mbar_init(smem_u32(&ring.empty_bar[tid]), warps_per_chunk);
        ring.armed_parity[tid] = -1;
    }
}

// Consumer: wait until the chunk at ring position gi has landed in its slot.  A parity wait is
// only sound when the barrier is at most one phase short of the one asked about.  Within an item
// a slot is taken by the same warps lap after lap (the ring has a multiple of four slots), and so
// it is across items as long as their first ring positions agree modulo the warp-group stride;
// where they do not, the slot's consumers in consecutive laps are different warps, and one of
// them may run a whole lap ahead of a chunk that is still in flight -- its wait would pass one
// phase early.  So for the first lap after such a change (positions below guard_until) the
// slot's previous chunk is first known to have been released, which implies it had landed.
struct RingRun {               // per consumer warp: the current run of items whose mapping agrees
    uint32_t key = 0xffffffffu;
    uint32_t guard_until = 0;  // ring positions below this need the extra wait
    __device__ __forceinline__ void begin_item(uint32_t g0, uint32_t item_key) {
        if (item_key != key) { key = item_key; guard_until = g0 + kRingSlots; }
    }
};
__device__ __forceinline__ void ring_wait_chunk(ChunkRing& ring, uint32_t gi, uint32_t guard_until,
                                                volatile int* err, int site) {
    const uint32_t s = gi % kRingSlots, lap = gi / kRingSlots;
    if (lap > 0 && gi < guard_until) mbar_wait(smem_u32(&ring.empty_bar[s]), (lap - 1) & 1, err, site);
    mbar_wait(smem_u32(&ring.full_bar[s]), lap & 1, err, site);
}

// Copy warp: issue chunks [ci0, ci1) of one item (rows interleaved chunk by chunk when there are
// two: chunk ci is chunk ci/2 of the target row for even ci, of the draft row for odd ci).  Chunk
// ci goes to ring position g0 + ci - ci0.  kCopyLanes lanes issue one chunk each per round: a
// single thread cannot issue 8 KB copies fast enough for an SM's share of HBM bandwidth.
// Returns false once a wait has failed.
__device__ __forceinline__ bool ring_issue_item(ChunkRing& ring, const char* src_p, const char* src_q, int ci0,
                                                int ci1, int64_t row_bytes, uint32_t g0, int lane,
                                                volatile int* err, int site) {
    const bool pair = src_q != nullptr;
    for (int c0 = ci0; c0 < ci1; c0 += kCopyLanes) {
        const int ci = c0 + lane;
        if (lane < kCopyLanes && ci < ci1) {
            const int k = pair ? (ci >> 1) : ci;
            const int64_t rem = row_bytes - (int64_t)k * kChunkBytes;
            const uint32_t bytes = rem < kChunkBytes ? (uint32_t)rem : kChunkBytes;
            const uint32_t gi = g0 + (uint32_t)(ci - ci0);
            const uint32_t s = gi % kRingSlots;
            mbar_wait(smem_u32(&ring.empty_bar[s]), ((gi / kRingSlots) & 1) ^ 1, err, site);
            if (!*err) {
                const uint32_t fb = smem_u32(&ring.full_bar[s]);
                mbar_expect_tx(fb, bytes);
                ring.armed_parity[s] = (signed char)((gi / kRingSlots) & 1);
                bulk_load(smem_u32(&ring.slot[s][0]), ((pair && (ci & 1)) ? src_q : src_p) + (int64_t)k * kChunkBytes,
                          bytes, fb);
            }
        }
        __syncwarp();
        if (*err) return false;
    }
    return true;
}

// Copy warp, after a failure: make sure no copy of ours is still in flight when the CTA ends --
// wait (with the limit) for the last phase armed on each slot.
__device__ __forceinline__ void ring_drain(ChunkRing& ring, int lane) {
    __syncwarp();
    if (lane < kRingSlots) {
        const int ap = ring.armed_parity[lane];
        const uint32_t fb = smem_u32(&ring.full_bar[lane]);
        const long long t0 = clock64();
        while (ap >= 0 && !mbar_try_wait(fb, (uint32_t)ap) && clock64() - t0 < kWaitLimitCycles) {}
    }
}

// ---------------------------------------------------------------------------------
// specv_ring_stats
// ---------------------------------------------------------------------------------
// Online-softmax update of one lane with its share of a warp's part of a chunk (NV 16-byte
// vectors per lane: 4 KB per warp with NV = 8): the lane keeps its own reference (the scaled
// maximum of what it has seen) and four partial sums, so nothing is exchanged between lanes
// until the item ends.
template <int DT, int NV>
__device__ __forceinline__ void part_stats(const unsigned char* quarter, int nvec_q, float c, int lane,
                                           float& ref, float (&s)[4]) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    uint4 a[NV];
    if (nvec_q >= NV * 32) {      // a whole part (all but a row's last chunk): no bounds to mind
#pragma unroll
        for (int i = 0; i < NV; ++i) a[i] = *reinterpret_cast<const uint4*>(quarter + (lane + 32 * i) * 16);
    } else {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int v = lane + 32 * i;
            a[i] = v < nvec_q ? *reinterpret_cast<const uint4*>(quarter + v * 16) : neg_inf_vec(E::kNegInfWord);
        }
    }
    float mx;
    if (DT == kBF16) {
        uint32_t m2 = 0xff80ff80u;
#pragma unroll
        for (int i = 0; i < NV; ++i)
            m2 = max_bf16x2(max_bf16x2(m2, a[i].x), max_bf16x2(a[i].y, max_bf16x2(a[i].z, a[i].w)));
        mx = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
    } else if (DT == kF16) {
        uint32_t m2 = 0xfc00fc00u;
#pragma unroll
        for (int i = 0; i < NV; ++i)
            m2 = max_f16x2(max_f16x2(m2, a[i].x), max_f16x2(a[i].y, max_f16x2(a[i].z, a[i].w)));
        float lo, hi;
        Elt<kF16>::unpack2(m2, lo, hi);
        mx = fmaxf(lo, hi);
    } else {
        mx = __uint_as_float(0xff800000u);
#pragma unroll
        for (int i = 0; i < NV; ++i)
            mx = fmaxf(fmaxf(mx, __uint_as_float(a[i].x)),
                       fmaxf(__uint_as_float(a[i].y), fmaxf(__uint_as_float(a[i].z), __uint_as_float(a[i].w))));
    }
    const float cand = mx * c;
    if (cand > ref) {   // rare after the first chunks
        const float f = ex2_approx(ref - cand);
        s[0] *= f; s[1] *= f; s[2] *= f; s[3] *= f;
        ref = cand;
    }
    // sums 0,1 and 2,3 ride in two packed registers; element k of a vector goes to sum k % 4
    const unsigned long long cc = pack_f32x2(c, c), nr = pack_f32x2(-ref, -ref);
    unsigned long long s01 = pack_f32x2(s[0], s[1]), s23 = pack_f32x2(s[2], s[3]);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        float x[N];
        E::unpack(a[i], x);
#pragma unroll
        for (int k = 0; k < N; k += 4) {
            float t0, t1, t2, t3;
            unpack_f32x2(fma_f32x2(pack_f32x2(x[k + 0], x[k + 1]), cc, nr), t0, t1);
            unpack_f32x2(fma_f32x2(pack_f32x2(x[k + 2], x[k + 3]), cc, nr), t2, t3);
            s01 = add_f32x2(s01, pack_f32x2(ex2_approx(t0), ex2_approx(t1)));
            s23 = add_f32x2(s23, pack_f32x2(ex2_approx(t2), ex2_approx(t3)));
        }
    }
    unpack_f32x2(s01, s[0], s[1]);
    unpack_f32x2(s23, s[2], s[3]);
}

// Statistics warp: this warp's share of chunks [ci0, ci1) of an item (ring positions g0 ..).  A
// group of two warps takes one chunk at a time, half each; for two-row items chunk parity =
// row, and (ci0 being even) so is group parity.  Returns the warp's (ref, sum), lanes already merged.
template <int DT>
__device__ __forceinline__ float2 consume_stats_unit(ChunkRing& ring, RingRun& run, uint32_t g0, bool pair, int ci0,
                                                     int ci1, int64_t row_bytes, float c, int warp, int lane,
                                                     volatile int* err, int site) {
    run.begin_item(g0, g0 % kStatsGroups);      // chunk ci of an item goes to warp group (ci - ci0) % 8
    const int group = warp / kStatsWarpsPerChunk, sub = warp % kStatsWarpsPerChunk;
    constexpr int kPartBytes = kChunkBytes / kStatsWarpsPerChunk;
    float ref = kNoMax;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int ci = ci0 + group; ci < ci1; ci += kStatsGroups) {
        const uint32_t gi = g0 + (uint32_t)(ci - ci0);
        const uint32_t s = gi % kRingSlots;
        ring_wait_chunk(ring, gi, run.guard_until, err, site);
        const int k = pair ? (ci >> 1) : ci;
        const int64_t rem = row_bytes - (int64_t)k * kChunkBytes;
        const int nvec = (int)((rem < kChunkBytes ? rem : kChunkBytes) / 16);
        part_stats<DT, kPartBytes / 16 / 32>(ring.slot[s] + sub * kPartBytes, nvec - sub * (kPartBytes / 16), c, lane,
                                             ref, acc);
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ring.empty_bar[s]));   // this warp's part consumed
    }
    float sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        merge_ref_sum(ref, sum, __shfl_xor_sync(0xffffffffu, ref, o), __shfl_xor_sync(0xffffffffu, sum, o));
    return make_float2(ref, sum);
}

// Merge warp: the sixteen warp partials of a unit -> (p_ref, p_sum, q_ref, q_sum), valid in lane 0.
__device__ __forceinline__ float4 merge_warp_partials(const float2* wpart, bool pair, int lane) {
    const float2 wp = lane < kCWarps ? wpart[lane] : make_float2(kNoMax, 0.f);
    const bool is_q = pair && ((lane / kStatsWarpsPerChunk) & 1);
    float Rp = is_q ? kNoMax : wp.x, Sp = is_q ? 0.f : wp.y;
    float Rq = is_q ? wp.x : kNoMax, Sq = is_q ? wp.y : 0.f;
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
        merge_ref_sum(Rp, Sp, __shfl_xor_sync(0xffffffffu, Rp, o), __shfl_xor_sync(0xffffffffu, Sp, o));
        merge_ref_sum(Rq, Sq, __shfl_xor_sync(0xffffffffu, Rq, o), __shfl_xor_sync(0xffffffffu, Sq, o));
    }
    return make_float4(Rp, Sp, Rq, Sq);
}

// Quotient of two non-negative 64-bit numbers.  The general 64-bit division is a long routine
// (several hundred cycles); batches that matter keep both operands below 2^32.
__device__ __forceinline__ int64_t div_nn(int64_t a, int64_t b) {
    if (((uint64_t)a | (uint64_t)b) >> 32) return a / b;
    return (int64_t)((uint32_t)a / (uint32_t)b);
}

// Block-wide exclusive prefix: out[b] = min(val(0) + ... + val(b-1), limit) for b in [0, n]; also
// calls each(b, val(0) + ... + val(b-1)) with the unclamped prefix for b in [0, n).
// Every thread of the block calls it (nthreads = blockDim.x); warp_tot holds one entry per warp.
template <class F, class G>
__device__ __forceinline__ void block_exclusive_prefix(F val, int32_t n, int64_t limit, int32_t* out,
                                                       long long* warp_tot, int tid, int nthreads, G each) {
    const int lane = tid & 31, warp = tid >> 5;
    const int32_t per = (n + nthreads - 1) / nthreads;
    const int32_t b0 = min(tid * per, n), b1 = min(b0 + per, n);
    long long local = 0;
    for (int32_t b = b0; b < b1; ++b) local += val(b);
    long long incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const long long up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    long long run = incl - local;
    for (int w = 0; w < warp; ++w) run += warp_tot[w];
    for (int32_t b = b0; b < b1; ++b) {
        out[b] = (int32_t)(run < limit ? run : limit);
        each(b, run);
        run += val(b);
    }
    if (tid == nthreads - 1) out[n] = (int32_t)(run < limit ? run : limit);   // its range ends at n
    __syncthreads();
}

// Offsets of the ragged batch in shared memory: off[b] = min(sum_{c<b} max(K_c, 0), n_draft_total),
// exactly what the prologue kernel stores.  With `publish` the calling CTA also does the
// prologue's other per-sequence work: argument checks into seq_status, tickets zeroed.
__device__ __forceinline__ void block_offsets(const BatchView& in, int32_t* off, long long* warp_tot, int tid,
                                              int nthreads, bool publish, int32_t* seq_status, int32_t* done) {
    const int32_t* kp = in.k_per_row;
    const int32_t ku = in.k_uniform;
    if (!kp) {
        // every sequence has the same lookahead: no scan (the host has checked B * k_uniform == n_draft_total)
        for (int32_t b = tid; b <= in.B; b += nthreads) {
            const long long excl = (long long)b * ku;
            off[b] = (int32_t)(excl < in.n_draft_total ? excl : in.n_draft_total);
            if (publish && b < in.B) {
                const float T = in.temperature[in.per_row_temperature ? b : 0];
                seq_status[b] = (!(T > 0.0f) || isinf(T)) ? 2 : 0;          // SPECV_ROW_BAD_TEMPERATURE
                done[b] = 0;
            }
        }
        __syncthreads();
        return;
    }
    auto lookahead = [&](int32_t b) { const int32_t k = kp ? kp[b] : ku; return (long long)(k > 0 ? k : 0); };
    block_exclusive_prefix(lookahead, in.B, in.n_draft_total, off, warp_tot, tid, nthreads,
                           [&](int32_t b, long long excl) {
                               if (!publish) return;
                               const int32_t k_raw = kp ? kp[b] : ku;
                               int status = 0;
                               if (k_raw < 0 || excl + lookahead(b) > in.n_draft_total) status |= 1;   // SPECV_ROW_BAD_K
                               const float T = in.temperature[in.per_row_temperature ? b : 0];
                               if (!(T > 0.0f) || isinf(T)) status |= 2;                 // SPECV_ROW_BAD_TEMPERATURE
                               seq_status[b] = status;
                               done[b] = 0;
                           });
}

// The statistics pass as one sequence of 16 KB units in row order.  Target row t of sequence b at
// position pos: nck units if pos is a draft position (unit k = chunk k of the target row and
// chunk k of the draft row), else (the sequence's last target row) h = ceil(nck / 2) units of two
// chunks.  With K_b = off[b+1] - off[b] (the offsets the prologue also computes, clamped to the
// buffers), sequence b starts at unit nck * off[b] + h * b.
struct StatsUnits {
    const int32_t* off;    // [B+1]
    int32_t B, nck, h;
    __device__ __forceinline__ int64_t seq_start(int32_t b) const { return (int64_t)nck * off[b] + (int64_t)h * b; }
    __device__ __forceinline__ int64_t total() const { return seq_start(B); }
    // packed target row that holds unit x (0 <= x < total)
    __device__ __forceinline__ int64_t row_of_unit(int64_t x) const {
        int32_t lo = 0, hi = B;   // invariant: seq_start(lo) <= x, answer in [lo, hi)
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (seq_start(mid) <= x) lo = mid; else hi = mid;
        }
        const int64_t r = x - seq_start(lo);
        const int64_t K = off[lo + 1] - off[lo];
        const int64_t pos = div_nn(r, nck) < K ? div_nn(r, nck) : K;
        return (int64_t)off[lo] + lo + pos;
    }
};

// One CTA's share of one item (a target row, with the draft row of the same position if there is one).
struct __align__(16) StatsItem {   // 32 bytes
    int64_t trow, drow;            // packed row indices; drow < 0: target row alone
    float c;                       // log2(e) / T of the row's sequence
    int32_t ci0, ci1;              // chunks of the item this CTA takes (numbering of ring_issue_item)
    int32_t slot;                  // bits 0-7: statistics slot of this part; bits 8-15: first slot to
                                   // blank (kStatParts: none) -- the CTA holding the row's first unit
                                   // blanks the slots no part will write
};

// Item t restricted to units [lo, hi) of the pass; q = units per CTA.  WITH_C: also the
// sequence's temperature constant (a global load the copy warp does not wait for).
template <bool WITH_C>
__device__ __forceinline__ StatsItem describe_item(const BatchView& in, const StatsUnits& g, int64_t t,
                                                   int64_t lo, int64_t hi, int64_t q) {
    const int32_t b = seq_of_target_row(g.off, g.B, t);
    const int64_t d0 = g.off[b];
    const int64_t pos = t - (d0 + b);
    const bool draft_pos = pos < (int64_t)g.off[b + 1] - d0;
    const int64_t n_units = draft_pos ? g.nck : g.h;
    const int64_t S = g.seq_start(b) + (int64_t)g.nck * pos;      // first unit of the item
    const int64_t u0 = lo > S ? lo - S : 0, u1 = hi - S < n_units ? hi - S : n_units;
    StatsItem d;
    d.trow = t;
    d.drow = draft_pos ? d0 + pos : -1;
    // tree-structured verification: the draft row of a context without children is never read
    // (its units then hold one chunk of the target row each)
    const bool childless = draft_pos && in.ctx_has_children && !in.ctx_has_children[d.drow];
    if (childless) d.drow = -1;
    if (d.drow >= 0) { d.ci0 = (int32_t)(2 * u0); d.ci1 = (int32_t)(2 * u1); }
    else if (childless) { d.ci0 = (int32_t)u0; d.ci1 = (int32_t)u1; }
    else { d.ci0 = (int32_t)(2 * u0); d.ci1 = (int32_t)(2 * u1 < g.nck ? 2 * u1 : g.nck); }
    d.c = WITH_C ? (float)(kLog2e / (double)in.temperature[in.per_row_temperature ? b : 0]) : 0.f;
    const int64_t first_cta = div_nn(S, q), last_cta = div_nn(S + n_units - 1, q);
    const int32_t slot = (int32_t)(div_nn(lo, q) - first_cta);
    d.slot = slot | ((slot == 0 ? (int32_t)(last_cta - first_cta + 1) : kStatParts) << 8);
    return d;
}

// Units per CTA: an equal share, but never so small that a row would have more than kStatParts parts.
__device__ __forceinline__ int64_t stats_units_per_cta(int64_t total, int64_t n_ctas, int64_t nck) {
    int64_t q = div_nn(total + n_ctas - 1, n_ctas);
    const int64_t q_min = (nck + kStatParts - 2) / (kStatParts - 1);
    if (q < q_min) q = q_min;
    return q > 0 ? q : 1;
}

struct RingStatsShared {
    ChunkRing ring;
    StatsItem desc[2][kDescBatch];
    unsigned long long batch_full[2], batch_empty[2];
    unsigned long long item_done[kItemDepth], item_free[kItemDepth];
    float2 wpart[kItemDepth][kCWarps];
    long long warp_tot[32];
    int32_t off[kMaxRingSeqs + 1];
    int err;
};
static_assert(sizeof(RingStatsShared) <= 227 * 1024, "RingStatsShared exceeds the shared memory of one CTA");

// prologue_too: no prologue kernel runs for this batch; CTA 0 does its per-sequence work (argument
// checks, tickets and error word zeroed) and the resolve kernel writes the -1 padding.
template <int DT>
__global__ void __launch_bounds__(kRingStatsThreads, 1)
specv_ring_stats(BatchView in, RingScratch ws, int prologue_too) {
    using E = Elt<DT>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RingStatsShared& sh = *reinterpret_cast<RingStatsShared*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row_bytes = in.V * E::kBytes;
    const int nck = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);

    // barriers: one thread each (the scan of the lookahead lengths below holds the CTA barrier that follows)
    ring_init(sh.ring, tid, kStatsWarpsPerChunk);
    if (tid >= 32 && tid < 34) {
        mbar_init(smem_u32(&sh.batch_full[tid - 32]), 1);
        mbar_init(smem_u32(&sh.batch_empty[tid - 32]), kCWarps + 1);   // statistics warps, merge warp
    } else if (tid >= 64 && tid < 64 + kItemDepth) {
        mbar_init(smem_u32(&sh.item_done[tid - 64]), kCWarps);
        mbar_init(smem_u32(&sh.item_free[tid - 64]), 1);
    } else if (tid == 96) {
        sh.err = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_launch_dependents();       // the next kernel may move in as SMs free up
    // Nothing a prologue kernel writes is needed here: every CTA scans the lookahead lengths
    // itself.  Only a tree batch has to wait -- the flags of contexts with children come from the
    // kernel before this one.
    if (in.ctx_has_children) pdl_wait_for_predecessor();
    if (prologue_too && blockIdx.x == 0 && tid == 0) ws.ctrl[0] = ws.ctrl[1] = 0;   // a wait can only expire a second from now
    block_offsets(in, sh.off, sh.warp_tot, tid, kRingStatsThreads, prologue_too && blockIdx.x == 0, ws.seq_status,
                  ws.done);

    StatsUnits g;
    g.off = sh.off; g.B = in.B; g.nck = nck; g.h = (nck + 1) / 2;
    const int64_t total = g.total();
    const int64_t q = stats_units_per_cta(total, gridDim.x, nck);
    const int64_t lo = (int64_t)blockIdx.x * q, hi = lo + q < total ? lo + q : total;
    int64_t t_first = 0;
    int32_t J = 0;                 // items (target rows) this CTA has a share of
    if (lo < total) {
        t_first = g.row_of_unit(lo);
        J = (int32_t)(g.row_of_unit(hi - 1) - t_first + 1);
    }
    volatile int* err = &sh.err;
    auto batch_of = [](int32_t j) { return (j / kDescBatch) & 1; };
    auto batch_parity = [](int32_t j) { return (uint32_t)((j / (2 * kDescBatch)) & 1); };
    auto batch_ends_at = [&](int32_t j) { return j % kDescBatch == kDescBatch - 1 || j == J - 1; };

    if (warp == kStatsCopyWarp) {
        // the copy warp works out its rows and chunks itself, 32 items at a time (one per lane), so
        // the first copy leaves as soon as the offsets are known; what the other warps need besides
        // (the temperature) arrives through the descriptor warp while the data is in flight
        uint32_t g0 = 0;
        StatsItem mine;
        mine.trow = 0; mine.drow = -1; mine.ci0 = mine.ci1 = 0;
        for (int32_t j = 0; j < J; ++j) {
            if (j % 32 == 0) {
                if (j + lane < J) mine = describe_item<false>(in, g, t_first + j + lane, lo, hi, q);
                __syncwarp();
            }
            const int src = j % 32;
            const int64_t trow = __shfl_sync(0xffffffffu, mine.trow, src);
            const int64_t drow = __shfl_sync(0xffffffffu, mine.drow, src);
            const int ci0 = __shfl_sync(0xffffffffu, mine.ci0, src), ci1 = __shfl_sync(0xffffffffu, mine.ci1, src);
            const char* src_p = in.target + trow * in.pitch_t;
            const char* src_q = drow >= 0 ? in.draft + drow * in.pitch_d : nullptr;
            if (!ring_issue_item(sh.ring, src_p, src_q, ci0, ci1, row_bytes, g0, lane, err, 2)) break;
            g0 += (uint32_t)(ci1 - ci0);
        }
        if (*err) ring_drain(sh.ring, lane);
    } else if (warp == kStatsDescWarp) {
        // descriptor warp: which rows and chunks make up each item, 32 items at a time
        for (int32_t jb = 0; jb < J; jb += kDescBatch) {
            const int bb = batch_of(jb);
            mbar_wait(smem_u32(&sh.batch_empty[bb]), batch_parity(jb) ^ 1, err, 3);
            const int32_t j = jb + lane;
            if (j < J) sh.desc[bb][lane] = describe_item<true>(in, g, t_first + j, lo, hi, q);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.batch_full[bb]));
        }
    } else if (warp < kCWarps) {
        uint32_t g0 = 0;
        RingRun run;
        for (int32_t j = 0; j < J; ++j) {
            const int bb = batch_of(j);
            if (j % kDescBatch == 0) mbar_wait(smem_u32(&sh.batch_full[bb]), batch_parity(j), err, 4);
            const StatsItem& dref = sh.desc[bb][j % kDescBatch];
            const bool pair = dref.drow >= 0;
            const float c = dref.c;
            const int ci0 = dref.ci0, ci1 = dref.ci1;
            __syncwarp();
            if (lane == 0 && batch_ends_at(j)) mbar_arrive(smem_u32(&sh.batch_empty[bb]));
            const float2 part = consume_stats_unit<DT>(sh.ring, run, g0, pair, ci0, ci1, row_bytes, c, warp, lane, err, 5);
            // hand the partial to the merge warp (slot reuse waits until it has read the old one)
            const int is = j % kItemDepth;
            if (lane == 0) {
                mbar_wait(smem_u32(&sh.item_free[is]), ((j / kItemDepth) & 1) ^ 1, err, 6);
                sh.wpart[is][warp] = part;
                mbar_arrive(smem_u32(&sh.item_done[is]));
            }
            g0 += (uint32_t)(ci1 - ci0);
        }
    } else if (warp == kMergeWarp) {
        // merge warp: sixteen partials -> (ref, sum) of this CTA's part of the item's one or two rows
        for (int32_t j = 0; j < J; ++j) {
            const int bb = batch_of(j);
            if (j % kDescBatch == 0) mbar_wait(smem_u32(&sh.batch_full[bb]), batch_parity(j), err, 7);
            const StatsItem& d = sh.desc[bb][j % kDescBatch];
            const int64_t trow = d.trow, drow = d.drow;
            const int slot = d.slot & 0xff, blank_from = (d.slot >> 8) & 0xff;
            const int is = j % kItemDepth;
            mbar_wait(smem_u32(&sh.item_done[is]), (j / kItemDepth) & 1, err, 8);
            const float4 st = merge_warp_partials(sh.wpart[is], drow >= 0, lane);
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.item_free[is]));   // partials are in registers (this warp is the only waiter)
                if (!*err) {
                    ws.stat_p[trow * kStatParts + slot] = make_float2(st.x, st.y);
                    if (drow >= 0) ws.stat_q[drow * kStatParts + slot] = make_float2(st.z, st.w);
                    for (int e = blank_from; e < kStatParts; ++e) {
                        ws.stat_p[trow * kStatParts + e] = make_float2(kNoMax, 0.f);
                        if (drow >= 0) ws.stat_q[drow * kStatParts + e] = make_float2(kNoMax, 0.f);
                    }
                }
                if (batch_ends_at(j)) mbar_arrive(smem_u32(&sh.batch_empty[bb]));
            }
            __syncwarp();
        }
    }
    __syncthreads();
    // when a prologue kernel zeroes the error word, report only once it has finished (this also
    // orders it before whatever waits for this grid)
    if (!prologue_too) pdl_wait_for_predecessor();
    if (tid == 0 && sh.err) atomicExch(&ws.ctrl[0], sh.err);
}

// ---------------------------------------------------------------------------------
// resolve building blocks
// ---------------------------------------------------------------------------------
struct SeqRecord {
    int32_t b, K, n, status;       // sequence (-1: no more work), lookahead, first rejection, status bits so far
    int32_t stream;                // 1: rows are streamed and a token is drawn; 0: nothing to draw
    int64_t t0, d0;
    SampleRows rows;               // the row (pair) the token is drawn from, with its constants
    float u2;
};

// Statistics of a whole row from its kStatParts slots: the largest reference and the sum on it, in
// double, slots in index order.  sum < 0 marks a row the early-exit form never evaluated.
struct RowStat {
    float ref;
    double sum;
};
__device__ __forceinline__ RowStat load_row_stat(const float2* stat, int64_t row) {
    static_assert(kStatParts == 4, "two 16-byte loads per row");
    const float4* p = reinterpret_cast<const float4*>(stat + row * kStatParts);
    const float4 a = p[0], b = p[1];
    RowStat r;
    if (a.y < 0.f) { r.ref = 0.f; r.sum = -1.0; return r; }
    r.ref = fmaxf(fmaxf(a.x, a.z), fmaxf(b.x, b.z));
    // a row that was not shared has one slot in use: no exponential at all then
    auto term = [&](float ref, float sum) -> double {
        if (sum == 0.f) return 0.0;
        return ref == r.ref ? (double)sum : (double)sum * exp2((double)ref - (double)r.ref);
    };
    r.sum = ((term(a.x, a.y) + term(a.z, a.w)) + term(b.x, b.y)) + term(b.z, b.w);
    return r;
}

// What a decision needs from the caller's buffers, loaded before the row statistics exist: per
// lane the drafted token of position `lane`, its accept uniform and its two logits.
struct SeqInputs {
    int64_t d0;
    int32_t K;          // lookahead as the clamped offsets give it (equals K_b for every valid sequence)
    float T, u2;
    int32_t x;
    float u, lp, lq;
};

template <int DT>
__device__ __forceinline__ void load_position(const BatchView& in, int64_t d0, int64_t t0, int32_t i, int32_t& x,
                                              float& u, float& lp, float& lq) {
    using E = Elt<DT>;
    x = in.tokens[d0 + i];
    u = in.uniforms[t0 + i];
    lp = lq = 0.f;
    if (x >= 0 && (int64_t)x < in.V) {
        lp = E::load1(in.target + (t0 + i) * in.pitch_t, x);
        lq = E::load1(in.draft + (d0 + i) * in.pitch_d, x);
    }
}

// `off` are the clamped offsets (any copy of them: shared or global), so every index formed here
// stays inside the buffers even for a sequence whose lookahead is nonsense.
template <int DT>
__device__ __forceinline__ SeqInputs prefetch_sequence(const BatchView& in, const int32_t* off, int32_t b, int lane) {
    SeqInputs s;
    s.d0 = off[b];
    s.K = off[b + 1] - off[b];
    const int64_t t0 = s.d0 + b;
    s.T = in.temperature[in.per_row_temperature ? b : 0];
    s.u2 = in.uniforms[t0 + s.K];
    s.x = 0; s.u = 0.f; s.lp = 0.f; s.lq = 0.f;
    if (lane < s.K) load_position<DT>(in, s.d0, t0, lane, s.x, s.u, s.lp, s.lq);
    return s;
}

// One warp: acceptance test of every draft position of sequence b in double (lanes =
// positions), first rejection, and the constants of the row (pair) the token is drawn from.
// `pre` holds what could be loaded before the statistics were complete; what remains is one
// round of loads (row statistics, the prologue's verdict on the sequence) and the arithmetic.
// The record is complete in lane 0.
template <int DT>
__device__ __forceinline__ SeqRecord decide_sequence(const BatchView& in, const RingScratch& ws, int32_t b,
                                                     const SeqInputs& pre, int lane, float* diag_p, float* diag_q) {
    const int32_t K = pre.K;
    const int64_t d0 = pre.d0, t0 = d0 + b;
    // one round of loads: the statistics of the first 32 positions are requested before the
    // prologue's verdict on the sequence is looked at (the clamped offsets keep every row index
    // inside the buffers whatever that verdict is)
    RowStat sp0{0.f, 1.0}, sq0{0.f, 1.0};
    if (lane < K) sq0 = load_row_stat(ws.stat_q, d0 + lane);
    if (lane <= K) sp0 = load_row_stat(ws.stat_p, t0 + lane);
    const int error_word = ws.ctrl[0];    // non-zero: the statistics kernel gave up -- report it, draw nothing
    int status = ws.seq_status[b] | (error_word ? (16 | (error_word << 8)) : 0);
    const float cf = (float)(kLog2e / (double)pre.T);
    const double c = (double)cf;

    SeqRecord r;
    r.b = b; r.K = K; r.n = K;
    r.t0 = t0; r.d0 = d0;
    r.u2 = 0.f;
    r.rows.p = nullptr; r.rows.q = nullptr;
    r.rows.p_aligned = r.rows.q_aligned = true;
    r.rows.c = cf; r.rows.p_ref = 0.f; r.rows.q_ref = 0.f; r.rows.kappa = 0.f;

    int32_t n = K;
    RowStat n_p{0.f, 1.0}, n_q{0.f, 1.0};    // statistics of the rows at the first rejection
    if (!(status & 1)) {                     // else the lookahead is nonsense: nothing of the sequence is judged
        for (int32_t base = 0; base <= K; base += 32) {
            const int32_t i = base + lane;
            const bool has_t = i <= K, has_d = i < K;
            int32_t x = pre.x;
            float u = pre.u, lp = pre.lp, lq = pre.lq;
            RowStat sp = sp0, sq = sq0;
            if (base > 0) {
                if (has_d) { load_position<DT>(in, d0, t0, i, x, u, lp, lq); sq = load_row_stat(ws.stat_q, d0 + i); }
                if (has_t) sp = load_row_stat(ws.stat_p, t0 + i);
            }
            const bool bad = has_d && (x < 0 || (int64_t)x >= in.V);
            if (__any_sync(0xffffffffu, bad)) status |= 4;   // SPECV_ROW_BAD_TOKEN
            bool rej = false;
            if (has_d && !bad && !(status & ~4)) {
                if (sp.sum < 0.0 || sq.sum < 0.0) {
                    // early-exit form: the position was skipped because an earlier one is rejected
                    // for certain; it cannot be the first rejection and has no probabilities
                    if (diag_p) diag_p[d0 + i] = __int_as_float(0x7fc00000);
                    if (diag_q) diag_q[d0 + i] = __int_as_float(0x7fc00000);
                } else {
                    const double p = exp2((double)lp * c - (double)sp.ref) / sp.sum;
                    const double q = exp2((double)lq * c - (double)sq.ref) / sq.sum;
                    if (diag_p) diag_p[d0 + i] = (float)p;
                    if (diag_q) diag_q[d0 + i] = (float)q;
                    rej = !((double)u * q < p);
                }
            }
            const unsigned mask = __ballot_sync(0xffffffffu, rej);
            const int32_t first = (mask && n == K) ? base + __ffs(mask) - 1 : n;
            // statistics of the deciding row (pair): the first rejection, or row K when this block holds it
            if (first != n || (n == K && K >= base && K - base < 32)) {
                const int src = (first != n ? first : K) - base;
                n_p.ref = __shfl_sync(0xffffffffu, sp.ref, src);
                n_p.sum = shfl_double(sp.sum, src);
                n_q.ref = __shfl_sync(0xffffffffu, sq.ref, src);
                n_q.sum = shfl_double(sq.sum, src);
            }
            n = first;
        }
        if (status == 0) {
            r.n = n;
            r.u2 = pre.u2;
            r.rows.p = in.target + (t0 + n) * in.pitch_t;
            r.rows.p_ref = n_p.ref;
            if (n < K) {
                r.rows.q = in.draft + (d0 + n) * in.pitch_d;
                r.rows.q_ref = n_q.ref;
                r.rows.kappa = (float)(n_p.sum / n_q.sum);
            }
        }
    }
    r.status = status;
    r.stream = status == 0;
    return r;
}

// Consumer warp: this warp's share of chunk columns [k0, k1) of the rows a token is drawn from
// (ring positions g0 ..).  A group of four warps takes one column at a time (the same vocabulary
// range of the target and the draft row; the target row's chunk alone when the token comes from
// it alone), a quarter each, and writes the masses of its 512-byte segments to seg[] (global).
template <int DT>
__device__ __forceinline__ void consume_resolve_unit(ChunkRing& ring, RingRun& run, uint32_t g0, const SampleRows& sr, int k0,
                                                     int k1, int32_t nvec_row, int32_t nseg, float* seg, int warp,
                                                     int lane, volatile int* err, int site) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    constexpr int kSegsPerChunk = kChunkBytes / 512;
    constexpr int kQuarterBytes = kChunkBytes / kWarpsPerChunk;
    const int group = warp / kWarpsPerChunk, sub = warp % kWarpsPerChunk;
    const bool pair = sr.q != nullptr;
    const unsigned long long cc = pack_f32x2(sr.c, sr.c), np_ref = pack_f32x2(-sr.p_ref, -sr.p_ref),
                             nq_ref = pack_f32x2(-sr.q_ref, -sr.q_ref), nkappa = pack_f32x2(-sr.kappa, -sr.kappa);
    // column u of a part goes to warp group (u - k0) % 4: two ring positions per column for a row pair
    run.begin_item(g0, pair ? (g0 % (2 * kChunkGroups)) : 16 + g0 % kChunkGroups);
    for (int u = k0 + group; u < k1; u += kChunkGroups) {
        const uint32_t gp = g0 + (uint32_t)(pair ? 2 * (u - k0) : (u - k0));
        const uint32_t slot_p = gp % kRingSlots, slot_q = (gp + 1) % kRingSlots;
        ring_wait_chunk(ring, gp, run.guard_until, err, site);
        if (pair) ring_wait_chunk(ring, gp + 1, run.guard_until, err, site);
        const unsigned char* pq = ring.slot[slot_p] + sub * kQuarterBytes;
        const unsigned char* qq = ring.slot[slot_q] + sub * kQuarterBytes;
        // four 512-byte segments per quarter: all loads first (the slots are released as soon as the
        // data is in registers), then the masses, then the four warp sums folded into one another
        // (six shuffles: after two exchange steps each lane carries one segment's partial sum)
        constexpr int kSegsPerQuarter = kQuarterBytes / 512;
        static_assert(kSegsPerQuarter == 4, "the folded warp sum below is written for four segments");
        const int32_t seg0 = u * kSegsPerChunk + sub * kSegsPerQuarter;
        uint4 rawp[kSegsPerQuarter], rawq[kSegsPerQuarter];
#pragma unroll
        for (int i = 0; i < kSegsPerQuarter; ++i) {
            rawp[i] = *reinterpret_cast<const uint4*>(pq + (i * 32 + lane) * 16);
            rawq[i] = pair ? *reinterpret_cast<const uint4*>(qq + (i * 32 + lane) * 16) : make_uint4(0u, 0u, 0u, 0u);
        }
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(smem_u32(&ring.empty_bar[slot_p]));
            if (pair) mbar_arrive(smem_u32(&ring.empty_bar[slot_q]));
        }
        float a[kSegsPerQuarter];
#pragma unroll
        for (int i = 0; i < kSegsPerQuarter; ++i) {
            a[i] = 0.f;
            if ((seg0 + i) * 32 + lane < nvec_row) {      // vector index within the row
                // the masses of mass_of_raw, two elements per instruction (even elements in the
                // low half, odd ones in the high half), summed per half and then together
                float xp[N], xq[N];
                E::unpack(rawp[i], xp);
                unsigned long long acc = pack_f32x2(0.f, 0.f);
                if (pair) {
                    E::unpack(rawq[i], xq);
#pragma unroll
                    for (int k = 0; k < N; k += 2) {
                        float tp0, tp1, tq0, tq1, d0, d1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(xp[k], xp[k + 1]), cc, np_ref), tp0, tp1);
                        unpack_f32x2(fma_f32x2(pack_f32x2(xq[k], xq[k + 1]), cc, nq_ref), tq0, tq1);
                        unpack_f32x2(fma_f32x2(nkappa, pack_f32x2(ex2_approx(tq0), ex2_approx(tq1)),
                                               pack_f32x2(ex2_approx(tp0), ex2_approx(tp1))), d0, d1);
                        acc = add_f32x2(acc, pack_f32x2(fmaxf(d0, 0.f), fmaxf(d1, 0.f)));
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < N; k += 2) {
                        float tp0, tp1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(xp[k], xp[k + 1]), cc, np_ref), tp0, tp1);
                        acc = add_f32x2(acc, pack_f32x2(ex2_approx(tp0), ex2_approx(tp1)));
                    }
                }
                float lo, hi;
                unpack_f32x2(acc, lo, hi);
                a[i] = lo + hi;
            }
        }
        const bool up16 = lane & 16, up8 = lane & 8;
        const float b0 = (up16 ? a[2] : a[0]) + __shfl_xor_sync(0xffffffffu, up16 ? a[0] : a[2], 16);
        const float b1 = (up16 ? a[3] : a[1]) + __shfl_xor_sync(0xffffffffu, up16 ? a[1] : a[3], 16);
        float v = (up8 ? b1 : b0) + __shfl_xor_sync(0xffffffffu, up8 ? b0 : b1, 8);
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        // lanes 8 s .. 8 s + 7 now hold the sum of segment s of the quarter
        if ((lane & 7) == 0 && seg0 + (lane >> 3) < nseg) seg[seg0 + (lane >> 3)] = v;
    }
}

// Locator warp: token from the finished segment table and the sequence's outputs.
template <int DT>
__device__ __forceinline__ void locate_and_emit(const BatchView& in, const SeqRecord& r, float* seg, int32_t nseg,
                                                int32_t* result_slot, int lane, int32_t* accepted_len,
                                                int32_t* emitted, int32_t* row_status, const NextLookahead& next) {
    auto wsync = [] { __syncwarp(); };
    int status = r.status;
    SampleRows sr = r.rows;
    int32_t token = locate_in_segments<DT, true>(sr, in.V, (double)r.u2, seg, nseg, lane);
    if (token < 0 && sr.q) {
        // the residual rounded to nothing: sample from the target row itself (rare; this
        // warp alone re-reads the row with plain loads)
        status |= 8;   // SPECV_ROW_ZERO_RESIDUAL
        sr.q = nullptr;
        token = block_inverse_cdf<DT, 1, true>(sr, in.V, (double)r.u2, seg, result_slot, 0, wsync);
    }
    if (token < 0) token = (int32_t)(in.V - 1);   // a row without any mass (all logits -inf)
    for (int32_t i = lane; i <= r.K; i += 32)
        emitted[r.t0 + i] = (i < r.n) ? in.tokens[r.d0 + i] : (i == r.n ? token : -1);
    if (lane == 0) {
        accepted_len[r.b] = r.n;
        if (row_status) row_status[r.b] = status;
        // a sequence that draws a token is valid, so r.K is its lookahead as the caller gave it
        if (next.out) next.out[r.b] = next_lookahead_of(r.K, r.n, next.k_min, next.k_max);
    }
}

// ---------------------------------------------------------------------------------
// specv_ring_resolve
// ---------------------------------------------------------------------------------
// A CTA's share of one sequence's rows: chunk columns [k0, k1), `units` 16 KB units.
struct PartRecord {
    SeqRecord r;                   // r.b < 0: no more work
    int32_t k0, k1, units, pad;
};

struct RingResolveShared {
    ChunkRing ring;
    PartRecord rec[kPartDepth];
    unsigned long long rec_full[kPartDepth], rec_empty[kPartDepth];
    unsigned long long seg_done[2], seg_free[2];
    float seg[kMaxSegs];           // locator: the finished sequence's segment sums
    long long warp_tot[32];
    int32_t off[kMaxRingSeqs + 1];
    int32_t result_slot;
    int err;
};
static_assert(sizeof(RingResolveShared) <= 227 * 1024, "RingResolveShared exceeds the shared memory of one CTA");
static_assert(kPartDepth == kCWarps, "the first kPartDepth records are produced by one consumer warp each");

// The rows a token is drawn from, as one sequence of chunk columns: sequence b owns columns
// [b nck, (b+1) nck) whether it draws from a row pair (16 KB per column), from its last target row
// alone (8 KB) or from nothing (a data error) -- the cut needs no decision to be known.  CTA c takes
// columns [c q, (c+1) q); part m of a CTA is its share of sequence b_first + m.  The CTA decides the
// sequences it touches itself, the first sixteen at once (one warp each, before those warps turn
// to the data), later ones in the fetch warp; a sequence shared by several CTAs is decided by each
// of them (same inputs, same code, same answer).  Everything a decision needs from the caller's
// buffers is loaded while the statistics kernel is still finishing.
template <int DT>
__global__ void __launch_bounds__(kRingResolveThreads, 1)
specv_ring_resolve(BatchView in, RingScratch ws, int32_t* __restrict__ accepted_len, int32_t* __restrict__ emitted,
                   int32_t* __restrict__ row_status, float* __restrict__ diag_p, float* __restrict__ diag_q,
                   NextLookahead next) {
    using E = Elt<DT>;
    constexpr int SEG = 32 * E::kPerVec;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RingResolveShared& sh = *reinterpret_cast<RingResolveShared*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row_bytes = in.V * E::kBytes;
    const int nck = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);
    const int32_t nvec_row = (int32_t)(row_bytes / 16);
    const int32_t nseg = (int32_t)((in.V + SEG - 1) / SEG);

    ring_init(sh.ring, tid);
    if (tid >= 32 && tid < 32 + kPartDepth) {
        mbar_init(smem_u32(&sh.rec_full[tid - 32]), 1);
        mbar_init(smem_u32(&sh.rec_empty[tid - 32]), kCWarps + 2);   // consumers, copy warp, locator
    } else if (tid >= 64 && tid < 66) {
        mbar_init(smem_u32(&sh.seg_done[tid - 64]), kCWarps);
        mbar_init(smem_u32(&sh.seg_free[tid - 64]), 1);
    } else if (tid == 96) {
        sh.err = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    block_offsets(in, sh.off, sh.warp_tot, tid, kRingResolveThreads, false, nullptr, nullptr);

    const int64_t total = (int64_t)in.B * nck;
    const int64_t q = div_nn(total + gridDim.x - 1, gridDim.x);
    const int64_t lo = (int64_t)blockIdx.x * q < total ? (int64_t)blockIdx.x * q : total;
    const int64_t hi = lo + q < total ? lo + q : total;
    const int32_t b_first = (int32_t)div_nn(lo, nck);
    const int32_t n_parts = hi > lo ? (int32_t)div_nn(hi - 1, nck) - b_first + 1 : 0;
    volatile int* err = &sh.err;
    auto rec_slot = [](int32_t m) { return m % kPartDepth; };
    auto rec_parity = [](int32_t m) { return (uint32_t)((m / kPartDepth) & 1); };

    // Record of part m (m == n_parts: the end marker), written by the calling warp.  With
    // after_wait == false the statistics kernel may still be running: only the caller's buffers are
    // read before the wait.
    auto produce = [&](int32_t m, bool wait_inside) {
        const int rs = rec_slot(m);
        const int32_t b = b_first + m;
        if (m >= n_parts) {
            if (wait_inside) pdl_wait_for_predecessor();
            if (lane == 0) sh.rec[rs].r.b = -1;
        } else {
            const int64_t c0 = (int64_t)b * nck;
            const int32_t u0 = (int32_t)(lo > c0 ? lo - c0 : 0), u1 = (int32_t)(hi - c0 < nck ? hi - c0 : nck);
            const SeqInputs pre = prefetch_sequence<DT>(in, sh.off, b, lane);
            if (wait_inside) pdl_wait_for_predecessor();    // every row statistic must be in memory
            const bool first_part = u0 == 0;                 // this CTA reports what only one CTA may report
            const SeqRecord r = decide_sequence<DT>(in, ws, b, pre, lane, first_part ? diag_p : nullptr,
                                                    first_part ? diag_q : nullptr);
            if (first_part) {
                // a sequence that draws a token reads as failed until its token is emitted; one
                // with a data error is final here: no accepted tokens, -1 in all its slots
                for (int32_t i = lane; i <= r.K; i += 32) emitted[r.t0 + i] = -1;
                if (lane == 0) {
                    accepted_len[b] = 0;
                    if (row_status) row_status[b] = r.stream ? 16 : r.status;   // 16: SPECV_ROW_INTERNAL
                    if (next.out)
                        next.out[b] = next_lookahead_of(in.k_per_row ? in.k_per_row[b] : in.k_uniform, 0, next.k_min,
                                                        next.k_max);
                }
            }
            if (lane == 0) {
                sh.rec[rs].r = r;
                sh.rec[rs].k0 = u0;
                sh.rec[rs].k1 = u1;
                sh.rec[rs].units = u1 - u0;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.rec_full[rs]));
    };

    if (warp < kCWarps && warp <= n_parts) produce(warp, true);
    else pdl_wait_for_predecessor();

    if (warp == kFetchWarp) {
        // token slots that belong to no sequence (the lookahead lengths add up to less than n_draft_total)
        if (blockIdx.x == 0)
            for (int64_t i = (int64_t)sh.off[in.B] + in.B + lane; i < in.n_draft_total + in.B; i += 32) emitted[i] = -1;
        // parts beyond the first kPartDepth, in order, as record slots come free
        for (int32_t m = kPartDepth; m <= n_parts; ++m) {
            mbar_wait(smem_u32(&sh.rec_empty[rec_slot(m)]), rec_parity(m) ^ 1, err, 21);
            if (__shfl_sync(0xffffffffu, (int)(*err != 0), 0)) break;
            produce(m, false);
        }
    } else if (warp == kResolveCopyWarp) {
        uint32_t g0 = 0;
        for (int32_t m = 0;; ++m) {
            const int rs = rec_slot(m);
            mbar_wait(smem_u32(&sh.rec_full[rs]), rec_parity(m), err, 22);
            if (*err) break;
            const PartRecord& pr = sh.rec[rs];
            const bool last = pr.r.b < 0;
            const char* src_p = pr.r.rows.p;
            const char* src_q = pr.r.rows.q;
            const int k0 = pr.k0, k1 = pr.k1;
            const bool stream = !last && pr.r.stream != 0;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.rec_empty[rs]));
            if (last) break;
            if (!stream) continue;     // a data error: nothing is drawn
            const int ci0 = src_q ? 2 * k0 : k0, ci1 = src_q ? 2 * k1 : k1;
            if (!ring_issue_item(sh.ring, src_p, src_q, ci0, ci1, row_bytes, g0, lane, err, 23)) break;
            g0 += (uint32_t)(ci1 - ci0);
        }
        if (*err) ring_drain(sh.ring, lane);
    } else if (warp < kCWarps) {
        uint32_t g0 = 0;
        RingRun run;
        int32_t drawn = 0;      // parts streamed so far
        for (int32_t m = 0;; ++m) {
            const int rs = rec_slot(m);
            mbar_wait(smem_u32(&sh.rec_full[rs]), rec_parity(m), err, 24);
            if (*err) break;
            const bool last = sh.rec[rs].r.b < 0;
            const bool stream = !last && sh.rec[rs].r.stream != 0;
            const SampleRows sr = sh.rec[rs].r.rows;
            const int32_t b = sh.rec[rs].r.b;
            const int k0 = sh.rec[rs].k0, k1 = sh.rec[rs].k1;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.rec_empty[rs]));
            if (last) break;
            if (!stream) continue;
            // the locator must have seen the completion of the part before the previous one before
            // this barrier moves on
            mbar_wait(smem_u32(&sh.seg_free[drawn & 1]), ((drawn >> 1) & 1) ^ 1, err, 25);
            consume_resolve_unit<DT>(sh.ring, run, g0, sr, k0, k1, nvec_row, nseg, ws.gseg + (int64_t)b * nseg, warp, lane,
                                     err, 26);
            // the segment sums are read by whichever CTA finishes the sequence: the arrival orders
            // them before the locator's wait, and the locator's fence and ticket (cumulative) before
            // that CTA's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.seg_done[drawn & 1]));
            g0 += (uint32_t)(sr.q ? 2 * (k1 - k0) : (k1 - k0));
            ++drawn;
        }
    } else if (warp == kLocatorWarp) {
        int32_t drawn = 0;
        for (int32_t m = 0;; ++m) {
            const int rs = rec_slot(m);
            mbar_wait(smem_u32(&sh.rec_full[rs]), rec_parity(m), err, 28);
            if (*err) break;
            const SeqRecord r = sh.rec[rs].r;
            const int32_t units = sh.rec[rs].units;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.rec_empty[rs]));
            if (r.b < 0) break;
            if (!r.stream) continue;
            mbar_wait(smem_u32(&sh.seg_done[drawn & 1]), (drawn >> 1) & 1, err, 29);
            if (*err) break;
            const int sd = drawn & 1;
            ++drawn;
            int32_t complete = 0;
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.seg_free[sd]));
                __threadfence();
                complete = atomicAdd(&ws.done[r.b], units) + units == nck;
                __threadfence();
            }
            complete = __shfl_sync(0xffffffffu, complete, 0);
            if (complete) {
                // every part of the sequence is in: this CTA draws the token
                const float* gs = ws.gseg + (int64_t)r.b * nseg;
                for (int32_t i = lane; i < nseg; i += 32) sh.seg[i] = __ldcg(gs + i);
                __syncwarp();
                locate_and_emit<DT>(in, r, sh.seg, nseg, &sh.result_slot, lane, accepted_len, emitted, row_status, next);
                __syncwarp();
            }
        }
    }
    __syncthreads();
    if (tid == 0 && sh.err) atomicExch(&ws.ctrl[0], sh.err);
}

// ---------------------------------------------------------------------------------
// Early-exit form of the statistics pass (optional; spec_verify_set_early_exit).
//
// The paper's theme is to skip work that the input makes unnecessary.  Here: once a draft
// position of a sequence is rejected for certain, nothing after it can be emitted, so the rows
// of its later positions need not be read at all.  Work items are ordered by position first
// (all sequences' position 0, then all position 1, ...), so that by the time position i+1 of a
// sequence comes up the verdict on its position i is in; the merge warp takes that verdict in
// fp32 as soon as an item's statistics exist and publishes clear rejections; the copy warp looks
// the sequence up right before it would stream an item and skips it if an earlier position is
// already rejected.  Verdicts closer than 1e-3 relative are not published (the resolve kernel
// settles every verdict in double anyway), so a skipped row can never be one the result needs.
// ---------------------------------------------------------------------------------
constexpr int kNoReject = 0x7fffffff;

constexpr int kPlanThreads = 1024;              // 32 warps: one level per warp and round

// Work list ordered by position: level i holds every valid sequence with K_b >= i.  One block.
__global__ void __launch_bounds__(kPlanThreads)
specv_plan_levels(BatchView in, RingScratch ws) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    asm volatile("griddepcontrol.wait;" ::: "memory");             // offsets and status from the prologue
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ int32_t kmax_s;
    if (tid == 0) kmax_s = -1;
    __syncthreads();
    auto k_of = [&](int32_t b) { return in.k_per_row ? in.k_per_row[b] : in.k_uniform; };
    for (int32_t b = tid; b < in.B; b += kPlanThreads) {
        ws.first_rej[b] = kNoReject;
        if (ws.seq_status[b] == 0) atomicMax(&kmax_s, k_of(b));
    }
    __syncthreads();
    const int32_t kmax = kmax_s;   // -1: no valid sequence
    auto in_level = [&](int32_t b, int32_t level) -> bool {
        return b < in.B && ws.seq_status[b] == 0 && k_of(b) >= level;
    };
    for (int32_t level = warp; level <= kmax; level += 32) {
        int32_t count = 0;
        for (int32_t base = 0; base < in.B; base += 32)
            count += __popc(__ballot_sync(0xffffffffu, in_level(base + lane, level)));
        if (lane == 0) ws.level_start[level] = count;
    }
    __syncthreads();
    if (warp == 0) {   // exclusive prefix over levels
        int32_t carry = 0;
        for (int32_t base = 0; base <= kmax; base += 32) {
            const int32_t level = base + lane;
            const int32_t v = level <= kmax ? ws.level_start[level] : 0;
            int32_t incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            if (level <= kmax) ws.level_start[level] = carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) { ws.ctrl[2] = carry; ws.ctrl[3] = 0; ws.ctrl[4] = 0; }
    }
    __syncthreads();
    for (int32_t level = warp; level <= kmax; level += 32) {
        int32_t next = ws.level_start[level];
        for (int32_t base = 0; base < in.B; base += 32) {
            const bool f = in_level(base + lane, level);
            const unsigned m = __ballot_sync(0xffffffffu, f);
            if (f) {
                const int32_t n = next + __popc(m & ((1u << lane) - 1u));
                ws.item_seq[n] = base + lane;
                ws.item_pos[n] = level;
            }
            next += __popc(m);
        }
    }
    // rows that end up skipped must read as "never evaluated" when the sequence is decided: a
    // negative sum in the first slot (this form writes whole-row statistics there, the other slots
    // stay empty)
    auto never = [](float2* stat, int64_t i) {
        stat[i] = (i % kStatParts) ? make_float2(kNoMax, 0.f) : make_float2(0.f, -1.f);
    };
    for (int64_t i = tid; i < (in.n_draft_total + in.B) * kStatParts; i += kPlanThreads) never(ws.stat_p, i);
    for (int64_t i = tid; i < in.n_draft_total * kStatParts; i += kPlanThreads) never(ws.stat_q, i);
}

struct __align__(16) EarlyItem {   // 48 bytes
    int64_t trow, drow;            // drow < 0: last target row of its sequence
    float c, lp_x, lq_x, u;        // logits of the drafted token in both rows, its accept uniform
    int32_t b, pos;
    int32_t token_ok;              // the drafted token is a valid id (else no verdict is taken here)
    int32_t dropped;               // already known to be skippable when it was described: nobody looks at it
};

constexpr int kEarlyDescDepth = 4;     // work items described ahead, in rounds of kEarlyFetch
constexpr int kEarlyFetch = 2;         // items taken from the global work counter at a time

struct RingEarlyShared {
    ChunkRing ring;
    EarlyItem desc[kEarlyDescDepth];
    unsigned long long desc_full[kEarlyDescDepth], desc_empty[kEarlyDescDepth];
    unsigned long long item_go[kItemDepth], item_done[kItemDepth], item_free[kItemDepth];
    float2 wpart[kItemDepth][kCWarps];
    int32_t skip[kItemDepth];
    int err;
};
static_assert(sizeof(RingEarlyShared) <= 227 * 1024, "RingEarlyShared exceeds the shared memory of one CTA");

// Work items come from a global counter over the position-major list, four at a time, so that
// all CTAs advance through the positions together: a CTA that skips a lot takes more items
// instead of running ahead into positions whose verdicts are not in yet.
template <int DT>
__global__ void __launch_bounds__(kRingStatsThreads, 1)
specv_ring_stats_early(BatchView in, RingScratch ws) {
    using E = Elt<DT>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RingEarlyShared& sh = *reinterpret_cast<RingEarlyShared*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row_bytes = in.V * E::kBytes;
    const int nck = (int)((row_bytes + kChunkBytes - 1) / kChunkBytes);

    ring_init(sh.ring, tid, kStatsWarpsPerChunk);
    if (tid >= 32 && tid < 32 + kEarlyDescDepth) {
        mbar_init(smem_u32(&sh.desc_full[tid - 32]), 1);
        mbar_init(smem_u32(&sh.desc_empty[tid - 32]), 1 + kCWarps + 1);   // copy warp, statistics warps, merge warp
    } else if (tid >= 64 && tid < 64 + kItemDepth) {
        mbar_init(smem_u32(&sh.item_go[tid - 64]), 1);
        mbar_init(smem_u32(&sh.item_done[tid - 64]), kCWarps);
        mbar_init(smem_u32(&sh.item_free[tid - 64]), 1);
    } else if (tid == 96) {
        sh.err = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    pdl_wait_for_predecessor();    // the work list
    pdl_launch_dependents();

    const int32_t n_items = ws.ctrl[2];
    volatile int* err = &sh.err;
    auto desc_slot = [](uint32_t e) { return (int)(e % kEarlyDescDepth); };
    auto desc_parity = [](uint32_t e) { return (uint32_t)((e / kEarlyDescDepth) & 1); };
    auto item_parity = [](uint32_t e) { return (uint32_t)((e / kItemDepth) & 1); };
    // every reader: next descriptor in order; false at the end of the work (or after a failure)
    auto next_item = [&](uint32_t e, EarlyItem& d, int site) -> bool {
        mbar_wait(smem_u32(&sh.desc_full[desc_slot(e)]), desc_parity(e), err, site);
        if (*err) return false;
        d = sh.desc[desc_slot(e)];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh.desc_empty[desc_slot(e)]));
        return d.b >= 0;
    };

    if (warp == kStatsCopyWarp) {
        uint32_t g0 = 0;
        int32_t skipped_rows = 0;
        EarlyItem d;
        uint32_t it = 0;    // items that entered the pipeline
        for (uint32_t e = 0; next_item(e, d, 61); ++e) {
            if (d.dropped) continue;
            // is an earlier position of this sequence already rejected for certain?  (asked again:
            // the verdict may have come in since the item was described)
            const int is = it % kItemDepth;
            const uint32_t ip = item_parity(it);
            ++it;
            int skip = 0;
            if (lane == 0) {
                skip = *reinterpret_cast<volatile int32_t*>(&ws.first_rej[d.b]) < d.pos;
                mbar_wait(smem_u32(&sh.item_free[is]), ip ^ 1, err, 62);   // slot's previous item fully merged
                sh.skip[is] = skip;
                mbar_arrive(smem_u32(&sh.item_go[is]));
            }
            skip = __shfl_sync(0xffffffffu, skip, 0);
            if (skip) { skipped_rows += d.drow >= 0 ? 2 : 1; continue; }
            const char* src_p = in.target + d.trow * in.pitch_t;
            const char* src_q = d.drow >= 0 ? in.draft + d.drow * in.pitch_d : nullptr;
            if (!ring_issue_item(sh.ring, src_p, src_q, 0, src_q ? 2 * nck : nck, row_bytes, g0, lane, err, 63)) break;
            g0 += src_q ? 2 * nck : nck;
        }
        if (lane == 0 && skipped_rows) atomicAdd(&ws.ctrl[3], skipped_rows);
        if (*err) ring_drain(sh.ring, lane);
    } else if (warp == kStatsDescWarp) {
        // descriptor warp: kEarlyFetch items per round from the global counter, one lane each
        for (uint32_t e0 = 0;; e0 += kEarlyFetch) {
            const uint32_t e = e0 + lane;
            if (lane < kEarlyFetch) mbar_wait(smem_u32(&sh.desc_empty[desc_slot(e)]), desc_parity(e) ^ 1, err, 64);
            __syncwarp();
            int32_t base = 0;
            if (lane == 0) base = *err ? n_items : atomicAdd(&ws.ctrl[4], kEarlyFetch);
            base = __shfl_sync(0xffffffffu, base, 0);
            if (lane < kEarlyFetch) {
                const int32_t n = base + lane;
                EarlyItem d;
                d.b = -1; d.pos = 0; d.trow = 0; d.drow = -1; d.c = 0.f;
                d.lp_x = 0.f; d.lq_x = 0.f; d.u = 0.f; d.token_ok = 0; d.dropped = 0;
                if (n < n_items) {
                    d.b = ws.item_seq[n];
                    d.pos = ws.item_pos[n];
                    const int64_t d0 = ws.off_d[d.b];
                    const int32_t K = in.k_per_row ? in.k_per_row[d.b] : in.k_uniform;
                    d.c = (float)(kLog2e / (double)in.temperature[in.per_row_temperature ? d.b : 0]);
                    d.trow = d0 + d.b + d.pos;
                    d.drow = d.pos < K ? d0 + d.pos : -1;
                    d.dropped = *reinterpret_cast<volatile int32_t*>(&ws.first_rej[d.b]) < d.pos;
                    if (d.dropped) {
                        atomicAdd(&ws.ctrl[3], d.drow >= 0 ? 2 : 1);
                    } else if (d.drow >= 0) {
                        const int32_t x = in.tokens[d.drow];
                        d.u = in.uniforms[d.trow];
                        if (x >= 0 && (int64_t)x < in.V) {
                            d.token_ok = 1;
                            d.lp_x = E::load1(in.target + d.trow * in.pitch_t, x);
                            d.lq_x = E::load1(in.draft + d.drow * in.pitch_d, x);
                        }
                    }
                }
                sh.desc[desc_slot(e)] = d;     // b < 0 marks the end of the work
                mbar_arrive(smem_u32(&sh.desc_full[desc_slot(e)]));
            }
            __syncwarp();
            if (base + kEarlyFetch > n_items) break;   // this round held an end marker
        }
    } else if (warp < kCWarps) {
        uint32_t g0 = 0;
        RingRun run;
        EarlyItem d;
        uint32_t it = 0;
        for (uint32_t e = 0; next_item(e, d, 65); ++e) {
            if (d.dropped) continue;
            const bool pair = d.drow >= 0;
            const int is = it % kItemDepth;
            const uint32_t ip = item_parity(it);
            ++it;
            mbar_wait(smem_u32(&sh.item_go[is]), ip, err, 66);
            const bool skip = sh.skip[is] != 0;
            float2 part = make_float2(kNoMax, 0.f);
            if (!skip) {
                part = consume_stats_unit<DT>(sh.ring, run, g0, pair, 0, pair ? 2 * nck : nck, row_bytes, d.c, warp, lane,
                                              err, 67);
                g0 += pair ? 2 * nck : nck;
            }
            __syncwarp();
            if (lane == 0) {
                sh.wpart[is][warp] = part;     // the slot is ours: the copy warp waited for it before item_go
                mbar_arrive(smem_u32(&sh.item_done[is]));
            }
        }
    } else if (warp == kMergeWarp) {
        // merge warp: statistics of the item, and the verdict on its draft token where it is clear
        EarlyItem d;
        uint32_t it = 0;
        for (uint32_t e = 0; next_item(e, d, 68); ++e) {
            if (d.dropped) continue;
            const int is = it % kItemDepth;
            const uint32_t ip = item_parity(it);
            ++it;
            mbar_wait(smem_u32(&sh.item_go[is]), ip, err, 69);
            const bool skip = sh.skip[is] != 0;
            mbar_wait(smem_u32(&sh.item_done[is]), ip, err, 70);
            const float4 st = merge_warp_partials(sh.wpart[is], d.drow >= 0, lane);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh.item_free[is]));
                if (!skip && !*err) {
                    ws.stat_p[d.trow * kStatParts] = make_float2(st.x, st.y);
                    if (d.drow >= 0) {
                        ws.stat_q[d.drow * kStatParts] = make_float2(st.z, st.w);
                        if (d.token_ok) {
                            const float ep = ex2_approx(fmaf(d.lp_x, d.c, -st.x));
                            const float eq = ex2_approx(fmaf(d.lq_x, d.c, -st.z));
                            const float lhs = d.u * eq * st.y, rhs = ep * st.w;     // accept iff u*q < p
                            const bool rejected = !(lhs < rhs);
                            const bool thin = !(fabsf(lhs - rhs) > 1e-3f * (lhs + rhs));
                            if (rejected && !thin) atomicMin(&ws.first_rej[d.b], d.pos);
                        }
                    }
                }
            }
            __syncwarp();
        }
    }
    __syncthreads();
    if (tid == 0 && sh.err) atomicExch(&ws.ctrl[0], sh.err);
}

}  // namespace specv
