// The streaming kernel set: works for every shape, pitch and alignment.
//
//   specv_prologue   offsets of the ragged batch, per-sequence checks, -1 fill
//   specv_row_stats  one read of every logits row: (reference, sum) of the tempered
//                    base-2 online softmax, per (row, split)
//   specv_resolve    per sequence: acceptance test of every draft position, first
//                    rejection, then ONE more read of the rows at that position for
//                    the residual (or bonus) inverse-CDF sample; emit
//
// Steps and formulas: the verify-and-resample pass of the paper's section
// "Speculative Sampling Results", with the accept / residual rule stated in
// include/spec_verify.h.
#pragma once

#include "specv_device.cuh"

namespace specv {

struct BatchView {
    const char* target;        // [n_draft_total + B] rows
    const char* draft;         // [n_draft_total] rows
    int64_t pitch_t, pitch_d;  // row pitch in BYTES
    int64_t V;
    const int32_t* tokens;
    const int32_t* k_per_row;  // may be null
    int32_t B, k_uniform;
    int64_t n_draft_total;
    const float* temperature;
    int per_row_temperature;
    const float* uniforms;
    // tree-structured verification only (null otherwise): parent of every node, and per draft
    // row whether its context has children (rows of contexts without children are never read)
    const int32_t* parent = nullptr;
    const int32_t* ctx_has_children = nullptr;
};

// Lookahead of the next speculation round, written by the kernel that emits a sequence's tokens
// (out == nullptr: not wanted): K+2 after a fully accepted draft, else K-1, within [k_min, k_max].
struct NextLookahead {
    int32_t* out;
    int32_t k_min, k_max;
};
__device__ __forceinline__ int32_t next_lookahead_of(int32_t k_raw, int32_t accepted, int32_t k_min, int32_t k_max) {
    const int32_t K = k_raw > 0 ? k_raw : 0;
    const int32_t next = accepted >= K ? K + 2 : K - 1;
    return min(max(next, k_min), k_max);
}

// ---------------------------------------------------------------------------------
// Prologue.  Block 0 scans max(K_b,0) into off_d[0..B] and records per-sequence
// argument errors; all blocks fill emitted_tokens with -1.
// ---------------------------------------------------------------------------------
constexpr int kPrologueThreads = 512;   // small enough to share an SM with a CTA of the ring statistics kernel

__global__ void __launch_bounds__(kPrologueThreads)
specv_prologue(BatchView in, int32_t* __restrict__ off_d, int32_t* __restrict__ seq_status,
               int32_t* __restrict__ emitted, int32_t* __restrict__ error_word, int32_t* __restrict__ done,
               int wait_at_end) {
    const int tid = threadIdx.x;
    // lets a kernel launched with programmatic stream serialization start its set-up now; it
    // waits for this grid to finish before reading what is written here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t n_slots = in.n_draft_total + in.B;
    for (int64_t s = (int64_t)blockIdx.x * kPrologueThreads + tid; s < n_slots;
         s += (int64_t)gridDim.x * kPrologueThreads)
        emitted[s] = -1;
    if (blockIdx.x == 0) {
        __shared__ int64_t warp_tot[32];
        __shared__ int64_t carry_s;
        if (tid == 0) {
            carry_s = 0;
            if (error_word) error_word[0] = error_word[1] = 0;   // ring kernels: expired-wait report, work counter
        }
        __syncthreads();
        const int lane = tid & 31, warp = tid >> 5;
        for (int32_t base = 0; base < in.B; base += kPrologueThreads) {
            const int32_t b = base + tid;
            int32_t k_raw = 0;
            if (b < in.B) k_raw = in.k_per_row ? in.k_per_row[b] : in.k_uniform;
            const int64_t k = k_raw > 0 ? k_raw : 0;
            int64_t incl = k;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int64_t up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            if (lane == 31) warp_tot[warp] = incl;
            __syncthreads();
            int64_t before = carry_s;
            for (int w = 0; w < warp; ++w) before += warp_tot[w];
            const int64_t excl = before + incl - k;
            if (b < in.B) {
                int status = 0;
                if (k_raw < 0 || excl + k > in.n_draft_total) status |= 1;   // SPECV_ROW_BAD_K
                // greedy verification has no temperature
                const float T = in.temperature ? in.temperature[in.per_row_temperature ? b : 0] : 1.0f;
                if (!(T > 0.0f) || isinf(T)) status |= 2;                    // SPECV_ROW_BAD_TEMPERATURE
                seq_status[b] = status;
                if (done) done[b] = 0;   // ring kernels: per-sequence count of finished chunk columns
                // keep offsets inside the buffers even for nonsense K, so later kernels never
                // form an out-of-range row index
                off_d[b] = (int32_t)(excl < in.n_draft_total ? excl : in.n_draft_total);
            }
            __syncthreads();
            if (tid == kPrologueThreads - 1) carry_s = before + incl;
            __syncthreads();
        }
        if (tid == 0) {
            const int64_t tot = carry_s;
            off_d[in.B] = (int32_t)(tot < in.n_draft_total ? tot : in.n_draft_total);
        }
    }
    // ring kernel set: this grid is launched after the statistics kernel and runs beside it; it ends
    // only when that kernel has, so that whatever waits for this grid has waited for both
    if (wait_at_end) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Sequence that owns packed draft row d: largest b with off_d[b] <= d.
__device__ __forceinline__ int32_t seq_of_draft_row(const int32_t* off_d, int32_t B, int64_t d) {
    int32_t lo = 0, hi = B;   // invariant: off_d[lo] <= d, answer in [lo, hi)
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if ((int64_t)off_d[mid] <= d) lo = mid; else hi = mid;
    }
    return lo;
}
// Sequence that owns packed target row t: largest b with off_d[b] + b <= t.
__device__ __forceinline__ int32_t seq_of_target_row(const int32_t* off_d, int32_t B, int64_t t) {
    int32_t lo = 0, hi = B;
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if ((int64_t)off_d[mid] + mid <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// ---------------------------------------------------------------------------------
// Row statistics.  Work item = (row, split); rows 0..n_target-1 are target rows, the
// rest draft rows.  A block owns items blockIdx.x, blockIdx.x + gridDim.x, ...
// For its slice of the row it produces (ref, sum) with  sum = sum_j 2^(l_j*c - ref),
// c = log2(e)/T, reading each element once.
// ---------------------------------------------------------------------------------
constexpr int kStatsThreads = 256;
constexpr int kStatsUnroll = 4;

template <int DT>
__global__ void __launch_bounds__(kStatsThreads)
specv_row_stats(BatchView in, const int32_t* __restrict__ off_d, int64_t n_target_rows,
                int64_t n_rows, int splits, float2* __restrict__ partial) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ float2 warp_part[kStatsThreads / 32];
    // launched with programmatic stream serialization: wait for the prologue's offsets, then let
    // the resolve kernel's blocks move in as this grid drains
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int64_t n_items = n_rows * splits;
    const int64_t nvec = (in.V + N - 1) / N;
    for (int64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int64_t row = item / splits;
        const int split = (int)(item - row * splits);
        const bool is_target = row < n_target_rows;
        if (!debug_in_range(row >= 0 && row < n_rows && split >= 0 && split < splits &&
                                (is_target || row - n_target_rows < in.n_draft_total), 101))
            continue;
        if (!is_target && in.ctx_has_children && !in.ctx_has_children[row - n_target_rows]) continue;   // block-uniform
        const char* rp = is_target ? in.target + row * in.pitch_t
                                   : in.draft + (row - n_target_rows) * in.pitch_d;
        float T = in.temperature[0];
        if (in.per_row_temperature) {
            const int32_t b = is_target ? seq_of_target_row(off_d, in.B, row)
                                        : seq_of_draft_row(off_d, in.B, row - n_target_rows);
            T = in.temperature[b];
        }
        const float c = (float)(kLog2e / (double)T);
        const bool aligned = (reinterpret_cast<uintptr_t>(rp) & 15u) == 0;
        const int64_t v0 = nvec * split / splits, v1 = nvec * (split + 1) / splits;

        float ref = kNoMax, s0 = 0.f, s1 = 0.f;
        for (int64_t v = v0 + tid; v < v1; v += kStatsThreads * kStatsUnroll) {
            uint4 raw[kStatsUnroll];
#pragma unroll
            for (int k = 0; k < kStatsUnroll; ++k) {
                const int64_t vv = v + (int64_t)k * kStatsThreads;
                raw[k] = (vv < v1) ? load_vec<DT>(rp, aligned, vv, in.V) : neg_inf_vec(E::kNegInfWord);
            }
            float x[kStatsUnroll * N];
#pragma unroll
            for (int k = 0; k < kStatsUnroll; ++k) E::unpack(raw[k], x + k * N);
            float mx = x[0];
#pragma unroll
            for (int k = 1; k < kStatsUnroll * N; ++k) mx = fmaxf(mx, x[k]);
            const float cand = mx * c;
            if (cand > ref) {           // rare after the first few iterations
                const float f = ex2_approx(ref - cand);
                s0 *= f; s1 *= f;
                ref = cand;
            }
            // two elements per instruction (packed f32x2, same results as the scalar forms)
            const unsigned long long cc = pack_f32x2(c, c), nr = pack_f32x2(-ref, -ref);
            unsigned long long acc = pack_f32x2(s0, s1);
#pragma unroll
            for (int k = 0; k < kStatsUnroll * N; k += 2) {
                float t0, t1;
                unpack_f32x2(fma_f32x2(pack_f32x2(x[k], x[k + 1]), cc, nr), t0, t1);
                acc = add_f32x2(acc, pack_f32x2(ex2_approx(t0), ex2_approx(t1)));
            }
            unpack_f32x2(acc, s0, s1);
        }
        float sum = s0 + s1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float oref = __shfl_xor_sync(0xffffffffu, ref, o);
            const float osum = __shfl_xor_sync(0xffffffffu, sum, o);
            merge_ref_sum(ref, sum, oref, osum);
        }
        if (lane == 0) warp_part[warp] = make_float2(ref, sum);
        __syncthreads();
        if (warp == 0) {
            float2 p = (lane < kStatsThreads / 32) ? warp_part[lane] : make_float2(kNoMax, 0.f);
            ref = p.x; sum = p.y;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float oref = __shfl_xor_sync(0xffffffffu, ref, o);
                const float osum = __shfl_xor_sync(0xffffffffu, sum, o);
                merge_ref_sum(ref, sum, oref, osum);
            }
            if (lane == 0) partial[item] = make_float2(ref, sum);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// Resolve.  One block per sequence.
// ---------------------------------------------------------------------------------
constexpr int kResolveThreads = 1024;
constexpr int kResolveWarps = kResolveThreads / 32;

struct RowNorm {     // sum_j 2^(l_j*c - ref) = sum   (sum in double, merged in split order)
    float ref;
    double sum;
};

// Merge of a row's split partials by a whole warp, one split per lane (splits <= 32), in a
// fixed shuffle order; every lane gets the result.
__device__ __forceinline__ RowNorm warp_merge_splits(const float2* partial, int64_t row, int splits, int lane) {
    const float2 v = lane < splits ? partial[row * splits + lane] : make_float2(kNoMax, 0.f);
    float ref = v.x;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ref = fmaxf(ref, __shfl_xor_sync(0xffffffffu, ref, o));
    double t = (double)v.y * exp2((double)v.x - (double)ref);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        int lo = __double2loint(t), hi = __double2hiint(t);
        lo = __shfl_xor_sync(0xffffffffu, lo, o);
        hi = __shfl_xor_sync(0xffffffffu, hi, o);
        t += __hiloint2double(hi, lo);
    }
    return RowNorm{ref, t};
}

// Constants of the one or two rows being sampled from.  With e_p(j) = 2^(lp_j*c - p_ref) and
// e_q(j) = 2^(lq_j*c - q_ref) the probabilities are p_j = e_p(j) / sum_p and q_j = e_q(j) / sum_q,
// so max(0, p_j - w q_j) = max(0, e_p(j) - kappa e_q(j)) / sum_p with kappa = w sum_p / sum_q
// (w = 1 for the plain residual).  The inverse CDF is indifferent to a common factor, so all
// masses are kept in units of 1 / sum_p: one fused multiply-add instead of two multiplies and
// a subtraction per element.
struct SampleRows {
    const char* p;
    const char* q;        // null: sample from p alone
    bool p_aligned, q_aligned;
    float c;              // log2(e)/T
    float p_ref, q_ref;
    float kappa;
};

// Masses of one 16-byte vector of the sampled distribution, max(0, p - q) or p in units of
// 1 / sum_p, from the raw vectors of the two rows.
template <int DT>
__device__ __forceinline__ void mass_of_raw(const SampleRows& sr, const uint4& rawp, const uint4& rawq, float* r) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    float xp[N];
    E::unpack(rawp, xp);
    if (sr.q) {
        float xq[N];
        E::unpack(rawq, xq);
#pragma unroll
        for (int k = 0; k < N; ++k) {
            const float ep = ex2_approx(fmaf(xp[k], sr.c, -sr.p_ref));
            const float eq = ex2_approx(fmaf(xq[k], sr.c, -sr.q_ref));
            r[k] = fmaxf(fmaf(-sr.kappa, eq, ep), 0.f);
        }
    } else {
#pragma unroll
        for (int k = 0; k < N; ++k) r[k] = ex2_approx(fmaf(xp[k], sr.c, -sr.p_ref));
    }
}

// Warp-level second half of the inverse CDF: prefix over the segment masses in double, find
// the segment where the running mass first exceeds u * total, then the token inside it
// (its vectors are re-read and their masses recomputed exactly as for the segment sums).
// Returns the token to every lane, or -1 if the total mass is 0.
// `load_pair(v, rawp, rawq)` supplies 16-byte vector v of the row(s) the masses are taken from.
template <int DT, class LoadPair>
__device__ int32_t locate_in_segments_with(const SampleRows& sr, double u, const float* seg, int32_t nseg, int lane,
                                           LoadPair load_pair) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    auto masses = [&](int64_t v, float* r) {
        uint4 rawp, rawq;
        load_pair(v, rawp, rawq);
        mass_of_raw<DT>(sr, rawp, rawq, r);
    };
    const int32_t per = (nseg + 31) / 32;
    const int32_t s_begin = min(lane * per, nseg), s_end = min(s_begin + per, nseg);
    double local = 0.0;
    for (int32_t s = s_begin; s < s_end; ++s) local += (double)seg[s];
    const double incl = warp_inclusive_scan(local, lane);
    const double total = shfl_double(incl, 31);
    int32_t token = -1;
    if (total > 0.0) {
        const double t = u * total;
        // lane whose block of segments holds the crossing; if rounding hides it, the
        // last lane that has any mass
        unsigned cross = __ballot_sync(0xffffffffu, incl > t);
        const unsigned has = __ballot_sync(0xffffffffu, local > 0.0);
        const int owner = cross ? (__ffs(cross) - 1) : (31 - __clz(has));
        int32_t found_seg = -1;
        double base = 0.0;
        if (lane == owner) {
            double run = incl - local;
            int32_t last_pos = -1;
            double last_base = 0.0;
            for (int32_t s = s_begin; s < s_end; ++s) {
                const double m = (double)seg[s];
                if (m > 0.0) { last_pos = s; last_base = run; }
                if (run + m > t) { found_seg = s; base = run; break; }
                run += m;
            }
            if (found_seg < 0) { found_seg = last_pos; base = last_base; }
        }
        found_seg = __shfl_sync(0xffffffffu, found_seg, owner);
        base = shfl_double(base, owner);
        if (!debug_in_range(found_seg >= 0 && found_seg < nseg, 104)) return -1;
        // inside the segment: recompute the masses exactly as pass A did
        float r[N];
        masses((int64_t)found_seg * 32 + lane, r);
        double lane_sum = 0.0;
#pragma unroll
        for (int k = 0; k < N; ++k) lane_sum += (double)r[k];
        const double lane_incl = warp_inclusive_scan(lane_sum, lane);
        double run = base + lane_incl - lane_sum;
        int hit = -1, last_mass = -1;
#pragma unroll
        for (int k = 0; k < N; ++k) {
            run += (double)r[k];
            if (r[k] > 0.f) last_mass = k;
            if (hit < 0 && r[k] > 0.f && run > t) hit = k;
        }
        const unsigned hits = __ballot_sync(0xffffffffu, hit >= 0);
        const unsigned massive = __ballot_sync(0xffffffffu, last_mass >= 0);
        const int src = hits ? (__ffs(hits) - 1) : (31 - __clz(massive));
        const int k_sel = hits ? hit : last_mass;
        token = (int32_t)(((int64_t)found_seg * 32 + src) * N + __shfl_sync(0xffffffffu, k_sel, src));
    }
    return token;
}

// The same with the vectors read from the rows in global memory.
template <int DT, bool FAST>
__device__ int32_t locate_in_segments(const SampleRows& sr, int64_t V, double u, const float* seg,
                                      int32_t nseg, int lane) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    auto load = [&](const char* row, bool aligned, int64_t v) -> uint4 {
        if (FAST) return v * N < V ? ld_stream16(row + v * 16) : neg_inf_vec(E::kNegInfWord);
        return load_vec<DT>(row, aligned, v, V);
    };
    return locate_in_segments_with<DT>(sr, u, seg, nseg, lane, [&](int64_t v, uint4& rawp, uint4& rawq) {
        rawp = load(sr.p, sr.p_aligned, v);
        rawq = sr.q ? load(sr.q, sr.q_aligned, v) : make_uint4(0u, 0u, 0u, 0u);
    });
}

// Segment masses of the distribution `sr` describes into seg[] (shared, one float per 32-vector
// segment); NWARPS warps take part, `warp` in [0, NWARPS) being the caller's index among them;
// `sync` is a barrier over exactly those warps and is called once at the end.
// FAST: both rows start on 16-byte boundaries and V is a whole number of vectors.
// `store(s, a)` receives the mass a of segment s from lane 0 of the warp that summed it.
template <int DT, int NWARPS, bool FAST, class StoreFn, class SyncFn>
__device__ void block_segment_sums_to(const SampleRows& sr, int64_t V, int warp, StoreFn store, SyncFn sync) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    constexpr int SEG = 32 * N;                 // elements per warp-wide segment
    const int lane = threadIdx.x & 31;
    const int32_t nseg = (int32_t)((V + SEG - 1) / SEG);
    auto load = [&](const char* row, bool aligned, int64_t v) -> uint4 {
        if (FAST) return v * N < V ? ld_stream16(row + v * 16) : neg_inf_vec(E::kNegInfWord);
        return load_vec<DT>(row, aligned, v, V);
    };
    // segments dealt round-robin to warps (vocabulary order kept by the segment index, so the
    // prefix taken later is over token ids); two segments per warp and step, and the loads of the
    // next step are issued before the arithmetic of this one (the exponentials of a step take as
    // long as its loads, so neither waits for the other)
    constexpr int U = 2;
    uint4 curp[U], curq[U], nxtp[U], nxtq[U];
    auto issue = [&](int32_t s0, uint4* rp, uint4* rq) {
#pragma unroll
        for (int i = 0; i < U; ++i) {
            const int32_t s = s0 + i * NWARPS;
            if (s < nseg) {
                rp[i] = load(sr.p, sr.p_aligned, (int64_t)s * 32 + lane);
                rq[i] = sr.q ? load(sr.q, sr.q_aligned, (int64_t)s * 32 + lane) : make_uint4(0u, 0u, 0u, 0u);
            }
        }
    };
    if (warp < nseg) issue(warp, curp, curq);
    for (int32_t s0 = warp; s0 < nseg; s0 += U * NWARPS) {
        if (s0 + U * NWARPS < nseg) issue(s0 + U * NWARPS, nxtp, nxtq);
#pragma unroll
        for (int i = 0; i < U; ++i) {
            const int32_t s = s0 + i * NWARPS;
            if (s < nseg) {      // warp-uniform
                float r[N];
                mass_of_raw<DT>(sr, curp[i], curq[i], r);
                float a = 0.f;
#pragma unroll
                for (int k = 0; k < N; ++k) a += r[k];
                a = warp_sum(a);
                if (lane == 0) store(s, a);
            }
        }
#pragma unroll
        for (int i = 0; i < U; ++i) { curp[i] = nxtp[i]; curq[i] = nxtq[i]; }
    }
    sync();
}
template <int DT, int NWARPS, bool FAST, class SyncFn>
__device__ void block_segment_sums(const SampleRows& sr, int64_t V, float* seg, int warp, SyncFn sync) {
    block_segment_sums_to<DT, NWARPS, FAST>(sr, V, warp, [seg](int32_t s, float a) { seg[s] = a; }, sync);
}

// Total of the segment masses, summed in double exactly as locate_in_segments sums them (a
// contiguous block of segments per lane, then across lanes); every lane gets it.
__device__ __forceinline__ double warp_segment_total(const float* seg, int32_t nseg, int lane) {
    const int32_t per = (nseg + 31) / 32;
    const int32_t s_begin = min(lane * per, nseg), s_end = min(s_begin + per, nseg);
    double local = 0.0;
    for (int32_t s = s_begin; s < s_end; ++s) local += (double)seg[s];
    return shfl_double(warp_inclusive_scan(local, lane), 31);
}

// Inverse-CDF sample from the distribution `sr` describes; whole block participates.
// seg[] is scratch.  Returns the token to every thread, or -1 if the total mass is 0.
template <int DT, int NWARPS, bool FAST, class SyncFn>
__device__ int32_t block_inverse_cdf(const SampleRows& sr, int64_t V, double u, float* seg,
                                     int32_t* result_slot, int warp, SyncFn sync) {
    constexpr int SEG = 32 * Elt<DT>::kPerVec;
    const int lane = threadIdx.x & 31;
    const int32_t nseg = (int32_t)((V + SEG - 1) / SEG);
    block_segment_sums<DT, NWARPS, FAST>(sr, V, seg, warp, sync);      // pass A
    if (warp == 0) {                                                   // pass B: prefix, locate
        const int32_t token = locate_in_segments<DT, FAST>(sr, V, u, seg, nseg, lane);
        if (lane == 0) *result_slot = token;
    }
    sync();
    const int32_t token = *result_slot;
    sync();
    return token;
}

template <int DT>
__global__ void __launch_bounds__(kResolveThreads)
specv_resolve(BatchView in, const int32_t* __restrict__ off_d, const int32_t* __restrict__ seq_status,
              const float2* __restrict__ partial, int splits, int64_t n_target_rows,
              int32_t* __restrict__ accepted_len, int32_t* __restrict__ emitted,
              int32_t* __restrict__ row_status, float* __restrict__ diag_p, float* __restrict__ diag_q,
              NextLookahead next) {
    using E = Elt<DT>;
    extern __shared__ float seg[];
    __shared__ int32_t first_reject;
    __shared__ int32_t bad_token;
    __shared__ int32_t result_slot;
    __shared__ SampleRows rows;

    const int tid = threadIdx.x;
    const int32_t b = blockIdx.x;
    asm volatile("griddepcontrol.wait;" ::: "memory");   // all row statistics must be in memory
    const int64_t d0 = off_d[b];
    const int64_t t0 = d0 + b;
    int status = seq_status[b];
    const int32_t k_raw = in.k_per_row ? in.k_per_row[b] : in.k_uniform;
    const int32_t K = k_raw > 0 ? k_raw : 0;
    // a valid sequence's rows lie inside the packed buffers
    if (!(status & 1) && !debug_in_range(d0 >= 0 && d0 + K <= in.n_draft_total && t0 + K < n_target_rows, 102))
        status |= 16;

    if (tid == 0) { first_reject = K; bad_token = 0; }
    __syncthreads();
    if (!(status & 1)) {
        for (int32_t i = tid; i < K; i += kResolveThreads) {
            const int32_t x = in.tokens[d0 + i];
            if (x < 0 || (int64_t)x >= in.V) bad_token = 1;
        }
    }
    __syncthreads();
    if (bad_token) status |= 4;   // SPECV_ROW_BAD_TOKEN
    if (status) {
        if (tid == 0) {
            accepted_len[b] = 0;
            if (row_status) row_status[b] = status;
            if (next.out) next.out[b] = next_lookahead_of(k_raw, 0, next.k_min, next.k_max);
        }
        return;   // the prologue already wrote -1 into every slot
    }

    const float T = in.temperature[in.per_row_temperature ? b : 0];
    const float c = (float)(kLog2e / (double)T);

    // acceptance test of every draft position, in double from the streamed statistics: one warp
    // per position, its lanes merging the row's split partials
    const int lane = tid & 31;
    for (int32_t i = tid >> 5; i < K; i += kResolveWarps) {
        const RowNorm np = warp_merge_splits(partial, t0 + i, splits, lane);
        const RowNorm nq = warp_merge_splits(partial, n_target_rows + d0 + i, splits, lane);
        if (lane == 0) {
            const int32_t x = in.tokens[d0 + i];
            const double lp = (double)E::load1(in.target + (t0 + i) * in.pitch_t, x);
            const double lq = (double)E::load1(in.draft + (d0 + i) * in.pitch_d, x);
            const double p = exp2(lp * (double)c - (double)np.ref) / np.sum;
            const double q = exp2(lq * (double)c - (double)nq.ref) / nq.sum;
            if (diag_p) diag_p[d0 + i] = (float)p;
            if (diag_q) diag_q[d0 + i] = (float)q;
            const double u = (double)in.uniforms[t0 + i];
            if (!(u * q < p)) atomicMin(&first_reject, i);
        }
    }
    __syncthreads();
    const int32_t n = first_reject;

    if (tid < 32) {
        const RowNorm np = warp_merge_splits(partial, t0 + n, splits, lane);
        RowNorm nq{0.f, 1.0};
        if (n < K) nq = warp_merge_splits(partial, n_target_rows + d0 + n, splits, lane);
        if (lane == 0) {
            rows.p = in.target + (t0 + n) * in.pitch_t;
            rows.p_aligned = (reinterpret_cast<uintptr_t>(rows.p) & 15u) == 0;
            rows.c = c;
            rows.p_ref = np.ref;
            rows.q = nullptr;
            rows.q_aligned = false;
            rows.q_ref = 0.f;
            rows.kappa = 0.f;
            if (n < K) {
                rows.q = in.draft + (d0 + n) * in.pitch_d;
                rows.q_aligned = (reinterpret_cast<uintptr_t>(rows.q) & 15u) == 0;
                rows.q_ref = nq.ref;
                rows.kappa = (float)(np.sum / nq.sum);
            }
        }
    }
    __syncthreads();
    const double u2 = (double)in.uniforms[t0 + K];
    SampleRows sr = rows;
    auto sync_all = [] { __syncthreads(); };
    int32_t token = block_inverse_cdf<DT, kResolveWarps, false>(sr, in.V, u2, seg, &result_slot, tid >> 5, sync_all);
    if (token < 0 && sr.q) {
        // the residual rounded to nothing: sample from the target row itself
        status |= 8;   // SPECV_ROW_ZERO_RESIDUAL
        sr.q = nullptr;
        token = block_inverse_cdf<DT, kResolveWarps, false>(sr, in.V, u2, seg, &result_slot, tid >> 5, sync_all);
    }
    if (token < 0) token = (int32_t)(in.V - 1);   // a row without any mass (all logits -inf)
    if (!debug_in_range(token >= 0 && (int64_t)token < in.V && n >= 0 && n <= K, 103)) token = -1;

    for (int32_t i = tid; i <= K; i += kResolveThreads)
        emitted[t0 + i] = (i < n) ? in.tokens[d0 + i] : (i == n ? token : -1);
    if (tid == 0) {
        accepted_len[b] = n;
        if (row_status) row_status[b] = status;
        if (next.out) next.out[b] = next_lookahead_of(k_raw, n, next.k_min, next.k_max);
    }
}

// ---------------------------------------------------------------------------------
// Lookahead of the next round: K+2 after a fully accepted draft, else K-1, within [k_min, k_max].
// ---------------------------------------------------------------------------------
__global__ void specv_next_lookahead(const int32_t* __restrict__ k_per_row, int32_t k_uniform,
                                     const int32_t* __restrict__ accepted_len, int32_t B, int32_t k_min,
                                     int32_t k_max, int32_t* __restrict__ next_k) {
    const int32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    next_k[b] = next_lookahead_of(k_per_row ? k_per_row[b] : k_uniform, accepted_len[b], k_min, k_max);
}

}  // namespace specv
