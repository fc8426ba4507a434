// The whole pass in ONE launch for small batches (one to a dozen sequences): a thread-block cluster
// of eight CTAs per sequence holds every logits row of the sequence in its shared memory.
//
// For a handful of sequences the pass is not bound by HBM but by latency: three dependent launches
// (offsets, row statistics, resolve), each with its own round of loads, and a second read of the
// row pair a token is drawn from.  Here every logit is fetched exactly once:
//   CTA r of a cluster takes the columns [r, r+1) * slice of EVERY row of its sequence (K+1 target
//   rows, K draft rows) with bulk async copies into shared memory (all in flight at once);
//   one warp per row computes the (reference, sum) of its slice and writes it into the partials
//   table of all eight CTAs through distributed shared memory; after one cluster barrier every CTA
//   holds the statistics of every row and takes the decisions (all positions in parallel, in
//   double, first rejection) redundantly and identically;
//   the segment sums of the distribution the token is drawn from are computed from the slices
//   still in shared memory and written to the segment table of all eight CTAs; after a second
//   cluster barrier CTA 0 locates the token (prefix over the table, one 512-byte segment re-read
//   from L2) and writes the sequence's outputs.
// No workspace, no atomics in global memory, no wait on another CTA other than the hardware cluster
// barrier; the one bounded wait is for the CTA's own copies.
//
// Same arithmetic as the streaming kernels: statistics merged per row in double in a fixed order
// (warp_merge_splits over the 32 partials of a row), decisions u q < p in double, masses by mass_of_raw,
// inverse CDF by locate_in_segments.
#pragma once

#include "specv_ring_kernels.cuh"

namespace specv {

constexpr int kClusterCtas = 8;
constexpr int kClusterThreads = 512;
constexpr int kClusterWarps = kClusterThreads / 32;
constexpr int kClusterMaxK = 32;                          // lookahead the shared-memory tables are sized for
constexpr int kClusterMaxRows = 2 * kClusterMaxK + 1;
constexpr int kClusterMaxSeqs = 18;                       // 8 CTAs each on 148 SMs; offsets are scanned by one warp
constexpr int kClusterSub = 4;                            // a CTA's slice of a row is summed in four parts (all warps busy)
constexpr int kClusterParts = kClusterCtas * kClusterSub; // partial statistics per row: one per lane of the merging warp

struct ClusterShared {
    float2 part[kClusterMaxRows * kClusterParts];         // [row][cta][sub]: partial (ref, sum) of every row from every CTA
    double norm_sum[kClusterMaxRows];                     // merged statistics of every row (each CTA merges for itself)
    float norm_ref[kClusterMaxRows];
    int err_of[kClusterCtas];                             // a CTA whose copies did not arrive reports here, everywhere
    unsigned long long bar;
    SampleRows rows;
    int32_t first_reject, bad_token, err, token;
    // what the decisions need of every draft position, fetched while the rows are on their way
    int32_t tok[kClusterMaxK];
    float lp[kClusterMaxK], lq[kClusterMaxK], u[kClusterMaxK + 1];
};

__device__ __forceinline__ uint32_t map_to_cta(const void* smem_ptr, uint32_t cta) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_u32(smem_ptr)), "r"(cta));
    return a;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Dynamic shared memory: the slices of the sequence's rows (row-major, `slice_bytes` each, 16-byte
// aligned), then the segment table (one float per 512-byte segment of a row).
template <int DT>
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kClusterThreads, 1)
specv_cluster_pass(BatchView in, int32_t slice_bytes, int32_t* __restrict__ accepted_len, int32_t* __restrict__ emitted,
                   int32_t* __restrict__ row_status, float* __restrict__ diag_p, float* __restrict__ diag_q,
                   NextLookahead next) {
    using E = Elt<DT>;
    constexpr int N = E::kPerVec;
    constexpr int SEG = 32 * N;
    extern __shared__ __align__(128) unsigned char cl_smem[];
    __shared__ ClusterShared sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int32_t b = blockIdx.x / kClusterCtas;
    const bool writer = rank == 0;
    const int64_t row_bytes = in.V * E::kBytes;
    const int32_t nseg = (int32_t)((in.V + SEG - 1) / SEG);

    // offsets over max(K_b, 0), clamped to the buffers like the prologue kernel's (every warp, B <= 18)
    int32_t k_raw = 0;
    if (lane < in.B) k_raw = in.k_per_row ? in.k_per_row[lane] : in.k_uniform;
    int64_t incl = k_raw > 0 ? k_raw : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    const int64_t D = in.n_draft_total;
    const int64_t excl_b = __shfl_sync(0xffffffffu, incl, b) - (__shfl_sync(0xffffffffu, k_raw, b) > 0 ? __shfl_sync(0xffffffffu, k_raw, b) : 0);
    const int64_t incl_b = __shfl_sync(0xffffffffu, incl, b);
    const int32_t kb_raw = __shfl_sync(0xffffffffu, k_raw, b);
    const int32_t K = kb_raw > 0 ? kb_raw : 0;
    const int64_t d0 = excl_b < D ? excl_b : D;                   // clamped like off_d[b]
    const int64_t d1 = incl_b < D ? incl_b : D;                   // off_d[b + 1]
    const int64_t t0 = d0 + b;

    int status = 0;
    if (kb_raw < 0 || excl_b + K > D) status |= 1;                // SPECV_ROW_BAD_K
    const float T = in.temperature[in.per_row_temperature ? b : 0];
    if (!(T > 0.0f) || isinf(T)) status |= 2;                     // SPECV_ROW_BAD_TEMPERATURE
    if (K > kClusterMaxK) status |= 16;                           // the host only sends batches that fit

    if (tid == 0) { sh.first_reject = K; sh.bad_token = 0; sh.err = 0; }
    if (tid < kClusterCtas) sh.err_of[tid] = 0;
    __syncthreads();

    // ---- every row's slice into shared memory, all copies in flight at once: issued first, everything
    // else the pass needs from global memory is fetched while they are on their way --------------------
    const int32_t n_rows = 2 * K + 1;                             // rows 0..K target, K+1..2K draft
    const int64_t slice_off = (int64_t)rank * slice_bytes;
    const int32_t my_bytes = (int32_t)(row_bytes - slice_off < slice_bytes ? (row_bytes - slice_off > 0 ? row_bytes - slice_off : 0)
                                                                           : slice_bytes);
    auto row_ptr = [&](int32_t r) {
        return r <= K ? in.target + (t0 + r) * in.pitch_t : in.draft + (d0 + (r - K - 1)) * in.pitch_d;
    };
    volatile int* err = &sh.err;
    const bool copying = !status && my_bytes > 0;                 // the same in every warp
    if (warp == 0) {
        if (lane == 0) {
            mbar_init(smem_u32(&sh.bar), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            if (copying) mbar_expect_tx(smem_u32(&sh.bar), (uint32_t)my_bytes * (uint32_t)n_rows);
        }
        __syncwarp();
        if (copying)
            for (int32_t r = lane; r < n_rows; r += 32)
                bulk_load(smem_u32(cl_smem + (size_t)r * slice_bytes), row_ptr(r) + slice_off, (uint32_t)my_bytes,
                          smem_u32(&sh.bar));
    }
    // the drafted tokens, their two logits and the uniforms (one thread per position)
    if (!(status & (1 | 16))) {
        for (int32_t i = tid; i <= K; i += kClusterThreads) {
            sh.u[i] = in.uniforms[t0 + i];
            if (i < K) {
                const int32_t x = in.tokens[d0 + i];
                const bool ok = x >= 0 && (int64_t)x < in.V;
                if (!ok) sh.bad_token = 1;
                sh.tok[i] = x;
                sh.lp[i] = ok ? E::load1(in.target + (t0 + i) * in.pitch_t, x) : 0.f;
                sh.lq[i] = ok ? E::load1(in.draft + (d0 + i) * in.pitch_d, x) : 0.f;
            }
        }
    }
    __syncthreads();
    if (sh.bad_token) status |= 4;                                // SPECV_ROW_BAD_TOKEN
    if (copying) mbar_wait(smem_u32(&sh.bar), 0, err, 71);        // also before giving up on a bad token: the copies target this CTA

    // slots of this sequence in the packed outputs (clamped offsets: together they tile [0, D + B));
    // the last cluster also owns the slots no sequence reaches
    const int64_t slot_end = (b == in.B - 1) ? D + in.B : d1 + b + 1;
    if (status) {                 // the same in every CTA of the cluster: no barrier is left behind
        if (writer) {
            for (int64_t s = t0 + tid; s < slot_end; s += kClusterThreads) emitted[s] = -1;
            if (tid == 0) {
                accepted_len[b] = 0;
                if (row_status) row_status[b] = status;
                if (next.out) next.out[b] = next_lookahead_of(kb_raw, 0, next.k_min, next.k_max);
            }
        }
        return;
    }
    const float c = (float)(kLog2e / (double)T);
    const int32_t my_vecs = my_bytes / 16;

    // ---- row statistics of the slices: a warp per (row, quarter of the slice) ------------------------
    for (int32_t item = warp; item < n_rows * kClusterSub; item += kClusterWarps) {
        const int32_t r = item / kClusterSub, sub = item % kClusterSub;
        const uint4* src = reinterpret_cast<const uint4*>(cl_smem + (size_t)r * slice_bytes);
        const int32_t v_begin = (int32_t)((int64_t)my_vecs * sub / kClusterSub);
        const int32_t v_end = (int32_t)((int64_t)my_vecs * (sub + 1) / kClusterSub);
        float ref = kNoMax, s0 = 0.f, s1 = 0.f;
        for (int32_t v = v_begin + lane; v < v_end; v += 32 * 2) {
            uint4 raw[2];
            raw[0] = src[v];
            raw[1] = v + 32 < v_end ? src[v + 32] : neg_inf_vec(E::kNegInfWord);
            float x[2 * N];
            E::unpack(raw[0], x);
            E::unpack(raw[1], x + N);
            float mx = x[0];
#pragma unroll
            for (int k = 1; k < 2 * N; ++k) mx = fmaxf(mx, x[k]);
            const float cand = mx * c;
            if (cand > ref) {
                const float f = ex2_approx(ref - cand);
                s0 *= f; s1 *= f;
                ref = cand;
            }
            const unsigned long long cc = pack_f32x2(c, c), nr = pack_f32x2(-ref, -ref);
            unsigned long long acc = pack_f32x2(s0, s1);
#pragma unroll
            for (int k = 0; k < 2 * N; k += 2) {
                float a0, a1;
                unpack_f32x2(fma_f32x2(pack_f32x2(x[k], x[k + 1]), cc, nr), a0, a1);
                acc = add_f32x2(acc, pack_f32x2(ex2_approx(a0), ex2_approx(a1)));
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
        // entry [r][rank][sub] of every CTA's table: lanes 0..7 write one CTA each
        if (lane < kClusterCtas) {
            const uint32_t dst = map_to_cta(&sh.part[r * kClusterParts + rank * kClusterSub + sub], (uint32_t)lane);
            asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(dst), "f"(ref), "f"(sum) : "memory");
        }
    }
    if (warp == kClusterWarps - 1 && lane < kClusterCtas) {       // this CTA's copies: arrived or not
        const uint32_t dst = map_to_cta(&sh.err_of[rank], (uint32_t)lane);
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(dst), "r"((uint32_t)*err) : "memory");
    }
    cluster_barrier();                                            // #1: all statistics everywhere
    int any_err = 0;
#pragma unroll
    for (int i = 0; i < kClusterCtas; ++i) any_err |= sh.err_of[i];
    if (any_err) {                // the same in every CTA; nothing more is exchanged
        if (writer) {
            for (int64_t s = t0 + tid; s < slot_end; s += kClusterThreads) emitted[s] = -1;
            if (tid == 0) {
                accepted_len[b] = 0;
                if (row_status) row_status[b] = 16 | (any_err << 8);          // SPECV_ROW_INTERNAL
                if (next.out) next.out[b] = next_lookahead_of(kb_raw, 0, next.k_min, next.k_max);
            }
        }
        if (*err && tid == 0) {   // copies that were issued may still land in this CTA's shared memory
            const long long t_wait = clock64();
            while (clock64() - t_wait < 200000) {}
        }
        __syncthreads();
        return;
    }

    // ---- every row's statistics merged (a warp per row, double, fixed order), then the decisions: every
    // draft position in parallel, in double; first rejection ------------------------------------------
    for (int32_t r = warp; r < n_rows; r += kClusterWarps) {
        const RowNorm nr = warp_merge_splits(sh.part, r, kClusterParts, lane);
        if (lane == 0) { sh.norm_ref[r] = nr.ref; sh.norm_sum[r] = nr.sum; }
    }
    __syncthreads();
    for (int32_t i = tid; i < K; i += kClusterThreads) {
        const double p = exp2((double)sh.lp[i] * (double)c - (double)sh.norm_ref[i]) / sh.norm_sum[i];
        const double q = exp2((double)sh.lq[i] * (double)c - (double)sh.norm_ref[K + 1 + i]) / sh.norm_sum[K + 1 + i];
        if (writer && diag_p) diag_p[d0 + i] = (float)p;
        if (writer && diag_q) diag_q[d0 + i] = (float)q;
        if (!((double)sh.u[i] * q < p)) atomicMin(&sh.first_reject, i);
    }
    __syncthreads();
    const int32_t n = sh.first_reject;
    if (tid == 0) {
        SampleRows& rows = sh.rows;
        rows.p = in.target + (t0 + n) * in.pitch_t;
        rows.p_aligned = true;                                    // the host sends aligned rows only
        rows.c = c;
        rows.p_ref = sh.norm_ref[n];
        rows.q = nullptr; rows.q_aligned = false; rows.q_ref = 0.f; rows.kappa = 0.f;
        if (n < K) {
            rows.q = in.draft + (d0 + n) * in.pitch_d;
            rows.q_aligned = true;
            rows.q_ref = sh.norm_ref[K + 1 + n];
            rows.kappa = (float)(sh.norm_sum[n] / sh.norm_sum[K + 1 + n]);
        }
    }
    __syncthreads();

    // ---- segment sums of the drawn-from distribution, from the slices in shared memory ---------------
    float* const seg = reinterpret_cast<float*>(cl_smem + (size_t)n_rows * slice_bytes);
    const int32_t seg0 = (int32_t)(slice_off / 512);              // first segment of this CTA's slice
    const int32_t my_segs = (my_vecs + 31) / 32;
    auto segment_pass = [&](const SampleRows& sr) {
        const uint4* sp = reinterpret_cast<const uint4*>(cl_smem + (size_t)n * slice_bytes);
        const uint4* sq = reinterpret_cast<const uint4*>(cl_smem + (size_t)(K + 1 + (n < K ? n : 0)) * slice_bytes);
        for (int32_t s = warp; s < my_segs; s += kClusterWarps) {
            const int32_t v = s * 32 + lane;
            float a = 0.f;
            if (v < my_vecs) {
                float r[N];
                mass_of_raw<DT>(sr, sp[v], sr.q ? sq[v] : make_uint4(0u, 0u, 0u, 0u), r);
#pragma unroll
                for (int k = 0; k < N; ++k) a += r[k];
            }
            a = warp_sum(a);
            if (lane < kClusterCtas) {
                const uint32_t dst = map_to_cta(&seg[seg0 + s], (uint32_t)lane);
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst), "f"(a) : "memory");
            }
        }
        cluster_barrier();
    };
    SampleRows sr = sh.rows;
    segment_pass(sr);                                             // #2
    // ---- CTA 0 locates the token: prefix over the table, then the crossing segment's vectors straight
    // from the shared memory of the CTA that holds them ---------------------------------------------
    if (writer) {
        if (warp == 0) {
            const int32_t row_p = n, row_q = K + 1 + (n < K ? n : 0);
            auto slice_vector = [&](int32_t row, int64_t v) -> uint4 {
                const int64_t byte = v * 16;
                if (byte >= row_bytes) return neg_inf_vec(E::kNegInfWord);
                const uint32_t owner = (uint32_t)(byte / slice_bytes);
                const uint32_t a = map_to_cta(cl_smem + (size_t)row * slice_bytes + (size_t)(byte - (int64_t)owner * slice_bytes), owner);
                uint4 r;
                asm volatile("ld.shared::cluster.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(a) : "memory");
                return r;
            };
            const int32_t token = locate_in_segments_with<DT>(sr, (double)sh.u[K], seg, nseg, lane,
                                                              [&](int64_t v, uint4& rawp, uint4& rawq) {
                                                                  rawp = slice_vector(row_p, v);
                                                                  rawq = sr.q ? slice_vector(row_q, v) : make_uint4(0u, 0u, 0u, 0u);
                                                              });
            if (lane == 0) sh.token = token;
        }
        __syncthreads();
        if (sh.token < 0 && sr.q) {       // block-uniform; rare
            // the residual rounded to nothing: sample from the target row itself.  This CTA alone, the row
            // read from global memory (the other CTAs have nothing more to contribute)
            status |= 8;                  // SPECV_ROW_ZERO_RESIDUAL
            sr.q = nullptr;
            block_segment_sums<DT, kClusterWarps, true>(sr, in.V, seg, warp, [] { __syncthreads(); });
            if (warp == 0) {
                const int32_t token = locate_in_segments<DT, true>(sr, in.V, (double)sh.u[K], seg, nseg, lane);
                if (lane == 0) sh.token = token;
            }
            __syncthreads();
        }
        if (tid == 0 && sh.token < 0) sh.token = (int32_t)(in.V - 1);     // a row without any mass (all logits -inf)
        __syncthreads();
        const int32_t token = sh.token;
        for (int64_t i = tid; t0 + i < slot_end; i += kClusterThreads)
            emitted[t0 + i] = (i < n) ? sh.tok[i] : (i == n ? token : -1);
        if (tid == 0) {
            accepted_len[b] = n;
            if (row_status) row_status[b] = status;
            if (next.out) next.out[b] = next_lookahead_of(kb_raw, n, next.k_min, next.k_max);
        }
    }
    cluster_barrier();            // nobody's shared memory goes away while CTA 0 may still read it
}

}  // namespace specv
