// Tree-structured verification: the draft proposes a tree of candidate tokens per sequence
// (several candidates for the same position), the target scores every node in one pass, and
// the verifier walks from the root, trying the children of the current context one after the
// other (recursive rejection sampling; rule and layout in include/spec_verify.h).  A chain is
// the special case the other kernels handle.
//
//   specv_prologue      (shared) offsets over the node counts, per-sequence checks, -1 fill
//   specv_tree_plan     per sequence: parent indices checked, contexts that have children marked
//                       (only their draft rows are read), accepted_nodes filled with -1
//   row statistics      the streaming or the ring statistics kernel, unchanged: (reference, sum)
//                       of every target row and of every draft row that is needed
//   specv_tree_resolve  one block, or a cluster of two, per sequence: probabilities of every node's
//                       token under its parent's context (all nodes in parallel), then the walk; each
//                       rejected child costs one more pass over the context's row pair
//
// With r = p_c at a fresh context, k rejected children leave r proportional to
// max(0, p_c - coef_k q_c), coef_0 = 0, coef_{k+1} = coef_k + norm_k, where norm_k is the sum of
// max(0, p_c - coef_k q_c) over the vocabulary (norm_0 = 1).  Child k+1 with token x is accepted
// iff u q_c(x) norm_k < max(0, p_c(x) - coef_k q_c(x)).  The walk keeps (coef, norm) instead of
// a vocabulary-sized vector; a pass with the next coefficient yields the next norm and, in the
// same sweep, the segment sums the final inverse-CDF draw needs.
#pragma once

#include "specv_stream_kernels.cuh"

namespace specv {

constexpr int kTreePlanThreads = 256;

__global__ void __launch_bounds__(kTreePlanThreads)
specv_tree_plan(BatchView in, const int32_t* __restrict__ off_d, int32_t* __restrict__ seq_status,
                int32_t* __restrict__ has_children, int32_t* __restrict__ accepted_nodes) {
    __shared__ int bad_parent;
    const int tid = threadIdx.x;
    const int32_t b = blockIdx.x;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (accepted_nodes) {
        const int64_t n_slots = in.n_draft_total + in.B;
        for (int64_t s = (int64_t)b * kTreePlanThreads + tid; s < n_slots; s += (int64_t)gridDim.x * kTreePlanThreads)
            accepted_nodes[s] = -1;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");      // offsets and status come from the prologue
    const int32_t n_raw = in.k_per_row ? in.k_per_row[b] : in.k_uniform;
    const int32_t N = n_raw > 0 ? n_raw : 0;
    const int64_t d0 = off_d[b];
    if (seq_status[b] & 1) return;     // the sequence's rows overrun the buffers: nothing of it is touched
    if (tid == 0) bad_parent = 0;
    for (int32_t j = tid; j < N; j += kTreePlanThreads) has_children[d0 + j] = 0;
    __syncthreads();
    for (int32_t j = tid; j < N; j += kTreePlanThreads) {
        const int32_t par = in.parent[d0 + j];
        if (par < -1 || par >= j) bad_parent = 1;
        else has_children[d0 + par + 1] = 1;               // context par+1 <= j < N
    }
    __syncthreads();
    if (tid == 0 && bad_parent) seq_status[b] |= 32;       // SPECV_ROW_BAD_PARENT
}

constexpr int kTreeThreads = 512;
constexpr int kTreeWarps = kTreeThreads / 32;
constexpr int kTreeCachedNodes = 1024;   // nodes whose token probabilities are kept in shared memory for the walk
constexpr int kTreeCachedCtx = 1024;     // contexts whose row normalisations are kept in shared memory
constexpr size_t kTreeCacheBytes = (size_t)kTreeCachedNodes * (2 * sizeof(double) + sizeof(float) + sizeof(int32_t)) +
                                   (size_t)kTreeCachedCtx * (2 * sizeof(double) + 2 * sizeof(float));

struct TreeWalk {          // block-wide state of the walk, written by warp 0 between barriers
    int32_t ctx;           // current context: 0 root, j+1 after node j
    int32_t n;             // accepted nodes so far
    int32_t cursor;        // smallest node index not yet examined as a child of ctx
    int32_t child;         // child under test, -1: none left
    int32_t accept;
    int32_t seg_valid;     // seg[] holds the segment sums of (ctx, coef)
    int32_t status;
    double coef, norm;     // r proportional to max(0, p - coef q), norm = its sum
    double cand;           // coefficient of the pass in flight
    double p_sum;          // the segment sums of the pass in flight are in units of 1 / p_sum
};

// CS CTAs (a thread-block cluster when CS > 1) per sequence.  A rejected child costs one pass over the
// context's row pair, and the passes of one walk depend on one another, so the time of the kernel is
// the longest chain of passes times the time of one pass -- which one SM's load bandwidth bounds.
// With CS = 2 each CTA sums half of the segments and writes its sums into the seg[] arrays of both
// CTAs through distributed shared memory; a cluster barrier replaces the block barrier after a pass.
// Everything else (node probabilities, the walk's state, the decisions) is computed redundantly and
// identically by every CTA of the cluster from the same inputs, so the CTAs never exchange anything
// but segment sums and always take the same branches; the CTA of rank 0 writes the results.
template <int DT, int CS>
__global__ void __launch_bounds__(kTreeThreads)
specv_tree_resolve(BatchView in, const int32_t* __restrict__ off_d, const int32_t* __restrict__ seq_status,
                   const float2* __restrict__ stat_t, const float2* __restrict__ stat_d, int splits,
                   const int32_t* __restrict__ error_word,
                   int32_t* __restrict__ accepted_len, int32_t* __restrict__ emitted,
                   int32_t* __restrict__ accepted_nodes, int32_t* __restrict__ row_status,
                   float* __restrict__ diag_p, float* __restrict__ diag_q) {
    using E = Elt<DT>;
    constexpr int SEG = 32 * E::kPerVec;
    extern __shared__ __align__(16) unsigned char tree_smem[];
    // per-node and per-context caches (what the walk needs of a node without touching memory), then
    // the two buffers of segment sums
    double* const node_p = reinterpret_cast<double*>(tree_smem);
    double* const node_q = node_p + kTreeCachedNodes;
    double* const ctx_sum_p = node_q + kTreeCachedNodes;
    double* const ctx_sum_q = ctx_sum_p + kTreeCachedCtx;
    float* const ctx_ref_p = reinterpret_cast<float*>(ctx_sum_q + kTreeCachedCtx);
    float* const ctx_ref_q = ctx_ref_p + kTreeCachedCtx;
    float* const node_u = ctx_ref_q + kTreeCachedCtx;
    int32_t* const node_par = reinterpret_cast<int32_t*>(node_u + kTreeCachedNodes);
    float* const seg = reinterpret_cast<float*>(node_par + kTreeCachedNodes);
    __shared__ TreeWalk w;
    __shared__ SampleRows rows;
    __shared__ int32_t bad_token;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t rank = 0;
    if (CS > 1) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int32_t b = blockIdx.x / CS;
    const bool writer = rank == 0;
    asm volatile("griddepcontrol.wait;" ::: "memory");   // all row statistics must be in memory
    const int64_t d0 = off_d[b];
    const int64_t t0 = d0 + b;
    const int err = error_word ? error_word[0] : 0;
    int status = seq_status[b] | (err ? (16 | (err << 8)) : 0);
    const int32_t n_raw = in.k_per_row ? in.k_per_row[b] : in.k_uniform;
    const int32_t N = n_raw > 0 ? n_raw : 0;
    const int32_t nseg = (int32_t)((in.V + SEG - 1) / SEG);

    if (tid == 0) bad_token = 0;
    __syncthreads();
    if (!(status & 1)) {
        for (int32_t j = tid; j < N; j += kTreeThreads) {
            const int32_t x = in.tokens[d0 + j];
            if (x < 0 || (int64_t)x >= in.V) bad_token = 1;
        }
    }
    __syncthreads();
    if (bad_token) status |= 4;   // SPECV_ROW_BAD_TOKEN
    if (status) {                 // the same in every CTA of the cluster: no barrier is left behind
        if (tid == 0 && writer) {
            accepted_len[b] = 0;
            if (row_status) row_status[b] = status;
        }
        return;   // emitted tokens and accepted nodes are already -1
    }

    const float T = in.temperature[in.per_row_temperature ? b : 0];
    const float cf = (float)(kLog2e / (double)T);
    const double cd = (double)cf;

    // probability of a token under context ctx, target and draft, from the streamed statistics
    auto prob_p = [&](int32_t ctx, int32_t x, const RowNorm& np) {
        return exp2((double)E::load1(in.target + (t0 + ctx) * in.pitch_t, x) * cd - (double)np.ref) / np.sum;
    };
    auto prob_q = [&](int32_t ctx, int32_t x, const RowNorm& nq) {
        return exp2((double)E::load1(in.draft + (d0 + ctx) * in.pitch_d, x) * cd - (double)nq.ref) / nq.sum;
    };

    // The rows of a context are asked for from L2 as soon as the walk can reach it: the statistics pass
    // has streamed far more than L2 holds, so a pass over rows that were not asked for ahead pays the
    // HBM latency once per wave of loads.  Warp 1 of the writing CTA, sixteen lanes, one chunk each.
    const int64_t row_bytes = in.V * E::kBytes;
    const bool can_prefetch = (row_bytes & 15) == 0;
    auto prefetch_ctx = [&](int32_t ctx) {
        if (!writer || !can_prefetch || lane >= 16) return;
        const bool is_q = lane >= 8;
        if (is_q && !(ctx < N && in.ctx_has_children[d0 + ctx])) return;      // a draft row exists for contexts with children
        const char* row = is_q ? in.draft + (d0 + ctx) * in.pitch_d : in.target + (t0 + ctx) * in.pitch_t;
        if (reinterpret_cast<uintptr_t>(row) & 15u) return;
        const int64_t chunk = ((row_bytes + 7) / 8 + 15) & ~(int64_t)15;
        const int64_t at = (int64_t)(lane & 7) * chunk;
        const int64_t n = row_bytes - at < chunk ? row_bytes - at : chunk;
        if (n > 0) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(row + at), "r"((uint32_t)n) : "memory");
    };
    if (warp == 1) prefetch_ctx(0);

    // every node's token under its parent's context, all nodes in parallel: kept for the walk
    // (which then takes a step without touching memory) and reported as diagnostics; the
    // normalisations of the parent's rows are kept too, for the passes over them
    {
        const int32_t n_cached = N < kTreeCachedNodes ? N : kTreeCachedNodes;
        const int32_t n_wanted = (diag_p || diag_q) ? N : n_cached;
        for (int32_t j = warp; j < n_wanted; j += kTreeWarps) {
            // every lane loads the same words: the logits of the token are on their way while the
            // row statistics are merged
            const int32_t par = in.parent[d0 + j], ctx = par + 1;
            const int32_t x = in.tokens[d0 + j];
            const double lp = (double)E::load1(in.target + (t0 + ctx) * in.pitch_t, x);
            const double lq = (double)E::load1(in.draft + (d0 + ctx) * in.pitch_d, x);
            const float u = in.uniforms[t0 + j];
            const RowNorm np = warp_merge_splits(stat_t, t0 + ctx, splits, lane);
            const RowNorm nq = warp_merge_splits(stat_d, d0 + ctx, splits, lane);
            if (lane == 0) {
                const double p = exp2(lp * cd - (double)np.ref) / np.sum, q = exp2(lq * cd - (double)nq.ref) / nq.sum;
                if (j < n_cached) { node_p[j] = p; node_q[j] = q; node_u[j] = u; node_par[j] = par; }
                if (ctx < kTreeCachedCtx) {       // siblings write the same values
                    ctx_ref_p[ctx] = np.ref; ctx_sum_p[ctx] = np.sum;
                    ctx_ref_q[ctx] = nq.ref; ctx_sum_q[ctx] = nq.sum;
                }
                if (diag_p && writer) diag_p[d0 + j] = (float)p;
                if (diag_q && writer) diag_q[d0 + j] = (float)q;
            }
        }
    }

    if (tid == 0) {
        w.ctx = 0; w.n = 0; w.cursor = 0; w.child = -1; w.accept = 0; w.seg_valid = 0; w.status = 0;
        w.coef = 0.0; w.norm = 1.0; w.cand = 0.0;
    }
    __syncthreads();

    // rows of context ctx with coefficient coef, for the mass routines: the coefficient is folded
    // into the draft row's normalisation, max(0, p_j - coef q_j).  `cached`: the context has children
    // among the cached nodes, so its normalisations are in shared memory.
    auto set_rows = [&](int32_t ctx, double coef, bool cached) {       // warp 0, all lanes
        RowNorm np, nq{0.f, 1.0};
        if (cached) {
            np = RowNorm{ctx_ref_p[ctx], ctx_sum_p[ctx]};
            nq = RowNorm{ctx_ref_q[ctx], ctx_sum_q[ctx]};
        } else {
            np = warp_merge_splits(stat_t, t0 + ctx, splits, lane);
            if (coef > 0.0) nq = warp_merge_splits(stat_d, d0 + ctx, splits, lane);
        }
        if (lane == 0) {
            rows.p = in.target + (t0 + ctx) * in.pitch_t;
            rows.p_aligned = (reinterpret_cast<uintptr_t>(rows.p) & 15u) == 0;
            rows.c = cf;
            rows.p_ref = np.ref;
            w.p_sum = np.sum;
            rows.q = nullptr; rows.q_aligned = false; rows.q_ref = 0.f; rows.kappa = 0.f;
            if (coef > 0.0) {
                rows.q = in.draft + (d0 + ctx) * in.pitch_d;
                rows.q_aligned = (reinterpret_cast<uintptr_t>(rows.q) & 15u) == 0;
                rows.q_ref = nq.ref;
                rows.kappa = (float)(coef * np.sum / nq.sum);
            }
        }
    };

    // one pass: the segment sums of the distribution `rows` describes, complete in the seg buffer of
    // every CTA of the cluster when it returns.  Two buffers, used in turn: a CTA that is already
    // in the next pass writes the other buffer, not the one its peer may still be summing up.
    const int32_t seg_stride = (nseg + 3) & ~3;
    int pb = CS > 1 ? 1 : 0;   // a single CTA has one buffer
    uint32_t seg_peer = 0;
    if (CS > 1) {
        const uint32_t mine = static_cast<uint32_t>(__cvta_generic_to_shared(seg));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(seg_peer) : "r"(mine), "r"(rank ^ 1u));
    }
    auto sync_pass = [] {
        if (CS > 1) asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        else __syncthreads();
    };
    const bool vec_rows = (in.V % E::kPerVec) == 0;
    auto pass = [&] {          // every thread of every CTA of the cluster, the same number of times
        if (CS > 1) pb ^= 1;
        float* const sg = seg + pb * seg_stride;
        const uint32_t sg_peer = seg_peer + 4u * (uint32_t)(pb * seg_stride);
        auto store_seg = [&](int32_t s, float a) {
            sg[s] = a;
            if (CS > 1) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(sg_peer + 4u * (uint32_t)s), "f"(a) : "memory");
        };
        const SampleRows sr = rows;
        if (vec_rows && sr.p_aligned && (!sr.q || sr.q_aligned))
            block_segment_sums_to<DT, kTreeWarps * CS, true>(sr, in.V, (int)rank * kTreeWarps + warp, store_seg, sync_pass);
        else
            block_segment_sums_to<DT, kTreeWarps * CS, false>(sr, in.V, (int)rank * kTreeWarps + warp, store_seg, sync_pass);
    };

    for (;;) {
        if (warp == 0) {
            // next child of the current context
            const int32_t ctx = w.ctx;
            int32_t child = -1;
            for (int32_t base = w.cursor; base < N && child < 0; base += 32) {
                const int32_t j = base + lane;
                const unsigned m = __ballot_sync(
                    0xffffffffu, j < N && (j < kTreeCachedNodes ? node_par[j] : in.parent[d0 + j]) == ctx - 1);
                if (m) child = base + __ffs(m) - 1;
            }
            int accept = 0;
            if (child >= 0) {
                double p, q, u;
                if (child < kTreeCachedNodes) {
                    p = node_p[child]; q = node_q[child]; u = (double)node_u[child];
                } else {
                    const RowNorm np = warp_merge_splits(stat_t, t0 + ctx, splits, lane);
                    const RowNorm nq = warp_merge_splits(stat_d, d0 + ctx, splits, lane);
                    const int32_t x = in.tokens[d0 + child];
                    p = prob_p(ctx, x, np); q = prob_q(ctx, x, nq);
                    u = (double)in.uniforms[t0 + child];
                }
                const double a = fmax(p - w.coef * q, 0.0);
                accept = u * q * w.norm < a;
            }
            __syncwarp();
            if (lane == 0) { w.child = child; w.accept = accept; }
        }
        __syncthreads();
        const int32_t child = w.child;
        if (child < 0) break;
        if (w.accept) {
            __syncthreads();       // everyone has read w.child / w.accept
            if (tid == 0) {
                if (writer) {
                    emitted[t0 + w.n] = in.tokens[d0 + child];
                    if (accepted_nodes) accepted_nodes[t0 + w.n] = child;
                }
                w.n += 1;
                w.ctx = child + 1; w.cursor = child + 1;      // children of node j have larger indices
                w.seg_valid = 0; w.coef = 0.0; w.norm = 1.0;
            }
            if (warp == 1) prefetch_ctx(child + 1);
            __syncthreads();
            continue;
        }
        // rejected: one pass over the context's rows with the next coefficient
        if (warp == 0) {
            const double cand = w.coef + w.norm;
            set_rows(w.ctx, cand, child < kTreeCachedNodes && w.ctx < kTreeCachedCtx);
            if (lane == 0) w.cand = cand;
        }
        __syncthreads();
        pass();
        if (warp == 0) {
            const double total = warp_segment_total(seg + pb * seg_stride, nseg, lane) / w.p_sum;
            if (lane == 0) {
                if (total > 0.0) { w.coef = w.cand; w.norm = total; w.seg_valid = 1; }
                else { w.status |= 8; w.seg_valid = 0; }      // SPECV_ROW_ZERO_RESIDUAL: r stays as it was
                w.cursor = child + 1;
            }
        }
        __syncthreads();
    }

    // no child accepted (or none exists): draw from r = max(0, p - coef q) / norm
    if (!w.seg_valid) {            // the same in every CTA of the cluster
        __syncthreads();
        if (warp == 0) set_rows(w.ctx, w.coef, false);
        __syncthreads();
        pass();
    }
    if (warp == 0 && writer) {
        const SampleRows sr = rows;
        int32_t token = locate_in_segments<DT, false>(sr, in.V, (double)in.uniforms[t0 + N], seg + pb * seg_stride, nseg, lane);
        if (token < 0) token = (int32_t)(in.V - 1);   // a row without any mass (all logits -inf)
        if (lane == 0) {
            emitted[t0 + w.n] = token;
            accepted_len[b] = w.n;
            if (row_status) row_status[b] = w.status;
        }
    }
}

}  // namespace specv
