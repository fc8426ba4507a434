// Host side of the C ABI declared in include/spec_verify.h: argument validation,
// workspace layout, kernel launches.  No device memory is allocated here.
#include "../../include/spec_verify.h"

#include <atomic>
#include <cstring>
#include <mutex>

#include "specv_cluster_kernels.cuh"
#include "specv_greedy_kernels.cuh"
#include "specv_lmhead_kernel.cuh"
#include "specv_ring_kernels.cuh"
#include "specv_stream_kernels.cuh"
#include "specv_tree_kernels.cuh"

namespace {

thread_local int g_last_cuda_error = 0;
thread_local cudaEvent_t g_trace[4] = {nullptr, nullptr, nullptr, nullptr};
thread_local bool g_trace_on = false;
thread_local int g_last_path = 0;
std::atomic<uint64_t> g_launches{0};

constexpr int64_t kMaxV = int64_t(1) << 22;          // segment table of the sampler must fit in shared memory
constexpr int kMaxSplits = 32;
constexpr int kMaxDevices = 64;

struct DeviceInfo {
    int state = 0;        // 0 unknown, 1 usable, -1 wrong architecture
    int sms = 0;
    int stats_blocks_per_sm[3] = {0, 0, 0};   // per dtype
    int ring_ready[3] = {0, 0, 0};
    int argmax_blocks_per_sm[3] = {0, 0, 0};
    int ring_argmax_ready[3] = {0, 0, 0};
    int tree_ready[3] = {0, 0, 0};
    int lm_head_ready = 0;
    int cluster_ready[3] = {0, 0, 0};
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;   // guards the lazy per-device set-up (first call on a device from any thread)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool cuda_ok(cudaError_t e) {
    if (e == cudaSuccess) return true;
    g_last_cuda_error = (int)e;
    return false;
}

// Splits per logits row for the statistics pass: enough (row, split) items to fill the
// machine when the batch has few rows.  A function of the shape only, so that the
// workspace size can be computed without a device.
int splits_for(int64_t n_rows, int64_t V) {
    constexpr int64_t kWantedItems = 148 * 8;
    int64_t s = (kWantedItems + n_rows - 1) / n_rows;
    const int64_t by_len = V / 2048 > 0 ? V / 2048 : 1;
    if (s > by_len) s = by_len;
    if (s > kMaxSplits) s = kMaxSplits;
    if (s < 1) s = 1;
    return (int)s;
}

bool shape_ok(int32_t B, int64_t n_draft_total, int64_t V) {
    if (B < 1 || V < 1 || V > kMaxV || n_draft_total < 0) return false;
    if (n_draft_total + (int64_t)B > (int64_t)0x7fffffff - 1) return false;
    return true;
}

struct Workspace {
    size_t off_d, seq_status, partial, total;
};
Workspace workspace_layout(int32_t B, int64_t n_draft_total, int64_t V) {
    const int64_t n_rows = 2 * n_draft_total + B;
    Workspace w;
    size_t o = 0;
    w.off_d = o;       o = align_up(o + sizeof(int32_t) * ((size_t)B + 1), 256);
    w.seq_status = o;  o = align_up(o + sizeof(int32_t) * (size_t)B, 256);
    w.partial = o;     o = align_up(o + sizeof(float2) * (size_t)n_rows * splits_for(n_rows, V), 256);
    w.total = o;
    return w;
}

// Scratch of the ring kernel set, placed after the streaming one (offsets and per-sequence
// status are shared with it).
struct RingLayout {
    size_t stat_p, stat_q, done, gseg, item_seq, item_pos, level_start, first_rej, ctrl, total;
};
// Segments (512 bytes of a logits row each) per row, for the widest element type: the workspace
// size does not depend on the dtype.  0: the ring kernels do not take the shape.
int64_t ring_segments(int32_t B, int64_t V) {
    if (B > specv::kMaxRingSeqs || (V * 2 + 511) / 512 > specv::kMaxSegs) return 0;
    return (V * 4 + 511) / 512;
}
RingLayout ring_layout(size_t base, int32_t B, int64_t D, int64_t V) {
    RingLayout f;
    size_t o = base;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const bool ring = ring_segments(B, V) > 0;
    f.stat_p = take(sizeof(float2) * (size_t)(D + B) * specv::kStatParts);
    f.stat_q = take(sizeof(float2) * (size_t)D * specv::kStatParts);
    f.done = take(ring ? 4 * (size_t)B : 0);
    f.gseg = take(sizeof(float) * (size_t)B * (size_t)ring_segments(B, V));
    f.item_seq = take(4 * (size_t)(D + B));
    f.item_pos = take(4 * (size_t)(D + B));
    f.level_start = take(4 * (size_t)(D + 2));
    f.first_rej = take(4 * (size_t)B);
    f.ctrl = take(64);
    f.total = o;
    return f;
}

// Whether a batch can take the ring kernels: bulk copies need every logits row to start on a
// 16-byte boundary and to be a whole number of 16-byte vectors, and the sampler keeps one
// float per 32-vector segment in shared memory.
bool ring_shape_ok(const specv::BatchView& in, int dtype) {
    const int64_t elt = dtype == SPECV_F32 ? 4 : 2;
    const int64_t seg = 32 * (16 / elt);
    if (in.B > specv::kMaxRingSeqs) return false;       // the kernels keep B + 1 offsets in shared memory
    if ((reinterpret_cast<uintptr_t>(in.target) & 15u) || (in.pitch_t & 15) || ((in.V * elt) & 15)) return false;
    if (in.n_draft_total > 0 && ((reinterpret_cast<uintptr_t>(in.draft) & 15u) || (in.pitch_d & 15))) return false;
    return (in.V + seg - 1) / seg <= specv::kMaxSegs;
}

// Lazy per-device set-up of the ring kernels (large dynamic shared memory).
template <int DT>
bool ensure_ring_ready(DeviceInfo& dev) {
    using namespace specv;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!dev.ring_ready[DT]) {
        if (!cuda_ok(cudaFuncSetAttribute(specv_ring_stats<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(RingStatsShared))) ||
            !cuda_ok(cudaFuncSetAttribute(specv_ring_resolve<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(RingResolveShared))) ||
            !cuda_ok(cudaFuncSetAttribute(specv_ring_stats_early<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(RingEarlyShared))))
            return false;
        dev.ring_ready[DT] = 1;
    }
    return true;
}

// Lazy per-device set-up of the streaming kernels.
template <int DT>
bool ensure_stream_ready(DeviceInfo& dev) {
    using namespace specv;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (dev.stats_blocks_per_sm[DT] == 0) {
        int per_sm = 0;
        if (!cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, specv_row_stats<DT>, kStatsThreads, 0)))
            return false;
        if (!cuda_ok(cudaFuncSetAttribute(specv_resolve<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024)))
            return false;
        dev.stats_blocks_per_sm[DT] = per_sm > 0 ? per_sm : 1;
    }
    return true;
}

template <int DT>
int launch_ring_path(const specv::BatchView& in, const Workspace& lay, const RingLayout& rl, char* ws,
                     DeviceInfo& dev, int32_t* accepted_len, int32_t* emitted, int32_t* row_status,
                     float* diag_p, float* diag_q, bool early, specv::NextLookahead next, cudaStream_t stream) {
    using namespace specv;
    const size_t smem_stats = sizeof(RingStatsShared), smem_resolve = sizeof(RingResolveShared);
    const size_t smem_early = sizeof(RingEarlyShared);
    if (!ensure_ring_ready<DT>(dev)) return SPECV_ERR_CUDA;
    RingScratch sc;
    sc.off_d = reinterpret_cast<int32_t*>(ws + lay.off_d);
    sc.seq_status = reinterpret_cast<int32_t*>(ws + lay.seq_status);
    sc.stat_p = reinterpret_cast<float2*>(ws + rl.stat_p);
    sc.stat_q = reinterpret_cast<float2*>(ws + rl.stat_q);
    sc.done = reinterpret_cast<int32_t*>(ws + rl.done);
    sc.gseg = reinterpret_cast<float*>(ws + rl.gseg);
    sc.ctrl = reinterpret_cast<int32_t*>(ws + rl.ctrl);
    sc.item_seq = reinterpret_cast<int32_t*>(ws + rl.item_seq);
    sc.item_pos = reinterpret_cast<int32_t*>(ws + rl.item_pos);
    sc.level_start = reinterpret_cast<int32_t*>(ws + rl.level_start);
    sc.first_rej = reinterpret_cast<int32_t*>(ws + rl.first_rej);

    auto trace = [&](int i) { if (g_trace_on) cudaEventRecord(g_trace[i], stream); };
    const int64_t n_slots = in.n_draft_total + in.B;
    const int64_t nck = (in.V * (int64_t)Elt<DT>::kBytes + kChunkBytes - 1) / kChunkBytes;
    // the kernels after the first are launched with programmatic stream serialization: their CTAs
    // may be scheduled while the previous kernel drains, and wait inside for its completion
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    trace(0);
    if (early) {
        // prologue, position-major work list (one block), then the statistics kernel that consults it
        int pro_blocks = (int)((n_slots + 8 * kPrologueThreads - 1) / (8 * kPrologueThreads));
        if (pro_blocks < 1) pro_blocks = 1;
        if (pro_blocks > dev.sms) pro_blocks = dev.sms;
        specv_prologue<<<pro_blocks, kPrologueThreads, 0, stream>>>(in, sc.off_d, sc.seq_status, emitted, sc.ctrl,
                                                                      sc.done, 0);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;
        trace(1);
        cfg.attrs = pdl;
        cfg.numAttrs = 1;
        cfg.gridDim = dim3(1, 1, 1);
        cfg.blockDim = dim3(kPlanThreads, 1, 1);
        cfg.dynamicSmemBytes = 0;
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_plan_levels, in, sc))) return SPECV_ERR_CUDA;
        g_launches.fetch_add(1, std::memory_order_relaxed);
        cfg.gridDim = dim3((unsigned)(n_slots < dev.sms ? n_slots : dev.sms), 1, 1);
        cfg.blockDim = dim3(kRingStatsThreads, 1, 1);
        cfg.dynamicSmemBytes = smem_early;
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_ring_stats_early<DT>, in, sc))) return SPECV_ERR_CUDA;
    } else {
        // the statistics kernel is the first of the pass: it does the prologue's per-sequence work
        // itself.  One persistent CTA per SM; a CTA whose share of the units is empty ends at once.
        trace(1);
        cfg.attrs = nullptr;
        cfg.numAttrs = 0;
        cfg.gridDim = dim3((unsigned)dev.sms, 1, 1);
        cfg.blockDim = dim3(kRingStatsThreads, 1, 1);
        cfg.dynamicSmemBytes = smem_stats;
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_ring_stats<DT>, in, sc, 1))) return SPECV_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    cfg.attrs = pdl;
    cfg.numAttrs = 1;

    trace(2);
    const int64_t max_units = (int64_t)in.B * nck;
    const int resolve_ctas = (int)(max_units < dev.sms ? max_units : dev.sms);
    cfg.gridDim = dim3((unsigned)resolve_ctas, 1, 1);
    cfg.blockDim = dim3(kRingResolveThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_resolve;
    if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_ring_resolve<DT>, in, sc, accepted_len, emitted, row_status, diag_p,
                                    diag_q, next)))
        return SPECV_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    trace(3);
    return SPECV_OK;
}

template <int DT>
int launch_stream_path(const specv::BatchView& in, const Workspace& lay, char* ws, DeviceInfo& dev,
                       int32_t* accepted_len, int32_t* emitted, int32_t* row_status,
                       float* diag_p, float* diag_q, specv::NextLookahead next, cudaStream_t stream) {
    using namespace specv;
    int32_t* off_d = reinterpret_cast<int32_t*>(ws + lay.off_d);
    int32_t* seq_status = reinterpret_cast<int32_t*>(ws + lay.seq_status);
    float2* partial = reinterpret_cast<float2*>(ws + lay.partial);
    const int64_t n_target = in.n_draft_total + in.B;
    const int64_t n_rows = n_target + in.n_draft_total;
    const int splits = splits_for(n_rows, in.V);

    auto trace = [&](int i) { if (g_trace_on) cudaEventRecord(g_trace[i], stream); };
    const int64_t n_slots = n_target;
    trace(0);
    int pro_blocks = (int)((n_slots + 8 * kPrologueThreads - 1) / (8 * kPrologueThreads));
    if (pro_blocks < 1) pro_blocks = 1;
    if (pro_blocks > dev.sms) pro_blocks = dev.sms;
    specv_prologue<<<pro_blocks, kPrologueThreads, 0, stream>>>(in, off_d, seq_status, emitted, nullptr, nullptr, 0);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;

    if (!ensure_stream_ready<DT>(dev)) return SPECV_ERR_CUDA;
    trace(1);
    const int64_t n_items = n_rows * splits;
    int64_t stats_blocks = (int64_t)dev.sms * dev.stats_blocks_per_sm[DT];
    if (stats_blocks > n_items) stats_blocks = n_items;
    // the two dependent kernels are launched with programmatic stream serialization: their blocks
    // may be scheduled while the previous kernel drains, and wait inside for its completion
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)stats_blocks, 1, 1);
    cfg.blockDim = dim3(kStatsThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    const int32_t* off_d_c = off_d;
    if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_row_stats<DT>, in, off_d_c, n_target, n_rows, splits, partial)))
        return SPECV_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);

    trace(2);
    const int seg_elems = 32 * Elt<DT>::kPerVec;
    const size_t seg_bytes = sizeof(float) * (size_t)((in.V + seg_elems - 1) / seg_elems);
    cfg.gridDim = dim3((unsigned)in.B, 1, 1);
    cfg.blockDim = dim3(kResolveThreads, 1, 1);
    cfg.dynamicSmemBytes = seg_bytes;
    const int32_t* seq_status_c = seq_status;
    const float2* partial_c = partial;
    if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_resolve<DT>, in, off_d_c, seq_status_c, partial_c, splits, n_target,
                                    accepted_len, emitted, row_status, diag_p, diag_q, next)))
        return SPECV_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    trace(3);
    return SPECV_OK;
}

int device_info(DeviceInfo** out) {
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return SPECV_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return SPECV_ERR_ARCH;
    DeviceInfo& d = g_dev[dev];
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (d.state == 0) {
        int major = 0, sms = 0;
        if (!cuda_ok(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev))) return SPECV_ERR_CUDA;
        if (!cuda_ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return SPECV_ERR_CUDA;
        d.sms = sms;
        d.state = (major == 10) ? 1 : -1;
    }
    if (d.state < 0) return SPECV_ERR_ARCH;
    *out = &d;
    return SPECV_OK;
}

int validate(const void* target_logits, const void* draft_logits, int dtype, int64_t V, int64_t ld_target,
             int64_t ld_draft, const int32_t* draft_tokens, const int32_t* k_per_row, int32_t B,
             int32_t k_uniform, int64_t n_draft_total, const float* temperature, const float* uniforms,
             const int32_t* accepted_len, const int32_t* emitted_tokens) {
    if (dtype != SPECV_F32 && dtype != SPECV_BF16 && dtype != SPECV_F16) return SPECV_ERR_DTYPE;
    if (!shape_ok(B, n_draft_total, V) || ld_target < V || ld_draft < V) return SPECV_ERR_SHAPE;
    if (!k_per_row && (k_uniform < 0 || (int64_t)B * k_uniform != n_draft_total)) return SPECV_ERR_SHAPE;
    if (!target_logits || !temperature || !uniforms || !accepted_len || !emitted_tokens) return SPECV_ERR_NULL;
    if (n_draft_total > 0 && (!draft_logits || !draft_tokens)) return SPECV_ERR_NULL;
    return SPECV_OK;
}

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" {

const char* spec_verify_strerror(int status) {
    switch (status) {
        case SPECV_OK: return "success";
        case SPECV_ERR_NULL: return "a required pointer is NULL";
        case SPECV_ERR_SHAPE: return "B, V, leading dimension, k_uniform or n_draft_total out of range";
        case SPECV_ERR_DTYPE: return "dtype is not a specv_dtype";
        case SPECV_ERR_ALIGN: return "a pointer is not aligned as required";
        case SPECV_ERR_WORKSPACE: return "workspace or arena too small";
        case SPECV_ERR_CUDA: return "a CUDA call failed (see spec_verify_last_cuda_error)";
        case SPECV_ERR_ARCH: return "the current device is not compute capability 10.x";
        case SPECV_ERR_TOO_LARGE:
            return "the batch needs more scratch than the built-in buffer of spec_verify_noalloc holds";
        case SPECV_ERR_FLAGS: return "unknown flag bits, both kernel-set flags, or a flag this call does not take";
        default: return "unknown status";
    }
}

int spec_verify_last_cuda_error(void) { return g_last_cuda_error; }

int spec_verify_set_trace_events(void* const* events) {
    g_trace_on = events != nullptr;
    for (int i = 0; i < 4; ++i) g_trace[i] = events ? static_cast<cudaEvent_t>(events[i]) : nullptr;
    return SPECV_OK;
}

uint64_t spec_verify_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t spec_verify_workspace_bytes(int32_t B, int64_t n_draft_total, int64_t V) {
    if (!shape_ok(B, n_draft_total, V)) return 0;
    return ring_layout(workspace_layout(B, n_draft_total, V).total, B, n_draft_total, V).total;
}

int spec_verify_next_lookahead(const int32_t* k_per_row, int32_t k_uniform, const int32_t* accepted_len,
                               int32_t B, int32_t k_min, int32_t k_max, int32_t* next_k, void* cuda_stream) {
    if (!accepted_len || !next_k) return SPECV_ERR_NULL;
    if (B < 1 || k_min < 0 || k_max < k_min || (!k_per_row && k_uniform < 0)) return SPECV_ERR_SHAPE;
    specv::specv_next_lookahead<<<(B + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        k_per_row, k_uniform, accepted_len, B, k_min, k_max, next_k);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cuda_ok(cudaGetLastError()) ? SPECV_OK : SPECV_ERR_CUDA;
}

int spec_verify_last_path(void) { return g_last_path; }

}  // extern "C"

namespace {

constexpr uint32_t kKnownFlags = SPECV_FLAG_STREAMING | SPECV_FLAG_RING | SPECV_FLAG_EARLY_EXIT | SPECV_FLAG_CLUSTER;
bool flags_ok(uint32_t flags) {
    const uint32_t set = flags & (SPECV_FLAG_STREAMING | SPECV_FLAG_RING | SPECV_FLAG_CLUSTER);
    return !(flags & ~kKnownFlags) && !(set & (set - 1));       // at most one kernel set
}

// The one-launch form for small batches (specv_cluster_kernels.cuh): a cluster of eight CTAs per
// sequence must hold every row of the sequence in shared memory.  The host knows the lookahead only
// when it is uniform; for a ragged batch the number of draft rows bounds it.
constexpr size_t kClusterSmemLimit = 200 * 1024;
struct ClusterPlan {
    bool ok = false;
    int32_t slice_bytes = 0;
    size_t smem = 0;
};
ClusterPlan cluster_plan(const specv::BatchView& in, int dtype, uint32_t flags) {
    ClusterPlan p;
    if (flags & (SPECV_FLAG_STREAMING | SPECV_FLAG_RING | SPECV_FLAG_EARLY_EXIT)) return p;
    const int64_t elt = dtype == SPECV_F32 ? 4 : 2;
    if (in.B > specv::kClusterMaxSeqs) return p;
    if ((reinterpret_cast<uintptr_t>(in.target) & 15u) || (in.pitch_t & 15) || ((in.V * elt) & 15)) return p;
    if (in.n_draft_total > 0 && ((reinterpret_cast<uintptr_t>(in.draft) & 15u) || (in.pitch_d & 15))) return p;
    const int64_t k_bound = in.k_per_row ? in.n_draft_total : (in.k_uniform > 0 ? in.k_uniform : 0);
    if (k_bound > specv::kClusterMaxK) return p;
    const int64_t row_bytes = in.V * elt;
    const int64_t nseg = (row_bytes + 511) / 512;
    const int64_t slice = ((nseg + specv::kClusterCtas - 1) / specv::kClusterCtas) * 512;
    const size_t smem = (size_t)(2 * k_bound + 1) * (size_t)slice + sizeof(float) * (size_t)nseg;
    if (smem > kClusterSmemLimit) return p;
    p.ok = true;
    p.slice_bytes = (int32_t)slice;
    p.smem = smem;
    return p;
}

template <int DT>
int launch_cluster_path(const specv::BatchView& in, const ClusterPlan& plan, DeviceInfo& dev, int32_t* accepted_len,
                        int32_t* emitted, int32_t* row_status, float* diag_p, float* diag_q, specv::NextLookahead next,
                        cudaStream_t stream) {
    using namespace specv;
    {
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        if (!dev.cluster_ready[DT]) {
            if (!cuda_ok(cudaFuncSetAttribute(specv_cluster_pass<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kClusterSmemLimit)))
                return SPECV_ERR_CUDA;
            dev.cluster_ready[DT] = 1;
        }
    }
    auto trace = [&](int i) { if (g_trace_on) cudaEventRecord(g_trace[i], stream); };
    trace(0);
    trace(1);
    specv_cluster_pass<DT><<<in.B * kClusterCtas, kClusterThreads, plan.smem, stream>>>(
        in, plan.slice_bytes, accepted_len, emitted, row_status, diag_p, diag_q, next);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    trace(2);
    trace(3);
    return cuda_ok(cudaGetLastError()) ? SPECV_OK : SPECV_ERR_CUDA;
}
// Kernel set for a batch of n_items work items whose shape the ring kernels can (or cannot) take.
// They give a whole (target row, draft row) item to one CTA, so they need enough items to occupy
// the machine; tiny batches are better served by the streaming kernels, which split rows over CTAs.
bool choose_ring(uint32_t flags, bool shape_allows, int64_t n_items) {
    if (!shape_allows || (flags & SPECV_FLAG_STREAMING)) return false;
    return (flags & SPECV_FLAG_RING) || n_items >= 64;
}

// Everything after the entry point's own checks of its scratch: the remaining argument checks, the
// kernel-set choice and the launches.  `ws` holds at least ring_layout(...).total bytes.
int run_pass(const void* target_logits, const void* draft_logits, int dtype, int64_t V, int64_t ld_target,
             int64_t ld_draft, const int32_t* draft_tokens, const int32_t* k_per_row, int32_t B, int32_t k_uniform,
             int64_t n_draft_total, const float* temperature, int temperature_per_row, const float* uniforms,
             int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status, float* diag_p_tok,
             float* diag_q_tok, char* ws, uint32_t flags, int32_t k_min, int32_t k_max, int32_t* next_k,
             cudaStream_t stream) {
    const size_t elt = dtype == SPECV_F32 ? 4 : 2;
    if (!aligned_to(target_logits, elt) || !aligned_to(draft_logits, elt) || !aligned_to(draft_tokens, 4) ||
        !aligned_to(k_per_row, 4) || !aligned_to(temperature, 4) || !aligned_to(uniforms, 4) ||
        !aligned_to(accepted_len, 4) || !aligned_to(emitted_tokens, 4) || !aligned_to(row_status, 4) ||
        !aligned_to(diag_p_tok, 4) || !aligned_to(diag_q_tok, 4) || !aligned_to(next_k, 4))
        return SPECV_ERR_ALIGN;
    const Workspace lay = workspace_layout(B, n_draft_total, V);
    const RingLayout rl = ring_layout(lay.total, B, n_draft_total, V);
    DeviceInfo* dev = nullptr;
    int rc = device_info(&dev);
    if (rc != SPECV_OK) return rc;

    specv::BatchView in;
    in.target = static_cast<const char*>(target_logits);
    in.draft = static_cast<const char*>(draft_logits);
    in.pitch_t = ld_target * (int64_t)elt;
    in.pitch_d = ld_draft * (int64_t)elt;
    in.V = V;
    in.tokens = draft_tokens;
    in.k_per_row = k_per_row;
    in.B = B;
    in.k_uniform = k_uniform;
    in.n_draft_total = n_draft_total;
    in.temperature = temperature;
    in.per_row_temperature = temperature_per_row ? 1 : 0;
    in.uniforms = uniforms;
    const specv::NextLookahead next{next_k, k_min, k_max};
    const bool early = (flags & SPECV_FLAG_EARLY_EXIT) != 0;

    // small batches: everything in one launch, if a cluster per sequence can hold the sequence's rows
    // and the device runs that many clusters at once
    const ClusterPlan cluster = cluster_plan(in, dtype, flags);
    if (cluster.ok && B * specv::kClusterCtas <= dev->sms) {
        g_last_path = 3;
        if (dtype == SPECV_F32)
            return launch_cluster_path<specv::kF32>(in, cluster, *dev, accepted_len, emitted_tokens, row_status,
                                                    diag_p_tok, diag_q_tok, next, stream);
        if (dtype == SPECV_F16)
            return launch_cluster_path<specv::kF16>(in, cluster, *dev, accepted_len, emitted_tokens, row_status,
                                                    diag_p_tok, diag_q_tok, next, stream);
        return launch_cluster_path<specv::kBF16>(in, cluster, *dev, accepted_len, emitted_tokens, row_status,
                                                 diag_p_tok, diag_q_tok, next, stream);
    }
    if (choose_ring(flags, ring_shape_ok(in, dtype), n_draft_total + B)) {
        g_last_path = 2;
        if (dtype == SPECV_F32)
            return launch_ring_path<specv::kF32>(in, lay, rl, ws, *dev, accepted_len, emitted_tokens, row_status,
                                                 diag_p_tok, diag_q_tok, early, next, stream);
        if (dtype == SPECV_F16)
            return launch_ring_path<specv::kF16>(in, lay, rl, ws, *dev, accepted_len, emitted_tokens, row_status,
                                                 diag_p_tok, diag_q_tok, early, next, stream);
        return launch_ring_path<specv::kBF16>(in, lay, rl, ws, *dev, accepted_len, emitted_tokens, row_status,
                                              diag_p_tok, diag_q_tok, early, next, stream);
    }
    g_last_path = 1;
    if (dtype == SPECV_F32)
        return launch_stream_path<specv::kF32>(in, lay, ws, *dev, accepted_len, emitted_tokens, row_status,
                                               diag_p_tok, diag_q_tok, next, stream);
    if (dtype == SPECV_F16)
        return launch_stream_path<specv::kF16>(in, lay, ws, *dev, accepted_len, emitted_tokens, row_status,
                                               diag_p_tok, diag_q_tok, next, stream);
    return launch_stream_path<specv::kBF16>(in, lay, ws, *dev, accepted_len, emitted_tokens, row_status,
                                            diag_p_tok, diag_q_tok, next, stream);
}

}  // namespace

extern "C" {

int spec_verify_ex(const void* target_logits, const void* draft_logits, int dtype, int64_t V, int64_t ld_target,
                   int64_t ld_draft, const int32_t* draft_tokens, const int32_t* k_per_row, int32_t B,
                   int32_t k_uniform, int64_t n_draft_total, const float* temperature, int temperature_per_row,
                   const float* uniforms, int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                   float* diag_p_tok, float* diag_q_tok, void* workspace, size_t workspace_bytes,
                   void* cuda_stream, uint32_t flags, int32_t k_min, int32_t k_max, int32_t* next_k) {
    int rc = validate(target_logits, draft_logits, dtype, V, ld_target, ld_draft, draft_tokens, k_per_row, B,
                      k_uniform, n_draft_total, temperature, uniforms, accepted_len, emitted_tokens);
    if (rc != SPECV_OK) return rc;
    if (!flags_ok(flags)) return SPECV_ERR_FLAGS;
    if (next_k && (k_min < 0 || k_max < k_min)) return SPECV_ERR_SHAPE;
    if (!workspace) return SPECV_ERR_NULL;
    if (!aligned_to(workspace, 256)) return SPECV_ERR_ALIGN;
    if (workspace_bytes < ring_layout(workspace_layout(B, n_draft_total, V).total, B, n_draft_total, V).total)
        return SPECV_ERR_WORKSPACE;
    return run_pass(target_logits, draft_logits, dtype, V, ld_target, ld_draft, draft_tokens, k_per_row, B, k_uniform,
                    n_draft_total, temperature, temperature_per_row, uniforms, accepted_len, emitted_tokens,
                    row_status, diag_p_tok, diag_q_tok, static_cast<char*>(workspace), flags, k_min, k_max, next_k,
                    static_cast<cudaStream_t>(cuda_stream));
}

int spec_verify(const void* target_logits, const void* draft_logits, int dtype, int64_t V, int64_t ld_target,
                int64_t ld_draft, const int32_t* draft_tokens, const int32_t* k_per_row, int32_t B,
                int32_t k_uniform, int64_t n_draft_total, const float* temperature, int temperature_per_row,
                const float* uniforms, int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                float* diag_p_tok, float* diag_q_tok, void* workspace, size_t workspace_bytes,
                void* cuda_stream) {
    return spec_verify_ex(target_logits, draft_logits, dtype, V, ld_target, ld_draft, draft_tokens, k_per_row, B,
                          k_uniform, n_draft_total, temperature, temperature_per_row, uniforms, accepted_len,
                          emitted_tokens, row_status, diag_p_tok, diag_q_tok, workspace, workspace_bytes, cuda_stream,
                          0u, 0, 0, nullptr);
}

namespace {
struct Arena {
    size_t target, draft, tokens, k, temperature, uniforms, accepted, emitted, status, diag_p, diag_q, ws, total;
};
Arena arena_layout(int dtype, int32_t B, int64_t D, int64_t V) {
    const size_t elt = dtype == SPECV_F32 ? 4 : 2;
    Arena a;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    a.target = take((size_t)(D + B) * V * elt);
    a.draft = take((size_t)D * V * elt);
    a.tokens = take((size_t)D * 4);
    a.k = take((size_t)B * 4);
    a.temperature = take((size_t)B * 4);
    a.uniforms = take((size_t)(D + B) * 4);
    a.accepted = take((size_t)B * 4);
    a.emitted = take((size_t)(D + B) * 4);
    a.status = take((size_t)B * 4);
    a.diag_p = take((size_t)D * 4);
    a.diag_q = take((size_t)D * 4);
    a.ws = take(ring_layout(workspace_layout(B, D, V).total, B, D, V).total);
    a.total = o;
    return a;
}
}  // namespace

size_t spec_verify_host_arena_bytes(int dtype, int32_t B, int64_t n_draft_total, int64_t V) {
    if ((dtype != SPECV_F32 && dtype != SPECV_BF16 && dtype != SPECV_F16) || !shape_ok(B, n_draft_total, V)) return 0;
    return arena_layout(dtype, B, n_draft_total, V).total;
}

int spec_verify_host(const void* target_logits, const void* draft_logits, int dtype, int64_t V,
                     int64_t ld_target, int64_t ld_draft, const int32_t* draft_tokens,
                     const int32_t* k_per_row, int32_t B, int32_t k_uniform, int64_t n_draft_total,
                     const float* temperature, int temperature_per_row, const float* uniforms,
                     int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status, float* diag_p_tok,
                     float* diag_q_tok, void* arena, size_t arena_bytes, void* cuda_stream, uint32_t flags) {
    int rc = validate(target_logits, draft_logits, dtype, V, ld_target, ld_draft, draft_tokens, k_per_row, B,
                      k_uniform, n_draft_total, temperature, uniforms, accepted_len, emitted_tokens);
    if (rc != SPECV_OK) return rc;
    if (!flags_ok(flags)) return SPECV_ERR_FLAGS;
    if (!arena) return SPECV_ERR_NULL;
    if (!aligned_to(arena, 256)) return SPECV_ERR_ALIGN;
    const Arena a = arena_layout(dtype, B, n_draft_total, V);
    if (arena_bytes < a.total) return SPECV_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* base = static_cast<char*>(arena);
    const size_t elt = dtype == SPECV_F32 ? 4 : 2;
    const int64_t D = n_draft_total;
    const size_t row = (size_t)V * elt;

    auto h2d = [&](size_t at, const void* src, size_t bytes) {
        return bytes == 0 || cuda_ok(cudaMemcpyAsync(base + at, src, bytes, cudaMemcpyHostToDevice, stream));
    };
    auto h2d_rows = [&](size_t at, const void* src, int64_t ld, int64_t rows) {
        if (rows == 0) return true;
        if (ld == V) return cuda_ok(cudaMemcpyAsync(base + at, src, row * rows, cudaMemcpyHostToDevice, stream));
        return cuda_ok(cudaMemcpy2DAsync(base + at, row, src, (size_t)ld * elt, row, (size_t)rows,
                                         cudaMemcpyHostToDevice, stream));
    };
    if (!h2d_rows(a.target, target_logits, ld_target, D + B) || !h2d_rows(a.draft, draft_logits, ld_draft, D) ||
        !h2d(a.tokens, draft_tokens, (size_t)D * 4) || (k_per_row && !h2d(a.k, k_per_row, (size_t)B * 4)) ||
        !h2d(a.temperature, temperature, temperature_per_row ? (size_t)B * 4 : 4) ||
        !h2d(a.uniforms, uniforms, (size_t)(D + B) * 4))
        return SPECV_ERR_CUDA;

    rc = spec_verify_ex(base + a.target, D ? base + a.draft : nullptr, dtype, V, V, V,
                     D ? reinterpret_cast<const int32_t*>(base + a.tokens) : nullptr,
                     k_per_row ? reinterpret_cast<const int32_t*>(base + a.k) : nullptr, B, k_uniform, D,
                     reinterpret_cast<const float*>(base + a.temperature), temperature_per_row,
                     reinterpret_cast<const float*>(base + a.uniforms),
                     reinterpret_cast<int32_t*>(base + a.accepted), reinterpret_cast<int32_t*>(base + a.emitted),
                     reinterpret_cast<int32_t*>(base + a.status),
                     diag_p_tok ? reinterpret_cast<float*>(base + a.diag_p) : nullptr,
                     diag_q_tok ? reinterpret_cast<float*>(base + a.diag_q) : nullptr, base + a.ws,
                     arena_bytes - a.ws, stream, flags, 0, 0, nullptr);
    if (rc != SPECV_OK) return rc;

    auto d2h = [&](void* dst, size_t at, size_t bytes) {
        return !dst || bytes == 0 || cuda_ok(cudaMemcpyAsync(dst, base + at, bytes, cudaMemcpyDeviceToHost, stream));
    };
    if (!d2h(accepted_len, a.accepted, (size_t)B * 4) || !d2h(emitted_tokens, a.emitted, (size_t)(D + B) * 4) ||
        !d2h(row_status, a.status, (size_t)B * 4) || !d2h(diag_p_tok, a.diag_p, (size_t)D * 4) ||
        !d2h(diag_q_tok, a.diag_q, (size_t)D * 4))
        return SPECV_ERR_CUDA;
    if (!cuda_ok(cudaStreamSynchronize(stream))) return SPECV_ERR_CUDA;
    return SPECV_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------
// spec_verify_tree
// ---------------------------------------------------------------------------------
namespace {

struct TreeLayout {
    Workspace lay;
    RingLayout rl;
    size_t has_children, total;
};
TreeLayout tree_layout(int32_t B, int64_t D, int64_t V) {
    TreeLayout t;
    t.lay = workspace_layout(B, D, V);
    t.rl = ring_layout(t.lay.total, B, D, V);
    t.has_children = t.rl.total;
    t.total = align_up(t.has_children + sizeof(int32_t) * (size_t)(D > 0 ? D : 1), 256);
    return t;
}

constexpr int kTreeMaxSmem = 200 * 1024;     // caches (52 KB) and the segment sums of the largest vocabulary (128 KB)

template <int DT>
int launch_tree(specv::BatchView in, const TreeLayout& tl, char* ws, DeviceInfo& dev, bool ring,
                int32_t* accepted_len, int32_t* emitted, int32_t* accepted_nodes, int32_t* row_status,
                float* diag_p, float* diag_q, cudaStream_t stream) {
    using namespace specv;
    int32_t* off_d = reinterpret_cast<int32_t*>(ws + tl.lay.off_d);
    int32_t* seq_status = reinterpret_cast<int32_t*>(ws + tl.lay.seq_status);
    int32_t* has_children = reinterpret_cast<int32_t*>(ws + tl.has_children);
    int32_t* ctrl = reinterpret_cast<int32_t*>(ws + tl.rl.ctrl);
    in.ctx_has_children = has_children;
    const int64_t n_target = in.n_draft_total + in.B;
    const int64_t n_rows = n_target + in.n_draft_total;
    if (ring ? !ensure_ring_ready<DT>(dev) : !ensure_stream_ready<DT>(dev)) return SPECV_ERR_CUDA;
    {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!dev.tree_ready[DT]) {
        if (!cuda_ok(cudaFuncSetAttribute(specv_tree_resolve<DT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTreeMaxSmem)) ||
            !cuda_ok(cudaFuncSetAttribute(specv_tree_resolve<DT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTreeMaxSmem)))
            return SPECV_ERR_CUDA;
        dev.tree_ready[DT] = 1;
    }
    }
    auto trace = [&](int i) { if (g_trace_on) cudaEventRecord(g_trace[i], stream); };
    trace(0);
    int pro_blocks = (int)((n_target + 8 * kPrologueThreads - 1) / (8 * kPrologueThreads));
    if (pro_blocks < 1) pro_blocks = 1;
    if (pro_blocks > dev.sms) pro_blocks = dev.sms;
    specv_prologue<<<pro_blocks, kPrologueThreads, 0, stream>>>(in, off_d, seq_status, emitted, ctrl, nullptr, 0);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;

    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)in.B, 1, 1);
    cfg.blockDim = dim3(kTreePlanThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    const int32_t* off_d_c = off_d;
    if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_tree_plan, in, off_d_c, seq_status, has_children, accepted_nodes)))
        return SPECV_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);

    trace(1);
    const float2* stat_t = nullptr;
    const float2* stat_d = nullptr;
    int splits = 1;
    if (ring) {
        RingScratch sc = {};
        sc.off_d = off_d;
        sc.seq_status = seq_status;
        sc.stat_p = reinterpret_cast<float2*>(ws + tl.rl.stat_p);
        sc.stat_q = reinterpret_cast<float2*>(ws + tl.rl.stat_q);
        sc.ctrl = ctrl;
        cfg.gridDim = dim3((unsigned)dev.sms, 1, 1);
        cfg.blockDim = dim3(kRingStatsThreads, 1, 1);
        cfg.dynamicSmemBytes = sizeof(RingStatsShared);
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_ring_stats<DT>, in, sc, 0))) return SPECV_ERR_CUDA;
        stat_t = sc.stat_p;
        stat_d = sc.stat_q;
        splits = kStatParts;          // the ring kernel stores up to kStatParts parts per row
    } else {
        float2* partial = reinterpret_cast<float2*>(ws + tl.lay.partial);
        splits = splits_for(n_rows, in.V);
        const int64_t n_items = n_rows * splits;
        int64_t stats_blocks = (int64_t)dev.sms * dev.stats_blocks_per_sm[DT];
        if (stats_blocks > n_items) stats_blocks = n_items;
        cfg.gridDim = dim3((unsigned)stats_blocks, 1, 1);
        cfg.blockDim = dim3(kStatsThreads, 1, 1);
        cfg.dynamicSmemBytes = 0;
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_row_stats<DT>, in, off_d_c, n_target, n_rows, splits, partial)))
            return SPECV_ERR_CUDA;
        stat_t = partial;
        stat_d = partial + n_target * splits;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);

    trace(2);
    const int seg_elems = 32 * Elt<DT>::kPerVec;
    const size_t nseg = (size_t)((in.V + seg_elems - 1) / seg_elems);
    // pairs of CTAs per sequence while every pair still gets SMs of its own: a walk is a chain of
    // dependent passes, and a pair halves the time of each
    const size_t seg_bytes = sizeof(float) * ((nseg + 3) & ~(size_t)3);
    const bool pairs = 2 * (int64_t)in.B <= dev.sms && kTreeCacheBytes + 2 * seg_bytes <= (size_t)kTreeMaxSmem;
    cudaLaunchAttribute attrs[2];
    attrs[0] = pdl[0];
    attrs[1].id = cudaLaunchAttributeClusterDimension;
    attrs[1].val.clusterDim.x = 2;
    attrs[1].val.clusterDim.y = 1;
    attrs[1].val.clusterDim.z = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = pairs ? 2 : 1;
    cfg.gridDim = dim3((unsigned)in.B * (pairs ? 2u : 1u), 1, 1);
    cfg.blockDim = dim3(kTreeThreads, 1, 1);
    cfg.dynamicSmemBytes = kTreeCacheBytes + (pairs ? 2 : 1) * seg_bytes;      // a pair alternates between two buffers
    const int32_t* seq_status_c = seq_status;
    const int32_t* err_c = ring ? ctrl : nullptr;
    const cudaError_t e =
        pairs ? cudaLaunchKernelEx(&cfg, specv_tree_resolve<DT, 2>, in, off_d_c, seq_status_c, stat_t, stat_d, splits, err_c,
                                   accepted_len, emitted, accepted_nodes, row_status, diag_p, diag_q)
              : cudaLaunchKernelEx(&cfg, specv_tree_resolve<DT, 1>, in, off_d_c, seq_status_c, stat_t, stat_d, splits, err_c,
                                   accepted_len, emitted, accepted_nodes, row_status, diag_p, diag_q);
    if (!cuda_ok(e)) return SPECV_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    trace(3);
    return SPECV_OK;
}

}  // namespace

extern "C" size_t spec_verify_tree_workspace_bytes(int32_t B, int64_t n_node_total, int64_t V) {
    if (!shape_ok(B, n_node_total, V)) return 0;
    return tree_layout(B, n_node_total, V).total;
}

extern "C" int spec_verify_tree(const void* target_logits, const void* draft_logits, int dtype, int64_t V,
                                int64_t ld_target, int64_t ld_draft, const int32_t* node_tokens,
                                const int32_t* node_parent, const int32_t* n_per_seq, int32_t B,
                                int32_t n_uniform, int64_t n_node_total, const float* temperature,
                                int temperature_per_seq, const float* uniforms, int32_t* accepted_len,
                                int32_t* emitted_tokens, int32_t* accepted_nodes, int32_t* row_status,
                                float* diag_p_tok, float* diag_q_tok, void* workspace, size_t workspace_bytes,
                                void* cuda_stream, uint32_t flags) {
    int rc = validate(target_logits, draft_logits, dtype, V, ld_target, ld_draft, node_tokens, n_per_seq, B,
                      n_uniform, n_node_total, temperature, uniforms, accepted_len, emitted_tokens);
    if (rc != SPECV_OK) return rc;
    if (!flags_ok(flags) || (flags & SPECV_FLAG_EARLY_EXIT)) return SPECV_ERR_FLAGS;
    if (!workspace || (n_node_total > 0 && !node_parent)) return SPECV_ERR_NULL;
    const size_t elt = dtype == SPECV_F32 ? 4 : 2;
    if (!aligned_to(workspace, 256) || !aligned_to(target_logits, elt) || !aligned_to(draft_logits, elt) ||
        !aligned_to(node_tokens, 4) || !aligned_to(node_parent, 4) || !aligned_to(n_per_seq, 4) ||
        !aligned_to(temperature, 4) || !aligned_to(uniforms, 4) || !aligned_to(accepted_len, 4) ||
        !aligned_to(emitted_tokens, 4) || !aligned_to(accepted_nodes, 4) || !aligned_to(row_status, 4) ||
        !aligned_to(diag_p_tok, 4) || !aligned_to(diag_q_tok, 4))
        return SPECV_ERR_ALIGN;
    const TreeLayout tl = tree_layout(B, n_node_total, V);
    if (workspace_bytes < tl.total) return SPECV_ERR_WORKSPACE;
    DeviceInfo* dev = nullptr;
    rc = device_info(&dev);
    if (rc != SPECV_OK) return rc;

    specv::BatchView in;
    in.target = static_cast<const char*>(target_logits);
    in.draft = static_cast<const char*>(draft_logits);
    in.pitch_t = ld_target * (int64_t)elt;
    in.pitch_d = ld_draft * (int64_t)elt;
    in.V = V;
    in.tokens = node_tokens;
    in.k_per_row = n_per_seq;
    in.B = B;
    in.k_uniform = n_uniform;
    in.n_draft_total = n_node_total;
    in.temperature = temperature;
    in.per_row_temperature = temperature_per_seq ? 1 : 0;
    in.uniforms = uniforms;
    in.parent = node_parent;
    const bool ring = choose_ring(flags, ring_shape_ok(in, dtype), n_node_total + B);
    g_last_path = ring ? 2 : 1;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    if (dtype == SPECV_F32)
        return launch_tree<specv::kF32>(in, tl, ws, *dev, ring, accepted_len, emitted_tokens, accepted_nodes,
                                        row_status, diag_p_tok, diag_q_tok, stream);
    if (dtype == SPECV_F16)
        return launch_tree<specv::kF16>(in, tl, ws, *dev, ring, accepted_len, emitted_tokens, accepted_nodes,
                                        row_status, diag_p_tok, diag_q_tok, stream);
    return launch_tree<specv::kBF16>(in, tl, ws, *dev, ring, accepted_len, emitted_tokens, accepted_nodes,
                                     row_status, diag_p_tok, diag_q_tok, stream);
}

// ---------------------------------------------------------------------------------
// spec_verify_greedy
// ---------------------------------------------------------------------------------
namespace {

struct GreedyLayout {
    size_t off_d, seq_status, argmax, ctrl, total;
};
GreedyLayout greedy_layout(int32_t B, int64_t D) {
    GreedyLayout g;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    g.off_d = take(sizeof(int32_t) * ((size_t)B + 1));
    g.seq_status = take(sizeof(int32_t) * (size_t)B);
    g.argmax = take(sizeof(int32_t) * (size_t)(D + B));
    g.ctrl = take(64);
    g.total = o;
    return g;
}

template <int DT>
int launch_greedy(const specv::BatchView& in, const GreedyLayout& gl, char* ws, DeviceInfo& dev, bool ring,
                  int32_t* accepted_len, int32_t* emitted, int32_t* row_status, int32_t* target_argmax,
                  cudaStream_t stream) {
    using namespace specv;
    int32_t* off_d = reinterpret_cast<int32_t*>(ws + gl.off_d);
    int32_t* seq_status = reinterpret_cast<int32_t*>(ws + gl.seq_status);
    int32_t* argmax = target_argmax ? target_argmax : reinterpret_cast<int32_t*>(ws + gl.argmax);
    int32_t* ctrl = reinterpret_cast<int32_t*>(ws + gl.ctrl);
    const int64_t n_rows = in.n_draft_total + in.B;
    {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (ring && !dev.ring_argmax_ready[DT]) {
        if (!cuda_ok(cudaFuncSetAttribute(specv_ring_argmax<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(RingArgmaxShared))))
            return SPECV_ERR_CUDA;
        dev.ring_argmax_ready[DT] = 1;
    }
    if (!ring && dev.argmax_blocks_per_sm[DT] == 0) {
        int per_sm = 0;
        if (!cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, specv_row_argmax<DT>, kArgmaxThreads, 0)))
            return SPECV_ERR_CUDA;
        dev.argmax_blocks_per_sm[DT] = per_sm > 0 ? per_sm : 1;
    }
    }
    auto trace = [&](int i) { if (g_trace_on) cudaEventRecord(g_trace[i], stream); };
    trace(0);
    int pro_blocks = (int)((n_rows + 8 * kPrologueThreads - 1) / (8 * kPrologueThreads));
    if (pro_blocks < 1) pro_blocks = 1;
    if (pro_blocks > dev.sms) pro_blocks = dev.sms;
    specv_prologue<<<pro_blocks, kPrologueThreads, 0, stream>>>(in, off_d, seq_status, emitted, ctrl, nullptr, 0);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;

    trace(1);
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (ring) {
        cfg.gridDim = dim3((unsigned)(n_rows < dev.sms ? n_rows : dev.sms), 1, 1);
        cfg.blockDim = dim3(kRingArgmaxThreads, 1, 1);
        cfg.dynamicSmemBytes = sizeof(RingArgmaxShared);
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_ring_argmax<DT>, in.target, in.pitch_t, in.V, n_rows, argmax, ctrl)))
            return SPECV_ERR_CUDA;
    } else {
        int64_t blocks = (int64_t)dev.sms * dev.argmax_blocks_per_sm[DT];
        if (blocks > n_rows) blocks = n_rows;
        cfg.gridDim = dim3((unsigned)blocks, 1, 1);
        cfg.blockDim = dim3(kArgmaxThreads, 1, 1);
        cfg.dynamicSmemBytes = 0;
        if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_row_argmax<DT>, in.target, in.pitch_t, in.V, n_rows, argmax)))
            return SPECV_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);

    trace(2);
    constexpr int kSeqPerBlock = kGreedyResolveThreads / 32;
    cfg.gridDim = dim3((unsigned)((in.B + kSeqPerBlock - 1) / kSeqPerBlock), 1, 1);
    cfg.blockDim = dim3(kGreedyResolveThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    const int32_t* off_d_c = off_d;
    const int32_t* seq_status_c = seq_status;
    const int32_t* argmax_c = argmax;
    const int32_t* ctrl_c = ctrl;
    if (!cuda_ok(cudaLaunchKernelEx(&cfg, specv_greedy_resolve, in, off_d_c, seq_status_c, argmax_c, ctrl_c,
                                    accepted_len, emitted, row_status)))
        return SPECV_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    trace(3);
    return SPECV_OK;
}

}  // namespace

extern "C" size_t spec_verify_greedy_workspace_bytes(int32_t B, int64_t n_draft_total) {
    if (!shape_ok(B, n_draft_total, 1)) return 0;
    return greedy_layout(B, n_draft_total).total;
}

extern "C" int spec_verify_greedy(const void* target_logits, int dtype, int64_t V, int64_t ld_target,
                                  const int32_t* draft_tokens, const int32_t* k_per_row, int32_t B,
                                  int32_t k_uniform, int64_t n_draft_total, int32_t* accepted_len,
                                  int32_t* emitted_tokens, int32_t* row_status, int32_t* target_argmax,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream, uint32_t flags) {
    if (dtype != SPECV_F32 && dtype != SPECV_BF16 && dtype != SPECV_F16) return SPECV_ERR_DTYPE;
    if (!flags_ok(flags) || (flags & SPECV_FLAG_EARLY_EXIT)) return SPECV_ERR_FLAGS;
    if (!shape_ok(B, n_draft_total, V) || ld_target < V) return SPECV_ERR_SHAPE;
    if (!k_per_row && (k_uniform < 0 || (int64_t)B * k_uniform != n_draft_total)) return SPECV_ERR_SHAPE;
    if (!target_logits || !accepted_len || !emitted_tokens || !workspace) return SPECV_ERR_NULL;
    if (n_draft_total > 0 && !draft_tokens) return SPECV_ERR_NULL;
    const size_t elt = dtype == SPECV_F32 ? 4 : 2;
    if (!aligned_to(workspace, 256) || !aligned_to(target_logits, elt) || !aligned_to(draft_tokens, 4) ||
        !aligned_to(k_per_row, 4) || !aligned_to(accepted_len, 4) || !aligned_to(emitted_tokens, 4) ||
        !aligned_to(row_status, 4) || !aligned_to(target_argmax, 4))
        return SPECV_ERR_ALIGN;
    const GreedyLayout gl = greedy_layout(B, n_draft_total);
    if (workspace_bytes < gl.total) return SPECV_ERR_WORKSPACE;
    DeviceInfo* dev = nullptr;
    int rc = device_info(&dev);
    if (rc != SPECV_OK) return rc;

    specv::BatchView in;
    in.target = static_cast<const char*>(target_logits);
    in.draft = nullptr;
    in.pitch_t = ld_target * (int64_t)elt;
    in.pitch_d = 0;
    in.V = V;
    in.tokens = draft_tokens;
    in.k_per_row = k_per_row;
    in.B = B;
    in.k_uniform = k_uniform;
    in.n_draft_total = n_draft_total;
    in.temperature = nullptr;
    in.per_row_temperature = 0;
    in.uniforms = nullptr;
    // the ring kernel gives a whole row to one CTA: it needs enough rows to occupy the machine
    const bool bulk_ok = !(reinterpret_cast<uintptr_t>(in.target) & 15u) && !(in.pitch_t & 15) && !((V * (int64_t)elt) & 15);
    const bool ring = choose_ring(flags, bulk_ok, n_draft_total + B);
    g_last_path = ring ? 2 : 1;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    if (dtype == SPECV_F32)
        return launch_greedy<specv::kF32>(in, gl, ws, *dev, ring, accepted_len, emitted_tokens, row_status,
                                          target_argmax, stream);
    if (dtype == SPECV_F16)
        return launch_greedy<specv::kF16>(in, gl, ws, *dev, ring, accepted_len, emitted_tokens, row_status,
                                          target_argmax, stream);
    return launch_greedy<specv::kBF16>(in, gl, ws, *dev, ring, accepted_len, emitted_tokens, row_status,
                                       target_argmax, stream);
}

// ---------------------------------------------------------------------------------
// spec_verify_noalloc: spec_verify with its scratch in a static device array.
// ---------------------------------------------------------------------------------
namespace {

// The scratch itself.  It is part of the library image on every GPU that loads the library
// and stays there until the process exits.  In HOST code this name is only a handle for
// cudaGetSymbolAddress, never an address to hand to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[SPECV_NOALLOC_SCRATCH_BYTES];

// Device address of g_static_scratch per device, looked up once per device.
void* g_static_scratch_ptr[kMaxDevices] = {};

int static_scratch_for_current_device(char** out) {
    int dev = 0;
    if (!cuda_ok(cudaGetDevice(&dev))) return SPECV_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return SPECV_ERR_ARCH;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_static_scratch_ptr[dev]) {
        void* p = nullptr;
        if (!cuda_ok(cudaGetSymbolAddress(&p, g_static_scratch)) || !p) return SPECV_ERR_CUDA;
        g_static_scratch_ptr[dev] = p;
    }
    *out = static_cast<char*>(g_static_scratch_ptr[dev]);
    return SPECV_OK;
}

}  // namespace

extern "C" int spec_verify_noalloc(const void* target_logits, const void* draft_logits, int dtype, int64_t V,
                                   int64_t ld_target, int64_t ld_draft, const int32_t* draft_tokens,
                                   const int32_t* k_per_row, int32_t B, int32_t k_uniform,
                                   int64_t n_draft_total, const float* temperature, int temperature_per_row,
                                   const float* uniforms, int32_t* accepted_len, int32_t* emitted_tokens,
                                   int32_t* row_status, float* diag_p_tok, float* diag_q_tok,
                                   void* cuda_stream) {
    int rc = validate(target_logits, draft_logits, dtype, V, ld_target, ld_draft, draft_tokens, k_per_row, B,
                      k_uniform, n_draft_total, temperature, uniforms, accepted_len, emitted_tokens);
    if (rc != SPECV_OK) return rc;
    if (ring_layout(workspace_layout(B, n_draft_total, V).total, B, n_draft_total, V).total >
        (size_t)SPECV_NOALLOC_SCRATCH_BYTES)
        return SPECV_ERR_TOO_LARGE;   // the documented limit is the public workspace size
    char* scratch = nullptr;
    rc = static_scratch_for_current_device(&scratch);
    if (rc != SPECV_OK) return rc;
    // Nothing in the scratch has to start at zero: whichever kernel set runs writes every word of
    // it (offsets, per-sequence status, statistics, tickets) before reading it.
    return run_pass(target_logits, draft_logits, dtype, V, ld_target, ld_draft, draft_tokens, k_per_row, B, k_uniform,
                    n_draft_total, temperature, temperature_per_row, uniforms, accepted_len, emitted_tokens,
                    row_status, diag_p_tok, diag_q_tok, scratch, 0u, 0, 0, nullptr,
                    static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------
// Self-test of the bounded waits
// ---------------------------------------------------------------------------------
extern "C" int spec_verify_selftest_bounded_wait(int64_t limit_cycles, int64_t* out4, void* cuda_stream) {
    if (!out4) return SPECV_ERR_NULL;
    if (limit_cycles < 1 || limit_cycles > 2000000000LL) return SPECV_ERR_SHAPE;
    if (!aligned_to(out4, 8)) return SPECV_ERR_ALIGN;
    specv::specv_selftest_bounded_wait<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        (long long)limit_cycles, reinterpret_cast<long long*>(out4));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cuda_ok(cudaGetLastError()) ? SPECV_OK : SPECV_ERR_CUDA;
}

// ---------------------------------------------------------------------------------
// Debug build: the recorded range violation
// ---------------------------------------------------------------------------------
extern "C" int spec_verify_debug_violation(void) {
#ifdef SPECV_DEBUG
    int v = 0;
    if (!cuda_ok(cudaMemcpyFromSymbol(&v, specv::g_debug_violation, sizeof(int)))) return -2;
    return v;
#else
    return -1;
#endif
}

// ---------------------------------------------------------------------------------
// spec_verify_from_hidden: LM-head products on the tensor cores with the row statistics in
// their epilogue, then the resolve kernel of the ring set
// ---------------------------------------------------------------------------------
namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 matrix [rows, cols] with a pitch of ld elements, boxes of box_rows x 64 elements, 128-byte swizzle
bool make_bf16_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)specv::kLmBK, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct HiddenLayout {
    Workspace lay;
    RingLayout rl;
    size_t c_target, c_draft, part_t, part_d, status, total;
};
HiddenLayout hidden_layout(int32_t B, int64_t D, int64_t V) {
    HiddenLayout h;
    h.lay = workspace_layout(B, D, V);
    h.rl = ring_layout(h.lay.total, B, D, V);
    size_t o = h.rl.total;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const size_t tiles_n = (size_t)((V + specv::kLmBN - 1) / specv::kLmBN);
    h.c_target = take(sizeof(float) * (size_t)(D + B));
    h.c_draft = take(sizeof(float) * (size_t)(D > 0 ? D : 1));
    h.part_t = take(sizeof(float2) * (size_t)(D + B) * tiles_n);
    h.part_d = take(sizeof(float2) * (size_t)(D > 0 ? D : 1) * tiles_n);
    h.status = take(64);
    h.total = o;
    return h;
}

bool lm_head_ready(DeviceInfo& dev) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!dev.lm_head_ready) {
        if (!cuda_ok(cudaFuncSetAttribute(specv::specv_lm_head, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(specv::LmHeadShared))))
            return false;
        dev.lm_head_ready = 1;
    }
    return true;
}

int launch_lm_head(const void* hidden, int64_t ld_h, const void* weight, int64_t ld_w, int64_t M, int64_t V, int64_t H,
                   const float* row_scale, void* logits, int64_t ld_out, float2* part, int32_t* status,
                   DeviceInfo& dev, cudaStream_t stream) {
    if (M == 0) return SPECV_OK;
    CUtensorMap map_a, map_b;
    if (!make_bf16_map(&map_a, hidden, M, H, ld_h, specv::kLmBM) || !make_bf16_map(&map_b, weight, V, H, ld_w, specv::kLmBN))
        return SPECV_ERR_CUDA;
    const int64_t tiles = ((M + specv::kLmBM - 1) / specv::kLmBM) * ((V + specv::kLmBN - 1) / specv::kLmBN);
    const int grid = (int)(tiles < dev.sms ? tiles : dev.sms);
    specv::specv_lm_head<<<grid, specv::kLmThreads, sizeof(specv::LmHeadShared), stream>>>(
        map_a, map_b, M, V, H, row_scale, static_cast<uint16_t*>(logits), ld_out, part, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cuda_ok(cudaGetLastError()) ? SPECV_OK : SPECV_ERR_CUDA;
}

bool hidden_shape_ok(const void* hidden, int64_t ld_h, const void* weight, int64_t ld_w, int64_t H) {
    // tensor maps: 16-byte aligned base addresses and pitches
    return H >= 1 && ld_h >= H && ld_w >= H && !(reinterpret_cast<uintptr_t>(hidden) & 15u) &&
           !(reinterpret_cast<uintptr_t>(weight) & 15u) && !((ld_h * 2) & 15) && !((ld_w * 2) & 15);
}

}  // namespace

extern "C" size_t spec_verify_from_hidden_workspace_bytes(int32_t B, int64_t n_draft_total, int64_t V) {
    if (!shape_ok(B, n_draft_total, V)) return 0;
    return hidden_layout(B, n_draft_total, V).total;
}

extern "C" int spec_verify_from_hidden(const void* target_hidden, int64_t ld_th, int64_t H_target,
                                       const void* target_weight, int64_t ld_tw, const void* draft_hidden,
                                       int64_t ld_dh, int64_t H_draft, const void* draft_weight, int64_t ld_dw,
                                       int64_t V, void* target_logits, int64_t ld_target, void* draft_logits,
                                       int64_t ld_draft, const int32_t* draft_tokens, const int32_t* k_per_row,
                                       int32_t B, int32_t k_uniform, int64_t n_draft_total, const float* temperature,
                                       int temperature_per_row, const float* uniforms, int32_t* accepted_len,
                                       int32_t* emitted_tokens, int32_t* row_status, float* diag_p_tok,
                                       float* diag_q_tok, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = validate(target_logits, draft_logits, SPECV_BF16, V, ld_target, ld_draft, draft_tokens, k_per_row, B,
                      k_uniform, n_draft_total, temperature, uniforms, accepted_len, emitted_tokens);
    if (rc != SPECV_OK) return rc;
    if (!target_hidden || !target_weight || !workspace) return SPECV_ERR_NULL;
    if (n_draft_total > 0 && (!draft_hidden || !draft_weight)) return SPECV_ERR_NULL;
    const int64_t D = n_draft_total;
    if (!hidden_shape_ok(target_hidden, ld_th, target_weight, ld_tw, H_target)) return SPECV_ERR_SHAPE;
    if (D > 0 && !hidden_shape_ok(draft_hidden, ld_dh, draft_weight, ld_dw, H_draft)) return SPECV_ERR_SHAPE;
    if (!aligned_to(workspace, 256) || !aligned_to(draft_tokens, 4) || !aligned_to(k_per_row, 4) ||
        !aligned_to(temperature, 4) || !aligned_to(uniforms, 4) || !aligned_to(accepted_len, 4) ||
        !aligned_to(emitted_tokens, 4) || !aligned_to(row_status, 4) || !aligned_to(diag_p_tok, 4) ||
        !aligned_to(diag_q_tok, 4))
        return SPECV_ERR_ALIGN;
    const HiddenLayout hl = hidden_layout(B, D, V);
    if (workspace_bytes < hl.total) return SPECV_ERR_WORKSPACE;
    DeviceInfo* dev = nullptr;
    rc = device_info(&dev);
    if (rc != SPECV_OK) return rc;

    specv::BatchView in;
    in.target = static_cast<const char*>(target_logits);
    in.draft = static_cast<const char*>(draft_logits);
    in.pitch_t = ld_target * 2;
    in.pitch_d = ld_draft * 2;
    in.V = V;
    in.tokens = draft_tokens;
    in.k_per_row = k_per_row;
    in.B = B;
    in.k_uniform = k_uniform;
    in.n_draft_total = D;
    in.temperature = temperature;
    in.per_row_temperature = temperature_per_row ? 1 : 0;
    in.uniforms = uniforms;
    // the resolve kernel of the ring set reads the logits this call writes: their layout must be one it takes
    if (!ring_shape_ok(in, SPECV_BF16)) return SPECV_ERR_SHAPE;
    if (!ensure_ring_ready<specv::kBF16>(*dev) || !lm_head_ready(*dev)) return SPECV_ERR_CUDA;

    char* ws = static_cast<char*>(workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    using namespace specv;
    RingScratch sc = {};
    sc.off_d = reinterpret_cast<int32_t*>(ws + hl.lay.off_d);
    sc.seq_status = reinterpret_cast<int32_t*>(ws + hl.lay.seq_status);
    sc.stat_p = reinterpret_cast<float2*>(ws + hl.rl.stat_p);
    sc.stat_q = reinterpret_cast<float2*>(ws + hl.rl.stat_q);
    sc.done = reinterpret_cast<int32_t*>(ws + hl.rl.done);
    sc.gseg = reinterpret_cast<float*>(ws + hl.rl.gseg);
    sc.ctrl = reinterpret_cast<int32_t*>(ws + hl.rl.ctrl);
    float* c_target = reinterpret_cast<float*>(ws + hl.c_target);
    float* c_draft = reinterpret_cast<float*>(ws + hl.c_draft);
    float2* part_t = reinterpret_cast<float2*>(ws + hl.part_t);
    float2* part_d = reinterpret_cast<float2*>(ws + hl.part_d);
    int32_t* lm_status = reinterpret_cast<int32_t*>(ws + hl.status);
    g_last_path = 2;

    // offsets, per-sequence checks, -1 fill, tickets and error word zeroed
    const int64_t n_slots = D + B;
    int pro_blocks = (int)((n_slots + 8 * kPrologueThreads - 1) / (8 * kPrologueThreads));
    if (pro_blocks < 1) pro_blocks = 1;
    if (pro_blocks > dev->sms) pro_blocks = dev->sms;
    specv_prologue<<<pro_blocks, kPrologueThreads, 0, stream>>>(in, sc.off_d, sc.seq_status, emitted_tokens, sc.ctrl,
                                                                  sc.done, 0);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;
    if (!cuda_ok(cudaMemsetAsync(lm_status, 0, 64, stream))) return SPECV_ERR_CUDA;
    const int64_t n_rows = n_slots + D;
    specv_row_scales<<<(unsigned)((n_rows + 255) / 256), 256, 0, stream>>>(in, sc.off_d, c_target, c_draft);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;

    rc = launch_lm_head(target_hidden, ld_th, target_weight, ld_tw, n_slots, V, H_target, c_target, target_logits,
                        ld_target, part_t, lm_status, *dev, stream);
    if (rc != SPECV_OK) return rc;
    rc = launch_lm_head(draft_hidden, ld_dh, draft_weight, ld_dw, D, V, H_draft, c_draft, draft_logits, ld_draft, part_d,
                        lm_status, *dev, stream);
    if (rc != SPECV_OK) return rc;
    const int64_t tiles_n = (V + kLmBN - 1) / kLmBN;
    specv_merge_tile_stats<<<(unsigned)((n_slots * 32 + 255) / 256), 256, 0, stream>>>(part_t, n_slots, tiles_n, sc.stat_p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (D > 0) {
        specv_merge_tile_stats<<<(unsigned)((D * 32 + 255) / 256), 256, 0, stream>>>(part_d, D, tiles_n, sc.stat_q);
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    if (!cuda_ok(cudaGetLastError())) return SPECV_ERR_CUDA;

    const int64_t nck = (V * 2 + kChunkBytes - 1) / kChunkBytes;
    const int64_t max_units = (int64_t)B * nck;
    const int resolve_ctas = (int)(max_units < dev->sms ? max_units : dev->sms);
    specv_ring_resolve<kBF16><<<resolve_ctas, kRingResolveThreads, sizeof(RingResolveShared), stream>>>(
        in, sc, accepted_len, emitted_tokens, row_status, diag_p_tok, diag_q_tok, NextLookahead{nullptr, 0, 0});
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cuda_ok(cudaGetLastError()) ? SPECV_OK : SPECV_ERR_CUDA;
}

// Status word of the LM-head kernels of the last spec_verify_from_hidden call on this workspace
// (0: no bounded wait expired).  Reads device memory: waits for the stream's work first.
extern "C" int spec_verify_from_hidden_status(const void* workspace, int32_t B, int64_t n_draft_total, int64_t V,
                                              void* cuda_stream) {
    if (!workspace || !shape_ok(B, n_draft_total, V)) return -1;
    const HiddenLayout hl = hidden_layout(B, n_draft_total, V);
    int32_t v = 0;
    if (!cuda_ok(cudaMemcpyAsync(&v, static_cast<const char*>(workspace) + hl.status, 4, cudaMemcpyDeviceToHost,
                                 static_cast<cudaStream_t>(cuda_stream))) ||
        !cuda_ok(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream))))
        return -2;
    return v;
}
