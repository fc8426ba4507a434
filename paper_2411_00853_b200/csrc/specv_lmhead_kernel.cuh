// The step in front of the verify pass, fused with its first half: the LM-head product
//   logits[r, v] = sum_k hidden[r, k] * weight[v, k]          (bf16 inputs, fp32 accumulation)
// on the fifth-generation tensor cores, with the row statistics of the verify pass computed in
// the epilogue while the accumulators are still on chip.  The paper's section "Speculative
// Sampling Results" has the target model score the drafted positions in one parallel pass whose
// output -- these logits -- is what the verify pass then reads; here the logits are written once
// (the resolve kernel re-reads the one or two rows per sequence a token is drawn from) and never
// read back for the statistics.
//
//   one persistent CTA per SM, 6 warps:
//     warp 0     TMA producer: per k-block a 128 x 64 tile of hidden and a 256 x 64 tile of weight
//                (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into a 4-stage ring
//     warp 1     MMA issuer: tcgen05.mma (cta_group::1, kind::f16, M 128 x N 256 x K 16) from the shared
//                memory descriptors into one of two 256-column accumulators in tensor memory;
//                tcgen05.commit hands smem stages back to the producer and accumulators to the epilogue
//     warps 2-5  epilogue: tcgen05.ld of the warp's 32 accumulator lanes (a thread = one output row),
//                rounding to bf16, the online (reference, sum) of 2^(x*c - ref) over the tile's columns
//                from the ROUNDED values (what the resolve kernel will read), logits stored, one
//                (reference, sum) per (row, column tile) stored
//   specv_merge_tile_stats then folds a row's column-tile partials into the four-slot format of the
//   ring kernels.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "specv_ring_kernels.cuh"

namespace specv {

constexpr int kLmBM = 128, kLmBN = 256, kLmBK = 64;          // CTA tile; BK * 2 bytes = one 128-byte swizzle row
constexpr int kLmStages = 4;
constexpr int kLmABytes = kLmBM * kLmBK * 2, kLmBBytes = kLmBN * kLmBK * 2;
constexpr int kLmStageBytes = kLmABytes + kLmBBytes;         // 48 KB
constexpr int kLmThreads = 192;
constexpr int kLmTmemCols = 512;                             // two accumulators of 256 fp32 columns
constexpr int kLmUmmaK = 16;

struct LmHeadShared {
    alignas(1024) unsigned char stage[kLmStages][kLmStageBytes];
    unsigned long long full_bar[kLmStages], empty_bar[kLmStages];
    unsigned long long acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int err;
};
static_assert(sizeof(LmHeadShared) <= 227 * 1024, "LmHeadShared exceeds the shared memory of one CTA");

// Instruction descriptor of tcgen05.mma kind::f16: fp32 accumulator, bf16 A and B, both K-major, N 256, M 128.
constexpr uint32_t kLmInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kLmBN >> 3) << 17) |
                                  ((uint32_t)(kLmBM >> 4) << 24);

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the 128-byte
// swizzle (what the TMA load writes): start address, leading offset 1 (unused for this layout),
// 1024 bytes between groups of eight rows, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t lm_smem_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    const uint32_t no_lane_off = 0;      // every accumulator lane is written
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(no_lane_off) : "memory");
}
// The barrier gets one arrival when every tcgen05.mma this thread has issued so far has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// hidden [M, H] and weight [V, H] through their tensor maps (boxes 64 x 128 and 64 x 256, 128-byte
// swizzle); row_scale[r] = log2(e) / T of row r's sequence; logits [M, ld_out] bf16 out;
// part [M, n_tiles_n] (reference, sum) out.  status[0] receives a non-zero code if a bounded wait expired.
__global__ void __launch_bounds__(kLmThreads, 1)
specv_lm_head(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, int64_t M,
              int64_t V, int64_t H, const float* __restrict__ row_scale, uint16_t* __restrict__ logits,
              int64_t ld_out, float2* __restrict__ part, int32_t* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    LmHeadShared& sh = *reinterpret_cast<LmHeadShared*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t tiles_m = (M + kLmBM - 1) / kLmBM, tiles_n = (V + kLmBN - 1) / kLmBN;
    const int64_t n_tiles = tiles_m * tiles_n;
    const int32_t k_blocks = (int32_t)((H + kLmBK - 1) / kLmBK);
    volatile int* err = &sh.err;

    if (tid < kLmStages) {
        mbar_init(smem_u32(&sh.full_bar[tid]), 1);
        mbar_init(smem_u32(&sh.empty_bar[tid]), 1);
    } else if (tid >= 32 && tid < 34) {
        mbar_init(smem_u32(&sh.acc_full[tid - 32]), 1);
        mbar_init(smem_u32(&sh.acc_empty[tid - 32]), 4);       // one arrival per epilogue warp
    } else if (tid == 64) {
        sh.err = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp == 1) {            // tensor memory: all 512 columns, allocated and freed by this warp
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sh.tmem_base)), "r"((uint32_t)kLmTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;    // k-blocks issued so far (stage = it % kLmStages)
            for (int64_t t = blockIdx.x; t < n_tiles && !*err; t += gridDim.x) {
                const int32_t m0 = (int32_t)(t % tiles_m) * kLmBM, n0 = (int32_t)(t / tiles_m) * kLmBN;
                for (int32_t kb = 0; kb < k_blocks; ++kb, ++it) {
                    const uint32_t s = it % kLmStages;
                    mbar_wait(smem_u32(&sh.empty_bar[s]), ((it / kLmStages) & 1) ^ 1, err, 91);
                    if (*err) break;
                    const uint32_t fb = smem_u32(&sh.full_bar[s]);
                    mbar_expect_tx(fb, kLmStageBytes);
                    tma_load_2d(smem_u32(&sh.stage[s][0]), &map_a, kb * kLmBK, m0, fb);
                    tma_load_2d(smem_u32(&sh.stage[s][kLmABytes]), &map_b, kb * kLmBK, n0, fb);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, tile_i = 0;
            for (int64_t t = blockIdx.x; t < n_tiles && !*err; t += gridDim.x, ++tile_i) {
                const uint32_t acc = tile_i & 1;
                mbar_wait(smem_u32(&sh.acc_empty[acc]), ((tile_i >> 1) & 1) ^ 1, err, 92);   // epilogue has drained it
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * kLmBN;
                for (int32_t kb = 0; kb < k_blocks && !*err; ++kb, ++it) {
                    const uint32_t s = it % kLmStages;
                    mbar_wait(smem_u32(&sh.full_bar[s]), (it / kLmStages) & 1, err, 93);
                    if (*err) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t da = lm_smem_desc(smem_u32(&sh.stage[s][0]));
                    const uint64_t db = lm_smem_desc(smem_u32(&sh.stage[s][kLmABytes]));
#pragma unroll
                    for (int kk = 0; kk < kLmBK / kLmUmmaK; ++kk)      // 32 bytes along K per instruction
                        umma_bf16(d_tmem, da + (uint64_t)(kk * kLmUmmaK * 2 >> 4), db + (uint64_t)(kk * kLmUmmaK * 2 >> 4),
                                  kLmInstrDesc, (kb | kk) != 0);
                    umma_commit(smem_u32(&sh.empty_bar[s]));           // the stage is free once these have read it
                }
                umma_commit(smem_u32(&sh.acc_full[acc]));              // the accumulator is complete
            }
        }
    } else {
        // epilogue: a warp may touch the 32 tensor-memory lanes 32 * (warp % 4) ..
        const int q = warp & 3;
        uint32_t tile_i = 0;
        for (int64_t t = blockIdx.x; t < n_tiles && !*err; t += gridDim.x, ++tile_i) {
            const uint32_t acc = tile_i & 1;
            const int64_t m0 = (t % tiles_m) * kLmBM, n0 = (t / tiles_m) * kLmBN;
            const int64_t r = m0 + q * 32 + lane;
            const bool row_ok = r < M;
            const float c = row_ok ? row_scale[r] : 1.0f;
            mbar_wait(smem_u32(&sh.acc_full[acc]), (tile_i >> 1) & 1, err, 94);
            if (*err) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float ref = kNoMax, sum = 0.f;
            uint16_t* out_row = logits + (row_ok ? r : 0) * ld_out;
#pragma unroll 1
            for (int ch = 0; ch < kLmBN / 32; ++ch) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * kLmBN + ch * 32, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int64_t col0 = n0 + ch * 32;
                uint32_t w[16];
                float x[32];
                float mx = __uint_as_float(0xff800000u);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    w[j] = cvt_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                    x[2 * j] = col0 + 2 * j < V ? __uint_as_float(w[j] << 16) : __uint_as_float(0xff800000u);
                    x[2 * j + 1] = col0 + 2 * j + 1 < V ? __uint_as_float(w[j] & 0xffff0000u) : __uint_as_float(0xff800000u);
                    mx = fmaxf(mx, fmaxf(x[2 * j], x[2 * j + 1]));
                }
                const float cand = mx * c;
                if (cand > ref) {
                    sum *= ex2_approx(ref - cand);
                    ref = cand;
                }
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    s0 += ex2_approx(fmaf(x[j], c, -ref));
                    s1 += ex2_approx(fmaf(x[j + 1], c, -ref));
                }
                sum += s0 + s1;
                if (row_ok) {
                    if (col0 + 32 <= V && ((reinterpret_cast<uintptr_t>(out_row + col0) & 15u) == 0)) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            *reinterpret_cast<uint4*>(out_row + col0 + 8 * j) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col0 + j < V) out_row[col0 + j] = (uint16_t)((j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xffffu));
                    }
                }
            }
            if (row_ok) part[r * tiles_n + (t / tiles_m)] = make_float2(ref, sum);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.acc_empty[acc]));
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kLmTmemCols) : "memory");
    }
    if (tid == 0 && sh.err) {
        // a wait gave up: copies already issued may still be landing in this CTA's shared memory;
        // give them time before the memory can go to another CTA
        const long long t0 = clock64();
        while (clock64() - t0 < 200000) {}
        atomicExch(status, sh.err);
    }
}

// Temperature constant of every logits row: c[row] = log2(e) / T of the row's sequence, for the
// target rows (packed as in spec_verify) followed by the draft rows.
__global__ void specv_row_scales(BatchView in, const int32_t* __restrict__ off_d, float* __restrict__ c_target,
                                 float* __restrict__ c_draft) {
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the offsets come from the prologue
    const int64_t n_target = in.n_draft_total + in.B;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_target + in.n_draft_total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const bool is_t = i < n_target;
        const int32_t b = is_t ? seq_of_target_row(off_d, in.B, i) : seq_of_draft_row(off_d, in.B, i - n_target);
        const float T = in.temperature[in.per_row_temperature ? b : 0];
        const float c = (T > 0.0f && !isinf(T)) ? (float)(kLog2e / (double)T) : 1.0f;     // a bad T is reported by the prologue
        if (is_t) c_target[i] = c; else c_draft[i - n_target] = c;
    }
}

// One warp per logits row: the column-tile partials of the row, merged in tile order into slot 0 of
// the ring kernels' four-slot statistics (the other slots blank).
__global__ void specv_merge_tile_stats(const float2* __restrict__ part, int64_t rows, int64_t tiles_n,
                                       float2* __restrict__ stat) {
    const int lane = threadIdx.x & 31;
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= rows) return;
    float ref = kNoMax, sum = 0.f;
    for (int64_t i = lane; i < tiles_n; i += 32) {
        const float2 p = part[row * tiles_n + i];
        merge_ref_sum(ref, sum, p.x, p.y);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        merge_ref_sum(ref, sum, __shfl_xor_sync(0xffffffffu, ref, o), __shfl_xor_sync(0xffffffffu, sum, o));
    if (lane == 0) {
        stat[row * kStatParts] = make_float2(ref, sum);
        for (int e = 1; e < kStatParts; ++e) stat[row * kStatParts + e] = make_float2(kNoMax, 0.f);
    }
}

}  // namespace specv
