// Split-combine step: merges the per-piece partial outputs of the split-KV pass by log-sum-exp,
//     lse = log sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * o_s,
// (partials are fp16, normalised, so their magnitude is bounded by max |v|) and writes bf16 out
// [B][T][Hq][128] and fp32 lse [B][Hq][T].  Pieces that saw no visible key carry lse_s = -inf and
// weigh zero; a row with no visible key anywhere gets out = 0, lse = -inf.
//
// One warp per query row, registers and shuffles only, so the same routine serves the finisher
// CTAs of the fused split-KV kernel (whose shared memory is taken) and the stand-alone combine
// kernel of the stream-ordered mode.  Lane l keeps the LSEs of pieces
// l, l+32, ...  The four quarter-warps take pieces q, q+4, q+8, ...; inside a quarter each of the 8
// lanes owns 16 of the 128 output dims (two 16-byte loads per piece), and the quarters' sums meet
// through two shuffle steps.  The code is kept small on purpose: every warp runs it exactly once,
// so instruction fetch, not arithmetic, is what a long unrolled body would pay for.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace sparrow {

struct CombineArgs {
    const __half* o_part;       // [n_items][part_rows] partial rows: 128 fp16 outputs + fp32 LSE (kPartRowHalves)
    __nv_bfloat16* out;
    float* lse;
    int32_t n_q_heads;
};

namespace combine {

constexpr int kWarps = 4;             // rows per CTA
constexpr int kPerLane = 8;           // pieces per lane held in registers (256 pieces per row)
constexpr int kIter = 5;              // pieces per quarter-warp fetched in one go (20 per warp pass)

__device__ __forceinline__ void fma8(float (&acc)[16], int base, float w, const uint4& v)
{
    const __half2* h = reinterpret_cast<const __half2*>(&v);
    #pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        acc[base + 2 * i] = fmaf(w, f.x, acc[base + 2 * i]);
        acc[base + 2 * i + 1] = fmaf(w, f.y, acc[base + 2 * i + 1]);
    }
}

// Merges the pieces of one (sequence b, KV head, draft token t, head g of the group) row; called
// by all 32 lanes of a warp.
__device__ __forceinline__ void combine_row(const SplitPlan& plan, const CombineArgs& args, int b, int kvh, int t, int g, int lane)
{
    const int block = t / plan.tok_per_block;               // 128-row block holding this token
    const int group = block / plan.blocks_per_group;
    const int lr = (block - group * plan.blocks_per_group) * kBlockRows + (t - block * plan.tok_per_block) * plan.group + g;
    const int ns = plan.seq[b].n_splits;
    if (ns == 1) return;                              // the split pass wrote this row's result itself
    const int item0 = plan.seq[b].item_begin + (kvh * plan.n_groups + group) * ns;
    const size_t lse_pitch = (size_t)plan.part_rows * (kPartRowHalves / 2);          // floats between pieces
    const float* lse_row = reinterpret_cast<const float*>(args.o_part + ((size_t)item0 * plan.part_rows + lr) * kPartRowHalves + kD);
    const int quarter = lane >> 3, sub = lane & 7;
    const __half* o_row = args.o_part + ((size_t)item0 * plan.part_rows + lr) * kPartRowHalves + sub * 16;
    const size_t o_pitch = (size_t)plan.part_rows * kPartRowHalves;

    // first pass of partial loads goes out together with the LSE loads (they are independent)
    uint4 o0[kIter], o1[kIter];
    #pragma unroll
    for (int i = 0; i < kIter; ++i) {
        const int s = 4 * i + quarter;
        if (s < ns) {
            const uint4* src = reinterpret_cast<const uint4*>(o_row + (size_t)s * o_pitch);
            o0[i] = __ldcg(src); o1[i] = __ldcg(src + 1);
        }
    }
    float lv[kPerLane];
    #pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        const int s = lane + 32 * i;
        lv[i] = s < ns ? __ldcg(lse_row + (size_t)s * lse_pitch) : -INFINITY;
    }
    float mx = -INFINITY;
    #pragma unroll
    for (int i = 0; i < kPerLane; ++i) mx = fmaxf(mx, lv[i]);
    for (int s = lane + 32 * kPerLane; s < ns; s += 32) mx = fmaxf(mx, __ldcg(lse_row + (size_t)s * lse_pitch));
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    const bool any = mx != -INFINITY;
    float sum = 0.f;
    #pragma unroll
    for (int i = 0; i < kPerLane; ++i) sum += any ? __expf(lv[i] - mx) : 0.f;        // 0 for absent pieces
    for (int s = lane + 32 * kPerLane; s < ns; s += 32) sum += any ? __expf(__ldcg(lse_row + (size_t)s * lse_pitch) - mx) : 0.f;
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
    const float total = any ? mx + logf(sum) : -INFINITY;
    #pragma unroll
    for (int i = 0; i < kPerLane; ++i) lv[i] = any ? __expf(lv[i] - total) : 0.f;     // now the weights

    float acc[16];
    #pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    #pragma unroll 1
    for (int s0 = 0; s0 < ns; s0 += 4 * kIter) {                 // warp-uniform trip count
        if (s0 > 0) {
            #pragma unroll
            for (int i = 0; i < kIter; ++i) {
                const int s = s0 + 4 * i + quarter;
                if (s < ns) {
                    const uint4* src = reinterpret_cast<const uint4*>(o_row + (size_t)s * o_pitch);
                    o0[i] = __ldcg(src); o1[i] = __ldcg(src + 1);
                }
            }
        }
        #pragma unroll
        for (int i = 0; i < kIter; ++i) {
            const int s = s0 + 4 * i + quarter;
            // weight of piece s lives in lane s & 31, register s >> 5 (the same register for all quarters)
            const int reg = (s0 + 4 * i) >> 5;
            float mine = 0.f;
            #pragma unroll
            for (int k = 0; k < kPerLane; ++k) if (reg == k) mine = lv[k];
            float w = __shfl_sync(0xffffffffu, mine, s & 31);
            if (reg >= kPerLane && s < ns) w = any ? __expf(__ldcg(lse_row + (size_t)s * lse_pitch) - total) : 0.f;
            if (s < ns) { fma8(acc, 0, w, o0[i]); fma8(acc, 8, w, o1[i]); }
        }
    }
    #pragma unroll
    for (int i = 0; i < 16; ++i) {
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 8);
        acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 16);
    }
    if (quarter == 0) {
        const int h = kvh * plan.group + g;
        __nv_bfloat16* dst = args.out + (((size_t)b * plan.T + t) * args.n_q_heads + h) * kD + sub * 16;
        uint4 pk[2];
        uint32_t* w32 = reinterpret_cast<uint32_t*>(pk);
        #pragma unroll
        for (int i = 0; i < 8; ++i) {
            __nv_bfloat162 v = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
            w32[i] = *reinterpret_cast<uint32_t*>(&v);
        }
        reinterpret_cast<uint4*>(dst)[0] = pk[0];
        reinterpret_cast<uint4*>(dst)[1] = pk[1];
        if (lane == 0) args.lse[((size_t)b * args.n_q_heads + h) * plan.T + t] = total;
    }
}

// The stand-alone combine kernel of the stream-ordered mode: grid-stride over the rows, one warp
// per row, launched behind the split-KV kernel (ordinarily, or programmatically in anchored mode).
__global__ void __launch_bounds__(kWarps * 32)
combine_kernel(const __grid_constant__ SplitPlan plan, const __grid_constant__ CombineArgs args)
{
    // Launched programmatically behind the split-KV kernel it may start early: wait for that grid
    // to complete (with its writes visible).  Without a programmatic dependency this returns at once.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows_total = plan.batch * plan.n_kv_heads * plan.M;
    for (int row_id = blockIdx.x * kWarps + warp; row_id < rows_total; row_id += gridDim.x * kWarps) {
        const int R = row_id % plan.M, unit_bh = row_id / plan.M;
        combine_row(plan, args, unit_bh / plan.n_kv_heads, unit_bh % plan.n_kv_heads, R / plan.group, R % plan.group, lane);
    }
}

}  // namespace combine
}  // namespace sparrow
