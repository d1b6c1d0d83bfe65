// Split-combine step: merges the per-piece partial outputs of the split-KV pass by log-sum-exp,
//     lse = log sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * o_s,
// (partials are fp16, normalised, so their magnitude is bounded by max |v|) and writes bf16 out [B][T][Hq][128] and fp32 lse [B][Hq][T].  Pieces that saw no visible key
// carry lse_s = -inf and weigh zero; a row with no visible key anywhere gets out = 0, lse = -inf.
//
// One CTA of 4 warps per packed query row.  The piece LSEs go to shared memory with one read per
// thread; warp w then accumulates pieces w, w+4, ... (each lane owns 4 of the 128 output dims, all
// its loads issued before the first use), and the four warp sums are added through shared memory.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace sparrow {

struct CombineArgs {
    const __half* o_part;       // [n_items][part_rows][128] normalised partial outputs (fp16)
    const float* lse_part;
    __nv_bfloat16* out;
    float* lse;
    int32_t n_q_heads;
    int32_t use_pdl;      // 1: launched with programmatic stream serialisation
};

namespace combine {

constexpr int kWarps = 4;
constexpr int kMaxPieces = 1024;       // upper bound on pieces per row held in shared memory

__global__ void __launch_bounds__(kWarps * 32)
combine_kernel(const __grid_constant__ SplitPlan plan, const __grid_constant__ CombineArgs args)
{
    __shared__ float lse_s[kMaxPieces];
    __shared__ float4 acc_s[kWarps][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row_id = blockIdx.x;
    const int R = row_id % plan.M;                    // packed row: t*7 + g
    const int unit_bh = row_id / plan.M;
    const int kvh = unit_bh % plan.n_kv_heads;
    const int b = unit_bh / plan.n_kv_heads;
    const int group = R / plan.rows_per_group;
    const int lr = R % plan.rows_per_group;
    const int ns = plan.n_splits[b];
    const int item0 = plan.item_begin[b] + (kvh * plan.n_groups + group) * ns;
    if (args.use_pdl) {
        asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
    }
    if (ns == 1) return;                              // the split pass wrote this row's result itself
    for (int s = threadIdx.x; s < ns; s += kWarps * 32)
        lse_s[s] = args.lse_part[(size_t)(item0 + s) * plan.part_rows + lr];
    __syncthreads();
    float mx = -INFINITY;
    for (int s = lane; s < ns; s += 32) mx = fmaxf(mx, lse_s[s]);
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    float sum = 0.f;
    if (mx != -INFINITY)
        for (int s = lane; s < ns; s += 32) sum += expf(lse_s[s] - mx);
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
    const float total = (mx == -INFINITY) ? -INFINITY : mx + logf(sum);

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (mx != -INFINITY) {
        constexpr int kBatch = 8;
        for (int s0 = warp; s0 < ns; s0 += kWarps * kBatch) {
            uint2 o[kBatch];                                   // 4 halves per lane and piece
            #pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int s = s0 + u * kWarps;
                if (s < ns)
                    o[u] = __ldcg(reinterpret_cast<const uint2*>(
                        args.o_part + ((size_t)(item0 + s) * plan.part_rows + lr) * kD + lane * 4));
            }
            #pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int s = s0 + u * kWarps;
                if (s < ns) {
                    const float w = expf(lse_s[s] - total);
                    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&o[u].x));
                    const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&o[u].y));
                    acc.x = fmaf(w, a.x, acc.x); acc.y = fmaf(w, a.y, acc.y);
                    acc.z = fmaf(w, c.x, acc.z); acc.w = fmaf(w, c.y, acc.w);
                }
            }
        }
    }
    acc_s[warp][lane] = acc;
    __syncthreads();
    if (warp == 0) {
        #pragma unroll
        for (int w = 1; w < kWarps; ++w) {
            const float4 o = acc_s[w][lane];
            acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
        }
        const int t = R / kGroup, g = R % kGroup;
        const int h = kvh * kGroup + g;
        __nv_bfloat16* dst = args.out + (((size_t)b * plan.T + t) * args.n_q_heads + h) * kD + lane * 4;
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t*>(&lo);
        packed.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(dst) = packed;
        if (lane == 0) args.lse[((size_t)b * args.n_q_heads + h) * plan.T + t] = total;
    }
}

}  // namespace combine
}  // namespace sparrow
