// Split-combine step: merges the per-piece partial outputs of the split-KV pass by log-sum-exp,
//     lse = log sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * o_s,
// and writes bf16 out [B][T][Hq][128] and fp32 lse [B][Hq][T].  Pieces that saw no visible key
// carry lse_s = -inf and weigh zero; a row with no visible key anywhere gets out = 0, lse = -inf.
// One warp per packed query row; each lane owns 4 of the 128 output dims.
#pragma once
#include "common.cuh"

namespace sparrow {

struct CombineArgs {
    const float* o_part;
    const float* lse_part;
    __nv_bfloat16* out;
    float* lse;
    int32_t n_q_heads;
    int32_t use_pdl;      // 1: launched with programmatic stream serialisation
};

namespace combine {

constexpr int kWarps = 4;

__global__ void __launch_bounds__(kWarps * 32)
combine_kernel(const __grid_constant__ SplitPlan plan, const __grid_constant__ CombineArgs args)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows_total = plan.batch * plan.n_kv_heads * plan.M;
    const int row_id = blockIdx.x * kWarps + warp;
    if (args.use_pdl) {
        asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
    }
    if (row_id >= rows_total) return;
    const int R = row_id % plan.M;                    // packed row: t*7 + g
    const int unit_bh = row_id / plan.M;
    const int kvh = unit_bh % plan.n_kv_heads;
    const int b = unit_bh / plan.n_kv_heads;
    const int group = R / plan.rows_per_group;
    const int lr = R % plan.rows_per_group;
    const int ns = plan.n_splits[b];
    const int item0 = plan.item_begin[b] + (kvh * plan.n_groups + group) * ns;

    float mx = -INFINITY;
    for (int s = lane; s < ns; s += 32)
        mx = fmaxf(mx, args.lse_part[(size_t)(item0 + s) * plan.part_rows + lr]);
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    float sum = 0.f;
    if (mx != -INFINITY)
        for (int s = lane; s < ns; s += 32)
            sum += expf(args.lse_part[(size_t)(item0 + s) * plan.part_rows + lr] - mx);
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
    const float total = (mx == -INFINITY) ? -INFINITY : mx + logf(sum);

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (mx != -INFINITY) {
        #pragma unroll 4
        for (int s = 0; s < ns; ++s) {
            const size_t prow = (size_t)(item0 + s) * plan.part_rows + lr;
            const float w = expf(args.lse_part[prow] - total);
            const float4 o = *reinterpret_cast<const float4*>(args.o_part + prow * kD + lane * 4);
            acc.x = fmaf(w, o.x, acc.x); acc.y = fmaf(w, o.y, acc.y);
            acc.z = fmaf(w, o.z, acc.z); acc.w = fmaf(w, o.w, acc.w);
        }
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

}  // namespace combine
}  // namespace sparrow
