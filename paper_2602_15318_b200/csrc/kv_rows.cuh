// Row movers around the two attention modes: appending the draft tokens' K/V rows to a cache,
// and compacting the text-anchored rows of a long cache into a short contiguous one (Section 3.1:
// the draft model keeps only the text-anchored states and discards the visual KV cache), after
// which the anchored mode is an ordinary contiguous stream for the tensor-core kernel.
//
// One thread moves 16 bytes; 16 consecutive threads move one 256-byte row of K and the same row
// of V.  Pure copies: results are bit-exact.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace sparrow {

struct RowMoveArgs {
    const __nv_bfloat16* k_src;
    const __nv_bfloat16* v_src;
    __nv_bfloat16* k_dst;
    __nv_bfloat16* v_dst;
    const int32_t* src_rows;         // DEV [batch][n_rows] source row of each moved row, or nullptr: rows 0 .. n_rows-1
    int32_t n_rows;                  // rows moved per (sequence, KV head)
    int32_t batch, n_kv_heads;
    int32_t src_capacity;            // valid source rows are [0, src_capacity)
    int64_t src_stride_batch, src_stride_head;      // in elements
    int64_t dst_stride_batch, dst_stride_head;
    int32_t dst_row0[kMaxBatch];     // first destination row per sequence
    unsigned* status;
};

// Moves 16 bytes of K and of V: chunk i of the (sequence, KV head, row, 16-byte column) index space.
__device__ __forceinline__ void move_row_chunk(const RowMoveArgs& a, long long i)
{
    const int c = (int)(i & 15);
    long long rest = i >> 4;
    const int r = (int)(rest % a.n_rows); rest /= a.n_rows;
    const int h = (int)(rest % a.n_kv_heads);
    const int b = (int)(rest / a.n_kv_heads);
    int src = a.src_rows ? __ldg(a.src_rows + (size_t)b * a.n_rows + r) : r;
    const bool bad = src < 0 || src >= a.src_capacity;       // never read: the row is written as zeros
    if (bad && c == 0 && h == 0) atomicOr(a.status, kStatAnchor);
    const size_t s_off = (size_t)b * a.src_stride_batch + (size_t)h * a.src_stride_head + (size_t)(bad ? 0 : src) * kD + c * 8;
    const size_t d_off = (size_t)b * a.dst_stride_batch + (size_t)h * a.dst_stride_head +
                         (size_t)(a.dst_row0[b] + r) * kD + c * 8;
    uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
    if (!bad) {
        kv = *reinterpret_cast<const uint4*>(a.k_src + s_off);
        vv = *reinterpret_cast<const uint4*>(a.v_src + s_off);
    }
    *reinterpret_cast<uint4*>(a.k_dst + d_off) = kv;
    *reinterpret_cast<uint4*>(a.v_dst + d_off) = vv;
}

__global__ void __launch_bounds__(256)
move_rows_kernel(const __grid_constant__ RowMoveArgs a)
{
    const long long total = (long long)a.batch * a.n_kv_heads * a.n_rows * 16;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
        move_row_chunk(a, i);
}

// One step's inputs straight from host memory that the GPU can address (pinned or registered):
// the queries and the tree go to device staging (the attention kernel fetches the queries by TMA),
// the draft tokens' K/V rows go to their cache rows.  One 16-byte load per thread and buffer, all
// in flight together, so the launch costs about one round trip over the host link.
struct IngestArgs {
    RowMoveArgs rows;                // k_src / v_src are host memory here
    const uint4* q_src;              // host view
    uint4* q_dst;
    const int32_t* parents_src;      // host view
    int32_t* parents_dst;
    int32_t q_chunks, n_parents;
};

__global__ void __launch_bounds__(256)
ingest_step_kernel(const __grid_constant__ IngestArgs a)
{
    const long long row_chunks = (long long)a.rows.batch * a.rows.n_kv_heads * a.rows.n_rows * 16;
    const long long total = row_chunks + a.q_chunks + a.n_parents;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        if (i < row_chunks) move_row_chunk(a.rows, i);
        else if (i < row_chunks + a.q_chunks) a.q_dst[i - row_chunks] = a.q_src[i - row_chunks];
        else a.parents_dst[i - row_chunks - a.q_chunks] = a.parents_src[i - row_chunks - a.q_chunks];
    }
}

}  // namespace sparrow
