// Lower window bound of the text-anchored mode on a compacted cache (Eq. 2 with the window rule
// "query at row qpos sees text anchor p iff qpos - window < p"): the anchors are strictly
// increasing, so the visible text anchors of a query are a contiguous run of the compacted cache
// and one index per query -- its first visible compact row -- describes it.
#pragma once
#include "common.cuh"

namespace sparrow {

// First index j in [0, n_text) with anchor[j] > bound (n_text if none); at most 32 halvings.
__host__ __device__ __forceinline__ int first_anchor_above(const int32_t* anchor, int n_text, long long bound)
{
    int lo = 0, hi = n_text;
    for (int step = 0; step < 32 && lo < hi; ++step) {
        const int mid = lo + (hi - lo) / 2;
        if ((long long)anchor[mid] > bound) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// One thread per (sequence, query token).  anchor_idx [B][n_anchor]: text anchors first, then the
// T_tree rows of the draft tree; the queries are its last T_new nodes.
__global__ void window_bounds_kernel(const int32_t* __restrict__ anchor_idx, int n_anchor, int window, int T_tree, int T_new,
                                     int batch, int32_t* __restrict__ first_visible)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch * T_new) return;
    const int b = i / T_new, t = i - b * T_new;
    const int32_t* a = anchor_idx + (size_t)b * n_anchor;
    const int n_text = n_anchor - T_tree;
    int first = 0;
    if (window > 0) first = first_anchor_above(a, n_text, (long long)a[n_anchor - T_new + t] - window);
    first_visible[i] = first;
}

}  // namespace sparrow
