// After the verification pass: which draft nodes the target keeps (greedy, temperature 0), and
// the move of their K/V rows to the front of the draft block (Appendix A: the target verifies the
// draft tree in one forward pass and keeps exactly what it would have produced itself).
// Integer work, bit-exact; a few microseconds of latency, no bandwidth to speak of.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace sparrow {

// One thread per sequence: parents[i] < i, so one pass in node order settles every node.
// accepted(i) = (root or accepted(parent)) and draft[i] == target_next[parent + 1].
// The deepest accepted node wins, the smallest index among equals.  path[0 .. n) = its chain
// from the root down, path[n .. T) = -1; bonus = target_next[last + 1] (target_next[0] if none).
// A parent outside [-1, i) sets the tree status bit and counts as "root".
__global__ void __launch_bounds__(kMaxBatch)
accept_greedy_kernel(const int32_t* __restrict__ draft_tokens, const int32_t* __restrict__ parents,
                     const int32_t* __restrict__ target_next, int batch, int T, int32_t* __restrict__ path,
                     int32_t* __restrict__ n_accept, int32_t* __restrict__ bonus, unsigned* status)
{
    const int b = threadIdx.x;
    if (b >= batch) return;
    const int32_t* tok = draft_tokens + (size_t)b * T;
    const int32_t* par = parents + (size_t)b * T;
    const int32_t* nxt = target_next + (size_t)b * (T + 1);
    unsigned long long acc = 0ull;              // bit i: node i accepted
    unsigned char depth[kMaxT];
    int best = -1, best_depth = 0;
    for (int i = 0; i < T; ++i) {
        int p = par[i];
        if (p < -1 || p >= i) { atomicOr(status, kStatTree); p = -1; }
        const bool ok = (p < 0 || ((acc >> p) & 1ull)) && tok[i] == nxt[p + 1];
        const int d = ok ? (p < 0 ? 1 : depth[p] + 1) : 0;
        depth[i] = (unsigned char)d;
        if (ok) acc |= 1ull << i;
        if (d > best_depth) { best_depth = d; best = i; }
    }
    int32_t* out = path + (size_t)b * T;
    for (int i = best_depth; i < T; ++i) out[i] = -1;
    int node = best;
    for (int i = best_depth - 1; i >= 0; --i) {
        out[i] = node;
        const int p = par[node];
        node = (p < -1 || p >= node) ? -1 : p;
    }
    n_accept[b] = best_depth;
    bonus[b] = nxt[best + 1];
}

struct KeepArgs {
    __nv_bfloat16* k;
    __nv_bfloat16* v;
    const int32_t* path;             // DEV [batch][T]
    const int32_t* n_accept;         // DEV [batch]
    int32_t T, n_kv_heads;
    int64_t stride_batch, stride_head;
    int32_t kv_len[kMaxBatch];
};

// One CTA per (sequence, KV head): rows kv_len + path[i] -> rows kv_len + i, i < n_accept.  The
// move is in place and sources and destinations overlap, so every row is read into shared
// memory before any is written.  256 threads, 16 per row and pass.
__global__ void __launch_bounds__(256)
keep_accepted_rows_kernel(const __grid_constant__ KeepArgs a)
{
    extern __shared__ uint4 rows_sm[];                       // [2][T][16] chunks of 16 bytes
    const int b = blockIdx.x / a.n_kv_heads, h = blockIdx.x % a.n_kv_heads;
    int n = a.n_accept[b];
    n = n < 0 ? 0 : (n > a.T ? a.T : n);
    const size_t base = (size_t)b * a.stride_batch + (size_t)h * a.stride_head + (size_t)a.kv_len[b] * kD;
    for (int e = threadIdx.x; e < n * 16; e += blockDim.x) {
        const int i = e >> 4, c = e & 15;
        int src = a.path[(size_t)b * a.T + i];
        src = src < 0 ? 0 : (src >= a.T ? a.T - 1 : src);   // (a well-formed path never needs this)
        rows_sm[e] = *reinterpret_cast<const uint4*>(a.k + base + (size_t)src * kD + c * 8);
        rows_sm[a.T * 16 + e] = *reinterpret_cast<const uint4*>(a.v + base + (size_t)src * kD + c * 8);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n * 16; e += blockDim.x) {
        const int i = e >> 4, c = e & 15;
        *reinterpret_cast<uint4*>(a.k + base + (size_t)i * kD + c * 8) = rows_sm[e];
        *reinterpret_cast<uint4*>(a.v + base + (size_t)i * kD + c * 8) = rows_sm[a.T * 16 + e];
    }
}

}  // namespace sparrow
