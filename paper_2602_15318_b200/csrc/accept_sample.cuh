// Acceptance at temperature 1: multi-round rejection sampling over the draft tree (Appendix A: the
// verification keeps the target's output distribution exactly; the paper relies on the standard
// procedure).  At the current node, with target distribution p and draft distribution q, the
// children are tried in index order; a child with token x is accepted with probability
// min(1, p(x) / q(x)); after a rejection p becomes the normalised positive part of (p - q), and q
// loses x (the siblings were drawn without replacement); when no child is accepted the next token
// is drawn from what p has become.
//
// The results are integers (accepted path, bonus token), so the arithmetic is integer too:
// probabilities are rounded once to 30-bit fixed point, P = floor(p 2^30 + 1/2), and with A = sum P,
// B = sum Q and a 32-bit uniform r
//     accept x          iff  Q[x] > 0 and r Q[x] A < P[x] B 2^32               (128-bit products)
//     after a rejection      P <- max(B P - A Q, 0) >> 30 (unless B == 0), A <- sum P, B <- B - Q[x], Q[x] <- 0
//     bonus                  the smallest v with P[0] + ... + P[v] > (r A) >> 32, P being the row's
//                            original target row again if A == 0.
// Integer sums do not depend on the order of summation, so any parallel reduction gives the same
// bits.  The residual rows are never stored: element v of the current P is recomputed from the two
// input rows and the level's short history of (A, B, x) triples.
//
// One CTA per sequence; every step is a pass of the whole CTA over the V entries of two rows.
#pragma once
#include "common.cuh"

namespace sparrow {
namespace sample {

constexpr int kThreads = 1024;
constexpr int kProbBits = 30;

__device__ __forceinline__ long long fixed_prob(float p)
{
    // exact in double for p in [0, 1]; anything else (NaN, negative, > 1) is clamped into the range
    const double d = (double)(p > 0.f ? (p < 1.f ? p : 1.f) : 0.f);
    return __double2ll_rd(d * 1073741824.0 + 0.5);
}

struct Level {                      // history of the rejections at the current node
    long long A[kMaxT], B[kMaxT];
    int x[kMaxT];
    int n;
};

// Current residual target weight and current draft weight of vocabulary entry v.
__device__ __forceinline__ void weights_at(const float* __restrict__ pt, const float* __restrict__ pq, int v, const Level& lv,
                                           long long* P_out, long long* Q_out)
{
    long long P = fixed_prob(pt[v]);
    const long long q0 = fixed_prob(pq[v]);
    bool gone = false;               // v was a rejected candidate: the draft distribution has lost it
    for (int s = 0; s < lv.n; ++s) {
        const long long Q = gone ? 0ll : q0;
        if (lv.B[s] > 0) {
            const long long d = lv.B[s] * P - lv.A[s] * Q;
            P = d > 0 ? d >> kProbBits : 0ll;
        }
        if (v == lv.x[s]) gone = true;
    }
    *P_out = P;
    *Q_out = gone ? 0ll : q0;
}

__device__ __forceinline__ long long block_sum(long long v, long long* scratch /*[32]*/)
{
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                                           // scratch may still be read from the call before
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    long long t = 0;
    for (int w = 0; w < kThreads / 32; ++w) t += scratch[w];   // same order in every thread
    return t;
}

__global__ void __launch_bounds__(kThreads)
accept_sample_kernel(const int32_t* __restrict__ draft_tokens, const int32_t* __restrict__ parents,
                     const float* __restrict__ p_target, const float* __restrict__ p_draft,
                     const uint32_t* __restrict__ u_node, const uint32_t* __restrict__ u_bonus, int T, int V,
                     int32_t* __restrict__ path, int32_t* __restrict__ n_accept, int32_t* __restrict__ bonus, unsigned* status)
{
    __shared__ Level lv;
    __shared__ int32_t tok_s[kMaxT], par_s[kMaxT];
    __shared__ long long red[32], red2[32];
    __shared__ long long chunk_sum[kThreads];
    __shared__ int found_v;
    const int b = blockIdx.x, tid = threadIdx.x;
    if (tid < T) {
        tok_s[tid] = draft_tokens[(size_t)b * T + tid];
        int p = parents[(size_t)b * T + tid];
        if (p < -1 || p >= tid) { atomicOr(status, kStatTree); p = -1; }
        par_s[tid] = p;
    }
    __syncthreads();
    int cur = -1, n_acc = 0;
    int32_t* out = path + (size_t)b * T;
    #pragma unroll 1
    for (int level = 0; level <= T; ++level) {
        const size_t row = (size_t)b * (T + 1) + (size_t)(cur + 1);
        const float* pt = p_target + row * V;
        const float* pq = p_draft + row * V;
        if (tid == 0) lv.n = 0;
        long long a = 0, q = 0;
        for (int v = tid; v < V; v += kThreads) { a += fixed_prob(pt[v]); q += fixed_prob(pq[v]); }
        long long A = block_sum(a, red), Bq = block_sum(q, red2);
        int taken = -1;
        #pragma unroll 1
        for (int c = cur + 1; c < T && taken < 0; ++c) {          // children of cur, in index order
            if (par_s[c] != cur) continue;
            const int x = tok_s[c];
            long long Px = 0, Qx = 0;
            if (x >= 0 && x < V) weights_at(pt, pq, x, lv, &Px, &Qx);
            else if (tid == 0) atomicOr(status, kStatTree);        // a token outside the vocabulary is never accepted
            const unsigned __int128 lhs = (unsigned __int128)u_node[(size_t)b * T + c] * (unsigned long long)Qx * (unsigned long long)A;
            const unsigned __int128 rhs = ((unsigned __int128)(unsigned long long)Px * (unsigned long long)Bq) << 32;
            if (Qx > 0 && lhs < rhs) { taken = c; break; }
            // rejected: the level's history grows by (A, B, x); the new A is the sum of the new residual
            __syncthreads();                                       // everybody has read the history as it was
            if (tid == 0) { lv.A[lv.n] = A; lv.B[lv.n] = Bq; lv.x[lv.n] = (x >= 0 && x < V) ? x : -1; lv.n += 1; }
            __syncthreads();
            if (Bq > 0) {
                long long s = 0;
                for (int v = tid; v < V; v += kThreads) {
                    long long P, Q;
                    weights_at(pt, pq, v, lv, &P, &Q);
                    s += P;
                }
                A = block_sum(s, red);
            }
            Bq -= Qx;
        }
        if (taken >= 0) {
            if (tid == 0) out[n_acc] = taken;
            n_acc += 1;
            cur = taken;
            __syncthreads();
            continue;
        }
        // nobody accepted: draw the next token from the residual (the original row if nothing is left of it)
        if (A == 0) {
            __syncthreads();
            if (tid == 0) lv.n = 0;
            __syncthreads();
            long long s = 0;
            for (int v = tid; v < V; v += kThreads) s += fixed_prob(pt[v]);
            A = block_sum(s, red);
        }
        const unsigned long long t = (unsigned long long)(((unsigned __int128)u_bonus[row] * (unsigned long long)A) >> 32);
        // thread i owns the contiguous entries [i per, (i + 1) per): its sum, a scan over the threads, then a walk
        const int per = (V + kThreads - 1) / kThreads;
        const int v0 = tid * per, v1 = min(V, v0 + per);
        long long mine = 0;
        for (int v = v0; v < v1; ++v) {
            long long P, Q;
            weights_at(pt, pq, v, lv, &P, &Q);
            mine += P;
        }
        chunk_sum[tid] = mine;
        if (tid == 0) found_v = V - 1;                             // (only reached if A > 0 failed to hold)
        __syncthreads();
        if (tid == 0) {
            long long before = 0;
            int owner = -1;
            for (int i = 0; i < kThreads; ++i) {
                if ((unsigned long long)(before + chunk_sum[i]) > t) { owner = i; break; }
                before += chunk_sum[i];
            }
            chunk_sum[0] = before;                                 // prefix in front of the owner's entries
            found_v = owner < 0 ? V - 1 : -1 - owner;              // negative: the owner still has to walk its entries
        }
        __syncthreads();
        if (found_v < 0 && tid == -1 - found_v) {
            long long acc = chunk_sum[0];
            int pick = v1 - 1;
            for (int v = v0; v < v1; ++v) {
                long long P, Q;
                weights_at(pt, pq, v, lv, &P, &Q);
                acc += P;
                if ((unsigned long long)acc > t) { pick = v; break; }
            }
            bonus[b] = pick;
        } else if (found_v >= 0 && tid == 0) {
            bonus[b] = found_v;
        }
        break;
    }
    if (tid == 0) n_accept[b] = n_acc;
    for (int i = n_acc + tid; i < T; i += kThreads) out[i] = -1;
}

}  // namespace sample
}  // namespace sparrow
