// Hidden-state reuse: the draft model's input z_t = FC(e_t (+) h_t) (Section 3.1, Eq. 1) -- the
// projection of [token embedding | target hidden state], 2 d features, down to d_out, for the
// M <= 64 tokens of a drafting step.  A weight-streaming GEMM: every weight byte crosses HBM -> SM
// once (d_out x 2 d bf16, 51 MB for a 7B-class model), the activations are tiny and come from L2,
// so the bound is HBM bandwidth.
//
// The concatenation is never materialised: the K dimension is walked in 64-wide tiles, a tile
// taking its activations from e (k < d) or from h (k >= d) through two tensor maps.
//
// Work item = (tile of 128 output features, slice of the K range); about one item per SM.  The
// weights are the M-side operand (128 features), the tokens the N side (64 columns, rows past M
// read as zero):  D[128 features x 64 tokens] += W_tile[128 x 16] X_tile[64 x 16]^T  on tcgen05,
// operands staged by TMA through a 6-stage mbarrier ring (16 KB of weights + 8 KB of activations per
// stage), accumulator in TMEM.  Each item stores its fp32 partial tile; the item that arrives last on
// its feature tile's counter adds the slices in fixed order (deterministic), adds the bias and
// writes z (bf16); it also puts the counter back to zero.  Every wait is bounded.
#pragma once
#include <cuda.h>

#include "verify_tc.cuh"

namespace sparrow {

struct HsrArgs {
    const __nv_bfloat16* bias;   // [d_out] or nullptr
    float* partial;              // [n_slices][64][d_out] fp32 (token rows past M are never touched)
    __nv_bfloat16* z;            // [M][d_out]
    unsigned* counters;          // [d_out / 128], zero between calls
    unsigned* status;
    int32_t M, d, d_out;
    int32_t n_slices;            // K-range slices per feature tile
    int32_t k_tiles;             // 2 d / 64
};

namespace hsr {

using namespace tc;

constexpr int kThreadsHsr = 192;                 // 4 epilogue warps, producer, MMA issuer
constexpr int kFeat = 128;                       // output features per item
constexpr int kTok = 64;                         // token columns (M <= 64)
constexpr int kKTile = 64;                       // K elements per TMA box (one 128-byte swizzled row)
constexpr int kBoxes = 1;                        // boxes per stage (wider stages were measured: no difference)
constexpr int kWBytes = kFeat * kKTile * 2;      // one weight box: 16 KB
constexpr int kXBytes = kTok * kKTile * 2;       // one activation box: 8 KB
constexpr int kStageBytes = kBoxes * (kWBytes + kXBytes);
constexpr int kStages = 6;
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 256;

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

__global__ void __launch_bounds__(kThreadsHsr, 1)
hsr_fuse_kernel(const __grid_constant__ HsrArgs args, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_e, const __grid_constant__ CUtensorMap tmap_h)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    unsigned char* misc = sm + kStages * kStageBytes;
    const uint32_t bar0 = smem_u32(misc);                               // full[6], empty[6], done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 128);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(misc + 132);
    volatile int32_t* is_last = reinterpret_cast<volatile int32_t*>(misc + 136);
    auto full = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto empty = [&](int i) { return bar0 + 48u + 8u * (uint32_t)i; };
    const uint32_t done = bar0 + 96u;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int f_tile = blockIdx.x / args.n_slices, slice = blockIdx.x - f_tile * args.n_slices;
    // K tiles of this slice: as even as whole tiles allow
    const int kt_begin = (int)((long long)args.k_tiles * slice / args.n_slices);
    const int kt_end = (int)((long long)args.k_tiles * (slice + 1) / args.n_slices);
    const int n_kt = kt_end - kt_begin;
    const int n_st = (n_kt + kBoxes - 1) / kBoxes;                      // ring fills of this item (the last may be short)
    const int d_tiles = args.d / kKTile;                                // K tiles that belong to e

    // Stage layout: kBoxes weight boxes, then kBoxes activation boxes.
    auto issue = [&](int i) {                                           // producer thread only
        const int st = i % kStages;
        const int boxes = min(kBoxes, n_kt - i * kBoxes);
        const uint32_t dst = smem_u32(sm + st * kStageBytes);
        mbar_expect_tx(full(st), boxes * (kWBytes + kXBytes));
        for (int bx = 0; bx < boxes; ++bx) {
            const int kt = kt_begin + i * kBoxes + bx;
            tma_load_2d(dst + bx * kWBytes, &tmap_w, kt * kKTile, f_tile * kFeat, full(st));
            if (kt < d_tiles) tma_load_2d(dst + kBoxes * kWBytes + bx * kXBytes, &tmap_e, kt * kKTile, 0, full(st));
            else tma_load_2d(dst + kBoxes * kWBytes + bx * kXBytes, &tmap_h, (kt - d_tiles) * kKTile, 0, full(st));
        }
    };

    if (warp == 4 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_e) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_h) : "memory");
        for (int i = 0; i < kStages; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
        mbar_init(done, 1);
        *abort_flag = 0;
        fence_barrier_init();
        for (int i = 0; i < n_st && i < kStages; ++i) issue(i);
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(64u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        if (lane == 0) {                                                // ---- TMA producer: refill freed stages
            #pragma unroll 1
            for (int i = kStages; i < n_st; ++i) {
                if (!mbar_wait(empty(i % kStages), (i / kStages - 1) & 1)) {
                    atomicOr(args.status, timeout_bits(kSiteProducer)); *abort_flag = 1; break;
                }
                issue(i);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {                                                // ---- MMA issuer
            constexpr uint32_t idesc = idesc_bf16(false, kTok);
            bool ok = true;
            #pragma unroll 1
            for (int i = 0; i < n_st && ok; ++i) {
                const int st = i % kStages;
                if (!mbar_wait(full(st), (i / kStages) & 1)) { ok = false; break; }
                tc_fence_after();
                const int boxes = min(kBoxes, n_kt - i * kBoxes);
                const uint32_t base = smem_u32(sm + st * kStageBytes);
                for (int bx = 0; bx < boxes; ++bx) {
                    const uint64_t wd = smem_desc(base + bx * kWBytes, 16, 1024);
                    const uint64_t xd = smem_desc(base + kBoxes * kWBytes + bx * kXBytes, 16, 1024);
                    #pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_ss(tmem, wd + (uint64_t)((ks * 32) >> 4), xd + (uint64_t)((ks * 32) >> 4), idesc,
                               (i > 0 || bx > 0 || ks > 0) ? 1u : 0u);
                }
                tc_commit(empty(st));
            }
            tc_commit(done);
            if (!ok) { atomicOr(args.status, timeout_bits(kSiteMma)); *abort_flag = 1; }
        }
    } else {
        // ---- epilogue warps: thread = one output feature (TMEM lane), 64 token columns
        bool ok = n_kt == 0 || mbar_wait_warp(done, 0);
        tc_fence_after();
        const int feat = f_tile * kFeat + warp * 32 + lane;
        float acc[64];
        if (ok && n_kt > 0) {
            tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16), acc);
            tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + 32, acc + 32);
            tmem_wait_ld();
        } else {
            #pragma unroll
            for (int t = 0; t < 64; ++t) acc[t] = 0.f;
        }
        if (!ok) { atomicOr(args.status, timeout_bits(kSiteSoftmax)); *abort_flag = 1; }
        const float b = args.bias ? __bfloat162float(args.bias[feat]) : 0.f;
        if (args.n_slices == 1) {
            #pragma unroll
            for (int t = 0; t < 64; ++t)
                if (t < args.M) args.z[(size_t)t * args.d_out + feat] = __float2bfloat16(acc[t] + b);
        } else {
            // partial sums as [slice][token][feature]: the 32 features of a warp are 128 contiguous bytes
            float* mine = args.partial + (size_t)slice * kTok * args.d_out + feat;
            #pragma unroll
            for (int t = 0; t < 64; ++t)
                if (t < args.M) mine[(size_t)t * args.d_out] = acc[t];
            asm volatile("bar.sync 1, 128;" ::: "memory");             // every store of this item has been issued
            if (tid == 0) {
                // release (cumulative over the stores the barrier ordered before it) and acquire in one
                unsigned old;
                asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(args.counters + f_tile) : "memory");
                *is_last = old == (unsigned)args.n_slices - 1u ? 1 : 0;
                if (*is_last) args.counters[f_tile] = 0u;              // back to zero for the next call
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (*is_last) {
                // The slices in fixed order, whoever arrived last (its own slice comes from its
                // registers: the same values it stored); all loads of a slice in flight at once.
                // (Two slices in flight, or a sum shared among the tile's items, measured slower.)
                float sum[64];
                #pragma unroll
                for (int t = 0; t < 64; ++t) sum[t] = 0.f;
                #pragma unroll 1
                for (int s2 = 0; s2 < args.n_slices; ++s2) {
                    if (s2 == slice) {
                        #pragma unroll
                        for (int t = 0; t < 64; ++t) sum[t] += acc[t];
                    } else {
                        const float* src = args.partial + (size_t)s2 * kTok * args.d_out + feat;
                        float v[64];
                        #pragma unroll
                        for (int t = 0; t < 64; ++t) v[t] = t < args.M ? __ldcg(src + (size_t)t * args.d_out) : 0.f;
                        #pragma unroll
                        for (int t = 0; t < 64; ++t) sum[t] += v[t];
                    }
                }
                #pragma unroll
                for (int t = 0; t < 64; ++t)
                    if (t < args.M) args.z[(size_t)t * args.d_out + feat] = __float2bfloat16(sum[t] + b);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        #pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(64u) : "memory");
    }
}

}  // namespace hsr
}  // namespace sparrow
