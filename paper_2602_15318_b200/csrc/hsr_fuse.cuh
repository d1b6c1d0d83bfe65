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
// stage), accumulator in TMEM.  The slices of one feature tile form a thread-block cluster (2, 4 or
// 8 CTAs).  The CTA of rank r finishes tokens [r 64/n, (r + 1) 64/n): every CTA pushes its fp32
// partial sums for those tokens into that CTA's shared memory, and after one cluster barrier each
// CTA adds the slices in fixed order (deterministic), adds the bias and writes z (bf16).  Nothing
// goes through global scratch and no counter is needed.  Every mbarrier wait is bounded; a CTA
// whose wait ran out still takes part in the cluster barrier.
#pragma once
#include <cuda.h>

#include "verify_tc.cuh"

namespace sparrow {

struct HsrArgs {
    const __nv_bfloat16* bias;   // [d_out] or nullptr
    __nv_bfloat16* z;            // [M][d_out]
    unsigned* status;
    int32_t M, d, d_out;
    int32_t n_slices;            // K-range slices per feature tile = CTAs per cluster (1 .. 8)
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
constexpr int kRecvBytes = (kTok + 4 * 8) * kFeat * 4;   // partial sums pushed by the cluster's CTAs: [slice][feature][share + 4] fp32
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kRecvBytes + 256;

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "r"(taddr) : "memory");
}

__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, float a, float b, float c, float d)
{
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// eight token columns of this thread's feature row (zeros when the item has no accumulator)
__device__ __forceinline__ void load8(bool have, uint32_t taddr, float (&v)[8])
{
    if (have) {
        tmem_ld8(taddr, v);
        tmem_wait_ld();
    } else {
        #pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
    }
}

__global__ void __launch_bounds__(kThreadsHsr, 1)
hsr_fuse_kernel(const __grid_constant__ HsrArgs args, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_e, const __grid_constant__ CUtensorMap tmap_h)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    unsigned char* recv = sm + kStages * kStageBytes;                    // [n_slices][128][share + 4] fp32 (rows padded against bank conflicts)
    unsigned char* misc = recv + kRecvBytes;
    const uint32_t bar0 = smem_u32(misc);                               // full[6], empty[6], done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 128);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(misc + 132);
    auto full = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto empty = [&](int i) { return bar0 + 48u + 8u * (uint32_t)i; };
    const uint32_t done = bar0 + 96u;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    SPARROW_TIMELINE_CALL(0);
    if (tid == 0) SPARROW_STAMP(0);                                     // entry
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
    if (tid == 0) SPARROW_STAMP(1);                                     // set-up done

    const int feat_local = (warp & 3) * 32 + lane;
    // n_slices is a power of two: each CTA of the cluster finishes `share` of the 64 token columns
    const int share = kTok / args.n_slices, lg_share = 31 - __clz(share), row_floats = share + 4;
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
                if (i == 0) SPARROW_STAMP(2);                           // first tile landed
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
            SPARROW_STAMP(3);                                           // last MMA issued
            if (!ok) { atomicOr(args.status, timeout_bits(kSiteMma)); *abort_flag = 1; }
        }
    } else {
        // ---- epilogue warps, part 1: thread = one output feature (TMEM lane), 64 token columns.
        // Everything from here on runs once per CTA, i.e. from a cold instruction cache: the loops
        // are kept rolled (8 token columns per trip) so that few distinct instructions are fetched.
        bool ok = n_kt == 0 || mbar_wait_warp(done, 0);
        tc_fence_after();
        if (!ok) { atomicOr(args.status, timeout_bits(kSiteSoftmax)); *abort_flag = 1; }
        const bool have = ok && n_kt > 0;
        if (tid == 0) SPARROW_STAMP(4);                                 // accumulator complete
        if (args.n_slices == 1) {                                       // a single slice writes z itself
            const float b = args.bias ? __bfloat162float(args.bias[f_tile * kFeat + feat_local]) : 0.f;
            #pragma unroll 1
            for (int c = 0; c < args.M; c += 8) {
                float v[8];
                load8(have, tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, v);
                #pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (c + i < args.M) args.z[(size_t)(c + i) * args.d_out + f_tile * kFeat + feat_local] = __float2bfloat16(v[i] + b);
            }
        } else {
            // The CTA of rank r finishes tokens [r share, (r + 1) share): this slice's partial sums
            // for them are pushed into that CTA's receive buffer, laid out [slice][feature][token in
            // share] with padded rows.  Remote stores are not waited for.  Columns past M hold
            // zeros (TMA fills the token rows past M with zeros), so whole chunks are pushed.
            const uint32_t row0 = smem_u32(recv) + (uint32_t)((slice * kFeat + feat_local) * row_floats) * 4u;
            #pragma unroll 1
            for (int c = 0; c < args.M; c += 8) {
                float v[8];
                load8(have, tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, v);
                const uint32_t dst = map_to_rank(row0 + (uint32_t)(c & (share - 1)) * 4u, (uint32_t)(c >> lg_share));
                st_cluster_v4(dst, v[0], v[1], v[2], v[3]);
                st_cluster_v4(dst + 16u, v[4], v[5], v[6], v[7]);
            }
        }
    }
    if (args.n_slices > 1) {
        // one cluster barrier: every slice's pushes have landed; after it nobody touches a peer
        if (tid == 0) SPARROW_STAMP(5);                                 // partial sums pushed
        cluster_arrive_release();
        cluster_wait_acquire();
        if (tid == 0) SPARROW_STAMP(6);                                 // cluster barrier passed
        if (warp < 4) {
            // part 2: the slices in fixed order (results do not depend on timing), bias, bf16 z
            const float b = args.bias ? __bfloat162float(args.bias[f_tile * kFeat + feat_local]) : 0.f;
            const float* mine = reinterpret_cast<const float*>(recv) + feat_local * row_floats;
            const int t0 = slice * share;
            const int n_mine = min(share, args.M - t0);                 // may be <= 0: nothing to finish
            #pragma unroll 1
            for (int j0 = 0; j0 < n_mine; j0 += 4) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                #pragma unroll 1
                for (int s2 = 0; s2 < args.n_slices; ++s2) {
                    const float4 p = *reinterpret_cast<const float4*>(mine + s2 * kFeat * row_floats + j0);
                    acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
                }
                __nv_bfloat16* zp = args.z + (size_t)(t0 + j0) * args.d_out + f_tile * kFeat + feat_local;
                zp[0] = __float2bfloat16(acc.x + b);
                if (j0 + 1 < n_mine) zp[args.d_out] = __float2bfloat16(acc.y + b);
                if (j0 + 2 < n_mine) zp[2 * (size_t)args.d_out] = __float2bfloat16(acc.z + b);
                if (j0 + 3 < n_mine) zp[3 * (size_t)args.d_out] = __float2bfloat16(acc.w + b);
            }
        }
    }
    if (tid == 0) SPARROW_STAMP(7);                                     // z written, leaving
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
