// Split-KV pass of the verification mode on the sm_100a tensor path.
//
// One CTA per SM-sized work item (sequence, KV head, group of up to 256 packed query rows, piece
// of the key range).  The GQA group's 7 heads x T draft tokens are packed into M = 7T query rows
// (row r = t*7 + g), so each K/V byte crosses HBM -> SM once per KV head.
//
//   producer warp (1 thread) TMA: K and V tiles of 128 keys x 128 dims (4 boxes of 128 x 64,
//                        128-byte swizzle) into a 2- or 3-stage shared-memory ring, mbarrier
//                        full / empty handshakes.
//   MMA warp (1 thread) tcgen05.mma issuer: S = Q K^T (A, B from shared memory, K-major) into a
//                        128x128 fp32 TMEM block; O += P V with P read from TMEM (bf16, aliasing
//                        the S block) and V from shared memory as an MN-major operand.
//   warps 0-3, 4-7      softmax warpgroups, one thread per query row (TMEM lane): tcgen05.ld of
//                        the score row, ancestor / range masking, fp32 online softmax with a lazy
//                        maximum (O is rescaled in TMEM only when the row maximum grows by more
//                        than 2^8), P packed to bf16 and stored back with tcgen05.st.
//
// With M <= 128 one warpgroup works through the key tiles on two alternating S blocks, so the
// tensor pipe computes tile j+1's scores while tile j's softmax runs.  With 128 < M <= 256 each
// warpgroup owns one 128-row block (its own S and O) and the two ping-pong on every key tile.
// Every mbarrier wait is bounded; a wait that gives up sets the timeout status bit and the CTA
// drains and exits.  TMEM is always released.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace sparrow {

struct TcArgs {
    const __nv_bfloat16* q;
    const int32_t* parents;      // DEV [B][T]
    int32_t n_q_heads;
    int32_t n_stages;            // K/V ring depth (3 when M <= 128, else 2)
    int32_t n_blocks;            // 128-row blocks per work item (1 or 2)
    int32_t use_pdl;
    float scale_log2e;           // softmax_scale * log2(e)
    __half* o_part;              // [n_items][part_rows][128] normalised partial outputs (fp16)
    float* lse_part;             // [n_items][part_rows]
    __nv_bfloat16* out;          // final output, written here directly for sequences with one piece
    float* lse;
    unsigned* status;
    unsigned long long* tl_all;  // tuning builds only: [n_items][8] wall-clock stamps
};

namespace tc {

// NB = 1: 4 softmax warps + producer + MMA issuer; NB = 2: 8 softmax warps + one more warpgroup
// holding the producer and the MMA issuer (register budget moved to the softmax warps).
__host__ __device__ constexpr int threads_for(int n_blocks) { return n_blocks == 1 ? 192 : 384; }
constexpr int kTile = 128;                       // keys per stage
constexpr int kSubTileBytes = 128 * 64 * 2;      // one 128 x 64 bf16 box: 16 KB
constexpr int kQBlockBytes = 2 * kSubTileBytes;  // 128 rows x 128 dims: 32 KB
constexpr int kStageBytes = 4 * kSubTileBytes;   // K (32 KB) + V (32 KB)
constexpr int kMiscBytes = 1024;                 // barriers, TMEM slot, flags, ancestor words
constexpr uint32_t kSpinLimit = 1u << 22;        // polls before a wait gives up
constexpr float kRescaleLog2 = 8.0f;             // lazy-max threshold in log2 units

__host__ __device__ constexpr int smem_bytes(int n_blocks, int n_stages)
{
    return 1024 /*alignment slack*/ + n_blocks * kQBlockBytes + n_stages * kStageBytes + kMiscBytes;
}

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the phase did not complete within kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Same, with a warp-uniform result (every lane polls; used around warp-collective tcgen05 ops).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity)
{
    return __all_sync(0xffffffffu, mbar_wait(bar, parity) ? 1 : 0) != 0;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
// K-major operand: rows of 128 bytes, 8-row groups 1024 bytes apart (stride offset); the leading
// offset is unused.  MN-major operand: 64-element (128-byte) runs along MN, 8 K-rows per 1024-byte
// group (stride offset), next 64-element MN run `lbo` bytes away (leading offset).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;          // descriptor version
    d |= (uint64_t)2 << 61;          // SWIZZLE_128B
    return d;
}
// Instruction descriptor, kind::f16: D fp32, A/B bf16, A K-major, M = 128, N = 128.
__host__ __device__ constexpr uint32_t idesc_bf16(bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// Shared-memory addresses of the mbarriers (8-byte slots).  K and V tiles have their own full /
// empty pairs: a K tile is released as soon as its S = Q K^T has been computed, a V tile only
// after its O += P V, so the K stream runs ahead of the V stream.
struct Bars {
    uint32_t base;
    __device__ __forceinline__ uint32_t k_full(int i) const { return base + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t k_empty(int i) const { return base + 32u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t v_full(int i) const { return base + 64u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t v_empty(int i) const { return base + 96u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t s_full(int i) const { return base + 128u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t p_full(int i) const { return base + 144u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t o_done(int i) const { return base + 160u + 8u * (uint32_t)i; }
};

// Optional timeline for tuning builds (-DSPARROW_TIMELINE): CTA 0 stores SM clock deltas into the
// spare words of the status block.  Compiled out of the product build.
#ifdef SPARROW_TIMELINE
#define SPARROW_TL(word) do { if (blockIdx.x == 0 && (word) < 240) args.status[16 + (word)] = (unsigned)(clock64() - tl_t0); } while (0)
// every CTA: wall-clock (globaltimer, ns) stamps into a per-CTA record of 8 words
#define SPARROW_TLG(word) do { unsigned long long gt_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt_)); args.tl_all[blockIdx.x * 8 + (word)] = gt_; } while (0)
#else
#define SPARROW_TL(word) do { } while (0)
#define SPARROW_TLG(word) do { } while (0)
#endif

template <int NB>
__global__ void __launch_bounds__(threads_for(NB), 1)
verify_tc_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                 const __grid_constant__ SplitPlan plan, const __grid_constant__ TcArgs args)
{
#ifdef SPARROW_TIMELINE
    const long long tl_t0 = clock64();
#endif
    extern __shared__ unsigned char smem_raw[];
    if (threadIdx.x == 0) { SPARROW_TLG(0); }
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const int NS = args.n_stages;
    constexpr int kProducerWarp = 4 * NB, kMmaWarp = 4 * NB + 1;
    unsigned char* q_sm = sm;
    unsigned char* kv_sm = sm + NB * kQBlockBytes;
    unsigned char* misc = kv_sm + NS * kStageBytes;
    uint64_t* bar_mem = reinterpret_cast<uint64_t*>(misc);                  // 22 barriers in 176 bytes
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 192);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(misc + 196);
    unsigned long long* anc_s = reinterpret_cast<unsigned long long*>(misc + 256);   // [64]

    Bars B;
    B.base = smem_u32(bar_mem);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Item it = decode_item(plan, blockIdx.x);
    const int T = plan.T, M = plan.M;
    const int kv_len = plan.kv_len[it.b];
    const int n_keys_seq = plan.n_keys[it.b];
    const int n_tiles = (it.key_end - it.key_begin + kTile - 1) / kTile;
    const int n_jobs = n_tiles * NB;                 // job n: tile n / NB, S block n % 2, row block n % NB

    // ---- setup: barriers, TMEM ------------------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) {
            mbar_init(B.k_full(i), 1); mbar_init(B.k_empty(i), 1); mbar_init(B.v_full(i), 1); mbar_init(B.v_empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(B.s_full(i), 1); mbar_init(B.p_full(i), 128); mbar_init(B.o_done(i), 1); }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp == kProducerWarp && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_v) : "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (tid == 0) SPARROW_TL(0);
    if (args.use_pdl) {
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    auto issue_k = [&](int j) {                     // producer thread only
        const int st = j % NS;
        const uint32_t dst = smem_u32(kv_sm + st * kStageBytes);
        const int row = it.key_begin + j * kTile;
        mbar_expect_tx(B.k_full(st), 2 * kSubTileBytes);
        tma_load_4d(dst, &tmap_k, 0, row, it.kvh, it.b, B.k_full(st));
        tma_load_4d(dst + kSubTileBytes, &tmap_k, 64, row, it.kvh, it.b, B.k_full(st));
    };
    auto issue_v = [&](int j) {
        const int st = j % NS;
        const uint32_t dst = smem_u32(kv_sm + st * kStageBytes + 2 * kSubTileBytes);
        const int row = it.key_begin + j * kTile;
        mbar_expect_tx(B.v_full(st), 2 * kSubTileBytes);
        tma_load_4d(dst, &tmap_v, 0, row, it.kvh, it.b, B.v_full(st));
        tma_load_4d(dst + kSubTileBytes, &tmap_v, 64, row, it.kvh, it.b, B.v_full(st));
    };

    // ---- prologue --------------------------------------------------------------------------------
    // The small reads (parents, the packed Q block) are issued first and the K/V stream second:
    // requests are served roughly in order, and Q queued behind a ring-full of K/V tiles would
    // hold up the first S = Q K^T for several microseconds.
    constexpr int kChunksPerThread = 16;             // 16-byte chunks of Q per softmax thread
    uint4 qv[kChunksPerThread];
    int32_t par0 = -1, par1 = -1;
    if (warp < 4 * NB) {
        if (warp == 0) {
            const int32_t* par_g = args.parents + (size_t)it.b * T;
            if (lane < T) par0 = __ldg(par_g + lane);
            if (lane + 32 < T) par1 = __ldg(par_g + lane + 32);
        }
        {
            // thread tid owns 16-byte chunk (tid & 15) of rows (tid >> 4) + u * 8 * NB, u = 0..15
            const int c = tid & 15;
            const __nv_bfloat16* qbase = args.q + ((size_t)it.b * T * args.n_q_heads + it.kvh * kGroup) * kD + c * 8;
            #pragma unroll
            for (int u = 0; u < kChunksPerThread; ++u) {
                const int r = (tid >> 4) + u * 8 * NB;
                const int R = it.group * plan.rows_per_group + r;
                qv[u] = make_uint4(0, 0, 0, 0);
                if (R < M && r < plan.rows_per_group) {
                    const int t = R / kGroup, g = R - t * kGroup;
                    qv[u] = __ldg(reinterpret_cast<const uint4*>(qbase + ((size_t)t * args.n_q_heads + g) * kD));
                }
            }
        }
    }
    __syncthreads();                                 // every Q / parents request is in flight
    if (warp == kProducerWarp && lane == 0)
        for (int j = 0; j < n_tiles && j < NS; ++j) { issue_k(j); issue_v(j); }
    if (warp < 4 * NB) {
        if (warp == 0) {
            int32_t* par_s = reinterpret_cast<int32_t*>(misc + 768);               // [64]
            if (lane < T) par_s[lane] = par0;
            if (lane + 32 < T) par_s[lane + 32] = par1;
            __syncwarp();
            for (int i = lane; i < T; i += 32) anc_s[i] = ancestor_word(par_s, T, i, args.status);
        }
        #pragma unroll
        for (int u = 0; u < kChunksPerThread; ++u) {
            const int i = tid + u * NB * 128;
            const int r = i >> 4, c = i & 15;
            const int blk = r >> 7, rr = r & 127;
            unsigned char* dst = q_sm + blk * kQBlockBytes + (c >> 3) * kSubTileBytes + rr * 128 + (((c & 7) ^ (rr & 7)) << 4);
            *reinterpret_cast<uint4*>(dst) = qv[u];
        }
        fence_proxy_async();
    }
    if (tid == 0) SPARROW_TL(1);
    __syncthreads();
    if (tid == 0) SPARROW_TL(2);

    if (warp == kProducerWarp) {
        // ================= TMA producer =================
        if (NB == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
        if (lane == 0) {
            // refill whichever ring has a free slot; K slots free up about one tile before V slots
            int jk = NS < n_tiles ? NS : n_tiles, jv = jk;
            uint32_t idle = 0;
            #pragma unroll 1
            while (jk < n_tiles || jv < n_tiles) {
                bool progress = false;
                if (jk < n_tiles && mbar_try_wait(B.k_empty(jk % NS), (jk / NS - 1) & 1)) { issue_k(jk); ++jk; progress = true; }
                if (jv < n_tiles && mbar_try_wait(B.v_empty(jv % NS), (jv / NS - 1) & 1)) { issue_v(jv); ++jv; progress = true; }
                if (progress) idle = 0;
                else if (++idle > kSpinLimit) { atomicOr(args.status, kStatTimeout); *abort_flag = 1; break; }
            }
        }
    } else if (warp == kMmaWarp) {
        // ================= MMA issuer =================
        if (NB == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(false);
            constexpr uint32_t idesc_pv = idesc_bf16(true);
            bool ok = true;
            // descriptors differ from tile to tile only in their 14-bit address field
            const uint64_t q_desc0 = smem_desc(smem_u32(q_sm), 16, 1024);
            const uint64_t k_desc0 = smem_desc(smem_u32(kv_sm), 16, 1024);
            const uint64_t v_desc0 = smem_desc(smem_u32(kv_sm) + 2 * kSubTileBytes, kSubTileBytes, 1024);
            #pragma unroll 1
            for (int n = -1; n < n_jobs && ok; ++n) {
                if (n + 1 < n_jobs) {                                     // S = Q K^T of the next job
                    const int m = n + 1;
                    const int j = m / NB, blk = m % NB, slot = m & 1, st = j % NS;
                    if (blk == 0) {                                       // first use of this K tile
                        if (!mbar_wait(B.k_full(st), (j / NS) & 1)) { ok = false; break; }
                        tc_fence_after();
                        SPARROW_TL(100 + 4 * m);
                        if (j == 0) { SPARROW_TLG(1); }
                        if (j == n_tiles - 1) { SPARROW_TLG(2); }
                    }
                    const uint64_t qd = q_desc0 + (uint64_t)((blk * kQBlockBytes) >> 4);
                    const uint64_t kd = k_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                    #pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t off = ((ks >> 2) * kSubTileBytes + (ks & 3) * 32) >> 4;
                        mma_ss(tmem + slot * 128, qd + off, kd + off, idesc_qk, ks > 0);
                    }
                    tc_commit(B.s_full(slot));
                    if (blk == NB - 1) tc_commit(B.k_empty(st));
                    SPARROW_TL(101 + 4 * m);
                }
                if (n < 0) continue;
                const int j = n / NB, blk = n % NB, slot = n & 1, st = j % NS;
                if (blk == 0 && !mbar_wait(B.v_full(st), (j / NS) & 1)) { ok = false; break; }
                if (!mbar_wait(B.p_full(slot), (n >> 1) & 1)) { ok = false; break; }
                tc_fence_after();
                SPARROW_TL(102 + 4 * n);
                const uint64_t vd = v_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                #pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem + 256 + blk * 128, tmem + slot * 128 + kk * 8, vd + (uint64_t)((kk * 2048) >> 4),
                           idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
                tc_commit(B.o_done(blk));
                if (blk == NB - 1) tc_commit(B.v_empty(st));
                SPARROW_TL(103 + 4 * n);
            }
            SPARROW_TLG(3);
            if (!ok) { atomicOr(args.status, kStatTimeout); *abort_flag = 1; }
        }
    } else if (warp < 4 * NB) {
        // ================= softmax warpgroups =================
        if (NB == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory");
        const int wg = warp >> 2;                        // row block handled (NB == 2) / 0
        const int row_local = (warp & 3) * 32 + lane;    // TMEM lane
        const int r_item = wg * 128 + row_local;
        const int R = it.group * plan.rows_per_group + r_item;
        const bool row_ok = R < M && r_item < plan.rows_per_group;
        const unsigned long long anc = anc_s[row_ok ? R / kGroup : 0];
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const float c2 = args.scale_log2e;
        const float thr = kRescaleLog2 / c2;             // threshold in raw score units
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;

        #pragma unroll 1
        for (int n = (NB == 2 ? wg : 0); n < n_jobs; n += NB) {
            const int j = n / NB, slot = n & 1, st = j % NS;
            if (!mbar_wait_warp(B.s_full(slot), (n >> 1) & 1)) { ok = false; break; }
            tc_fence_after();
            if (tid == 0) SPARROW_TL(8 + 6 * n);
            float s[128];
            const uint32_t s_addr = lane_addr + slot * 128;
            tmem_ld32(s_addr, s); tmem_ld32(s_addr + 32, s + 32);
            tmem_ld32(s_addr + 64, s + 64); tmem_ld32(s_addr + 96, s + 96);
            tmem_wait_ld();
            if (tid == 0) SPARROW_TL(9 + 6 * n);

            const int j0 = it.key_begin + j * kTile;
            if (j0 + kTile > it.key_end || j0 + kTile > kv_len) {          // tile touches the draft block / range end
                // 128-bit visibility word of this row for the tile's columns: prefix columns, then the
                // ancestor word shifted to the draft block's column, cut at the end of the key range.
                const int d0 = kv_len - j0;                                 // column of draft token 0 (any sign)
                const int nval = it.key_end - j0;                           // valid columns (>= 1)
                unsigned long long lo, hi;
                if (d0 >= 128) { lo = ~0ull; hi = ~0ull; }
                else if (d0 >= 64) { lo = ~0ull; hi = ((1ull << (d0 - 64)) - 1ull) | (anc << (d0 - 64)); }
                else if (d0 > 0) { lo = ((1ull << d0) - 1ull) | (anc << d0); hi = anc >> (64 - d0); }
                else if (d0 > -64) { lo = anc >> (-d0); hi = 0ull; }
                else { lo = 0ull; hi = 0ull; }
                if (nval < 64) { lo &= (1ull << nval) - 1ull; hi = 0ull; }
                else if (nval < 128) { hi &= (1ull << (nval - 64)) - 1ull; }
                const uint32_t w0 = (uint32_t)lo, w1 = (uint32_t)(lo >> 32), w2 = (uint32_t)hi, w3 = (uint32_t)(hi >> 32);
                #pragma unroll
                for (int c = 0; c < 32; ++c) {
                    if (!((w0 >> c) & 1u)) s[c] = -INFINITY;
                    if (!((w1 >> c) & 1u)) s[32 + c] = -INFINITY;
                    if (!((w2 >> c) & 1u)) s[64 + c] = -INFINITY;
                    if (!((w3 >> c) & 1u)) s[96 + c] = -INFINITY;
                }
                // V rows past the end of the sequence may hold anything: zero them so 0 * x stays 0
                if (wg == 0 && j0 + kTile > n_keys_seq && row_local >= n_keys_seq - j0) {
                    mbar_wait(B.v_full(st), (j / NS) & 1);
                    unsigned char* vrow = kv_sm + st * kStageBytes + 2 * kSubTileBytes + row_local * 128;
                    #pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(vrow + kSubTileBytes + c * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                }
            }
            float mx4[4] = {s[0], s[1], s[2], s[3]};                   // four independent chains
            #pragma unroll
            for (int c = 4; c < 128; c += 4) {
                mx4[0] = fmaxf(mx4[0], s[c]); mx4[1] = fmaxf(mx4[1], s[c + 1]);
                mx4[2] = fmaxf(mx4[2], s[c + 2]); mx4[3] = fmaxf(mx4[3], s[c + 3]);
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));

            if (tid == 0) SPARROW_TL(10 + 6 * n);
            const bool need = mx > m_ref + thr || (m_ref == -INFINITY && mx > -INFINITY);
            if (__any_sync(0xffffffffu, need)) {
                float alpha = 1.f;
                if (need) {
                    alpha = (m_ref == -INFINITY) ? 0.f : ex2((m_ref - mx) * c2);
                    m_ref = mx;
                    l_run *= alpha;
                }
                if (j > 0) {                                          // O holds earlier tiles: rescale it in TMEM
                    const int i_blk = n / NB;                         // jobs of this row block issued so far
                    if (!mbar_wait_warp(B.o_done(NB == 2 ? wg : 0), (i_blk - 1) & 1)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t o_addr = lane_addr + 256 + (NB == 2 ? wg : 0) * 128;
                    #pragma unroll 1
                    for (int ch = 0; ch < 4; ++ch) {
                        float o[32];
                        tmem_ld32(o_addr + ch * 32, o);
                        tmem_wait_ld();
                        #pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] *= alpha;
                        tmem_st32(o_addr + ch * 32, reinterpret_cast<uint32_t*>(o));
                    }
                    tmem_wait_st();
                }
            }
            if (tid == 0) SPARROW_TL(11 + 6 * n);
            const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * c2;
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            #pragma unroll
            for (int ch = 0; ch < 4; ++ch) {                          // 32 scores -> 16 packed bf16 pairs
                uint32_t p[16];
                #pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const float p0 = ex2(fmaf(s[ch * 32 + 2 * c], c2, -mc));
                    const float p1 = ex2(fmaf(s[ch * 32 + 2 * c + 1], c2, -mc));
                    sum4[c & 3] += p0 + p1;
                    p[c] = pack_bf16x2(p0, p1);
                }
                tmem_st16(s_addr + ch * 16, p);
            }
            l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            if (tid == 0) SPARROW_TL(12 + 6 * n);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(B.p_full(slot));
            if (tid == 0) SPARROW_TL(13 + 6 * n);
        }

        // ---- epilogue: normalised partial output + natural-log LSE -------------------------------
        if (ok && n_tiles > 0) {
            const int blk = NB == 2 ? wg : 0;
            if (mbar_wait_warp(B.o_done(blk), (n_tiles - 1) & 1)) {
                tc_fence_after();
                if (tid == 0) { SPARROW_TL(3); SPARROW_TLG(4); }
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
                const float lse_val = l_run > 0.f ? (m_ref * c2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                const uint32_t o_addr = lane_addr + 256 + blk * 128;
                const bool direct = plan.n_splits[it.b] == 1;           // the only piece: write the final result
                const size_t prow0 = (size_t)blockIdx.x * plan.part_rows + blk * 128;    // first partial row of this block
                const int t_row = row_ok ? R / kGroup : 0, h_row = it.kvh * kGroup + (row_ok ? R % kGroup : 0);
                // Staging area: this row block's Q tile (every MMA that read it has completed).  Row r
                // holds 16 chunks of 16 bytes (128 halves), chunk c stored at position c ^ (r & 15).
                unsigned char* stage = q_sm + blk * kQBlockBytes;
                #pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    float o[32];
                    tmem_ld32(o_addr + ch * 32, o);
                    tmem_wait_ld();
                    uint4 pk[4];
                    uint32_t* w = reinterpret_cast<uint32_t*>(pk);
                    if (direct) {
                        if (row_ok) {
                            #pragma unroll
                            for (int c = 0; c < 16; ++c) w[c] = pack_bf16x2(o[2 * c] * inv, o[2 * c + 1] * inv);
                            uint4* dst = reinterpret_cast<uint4*>(
                                args.out + (((size_t)it.b * T + t_row) * args.n_q_heads + h_row) * kD + ch * 32);
                            #pragma unroll
                            for (int c = 0; c < 4; ++c) dst[c] = pk[c];
                        }
                    } else {
                        #pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const __half2 h2 = __floats2half2_rn(o[2 * c] * inv, o[2 * c + 1] * inv);
                            w[c] = *reinterpret_cast<const uint32_t*>(&h2);
                        }
                        #pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(stage + row_local * 256 + (((ch * 4 + c) ^ (row_local & 15)) << 4)) = pk[c];
                    }
                }
                if (tid == 0) SPARROW_TL(6);
                if (row_ok) {
                    if (direct) args.lse[((size_t)it.b * args.n_q_heads + h_row) * T + t_row] = lse_val;
                    else args.lse_part[prow0 + row_local] = lse_val;
                }
                if (tid == 0) SPARROW_TL(7);
                if (!direct) {
                    // each warp wrote its own 32 rows; read them back two rows per instruction so a warp
                    // store covers 512 contiguous bytes of the partial buffer
                    __syncwarp();
                    const int rows_here = min(128, min(plan.rows_per_group - blk * 128, M - (it.group * plan.rows_per_group + blk * 128)));
                    #pragma unroll 4
                    for (int i = 0; i < 16; ++i) {
                        const int r = (warp & 3) * 32 + 2 * i + (lane >> 4), c = lane & 15;
                        if (r < rows_here) {
                            const uint4 val = *reinterpret_cast<const uint4*>(stage + r * 256 + ((c ^ (r & 15)) << 4));
                            *reinterpret_cast<uint4*>(args.o_part + (prow0 + r) * kD + c * 8) = val;
                        }
                    }
                }
                if (tid == 0) SPARROW_TL(4);
            } else {
                ok = false;
            }
        }
        if (!ok) { atomicOr(args.status, kStatTimeout); *abort_flag = 1; }
    } else if (NB == 2) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");     // the two spare warps of the third warpgroup
    }

    // ---- teardown -------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // give copies that are still in flight time to land before the CTA's memory is released
        #pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (tid == 0) { SPARROW_TL(5); SPARROW_TLG(5); }
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

}  // namespace tc
}  // namespace sparrow
