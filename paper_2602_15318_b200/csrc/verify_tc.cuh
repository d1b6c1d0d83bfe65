// Split-KV pass of the verification mode on the sm_100a tensor path.
//
// One CTA per SM-sized work item (sequence, KV head, row group of 1 or 2 128-row blocks, piece of
// the key range).  A block packs the GQA group's 7 heads x 18 draft tokens (row r = (t % 18)*7 + g,
// 2 rows of padding), so each K/V byte crosses HBM -> SM once per KV head and row group.
//
//   warp 8, one thread   TMA producer: the Q block(s) (two boxes of 64 dims x 7 heads x 18 tokens
//                        each, which land exactly in the K-major 128-byte-swizzled operand
//                        layout), then K and V tiles of 128 keys x 128 dims (4 boxes of 128 x 64)
//                        into a 2- or 3-stage shared-memory ring, mbarrier full / empty handshakes.
//   warp 9, one thread   tcgen05.mma issuer: S = Q K^T (A, B from shared memory, K-major) into a
//                        128x128 fp32 TMEM block; O += P V with P read from TMEM (bf16, aliasing
//                        the S block) and V from shared memory as an MN-major operand.
//   warps 0-3, 4-7       two softmax warpgroups, one thread per query row (TMEM lane): tcgen05.ld
//                        of the score row, ancestor / range masking, fp32 online softmax with a
//                        lazy maximum (O is rescaled in TMEM only when the row maximum grows by
//                        more than 2^8), P packed to bf16 and stored back with tcgen05.st.
//
// Warpgroup w owns S block w and O accumulator w.  With one row block (T <= 18) the warpgroups
// take alternate key tiles of the same rows and their two (max, sum, O) states are merged in the
// epilogue; with two row blocks each warpgroup owns one block and both process every key tile.
// Either way the tensor pipe computes one job's scores while the other job's softmax runs.
//
// Ordering against neighbouring kernels in the stream (programmatic dependent launch): all reads
// of q / k / v / parents are issued as soon as the CTA starts; griddepcontrol.wait is executed only
// in front of the first global write (partials, out, lse), so the K/V stream of this call overlaps
// the tail and the combine step of the previous one.
//
// Every mbarrier wait is bounded; a wait that gives up sets the timeout status bit and the CTA
// drains and exits.  TMEM is always released.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace sparrow {

struct TcArgs {
    const int32_t* parents;      // DEV [B][T]
    int32_t n_q_heads;
    int32_t n_stages;            // K/V ring depth (3 with one row block, 2 with two)
    int32_t use_pdl;
    float scale_log2e;           // softmax_scale * log2(e)
    __half* o_part;              // [n_items][part_rows][128] normalised partial outputs (fp16)
    float* lse_part;             // [n_items][part_rows]
    __nv_bfloat16* out;          // final output, written here directly for sequences with one piece
    float* lse;
    unsigned* status;
};

namespace tc {

constexpr int kThreads = 320;                    // 8 softmax warps, producer, MMA issuer
// Declared thread bound: caps the kernel at 65536 / 512 = 128 registers per thread, so that a CTA
// (320 x 128 registers) leaves room on the SM for the combine kernel's CTAs.
constexpr int kBoundThreads = 512;
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr int kTile = 128;                       // keys per stage
constexpr int kSubTileBytes = 128 * 64 * 2;      // one 128 x 64 bf16 box: 16 KB
constexpr int kQBlockBytes = 2 * kSubTileBytes;  // 128 rows x 128 dims: 32 KB
constexpr int kQBoxBytes = 64 * kGroup * kTokPerBlock * 2;   // one Q box: 64 dims x 7 heads x 18 tokens
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
// barrier among the 256 softmax threads only (id 1; id 0 is __syncthreads)
__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
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
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    const __half2 h2 = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h2);
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

// ---- softmax helpers on a 32-column chunk of one score row ---------------------------------------
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ void mask_chunk(float (&x)[32], uint32_t visible)
{
    #pragma unroll
    for (int c = 0; c < 32; ++c)
        if (!((visible >> c) & 1u)) x[c] = -INFINITY;
}
__device__ __forceinline__ float chunk_max(const float (&x)[32])
{
    float a = max3(x[0], x[1], x[2]), b = max3(x[3], x[4], x[5]);
    #pragma unroll
    for (int c = 6; c < 30; c += 4) { a = max3(a, x[c], x[c + 1]); b = max3(b, x[c + 2], x[c + 3]); }
    return max3(a, b, fmaxf(x[30], x[31]));
}
// p = 2^(x c2 - mc) for 32 scores; adds the unrounded p to sum4 and stores the 16 packed bf16
// pairs to 16 TMEM columns at p_addr.
__device__ __forceinline__ void exp_chunk(const float (&x)[32], float c2, float mc, float (&sum4)[4], uint32_t p_addr)
{
    uint32_t p[16];
    #pragma unroll
    for (int c = 0; c < 16; ++c) {
        const float p0 = ex2(fmaf(x[2 * c], c2, -mc));
        const float p1 = ex2(fmaf(x[2 * c + 1], c2, -mc));
        sum4[c & 3] += p0 + p1;
        p[c] = pack_bf16x2(p0, p1);
    }
    tmem_st16(p_addr, p);
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
    __device__ __forceinline__ uint32_t q_full() const { return base + 176u; }
};

template <int NB>
__global__ void __launch_bounds__(kBoundThreads, 1)
verify_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ SplitPlan plan,
                 const __grid_constant__ TcArgs args)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const int NS = args.n_stages;
    unsigned char* q_sm = sm;
    unsigned char* kv_sm = sm + NB * kQBlockBytes;
    unsigned char* misc = kv_sm + NS * kStageBytes;
    uint64_t* bar_mem = reinterpret_cast<uint64_t*>(misc);                  // 23 barriers in 184 bytes
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 192);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(misc + 196);
    unsigned long long* anc_s = reinterpret_cast<unsigned long long*>(misc + 256);   // [64]
    int32_t* par_s = reinterpret_cast<int32_t*>(misc + 768);                          // [64]

    Bars B;
    B.base = smem_u32(bar_mem);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Item it = decode_item(plan, blockIdx.x);
    const int T = plan.T;
    const int kv_len = plan.kv_len[it.b];
    const int n_keys_seq = plan.n_keys[it.b];
    const int n_tiles = (it.key_end - it.key_begin + kTile - 1) / kTile;
    // job n: key tile n / NB; S block, O accumulator and softmax warpgroup n % 2; row block n % NB
    const int n_jobs = n_tiles * NB;
    const int block0 = it.group * NB;                       // first 128-row block of this item

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

    // ---- setup: barriers and the first ring-full of loads, TMEM, ancestor words ------------------
    if (warp == kProducerWarp && lane == 0) {
        for (int i = 0; i < 4; ++i) {
            mbar_init(B.k_full(i), 1); mbar_init(B.k_empty(i), 1); mbar_init(B.v_full(i), 1); mbar_init(B.v_empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(B.s_full(i), 1); mbar_init(B.p_full(i), 128); mbar_init(B.o_done(i), 1); }
        mbar_init(B.q_full(), 1);
        *abort_flag = 0;
        fence_barrier_init();
        // Q first (the first S = Q K^T needs it and it is small), then K and V tiles in the order
        // they are consumed.  Nothing here depends on the previous kernel in the stream.
        mbar_expect_tx(B.q_full(), NB * 2 * kQBoxBytes);
        #pragma unroll
        for (int blk = 0; blk < NB; ++blk) {
            const uint32_t dst = smem_u32(q_sm + blk * kQBlockBytes);
            const int tok = it.b * T + (block0 + blk) * kTokPerBlock;
            tma_load_4d(dst, &tmap_q, 0, 0, it.kvh, tok, B.q_full());
            tma_load_4d(dst + kSubTileBytes, &tmap_q, 64, 0, it.kvh, tok, B.q_full());
        }
        for (int j = 0; j < n_tiles && j < NS; ++j) { issue_k(j); issue_v(j); }
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp == 0 && it.key_end > kv_len) {          // this piece reaches the draft block: it needs the tree
        const int32_t* par_g = args.parents + (size_t)it.b * T;
        if (lane < T) par_s[lane] = __ldg(par_g + lane);
        if (lane + 32 < T) par_s[lane + 32] = __ldg(par_g + lane + 32);
        __syncwarp();
        for (int i = lane; i < T; i += 32) anc_s[i] = ancestor_word(par_s, T, i, args.status);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (args.use_pdl) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kProducerWarp) {
        // ================= TMA producer =================
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
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(false);
            constexpr uint32_t idesc_pv = idesc_bf16(true);
            // descriptors differ from tile to tile only in their 14-bit address field
            const uint64_t q_desc0 = smem_desc(smem_u32(q_sm), 16, 1024);
            const uint64_t k_desc0 = smem_desc(smem_u32(kv_sm), 16, 1024);
            const uint64_t v_desc0 = smem_desc(smem_u32(kv_sm) + 2 * kSubTileBytes, kSubTileBytes, 1024);
            bool ok = mbar_wait(B.q_full(), 0);
            #pragma unroll 1
            for (int n = -1; n < n_jobs && ok; ++n) {
                if (n + 1 < n_jobs) {                                     // S = Q K^T of the next job
                    const int m = n + 1;
                    const int j = m / NB, blk = m % NB, slot = m & 1, st = j % NS;
                    if (blk == 0) {                                       // first use of this K tile
                        if (!mbar_wait(B.k_full(st), (j / NS) & 1)) { ok = false; break; }
                        tc_fence_after();
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
                }
                if (n < 0) continue;
                const int j = n / NB, blk = n % NB, slot = n & 1, st = j % NS;
                if (blk == 0 && !mbar_wait(B.v_full(st), (j / NS) & 1)) { ok = false; break; }
                if (!mbar_wait(B.p_full(slot), (n >> 1) & 1)) { ok = false; break; }
                tc_fence_after();
                const uint64_t vd = v_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                #pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem + 256 + slot * 128, tmem + slot * 128 + kk * 8, vd + (uint64_t)((kk * 2048) >> 4),
                           idesc_pv, (n >= 2 || kk > 0) ? 1u : 0u);
                tc_commit(B.o_done(slot));
                if (blk == NB - 1) tc_commit(B.v_empty(st));
            }
            if (!ok) { atomicOr(args.status, kStatTimeout); *abort_flag = 1; }
        }
    } else if (warp < 8) {
        // ================= softmax warpgroups =================
        const int wg = warp >> 2;                        // S block / O accumulator owned
        const int row_local = (warp & 3) * 32 + lane;    // TMEM lane = row inside the 128-row block
        const int blk = NB == 2 ? wg : 0;                // row block this warpgroup works on
        const int tok0 = (block0 + blk) * kTokPerBlock;  // first token of that block
        const int t_row = tok0 + row_local / kGroup, g_row = row_local % kGroup;
        const bool row_ok = row_local < kTokPerBlock * kGroup && t_row < T;
        const unsigned long long anc = (row_ok && it.key_end > kv_len) ? anc_s[t_row] : 0ull;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t s_addr = lane_addr + wg * 128;
        const uint32_t o_addr = lane_addr + 256 + wg * 128;
        const float c2 = args.scale_log2e;
        const float thr = kRescaleLog2 / c2;             // threshold in raw score units
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;

        #pragma unroll 1
        for (int n = wg; n < n_jobs; n += 2) {
            const int j = n / NB, st = j % NS;
            if (!mbar_wait_warp(B.s_full(wg), (n >> 1) & 1)) { ok = false; break; }
            tc_fence_after();
            // Visibility words of this row for the tile's 128 columns (all ones away from the draft
            // block and the end of the key range).
            const int j0 = it.key_begin + j * kTile;
            const bool boundary = j0 + kTile > it.key_end || j0 + kTile > kv_len;
            unsigned long long vis_lo = ~0ull, vis_hi = ~0ull;      // columns 0-63 / 64-127
            if (boundary) {
                // prefix columns, then the ancestor word shifted to the draft block's column, cut at
                // the end of the key range
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
                vis_lo = lo; vis_hi = hi;
                // V rows past the end of the sequence may hold anything: zero them so 0 * x stays 0.
                // Done by the warpgroup whose P V product is the first to read this V tile.
                if ((NB == 1 || wg == 0) && j0 + kTile > n_keys_seq && row_local >= n_keys_seq - j0) {
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

            // ---- pass 1: row maximum, 32 columns at a time (two chunks in flight) ----
            float x0[32], x1[32];
            float mx = -INFINITY;
            #pragma unroll 1
            for (int hf = 0; hf < 2; ++hf) {
                tmem_ld32(s_addr + hf * 64, x0);
                tmem_ld32(s_addr + hf * 64 + 32, x1);
                tmem_wait_ld();
                const unsigned long long vw = hf ? vis_hi : vis_lo;
                if (boundary) { mask_chunk(x0, (uint32_t)vw); mask_chunk(x1, (uint32_t)(vw >> 32)); }
                mx = fmaxf(mx, fmaxf(chunk_max(x0), chunk_max(x1)));
            }

            // rows of padding hold whatever the Q box left there: they never force a rescale
            const bool need = row_ok && (mx > m_ref + thr || (m_ref == -INFINITY && mx > -INFINITY));
            if (__any_sync(0xffffffffu, need)) {
                float alpha = 1.f;
                if (need) {
                    alpha = (m_ref == -INFINITY) ? 0.f : ex2((m_ref - mx) * c2);
                    m_ref = mx;
                    l_run *= alpha;
                }
                if (n >= 2) {                                         // O holds earlier tiles: rescale it in TMEM
                    if (!mbar_wait_warp(B.o_done(wg), ((n >> 1) - 1) & 1)) { ok = false; break; }
                    tc_fence_after();
                    #pragma unroll 1
                    for (int ch = 0; ch < 4; ++ch) {
                        tmem_ld32(o_addr + ch * 32, x0);
                        tmem_wait_ld();
                        #pragma unroll
                        for (int c = 0; c < 32; ++c) x0[c] *= alpha;
                        tmem_st32(o_addr + ch * 32, reinterpret_cast<uint32_t*>(x0));
                    }
                    tmem_wait_st();
                }
            }

            // ---- pass 2: p = 2^(s c2 - m c2), row sum from the unrounded p, P (bf16) over the S block.
            // P chunk ch lands on columns [16 ch, 16 ch + 16), which hold scores already consumed.
            const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * c2;
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            tmem_ld32(s_addr, x0);
            #pragma unroll 1
            for (int hf = 0; hf < 2; ++hf) {
                const unsigned long long vw = hf ? vis_hi : vis_lo;
                tmem_wait_ld();
                tmem_ld32(s_addr + hf * 64 + 32, x1);                  // next chunk in flight
                if (boundary) mask_chunk(x0, (uint32_t)vw);
                exp_chunk(x0, c2, mc, sum4, s_addr + hf * 32);
                tmem_wait_ld();
                if (hf == 0) tmem_ld32(s_addr + 64, x0);
                if (boundary) mask_chunk(x1, (uint32_t)(vw >> 32));
                exp_chunk(x1, c2, mc, sum4, s_addr + hf * 32 + 16);
            }
            l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(B.p_full(wg));
        }

        // ---- epilogue: normalised partial output + natural-log LSE -------------------------------
        const int my_jobs = (n_jobs - wg + 1) / 2;                     // jobs this warpgroup ran
        // A warpgroup without a job (a single-tile item has one job) waits for that one job instead:
        // nothing below may touch shared memory while a load or an MMA can still use it.
        if (ok && !mbar_wait_warp(B.o_done(my_jobs > 0 ? wg : wg ^ 1), my_jobs > 0 ? (my_jobs - 1) & 1 : 0)) ok = false;
        tc_fence_after();
        const bool direct = plan.n_splits[it.b] == 1;                  // the only piece: write the final result
        const int h_row = it.kvh * kGroup + g_row;
        // Staging area for coalesced stores: the Q block(s) (every MMA that read them has completed
        // once both warpgroups are past their last o_done).  Row r holds 16 chunks of 16 bytes
        // (128 halves), chunk c stored at position c ^ (r & 15).
        unsigned char* stage = q_sm + blk * kQBlockBytes;
        const size_t prow0 = (size_t)blockIdx.x * plan.part_rows + blk * kBlockRows;   // first partial row of this block
        const int tok_here = min(kTokPerBlock, max(0, T - tok0));
        const int rows_here = tok_here * kGroup;

        if (NB == 1) {
            // The two warpgroups hold two (max, sum, O) states of the same rows: exchange (max, sum)
            // through shared memory (first bytes of the K/V ring, idle by now), then warpgroup w
            // merges and writes output dims [64 w, 64 w + 64).
            float2* ml = reinterpret_cast<float2*>(kv_sm);
            ml[wg * 128 + row_local] = make_float2(m_ref, l_run);
            softmax_bar_sync();
            const float2 other = ml[(wg ^ 1) * 128 + row_local];
            const float m_all = fmaxf(m_ref, other.x);
            const float a_me = (m_ref == -INFINITY) ? 0.f : ex2((m_ref - m_all) * c2);
            const float a_ot = (other.x == -INFINITY) ? 0.f : ex2((other.x - m_all) * c2);
            const float l_all = a_me * l_run + a_ot * other.y;
            const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
            const float lse_val = l_all > 0.f ? (m_all * c2 + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
            const float w0 = (wg == 0 ? a_me : a_ot) * inv, w1 = (wg == 0 ? a_ot : a_me) * inv;
            const bool has1 = n_jobs >= 2;                             // accumulator 1 was written at all
            if (args.use_pdl) pdl_wait();                              // global writes start here
            if (ok) {
                #pragma unroll 1
                for (int hf = 0; hf < 2; ++hf) {
                    const int col = wg * 64 + hf * 32;
                    float oa[32], ob[32];
                    tmem_ld32(lane_addr + 256 + col, oa);
                    if (has1) tmem_ld32(lane_addr + 384 + col, ob);
                    tmem_wait_ld();
                    #pragma unroll
                    for (int c = 0; c < 32; ++c) oa[c] = has1 ? fmaf(ob[c], w1, oa[c] * w0) : oa[c] * w0;
                    uint4 pk[4];
                    uint32_t* w = reinterpret_cast<uint32_t*>(pk);
                    if (direct) {
                        if (row_ok) {
                            #pragma unroll
                            for (int c = 0; c < 16; ++c) w[c] = pack_bf16x2(oa[2 * c], oa[2 * c + 1]);
                            uint4* dst = reinterpret_cast<uint4*>(
                                args.out + (((size_t)it.b * T + t_row) * args.n_q_heads + h_row) * kD + col);
                            #pragma unroll
                            for (int c = 0; c < 4; ++c) dst[c] = pk[c];
                        }
                    } else {
                        #pragma unroll
                        for (int c = 0; c < 16; ++c) w[c] = pack_half2(oa[2 * c], oa[2 * c + 1]);
                        #pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(stage + row_local * 256 + ((((col >> 3) + c) ^ (row_local & 15)) << 4)) = pk[c];
                    }
                }
                if (row_ok && wg == 0) {
                    if (direct) args.lse[((size_t)it.b * args.n_q_heads + h_row) * T + t_row] = lse_val;
                    else args.lse_part[prow0 + row_local] = lse_val;
                }
            }
            softmax_bar_sync();                                        // both halves of every staged row are in place
            if (ok && !direct) {
                // warp w copies rows [16 w, 16 w + 16), two rows (512 contiguous bytes) per instruction
                #pragma unroll 4
                for (int i = 0; i < 8; ++i) {
                    const int r = warp * 16 + 2 * i + (lane >> 4), c = lane & 15;
                    if (r < rows_here) {
                        const uint4 val = *reinterpret_cast<const uint4*>(stage + r * 256 + ((c ^ (r & 15)) << 4));
                        *reinterpret_cast<uint4*>(args.o_part + (prow0 + r) * kD + c * 8) = val;
                    }
                }
            }
        } else {
            softmax_bar_sync();                                        // both warpgroups are done with the MMAs' operands
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const float lse_val = l_run > 0.f ? (m_ref * c2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            if (args.use_pdl) pdl_wait();                              // global writes start here
            if (ok) {
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
                        for (int c = 0; c < 16; ++c) w[c] = pack_half2(o[2 * c] * inv, o[2 * c + 1] * inv);
                        #pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(stage + row_local * 256 + (((ch * 4 + c) ^ (row_local & 15)) << 4)) = pk[c];
                    }
                }
                if (row_ok) {
                    if (direct) args.lse[((size_t)it.b * args.n_q_heads + h_row) * T + t_row] = lse_val;
                    else args.lse_part[prow0 + row_local] = lse_val;
                }
                if (!direct) {
                    // each warp wrote its own 32 rows; read them back two rows per instruction so a
                    // warp store covers 512 contiguous bytes of the partial buffer
                    __syncwarp();
                    #pragma unroll 4
                    for (int i = 0; i < 16; ++i) {
                        const int r = (warp & 3) * 32 + 2 * i + (lane >> 4), c = lane & 15;
                        if (r < rows_here) {
                            const uint4 val = *reinterpret_cast<const uint4*>(stage + r * 256 + ((c ^ (r & 15)) << 4));
                            *reinterpret_cast<uint4*>(args.o_part + (prow0 + r) * kD + c * 8) = val;
                        }
                    }
                }
            }
        }
        if (!ok) { atomicOr(args.status, kStatTimeout); *abort_flag = 1; }
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
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

}  // namespace tc
}  // namespace sparrow
