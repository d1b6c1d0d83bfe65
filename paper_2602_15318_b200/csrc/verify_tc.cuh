// Split-KV pass of the verification mode on the sm_100a tensor path.
//
// One CTA per SM-sized work item (sequence, KV head, row group of 1 or 2 128-row blocks, piece of
// the key range).  A block packs the GQA group's g heads x p = 128 / g draft tokens (row r = (t % p) g + head;
// g = 7: 18 tokens, 2 rows of padding), so each K/V byte crosses HBM -> SM once per KV head and row group.
//
//   warp 8, one thread   TMA producer: the Q block(s) (two boxes of 64 dims x g heads x p tokens
//                        each, which land exactly in the K-major 128-byte-swizzled operand
//                        layout), then K and V tiles of 128 keys x 128 dims (4 boxes of 128 x 64)
//                        into a 2- or 3-stage shared-memory ring, mbarrier full / empty handshakes.
//   warp 9, one thread   tcgen05.mma issuer.  A job is one key tile against one row block:
//                        S = Q K^T (A, B from shared memory, K-major) into a 128 x 128 fp32 TMEM
//                        block; O += P V with P read from TMEM (bf16, aliasing the S block) and V
//                        from shared memory as an MN-major operand.  The scores of up to three
//                        jobs are kept ahead of the softmax.
//   warps 0-7            softmax, TMEM lane = query row: tcgen05.ld, ancestor / range / window
//                        masking, fp32 online softmax with a lazy maximum, P packed to bf16 and
//                        stored back with tcgen05.st.
//                        One row block (T <= 18): the two threads with the same lane (warps w and
//                        w + 4) share a row, warpgroup g taking key columns [64 g, 64 g + 64) of every
//                        job.  They keep the same reference maximum: one barrier with an OR reduction
//                        per job tells whether any row's maximum grew by more than 2^8; only then the
//                        halves' maxima meet in shared memory and O is rescaled in TMEM.  Each
//                        thread sums its own columns; the halves' sums meet once, in the epilogue.
//                        Two row blocks: warpgroup g owns block g, one thread per row and all 128
//                        keys of a tile, and works through its block's tiles on its own (no
//                        barrier between the warpgroups); per block the chain is scores -> softmax
//                        -> O += P V -> next scores, and the two chains interleave on the tensor
//                        pipe and the exponential unit.
//   warp 10, one thread  gatekeeper (overlapped mode): waits, beside the main loop, for the counters
//                        that allow this CTA's first global write.
//
// With one row block there are three S blocks and one O accumulator, with two row blocks one S
// block and one accumulator per block.
//
// Ordering against neighbouring kernels in the stream (see SyncArgs).  Overlapped mode: the kernel
// is launched with programmatic stream serialisation and never waits for the previous grid as a
// whole.  All reads of q / k / v / parents are issued as soon as the CTA starts, so the K/V stream
// of this call overlaps the tail of the previous one; in front of its first global write a CTA
// waits on the finisher counters.  A CTA publishes its item after storing its partials, and the
// call's finisher CTAs wait for the arrivals, share the call's rows among them, merge each row's
// pieces by log-sum-exp and write out / lse.  Stream-ordered mode (a call captured into a graph, or
// with programmatic launch switched off): the kernel touches no counter, only stores partials and
// direct results, and the combine kernel follows.
//
// Every wait is bounded; a wait that gives up sets the timeout status bit and the CTA drains and
// exits.  TMEM is always released.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>

#include "combine.cuh"
#include "common.cuh"

namespace sparrow {

struct TcArgs {
    const int32_t* parents;      // DEV [B][T_tree]
    const int32_t* first_visible;   // DEV [B][T] or nullptr: query t sees prefix key j only if j >= first_visible[b][t]
    int32_t n_q_heads;
    float scale_log2e;           // softmax_scale * log2(e)
    __half* o_part;              // [n_items][part_rows] partial rows: 128 fp16 outputs + fp32 LSE (kPartRowHalves)
    __nv_bfloat16* out;          // final output
    float* lse;
    unsigned* status;
};

namespace tc {

constexpr int kThreads = 352;                    // 8 softmax warps, producer, MMA issuer, gatekeeper
// Declared thread bound: caps the kernel at 65536 / 384 = 170 registers per thread.
constexpr int kBoundThreads = 384;
constexpr int kProducerWarp = 8, kMmaWarp = 9, kGateWarp = 10;
constexpr int kTile = 128;                       // keys per stage and per job
constexpr int kSubTileBytes = 128 * 64 * 2;      // one 128 x 64 bf16 box: 16 KB
constexpr int kQBlockBytes = 2 * kSubTileBytes;  // 128 rows x 128 dims: 32 KB
constexpr int kStageBytes = 4 * kSubTileBytes;   // K (32 KB) + V (32 KB)
constexpr int kMiscBytes = 2048;                 // barriers, flags, ancestor words, maxima exchange
constexpr uint32_t kSpinLimit = 1u << 22;        // polls before a wait gives up
constexpr float kRescaleLog2 = 8.0f;             // lazy-max threshold in log2 units

__host__ __device__ constexpr int smem_bytes(int n_blocks, int n_stages)
{
    // two row blocks: 1 KB more for the per-row results the two warpgroups hand each other
    return 1024 /*alignment slack*/ + n_blocks * kQBlockBytes + n_stages * kStageBytes + kMiscBytes + (n_blocks == 2 ? 1024 : 0);
}
// S blocks (score tiles in flight) for a given number of row blocks; TMEM: S blocks first, then
// one 128-column O accumulator per row block, 512 columns in all.
__host__ __device__ constexpr int s_blocks(int n_blocks) { return n_blocks == 1 ? 3 : 2; }

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
// Non-blocking probe of a phase.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
// Same for a whole warp, with a warp-uniform result.  One lane polls (32 lanes hammering the same
// barrier word serialise and cost hundreds of cycles per wait); the shuffle carries the verdict to
// the others and orders their later accesses behind the observation.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
// 1-D bulk copy global -> shared (16-byte aligned, size a multiple of 16), completion on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Orders generic-proxy accesses to global memory that this thread has observed before its later
// async-proxy (bulk copy) accesses to it.
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// barrier among the 256 softmax threads only (id 1; id 0 is __syncthreads)
__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
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
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void lds_v4(uint32_t addr, uint32_t (&v)[4])
{
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// Two non-negative finite floats -> packed bf16, rounded to nearest (ties up) with integer
// instructions: the conversion instruction shares the quarter-rate pipe with ex2, which is the
// softmax's bottleneck.
__device__ __forceinline__ uint32_t pack_bf16x2_pos(float lo, float hi)
{
    return __byte_perm(__float_as_uint(lo) + 0x8000u, __float_as_uint(hi) + 0x8000u, 0x7632);
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
// Instruction descriptor, kind::f16: D fp32, A/B bf16, A K-major, M = 128, N = n (128 or 64).
__host__ __device__ constexpr uint32_t idesc_bf16(bool b_mn_major, uint32_t n = 128u)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
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
        p[c] = pack_bf16x2_pos(p0, p1);
    }
    tmem_st16(p_addr, p);
}

// Barrier among the 256 softmax threads with an OR reduction of a predicate (id 2).
__device__ __forceinline__ bool softmax_bar_or(bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 2, 256, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// Shared-memory addresses of the mbarriers (8-byte slots).  K and V tiles have their own full /
// empty pairs: a K tile is released as soon as its last S = Q K^T has been computed, a V tile
// only after its last O += P V, so the K stream runs ahead of the V stream.
struct Bars {
    uint32_t base;
    // at most 3 stages and 3 S blocks: 28 slots in all
    __device__ __forceinline__ uint32_t k_full(int i) const { return base + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t k_empty(int i) const { return base + 24u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t v_full(int i) const { return base + 48u + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t v_empty(int i) const { return base + 72u + 8u * (uint32_t)i; }
    // (a fourth score / P slot, used with two row blocks, sits behind the other barriers)
    __device__ __forceinline__ uint32_t s_full(int i) const { return i < 3 ? base + 96u + 8u * (uint32_t)i : base + 240u; }
    __device__ __forceinline__ uint32_t p_full(int i) const { return i < 3 ? base + 120u + 8u * (uint32_t)i : base + 248u; }
    __device__ __forceinline__ uint32_t q_full() const { return base + 144u; }
    __device__ __forceinline__ uint32_t fin() const { return base + 152u; }       // finishers' bulk copies
    // Completion of O += P V of key tile j on row block blk: a ring of four barriers per block,
    // tile j on barrier j % 4 with phase parity (j / 4) & 1.  The softmax only looks at it when a
    // row maximum moves and in the epilogue, asking for tile j - 1 while it works on tile j.  A
    // parity wait is only meaningful for the phase in progress or the one just completed; here the
    // barrier is in exactly that state: its previous use (tile j - 5) completed before the scores
    // of tile j, which the warp has seen (the tensor pipe completes in issue order and the scores
    // of tile j were issued after the product of tile j - 3), and its next use (tile j + 3) needs
    // this warp's P of that tile.
    __device__ __forceinline__ uint32_t o_done(int blk, int j) const { return base + 160u + 32u * (uint32_t)blk + 8u * (uint32_t)(j & 3); }
};

template <int NB>
__global__ void __launch_bounds__(kBoundThreads, 1)
verify_tc_kernel(const __grid_constant__ TcArgs args, const __grid_constant__ SyncArgs sync,
                 const __grid_constant__ SplitPlan plan, const __grid_constant__ CUtensorMap tmap_q,
                 const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v)
{
    constexpr int NSB = s_blocks(NB);                 // S blocks
    constexpr uint32_t kOCol = 512 - 128 * NB;        // first accumulator's TMEM column
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    constexpr int NS = NB == 1 ? 3 : 2;               // K/V ring depth
    unsigned char* q_sm = sm;
    unsigned char* kv_sm = sm + NB * kQBlockBytes;
    unsigned char* misc = kv_sm + NS * kStageBytes;
    uint64_t* bar_mem = reinterpret_cast<uint64_t*>(misc);                  // 28 barrier slots in 224 bytes
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 224);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(misc + 228);
    volatile uint32_t* write_ok = reinterpret_cast<volatile uint32_t*>(misc + 232);   // the counters allow global writes
    volatile int32_t* fin_go = reinterpret_cast<volatile int32_t*>(misc + 236);       // finishers: their waits succeeded
    unsigned long long* anc_s = reinterpret_cast<unsigned long long*>(misc + 256);   // [64]
    int32_t* par_s = reinterpret_cast<int32_t*>(misc + 768);                          // [64]: parents in the prologue, then the rows' first visible keys
    float* xch = reinterpret_cast<float*>(misc + 1024);                               // [2][128] maxima / sums exchange

    Bars B;
    SPARROW_TIMELINE_CALL(sync.call);
    if (threadIdx.x == 0) SPARROW_STAMP(0);                             // entry
    B.base = smem_u32(bar_mem);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Item it = decode_item(plan, blockIdx.x);
    const int T = plan.T;
    const int qg = plan.group, tpb = plan.tok_per_block;   // query heads per KV head, tokens per 128-row block
    const int kv_len = plan.seq[it.b].kv_len;
    const int n_keys_seq = plan.seq[it.b].n_keys;
    const int n_tiles = (it.key_end - it.key_begin + kTile - 1) / kTile;
    // job n: key tile n / NB, row block (and O accumulator) n % NB, S block n % NSB
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
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_v) : "memory");
        for (int i = 0; i < 3; ++i) { mbar_init(B.k_full(i), 1); mbar_init(B.k_empty(i), 1); mbar_init(B.v_full(i), 1); mbar_init(B.v_empty(i), 1); }
        // one row block: a P block comes from all 256 softmax threads; two: from the block's own warpgroup
        for (int i = 0; i < 4; ++i) { mbar_init(B.s_full(i), 1); mbar_init(B.p_full(i), NB == 1 ? 256 : 128); }
        for (int i = 0; i < 4; ++i) { mbar_init(B.o_done(0, i), 1); mbar_init(B.o_done(1, i), 1); }
        mbar_init(B.q_full(), 1);
        mbar_init(B.fin(), 1);
        *abort_flag = 0;
        *write_ok = sync.enabled ? 0u : 1u;
        fence_barrier_init();
        // Q first (the first S = Q K^T needs it and it is small), then K and V tiles in the order
        // they are consumed.  Nothing here depends on the previous kernel in the stream.
        mbar_expect_tx(B.q_full(), (uint32_t)(NB * 2 * 64 * qg * tpb * 2));   // two boxes of 64 dims x g heads x p tokens per block
        #pragma unroll
        for (int blk = 0; blk < NB; ++blk) {
            const uint32_t dst = smem_u32(q_sm + blk * kQBlockBytes);
            const int tok = it.b * T + (block0 + blk) * tpb;
            tma_load_4d(dst, &tmap_q, 0, 0, it.kvh, tok, B.q_full());
            tma_load_4d(dst + kSubTileBytes, &tmap_q, 64, 0, it.kvh, tok, B.q_full());
        }
        for (int j = 0; j < n_tiles && j < NS; ++j) { issue_k(j); issue_v(j); }
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp == 0) {
        const int Tt = plan.T_tree;
        if (it.key_end > kv_len) {                   // this piece reaches the draft block: it needs the tree
            const int32_t* par_g = args.parents + (size_t)it.b * Tt;
            if (lane < Tt) par_s[lane] = __ldg(par_g + lane);
            if (lane + 32 < Tt) par_s[lane + 32] = __ldg(par_g + lane + 32);
            __syncwarp();
            for (int i = lane; i < Tt; i += 32) anc_s[i] = ancestor_word(par_s, Tt, i, args.status);
            __syncwarp();
        }
        // Lower window bound of every query token, clamped to what this call streams: a bound
        // left of the first streamed key cannot be honoured (the keys in between were not planned)
        // and is reported.
        for (int t = lane; t < T; t += 32) {
            int lo = args.first_visible ? __ldg(args.first_visible + (size_t)it.b * T + t) : 0;
            if (lo < plan.seq[it.b].key0) {
                if (args.first_visible) atomicOr(args.status, kStatAnchor);
                lo = plan.seq[it.b].key0;
            }
            par_s[t] = lo < kv_len ? lo : kv_len;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (threadIdx.x == 0) SPARROW_STAMP(1);                             // set-up done
    if (sync.enabled) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kProducerWarp) {
        // ================= TMA producer =================
        if (lane == 0) {
            // refill whichever ring has a free slot; K slots free up ahead of V slots
            int jk = NS < n_tiles ? NS : n_tiles, jv = jk;
            uint32_t idle = 0;
            #pragma unroll 1
            while (jk < n_tiles || jv < n_tiles) {
                bool progress = false;
                if (jk < n_tiles && mbar_try_wait(B.k_empty(jk % NS), (jk / NS - 1) & 1)) { issue_k(jk); ++jk; progress = true; }
                if (jv < n_tiles && mbar_try_wait(B.v_empty(jv % NS), (jv / NS - 1) & 1)) { issue_v(jv); ++jv; progress = true; }
                if (progress) idle = 0;
                else if (++idle > kSpinLimit) { atomicOr(args.status, timeout_bits(kSiteProducer)); *abort_flag = 1; break; }
            }
        }
    } else if (warp == kMmaWarp) {
        // ================= MMA issuer =================
        if (lane == 0) {
            // descriptors differ from job to job only in their 14-bit address field
            const uint64_t q_desc0 = smem_desc(smem_u32(q_sm), 16, 1024);
            const uint64_t k_desc0 = smem_desc(smem_u32(kv_sm), 16, 1024);
            const uint64_t v_desc0 = smem_desc(smem_u32(kv_sm) + 2 * kSubTileBytes, kSubTileBytes, 1024);
            bool ok = mbar_wait(B.q_full(), 0);
            SPARROW_STAMP(2);                                           // Q landed
            if constexpr (NB == 2) {
                // Two row blocks, each with its own softmax warpgroup.  Job n = (key tile j = n / 2,
                // block b = n % 2).  Block b owns TMEM columns [128 b, 128 b + 128) for its scores,
                // with its P (bf16, 64 columns) written over the upper half, and the accumulator at
                // 256 + 128 b.  Per block the chain is scores -> softmax -> O += P V -> next scores;
                // the two blocks' chains interleave, so the tensor pipe works for one block while
                // the other block's warpgroup is in its exponentials.
                constexpr uint32_t idesc_qk = idesc_bf16(false);
                constexpr uint32_t idesc_pv = idesc_bf16(true);
                auto issue_qk2 = [&](int m) -> bool {
                    const int j = m >> 1, b = m & 1, st = j % NS;
                    if (b == 0) {                                             // first use of this K tile
                        if (!mbar_wait(B.k_full(st), (j / NS) & 1)) return false;
                        tc_fence_after();
                        if (j == 0) SPARROW_STAMP(3);                   // first K tile landed
                    }
                    const uint64_t qd = q_desc0 + (uint64_t)((b * kQBlockBytes) >> 4);
                    const uint64_t kd = k_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                    #pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t off = ((ks >> 2) * kSubTileBytes + (ks & 3) * 32) >> 4;
                        mma_ss(tmem + b * 128, qd + off, kd + off, idesc_qk, ks > 0);
                    }
                    tc_commit(B.s_full(b));
                    if (b == 1) tc_commit(B.k_empty(st));                     // last use of the tile
                    return true;
                };
                for (int m = 0; m < 2 && m < n_jobs && ok; ++m) ok = issue_qk2(m);
                #pragma unroll 1
                for (int n = 0; n < n_jobs && ok; ++n) {
                    const int j = n >> 1, b = n & 1, st = j % NS;
                    if (b == 0 && !mbar_wait(B.v_full(st), (j / NS) & 1)) { ok = false; break; }
                    if (!mbar_wait(B.p_full(b), j & 1)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t vd = v_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                    #pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_ts(tmem + 256 + b * 128, tmem + b * 128 + 64 + kk * 8, vd + (uint64_t)((kk * 2048) >> 4),
                               idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(B.o_done(b, j));
                    if (b == 1) tc_commit(B.v_empty(st));
                    if (n + 2 < n_jobs) ok = issue_qk2(n + 2);                // this block's next scores
                }
            } else {
            constexpr uint32_t idesc_qk = idesc_bf16(false);
            constexpr uint32_t idesc_pv = idesc_bf16(true);
            // S = Q K^T of job m into S block m % NSB
            auto issue_qk = [&](int m) -> bool {
                const int j = m / NB, blk = m % NB, sb = m % NSB, st = j % NS;
                if (blk == 0) {                                           // first use of this K tile
                    if (!mbar_wait(B.k_full(st), (j / NS) & 1)) return false;
                    tc_fence_after();
                    if (j == 0) SPARROW_STAMP(3);                       // first K tile landed
                }
                const uint64_t qd = q_desc0 + (uint64_t)((blk * kQBlockBytes) >> 4);
                const uint64_t kd = k_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                #pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = ((ks >> 2) * kSubTileBytes + (ks & 3) * 32) >> 4;
                    mma_ss(tmem + sb * 128, qd + off, kd + off, idesc_qk, ks > 0);
                }
                tc_commit(B.s_full(sb));
                if (blk == NB - 1) tc_commit(B.k_empty(st));              // last use of the tile
                return true;
            };
            for (int m = 0; m < NSB && m < n_jobs && ok; ++m) ok = issue_qk(m);
            #pragma unroll 1
            for (int n = 0; n < n_jobs && ok; ++n) {
                const int j = n / NB, blk = n % NB, sb = n % NSB, st = j % NS;
                if (blk == 0 && !mbar_wait(B.v_full(st), (j / NS) & 1)) { ok = false; break; }
                if (!mbar_wait(B.p_full(sb), (n / NSB) & 1)) { ok = false; break; }
                tc_fence_after();
                const uint64_t vd = v_desc0 + (uint64_t)((st * kStageBytes) >> 4);
                #pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem + kOCol + blk * 128, tmem + sb * 128 + kk * 8, vd + (uint64_t)((kk * 2048) >> 4),
                           idesc_pv, (n >= NB || kk > 0) ? 1u : 0u);
                tc_commit(B.o_done(blk, j));
                if (blk == NB - 1) tc_commit(B.v_empty(st));
                if (n + NSB < n_jobs) ok = issue_qk(n + NSB);             // its S block was job n's
            }
            }
            SPARROW_STAMP(4);                                           // last product issued
            if (!ok) { atomicOr(args.status, timeout_bits(kSiteMma)); *abort_flag = 1; }
        }
    } else if (warp == kGateWarp) {
        if (lane == 0 && sync.enabled) {
            // Overlapped mode: whoever read this parity's partial buffer two calls ago must be done
            // before this CTA's first global write, and final results may only follow every earlier
            // call's.  Waiting here, beside the main loop, keeps the round trip to the counters off the
            // epilogue's critical path.  1 = go, 2 = a wait gave up.
            bool go = wait_counter(sync.fin_done + sync.parity, sync.fin_wait_same);
            if (!go) atomicOr(args.status, timeout_bits(kSiteWriteSame));
            if (go && plan.seq[it.b].n_splits == 1) {
                go = wait_counter(sync.fin_done + (sync.parity ^ 1), sync.fin_wait_other);
                if (!go) atomicOr(args.status, timeout_bits(kSiteWriteOther));
            }
            __threadfence_block();
            *write_ok = go ? 1u : 2u;
        }
    } else if (warp < 8) {
        // ================= softmax =================
        const int wg = warp >> 2;                        // key-column half this thread takes
        const int row_local = (warp & 3) * 32 + lane;    // TMEM lane = row inside the 128-row block
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const float c2 = args.scale_log2e;
        const float thr = kRescaleLog2 / c2;             // threshold in raw score units
        const int g_row = row_local % qg;
        int t_row[NB], lo_row[NB];
        bool row_ok[NB];
        unsigned long long anc[NB];
        float m_ref[NB], l_run[NB];
        #pragma unroll
        for (int blk = 0; blk < NB; ++blk) {
            t_row[blk] = (block0 + blk) * tpb + row_local / qg;
            row_ok[blk] = row_local < tpb * qg && t_row[blk] < T;
            // the queries are the last T nodes of the tree
            anc[blk] = (row_ok[blk] && it.key_end > kv_len) ? anc_s[plan.T_tree - T + t_row[blk]] : 0ull;
            lo_row[blk] = row_ok[blk] ? par_s[t_row[blk]] : 0;
            m_ref[blk] = -INFINITY; l_run[blk] = 0.f;
        }
        bool ok = true;

        float my_m = -INFINITY, my_l = 0.f;       // two row blocks: the state of this warpgroup's own block
        if constexpr (NB == 2) {
            // ---- two row blocks: warpgroup g owns block g, one thread per query row, and works
            // through the block's half-tile jobs on its own -- no exchange with the other warpgroup,
            // whose exponentials fill the gaps this one leaves while it waits for the tensor pipe.
            const int blk = wg;
            // this warpgroup's block, in scalars (indexing the per-block arrays with wg would put them in local memory)
            const unsigned long long my_anc = wg ? anc[NB - 1] : anc[0];
            const int my_lo = wg ? lo_row[NB - 1] : lo_row[0];
            const bool my_ok = wg ? row_ok[NB - 1] : row_ok[0];
            const uint32_t s_addr = lane_addr + blk * 128;
            // visibility word of this row for the 64 keys that start at key j0
            auto vis_word = [&](int j0) -> unsigned long long {
                if (!(j0 + 64 > it.key_end || j0 + 64 > kv_len || j0 < my_lo)) return ~0ull;
                const int d0 = kv_len - j0;                                 // column of draft token 0 (any sign)
                const int nval = it.key_end - j0;                           // valid columns (may be <= 0)
                unsigned long long vis;
                if (d0 >= 64) vis = ~0ull;
                else if (d0 > 0) vis = ((1ull << d0) - 1ull) | (my_anc << d0);
                else if (d0 > -64) vis = my_anc >> (-d0);
                else vis = 0ull;
                if (nval <= 0) vis = 0ull;
                else if (nval < 64) vis &= (1ull << nval) - 1ull;
                const int cut = my_lo - j0;
                if (cut >= 64) vis = 0ull;
                else if (cut > 0) vis &= ~((1ull << cut) - 1ull);
                return vis;
            };
            float x0[32], x1[32];
            #pragma unroll 1
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int st = j % NS;
                const int tile0 = it.key_begin + j * kTile;
                if (!mbar_wait_warp(B.s_full(blk), j & 1)) { ok = false; break; }
                tc_fence_after();
                // first pass over the row's 128 scores, 64 at a time: the maximum.  The upper 64 stay
                // in registers; the lower 64 are fetched again for the second pass.
                tmem_ld32(s_addr, x0);
                tmem_ld32(s_addr + 32, x1);
                const unsigned long long vis_lo = vis_word(tile0), vis_hi = vis_word(tile0 + 64);
                // V rows past the end of the sequence may hold anything: zero them so 0 * x stays 0
                // (once per tile, by the threads of the first block, thread r taking key row r)
                if (blk == 0 && tile0 + kTile > n_keys_seq && tile0 + row_local >= n_keys_seq) {
                    mbar_wait(B.v_full(st), (j / NS) & 1);
                    unsigned char* vrow = kv_sm + st * kStageBytes + 2 * kSubTileBytes + row_local * 128;
                    #pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(vrow + kSubTileBytes + c * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                }
                tmem_wait_ld();
                if (vis_lo != ~0ull) { mask_chunk(x0, (uint32_t)vis_lo); mask_chunk(x1, (uint32_t)(vis_lo >> 32)); }
                float mx = fmaxf(chunk_max(x0), chunk_max(x1));
                tmem_ld32(s_addr + 64, x0);
                tmem_ld32(s_addr + 96, x1);
                tmem_wait_ld();
                if (vis_hi != ~0ull) { mask_chunk(x0, (uint32_t)vis_hi); mask_chunk(x1, (uint32_t)(vis_hi >> 32)); }
                mx = fmaxf(mx, fmaxf(chunk_max(x0), chunk_max(x1)));
                // lazy reference maximum, per row; the accumulator is rescaled by the whole warp (the
                // TMEM accesses are warp-wide) whenever one of its rows moved
                const bool need = my_ok && (mx > my_m + thr || (my_m == -INFINITY && mx > -INFINITY));
                if (__any_sync(0xffffffffu, need)) {
                    float alpha = 1.f;
                    if (need) {
                        alpha = (my_m == -INFINITY) ? 0.f : ex2((my_m - mx) * c2);
                        my_m = mx;
                        my_l *= alpha;
                    }
                    if (j > 0) {                                            // O holds earlier tiles
                        if (!mbar_wait_warp(B.o_done(blk, j - 1), ((j - 1) >> 2) & 1)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t o_addr = lane_addr + kOCol + blk * 128;
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
                // second pass: p = 2^(s c2 - m c2), row sum from the unrounded p, P (bf16) over the upper
                // half of the score block -- first the upper 64 keys (their scores are in registers and
                // their columns are the ones P overwrites), then the lower 64, fetched again
                const float mc = (my_m == -INFINITY) ? 0.f : my_m * c2;
                float sum4[4] = {0.f, 0.f, 0.f, 0.f};
                exp_chunk(x0, c2, mc, sum4, s_addr + 64 + 32);
                exp_chunk(x1, c2, mc, sum4, s_addr + 64 + 48);
                tmem_ld32(s_addr, x0);
                tmem_ld32(s_addr + 32, x1);
                tmem_wait_ld();
                if (vis_lo != ~0ull) { mask_chunk(x0, (uint32_t)vis_lo); mask_chunk(x1, (uint32_t)(vis_lo >> 32)); }
                exp_chunk(x0, c2, mc, sum4, s_addr + 64);
                exp_chunk(x1, c2, mc, sum4, s_addr + 64 + 16);
                my_l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                tmem_wait_st();                                            // this job's P is in TMEM
                tc_fence_before();
                mbar_arrive(B.p_full(blk));
            }
        } else {
        // The scores of a job are requested from TMEM at the end of the job before it, ahead of the
        // wait for that job's P stores, so the two latencies overlap; whether those scores are there
        // is probed before the exponentials and only waited for if the probe said no.
        float x0[32], x1[32];
        if (n_jobs > 0) {
            ok = mbar_wait_warp(B.s_full(0), 0);
            tc_fence_after();
            if (ok) { tmem_ld32(lane_addr + 64 * wg, x0); tmem_ld32(lane_addr + 64 * wg + 32, x1); }
        }

        #pragma unroll 1
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int st = j % NS;
            const int tile0 = it.key_begin + j * kTile;          // first key of the tile
            const int j0 = tile0 + 64 * wg;                       // first key of this thread's columns
            #pragma unroll
            for (int blk = 0; blk < NB; ++blk) {
                const int n = j * NB + blk, sb = n % NSB;
                // Visibility word of this row for the thread's 64 columns (all ones away from the
                // draft block and the end of the key range).
                const bool boundary = j0 + 64 > it.key_end || j0 + 64 > kv_len || j0 < lo_row[blk];
                unsigned long long vis = ~0ull;
                if (boundary) {
                    // prefix columns, then the ancestor word shifted to the draft block's column, cut
                    // at the end of the key range
                    const int d0 = kv_len - j0;                             // column of draft token 0 (any sign)
                    const int nval = it.key_end - j0;                       // valid columns (may be <= 0)
                    if (d0 >= 64) vis = ~0ull;
                    else if (d0 > 0) vis = ((1ull << d0) - 1ull) | (anc[blk] << d0);
                    else if (d0 > -64) vis = anc[blk] >> (-d0);
                    else vis = 0ull;
                    if (nval <= 0) vis = 0ull;
                    else if (nval < 64) vis &= (1ull << nval) - 1ull;
                    // prefix keys left of the row's window (the bound never exceeds kv_len, so
                    // the draft block's columns are not touched)
                    const int cut = lo_row[blk] - j0;
                    if (cut >= 64) vis = 0ull;
                    else if (cut > 0) vis &= ~((1ull << cut) - 1ull);
                }
                // V rows past the end of the sequence may hold anything: zero them so 0 * x stays 0
                // (once per tile, by the threads of the first half, thread r taking key row r).
                if (blk == 0 && wg == 0 && tile0 + kTile > n_keys_seq && tile0 + row_local >= n_keys_seq) {
                    mbar_wait(B.v_full(st), (j / NS) & 1);
                    unsigned char* vrow = kv_sm + st * kStageBytes + 2 * kSubTileBytes + row_local * 128;
                    #pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(vrow + kSubTileBytes + c * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                }
                tmem_wait_ld();
                if (boundary) { mask_chunk(x0, (uint32_t)vis); mask_chunk(x1, (uint32_t)(vis >> 32)); }
                const float mx = fmaxf(chunk_max(x0), chunk_max(x1));

                // Rows of padding hold whatever the Q box left there: they never force a rescale.  The
                // barrier also orders both halves' score loads before anyone's P stores (P aliases S).
                const bool need = row_ok[blk] && (mx > m_ref[blk] + thr || (m_ref[blk] == -INFINITY && mx > -INFINITY));
                if (softmax_bar_or(need)) {
                    // some row's maximum moved: the two halves of every row agree on the new reference
                    xch[wg * 128 + row_local] = need ? mx : -INFINITY;
                    softmax_bar_sync();
                    const float cand = fmaxf(need ? mx : -INFINITY, xch[(wg ^ 1) * 128 + row_local]);
                    float alpha = 1.f;
                    if (cand > -INFINITY) {
                        alpha = (m_ref[blk] == -INFINITY) ? 0.f : ex2((m_ref[blk] - cand) * c2);
                        m_ref[blk] = cand;
                        l_run[blk] *= alpha;
                    }
                    if (j > 0 && __any_sync(0xffffffffu, cand > -INFINITY)) {     // O holds earlier tiles: rescale this half of it
                        // every earlier tile's product has been added (they complete in order)
                        if (!mbar_wait_warp(B.o_done(blk, j - 1), ((j - 1) >> 2) & 1)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t o_addr = lane_addr + kOCol + blk * 128 + 64 * wg;
                        #pragma unroll 1
                        for (int ch = 0; ch < 2; ++ch) {
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

                // are the next job's scores there already?  (asked now, used after the exponentials)
                const bool has_next = n + 1 < n_jobs;
                const int sb_next = (n + 1) % NSB;
                const uint32_t par_next = (uint32_t)((n + 1) / NSB) & 1u;
                uint32_t next_ready = 0;
                if (has_next && lane == 0) next_ready = mbar_test_wait(B.s_full(sb_next), par_next) ? 1u : 0u;

                // p = 2^(s c2 - m c2), row sum from the unrounded p, P (bf16) over the S block: this
                // thread's 64 keys land on columns [32 wg, 32 wg + 32) of the block.
                const float mc = (m_ref[blk] == -INFINITY) ? 0.f : m_ref[blk] * c2;
                float sum4[4] = {0.f, 0.f, 0.f, 0.f};
                const uint32_t p_addr = lane_addr + sb * 128 + 32 * wg;
                exp_chunk(x0, c2, mc, sum4, p_addr);
                exp_chunk(x1, c2, mc, sum4, p_addr + 16);
                l_run[blk] += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);

                if (has_next) {                                            // request the next job's scores
                    if (__shfl_sync(0xffffffffu, next_ready, 0) == 0u && !mbar_wait_warp(B.s_full(sb_next), par_next)) {
                        ok = false;
                    } else {
                        tc_fence_after();
                        const uint32_t s_next = lane_addr + sb_next * 128 + 64 * wg;
                        tmem_ld32(s_next, x0);
                        tmem_ld32(s_next + 32, x1);
                    }
                }
                tmem_wait_st();                                            // this job's P is in TMEM
                tc_fence_before();
                mbar_arrive(B.p_full(sb));
                if (!ok) break;
            }
        }

        }
        // ---- epilogue: normalised partial output + natural-log LSE -------------------------------
        if (tid == 0) SPARROW_STAMP(5);                                 // softmax loop left
        const bool direct = plan.seq[it.b].n_splits == 1;                  // the only piece: write the final result
        if (tid == 0) {
            // Global writes start below.  In overlapped mode a lane of the MMA warp has been waiting,
            // since the kernel started, for the counters that allow them (see there).
            uint32_t w = *write_ok;
            for (uint32_t i = 0; w == 0u && i < (1u << 26); ++i) { __nanosleep(20); w = *write_ok; }
            __threadfence_block();
            if (w == 1u && sync.enabled && blockIdx.x == 0) sync.arrivals[(sync.slot + 2) & 3] = 0u;   // the call after next: unused by now
            *write_ok = w == 1u ? 1u : 2u;
        }
        float* xch2 = reinterpret_cast<float*>(misc + kMiscBytes);         // [2][128], two row blocks only
        if constexpr (NB == 2) {
            // each warpgroup hands over its block's per-row results: both warpgroups store both blocks
            xch[wg * 128 + row_local] = my_l > 0.f ? 1.f / my_l : 0.f;
            xch2[wg * 128 + row_local] = my_l > 0.f ? (my_m * c2 + log2f(my_l)) * 0.6931471805599453f : -INFINITY;
            softmax_bar_sync();
        }
        #pragma unroll
        for (int blk = 0; blk < NB; ++blk) {
            const int last_product = n_tiles - 1;
            if (ok) ok = mbar_wait_warp(B.o_done(blk, last_product), (last_product >> 2) & 1);    // the last product is in
            tc_fence_after();
            if (tid == 0 && blk == 0) SPARROW_STAMP(6);                // last product complete
            float inv, lse_val;
            if constexpr (NB == 2) {
                inv = xch[blk * 128 + row_local];
                lse_val = xch2[blk * 128 + row_local];
            } else {
                // the two halves' sums meet (the maxima are already the same)
                xch[wg * 128 + row_local] = l_run[blk];
                softmax_bar_sync();
                const float l_all = l_run[blk] + xch[(wg ^ 1) * 128 + row_local];
                softmax_bar_sync();                                    // xch is reused by the next block
                inv = l_all > 0.f ? 1.f / l_all : 0.f;
                lse_val = l_all > 0.f ? (m_ref[blk] * c2 + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
            }
            ok = ok && *write_ok == 1u;                                // (thread 0 settled it before the barriers above)
            const int h_row = it.kvh * qg + g_row;
            // Staging area for coalesced stores: the Q block (every MMA has completed by now).  Row r
            // holds 16 chunks of 16 bytes (128 halves), chunk c stored at position c ^ (r & 15).
            unsigned char* stage = q_sm + blk * kQBlockBytes;
            const size_t prow0 = (size_t)blockIdx.x * plan.part_rows + blk * kBlockRows;   // first partial row of this block
            if (ok) {
                #pragma unroll 1
                for (int hf = 0; hf < 2; ++hf) {                       // this thread's output dims [64 wg, 64 wg + 64)
                    const int col = wg * 64 + hf * 32;
                    float o[32];
                    tmem_ld32(lane_addr + kOCol + blk * 128 + col, o);
                    tmem_wait_ld();
                    uint4 pk[4];
                    uint32_t* w = reinterpret_cast<uint32_t*>(pk);
                    if (direct) {
                        if (row_ok[blk]) {
                            #pragma unroll
                            for (int c = 0; c < 16; ++c) w[c] = pack_bf16x2(o[2 * c] * inv, o[2 * c + 1] * inv);
                            uint4* dst = reinterpret_cast<uint4*>(
                                args.out + (((size_t)it.b * T + t_row[blk]) * args.n_q_heads + h_row) * kD + col);
                            #pragma unroll
                            for (int c = 0; c < 4; ++c) dst[c] = pk[c];
                        }
                    } else {
                        #pragma unroll
                        for (int c = 0; c < 16; ++c) w[c] = pack_half2(o[2 * c] * inv, o[2 * c + 1] * inv);
                        #pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(stage + row_local * 256 + ((((col >> 3) + c) ^ (row_local & 15)) << 4)) = pk[c];
                    }
                }
                if (row_ok[blk] && wg == 0) {
                    if (direct) args.lse[((size_t)it.b * args.n_q_heads + h_row) * T + t_row[blk]] = lse_val;
                    else *reinterpret_cast<float*>(args.o_part + (prow0 + row_local) * kPartRowHalves + kD) = lse_val;
                }
            }
            softmax_bar_sync();                                        // both halves of every staged row are in place
            if (ok && !direct) {
                // warp w copies rows [16 w, 16 w + 16), two rows (512 contiguous bytes) per instruction
                const int tok_here = min(tpb, max(0, T - (block0 + blk) * tpb));
                const int rows_here = tok_here * qg;
                #pragma unroll 4
                for (int i = 0; i < 8; ++i) {
                    const int r = warp * 16 + 2 * i + (lane >> 4), c = lane & 15;
                    if (r < rows_here) {
                        const uint4 val = *reinterpret_cast<const uint4*>(stage + r * 256 + ((c ^ (r & 15)) << 4));
                        *reinterpret_cast<uint4*>(args.o_part + (prow0 + r) * kPartRowHalves + c * 8) = val;
                    }
                }
            }
        }

        // ---- publish this item; the call's finisher CTAs merge its partials ---------------------------
        // (overlapped mode: arrival words and finisher counters as described at SyncArgs; a
        // stream-ordered call only stores its partials, and a combine kernel follows)
        if (sync.enabled) {
            const int fin_idx = (int)blockIdx.x - (plan.n_items - sync.n_fin);     // >= 0: this CTA is a finisher
            const int kRowsPerBlock = tpb * qg;                        // 126 for 7 heads x 18 tokens
            // The call's row list: for every unit (sequence, KV head, row group) with several pieces,
            // its valid query rows (7 per draft token).  Finisher f takes rows [f chunk, (f + 1) chunk).
            int total = 0;
            for (int b = 0; b < plan.batch; ++b)
                if (plan.seq[b].n_splits > 1) total += plan.n_kv_heads * qg * T;
            const int chunk = sync.n_fin > 0 ? (total + sync.n_fin - 1) / sync.n_fin : 0;
            const int my_begin = fin_idx >= 0 ? min(total, fin_idx * chunk) : 0;
            const int my_end = fin_idx >= 0 ? min(total, my_begin + chunk) : 0;
            const bool merges = my_begin < my_end;
            unsigned* arrive_word = sync.arrivals + sync.slot;
            // the pieces are read by the finishers' bulk copies (async proxy): order this thread's stores ahead of them
            if (!direct) fence_proxy_async_global();
            softmax_bar_sync();                                        // every global store of this CTA has been issued
            if (tid == 0) SPARROW_STAMP(7);                            // partial rows stored
            if (tid == 0) {
                if (!direct) publish_counter(arrive_word);
                if (merges) {
                    // every partial of the call in place, and (overlapped mode) the previous call's final results written
                    // (both words are polled in one loop: the second is usually there already)
                    bool have_all = false, prev_done = false;
                    #pragma unroll 1
                    for (uint32_t i = 0; i < kCounterPolls && !(have_all && prev_done); ++i) {
                        if (!have_all) have_all = ld_acquire(arrive_word) == (unsigned)sync.n_arrive;
                        if (!prev_done) prev_done = (int32_t)(ld_acquire(sync.fin_done + (sync.parity ^ 1)) - sync.fin_wait_other) >= 0;
                        if (!(have_all && prev_done)) __nanosleep(i < 256 ? 20 : 200);
                    }
                    SPARROW_STAMP(8);                                   // all arrivals seen
                    if (!have_all) atomicOr(args.status, timeout_bits(kSiteArrivals));
                    else if (!prev_done) atomicOr(args.status, timeout_bits(kSiteFinOther));
                    SPARROW_STAMP(9);                                   // previous call's finishers seen
                    *fin_go = (have_all && prev_done) ? 1 : 0;
                }
            }
            if (merges) {
                softmax_bar_sync();
                if (*fin_go) {
                    // 16 R G threads merge R rows at a time.  The rows' pieces are first brought into the
                    // (idle) K/V ring by bulk copies, [piece][row][272 bytes], one copy per piece and
                    // block touched -- far fewer and larger requests than per-thread loads.  (The pieces
                    // were written with ordinary stores and the copies read through the async proxy: the
                    // writers issued the proxy fence, before they published their piece.)
                    // Thread (row i, 16-byte chunk c, piece group g) then folds pieces g, g + G, ... of its
                    // row into a running (max, sum, weighted output); the groups' results meet in shared
                    // memory (the Q blocks, idle by now).
                    constexpr int kRowBytes = kPartRowHalves * 2;               // 272
                    float* red = reinterpret_cast<float*>(q_sm);                // [256][10]: 8 outputs, sum, max
                    int ubase = 0, phase = 0;
                    bool fin_ok = true;
                    #pragma unroll 1
                    for (int b = 0; b < plan.batch; ++b) {
                        const int ns = plan.seq[b].n_splits;
                        if (ns == 1) continue;
                        // rows per pass: a power of two, no more than this finisher has, than fit the ring
                        // with all their pieces, or than 16
                        int R = 1;
                        while (R < 16 && R < chunk) R <<= 1;
                        while (R > 1 && R * ns * kRowBytes > NS * kStageBytes) R >>= 1;
                        const int G = 16 / R;                                   // piece groups
                        const int c16 = tid & 15, grp_p = (tid >> 4) % G, row_i = tid / (16 * G);
                        const size_t piece_pitch = (size_t)plan.part_rows * kPartRowHalves;      // halves between pieces
                        #pragma unroll 1
                        for (int u = 0; u < plan.n_kv_heads * plan.n_groups; ++u) {
                            const int kvh = u / plan.n_groups, grp = u - kvh * plan.n_groups;
                            const int tok0 = grp * NB * tpb;                        // first token of this row group
                            const int list_len = qg * min(NB * tpb, T - tok0);  // its valid rows
                            const int row_begin = max(my_begin, ubase) - ubase, row_end = min(my_end, ubase + list_len) - ubase;
                            ubase += list_len;
                            if (row_begin >= row_end) continue;                    // (the same in every thread of the CTA)
                            const size_t item0 = (size_t)plan.seq[b].item_begin + (size_t)u * ns;
                            #pragma unroll 1
                            for (int r0 = row_begin; r0 < row_end; r0 += R, phase ^= 1) {
                                const int n_here = min(R, row_end - r0);
                                // the rows may straddle the unit's two blocks: rows [r0, split) and [split, r0 + n_here)
                                const int split = (r0 < kRowsPerBlock && r0 + n_here > kRowsPerBlock) ? kRowsPerBlock : r0 + n_here;
                                if (tid == 0) mbar_expect_tx(B.fin(), (uint32_t)(n_here * ns * kRowBytes));
                                softmax_bar_sync();                                // the ring's previous contents have been read, the byte count is posted
                                {
                                    const int bk0 = r0 / kRowsPerBlock;
                                    const __half* first = args.o_part + (item0 * plan.part_rows + (size_t)(bk0 * kBlockRows + r0 - bk0 * kRowsPerBlock)) * kPartRowHalves;
                                    const __half* second = args.o_part + (item0 * plan.part_rows + (size_t)kBlockRows) * kPartRowHalves;
                                    for (int sp = tid; sp < ns; sp += 256) {           // thread sp brings piece sp
                                        const uint32_t dst = smem_u32(kv_sm) + (uint32_t)(sp * n_here * kRowBytes);
                                        bulk_load(dst, first + (size_t)sp * piece_pitch, (uint32_t)(split - r0) * kRowBytes, B.fin());
                                        if (split < r0 + n_here)
                                            bulk_load(dst + (uint32_t)(split - r0) * kRowBytes, second + (size_t)sp * piece_pitch,
                                                      (uint32_t)(r0 + n_here - split) * kRowBytes, B.fin());
                                    }
                                }
                                if (tid == 0) SPARROW_STAMP(12);        // bulk copies issued
                                fin_ok = fin_ok && mbar_wait_warp(B.fin(), phase);
                                if (tid == 0) SPARROW_STAMP(15);        // bulk copies landed
                                const int idx = r0 + row_i;                            // row of the unit's list: token idx / 7, head idx % 7
                                const bool active = fin_ok && row_i < n_here;
                                const uint32_t pstride = (uint32_t)n_here * kRowBytes;     // bytes between pieces in the ring
                                const uint32_t row_sm = smem_u32(kv_sm) + (uint32_t)row_i * kRowBytes;
                                float m_run = -INFINITY, s_run = 0.f;                  // natural-log units
                                float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                                if (active) {
                                    #pragma unroll 2
                                    for (uint32_t sp = grp_p, a_o = row_sm + grp_p * pstride; sp < (uint32_t)ns; sp += G, a_o += G * pstride) {
                                        const float l = lds_f32(a_o + 2 * kD);
                                        uint32_t raw[4];
                                        lds_v4(a_o + c16 * 16, raw);
                                        if (l == -INFINITY) continue;                  // a piece that saw no visible key
                                        const float m_new = fmaxf(m_run, l);
                                        const float a = ex2((m_run - m_new) * 1.4426950408889634f);   // 0 for the first piece
                                        const float w = ex2((l - m_new) * 1.4426950408889634f);
                                        s_run = fmaf(s_run, a, w);
                                        #pragma unroll
                                        for (int q = 0; q < 4; ++q) {
                                            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&raw[q]));
                                            acc[2 * q] = fmaf(acc[2 * q], a, w * f.x); acc[2 * q + 1] = fmaf(acc[2 * q + 1], a, w * f.y);
                                        }
                                        m_run = m_new;
                                    }
                                }
                                if (tid == 0) SPARROW_STAMP(13);        // pieces folded
                                if (G > 1) {                                           // (G is the same in every thread)
                                    softmax_bar_sync();                                // the pass before has been read
                                    #pragma unroll
                                    for (int q = 0; q < 8; ++q) red[tid * 10 + q] = acc[q];
                                    red[tid * 10 + 8] = s_run;
                                    red[tid * 10 + 9] = m_run;
                                    softmax_bar_sync();
                                    if (grp_p == 0) {
                                        const float* mine = red + tid * 10;
                                        float m_all = m_run;
                                        for (int g2 = 1; g2 < G; ++g2) m_all = fmaxf(m_all, mine[g2 * 160 + 9]);
                                        const float a0 = m_run == -INFINITY ? 0.f : ex2((m_run - m_all) * 1.4426950408889634f);
                                        s_run *= a0;
                                        #pragma unroll
                                        for (int q = 0; q < 8; ++q) acc[q] *= a0;
                                        for (int g2 = 1; g2 < G; ++g2) {
                                            const float* o = mine + g2 * 160;
                                            if (o[9] == -INFINITY) continue;
                                            const float ag = ex2((o[9] - m_all) * 1.4426950408889634f);
                                            s_run = fmaf(o[8], ag, s_run);
                                            #pragma unroll
                                            for (int q = 0; q < 8; ++q) acc[q] = fmaf(o[q], ag, acc[q]);
                                        }
                                        m_run = m_all;
                                    }
                                }
                                if (tid == 0) SPARROW_STAMP(14);        // groups reduced
                                if (active && grp_p == 0) {
                                    const int t = tok0 + idx / qg;
                                    const int h = kvh * qg + idx % qg;
                                    const float inv = s_run > 0.f ? __fdividef(1.f, s_run) : 0.f;
                                    uint4 pk;
                                    pk.x = pack_bf16x2(acc[0] * inv, acc[1] * inv); pk.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
                                    pk.z = pack_bf16x2(acc[4] * inv, acc[5] * inv); pk.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
                                    *reinterpret_cast<uint4*>(args.out + (((size_t)b * T + t) * args.n_q_heads + h) * kD + c16 * 8) = pk;
                                    if (c16 == 0) args.lse[((size_t)b * args.n_q_heads + h) * T + t] = s_run > 0.f ? m_run + __logf(s_run) : -INFINITY;
                                }
                            }
                        }
                    }
                    if (!fin_ok) atomicOr(args.status, timeout_bits(kSiteFinCopies));
                }
                if (tid == 0) SPARROW_STAMP(10);                        // merged rows written
                softmax_bar_sync();
            }
            if (tid == 0) {
                if (direct) publish_counter(sync.fin_done + sync.parity);
                if (fin_idx >= 0) publish_counter(sync.fin_done + sync.parity);
            }
        }
        if (!ok) { atomicOr(args.status, timeout_bits(kSiteSoftmax)); *abort_flag = 1; }
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
    if (threadIdx.x == 0) SPARROW_STAMP(11);                            // leaving
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

}  // namespace tc
}  // namespace sparrow
