// Split-KV pass with row-gathered K/V loads: the kernel behind the text-anchored window mode
// (Eq. 2: keys/values restricted to the anchor list) and a general path for any key layout.
//
// One CTA = one work item (sequence, KV head, one 128-row block of packed query rows, key-range
// piece).  The g query heads of the GQA group times p = 128 / g draft tokens form one block (row
// r = (t % p) g + head; g = 7: 18 tokens, two rows of padding), so every gathered K/V row is loaded once per KV head
// and block.  K/V rows are fetched
// with 16-byte cp.async (row index = key index, or anchor_idx[key] when gathering) into a
// two-stage XOR-swizzled shared-memory ring; S = QK^T and O += PV run on mma.sync m16n8k16 bf16
// with fp32 accumulation; the online softmax is fp32 with quad shuffles.  Per item the kernel
// writes a normalised fp16 partial output and a natural-log LSE for the combine step (or, when
// the sequence has a single piece, the final bf16 output and LSE).
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace sparrow {

struct SplitArgs {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const int32_t* parents;      // verification: DEV [B][T]; anchored: DEV [B][tree_nodes] or nullptr (chain)
    const int32_t* anchor_idx;   // anchored: DEV [B][n_anchor]; nullptr in verification mode
    int32_t n_anchor;
    int32_t window;
    int32_t tree_nodes;          // anchored mode with a draft tree: its nodes are the last tree_nodes anchors, the
                                 // queries the last T of them; 0 = chain rule for every anchor
    int32_t n_q_heads;
    int32_t kv_capacity;
    int64_t kv_stride_batch;
    int64_t kv_stride_head;
    float scale_log2e;           // softmax_scale * log2(e)
    __half* o_part;              // [n_items][part_rows] partial rows: 128 fp16 outputs + fp32 LSE (kPartRowHalves)
    __nv_bfloat16* out;          // final output, written directly for sequences with one piece
    float* lse;
    unsigned* status;
    int32_t early_dependents;    // the next kernel in the stream is this call's combine step, launched programmatically
};

namespace gather {

constexpr int kThreads = 256;
constexpr int kRows = 128;        // packed query rows per CTA (8 warps x 16)
constexpr int kTile = 64;         // keys per stage
constexpr int kStageBytes = kTile * kD * 2;            // one K or V tile: 16 KB
constexpr int kSmemBytes = 4 * kStageBytes + kMaxT * 8 + kMaxT * 4 + 2 * kTile * 4;

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}
// byte offset of 16-byte chunk c of row r inside a [rows][128] bf16 tile (XOR swizzle)
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 256 + ((c ^ (r & 7)) << 4)); }

__global__ void __launch_bounds__(kThreads, 1)
split_gather_kernel(const __grid_constant__ SplitPlan plan, const __grid_constant__ SplitArgs args)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* kv_smem = smem;                                   // [2 stages][K 16K | V 16K]
    unsigned char* q_stage = smem + 2 * kStageBytes;                 // stage 1 doubles as the staging area of the Q block
    unsigned long long* anc_s = reinterpret_cast<unsigned long long*>(smem + 4 * kStageBytes);
    int32_t* qpos_s = reinterpret_cast<int32_t*>(smem + 4 * kStageBytes + kMaxT * 8);
    int32_t* apos_s = qpos_s + kMaxT;                                // [2][kTile] gathered row ids

    // The combine kernel may be scheduled now: it waits for this grid as a whole before it reads.
    if (args.early_dependents) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g4 = lane >> 2, c4 = lane & 3;
    const Item it = decode_item(plan, blockIdx.x);
    const int T = plan.T;
    const bool anchored = args.anchor_idx != nullptr;
    const int kv_len = anchored ? 0 : plan.seq[it.b].kv_len;
    const int32_t* aidx = anchored ? args.anchor_idx + (size_t)it.b * args.n_anchor : nullptr;

    const __nv_bfloat16* kbase = args.k + (size_t)it.b * args.kv_stride_batch + (size_t)it.kvh * args.kv_stride_head;
    const __nv_bfloat16* vbase = args.v + (size_t)it.b * args.kv_stride_batch + (size_t)it.kvh * args.kv_stride_head;
    const int n_tiles = (it.key_end - it.key_begin + kTile - 1) / kTile;

    // Row indices of a tile, four per thread (one per 16-byte chunk this thread copies).  In anchored
    // mode they come from the anchor list: a memory round trip that the row copies depend on, so
    // the indices of a tile are fetched one whole tile ahead of its copies.
    constexpr int kAbsent = -2147483647 - 1;                 // key past the end of the piece
    constexpr int kPerThread = (kTile * 16) / kThreads;      // 4
    // The thread that owns chunk 0 of a row also fetches the anchor before it: the list must be
    // strictly increasing (the window rule and the position of the tree nodes rely on it).
    const bool checks_order = anchored && (tid & 15) == 0;
    auto fetch_rows = [&](int tile, int (&rows)[kPerThread], int (&before)[kPerThread]) {
        #pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int r = (tid + i * kThreads) >> 4;
            const int j = it.key_begin + tile * kTile + r;
            rows[i] = j < it.key_end ? (anchored ? __ldg(aidx + j) : j) : kAbsent;
            before[i] = (checks_order && j > 0 && j < it.key_end) ? __ldg(aidx + j - 1) : kAbsent;
        }
    };
    auto issue_tile = [&](int stage, const int (&rows)[kPerThread], const int (&before)[kPerThread]) {
        unsigned char* ks = kv_smem + stage * 2 * kStageBytes;
        unsigned char* vs = ks + kStageBytes;
        #pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int idx = tid + i * kThreads;
            const int r = idx >> 4, c = idx & 15;
            int row = rows[i];
            if (checks_order && row != kAbsent && before[i] != kAbsent && row <= before[i]) atomicOr(args.status, kStatAnchor);
            if (row == kAbsent) {
                row = -1;
            } else if (row < 0 || row >= args.kv_capacity) {
                atomicOr(args.status, kStatAnchor);
                row = -1;
            }
            if (anchored && c == 0) apos_s[stage * kTile + r] = row;
            const size_t off = (size_t)(row < 0 ? 0 : row) * kD + c * 8;
            const int bytes = row < 0 ? 0 : 16;          // 0 -> the 16 bytes are zero-filled
            cp_async16(smem_u32(ks + swz(r, c)), kbase + off, bytes);
            cp_async16(smem_u32(vs + swz(r, c)), vbase + off, bytes);
        }
    };
    int rows_next[kPerThread], before_next[kPerThread];

    // Tile 0 is requested before anything else: its two dependent round trips (anchor indices,
    // then the rows) overlap the loads of the prologue.  It lands in stage 0; the packed Q block is
    // staged in stage 1, which the ring only reuses after Q has moved to registers.
    if (n_tiles > 0) { fetch_rows(0, rows_next, before_next); issue_tile(0, rows_next, before_next); }
    cp_async_commit();
    if (n_tiles > 1) fetch_rows(1, rows_next, before_next);

    // ---- prologue: masks / query positions, packed Q block -> registers --------------------
    const int tree_nodes = anchored ? args.tree_nodes : 0;
    // The parent array is staged in shared memory first: the walk up the tree is a chain of
    // dependent reads, one memory round trip each if it went to global memory.
    __shared__ int32_t par_s[kMaxT];
    const int n_par = anchored ? tree_nodes : T;
    if (tid < n_par) par_s[tid] = __ldg(args.parents + (size_t)it.b * n_par + tid);
    if (anchored && tid < T) {
        int p = aidx[args.n_anchor - T + tid];
        if (p < 0 || p >= args.kv_capacity) { atomicOr(args.status, kStatAnchor); p = -1; }
        qpos_s[tid] = p;
    }
    __syncthreads();
    if (tid < n_par) anc_s[tid] = ancestor_word(par_s, n_par, tid, args.status);
    {
        constexpr int kChunksPerThread = kRows * 16 / kThreads;      // 8: all loads first, then the stores
        uint4 val[kChunksPerThread];
        #pragma unroll
        for (int u = 0; u < kChunksPerThread; ++u) {
            const int i = tid + u * kThreads;
            const int r = i >> 4, c = i & 15;
            const int t = it.group * plan.tok_per_block + r / plan.group, g = r % plan.group;
            val[u] = make_uint4(0, 0, 0, 0);
            if (r < plan.tok_per_block * plan.group && t < T) {
                val[u] = __ldg(reinterpret_cast<const uint4*>(
                    args.q + (((size_t)it.b * T + t) * args.n_q_heads + it.kvh * plan.group + g) * kD + c * 8));
            }
        }
        #pragma unroll
        for (int u = 0; u < kChunksPerThread; ++u) {
            const int i = tid + u * kThreads;
            *reinterpret_cast<uint4*>(q_stage + swz(i >> 4, i & 15)) = val[u];
        }
    }
    __syncthreads();
    uint32_t qf[8][4];
    {
        const int r = warp * 16 + (lane & 15);
        #pragma unroll
        for (int ks = 0; ks < 8; ++ks)
            ldsm_x4(smem_u32(q_stage + swz(r, ks * 2 + (lane >> 4))), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    // per-thread row state: rows lr0 = warp*16+g4 and lr0+8
    int row_t[2]; bool row_ok[2]; unsigned long long row_anc[2]; int row_qpos[2];
    #pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const int lr = warp * 16 + g4 + rr * 8;
        row_t[rr] = it.group * plan.tok_per_block + lr / plan.group;
        row_ok[rr] = lr < plan.tok_per_block * plan.group && row_t[rr] < T;
        const int t = row_ok[rr] ? row_t[rr] : 0;
        row_anc[rr] = anchored ? (tree_nodes > 0 ? anc_s[tree_nodes - T + t] : 0ull) : anc_s[t];
        row_qpos[rr] = anchored ? qpos_s[t] : 0;
    }
    const bool warp_has_rows = __any_sync(0xffffffffu, row_ok[0] || row_ok[1]);
    __syncthreads();                      // Q staging area is reused by the K/V ring from here on

    float o[16][4];
    #pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    const float c2 = args.scale_log2e;

    for (int tile = 0; tile < n_tiles; ++tile) {
        const int stage = tile & 1;
        if (tile + 1 < n_tiles) issue_tile(stage ^ 1, rows_next, before_next);
        cp_async_commit();
        if (tile + 2 < n_tiles) fetch_rows(tile + 2, rows_next, before_next);     // arrives while this tile is being worked on
        cp_async_wait<1>();
        __syncthreads();
        const unsigned char* ks = kv_smem + stage * 2 * kStageBytes;
        const unsigned char* vs = ks + kStageBytes;

        // A warp whose 16 rows are all padding (fewer than 126 packed rows in this block) has no
        // arithmetic to do: it only takes part in the loads and the barriers.
        if (warp_has_rows) {
        // S = Q K^T for 16 rows x 64 keys
        float s[8][4];
        #pragma unroll
        for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
        #pragma unroll
        for (int kstep = 0; kstep < 8; ++kstep) {
            #pragma unroll
            for (int np = 0; np < 4; ++np) {
                const int mi = lane >> 3;
                const int key = np * 16 + (mi >> 1) * 8 + (lane & 7);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(smem_u32(ks + swz(key, kstep * 2 + (mi & 1))), b0, b1, b2, b3);
                mma_bf16(s[2 * np], qf[kstep], b0, b1);
                mma_bf16(s[2 * np + 1], qf[kstep], b2, b3);
            }
        }
        // visibility
        const int j0 = it.key_begin + tile * kTile;
        const bool need_mask = anchored || (j0 + kTile > it.key_end) || (j0 + kTile > kv_len);
        if (need_mask) {
            #pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                #pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int rr = e >> 1;
                    const int col = nt * 8 + 2 * c4 + (e & 1);
                    const int j = j0 + col;
                    bool vis = j < it.key_end;
                    if (vis) {
                        if (anchored) {
                            const int p = apos_s[stage * kTile + col];
                            const int qp = row_qpos[rr];
                            const int node = j - (args.n_anchor - tree_nodes);     // >= 0: a node of the draft tree
                            if (tree_nodes > 0 && node >= 0)
                                vis = p >= 0 && qp >= 0 && ((row_anc[rr] >> node) & 1ull);
                            else
                                vis = p >= 0 && qp >= 0 && p <= qp && (args.window <= 0 || qp - args.window < p);
                        } else if (j >= kv_len) {
                            vis = (row_anc[rr] >> (j - kv_len)) & 1ull;
                        }
                    }
                    if (!vis) s[nt][e] = -INFINITY;
                }
            }
        }
        // online softmax (fp32); the row sum uses the unrounded probabilities
        float alpha[2];
        #pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
            float mx = -INFINITY;
            #pragma unroll
            for (int nt = 0; nt < 8; ++nt) mx = fmaxf(mx, fmaxf(s[nt][2 * rr], s[nt][2 * rr + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[rr], mx);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            alpha[rr] = exp2f((m_run[rr] - m_use) * c2);
            m_run[rr] = m_new;
            const float mc = m_use * c2;
            float sum = 0.f;
            #pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                s[nt][2 * rr] = exp2f(fmaf(s[nt][2 * rr], c2, -mc));
                s[nt][2 * rr + 1] = exp2f(fmaf(s[nt][2 * rr + 1], c2, -mc));
                sum += s[nt][2 * rr] + s[nt][2 * rr + 1];
            }
            l_run[rr] = l_run[rr] * alpha[rr] + sum;
        }
        #pragma unroll
        for (int i = 0; i < 16; ++i) {
            o[i][0] *= alpha[0]; o[i][1] *= alpha[0];
            o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
        }
        // O += P V
        #pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t a[4];
            a[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
            a[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
            a[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
            a[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
            #pragma unroll
            for (int dn = 0; dn < 8; ++dn) {
                const int mi = lane >> 3;
                const int key = kk * 16 + (mi & 1) * 8 + (lane & 7);
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(smem_u32(vs + swz(key, dn * 2 + (mi >> 1))), b0, b1, b2, b3);
                mma_bf16(o[2 * dn], a, b0, b1);
                mma_bf16(o[2 * dn + 1], a, b2, b3);
            }
        }
        }   // warp_has_rows
        __syncthreads();                  // this stage is refilled by the next iteration's loads
    }
    cp_async_wait<0>();

    // ---- epilogue: normalised partial output + natural-log LSE ------------------------------
    #pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        float l = l_run[rr];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        if (!row_ok[rr]) continue;
        const int lr = warp * 16 + g4 + rr * 8;
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const float lse_val = l > 0.f ? (m_run[rr] * c2 + log2f(l)) * 0.6931471805599453f : -INFINITY;
        if (plan.seq[it.b].n_splits == 1) {                 // the only piece: write the final result
            const int t = row_t[rr], h = it.kvh * plan.group + lr % plan.group;
            __nv_bfloat16* dst = args.out + (((size_t)it.b * T + t) * args.n_q_heads + h) * kD;
            #pragma unroll
            for (int nt = 0; nt < 16; ++nt)
                *reinterpret_cast<uint32_t*>(dst + nt * 8 + 2 * c4) = pack_bf16(o[nt][2 * rr] * inv, o[nt][2 * rr + 1] * inv);
            if (c4 == 0) args.lse[((size_t)it.b * args.n_q_heads + h) * T + t] = lse_val;
        } else {
            const size_t prow = (size_t)blockIdx.x * plan.part_rows + lr;
            __half* dst = args.o_part + prow * kPartRowHalves;
            #pragma unroll
            for (int nt = 0; nt < 16; ++nt)
                *reinterpret_cast<__half2*>(dst + nt * 8 + 2 * c4) = __floats2half2_rn(o[nt][2 * rr] * inv, o[nt][2 * rr + 1] * inv);
            if (c4 == 0) *reinterpret_cast<float*>(dst + kD) = lse_val;
        }
    }
}

}  // namespace gather
}  // namespace sparrow
