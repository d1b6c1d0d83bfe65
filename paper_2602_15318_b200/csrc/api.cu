// Host side of libsparrow_attn: context, argument validation, split planning and kernel launches
// behind the C ABI declared in include/sparrow_attn.h.  No torch types, no allocation on the hot
// calls, no host synchronisation on the hot calls.
#include "sparrow_attn.h"

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "combine.cuh"
#include "common.cuh"
#include "accept.cuh"
#include "accept_sample.cuh"
#include "kv_rows.cuh"
#include "split_gather.cuh"
#include "verify_tc.cuh"
#include "hsr_fuse.cuh"
#include "window.cuh"

using namespace sparrow;

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TensorMapEntry {
    const void* base;        // nullptr: free slot
    int tag;                 // 0: K/V cache map; n > 0: Q map for n = batch * T tokens
    CUtensorMap map;
};
// Hashed by (base pointer, tag), a bucket being kMapWays consecutive slots: room for the q / K / V
// buffers of a few hundred layers or rotation slots before anything is encoded twice.
constexpr int kMapCacheSize = 1024;
constexpr int kMapWays = 8;

// Fused calls that can still be resident on the GPU when a new one starts: each has at least one
// CTA on an SM of its own, so there are fewer of them than SMs.
constexpr int kRecentCalls = 192;
struct RecentCall {
    uintptr_t out[2], lse[2];    // [begin, end) of what the call writes
};

struct sparrow_ctx {
    TensorMapEntry maps[kMapCacheSize];      // Q / K / V tensor maps, keyed by base pointer (and token count)
    unsigned evict_tick;
    TensorMapEncodeFn encode;
    sparrow_layout layout;
    int device;
    int n_sm;
    int plan_policy;                         // sparrow_plan_policy
    unsigned char* ws;
    size_t ws_bytes;
    size_t part_offset;                      // first byte of the split-KV partials in the workspace
    int part_buffers;                        // 2: alternate by call parity (fused mode); 1: stream-ordered calls only
    std::atomic<long long> launches;
    bool use_pdl;
    bool log_plans;                          // SPARROW_LOG=1 when the context was created: one line per call on stderr
    bool overlap_single_calls;               // sparrow_set_call_overlap()
    bool chain_next;                         // the call being enqueued directly follows this context's previous fused call
    // Host mirror of the ordering counters in the workspace (see SyncArgs): call sequence number
    // of the fused calls and, per call parity, the cumulative number of finishers launched so far.
    uint32_t seq;
    uint32_t fin_total[2];
    uint32_t fin_before_last[2];             // fin_total[p] as it was before the last call of parity p
    // Memory the previous fused call touches (out, lse, q, parents, k, v, window bounds), as [begin, end) addresses:
    // a call whose outputs overlap none of it need not wait for that call's merge.
    uintptr_t prev_ranges[7][2];
    bool prev_valid;
    // Outputs of the fused calls launched since this context's last launch in plain stream order.
    RecentCall recent[kRecentCalls];
    int n_recent, recent_head;
    uint32_t last_status_word;   // raw word read by the last sparrow_last_device_status()
};

namespace {

constexpr size_t kStatusBytes = 1024;      // word 0: sticky status; words 16, 17: finisher counters
constexpr size_t kFinDoneOffset = 64;
constexpr size_t kArrivalsOffset = 128;     // words 32..35: arrival words of the four call slots
constexpr int kMinPieceKeys = 128;
// The gathered kernel works on 64-key tiles and pays two dependent memory round trips per tile
// (anchor indices, then the rows), which a CTA with several tiles takes one after the other: short
// anchor lists are cut down to single tiles, one CTA each.
constexpr int kMinGatherPieceKeys = 64;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Staging {
    size_t q, out, lse, parents, k_new, v_new, total;
};

Staging staging_layout(const sparrow_layout& L)
{
    Staging s;
    const size_t B = (size_t)L.batch;
    s.q = 0;
    s.out = s.q + align_up(B * kMaxT * L.n_q_heads * kD * 2, 256);
    s.lse = s.out + align_up(B * kMaxT * L.n_q_heads * kD * 2, 256);
    s.parents = s.lse + align_up(B * kMaxT * L.n_q_heads * 4, 256);
    s.k_new = s.parents + align_up(B * kMaxT * 4, 256);
    s.v_new = s.k_new + align_up(B * L.n_kv_heads * kMaxT * kD * 2, 256);
    s.total = s.v_new + align_up(B * L.n_kv_heads * kMaxT * kD * 2, 256);
    return s;
}

// 128-row blocks (18 draft tokens each) one work item of the tensor-core pass handles
int blocks_per_group_tc(int T, int group) { return T <= tokens_per_block(group) ? 1 : 2; }

int max_items(int n_sm, int batch, int n_kv_heads, int n_groups)
{
    return n_sm + batch * n_kv_heads * n_groups;
}

// Chooses the number of key-range pieces per sequence so that the total number of work items is
// close to (and not above) the SM count while every item streams about the same number of keys.
// key0 (optional): per sequence, the first key that is streamed at all (a multiple of 128).
sparrow_status make_plan(int n_sm, int batch, int n_kv_heads, int group, const int32_t* n_keys, int T, int blocks_per_group,
                         SplitPlan* p, int min_piece_keys = kMinPieceKeys, const int32_t* key0 = nullptr)
{
    if (batch < 1 || batch > kMaxBatch || T < 1 || T > kMaxT || n_kv_heads < 1 || n_sm < 1 || group < 1 || group > kMaxGroup)
        return SPARROW_ERR_SHAPE;
    const int tpb = tokens_per_block(group);
    std::memset(p, 0, sizeof(*p));
    p->batch = batch;
    p->T = T;
    p->T_tree = T;
    p->group = group;
    p->tok_per_block = tpb;
    p->M = group * T;
    p->blocks_per_group = blocks_per_group;
    p->n_groups = (T + tpb * blocks_per_group - 1) / (tpb * blocks_per_group);
    p->n_kv_heads = n_kv_heads;
    p->piece_tile = min_piece_keys < kKeyTile ? min_piece_keys : kKeyTile;
    p->part_rows = blocks_per_group * kBlockRows + 1;    // odd pitch: partial rows of successive pieces must not share L2 sets
    const int units = n_kv_heads * p->n_groups;
    int max_keys = 1;
    int32_t streamed[kMaxBatch];                  // keys each sequence streams
    for (int b = 0; b < batch; ++b) {
        const int32_t k0 = key0 ? key0[b] : 0;
        if (n_keys[b] < 1 || k0 < 0 || k0 >= n_keys[b] || (k0 % kKeyTile) != 0) return SPARROW_ERR_SHAPE;
        streamed[b] = n_keys[b] - k0;
        if (streamed[b] > max_keys) max_keys = streamed[b];
    }
    auto items_for = [&](long long L) {
        long long n = 0;
        for (int b = 0; b < batch; ++b) n += (long long)units * ((streamed[b] + L - 1) / L);
        return n;
    };
    long long lo = min_piece_keys, hi = max_keys > min_piece_keys ? max_keys : min_piece_keys;
    if (items_for(lo) > n_sm) {                 // smallest piece length that fits the SM count
        while (lo < hi) {
            const long long mid = (lo + hi) / 2;
            if (items_for(mid) <= n_sm) hi = mid; else lo = mid + 1;
        }
    }
    int total = 0;
    for (int b = 0; b < batch; ++b) {
        p->seq[b].n_keys = n_keys[b];
        p->seq[b].key0 = key0 ? key0[b] : 0;
        p->seq[b].n_splits = (int)((streamed[b] + lo - 1) / lo);
        p->seq[b].item_begin = total;
        total += units * p->seq[b].n_splits;
    }
    p->n_items = total;
    return SPARROW_OK;
}

// n_q_heads = g * n_kv_heads with 1 <= g <= kMaxGroup
bool layout_heads_ok(const sparrow_layout& L)
{
    return L.n_kv_heads >= 1 && L.n_q_heads >= L.n_kv_heads && L.n_q_heads % L.n_kv_heads == 0 && L.n_q_heads / L.n_kv_heads <= kMaxGroup;
}
int layout_group(const sparrow_layout& L) { return L.n_q_heads / L.n_kv_heads; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Device-side address of a host buffer that kernels can reach themselves (page-locked memory,
// which unified addressing maps into every device; 16-byte aligned), else nullptr: the caller
// then goes through copies.
template <class P>
P* device_view(P* host)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer || !aligned16(at.devicePointer)) return nullptr;
    return static_cast<P*>(at.devicePointer);
}


size_t fixed_bytes(const sparrow_layout& L) { return kStatusBytes + staging_layout(L).total; }
size_t part_bytes(size_t rows) { return align_up(rows * kPartRowHalves * sizeof(__half), 256); }

// The partial outputs start at part_offset (behind the header and, for a caller-provided
// workspace, the staging area) and are double-buffered by call parity where calls can overlap.
size_t part_half_bytes(const sparrow_ctx* c)
{
    return c->ws_bytes > c->part_offset ? ((c->ws_bytes - c->part_offset) / c->part_buffers) & ~(size_t)255 : 0;
}

sparrow_status check_ws(const sparrow_ctx* c, const SplitPlan& p)
{
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    return part_bytes((size_t)p.n_items * p.part_rows) <= part_half_bytes(c) ? SPARROW_OK : SPARROW_ERR_WORKSPACE;
}

__half* o_part_ptr(const sparrow_ctx* c, int parity)
{
    return reinterpret_cast<__half*>(c->ws + c->part_offset + (c->part_buffers > 1 ? parity : 0) * part_half_bytes(c));
}

// Ordering arguments of the next call and, once it is enqueued, the advance of the host mirror.
// Calls that are being captured into a graph, or made with programmatic launch switched off, or
// served by the gathered kernel run in stream-ordered mode: their kernels touch no counter.
// Will this call run in fused mode, i.e. may it overlap its neighbours in the stream?  Not while the
// stream is being captured, not with programmatic launch switched off, not on the gathered kernel.
bool call_overlaps(const sparrow_ctx* c, cudaStream_t st, bool fused_kernel)
{
    if (!fused_kernel || !c->use_pdl) return false;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); return false; }
    return cap == cudaStreamCaptureStatusNone;
}

// Work items a policy aims for.  Fewer, longer pieces leave SMs free for the next calls in the
// stream, which then overlap this one: better sustained throughput, longer single-call latency.
int policy_target(int n_sm, int policy)
{
    switch (policy) {
        case SPARROW_PLAN_THROUGHPUT: return n_sm / 7 > 1 ? n_sm / 7 : 1;
        case SPARROW_PLAN_BALANCED: return (3 * n_sm) / 8 > 1 ? (3 * n_sm) / 8 : 1;
        default: return n_sm;
    }
}

// Calls that cannot overlap others always get one wave over all SMs.
int plan_target(const sparrow_ctx* c, bool overlaps)
{
    return overlaps ? policy_target(c->n_sm, c->plan_policy) : c->n_sm;
}

constexpr int kCallRanges = 7;
struct CallRanges {
    uintptr_t r[kCallRanges][2];     // out, lse (written), q, parents, k, v, window bounds (read)
};

CallRanges call_ranges(const sparrow_ctx* c, const void* q, const void* k, const void* v, const int32_t* parents, int T_tree,
                       int T, const int32_t* first_visible, const void* out, const float* lse)
{
    const sparrow_layout& L = c->layout;
    const size_t tok_bytes = (size_t)L.batch * T * L.n_q_heads * kD * 2;
    const size_t kv_bytes = ((size_t)(L.batch - 1) * L.kv_stride_batch + (size_t)(L.n_kv_heads - 1) * L.kv_stride_head +
                             (size_t)L.kv_capacity * kD) * 2;
    CallRanges cr;
    auto set = [&](int i, const void* p, size_t n) {
        cr.r[i][0] = reinterpret_cast<uintptr_t>(p);
        cr.r[i][1] = cr.r[i][0] + n;
    };
    set(0, out, tok_bytes);
    set(1, lse, (size_t)L.batch * L.n_q_heads * T * 4);
    set(2, q, tok_bytes);
    set(3, parents, (size_t)L.batch * T_tree * 4);
    set(4, k, kv_bytes);
    set(5, v, kv_bytes);
    set(6, first_visible, first_visible ? (size_t)L.batch * T * 4 : 0);
    return cr;
}

// Do this call's outputs overlap anything the previous fused call reads or writes?
bool outputs_touch_previous(const sparrow_ctx* c, const CallRanges& cr)
{
    if (!c->prev_valid) return false;
    for (int o = 0; o < 2; ++o)
        for (int i = 0; i < kCallRanges; ++i)
            if (cr.r[o][0] < c->prev_ranges[i][1] && c->prev_ranges[i][0] < cr.r[o][1]) return true;
    return false;
}

// Does this call read (q, parents, k, v) anything that a fused call which may still be running
// writes?  Such a call must not start early: it is launched in plain stream order.
bool inputs_touch_recent_outputs(const sparrow_ctx* c, const CallRanges& cr)
{
    uintptr_t lo = cr.r[2][0], hi = cr.r[2][1];
    for (int i = 3; i < kCallRanges; ++i) {
        if (cr.r[i][0] == cr.r[i][1]) continue;            // absent
        if (cr.r[i][0] < lo) lo = cr.r[i][0];
        if (cr.r[i][1] > hi) hi = cr.r[i][1];
    }
    for (int n = 0; n < c->n_recent; ++n) {
        const RecentCall& rc = c->recent[n];
        const uintptr_t w_lo = rc.out[0] < rc.lse[0] ? rc.out[0] : rc.lse[0];
        const uintptr_t w_hi = rc.out[1] > rc.lse[1] ? rc.out[1] : rc.lse[1];
        if (hi <= w_lo || w_hi <= lo) continue;            // nothing of this call near what that one writes
        for (int i = 2; i < kCallRanges; ++i)
            if ((cr.r[i][0] < rc.out[1] && rc.out[0] < cr.r[i][1]) || (cr.r[i][0] < rc.lse[1] && rc.lse[0] < cr.r[i][1]))
                return true;
    }
    return false;
}

// Book-keeping after a fused launch.  A launch in plain stream order follows everything enqueued
// before it, so the calls before it cannot be running beside any later call; otherwise the list
// keeps the last kRecentCalls calls, which is more than can be resident at once.
void note_fused_launch(sparrow_ctx* c, const CallRanges& cr, bool launched_early)
{
    if (!launched_early) c->n_recent = c->recent_head = 0;
    RecentCall& rc = c->recent[c->recent_head];
    rc.out[0] = cr.r[0][0]; rc.out[1] = cr.r[0][1];
    rc.lse[0] = cr.r[1][0]; rc.lse[1] = cr.r[1][1];
    c->recent_head = (c->recent_head + 1) % kRecentCalls;
    if (c->n_recent < kRecentCalls) ++c->n_recent;
}

// `after_previous`: the call's final results must wait for the previous fused call as a whole (its
// outputs overlap that call's memory); otherwise they only wait for the calls before that one.
SyncArgs next_sync(const sparrow_ctx* c, const SplitPlan& p, bool overlaps, bool after_previous)
{
    SyncArgs sy;
    const int parity = (int)(c->seq & 1u);
    sy.arrivals = reinterpret_cast<unsigned*>(c->ws + kArrivalsOffset);
    sy.fin_done = reinterpret_cast<unsigned*>(c->ws + kFinDoneOffset);
    sy.enabled = overlaps ? 1 : 0;
    sy.parity = parity;
    sy.slot = (int)(c->seq & 3u);
    int n_arrive = 0;
    for (int b = 0; b < p.batch; ++b)
        if (p.seq[b].n_splits > 1) n_arrive += p.n_kv_heads * p.n_groups * p.seq[b].n_splits;
    sy.n_arrive = n_arrive;
    // Finishers wait, holding their SM, until the call's last piece is in: few of them where later
    // calls should move in beside this one, all CTAs under the one-wave latency policy.
    const bool all_finish = overlaps && c->plan_policy == SPARROW_PLAN_LATENCY;
    sy.n_fin = n_arrive == 0 ? 0 : ((all_finish || p.n_items < kFinisherCtas) ? p.n_items : kFinisherCtas);
    sy.fin_wait_same = c->fin_total[parity];
    sy.fin_wait_other = after_previous ? c->fin_total[parity ^ 1] : c->fin_before_last[parity ^ 1];
    sy.call = c->seq;
    return sy;
}

void advance_sync(sparrow_ctx* c, const SplitPlan& p, const SyncArgs& sy)
{
    if (!sy.enabled) return;         // stream-ordered calls leave the fused sequence where it is
    c->fin_before_last[sy.parity] = c->fin_total[sy.parity];
    c->fin_total[sy.parity] += (uint32_t)(p.n_items - sy.n_arrive + sy.n_fin);    // single-piece items + finishers
    c->seq += 1;
}

// Context of the most recent fused launch in this process (any stream): see launch_verify_tc().
std::atomic<sparrow_ctx*> g_last_fused_ctx{nullptr};
// Any other kernel this library enqueues breaks the "directly before" knowledge: the next
// verification call takes a plain launch behind it.
inline void other_kernel_enqueued() { g_last_fused_ctx.store(nullptr); }

sparrow_status launch_combine(sparrow_ctx* c, const SplitPlan& plan, const SyncArgs& sy, void* out, float* lse, cudaStream_t st,
                              bool programmatic = false)
{
    CombineArgs ca;
    ca.o_part = o_part_ptr(c, sy.parity);
    ca.out = static_cast<__nv_bfloat16*>(out);
    ca.lse = lse;
    ca.n_q_heads = c->layout.n_q_heads;
    const int rows = plan.batch * plan.n_kv_heads * plan.M;
    int ctas = (rows + combine::kWarps - 1) / combine::kWarps;
    if (ctas > 8 * c->n_sm) ctas = 8 * c->n_sm;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(combine::kWarps * 32);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;       // its CTAs become resident while the split-KV pass runs and wait for it
    if (cudaLaunchKernelEx(&cfg, combine::combine_kernel, plan, ca) != cudaSuccess) { cudaGetLastError(); return SPARROW_ERR_CUDA; }
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status launch_split_gather(sparrow_ctx* c, const SplitPlan& plan, const SyncArgs& sy, const void* q, const void* k, const void* v,
                                   const int32_t* parents, const int32_t* anchor_idx, int n_anchor, int window,
                                   void* out, float* lse, cudaStream_t st, bool early_dependents = false, int tree_nodes = 0)
{
    SplitArgs a;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.k = static_cast<const __nv_bfloat16*>(k);
    a.v = static_cast<const __nv_bfloat16*>(v);
    a.parents = parents;
    a.anchor_idx = anchor_idx;
    a.n_anchor = n_anchor;
    a.window = window;
    a.tree_nodes = tree_nodes;
    a.n_q_heads = c->layout.n_q_heads;
    a.kv_capacity = c->layout.kv_capacity;
    a.kv_stride_batch = c->layout.kv_stride_batch;
    a.kv_stride_head = c->layout.kv_stride_head;
    a.scale_log2e = c->layout.softmax_scale * 1.4426950408889634f;
    a.o_part = o_part_ptr(c, sy.parity);
    a.out = static_cast<__nv_bfloat16*>(out);
    a.lse = lse;
    a.status = reinterpret_cast<unsigned*>(c->ws);
    a.early_dependents = early_dependents ? 1 : 0;
    other_kernel_enqueued();
    gather::split_gather_kernel<<<plan.n_items, gather::kThreads, gather::kSmemBytes, st>>>(plan, a);
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

// Cached tensor maps.  tag == 0: one K or V buffer, dims (128 dims, capacity rows, KV heads,
// batch), boxes of 64 dims x 128 rows; rows past the capacity read as zero.  tag == n_tok > 0: the
// query tensor [n_tok][KV heads][7][128], boxes of 64 dims x 7 heads x 18 tokens, which land in
// shared memory as the rows (t * 7 + g) of a K-major operand block; tokens past n_tok read as zero.
// Both use the 128-byte swizzle.
bool tensor_map_for(sparrow_ctx* c, const void* base, int tag, CUtensorMap* out)
{
    // The map is copied out: a later lookup of the same call may evict the slot it came from.
    size_t h = reinterpret_cast<uintptr_t>(base) >> 8;
    h = (h ^ (h >> 11) ^ ((size_t)tag * 0x9E3779B1u)) * 0x9E3779B97F4A7C15ull;
    const int bucket = (int)((h >> 40) % (kMapCacheSize / kMapWays)) * kMapWays;
    int free_slot = -1;
    for (int w = 0; w < kMapWays; ++w) {
        TensorMapEntry& e = c->maps[bucket + w];
        if (e.base == base && e.tag == tag) { *out = e.map; return true; }
        if (!e.base && free_slot < 0) free_slot = bucket + w;
    }
    if (!c->encode) return false;
    const sparrow_layout& L = c->layout;
    const int slot = free_slot >= 0 ? free_slot : bucket + (int)(c->evict_tick++ % kMapWays);
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r;
    if (tag == 0) {
        const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)L.kv_capacity, (cuuint64_t)L.n_kv_heads, (cuuint64_t)L.batch};
        const cuuint64_t batch_stride = L.batch > 1 ? (cuuint64_t)L.kv_stride_batch : (cuuint64_t)L.kv_stride_head * L.n_kv_heads;
        const cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)L.kv_stride_head * 2, batch_stride * 2};
        const cuuint32_t box[4] = {64, 128, 1, 1};
        r = c->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const int group = L.n_q_heads / L.n_kv_heads;
        const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)group, (cuuint64_t)L.n_kv_heads, (cuuint64_t)tag};
        const cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)group * kD * 2, (cuuint64_t)L.n_q_heads * kD * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)group, 1, (cuuint32_t)tokens_per_block(group)};
        r = c->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return false;
    c->maps[slot].base = base;
    c->maps[slot].tag = tag;
    c->maps[slot].map = *out;
    return true;
}

void clear_tensor_maps(sparrow_ctx* c)
{
    for (int i = 0; i < kMapCacheSize; ++i) c->maps[i].base = nullptr;
    c->evict_tick = 0;
}

sparrow_status launch_verify_tc(sparrow_ctx* c, const SplitPlan& plan, const SyncArgs& sy, const void* q, const void* k, const void* v,
                                const int32_t* parents, const int32_t* first_visible, void* out, float* lse, cudaStream_t st,
                                bool start_early)
{
    CUtensorMap mq, mk, mv;
    if (!tensor_map_for(c, q, plan.batch * plan.T, &mq) || !tensor_map_for(c, k, 0, &mk) || !tensor_map_for(c, v, 0, &mv))
        return SPARROW_ERR_CUDA;
    const int nb = plan.blocks_per_group;
    TcArgs a;
    a.parents = parents;
    a.first_visible = first_visible;
    a.n_q_heads = c->layout.n_q_heads;
    a.scale_log2e = c->layout.softmax_scale * 1.4426950408889634f;
    a.o_part = o_part_ptr(c, sy.parity);
    a.out = static_cast<__nv_bfloat16*>(out);
    a.lse = lse;
    a.status = reinterpret_cast<unsigned*>(c->ws);
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(plan.n_items);
    cfg.blockDim = dim3(tc::kThreads);
    cfg.dynamicSmemBytes = tc::smem_bytes(nb, nb == 1 ? 3 : 2);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    // A call may start early behind the kernel launched directly before it in the stream only
    // where the caller of this function has made sure that that kernel is this context's previous
    // call; every other launch takes plain stream order.
    cfg.numAttrs = start_early ? 1 : 0;
    const cudaError_t e = nb == 1 ? cudaLaunchKernelEx(&cfg, tc::verify_tc_kernel<1>, a, sy, plan, mq, mk, mv)
                                  : cudaLaunchKernelEx(&cfg, tc::verify_tc_kernel<2>, a, sy, plan, mq, mk, mv);
    if (e != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

__global__ void ancestor_masks_kernel(const int32_t* parents, int T, unsigned long long* masks, unsigned* status)
{
    const int i = threadIdx.x;
    if (i < T) masks[i] = ancestor_word(parents, T, i, status);
}

// One thread waits (bounded) on a finisher counter; see sparrow_debug_wait_counter().
__global__ void wait_counter_kernel(const unsigned* counter, unsigned target, unsigned* status)
{
    if (!wait_counter(counter, target)) atomicOr(status, timeout_bits(kSiteDebug));
}

// A stand-in for a foreign kernel that lets its dependents launch early and only then produces
// its output (as many library GEMM / norm kernels do): see sparrow_debug_early_trigger_copy().
__global__ void early_trigger_copy_kernel(const uint4* src, uint4* dst, size_t n_vec, unsigned delay_us)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (delay_us > 10000u) delay_us = 10000u;
    for (unsigned i = 0; i < delay_us; ++i) __nanosleep(1000);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (size_t)gridDim.x * blockDim.x) dst[i] = src[i];
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        want = dev;
    }
    ~DeviceGuard() { if (ok && prev != want) cudaSetDevice(prev); }
    int want = -1;
};

sparrow_status check_tree_host(const int32_t* parents, int T)
{
    for (int i = 0; i < T; ++i)
        if (parents[i] < -1 || parents[i] >= i) return SPARROW_ERR_TREE;
    return SPARROW_OK;
}

// One verification call: T query tokens, the last T of the T_tree nodes whose K/V rows sit at
// [kv_len, kv_len + T_tree); optional per-token lower window bound over the prefix keys.
sparrow_status verify_call(sparrow_ctx* c, const void* q, const void* k, const void* v, const int32_t* kv_len,
                           const int32_t* parents, int32_t T_tree, int32_t T, const int32_t* first_visible,
                           const int32_t* first_visible_min, void* out, float* lse, void* stream)
{
    if (!c || !q || !k || !v || !kv_len || !parents || !out || !lse) return SPARROW_ERR_NULL;
    if (T < 1 || T > T_tree || T_tree > kMaxT) return SPARROW_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return SPARROW_ERR_SHAPE;
    int32_t n_keys[kMaxBatch], key0[kMaxBatch];
    for (int b = 0; b < c->layout.batch; ++b) {
        if (kv_len[b] < 0 || (int64_t)kv_len[b] + T_tree > c->layout.kv_capacity) return SPARROW_ERR_SHAPE;
        n_keys[b] = kv_len[b] + T_tree;
        key0[b] = 0;
        if (first_visible_min) {                 // nothing left of every row's bound is streamed
            if (first_visible_min[b] < 0 || first_visible_min[b] > kv_len[b]) return SPARROW_ERR_SHAPE;
            key0[b] = first_visible_min[b] / kKeyTile * kKeyTile;
        }
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Outside stream capture (and with programmatic launch on) a call takes part in the counter
    // protocol and merges its own pieces.  Whether it also STARTS EARLY, overlapping the previous
    // call, is a separate decision: only where the kernel directly before it in the stream is known
    // to be this context's previous call (the counters order this context's own calls and know
    // nothing about another context's writes; nothing else can sit in between for the calls after
    // the first of sparrow_verify_attn_batch(), or once the caller has vouched for the stream with
    // sparrow_set_call_overlap()), and where it reads nothing that a call which may still be
    // running writes.  Every other launch takes plain stream order.  A captured call is two plain
    // launches: the split-KV pass and the combine kernel.
    const CallRanges cr = call_ranges(c, q, k, v, parents, T_tree, T, first_visible, out, lse);
    const bool protocol = call_overlaps(c, st, true);                // not capturing, programmatic launch on
    const bool same_ctx_before = g_last_fused_ctx.exchange(c) == c;
    const bool early = protocol && same_ctx_before && (c->chain_next || c->overlap_single_calls) &&
                       !inputs_touch_recent_outputs(c, cr);
    SplitPlan plan;
    const int group = layout_group(c->layout);
    sparrow_status s = make_plan(plan_target(c, protocol), c->layout.batch, c->layout.n_kv_heads, group, n_keys, T,
                                 blocks_per_group_tc(T, group), &plan, kMinPieceKeys, key0);
    if (s != SPARROW_OK) return s;
    plan.T_tree = T_tree;
    for (int b = 0; b < c->layout.batch; ++b) plan.seq[b].kv_len = kv_len[b];
    if ((s = check_ws(c, plan)) != SPARROW_OK) return s;
    const SyncArgs sy = next_sync(c, plan, protocol, outputs_touch_previous(c, cr));
    if (c->log_plans) {
        std::fprintf(stderr, "[sparrow] verify call %u: T %d of %d nodes, %d row block(s) x %d group(s), %d items (target %d), %s, %s;",
                     c->seq, T, T_tree, plan.blocks_per_group, plan.n_groups, plan.n_items, plan_target(c, protocol),
                     protocol ? "counter protocol" : "stream-ordered", early ? "starts early" : "plain launch");
        for (int b = 0; b < plan.batch; ++b)
            std::fprintf(stderr, " seq %d: keys [%d, %d) in %d piece(s)", b, plan.seq[b].key0, plan.seq[b].n_keys, plan.seq[b].n_splits);
        std::fprintf(stderr, "; %d finisher(s)\n", sy.n_fin);
    }
    if ((s = launch_verify_tc(c, plan, sy, q, k, v, parents, first_visible, out, lse, st, early)) != SPARROW_OK) return s;
    if (protocol) {
        advance_sync(c, plan, sy);
        std::memcpy(c->prev_ranges, cr.r, sizeof(cr.r));
        c->prev_valid = true;
        note_fused_launch(c, cr, early);
        return SPARROW_OK;                                   // the kernel merges its own partials
    }
    bool needs_combine = false;
    for (int b = 0; b < plan.batch; ++b) needs_combine = needs_combine || plan.seq[b].n_splits > 1;
    return needs_combine ? launch_combine(c, plan, sy, out, lse, st) : SPARROW_OK;
}

}  // namespace

extern "C" {

const char* sparrow_status_string(sparrow_status s)
{
    switch (s) {
        case SPARROW_OK: return "ok";
        case SPARROW_ERR_NULL: return "null pointer";
        case SPARROW_ERR_SHAPE: return "unsupported shape or size";
        case SPARROW_ERR_TREE: return "parents[] is not a topologically ordered forest";
        case SPARROW_ERR_ANCHOR: return "bad anchor list";
        case SPARROW_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SPARROW_ERR_CUDA: return "CUDA call failed";
        case SPARROW_ERR_TIMEOUT: return "device-side wait timed out";
        case SPARROW_ERR_ARCH: return "device is not sm_100";
    }
    return "unknown status";
}

sparrow_status sparrow_create(sparrow_ctx** out, const sparrow_layout* L, int device)
{
    if (!out || !L) return SPARROW_ERR_NULL;
    *out = nullptr;
    if (L->batch < 1 || L->batch > kMaxBatch || L->head_dim != kD || L->n_kv_heads < 1 ||
        !layout_heads_ok(*L) || L->kv_capacity < 1 ||
        !(L->softmax_scale > 0.f) || !std::isfinite(L->softmax_scale) ||
        L->kv_stride_head < (int64_t)L->kv_capacity * kD || (L->kv_stride_head % 8) != 0 ||
        (L->kv_stride_batch % 8) != 0 ||
        (L->batch > 1 && L->kv_stride_batch < L->kv_stride_head * (int64_t)L->n_kv_heads))
        return SPARROW_ERR_SHAPE;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) { cudaGetLastError(); return SPARROW_ERR_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (prop.major != 10) return SPARROW_ERR_ARCH;
    DeviceGuard guard(device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    if (cudaFuncSetAttribute(gather::split_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             gather::kSmemBytes) != cudaSuccess)
        return SPARROW_ERR_CUDA;
    if (cudaFuncSetAttribute(tc::verify_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             tc::smem_bytes(1, 3)) != cudaSuccess ||
        cudaFuncSetAttribute(tc::verify_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             tc::smem_bytes(2, 2)) != cudaSuccess)
        return SPARROW_ERR_CUDA;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn)
        return SPARROW_ERR_CUDA;
    sparrow_ctx* c = new (std::nothrow) sparrow_ctx();
    if (!c) return SPARROW_ERR_CUDA;
    clear_tensor_maps(c);
    c->encode = reinterpret_cast<TensorMapEncodeFn>(fn);
    c->layout = *L;
    c->device = device;
    c->n_sm = prop.multiProcessorCount;
    c->plan_policy = SPARROW_PLAN_BALANCED;
    c->ws = nullptr;
    c->ws_bytes = 0;
    c->part_offset = fixed_bytes(*L);
    c->part_buffers = 2;
    c->launches.store(0);
    const char* e = std::getenv("SPARROW_NO_PDL");
    // more SMs than the list of possibly-resident calls can hold: calls never start early
    c->use_pdl = !(e && e[0] == '1') && c->n_sm < kRecentCalls;
    c->overlap_single_calls = false;
    const char* lg = std::getenv("SPARROW_LOG");
    c->log_plans = lg && lg[0] == '1';
    c->chain_next = false;
    c->n_recent = c->recent_head = 0;
    c->seq = 0;
    c->fin_total[0] = c->fin_total[1] = 0;
    c->fin_before_last[0] = c->fin_before_last[1] = 0;
    c->prev_valid = false;
    c->last_status_word = 0;
    *out = c;
    return SPARROW_OK;
}

sparrow_status sparrow_destroy(sparrow_ctx* c)
{
    if (!c) return SPARROW_ERR_NULL;
    sparrow_ctx* expected = c;
    g_last_fused_ctx.compare_exchange_strong(expected, nullptr);      // a later context may reuse the address
    delete c;
    return SPARROW_OK;
}

size_t sparrow_workspace_bytes(const sparrow_ctx* c, int32_t max_T)
{
    if (!c || max_T < 1 || max_T > kMaxT) return 0;
    size_t worst = 0;
    const int tpb = tokens_per_block(layout_group(c->layout));
    for (int nb : {1, blocks_per_group_tc(max_T, layout_group(c->layout))}) {         // the gathered pass uses single blocks
        const int groups = (max_T + tpb * nb - 1) / (tpb * nb);
        const size_t rows = (size_t)max_items(c->n_sm, c->layout.batch, c->layout.n_kv_heads, groups) * (nb * kBlockRows + 1);
        const size_t need = part_bytes(rows);
        if (need > worst) worst = need;
    }
    return fixed_bytes(c->layout) + 2 * worst + 512;
}

sparrow_status sparrow_set_workspace(sparrow_ctx* c, void* p, size_t bytes)
{
    if (!c || !p) return SPARROW_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(p) & 255u) != 0 || bytes < fixed_bytes(c->layout)) return SPARROW_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    // Kernels of earlier calls may still be using the old workspace and its counters.
    if (cudaDeviceSynchronize() != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaMemset(p, 0, kStatusBytes) != cudaSuccess) return SPARROW_ERR_CUDA;
    c->ws = static_cast<unsigned char*>(p);
    c->ws_bytes = bytes;
    c->seq = 0;
    c->fin_total[0] = c->fin_total[1] = 0;
    c->fin_before_last[0] = c->fin_before_last[1] = 0;
    c->prev_valid = false;
    c->n_recent = c->recent_head = 0;
    return SPARROW_OK;
}

sparrow_status sparrow_plan_splits(int32_t n_sm, int32_t batch, int32_t n_kv_heads, int32_t gqa_group, const int32_t* n_keys,
                                   int32_t T, int32_t* splits_out, int32_t* n_items_out)
{
    if (!n_keys || !splits_out || !n_items_out) return SPARROW_ERR_NULL;
    SplitPlan p;
    if (T < 1 || T > kMaxT || gqa_group < 1 || gqa_group > kMaxGroup) return SPARROW_ERR_SHAPE;
    const sparrow_status s = make_plan(n_sm, batch, n_kv_heads, gqa_group, n_keys, T, blocks_per_group_tc(T, gqa_group), &p);
    if (s != SPARROW_OK) return s;
    for (int b = 0; b < batch; ++b) splits_out[b] = p.seq[b].n_splits;
    *n_items_out = p.n_items;
    return SPARROW_OK;
}

sparrow_status sparrow_plan_piece_range(int32_t n_keys, int32_t n_splits, int32_t piece, int32_t* begin_out, int32_t* end_out)
{
    if (!begin_out || !end_out) return SPARROW_ERR_NULL;
    if (n_keys < 1 || n_splits < 1 || piece < 0 || piece >= n_splits || n_splits > (n_keys + kKeyTile - 1) / kKeyTile)
        return SPARROW_ERR_SHAPE;
    int b, e;
    piece_range(n_keys, n_splits, piece, kKeyTile, &b, &e);
    *begin_out = b;
    *end_out = e;
    return SPARROW_OK;
}

sparrow_status sparrow_verify_attn(sparrow_ctx* c, const void* q, const void* k, const void* v,
                                   const int32_t* kv_len, const int32_t* parents, int32_t T, void* out,
                                   float* lse, void* stream)
{
    return verify_call(c, q, k, v, kv_len, parents, T, T, nullptr, nullptr, out, lse, stream);
}

sparrow_status sparrow_verify_attn_window(sparrow_ctx* c, const void* q, const void* k, const void* v,
                                          const int32_t* kv_len, const int32_t* parents, int32_t T_tree, int32_t T_new,
                                          const int32_t* first_visible, const int32_t* first_visible_min, void* out,
                                          float* lse, void* stream)
{
    if (T_tree < 1 || T_tree > kMaxT || T_new < 1 || T_new > T_tree) return SPARROW_ERR_SHAPE;
    return verify_call(c, q, k, v, kv_len, parents, T_tree, T_new, first_visible, first_visible_min, out, lse, stream);
}

}  // extern "C"  (closed for the file-scope objects of the no-allocation entry point)

// Scratch of sparrow_verify_attn_static(): part of the device image, one copy per GPU that loads
// the library.  In host code this name is only a handle for cudaGetSymbolAddress().
static __device__ __align__(256) unsigned char g_static_scratch[SPARROW_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxStaticDevices = 16;
struct StaticSlot {
    bool ready;
    sparrow_ctx ctx;
};
StaticSlot g_static_slots[kMaxStaticDevices];      // static storage: no heap behind the entry point

bool same_layout(const sparrow_layout& a, const sparrow_layout& b)
{
    return a.batch == b.batch && a.n_q_heads == b.n_q_heads && a.n_kv_heads == b.n_kv_heads && a.head_dim == b.head_dim &&
           a.kv_capacity == b.kv_capacity && a.softmax_scale == b.softmax_scale &&
           a.kv_stride_batch == b.kv_stride_batch && a.kv_stride_head == b.kv_stride_head;
}
}  // namespace

extern "C" {

sparrow_status sparrow_verify_attn_static(const sparrow_layout* L, const void* q, const void* k, const void* v,
                                          const int32_t* kv_len, const int32_t* parents, int32_t T, void* out,
                                          float* lse, void* stream)
{
    // every argument check comes first: a refused call has not touched the GPU
    if (!L || !q || !k || !v || !kv_len || !parents || !out || !lse) return SPARROW_ERR_NULL;
    if (L->batch < 1 || L->batch > kMaxBatch || L->head_dim != kD || L->n_kv_heads < 1 ||
        !layout_heads_ok(*L) || L->kv_capacity < 1 ||
        !(L->softmax_scale > 0.f) || !std::isfinite(L->softmax_scale) ||
        L->kv_stride_head < (int64_t)L->kv_capacity * kD || (L->kv_stride_head % 8) != 0 ||
        (L->kv_stride_batch % 8) != 0 ||
        (L->batch > 1 && L->kv_stride_batch < L->kv_stride_head * (int64_t)L->n_kv_heads))
        return SPARROW_ERR_SHAPE;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return SPARROW_ERR_SHAPE;
    int32_t n_keys[kMaxBatch];
    for (int b = 0; b < L->batch; ++b) {
        if (kv_len[b] < 0 || (int64_t)kv_len[b] + T > L->kv_capacity) return SPARROW_ERR_SHAPE;
        n_keys[b] = kv_len[b] + T;
    }
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return SPARROW_ERR_CUDA; }
    if (device < 0 || device >= kMaxStaticDevices) return SPARROW_ERR_SHAPE;
    StaticSlot& slot = g_static_slots[device];
    sparrow_ctx* c = &slot.ctx;
    if (!slot.ready) {
        // one-time set-up for this device (it is the current one)
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SPARROW_ERR_CUDA;
        if (prop.major != 10) return SPARROW_ERR_ARCH;
        if (cudaFuncSetAttribute(gather::split_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 gather::kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(tc::verify_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 tc::smem_bytes(1, 3)) != cudaSuccess ||
            cudaFuncSetAttribute(tc::verify_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 tc::smem_bytes(2, 2)) != cudaSuccess)
            return SPARROW_ERR_CUDA;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn)
            return SPARROW_ERR_CUDA;
        void* scratch = nullptr;               // the array's device address on THIS device
        if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) return SPARROW_ERR_CUDA;
        if (cudaMemset(scratch, 0, kStatusBytes) != cudaSuccess) return SPARROW_ERR_CUDA;
        clear_tensor_maps(c);
        c->encode = reinterpret_cast<TensorMapEncodeFn>(fn);
        c->layout = *L;
        c->device = device;
        c->n_sm = prop.multiProcessorCount;
        c->plan_policy = SPARROW_PLAN_LATENCY;
        c->ws = static_cast<unsigned char*>(scratch);
        c->ws_bytes = SPARROW_STATIC_SCRATCH_BYTES;
        // Stream-ordered calls only: no counters live in the shared array, nothing is double-buffered,
        // and there is no staging area -- the partials take everything behind the 1 KiB header.
        c->part_offset = kStatusBytes;
        c->part_buffers = 1;
        c->launches.store(0);
        c->use_pdl = false;
        c->overlap_single_calls = false;
        c->chain_next = false;
        c->n_recent = c->recent_head = 0;
        c->seq = 0;
        c->fin_total[0] = c->fin_total[1] = 0;
        c->fin_before_last[0] = c->fin_before_last[1] = 0;
        c->prev_valid = false;
        c->last_status_word = 0;
        slot.ready = true;
    }
    if (!same_layout(c->layout, *L)) {         // tensor maps depend on the layout
        c->layout = *L;
        clear_tensor_maps(c);
    }
    // refuse what does not fit the array before anything is enqueued
    SplitPlan plan;
    if (make_plan(c->n_sm, L->batch, L->n_kv_heads, layout_group(*L), n_keys, T, blocks_per_group_tc(T, layout_group(*L)), &plan) != SPARROW_OK)
        return SPARROW_ERR_SHAPE;
    if (check_ws(c, plan) != SPARROW_OK) return SPARROW_ERR_WORKSPACE;
    // the status word is the one thing that must start clean
    // the status word is the one thing that must start clean
    if (cudaMemsetAsync(c->ws, 0, sizeof(unsigned), static_cast<cudaStream_t>(stream)) != cudaSuccess) return SPARROW_ERR_CUDA;
    return sparrow_verify_attn(c, q, k, v, kv_len, parents, T, out, lse, stream);
}

sparrow_status sparrow_verify_attn_batch(sparrow_ctx* c, const sparrow_verify_call* calls, int32_t n_calls, void* stream)
{
    if (!c || !calls) return SPARROW_ERR_NULL;
    if (n_calls < 0) return SPARROW_ERR_SHAPE;
    for (int i = 0; i < n_calls; ++i) {
        const sparrow_verify_call& k = calls[i];
        // from the second call on, the kernel directly before this one in the stream is the previous call's
        c->chain_next = i > 0;
        const sparrow_status s = sparrow_verify_attn(c, k.q, k.k_cache, k.v_cache, k.kv_len, k.parents, k.T, k.out, k.lse, stream);
        c->chain_next = false;
        if (s != SPARROW_OK) return s;
    }
    return SPARROW_OK;
}

}  // extern "C"

namespace {
// Both anchored entry points: parents == nullptr / tree_nodes == 0 is the chain rule.
sparrow_status anchor_call(sparrow_ctx* c, const void* q, const void* k, const void* v, const int32_t* anchor_idx,
                           int32_t n_anchor, int32_t window, const int32_t* parents, int32_t tree_nodes, int32_t T,
                           void* out, float* lse, void* stream)
{
    if (!c || !q || !k || !v || !anchor_idx || !out || !lse) return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (n_anchor < T || n_anchor > c->layout.kv_capacity) return SPARROW_ERR_ANCHOR;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return SPARROW_ERR_SHAPE;
    int32_t n_keys[kMaxBatch];
    for (int b = 0; b < c->layout.batch; ++b) n_keys[b] = n_anchor;
    SplitPlan plan;
    sparrow_status s = make_plan(c->n_sm, c->layout.batch, c->layout.n_kv_heads, layout_group(c->layout), n_keys, T, 1, &plan, kMinGatherPieceKeys);
    if (s != SPARROW_OK) return s;
    if ((s = check_ws(c, plan)) != SPARROW_OK) return s;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const SyncArgs sy = next_sync(c, plan, false, true);
    // the two kernels of the call are chained programmatically unless the stream is being captured
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusActive; }
    const bool chained = c->use_pdl && cap == cudaStreamCaptureStatusNone;
    if ((s = launch_split_gather(c, plan, sy, q, k, v, parents, anchor_idx, n_anchor, window, out, lse, st, chained,
                                 tree_nodes)) != SPARROW_OK)
        return s;
    return launch_combine(c, plan, sy, out, lse, st, chained);
}
}  // namespace

extern "C" {

sparrow_status sparrow_anchor_attn(sparrow_ctx* c, const void* q, const void* k, const void* v,
                                   const int32_t* anchor_idx, int32_t n_anchor, int32_t window, int32_t T,
                                   void* out, float* lse, void* stream)
{
    return anchor_call(c, q, k, v, anchor_idx, n_anchor, window, nullptr, 0, T, out, lse, stream);
}

sparrow_status sparrow_anchor_attn_tree(sparrow_ctx* c, const void* q, const void* k, const void* v,
                                        const int32_t* anchor_idx, int32_t n_anchor, int32_t window,
                                        const int32_t* parents, int32_t T_tree, int32_t T_new, void* out, float* lse,
                                        void* stream)
{
    if (!parents) return SPARROW_ERR_NULL;
    if (T_tree < 1 || T_tree > kMaxT || T_new < 1 || T_new > T_tree) return SPARROW_ERR_SHAPE;
    if (n_anchor < T_tree) return SPARROW_ERR_ANCHOR;
    return anchor_call(c, q, k, v, anchor_idx, n_anchor, window, parents, T_tree, T_new, out, lse, stream);
}

sparrow_status sparrow_kv_append(sparrow_ctx* c, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                 const int32_t* kv_len, int32_t T, void* stream)
{
    if (!c || !k_new || !v_new || !k_cache || !v_cache || !kv_len) return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache)) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    const sparrow_layout& L = c->layout;
    RowMoveArgs a;
    std::memset(&a, 0, sizeof a);
    for (int b = 0; b < L.batch; ++b) {
        if (kv_len[b] < 0 || (int64_t)kv_len[b] + T > L.kv_capacity) return SPARROW_ERR_SHAPE;
        a.dst_row0[b] = kv_len[b];
    }
    a.k_src = static_cast<const __nv_bfloat16*>(k_new);
    a.v_src = static_cast<const __nv_bfloat16*>(v_new);
    a.k_dst = static_cast<__nv_bfloat16*>(k_cache);
    a.v_dst = static_cast<__nv_bfloat16*>(v_cache);
    a.src_rows = nullptr;
    a.n_rows = T;
    a.batch = L.batch;
    a.n_kv_heads = L.n_kv_heads;
    a.src_capacity = T;
    a.src_stride_head = (int64_t)T * kD;
    a.src_stride_batch = a.src_stride_head * L.n_kv_heads;
    a.dst_stride_batch = L.kv_stride_batch;
    a.dst_stride_head = L.kv_stride_head;
    a.status = reinterpret_cast<unsigned*>(c->ws);
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    const long long threads = (long long)L.batch * L.n_kv_heads * T * 16;
    other_kernel_enqueued();
    move_rows_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_compact_anchors(sparrow_ctx* c, const void* k, const void* v, const int32_t* anchor_idx,
                                       int32_t n_anchor, void* k_compact, void* v_compact, int32_t compact_capacity,
                                       int32_t dst_row, void* stream)
{
    if (!c || !k || !v || !anchor_idx || !k_compact || !v_compact) return SPARROW_ERR_NULL;
    if (!aligned16(k) || !aligned16(v) || !aligned16(k_compact) || !aligned16(v_compact)) return SPARROW_ERR_SHAPE;
    if (n_anchor < 1 || n_anchor > c->layout.kv_capacity) return SPARROW_ERR_ANCHOR;
    if (compact_capacity < 1 || dst_row < 0 || (int64_t)dst_row + n_anchor > compact_capacity) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    const sparrow_layout& L = c->layout;
    RowMoveArgs a;
    std::memset(&a, 0, sizeof a);
    for (int b = 0; b < L.batch; ++b) a.dst_row0[b] = dst_row;
    a.k_src = static_cast<const __nv_bfloat16*>(k);
    a.v_src = static_cast<const __nv_bfloat16*>(v);
    a.k_dst = static_cast<__nv_bfloat16*>(k_compact);
    a.v_dst = static_cast<__nv_bfloat16*>(v_compact);
    a.src_rows = anchor_idx;
    a.n_rows = n_anchor;
    a.batch = L.batch;
    a.n_kv_heads = L.n_kv_heads;
    a.src_capacity = L.kv_capacity;
    a.src_stride_batch = L.kv_stride_batch;
    a.src_stride_head = L.kv_stride_head;
    a.dst_stride_head = (int64_t)compact_capacity * kD;
    a.dst_stride_batch = a.dst_stride_head * L.n_kv_heads;
    a.status = reinterpret_cast<unsigned*>(c->ws);
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    const long long threads = (long long)L.batch * L.n_kv_heads * n_anchor * 16;
    long long blocks = (threads + 255) / 256;
    if (blocks > 8LL * c->n_sm) blocks = 8LL * c->n_sm;
    other_kernel_enqueued();
    move_rows_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_window_first_visible(const int32_t* anchor_idx, int32_t n_anchor, int32_t window, int32_t T_tree,
                                            int32_t T_new, int32_t* first_visible, int32_t* first_visible_min)
{
    if (!anchor_idx || !first_visible) return SPARROW_ERR_NULL;
    if (T_tree < 1 || T_tree > kMaxT || T_new < 1 || T_new > T_tree) return SPARROW_ERR_SHAPE;
    if (n_anchor < T_tree) return SPARROW_ERR_ANCHOR;
    for (int j = 1; j < n_anchor; ++j)
        if (anchor_idx[j] <= anchor_idx[j - 1]) return SPARROW_ERR_ANCHOR;
    const int n_text = n_anchor - T_tree;
    int32_t lowest = n_text;
    for (int t = 0; t < T_new; ++t) {
        int32_t f = 0;
        if (window > 0) f = first_anchor_above(anchor_idx, n_text, (long long)anchor_idx[n_anchor - T_new + t] - window);
        first_visible[t] = f;
        if (f < lowest) lowest = f;
    }
    if (first_visible_min) *first_visible_min = lowest;
    return SPARROW_OK;
}

sparrow_status sparrow_window_first_visible_device(sparrow_ctx* c, const int32_t* anchor_idx, int32_t n_anchor, int32_t window,
                                                   int32_t T_tree, int32_t T_new, int32_t* first_visible, void* stream)
{
    if (!c || !anchor_idx || !first_visible) return SPARROW_ERR_NULL;
    if (T_tree < 1 || T_tree > kMaxT || T_new < 1 || T_new > T_tree) return SPARROW_ERR_SHAPE;
    if (n_anchor < T_tree) return SPARROW_ERR_ANCHOR;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    const int n = c->layout.batch * T_new;
    other_kernel_enqueued();
    window_bounds_kernel<<<(n + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(anchor_idx, n_anchor, window, T_tree, T_new,
                                                                                         c->layout.batch, first_visible);
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

// K-range slices per feature tile: about one work item per SM, never more slices than K tiles.
static int hsr_slices(int n_sm, int d, int d_out)
{
    // slices of one feature tile = CTAs of one cluster: a power of two up to the portable limit of
    // 8, at most one wave over the SMs (clusters of 5 x 28 tiles did not all fit at once: slower)
    const int f_tiles = d_out / hsr::kFeat, k_tiles = 2 * d / hsr::kKTile;
    int s = 1;
    while (s < 8 && 2 * s * f_tiles <= n_sm && 2 * s <= k_tiles) s *= 2;
    return s;
}

sparrow_status sparrow_hsr_fuse(sparrow_ctx* c, const void* e, const void* h, const void* w, const void* bias, int32_t M,
                                int32_t d, int32_t d_out, void* z, void* stream)
{
    if (!c || !e || !h || !w || !z) return SPARROW_ERR_NULL;
    if (M < 1 || M > hsr::kTok || d < 64 || (d % 64) != 0 || d_out < 128 || (d_out % 128) != 0)
        return SPARROW_ERR_SHAPE;
    if (!aligned16(e) || !aligned16(h) || !aligned16(w) || !aligned16(z)) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;                       // the status word lives there
    const int n_slices = hsr_slices(c->n_sm, d, d_out);
    if (!c->encode) return SPARROW_ERR_CUDA;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    static bool attr_set[kMaxStaticDevices] = {};
    if (c->device >= 0 && c->device < kMaxStaticDevices && !attr_set[c->device]) {
        if (cudaFuncSetAttribute(hsr::hsr_fuse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, hsr::kSmemBytes) != cudaSuccess)
            return SPARROW_ERR_CUDA;
        attr_set[c->device] = true;
    }
    // W: [d_out][2 d], boxes of 64 k x 128 features; e, h: [M][d], boxes of 64 k x 64 tokens (rows past M read as zero)
    CUtensorMap mw, me, mh;
    const cuuint32_t estr[2] = {1, 1};
    auto encode2d = [&](CUtensorMap* m, const void* base, cuuint64_t cols, cuuint64_t rows, cuuint32_t box_rows) {
        const cuuint64_t dims[2] = {cols, rows};
        const cuuint64_t strides[1] = {cols * 2};
        const cuuint32_t box[2] = {(cuuint32_t)hsr::kKTile, box_rows};
        return c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    if (!encode2d(&mw, w, (cuuint64_t)2 * d, (cuuint64_t)d_out, hsr::kFeat) || !encode2d(&me, e, (cuuint64_t)d, (cuuint64_t)M, hsr::kTok) ||
        !encode2d(&mh, h, (cuuint64_t)d, (cuuint64_t)M, hsr::kTok))
        return SPARROW_ERR_CUDA;
    HsrArgs a;
    a.bias = static_cast<const __nv_bfloat16*>(bias);
    a.z = static_cast<__nv_bfloat16*>(z);
    a.status = reinterpret_cast<unsigned*>(c->ws);
    a.M = M; a.d = d; a.d_out = d_out;
    a.n_slices = n_slices;
    a.k_tiles = 2 * d / hsr::kKTile;
    other_kernel_enqueued();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((d_out / hsr::kFeat) * n_slices));
    cfg.blockDim = dim3(hsr::kThreadsHsr);
    cfg.dynamicSmemBytes = hsr::kSmemBytes;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;              // the slices of a feature tile share a cluster
    attr[0].val.clusterDim.x = (unsigned)n_slices;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, hsr::hsr_fuse_kernel, a, mw, me, mh) != cudaSuccess) { cudaGetLastError(); return SPARROW_ERR_CUDA; }
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_accept_greedy(sparrow_ctx* c, const int32_t* draft_tokens, const int32_t* parents,
                                     const int32_t* target_next, int32_t T, int32_t* path_out, int32_t* n_accept_out,
                                     int32_t* bonus_out, void* stream)
{
    if (!c || !draft_tokens || !parents || !target_next || !path_out || !n_accept_out || !bonus_out) return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    other_kernel_enqueued();
    accept_greedy_kernel<<<1, kMaxBatch, 0, static_cast<cudaStream_t>(stream)>>>(
        draft_tokens, parents, target_next, c->layout.batch, T, path_out, n_accept_out, bonus_out,
        reinterpret_cast<unsigned*>(c->ws));
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_accept_sample(sparrow_ctx* c, const int32_t* draft_tokens, const int32_t* parents, const float* p_target,
                                     const float* p_draft, const uint32_t* u_node, const uint32_t* u_bonus, int32_t vocab,
                                     int32_t T, int32_t* path_out, int32_t* n_accept_out, int32_t* bonus_out, void* stream)
{
    if (!c || !draft_tokens || !parents || !p_target || !p_draft || !u_node || !u_bonus || !path_out || !n_accept_out || !bonus_out)
        return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT || vocab < 1) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    other_kernel_enqueued();
    sample::accept_sample_kernel<<<c->layout.batch, sample::kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        draft_tokens, parents, p_target, p_draft, u_node, u_bonus, T, vocab, path_out, n_accept_out, bonus_out,
        reinterpret_cast<unsigned*>(c->ws));
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_kv_keep_accepted(sparrow_ctx* c, void* k_cache, void* v_cache, const int32_t* kv_len,
                                        const int32_t* path, const int32_t* n_accept, int32_t T, void* stream)
{
    if (!c || !k_cache || !v_cache || !kv_len || !path || !n_accept) return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (!aligned16(k_cache) || !aligned16(v_cache)) return SPARROW_ERR_SHAPE;
    const sparrow_layout& L = c->layout;
    KeepArgs a;
    std::memset(&a, 0, sizeof a);
    for (int b = 0; b < L.batch; ++b) {
        if (kv_len[b] < 0 || (int64_t)kv_len[b] + T > L.kv_capacity) return SPARROW_ERR_SHAPE;
        a.kv_len[b] = kv_len[b];
    }
    a.k = static_cast<__nv_bfloat16*>(k_cache);
    a.v = static_cast<__nv_bfloat16*>(v_cache);
    a.path = path;
    a.n_accept = n_accept;
    a.T = T;
    a.n_kv_heads = L.n_kv_heads;
    a.stride_batch = L.kv_stride_batch;
    a.stride_head = L.kv_stride_head;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    other_kernel_enqueued();
    keep_accepted_rows_kernel<<<L.batch * L.n_kv_heads, 256, (size_t)2 * T * 256, static_cast<cudaStream_t>(stream)>>>(a);
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_verify_step_host(sparrow_ctx* c, const void* q_host, const void* k_new_host,
                                        const void* v_new_host, void* k_cache, void* v_cache,
                                        const int32_t* kv_len, const int32_t* parents_host, int32_t T,
                                        void* out_host, float* lse_host, void* stream)
{
    if (!c || !q_host || !k_new_host || !v_new_host || !k_cache || !v_cache || !kv_len || !parents_host ||
        !out_host || !lse_host)
        return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    const sparrow_layout& L = c->layout;
    for (int b = 0; b < L.batch; ++b) {
        if (kv_len[b] < 0 || (int64_t)kv_len[b] + T > L.kv_capacity) return SPARROW_ERR_SHAPE;
        const sparrow_status ts = check_tree_host(parents_host + (size_t)b * T, T);
        if (ts != SPARROW_OK) return ts;
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Staging sl = staging_layout(L);
    unsigned char* base = c->ws + kStatusBytes;
    void* q_dev = base + sl.q;
    void* out_dev = base + sl.out;
    float* lse_dev = reinterpret_cast<float*>(base + sl.lse);
    int32_t* par_dev = reinterpret_cast<int32_t*>(base + sl.parents);
    const size_t q_bytes = (size_t)L.batch * T * L.n_q_heads * kD * 2;
    const size_t lse_bytes = (size_t)L.batch * L.n_q_heads * T * 4;
    const size_t new_bytes = (size_t)L.batch * L.n_kv_heads * T * kD * 2;
    // Host buffers the GPU can address itself (pinned or registered memory) are not copied by the
    // copy engine at all: one kernel reads q, the tree and the new K/V rows over the host link,
    // and the attention kernel writes out / lse straight into the host buffers.
    const void* q_view = device_view(q_host);
    const void* kn_view = device_view(k_new_host);
    const void* vn_view = device_view(v_new_host);
    const void* par_view = device_view(parents_host);
    void* out_view = device_view(out_host);
    void* lse_view = device_view(lse_host);
    if (q_view && kn_view && vn_view && par_view && out_view && lse_view) {
        IngestArgs ia;
        std::memset(&ia, 0, sizeof ia);
        for (int b = 0; b < L.batch; ++b) ia.rows.dst_row0[b] = kv_len[b];
        ia.rows.k_src = static_cast<const __nv_bfloat16*>(kn_view);
        ia.rows.v_src = static_cast<const __nv_bfloat16*>(vn_view);
        ia.rows.k_dst = static_cast<__nv_bfloat16*>(k_cache);
        ia.rows.v_dst = static_cast<__nv_bfloat16*>(v_cache);
        ia.rows.n_rows = T;
        ia.rows.batch = L.batch;
        ia.rows.n_kv_heads = L.n_kv_heads;
        ia.rows.src_capacity = T;
        ia.rows.src_stride_head = (int64_t)T * kD;
        ia.rows.src_stride_batch = ia.rows.src_stride_head * L.n_kv_heads;
        ia.rows.dst_stride_batch = L.kv_stride_batch;
        ia.rows.dst_stride_head = L.kv_stride_head;
        ia.rows.status = reinterpret_cast<unsigned*>(c->ws);
        ia.q_src = static_cast<const uint4*>(q_view);
        ia.q_dst = static_cast<uint4*>(q_dev);
        ia.q_chunks = (int32_t)(q_bytes / 16);
        ia.parents_src = static_cast<const int32_t*>(par_view);
        ia.parents_dst = par_dev;
        ia.n_parents = L.batch * T;
        const long long work = (long long)(new_bytes / 16) + ia.q_chunks + ia.n_parents;
        other_kernel_enqueued();
        ingest_step_kernel<<<(unsigned)((work + 255) / 256), 256, 0, st>>>(ia);
        if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
        c->launches.fetch_add(1);
        const sparrow_status s = sparrow_verify_attn(c, q_dev, k_cache, v_cache, kv_len, par_dev, T, out_view,
                                                     static_cast<float*>(lse_view), stream);
        if (s != SPARROW_OK) return s;
        return cudaStreamSynchronize(st) == cudaSuccess ? SPARROW_OK : SPARROW_ERR_CUDA;
    }
    if (cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaMemcpyAsync(par_dev, parents_host, (size_t)L.batch * T * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return SPARROW_ERR_CUDA;
    // the new rows: one contiguous copy each into the staging area, then the append kernel puts them
    // into the cache rows
    void* k_new_dev = base + sl.k_new;
    void* v_new_dev = base + sl.v_new;
    if (cudaMemcpyAsync(k_new_dev, k_new_host, new_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaMemcpyAsync(v_new_dev, v_new_host, new_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    const sparrow_status as = sparrow_kv_append(c, k_new_dev, v_new_dev, k_cache, v_cache, kv_len, T, stream);
    if (as != SPARROW_OK) return as;
    const sparrow_status s = sparrow_verify_attn(c, q_dev, k_cache, v_cache, kv_len, par_dev, T, out_dev, lse_dev, stream);
    if (s != SPARROW_OK) return s;
    if (cudaMemcpyAsync(out_host, out_dev, q_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaMemcpyAsync(lse_host, lse_dev, lse_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPARROW_ERR_CUDA;
    return SPARROW_OK;
}

sparrow_status sparrow_build_ancestor_masks(const int32_t* parents, int32_t T, uint64_t* masks)
{
    if (!parents || !masks) return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    const sparrow_status s = check_tree_host(parents, T);
    if (s != SPARROW_OK) return s;
    for (int i = 0; i < T; ++i) {                  // walk each node up to its root
        uint64_t m = 0;
        for (int a = i; a >= 0; a = parents[a]) m |= (uint64_t)1 << a;
        masks[i] = m;
    }
    return SPARROW_OK;
}

sparrow_status sparrow_build_anchor_idx(int32_t seq_len, const int32_t* spans, int32_t n_spans, int32_t window,
                                        int32_t T, int32_t* idx, int32_t* n_out)
{
    if (!idx || !n_out || (n_spans > 0 && !spans)) return SPARROW_ERR_NULL;
    if (seq_len < 0 || T < 0 || n_spans < 0) return SPARROW_ERR_SHAPE;
    for (int s = 0; s < n_spans; ++s)
        if (spans[2 * s] > spans[2 * s + 1]) return SPARROW_ERR_ANCHOR;
    const int32_t first = window > 0 && seq_len > window ? seq_len - window : 0;
    int32_t n = 0;
    for (int32_t p = first; p < seq_len; ++p) {
        bool text = true;
        for (int s = 0; s < n_spans && text; ++s) text = !(spans[2 * s] <= p && p < spans[2 * s + 1]);
        if (text) idx[n++] = p;
    }
    for (int32_t t = 0; t < T; ++t) idx[n++] = seq_len + t;
    *n_out = n;
    return SPARROW_OK;
}

sparrow_status sparrow_debug_ancestor_masks_device(sparrow_ctx* c, const int32_t* parents_dev, int32_t T,
                                                   uint64_t* masks_dev, void* stream)
{
    if (!c || !parents_dev || !masks_dev) return SPARROW_ERR_NULL;
    if (T < 1 || T > kMaxT) return SPARROW_ERR_SHAPE;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    other_kernel_enqueued();
    ancestor_masks_kernel<<<1, kMaxT, 0, static_cast<cudaStream_t>(stream)>>>(
        parents_dev, T, reinterpret_cast<unsigned long long*>(masks_dev), reinterpret_cast<unsigned*>(c->ws));
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_debug_wait_counter(sparrow_ctx* c, uint32_t ahead, void* stream)
{
    if (!c) return SPARROW_ERR_NULL;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    const unsigned* counter = reinterpret_cast<const unsigned*>(c->ws + kFinDoneOffset);
    wait_counter_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(counter, c->fin_total[0] + ahead,
                                                                         reinterpret_cast<unsigned*>(c->ws));
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_debug_early_trigger_copy(sparrow_ctx* c, const void* src, void* dst, size_t bytes,
                                               uint32_t delay_us, void* stream)
{
    if (!c || !src || !dst) return SPARROW_ERR_NULL;
    if (!aligned16(src) || !aligned16(dst) || (bytes & 15u) != 0) return SPARROW_ERR_SHAPE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    early_trigger_copy_kernel<<<8, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), bytes / 16, delay_us);
    if (cudaGetLastError() != cudaSuccess) return SPARROW_ERR_CUDA;
    c->launches.fetch_add(1);
    return SPARROW_OK;
}

sparrow_status sparrow_last_device_status(sparrow_ctx* c, void* stream)
{
    if (!c) return SPARROW_ERR_NULL;
    if (!c->ws) return SPARROW_ERR_WORKSPACE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SPARROW_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned word = 0;
    if (cudaMemcpyAsync(&word, c->ws, sizeof word, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaMemsetAsync(c->ws, 0, sizeof word, st) != cudaSuccess) return SPARROW_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPARROW_ERR_CUDA;
    c->last_status_word = word;
    if (word & kStatTimeout) {
        // A wait that gave up leaves the ordering counters in an unknown state: start them over.
        if (cudaMemsetAsync(c->ws, 0, kStatusBytes, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) return SPARROW_ERR_CUDA;
        c->seq = 0;
        c->fin_total[0] = c->fin_total[1] = 0;
        c->fin_before_last[0] = c->fin_before_last[1] = 0;
        c->prev_valid = false;
        c->n_recent = c->recent_head = 0;
    }
    if (word & kStatTimeout) return SPARROW_ERR_TIMEOUT;
    if (word & kStatTree) return SPARROW_ERR_TREE;
    if (word & kStatAnchor) return SPARROW_ERR_ANCHOR;
    return SPARROW_OK;
}

sparrow_status sparrow_set_plan_policy(sparrow_ctx* c, int32_t policy)
{
    if (!c) return SPARROW_ERR_NULL;
    if (policy != SPARROW_PLAN_LATENCY && policy != SPARROW_PLAN_BALANCED && policy != SPARROW_PLAN_THROUGHPUT)
        return SPARROW_ERR_SHAPE;
    c->plan_policy = policy;
    return SPARROW_OK;
}

sparrow_status sparrow_set_call_overlap(sparrow_ctx* c, int32_t enable)
{
    if (!c) return SPARROW_ERR_NULL;
    c->overlap_single_calls = enable != 0;
    return SPARROW_OK;
}

int32_t sparrow_plan_target_items(const sparrow_ctx* c) { return c ? plan_target(c, c->use_pdl) : 0; }

uint32_t sparrow_debug_status_word(const sparrow_ctx* c) { return c ? c->last_status_word : 0u; }

int64_t sparrow_launch_count(const sparrow_ctx* c) { return c ? (int64_t)c->launches.load() : 0; }

#ifdef SPARROW_TIMELINE
// Timeline build only (see common.cuh): read / clear the stamp table, and a one-thread kernel that
// stamps the stream position (so that a call's launch gap can be seen).
namespace {
__global__ void timeline_mark_kernel(unsigned long long* dst) { *dst = sparrow::global_timer_ns(); }
}
int sparrow_timeline_read(void* host_dst)
{
    return (int)cudaMemcpyFromSymbol(host_dst, sparrow::g_timeline, sizeof(sparrow::g_timeline));
}
int sparrow_timeline_clear()
{
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, sparrow::g_timeline) != cudaSuccess) return 1;
    return (int)cudaMemset(p, 0, sizeof(sparrow::g_timeline));
}
int sparrow_timeline_mark(void* dev_dst, void* stream)
{
    timeline_mark_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned long long*>(dev_dst));
    return (int)cudaGetLastError();
}
#endif

}  // extern "C"
