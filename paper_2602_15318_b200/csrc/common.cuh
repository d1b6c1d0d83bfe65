// Shared declarations of the CUDA path: the work decomposition handed to the kernels, the sticky
// device status bits, and the device-side ancestor-mask construction.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

// Timeline build (-DSPARROW_TIMELINE, made by `python -m paper_2602_15318_b200.timeline`; never
// the shipped library): SPARROW_STAMP(slot) records %globaltimer for (call, CTA, slot), and three
// extra exported calls read the table back.  A kernel names the call it belongs to once with
// SPARROW_TIMELINE_CALL(index) (kept modulo 32).  In the ordinary build both macros expand to nothing.
#ifdef SPARROW_TIMELINE
namespace sparrow {
constexpr int kTimelineCalls = 32, kTimelineCtas = 256, kTimelineSlots = 16;
__device__ unsigned long long g_timeline[kTimelineCalls * kTimelineCtas * kTimelineSlots];
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
}  // namespace sparrow
#define SPARROW_TIMELINE_CALL(index) const unsigned sparrow_tl_call = (unsigned)(index) % ::sparrow::kTimelineCalls
#define SPARROW_STAMP(slot)                                                                        \
    do {                                                                                           \
        if (blockIdx.x < ::sparrow::kTimelineCtas)                                                 \
            ::sparrow::g_timeline[((size_t)sparrow_tl_call * ::sparrow::kTimelineCtas + blockIdx.x) * ::sparrow::kTimelineSlots + (slot)] = \
                ::sparrow::global_timer_ns();                                                      \
    } while (0)
#else
#define SPARROW_TIMELINE_CALL(index) ((void)0)
#define SPARROW_STAMP(slot) ((void)0)
#endif

namespace sparrow {

constexpr int kD = 128;           // head_dim
constexpr int kMaxGroup = 16;      // query heads per KV head: 1 .. 16 (7 for the Qwen2-7B-shaped models of the paper)
constexpr int kMaxT = 64;
constexpr int kMaxBatch = 64;
// draft tokens per 128-row block for a group of g query heads: 18 for g = 7 (126 rows, 2 rows of padding)
__host__ __device__ constexpr int tokens_per_block(int g) { return 128 / g < 64 ? 128 / g : 64; }
constexpr int kBlockRows = 128;
constexpr int kKeyTile = 128;      // keys per tile of the tensor-core kernel; pieces of the key range are whole tiles

// device status bits (sticky, OR-ed into the first word of the workspace)
constexpr unsigned kStatTree = 1u;
constexpr unsigned kStatAnchor = 2u;
constexpr unsigned kStatTimeout = 4u;
// A wait that gives up also sets bit (8 + site) of the status word, so that the raw word tells which wait it was.
__host__ __device__ constexpr unsigned timeout_bits(int site) { return kStatTimeout | (1u << (8 + site)); }
enum WaitSite { kSiteProducer = 0, kSiteMma = 1, kSiteSoftmax = 2, kSiteWriteSame = 3, kSiteWriteOther = 4,
                kSiteArrivals = 5, kSiteFinOther = 6, kSiteFinCopies = 7, kSiteDebug = 8 };

// The GQA group's g query heads x T draft tokens are packed into 128-row blocks of p = 128 / g
// tokens: block i holds tokens [p i, p i + p), row r of a block is (token p i + r / g, head r % g),
// rows from g p on are padding (g = 7: 18 tokens, rows 126 and 127).  A row group is 1 or 2
// consecutive blocks, handled by one work item.
//
// One work item = (sequence b, KV head, row group, key-range piece).  Items of sequence b occupy
// [seq[b].item_begin, seq[b+1].item_begin); inside, the index runs (kv head, row group, piece) with the
// piece fastest.  Piece s of n covers keys [n_keys*s/n, n_keys*(s+1)/n).
struct SeqPlan {                  // per sequence
    int32_t item_begin;           // first work item of the sequence
    int32_t n_splits;             // key-range pieces per unit
    int32_t n_keys;               // kv_len + draft-tree nodes (verify) or n_anchor (anchored)
    int32_t kv_len;               // verify mode only
    int32_t key0;                 // first key that is streamed at all (a multiple of the tile; 0 unless a window cuts the prefix)
};
// Scalars first and the per-sequence entries as an array of structs: what a CTA reads of the plan
// then sits in one or two lines of the constant bank the kernel parameters live in.
struct SplitPlan {
    int32_t n_items;
    int32_t batch;
    int32_t T;                    // query tokens
    int32_t T_tree;               // nodes of the draft tree = rows of the draft block; the queries are its last T nodes
    int32_t group;                // g: query heads per KV head
    int32_t tok_per_block;        // p = tokens_per_block(g)
    int32_t M;                    // query rows per KV head = g*T
    int32_t blocks_per_group;     // 128-row blocks one work item handles (1 or 2)
    int32_t n_groups;             // ceil(T / (18 * blocks_per_group))
    int32_t n_kv_heads;
    int32_t part_rows;            // row pitch of one item's partial block in the workspace
    int32_t piece_tile;           // pieces of the key range are whole tiles of this many keys (128 or 64)
    SeqPlan seq[kMaxBatch];
};

constexpr int kFinisherCtas = 32;  // CTAs of a call that share its combine step
constexpr int kMaxGroups = 4;      // row groups per (sequence, KV head): at most 8 blocks (g = 16), 2 per group
constexpr int kArrivalSlots = 4;   // arrival words rotate over the call number modulo 4
// A partial row in the workspace: 128 fp16 outputs, then the row's fp32 LSE, padded to 16 bytes,
// so that one bulk copy brings a run of rows with everything needed to merge them.
constexpr int kPartRowHalves = 136;

// Overlapped mode: ordering between the CTAs of one call and between consecutive calls.
//
// The split-KV kernel is launched with programmatic stream serialisation and never waits for the
// previous grid as a whole, so the next call's CTAs start (and read their inputs) while the
// previous call is still finishing.  What must be ordered goes through counters in the workspace,
// released / acquired at GPU scope.  Partial buffers are double-buffered by the parity of the call
// number n, arrival words rotate over n modulo 4.
//   arrivals[n % 4]   items of call n that have published their partials
//   fin_done[n % 2]   final-result writers of calls with this parity that are done, cumulative
// An item whose unit (sequence, KV head, row group) has several key-range pieces stores a partial
// and arrives; an item that is its unit's only piece writes final results itself.  The last
// n_fin CTAs of the grid are the call's finishers (all of them where the call has the GPU to
// itself anyway) -- they are the last to start, so by the time
// they are through with their own items little is left to wait for: they wait until every
// partial of the call has arrived, then each merges a contiguous share of the call's rows by
// log-sum-exp and writes the final out / lse.  Every final-result writer (finisher or single
// piece) bumps fin_done once.
// Before its first global write an item of call n waits until the writers of call n-2 are done
// (fin_wait_same: the finishers among them read the partial buffer it is about to overwrite);
// whoever writes final results also waits for the writers of call n-1 (fin_wait_other), so
// results land in call order.  CTA 0 then clears the arrival word of slot (n + 2) % 4: its last
// user was call n-2, and the items of call n+2 cannot arrive before the finishers of call n are
// done, which in turn have seen CTA 0's arrival (or, if it had none, follow it in the stream).
// With enabled == 0 the kernels are ordered by the stream alone: they touch no counter, and a
// separate combine kernel follows the split-KV kernel.
struct SyncArgs {
    unsigned* arrivals;      // [4]
    unsigned* fin_done;      // [2]
    int32_t enabled;         // overlapped mode
    int32_t parity;          // n % 2
    int32_t slot;            // n % 4
    int32_t n_arrive;        // items of this call that store partials
    int32_t n_fin;           // finisher CTAs of this call (0 when no unit has several pieces)
    uint32_t fin_wait_same;
    uint32_t fin_wait_other;
    uint32_t call;           // running number of the context's fused calls (the timeline build files its stamps under it)
};

__device__ __forceinline__ unsigned ld_acquire(const unsigned* addr)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
    return v;
}
// Polls of a counter wait before it gives up: with the pause between polls this is of the order of
// a second.  The bound counts polls rather than reading a timer, so it cannot misfire on a timer
// glitch and does not depend on the timer's resolution.
constexpr uint32_t kCounterPolls = 1u << 22;
// Bounded acquire-wait until a cumulative counter has reached `target` (wrap-safe compare).
__device__ __forceinline__ bool wait_counter(const unsigned* addr, uint32_t target)
{
    #pragma unroll 1
    for (uint32_t i = 0; i < kCounterPolls; ++i) {
        if ((int32_t)(ld_acquire(addr) - target) >= 0) return true;
        __nanosleep(i < 64 ? 40 : 200);
    }
    return false;
}
// Bounded acquire-wait until a word equals `value`.
__device__ __forceinline__ bool wait_equal(const unsigned* addr, uint32_t value)
{
    #pragma unroll 1
    for (uint32_t i = 0; i < kCounterPolls; ++i) {
        if (ld_acquire(addr) == value) return true;
        __nanosleep(i < 64 ? 40 : 200);
    }
    return false;
}
// Release-increment of a counter: orders every write this thread has observed (its own and, after
// a CTA barrier, its CTA's) before the increment.
__device__ __forceinline__ void publish_counter(unsigned* addr)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(addr) : "memory");
}

struct Item {
    int b, kvh, group, split, key_begin, key_end;
};

// Key range of piece `split` of `ns` over `n_keys` keys: pieces are whole tiles of `tile` keys (the
// kernel's unit of work: 128 on the tensor-core path, 64 on the gathered one), as even as whole
// tiles allow; the last piece takes the ragged end.  Needs ns <= number of tiles, which the
// planner guarantees (pieces of at least one tile).
__host__ __device__ __forceinline__ void piece_range(int n_keys, int ns, int split, int tile, int* begin, int* end)
{
    const long long n_tiles = (n_keys + tile - 1) / tile;
    const long long b = n_tiles * split / ns * tile, e = n_tiles * (split + 1) / ns * tile;
    *begin = (int)b;
    *end = (int)(e < n_keys ? e : n_keys);
}

__device__ __forceinline__ Item decode_item(const SplitPlan& p, int item)
{
    int b = 0;
    while (b + 1 < p.batch && item >= p.seq[b + 1].item_begin) ++b;
    const int local = item - p.seq[b].item_begin;
    const int ns = p.seq[b].n_splits;
    Item it;
    it.b = b;
    it.split = local % ns;
    const int unit = local / ns;
    it.group = unit % p.n_groups;
    it.kvh = unit / p.n_groups;
    const int key0 = p.seq[b].key0;
    piece_range(p.seq[b].n_keys - key0, ns, it.split, p.piece_tile, &it.key_begin, &it.key_end);
    it.key_begin += key0;
    it.key_end += key0;
    return it;
}

// Ancestor word of draft node i: bit a set iff a == i or a is an ancestor of i.  Walks the parent
// chain (at most T steps, so a malformed array cannot loop).  A parent outside [-1, node) is
// treated as "root" and reported.
__device__ __forceinline__ unsigned long long ancestor_word(const int32_t* __restrict__ parents,
                                                            int T, int i, unsigned* status)
{
    unsigned long long m = 1ull << i;
    int node = i;
    for (int step = 0; step < T; ++step) {
        const int p = parents[node];
        if (p == -1) break;
        if (p < -1 || p >= node) {
            if (status) atomicOr(status, kStatTree);
            break;
        }
        m |= 1ull << p;
        node = p;
    }
    return m;
}

}  // namespace sparrow
