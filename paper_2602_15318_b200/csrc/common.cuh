// Shared declarations of the CUDA path: the work decomposition handed to the kernels, the sticky
// device status bits, and the device-side ancestor-mask construction.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sparrow {

constexpr int kD = 128;           // head_dim
constexpr int kGroup = 7;         // query heads per KV head
constexpr int kMaxT = 64;
constexpr int kMaxBatch = 64;
constexpr int kTokPerBlock = 18;  // draft tokens per 128-row block: 18 x 7 = 126 rows, 2 rows of padding
constexpr int kBlockRows = 128;

// device status bits (sticky, OR-ed into the first word of the workspace)
constexpr unsigned kStatTree = 1u;
constexpr unsigned kStatAnchor = 2u;
constexpr unsigned kStatTimeout = 4u;

// The GQA group's 7 query heads x T draft tokens are packed into 128-row blocks: block i holds
// tokens [18 i, 18 i + 18), row r of a block is (token 18 i + r / 7, head r % 7), rows 126 and 127
// are padding.  A row group is 1 or 2 consecutive blocks, handled by one work item.
//
// One work item = (sequence b, KV head, row group, key-range piece).  Items of sequence b occupy
// [item_begin[b], item_begin[b+1]); inside, the index runs (kv head, row group, piece) with the
// piece fastest.  Piece s of n covers keys [n_keys*s/n, n_keys*(s+1)/n).
struct SplitPlan {
    int32_t n_items;
    int32_t batch;
    int32_t T;                    // draft tokens
    int32_t M;                    // query rows per KV head = 7*T
    int32_t blocks_per_group;     // 128-row blocks one work item handles (1 or 2)
    int32_t n_groups;             // ceil(T / (18 * blocks_per_group))
    int32_t n_kv_heads;
    int32_t part_rows;            // row pitch of one item's partial block in the workspace
    int32_t item_begin[kMaxBatch + 1];
    int32_t n_splits[kMaxBatch];
    int32_t n_keys[kMaxBatch];    // keys per sequence: kv_len + T (verify) or n_anchor (anchored)
    int32_t kv_len[kMaxBatch];    // verify mode only
};

struct Item {
    int b, kvh, group, split, key_begin, key_end;
};

__device__ __forceinline__ Item decode_item(const SplitPlan& p, int item)
{
    int b = 0;
    while (b + 1 < p.batch && item >= p.item_begin[b + 1]) ++b;
    const int local = item - p.item_begin[b];
    const int ns = p.n_splits[b];
    Item it;
    it.b = b;
    it.split = local % ns;
    const int unit = local / ns;
    it.group = unit % p.n_groups;
    it.kvh = unit / p.n_groups;
    const long long nk = p.n_keys[b];
    it.key_begin = (int)(nk * it.split / ns);
    it.key_end = (int)(nk * (it.split + 1) / ns);
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
