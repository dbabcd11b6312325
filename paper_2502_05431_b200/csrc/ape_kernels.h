// Internal launch interface between the host API (ape_api.cu) and the kernels.
#pragma once

#include "ape_common.cuh"

namespace ape {

constexpr int kDecodeTile = 64;     // tokens per pipeline stage of the decode kernel
constexpr int kAttnTileN = 128;     // keys per tile of the tensor-core (prefill / encode) kernel
constexpr int kAttnRows = 256;      // packed (token, head-in-group) rows per row block of that kernel (two 128-row halves)

struct DecodeParams {
    const DevTile* tiles;
    const DevItem* items;
    const int32_t* cta_item_begin;   // [n_cta + 1]
    const DevReq* reqs;
    RowsDesc q;
    float* ws_o;                     // [n_slots][G][D]  unnormalised partial outputs
    float* ws_ml;                    // [n_slots][G][2]  running maximum (base-2 logits) and sum
    float scale_oth_log2;            // c * log2(e)
    float scale_ctx_log2;            // c / T * log2(e)
    int32_t kv_extra;
    int32_t G;
    int32_t n_stages;
    int* status;
};

size_t decode_smem_bytes(int D, int G, int n_stages);
int decode_pick_stages(int D, int G, size_t smem_limit);
cudaError_t decode_set_smem_attr(int D, size_t smem_bytes);
cudaError_t launch_decode(int D, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const DecodeParams& p,
                          int n_cta, size_t smem_bytes, cudaStream_t stream);

// Tensor-core attention kernel shared by query prefill and context encoding.
enum : int32_t {
    kAttnPrefill = 0,   // long items, one Q buffer, two stages each of K and V
    kAttnEncode = 1,    // many short items with a row block each: two Q buffers, one V stage
    kAttnAlt = 2,       // row blocks of 128 rows: both halves read the same rows and take alternate tiles (three K/V stages)
    kAttnStats = 3,     // first pass of a plan with separately scaled context nodes: per row and node, (max, sum) of its own tokens
    kAttnBias = 4       // second pass of such a plan: prefill with a per-row, per-node bias on the context logits
};
struct AttnParams {
    const DevTile* tiles;
    const DevItem* items;
    const int32_t* cta_item_begin;   // [n_groups + 1]; CTA b serves group b / n_sib as sibling b % n_sib
    const DevReq* reqs;
    RowsDesc out;                    // SEG_FINAL items write here
    float* lse_out;                  // nullable, [rows, H_q] natural-log LSE for SEG_FINAL items
    float* ws_o;                     // [n_slots][kAttnRows][D]
    float* ws_ml;                    // [n_slots][kAttnRows][2]
    float scale_oth_log2;
    float scale_ctx_log2;
    int32_t G;
    int32_t H_q;
    int32_t n_sib;                   // sibling CTAs per group (row blocks that stream the same tiles together)
    int32_t q_rows_are_pool;         // encode: Q / O rows are pool tokens (row = context start + i)
    int32_t split_r;                 // rows of a TILE_SPLIT tile that come from the prefix (a multiple of 8; 0: no such tiles)
    int32_t o_via_tma;               // two-buffer plans whose items all have their own Q: full halves of O leave through shared
                                     // memory (the item's Q buffer) and a bulk tensor store described by tm_o
    int32_t mode;                    // kAttnPrefill ... kAttnBias; kAttnAlt: a slot holds two partials of 128 rows (half 0, half 1)
    // kAttnStats / kAttnBias: context tiles carry their node in key_base and TILE_CTX_END on a node's last tile; the value of
    // node n for row (request row base + token) * H_q + head is at index n * stat_rows + row; an item's ctx_id is its
    // request's row base
    float2* stats;                   // kAttnStats writes (running maximum, sum) in base-2 units
    const float* bias;               // kAttnBias reads the bias (base-2 units) of the node's tokens
    int64_t stat_rows;
    int* status;
};

size_t attn_smem_bytes(int D, int mode);
cudaError_t attn_set_smem_attr(int D, int mode, size_t smem_bytes);
// K and V boxes of split_r rows (prefix part) and 128 - split_r rows (context part) for TILE_SPLIT tiles
struct SplitMaps { CUtensorMap ka, kb, va, vb; };
cudaError_t launch_attn(int D, const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const CUtensorMap& tm_o,
                        const SplitMaps& split, const AttnParams& p, int n_cta, size_t smem_bytes, cudaStream_t stream);

// Merge of the partials: hierarchical softmax identity inside each segment, then Eq. 5's scaling factor.
struct MergeParams {
    const DevMerge* groups;
    const DevReq* reqs;
    const DevItem* items;            // per-context mode: the context ordinal of a partial is items[slot / slot_stride].ctx_id
    int32_t per_context;             // 0: Eq. 5 (S on the LSE of all contexts together); 1: Eq. 11-12 (S on every context's own LSE);
                                     // 2: context trees (the hierarchical formula node by node, S where a node is marked)
    const DevNode* nodes;            // tree plans: all requests' nodes
    int32_t n_groups;
    int32_t rows_per_slot;           // G (decode) or kAttnRows (prefill)
    int32_t tokens_per_block;        // query tokens per row block: rows_per_slot / G
    const float* ws_o;
    const float* ws_ml;
    // context partials; ordinary plans keep them in the same workspace with the same geometry as the others
    const float* ws_o_ctx;
    const float* ws_ml_ctx;
    int32_t rows_per_slot_ctx;
    RowsDesc out;
    float* lse_out;                  // nullable, [rows, H_q]
    // When part_o_ctx is set the kernel stops after the per-segment combine and writes each segment's normalised output
    // (fp32 [rows, H_q, D]) and natural-log LSE (fp32 [rows, H_q]) instead of the merged result: one shard of a
    // context-sharded attend.
    float* part_o_ctx;
    float* part_lse_ctx;
    float* part_o_oth;
    float* part_lse_oth;
    float S;
    int32_t G;
    int32_t H_q;
    int32_t D;
};
cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream);

// Between the two passes of a plan with separately scaled context nodes (per-context form: every context a marked
// top-level node; context trees): from the (maximum, sum) of every node's own tokens to the bias of its tokens' logits.
// Bottom-up, a node's log2 mass A_n combines its own tokens and its children (a marked child enters with S * A_c, Eq. 11,
// an unmarked one with A_c); top-down, the bias of a node is the sum of (S - 1) * A_a over the marked nodes a on its
// path to the root, itself included: with it, one plain softmax over all context keys gives every node's tokens the
// weight the hierarchical formula gives them.  A node's parent has a smaller index than the node.
struct NodeBiasParams {
    const DevNode* nodes;            // all requests' nodes; pad != 0: the node has tokens of its own
    const DevReq* reqs;              // pad: the request's row base (rows before it in the plan)
    const int32_t* req_node0;        // [n_req + 1]: the nodes of request r are req_node0[r] .. req_node0[r + 1] - 1
    int32_t n_req;
    const float2* stats;             // [n_nodes][stat_rows] from the statistics pass (base-2 units)
    float* mass;                     // [n_nodes][stat_rows] scratch: A_n
    float* bias;                     // [n_nodes][stat_rows] out
    int64_t stat_rows;
    float S;
    int32_t H_q;
    int32_t max_rows;                // largest q_len * H_q of a request
    int32_t max_nodes;               // most nodes of a request
    size_t smem_limit;               // dynamic shared memory a CTA may ask for on this device
};
cudaError_t launch_node_bias(const NodeBiasParams& p, cudaStream_t stream);

// Merge of the shards of a context-sharded attend: the context segments of all shards combine by the hierarchical softmax
// identity, then Eq. 5's scaling factor and the merge with the non-context segment.
struct ShardMergeParams {
    const float* o_ctx;              // [n_shards][rows][H_q][D]
    const float* lse_ctx;            // [n_shards][rows][H_q], natural log
    const float* o_oth;              // [rows][H_q][D]
    const float* lse_oth;            // [rows][H_q]
    int32_t n_shards;
    int64_t n_rows;
    RowsDesc out;
    float* lse_out;                  // nullable
    float S;
    int32_t H_q;
    int32_t D;
};
cudaError_t launch_shard_merge(const ShardMergeParams& p, cudaStream_t stream);

// Rotary embedding with position re-use, fused with the copy to its destination.
constexpr int kRopeChunkTokens = 16;   // tokens per work item
struct RopeChunk {
    int32_t src_tok, dst_tok;        // first source / destination row
    int32_t n_tok;                   // 1 .. kRopeChunkTokens
    int32_t pos0;                    // position of the first row; the following rows count up from it
};
struct RopeParams {
    const RopeChunk* chunks;
    int32_t n_chunks;
    struct { const __nv_bfloat16* data; int64_t token_stride, head_stride; } src;
    RowsDesc dst;
    int32_t n_heads;
    int32_t rotate;                  // 0: plain copy (V), 1: rotate (K, Q)
    double log2_theta;
};
cudaError_t launch_rope(int D, const RopeParams& p, int n_cta, cudaStream_t stream);

// Append of one new token per request to the cache (decode step D0): dense staged rows -> pool rows.
struct AppendParams {
    const __nv_bfloat16* k_new;      // [n_req][H_kv][D], dense
    const __nv_bfloat16* v_new;
    __nv_bfloat16* k_pool;
    __nv_bfloat16* v_pool;
    const int64_t* rows;             // [n_req]: pool row of the newest token when kv_extra = 0
    int64_t kv_extra;
    int64_t token_stride, head_stride;
    int32_t n_req, H_kv, D;
};
cudaError_t launch_append(const AppendParams& p, cudaStream_t stream);

}  // namespace ape
