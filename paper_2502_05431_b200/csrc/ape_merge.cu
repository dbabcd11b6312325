// Merge kernel: turns the per-item partials (m, l, O~), kept in base-2 units, into the final output.
//   1. inside each segment (context / non-context) the partials of all splits are combined by the
//      hierarchical softmax identity (appendix "Hierarchical Formula for Softmax Attention"):
//      LSE = logsumexp_s(m_s + log2 l_s),  O = sum_s 2^(LSE_s - LSE) O_s;
//   2. the context log-sum-exp is multiplied by the scaling factor S and the two segments are merged by a
//      softmax over [S * LSE_C, LSE_other] (Eq. 5; appendix "Efficient Implementation").
// One warp per output row (query token, query head); lanes cover the head dimension.
#include "ape_common.cuh"
#include "ape_kernels.h"

namespace ape {

namespace {

constexpr float kLn2 = 0.6931471805599453f;

template <int VEC>
__device__ __forceinline__ void combine_segment(const float* __restrict__ ws_o, const float* __restrict__ ws_ml,
                                                int slot0, int n, int stride, int rows_per_slot, int row, int D,
                                                int lane, float& M, float& L, float (&acc)[VEC])
{
    M = -INFINITY; L = 0.f;
    #pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    // The partials are independent of each other: their loads are issued eight at a time, then folded in order (a merge
    // with many partials per row, such as a decode batch that shares its contexts, is bound by the latency of these loads).
    constexpr int kBatch = 8;
    for (int i0 = 0; i0 < n; i0 += kBatch) {
        float2 ml[kBatch];
        float x[kBatch][VEC];
        #pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const size_t slot = static_cast<size_t>(slot0) + static_cast<size_t>(i0 + u) * stride;
            ml[u] = (i0 + u < n) ? *reinterpret_cast<const float2*>(ws_ml + (slot * rows_per_slot + row) * 2) : make_float2(-INFINITY, 0.f);
        }
        #pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const size_t slot = static_cast<size_t>(slot0) + static_cast<size_t>(i0 + u) * stride;
            const float* src = ws_o + (slot * rows_per_slot + row) * D + lane * VEC;
            // Issued without waiting for (m, l): the row of an empty partial was never written, but it lies inside the
            // workspace, and the fold below never looks at what was read from it.
            if (i0 + u < n) {
                if constexpr (VEC == 4) { const float4 t = *reinterpret_cast<const float4*>(src); x[u][0] = t.x; x[u][1] = t.y; x[u][2] = t.z; x[u][3] = t.w; }
                else { const float2 t = *reinterpret_cast<const float2*>(src); x[u][0] = t.x; x[u][1] = t.y; }
            } else {
                #pragma unroll
                for (int v = 0; v < VEC; ++v) x[u][v] = 0.f;
            }
        }
        #pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (!(ml[u].y > 0.f)) continue;          // empty partial
            const float Mn = fmaxf(M, ml[u].x);
            const float f_old = fast_exp2(M - Mn), f_new = fast_exp2(ml[u].x - Mn);
            #pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] = acc[v] * f_old + x[u][v] * f_new;
            L = L * f_old + ml[u].y * f_new;
            M = Mn;
        }
    }
}

// Per-context form (appendix "Hierarchical Formula for APE", Eq. 11-12): every context C_i keeps its own normalised
// output and enters the final softmax with S * LSE_i.  Partials arrive grouped by context (consecutive slots with the same
// context ordinal); the result is the context segment's normalised output `acc` (to be divided by `norm`) and its
// scaled base-2 log weight `lse` = log2 sum_i 2^(S * LSE_i).
template <int VEC>
__device__ __forceinline__ void combine_per_context(const MergeParams& p, const DevMerge& g, int row, int lane,
                                                    float& lse, float& norm, float (&acc)[VEC])
{
    float top = -INFINITY, Z = 0.f;                   // running maximum of S * LSE_i and sum of 2^(S * LSE_i - top)
    #pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    float M = -INFINITY, L = 0.f, a[VEC];
    #pragma unroll
    for (int v = 0; v < VEC; ++v) a[v] = 0.f;
    const int item0 = g.ctx_slot0 / g.slot_stride;
    int cur = (g.ctx_n > 0) ? p.items[item0].ctx_id : 0;
    auto fold = [&]() {                               // close the current context
        if (L > 0.f) {
            const float li = p.S * (M + fast_log2(L));
            const float tn = fmaxf(top, li);
            const float f_old = fast_exp2(top - tn), f_new = fast_exp2(li - tn) / L;
            #pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] = acc[v] * f_old + a[v] * f_new;
            Z = Z * f_old + fast_exp2(li - tn);
            top = tn;
        }
        M = -INFINITY; L = 0.f;
        #pragma unroll
        for (int v = 0; v < VEC; ++v) a[v] = 0.f;
    };
    for (int i = 0; i < g.ctx_n; ++i) {
        const int cid = p.items[item0 + i].ctx_id;
        if (cid != cur) { fold(); cur = cid; }
        const size_t slot = static_cast<size_t>(g.ctx_slot0) + static_cast<size_t>(i) * g.slot_stride;
        const float2 ml = *reinterpret_cast<const float2*>(p.ws_ml + (slot * p.rows_per_slot + row) * 2);
        if (!(ml.y > 0.f)) continue;
        const float Mn = fmaxf(M, ml.x);
        const float f_old = fast_exp2(M - Mn), f_new = fast_exp2(ml.x - Mn);
        const float* src = p.ws_o + (slot * p.rows_per_slot + row) * p.D + lane * VEC;
        float x[VEC];
        if constexpr (VEC == 4) { const float4 t = *reinterpret_cast<const float4*>(src); x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
        else { const float2 t = *reinterpret_cast<const float2*>(src); x[0] = t.x; x[1] = t.y; }
        #pragma unroll
        for (int v = 0; v < VEC; ++v) a[v] = a[v] * f_old + x[v] * f_new;
        L = L * f_old + ml.y * f_new;
        M = Mn;
    }
    fold();
    norm = Z;
    lse = (Z > 0.f) ? top + fast_log2(Z) : -INFINITY;
}

// Context trees (appendix "Future Directions" on top of "Hierarchical Formula for APE"): the partials of a row arrive in
// depth-first order of the nodes their tiles belong to (a node's own tokens, then its subtrees).  A stack of accumulators,
// one per open tree level, follows that order: a partial is added to its node's accumulator; when the walk leaves a node,
// the node is finished -- log-sum-exp A_n and normalised output V_n of its members, by the plain hierarchical softmax
// identity -- and handed to its parent's accumulator as one member with log weight S * A_n if the node is marked, A_n
// otherwise.  Level 0 collects the top-level nodes; its content is the context side of the final softmax.
template <int VEC>
__device__ __forceinline__ void combine_tree(const MergeParams& p, const DevMerge& g, int row, int lane,
                                             float& lse, float& norm, float (&acc)[VEC])
{
    float top[kMaxTreeDepth + 1], Z[kMaxTreeDepth + 1], a[kMaxTreeDepth + 1][VEC];
    int node_at[kMaxTreeDepth + 1];
    top[0] = -INFINITY; Z[0] = 0.f; node_at[0] = -1;
    #pragma unroll
    for (int v = 0; v < VEC; ++v) a[0][v] = 0.f;
    int sp = 0;                                       // deepest open level; level k + 1 holds an open node of depth k
    auto add = [&](int lv, float m, float l, const float (&o)[VEC]) {
        const float Mn = fmaxf(top[lv], m);
        const float f_old = fast_exp2(top[lv] - Mn), f_new = fast_exp2(m - Mn);
        #pragma unroll
        for (int v = 0; v < VEC; ++v) a[lv][v] = a[lv][v] * f_old + o[v] * f_new;
        Z[lv] = Z[lv] * f_old + l * f_new;
        top[lv] = Mn;
    };
    auto close = [&](int lv) {                        // finish the node at level lv and hand it to level lv - 1
        if (Z[lv] > 0.f) {
            const float A = top[lv] + fast_log2(Z[lv]);
            const float handed = p.nodes[node_at[lv]].scaled ? p.S * A : A;
            const float inv = 1.f / Z[lv];
            float o[VEC];
            #pragma unroll
            for (int v = 0; v < VEC; ++v) o[v] = a[lv][v] * inv;
            add(lv - 1, handed, 1.f, o);
        }
    };
    auto ancestor = [&](int node, int depth_now, int depth_want) {
        for (; depth_now > depth_want; --depth_now) node = p.nodes[node].parent;
        return node;
    };
    const int item0 = g.ctx_slot0 / g.slot_stride;
    for (int i = 0; i < g.ctx_n; ++i) {
        const int node = p.items[item0 + i].ctx_id;
        const int depth = p.nodes[node].depth;
        // leave every open node that is not on the path from the top level down to `node`
        while (sp > 0 && (sp - 1 > depth || ancestor(node, depth, sp - 1) != node_at[sp])) { close(sp); --sp; }
        // open the rest of that path
        while (sp < depth + 1) {
            ++sp;
            node_at[sp] = ancestor(node, depth, sp - 1);
            top[sp] = -INFINITY; Z[sp] = 0.f;
            #pragma unroll
            for (int v = 0; v < VEC; ++v) a[sp][v] = 0.f;
        }
        const size_t slot = static_cast<size_t>(g.ctx_slot0) + static_cast<size_t>(i) * g.slot_stride;
        const float2 ml = *reinterpret_cast<const float2*>(p.ws_ml + (slot * p.rows_per_slot + row) * 2);
        if (!(ml.y > 0.f)) continue;
        const float* src = p.ws_o + (slot * p.rows_per_slot + row) * p.D + lane * VEC;
        float x[VEC];
        if constexpr (VEC == 4) { const float4 t = *reinterpret_cast<const float4*>(src); x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
        else { const float2 t = *reinterpret_cast<const float2*>(src); x[0] = t.x; x[1] = t.y; }
        add(sp, ml.x, ml.y, x);
    }
    while (sp > 0) { close(sp); --sp; }
    #pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = a[0][v];
    norm = Z[0];
    lse = (Z[0] > 0.f) ? top[0] + fast_log2(Z[0]) : -INFINITY;
}

template <int VEC>
__global__ void __launch_bounds__(256) ape_merge_kernel(const MergeParams p)
{
    const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int group = warp_global / p.rows_per_slot;
    const int row = warp_global - group * p.rows_per_slot;
    if (group >= p.n_groups) return;
    const DevMerge g = p.groups[group];
    const DevReq rq = p.reqs[g.req];
    const int tok = g.row_block * p.tokens_per_block + row / p.G;     // query row inside the request
    const int hg = row % p.G;
    if (tok >= rq.q_len) return;

    float Mc, Lc, Mo, Lo, ac[VEC], ao[VEC];
    float lse_c;
    if (p.per_context == 2) {
        combine_tree<VEC>(p, g, row, lane, lse_c, Lc, ac);             // Lc: the normaliser of ac
    } else if (p.per_context == 1) {
        combine_per_context<VEC>(p, g, row, lane, lse_c, Lc, ac);      // Lc: the normaliser of ac
    } else {
        combine_segment<VEC>(p.ws_o_ctx, p.ws_ml_ctx, g.ctx_slot0, g.ctx_n, g.ctx_stride, p.rows_per_slot_ctx, row + g.ctx_row_off,
                             p.D, lane, Mc, Lc, ac);
        // base-2 log-sum-exp of the context segment, multiplied by S (Eq. 5: Z_C^S)
        lse_c = (Lc > 0.f) ? p.S * (Mc + fast_log2(Lc)) : -INFINITY;
    }
    combine_segment<VEC>(p.ws_o, p.ws_ml, g.oth_slot0, g.oth_n, g.slot_stride, p.rows_per_slot, row, p.D, lane, Mo, Lo, ao);

    const int h = g.kv_head * p.G + hg;
    if (p.part_o_ctx != nullptr) {
        // one shard of a context-sharded attend: hand out the two segments as they are (Eq. 5 form only)
        const int64_t rh = static_cast<int64_t>(rq.q_row0 + tok) * p.H_q + h;
        const float ic = (Lc > 0.f) ? 1.f / Lc : 0.f, io = (Lo > 0.f) ? 1.f / Lo : 0.f;
        #pragma unroll
        for (int v = 0; v < VEC; ++v) {
            p.part_o_ctx[rh * p.D + lane * VEC + v] = ac[v] * ic;
            p.part_o_oth[rh * p.D + lane * VEC + v] = ao[v] * io;
        }
        if (lane == 0) {
            p.part_lse_ctx[rh] = (Lc > 0.f) ? (Mc + fast_log2(Lc)) * kLn2 : -INFINITY;
            p.part_lse_oth[rh] = (Lo > 0.f) ? (Mo + fast_log2(Lo)) * kLn2 : -INFINITY;
        }
        return;
    }
    const float lse_o = (Lo > 0.f) ? (Mo + fast_log2(Lo)) : -INFINITY;
    const float top = fmaxf(lse_c, lse_o);
    float wc = 0.f, wo = 0.f, lam = -INFINITY;
    if (top > -INFINITY) {
        const float ec = fast_exp2(lse_c - top), eo = fast_exp2(lse_o - top);
        const float inv = 1.f / (ec + eo);
        wc = (Lc > 0.f) ? ec * inv / Lc : 0.f;        // weight of the context segment over its own normaliser
        wo = (Lo > 0.f) ? eo * inv / Lo : 0.f;
        lam = (top + fast_log2(ec + eo)) * kLn2;
    }
    __nv_bfloat16* dst = p.out.data + static_cast<int64_t>(rq.q_row0 + tok) * p.out.token_stride
                         + static_cast<int64_t>(h) * p.out.head_stride + lane * VEC;
    float r[VEC];
    #pragma unroll
    for (int v = 0; v < VEC; ++v) r[v] = wc * ac[v] + wo * ao[v];
    if constexpr (VEC == 4) {
        uint2 pk; pk.x = pack_bf16x2(r[0], r[1]); pk.y = pack_bf16x2(r[2], r[3]);
        *reinterpret_cast<uint2*>(dst) = pk;
    } else {
        *reinterpret_cast<uint32_t*>(dst) = pack_bf16x2(r[0], r[1]);
    }
    if (p.lse_out != nullptr && lane == 0)
        p.lse_out[static_cast<int64_t>(rq.q_row0 + tok) * p.H_q + h] = lam;
}

// Shards of a context-sharded attend (each holds a subset of the contexts): LSE_C = log sum_s e^{LSE_s},
// O_C = sum_s e^{LSE_s - LSE_C} O_s (appendix "Hierarchical Formula for Softmax Attention"), then Eq. 5 as above.
template <int VEC>
__global__ void __launch_bounds__(256) ape_shard_merge_kernel(const ShardMergeParams p)
{
    constexpr float kLog2e = 1.4426950408889634f;
    const int64_t warp_global = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp_global >= p.n_rows * p.H_q) return;
    const int64_t row = warp_global / p.H_q;
    const int h = static_cast<int>(warp_global - row * p.H_q);
    float M = -INFINITY, Z = 0.f, acc[VEC];
    #pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    for (int s = 0; s < p.n_shards; ++s) {
        const int64_t rh = (static_cast<int64_t>(s) * p.n_rows + row) * p.H_q + h;
        const float l = p.lse_ctx[rh] * kLog2e;
        if (!(l > -INFINITY)) continue;
        const float Mn = fmaxf(M, l);
        const float f_old = fast_exp2(M - Mn), f_new = fast_exp2(l - Mn);
        #pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = acc[v] * f_old + p.o_ctx[rh * p.D + lane * VEC + v] * f_new;
        Z = Z * f_old + f_new;
        M = Mn;
    }
    const float lse_c = (Z > 0.f) ? p.S * (M + fast_log2(Z)) : -INFINITY;
    const int64_t rh = row * p.H_q + h;
    const float lo_nat = p.lse_oth[rh];
    const float lse_o = (lo_nat > -INFINITY) ? lo_nat * kLog2e : -INFINITY;
    const float top = fmaxf(lse_c, lse_o);
    float wc = 0.f, wo = 0.f, lam = -INFINITY;
    if (top > -INFINITY) {
        const float ec = fast_exp2(lse_c - top), eo = fast_exp2(lse_o - top);
        const float inv = 1.f / (ec + eo);
        wc = (Z > 0.f) ? ec * inv / Z : 0.f;
        wo = (lse_o > -INFINITY) ? eo * inv : 0.f;
        lam = (top + fast_log2(ec + eo)) * kLn2;
    }
    __nv_bfloat16* dst = p.out.data + row * p.out.token_stride + static_cast<int64_t>(h) * p.out.head_stride + lane * VEC;
    float r[VEC];
    #pragma unroll
    for (int v = 0; v < VEC; ++v) r[v] = wc * acc[v] + wo * p.o_oth[rh * p.D + lane * VEC + v];
    if constexpr (VEC == 4) {
        uint2 pk; pk.x = pack_bf16x2(r[0], r[1]); pk.y = pack_bf16x2(r[2], r[3]);
        *reinterpret_cast<uint2*>(dst) = pk;
    } else {
        *reinterpret_cast<uint32_t*>(dst) = pack_bf16x2(r[0], r[1]);
    }
    if (p.lse_out != nullptr && lane == 0) p.lse_out[rh] = lam;
}

}  // namespace

cudaError_t launch_shard_merge(const ShardMergeParams& p, cudaStream_t stream)
{
    const long long warps = static_cast<long long>(p.n_rows) * p.H_q;
    if (warps == 0) return cudaSuccess;
    const int blocks = static_cast<int>((warps * 32 + 255) / 256);
    if (p.D == 128) ape_shard_merge_kernel<4><<<blocks, 256, 0, stream>>>(p);
    else ape_shard_merge_kernel<2><<<blocks, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

namespace {

__device__ __forceinline__ float logaddexp2(float a, float b) {
    const float m = fmaxf(a, b);
    if (m == -INFINITY) return -INFINITY;
    return m + log2f(exp2f(a - m) + exp2f(b - m));
}

// One thread per query row (token, head) of a request; consecutive threads hold consecutive rows, so every access to the
// [node][row] arrays is coalesced.
__global__ void __launch_bounds__(256)
ape_node_bias_kernel(const NodeBiasParams p)
{
    const int r = blockIdx.y;
    const DevReq rq = p.reqs[r];
    const int64_t local = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (local >= static_cast<int64_t>(rq.q_len) * p.H_q) return;
    const int64_t row = static_cast<int64_t>(rq.pad) * p.H_q + local;
    const int n0 = p.req_node0[r], n1 = p.req_node0[r + 1];
    for (int n = n0; n < n1; ++n) p.mass[static_cast<int64_t>(n) * p.stat_rows + row] = -INFINITY;
    for (int n = n1 - 1; n >= n0; --n) {                     // children before parents
        const DevNode nd = p.nodes[n];
        float own = -INFINITY;
        if (nd.pad) {
            const float2 st = p.stats[static_cast<int64_t>(n) * p.stat_rows + row];
            if (st.y > 0.f) own = st.x + log2f(st.y);
        }
        const float A = logaddexp2(own, p.mass[static_cast<int64_t>(n) * p.stat_rows + row]);
        p.mass[static_cast<int64_t>(n) * p.stat_rows + row] = A;
        if (nd.parent >= 0) {
            float* up = p.mass + static_cast<int64_t>(nd.parent) * p.stat_rows + row;
            *up = logaddexp2(*up, nd.scaled ? p.S * A : A);
        }
    }
    for (int n = n0; n < n1; ++n) {                          // parents before children
        const DevNode nd = p.nodes[n];
        const float A = p.mass[static_cast<int64_t>(n) * p.stat_rows + row];
        float b = (nd.parent >= 0) ? p.bias[static_cast<int64_t>(nd.parent) * p.stat_rows + row] : 0.f;
        if (nd.scaled && A > -INFINITY) b += (p.S - 1.f) * A;
        p.bias[static_cast<int64_t>(n) * p.stat_rows + row] = b;
    }
}

// The same computation with a request's nodes x 32 rows in shared memory: a CTA takes 32 consecutive rows (lane = row).
// Reading the statistics and writing the biases is spread over the eight warps (node n goes to warp n mod 8, 256
// contiguous bytes per node); the two walks over the tree, which are sequential in the node index, are one warp's work
// on shared memory instead of a chain of dependent global-memory accesses per node.
constexpr int kBiasRows = 32;
__device__ __forceinline__ float logaddexp2_fast(float a, float b) {
    const float m = fmaxf(a, b);
    if (m == -INFINITY) return -INFINITY;
    return m + fast_log2(fast_exp2(a - m) + fast_exp2(b - m));
}
__global__ void __launch_bounds__(256)
ape_node_bias_smem_kernel(const NodeBiasParams p)
{
    extern __shared__ float val[];                           // [nodes of the request][32]: own mass, then A_n, then the bias
    const int r = blockIdx.y;
    const DevReq rq = p.reqs[r];
    const int64_t n_rows = static_cast<int64_t>(rq.q_len) * p.H_q;
    const int64_t local = static_cast<int64_t>(blockIdx.x) * kBiasRows + (threadIdx.x & 31);
    if (static_cast<int64_t>(blockIdx.x) * kBiasRows >= n_rows) return;
    const bool live = local < n_rows;
    const int64_t row = static_cast<int64_t>(rq.pad) * p.H_q + (live ? local : 0);
    const int n0 = p.req_node0[r], n_nodes = p.req_node0[r + 1] - n0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the node records (parent; scaled | 2 * has tokens) behind the values, so that everything below reads shared memory only
    int2* rec = reinterpret_cast<int2*>(val + static_cast<size_t>(n_nodes) * kBiasRows);
    for (int i = threadIdx.x; i < n_nodes; i += 256) {
        const DevNode nd = p.nodes[n0 + i];
        rec[i] = make_int2(nd.parent >= 0 ? nd.parent - n0 : -1, (nd.scaled ? 1 : 0) | (nd.pad ? 2 : 0));
    }
    __syncthreads();
    #pragma unroll 4
    for (int i = warp; i < n_nodes; i += 8) {                // independent loads: several in flight per warp
        float2 st = make_float2(0.f, 0.f);
        if (live && (rec[i].y & 2)) st = p.stats[static_cast<int64_t>(n0 + i) * p.stat_rows + row];
        val[i * kBiasRows + lane] = (st.y > 0.f) ? st.x + fast_log2(st.y) : -INFINITY;
    }
    __syncthreads();
    if (warp == 0) {
        for (int i = n_nodes - 1; i >= 0; --i) {             // children before parents
            const int2 nd = rec[i];
            if (nd.x >= 0) {
                const float A = val[i * kBiasRows + lane];
                float* up = &val[nd.x * kBiasRows + lane];
                *up = logaddexp2_fast(*up, (nd.y & 1) ? p.S * A : A);
            }
        }
        for (int i = 0; i < n_nodes; ++i) {                  // parents before children
            const int2 nd = rec[i];
            const float A = val[i * kBiasRows + lane];
            float b = (nd.x >= 0) ? val[nd.x * kBiasRows + lane] : 0.f;
            if ((nd.y & 1) && A > -INFINITY) b += (p.S - 1.f) * A;
            val[i * kBiasRows + lane] = b;
        }
    }
    __syncthreads();
    if (live)
        for (int i = warp; i < n_nodes; i += 8) p.bias[static_cast<int64_t>(n0 + i) * p.stat_rows + row] = val[i * kBiasRows + lane];
}

}  // namespace

cudaError_t launch_node_bias(const NodeBiasParams& p, cudaStream_t stream)
{
    if (p.n_req <= 0 || p.max_rows <= 0) return cudaSuccess;
    const size_t smem = static_cast<size_t>(p.max_nodes) * (kBiasRows * sizeof(float) + sizeof(int2));
    if (p.max_nodes > 0 && smem <= p.smem_limit) {
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(ape_node_bias_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
            return cudaGetLastError();
        const dim3 grid(static_cast<unsigned>((p.max_rows + kBiasRows - 1) / kBiasRows), static_cast<unsigned>(p.n_req));
        ape_node_bias_smem_kernel<<<grid, 256, smem, stream>>>(p);
        return cudaGetLastError();
    }
    // too many nodes for shared memory: the per-node arrays stay in global memory
    const dim3 grid(static_cast<unsigned>((p.max_rows + 255) / 256), static_cast<unsigned>(p.n_req));
    ape_node_bias_kernel<<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t stream)
{
    const long long warps = static_cast<long long>(p.n_groups) * p.rows_per_slot;
    if (warps == 0) return cudaSuccess;
    const int blocks = static_cast<int>((warps * 32 + 255) / 256);
    if (p.D == 128) ape_merge_kernel<4><<<blocks, 256, 0, stream>>>(p);
    else ape_merge_kernel<2><<<blocks, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace ape
