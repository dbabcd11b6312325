// Host side of libape: argument validation, planning (tile lists, work assignment, copy-engine descriptors)
// and the launches behind the C ABI declared in include/ape.h.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/ape.h"
#include "ape_kernels.h"

using namespace ape;

namespace {

enum PlanKind { PLAN_PREFILL = 0, PLAN_DECODE = 1, PLAN_ENCODE = 2, PLAN_ROPE = 3, PLAN_SHARED = 4 };

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct ape_handle_s {
    int device = 0;
    int n_sm = 0;                   // CTAs a plan may use: the device's SM count unless ape_set_sm_budget lowered it
    int n_sm_device = 0;
    size_t smem_optin = 0;
    int* d_status = nullptr;
    EncodeTiledFn encode_tiled = nullptr;
};

struct ape_plan_s {
    ape_handle_t h = nullptr;
    PlanKind kind = PLAN_PREFILL;
    ape_shape_t shape{};
    float c = 0.f;
    int G = 1;
    ape_kv_pool_t pool{};
    ape_rows_t q{}, out{};
    float* lse = nullptr;
    // device metadata (one allocation)
    void* d_blob = nullptr;
    DevTile* d_tiles = nullptr;
    DevItem* d_items = nullptr;
    int32_t* d_cta_begin = nullptr;
    DevReq* d_reqs = nullptr;
    DevMerge* d_merge = nullptr;
    int n_items = 0, n_cta = 0, n_merge = 0, n_sib = 1, n_slots = 0;
    int n_stages = 0;
    size_t smem_bytes = 0;
    size_t ws_bytes = 0;
    int64_t max_kv_extra = 0;
    CUtensorMap tm_q{}, tm_k{}, tm_v{}, tm_o{};
    SplitMaps tm_split{};           // encode plans with split_r > 0
    int split_r = 0;
    bool o_via_tma = false;         // encode plans: tm_o describes the output rows
    bool alt_halves = false;        // context pass of a shared plan with at most 128 rows: the halves take alternate tiles
    int32_t last_launches = 0;
    int per_context = 0;             // merge form: 0 Eq. 5, 1 Eq. 11-12 (per context), 2 context trees
    DevNode* d_nodes = nullptr;      // tree plans; two-pass plans
    // Prefill plans of the per-context and tree forms run in two passes (statistics of every node's own tokens, then
    // the prefill with per-row, per-node biases): their per-node arrays live behind the partials in the workspace.
    bool two_pass = false;
    int32_t* d_req_node0 = nullptr;  // [n_req + 1]
    int n_nodes = 0, max_rows = 0, max_nodes = 0;
    int64_t stat_rows = 0;
    size_t off_stats = 0, off_mass = 0, off_bias = 0;
    // shared-context decode plans: the context pass of all requests (tensor-core kernel) and the per-request rest (decode kernel)
    ape_plan_s* child_ctx = nullptr;
    ape_plan_s* child_oth = nullptr;
    // decode plans: what the host-buffer step needs (staging for the new token's Q is the plan's Q tensor itself)
    int n_req = 0;
    std::vector<int64_t> q_rows;     // Q / O row of every request
    void* d_step = nullptr;          // [n_req] int64 append rows, then dense staging for the new K and V rows
    // rotary-embedding plans
    RopeChunk* d_rope_chunks = nullptr;
    int n_rope_chunks = 0;
    double rope_log2_theta = 0.0;
    int64_t rope_src_rows = 0, rope_dst_rows = 0;    // one past the largest row the runs touch
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(const ape_shape_t* s, int* G_out, float* c_out) {
    if (!s) return APE_ERR_INVALID_ARG;
    if (s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->n_q_heads % s->n_kv_heads) return APE_ERR_SHAPE;
    const int G = s->n_q_heads / s->n_kv_heads;
    if (G > 16 || (G & (G - 1))) return APE_ERR_SHAPE;
    if (s->head_dim != 64 && s->head_dim != 128) return APE_ERR_SHAPE;
    if (!(s->softmax_scale >= 0.f) || !std::isfinite(s->softmax_scale)) return APE_ERR_RANGE;
    *G_out = G;
    *c_out = s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / std::sqrt(static_cast<float>(s->head_dim));
    return APE_OK;
}

int check_pool(const ape_kv_pool_t* p, const ape_shape_t* s) {
    if (!p || !p->k || !p->v || p->n_tokens <= 0) return APE_ERR_INVALID_ARG;
    if (!aligned16(p->k) || !aligned16(p->v)) return APE_ERR_ALIGN;
    if (p->head_stride % 8 || p->token_stride % 8) return APE_ERR_ALIGN;
    if (p->head_stride < s->head_dim || p->token_stride < static_cast<int64_t>(s->n_kv_heads - 1) * p->head_stride + s->head_dim)
        return APE_ERR_INVALID_ARG;
    if (p->n_tokens >= (1ll << 31) - 256) return APE_ERR_LAYOUT;
    return APE_OK;
}

int check_rows(const ape_rows_t* r, const ape_shape_t* s) {
    if (!r || !r->data || r->n_rows <= 0) return APE_ERR_INVALID_ARG;
    if (!aligned16(r->data)) return APE_ERR_ALIGN;
    if (r->head_stride % 8 || r->token_stride % 8) return APE_ERR_ALIGN;
    if (r->head_stride < s->head_dim || r->token_stride < static_cast<int64_t>(s->n_q_heads - 1) * r->head_stride + s->head_dim)
        return APE_ERR_INVALID_ARG;
    if (r->n_rows >= (1ll << 31) - 256) return APE_ERR_LAYOUT;
    return APE_OK;
}

// the optional fp32 log-sum-exp output: one float per (row, head), so the pointer must be float-aligned
int check_lse(const float* lse) { return (reinterpret_cast<uintptr_t>(lse) & 3u) ? APE_ERR_ALIGN : APE_OK; }

bool span_ok(const ape_span_t& s, int64_t n_tokens) {
    return s.len >= 0 && s.start >= 0 && s.start <= n_tokens && s.len <= n_tokens - s.start;
}

// bf16 [rows, heads, d] described to the copy engine as (d, heads, rows) with a 64-element (128-byte) swizzled box row.
int make_map(ape_handle_t h, CUtensorMap* tm, const void* base, int d, int64_t heads, int64_t rows,
             int64_t head_stride, int64_t token_stride, int box_heads, int box_rows) {
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(head_stride) * 2, static_cast<cuuint64_t>(token_stride) * 2};
    cuuint32_t box[3] = {64u, static_cast<cuuint32_t>(box_heads), static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    if (box_rows > 256 || box_heads > 256) return APE_ERR_LAYOUT;
    const CUresult r = h->encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? APE_OK : APE_ERR_LAYOUT;
}

void add_span_tiles(std::vector<DevTile>& tiles, int64_t start, int64_t len, int tile, int32_t flags, int64_t grow_capacity) {
    const int64_t extent = (flags & TILE_GROWS) ? grow_capacity : len;
    for (int64_t off = 0; off < extent; off += tile) {
        DevTile t;
        t.tok = static_cast<int32_t>(start + off);
        t.n_valid = static_cast<int32_t>(std::max<int64_t>(0, std::min<int64_t>(tile, len - off)));
        t.key_base = static_cast<int32_t>(off);
        t.flags = flags;
        tiles.push_back(t);
    }
}

// Context spans in any order -> sorted, with touching spans fused (Eq. 5 treats all contexts as one segment,
// so boundaries between contexts do not matter to attend).
std::vector<ape_span_t> fuse_spans(const ape_span_t* ctx, int n) {
    std::vector<ape_span_t> v;
    for (int i = 0; i < n; ++i) if (ctx[i].len > 0) v.push_back(ctx[i]);
    std::sort(v.begin(), v.end(), [](const ape_span_t& a, const ape_span_t& b) { return a.start < b.start; });
    std::vector<ape_span_t> out;
    for (const auto& s : v) {
        if (!out.empty() && out.back().start + out.back().len == s.start) out.back().len += s.len;
        else out.push_back(s);
    }
    return out;
}

// Tile ranges of the context segment: one range over the fused spans (Eq. 5 form), or one range per non-empty
// context in the caller's order (per-context form; `id` is the context's ordinal among the non-empty ones).
struct CtxRange { int t0, t1, id; };
std::vector<CtxRange> add_context_tiles(std::vector<DevTile>& tiles, const ape_span_t* ctx, int n, int tile, bool per_context) {
    std::vector<CtxRange> ranges;
    if (!per_context) {
        const int t0 = static_cast<int>(tiles.size());
        for (const auto& s : fuse_spans(ctx, n)) add_span_tiles(tiles, s.start, s.len, tile, 0, 0);
        if (static_cast<int>(tiles.size()) > t0) ranges.push_back({t0, static_cast<int>(tiles.size()), 0});
    } else {
        for (int i = 0; i < n; ++i) {
            if (ctx[i].len <= 0) continue;
            const int t0 = static_cast<int>(tiles.size());
            add_span_tiles(tiles, ctx[i].start, ctx[i].len, tile, 0, 0);
            ranges.push_back({t0, static_cast<int>(tiles.size()), static_cast<int>(ranges.size())});
        }
    }
    return ranges;
}

// Context trees: the nodes of one request in depth-first order (a node's own tokens, then its subtrees, children in
// index order), one tile range per node that holds tokens; `id` is the node's index in the plan-wide node array.  The
// merge kernel relies on this order: once the walk has left a subtree it never returns to it.
std::vector<CtxRange> add_tree_tiles(std::vector<DevTile>& tiles, const ape_span_t* ctx, const int32_t* parent, int n, int tile,
                                     int node_base) {
    std::vector<std::vector<int>> children(n);
    std::vector<int> roots, stack;
    for (int i = 0; i < n; ++i) (parent[i] < 0 ? roots : children[parent[i]]).push_back(i);
    std::vector<CtxRange> ranges;
    for (auto r = roots.rbegin(); r != roots.rend(); ++r) stack.push_back(*r);
    while (!stack.empty()) {
        const int i = stack.back(); stack.pop_back();
        if (ctx[i].len > 0) {
            const int t0 = static_cast<int>(tiles.size());
            add_span_tiles(tiles, ctx[i].start, ctx[i].len, tile, 0, 0);
            ranges.push_back({t0, static_cast<int>(tiles.size()), node_base + i});
        }
        for (auto c = children[i].rbegin(); c != children[i].rend(); ++c) stack.push_back(*c);
    }
    return ranges;
}

struct HostMeta {
    std::vector<DevTile> tiles;
    std::vector<DevItem> items;
    std::vector<int32_t> cta_begin;
    std::vector<DevReq> reqs;
    std::vector<DevMerge> merge;
    std::vector<DevNode> nodes;      // tree plans; two-pass plans
    std::vector<int32_t> req_node0;  // two-pass plans: first node of every request, and the total
};

struct Run {   // a run of tiles of one segment for one (request, kv head, row-block group)
    int req, kv_head, row_block, n_sib, seg, t0, t1, merge0;
    int ctx_id = 0;   // per-context plans: ordinal of the context of a SEG_CTX run
};

// Split the concatenation of all runs evenly over n_bins bins (each bin = one CTA or one sibling group);
// a run that straddles a bin boundary becomes several items, each with its own partial slot.
// With align_nodes (two-pass plans) a context run is only cut behind a tile that ends a node: the statistics pass keeps a
// node's running (maximum, sum) in registers and writes it once, so a node's tiles must not be spread over two items.
void assign_stream(const std::vector<Run>& runs, int n_bins, int slot_mult, HostMeta& m, bool align_nodes = false) {
    long long total = 0;
    for (const auto& r : runs) total += r.t1 - r.t0;
    const long long chunk = std::max<long long>(1, (total + n_bins - 1) / n_bins);
    m.cta_begin.assign(1, 0);
    long long room = chunk;
    for (const auto& r : runs) {
        int t = r.t0;
        while (t < r.t1) {
            int take = static_cast<int>(std::min<long long>(room, r.t1 - t));
            if (align_nodes && r.seg == SEG_CTX)
                while (t + take < r.t1 && !(m.tiles[t + take - 1].flags & TILE_CTX_END)) ++take;
            DevItem it;
            it.req = r.req; it.kv_head = r.kv_head; it.row_block = r.row_block;
            it.tile_begin = t; it.tile_end = t + take;
            it.slot = static_cast<int32_t>(m.items.size()) * slot_mult;
            it.seg = r.seg; it.n_sib = r.n_sib; it.ctx_id = r.ctx_id;
            // bookkeeping for the merge: every live sibling's group record learns about this partial
            for (int s = 0; s < r.n_sib; ++s) {
                DevMerge& g = m.merge[r.merge0 + s];
                g.slot_stride = slot_mult; g.ctx_stride = slot_mult;
                if (r.seg == SEG_CTX) { if (g.ctx_n == 0) g.ctx_slot0 = it.slot + s; g.ctx_n++; }
                else { if (g.oth_n == 0) g.oth_slot0 = it.slot + s; g.oth_n++; }
            }
            m.items.push_back(it);
            t += take; room -= take;
            if (room <= 0) { m.cta_begin.push_back(static_cast<int32_t>(m.items.size())); room = chunk; }
        }
    }
    while (static_cast<int>(m.cta_begin.size()) < n_bins + 1) m.cta_begin.push_back(static_cast<int32_t>(m.items.size()));
}

// Every item carries a copy of its request's geometry and of its first tile record.
void finish_items(HostMeta& m) {
    for (auto& it : m.items) {
        const DevReq& rq = m.reqs[it.req];
        it.q_row0 = rq.q_row0; it.q_len = rq.q_len; it.l_k = rq.l_k;
        if (it.tile_begin < static_cast<int32_t>(m.tiles.size())) it.first_tile = m.tiles[it.tile_begin];
        else it.first_tile = DevTile{0, 0, 0, 0};
    }
}

int upload(ape_plan_t p, const HostMeta& m) {
    auto rnd = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t b_tiles = rnd(m.tiles.size() * sizeof(DevTile) + 16), b_items = rnd(m.items.size() * sizeof(DevItem) + 16),
                 b_cta = rnd(m.cta_begin.size() * 4 + 16), b_reqs = rnd(m.reqs.size() * sizeof(DevReq) + 16),
                 b_merge = rnd(m.merge.size() * sizeof(DevMerge) + 16), b_nodes = rnd(m.nodes.size() * sizeof(DevNode) + 16),
                 b_rn = rnd(m.req_node0.size() * 4 + 16);
    const size_t total = b_tiles + b_items + b_cta + b_reqs + b_merge + b_nodes + b_rn;
    std::vector<uint8_t> host(total, 0);
    size_t o = 0;
    auto put = [&](const void* src, size_t n, size_t padded) { if (n) std::memcpy(host.data() + o, src, n); size_t at = o; o += padded; return at; };
    const size_t o_tiles = put(m.tiles.data(), m.tiles.size() * sizeof(DevTile), b_tiles);
    const size_t o_items = put(m.items.data(), m.items.size() * sizeof(DevItem), b_items);
    const size_t o_cta = put(m.cta_begin.data(), m.cta_begin.size() * 4, b_cta);
    const size_t o_reqs = put(m.reqs.data(), m.reqs.size() * sizeof(DevReq), b_reqs);
    const size_t o_merge = put(m.merge.data(), m.merge.size() * sizeof(DevMerge), b_merge);
    const size_t o_nodes = put(m.nodes.data(), m.nodes.size() * sizeof(DevNode), b_nodes);
    const size_t o_rn = put(m.req_node0.data(), m.req_node0.size() * 4, b_rn);
    if (cudaMalloc(&p->d_blob, total) != cudaSuccess) { p->d_blob = nullptr; return APE_ERR_NOMEM; }
    if (cudaMemcpy(p->d_blob, host.data(), total, cudaMemcpyHostToDevice) != cudaSuccess) return APE_ERR_CUDA;
    uint8_t* b = static_cast<uint8_t*>(p->d_blob);
    p->d_tiles = reinterpret_cast<DevTile*>(b + o_tiles);
    p->d_items = reinterpret_cast<DevItem*>(b + o_items);
    p->d_cta_begin = reinterpret_cast<int32_t*>(b + o_cta);
    p->d_reqs = reinterpret_cast<DevReq*>(b + o_reqs);
    p->d_merge = reinterpret_cast<DevMerge*>(b + o_merge);
    p->d_nodes = reinterpret_cast<DevNode*>(b + o_nodes);
    p->d_req_node0 = reinterpret_cast<int32_t*>(b + o_rn);
    p->n_items = static_cast<int>(m.items.size());
    p->n_merge = static_cast<int>(m.merge.size());
    return APE_OK;
}

RowsDesc rows_desc(const ape_rows_t& r) {
    RowsDesc d; d.data = static_cast<__nv_bfloat16*>(r.data); d.token_stride = r.token_stride; d.head_stride = r.head_stride; return d;
}

// Makes `device` current for the lifetime of the object and puts the caller's current device back afterwards: an entry
// point never leaves a different device current than the one it found.
struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int device) {
        int cur = -1;
        if (cudaGetDevice(&cur) != cudaSuccess) cur = -1;
        if (cur == device) { ok = true; return; }
        ok = cudaSetDevice(device) == cudaSuccess;
        if (ok) prev = cur;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
    DeviceGuard(const DeviceGuard&) = delete;
    DeviceGuard& operator=(const DeviceGuard&) = delete;
};

// Decode plans keep, per request, the pool row of its newest token and a small dense staging area for the K and V rows of
// the next one, so that a step whose inputs arrive in host memory needs three copies and no allocation.
int setup_decode_step(ape_plan_t p, const ape_request_t* reqs, int n_req) {
    p->n_req = n_req;
    std::vector<int64_t> rows(n_req);
    p->q_rows.resize(n_req);
    for (int r = 0; r < n_req; ++r) { rows[r] = reqs[r].query_kv.start + reqs[r].query_kv.len - 1; p->q_rows[r] = reqs[r].q_start; }
    const size_t b_rows = (static_cast<size_t>(n_req) * 8 + 255) & ~size_t(255);
    const size_t b_stage = static_cast<size_t>(n_req) * p->shape.n_kv_heads * p->shape.head_dim * 2;
    if (cudaMalloc(&p->d_step, b_rows + 2 * b_stage) != cudaSuccess) { p->d_step = nullptr; return APE_ERR_NOMEM; }
    if (cudaMemcpy(p->d_step, rows.data(), static_cast<size_t>(n_req) * 8, cudaMemcpyHostToDevice) != cudaSuccess) return APE_ERR_CUDA;
    return APE_OK;
}

}  // namespace

extern "C" {

int ape_create(ape_handle_t* handle, int device) {
    if (!handle) return APE_ERR_INVALID_ARG;
    *handle = nullptr;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess) return APE_ERR_CUDA;
    if (device < 0 || device >= n_dev) return APE_ERR_INVALID_ARG;
    ape_handle_t h = new (std::nothrow) ape_handle_s();
    if (!h) return APE_ERR_NOMEM;
    h->device = device;
    DeviceGuard guard(device);
    cudaDeviceProp prop;
    if (!guard.ok || cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete h; return APE_ERR_CUDA; }
    if (prop.major != 10) { delete h; return APE_ERR_CUDA; }      // the kernels are built for sm_100a only
    h->n_sm = h->n_sm_device = prop.multiProcessorCount;
    h->smem_optin = prop.sharedMemPerBlockOptin;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) { delete h; return APE_ERR_CUDA; }
    h->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    if (cudaMalloc(&h->d_status, sizeof(int)) != cudaSuccess) { delete h; return APE_ERR_NOMEM; }
    if (cudaMemset(h->d_status, 0, sizeof(int)) != cudaSuccess) { cudaFree(h->d_status); delete h; return APE_ERR_CUDA; }
    *handle = h;
    return APE_OK;
}

int ape_destroy(ape_handle_t h) {
    if (!h) return APE_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (h->d_status) cudaFree(h->d_status);
    delete h;
    return APE_OK;
}

int ape_plan_destroy(ape_plan_t p) {
    if (!p) return APE_ERR_INVALID_ARG;
    if (p->child_ctx) ape_plan_destroy(p->child_ctx);
    if (p->child_oth) ape_plan_destroy(p->child_oth);
    if (p->d_blob || p->d_step) { DeviceGuard guard(p->h->device); if (p->d_blob) cudaFree(p->d_blob); if (p->d_step) cudaFree(p->d_step); }
    delete p;
    return APE_OK;
}

static int attend_plan_impl(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                            const ape_rows_t* out, float* lse, const ape_request_t* reqs, int32_t n_req, ape_mode_t mode,
                            int per_context, const int32_t* const* parent, const uint8_t* const* scaled, ape_plan_t* plan_out)
{
    if (!h || !plan_out) return APE_ERR_INVALID_ARG;
    *plan_out = nullptr;
    int G = 1; float c = 0.f;
    int rc = check_shape(shape, &G, &c);              if (rc) return rc;
    rc = check_pool(pool, shape);                     if (rc) return rc;
    rc = check_rows(q, shape);                        if (rc) return rc;
    rc = check_rows(out, shape);                      if (rc) return rc;
    rc = check_lse(lse);                              if (rc) return rc;
    if (!reqs || n_req <= 0) return APE_ERR_INVALID_ARG;
    if (mode != APE_PREFILL && mode != APE_DECODE) return APE_ERR_INVALID_ARG;
    if (out->n_rows < q->n_rows) return APE_ERR_INVALID_ARG;
    int64_t max_extra = INT64_MAX;
    for (int r = 0; r < n_req; ++r) {
        const ape_request_t& rq = reqs[r];
        if (rq.q_len < 1 || rq.q_start < 0 || rq.q_start + rq.q_len > q->n_rows) return APE_ERR_INVALID_ARG;
        if (mode == APE_DECODE && rq.q_len != 1) return APE_ERR_INVALID_ARG;
        if (rq.n_ctx < 0 || (rq.n_ctx > 0 && !rq.ctx)) return APE_ERR_INVALID_ARG;
        if (!span_ok(rq.prefix, pool->n_tokens) || !span_ok(rq.query_kv, pool->n_tokens)) return APE_ERR_INVALID_ARG;
        for (int i = 0; i < rq.n_ctx; ++i) if (!span_ok(rq.ctx[i], pool->n_tokens)) return APE_ERR_INVALID_ARG;
        if (rq.query_kv.len < rq.q_len) return APE_ERR_INVALID_ARG;
        if (rq.query_kv_capacity < rq.query_kv.len || rq.query_kv.start + rq.query_kv_capacity > pool->n_tokens) return APE_ERR_INVALID_ARG;
        max_extra = std::min(max_extra, rq.query_kv_capacity - rq.query_kv.len);
    }
    HostMeta m;
    std::vector<int> node_base(n_req, 0);
    if (per_context == 2) {
        // the trees: parent[i] < i keeps them acyclic; depth is bounded by what the merge kernel's stack holds
        if (!parent) return APE_ERR_INVALID_ARG;
        try {
            for (int r = 0; r < n_req; ++r) {
                const int n = reqs[r].n_ctx;
                if (n > 0 && !parent[r]) return APE_ERR_INVALID_ARG;
                node_base[r] = static_cast<int>(m.nodes.size());
                for (int i = 0; i < n; ++i) {
                    const int par = parent[r][i];
                    if (par < -1 || par >= i) return APE_ERR_INVALID_ARG;
                    DevNode nd;
                    nd.parent = par < 0 ? -1 : node_base[r] + par;
                    nd.depth = par < 0 ? 0 : m.nodes[node_base[r] + par].depth + 1;
                    if (nd.depth >= kMaxTreeDepth) return APE_ERR_INVALID_ARG;
                    nd.scaled = (scaled && scaled[r]) ? (scaled[r][i] ? 1 : 0) : (par < 0 ? 1 : 0);
                    nd.pad = 0;
                    m.nodes.push_back(nd);
                }
            }
        } catch (const std::bad_alloc&) {
            return APE_ERR_NOMEM;
        }
    }
    if (per_context == 1 && mode != APE_DECODE) {
        // Eq. 11-12 as a forest of depth 0: every context a marked top-level node (the prefill plan runs in two passes)
        try {
            for (int r = 0; r < n_req; ++r) {
                node_base[r] = static_cast<int>(m.nodes.size());
                for (int i = 0; i < reqs[r].n_ctx; ++i) m.nodes.push_back(DevNode{-1, 0, 1, 0});
            }
        } catch (const std::bad_alloc&) {
            return APE_ERR_NOMEM;
        }
    }
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;

    ape_plan_t p = new (std::nothrow) ape_plan_s();
    if (!p) return APE_ERR_NOMEM;
    p->h = h; p->kind = (mode == APE_DECODE) ? PLAN_DECODE : PLAN_PREFILL;
    p->shape = *shape; p->c = c; p->G = G; p->pool = *pool; p->q = *q; p->out = *out; p->lse = lse; p->per_context = per_context;
    p->max_kv_extra = (mode == APE_DECODE) ? max_extra : 0;
    p->n_req = n_req;
    const int D = shape->head_dim, H_kv = shape->n_kv_heads;

    std::vector<Run> runs;
    try {
        if (mode == APE_DECODE) {
            const int tile = kDecodeTile;
            p->n_sib = 1;
            m.merge.reserve(static_cast<size_t>(n_req) * H_kv);
            for (int r = 0; r < n_req; ++r) {
                const ape_request_t& rq = reqs[r];
                DevReq dr{static_cast<int32_t>(rq.q_start), 1, static_cast<int32_t>(rq.query_kv.len), 0};
                m.reqs.push_back(dr);
                const int o0 = static_cast<int>(m.tiles.size());
                add_span_tiles(m.tiles, rq.prefix.start, rq.prefix.len, tile, 0, 0);
                add_span_tiles(m.tiles, rq.query_kv.start, rq.query_kv.len, tile, TILE_GROWS, rq.query_kv_capacity);
                const int o1 = static_cast<int>(m.tiles.size());
                const auto ctx_ranges = (per_context == 2) ? add_tree_tiles(m.tiles, rq.ctx, parent[r], rq.n_ctx, tile, node_base[r])
                                                            : add_context_tiles(m.tiles, rq.ctx, rq.n_ctx, tile, per_context == 1);
                for (int hh = 0; hh < H_kv; ++hh) {
                    DevMerge g{r, hh, 0, 0, 0, 0, 0, 1};
                    const int mi = static_cast<int>(m.merge.size());
                    m.merge.push_back(g);
                    runs.push_back(Run{r, hh, 0, 1, SEG_OTHER, o0, o1, mi});
                    for (size_t ci = 0; ci < ctx_ranges.size(); ++ci)
                        runs.push_back(Run{r, hh, 0, 1, SEG_CTX, ctx_ranges[ci].t0, ctx_ranges[ci].t1, mi, ctx_ranges[ci].id});
                }
            }
            p->n_cta = h->n_sm;
            assign_stream(runs, p->n_cta, 1, m);
            p->n_slots = static_cast<int>(m.items.size());
            p->n_stages = decode_pick_stages(D, G, h->smem_optin - 2048);
            if (p->n_stages < 2) { delete p; return APE_ERR_SHAPE; }
            p->smem_bytes = decode_smem_bytes(D, G, p->n_stages);
            const size_t rows = static_cast<size_t>(p->n_slots) * G;
            p->ws_bytes = ((rows * D * 4 + 255) & ~size_t(255)) + ((rows * 2 * 4 + 255) & ~size_t(255));
            rc = make_map(h, &p->tm_k, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
            if (!rc) rc = make_map(h, &p->tm_v, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
            if (!rc && decode_set_smem_attr(D, p->smem_bytes) != cudaSuccess) rc = APE_ERR_CUDA;
            if (!rc) rc = setup_decode_step(p, reqs, n_req);
        } else {
            const int tile = kAttnTileN;
            const int TB = kAttnRows / G;                 // query tokens per row block
            int max_rb = 1;
            for (int r = 0; r < n_req; ++r) max_rb = std::max<int>(max_rb, static_cast<int>((reqs[r].q_len + TB - 1) / TB));
            p->n_sib = std::max(1, std::min({4, max_rb, h->n_sm}));
            const int n_groups = std::max(1, h->n_sm / p->n_sib);
            int64_t row_base = 0;                          // query rows of the requests before this one
            bool any_node_tiles = false;
            for (int r = 0; r < n_req; ++r) {
                const ape_request_t& rq = reqs[r];
                // (pad: the request's row base, which the two-pass plans index their per-node arrays with)
                DevReq dr{static_cast<int32_t>(rq.q_start), static_cast<int32_t>(rq.q_len), static_cast<int32_t>(rq.query_kv.len),
                          static_cast<int32_t>(row_base)};
                m.reqs.push_back(dr);
                m.req_node0.push_back(node_base[r]);
                p->max_nodes = std::max(p->max_nodes, rq.n_ctx);
                const int o0 = static_cast<int>(m.tiles.size());
                add_span_tiles(m.tiles, rq.prefix.start, rq.prefix.len, tile, 0, 0);
                add_span_tiles(m.tiles, rq.query_kv.start, rq.query_kv.len, tile, TILE_CAUSAL, 0);
                const int o1 = static_cast<int>(m.tiles.size());
                std::vector<CtxRange> ctx_ranges;
                if (per_context == 2) ctx_ranges = add_tree_tiles(m.tiles, rq.ctx, parent[r], rq.n_ctx, tile, node_base[r]);
                else if (per_context == 1) {
                    for (int i = 0; i < rq.n_ctx; ++i) {
                        if (rq.ctx[i].len <= 0) continue;
                        const int c0 = static_cast<int>(m.tiles.size());
                        add_span_tiles(m.tiles, rq.ctx[i].start, rq.ctx[i].len, tile, 0, 0);
                        ctx_ranges.push_back({c0, static_cast<int>(m.tiles.size()), node_base[r] + i});
                    }
                } else ctx_ranges = add_context_tiles(m.tiles, rq.ctx, rq.n_ctx, tile, false);
                if (per_context != 0 && !ctx_ranges.empty()) {
                    // Two passes instead of a partial per node: every context tile names its node (key_base is free, these
                    // tiles are not causal) and a node's last tile is marked; the context segment is then ONE run of tiles
                    // (the ranges follow each other in the tile list), as in the Eq. 5 plan, and long items stay long.
                    for (const auto& cr : ctx_ranges) {
                        for (int t = cr.t0; t < cr.t1; ++t) m.tiles[t].key_base = cr.id;
                        m.tiles[cr.t1 - 1].flags |= TILE_CTX_END;
                        m.nodes[cr.id].pad = 1;
                    }
                    ctx_ranges = {CtxRange{ctx_ranges.front().t0, ctx_ranges.back().t1, static_cast<int>(row_base)}};
                    any_node_tiles = true;
                }
                row_base += rq.q_len;
                p->max_rows = std::max<int>(p->max_rows, static_cast<int>(rq.q_len) * shape->n_q_heads);
                const int RB = static_cast<int>((rq.q_len + TB - 1) / TB);
                for (int hh = 0; hh < H_kv; ++hh) {
                    for (int rb0 = 0; rb0 < RB; rb0 += p->n_sib) {
                        const int live = std::min(p->n_sib, RB - rb0);
                        const int mi = static_cast<int>(m.merge.size());
                        for (int s = 0; s < live; ++s) m.merge.push_back(DevMerge{r, hh, rb0 + s, 0, 0, 0, 0, 1});
                        runs.push_back(Run{r, hh, rb0, live, SEG_OTHER, o0, o1, mi});
                        for (size_t ci = 0; ci < ctx_ranges.size(); ++ci)
                            runs.push_back(Run{r, hh, rb0, live, SEG_CTX, ctx_ranges[ci].t0, ctx_ranges[ci].t1, mi, ctx_ranges[ci].id});
                    }
                }
            }
            assign_stream(runs, n_groups, p->n_sib, m, per_context != 0);
            p->n_cta = n_groups * p->n_sib;
            p->n_slots = static_cast<int>(m.items.size()) * p->n_sib;
            p->smem_bytes = attn_smem_bytes(D, kAttnPrefill);
            const size_t rows = static_cast<size_t>(p->n_slots) * kAttnRows;
            p->ws_bytes = ((rows * D * 4 + 255) & ~size_t(255)) + ((rows * 2 * 4 + 255) & ~size_t(255));
            m.req_node0.push_back(static_cast<int32_t>(m.nodes.size()));
            if (per_context != 0 && any_node_tiles) {
                if (row_base * shape->n_q_heads >= (1ll << 31)) { delete p; return APE_ERR_LAYOUT; }
                p->two_pass = true;
                p->n_nodes = static_cast<int>(m.nodes.size());
                p->stat_rows = row_base * shape->n_q_heads;
                const size_t cells = static_cast<size_t>(p->n_nodes) * static_cast<size_t>(p->stat_rows);
                auto rnd = [](size_t x) { return (x + 255) & ~size_t(255); };
                p->off_stats = p->ws_bytes;
                p->off_mass = p->off_stats + rnd(cells * 8);
                p->off_bias = p->off_mass + rnd(cells * 4);
                p->ws_bytes = p->off_bias + rnd(cells * 4);
            }
            rc = make_map(h, &p->tm_k, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
            if (!rc) rc = make_map(h, &p->tm_v, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
            if (!rc) rc = make_map(h, &p->tm_q, q->data, D, shape->n_q_heads, q->n_rows, q->head_stride, q->token_stride, G, 128 / G);
            if (!rc && attn_set_smem_attr(D, kAttnPrefill, p->smem_bytes) != cudaSuccess) rc = APE_ERR_CUDA;
            if (!rc && p->two_pass && (attn_set_smem_attr(D, kAttnStats, p->smem_bytes) != cudaSuccess ||
                                       attn_set_smem_attr(D, kAttnBias, p->smem_bytes) != cudaSuccess)) rc = APE_ERR_CUDA;
        }
        if (!rc) { finish_items(m); rc = upload(p, m); }
    } catch (const std::bad_alloc&) {
        rc = APE_ERR_NOMEM;
    }
    if (rc) { ape_plan_destroy(p); return rc; }
    *plan_out = p;
    return APE_OK;
}

int ape_attend_plan(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                    const ape_rows_t* out, float* lse, const ape_request_t* reqs, int32_t n_req, ape_mode_t mode,
                    ape_plan_t* plan_out)
{
    return attend_plan_impl(h, shape, pool, q, out, lse, reqs, n_req, mode, 0, nullptr, nullptr, plan_out);
}

int ape_attend_plan_per_context(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                                const ape_rows_t* out, float* lse, const ape_request_t* reqs, int32_t n_req, ape_mode_t mode,
                                ape_plan_t* plan_out)
{
    return attend_plan_impl(h, shape, pool, q, out, lse, reqs, n_req, mode, 1, nullptr, nullptr, plan_out);
}

int ape_attend_plan_tree(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                         const ape_rows_t* out, float* lse, const ape_request_t* reqs, int32_t n_req,
                         const int32_t* const* parent, const uint8_t* const* scaled, ape_mode_t mode, ape_plan_t* plan_out)
{
    return attend_plan_impl(h, shape, pool, q, out, lse, reqs, n_req, mode, 2, parent, scaled, plan_out);
}

int ape_attend_plan_shared(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                           const ape_rows_t* out, float* lse, const ape_request_t* reqs, int32_t n_req, ape_plan_t* plan_out)
{
    if (!h || !plan_out) return APE_ERR_INVALID_ARG;
    *plan_out = nullptr;
    int G = 1; float c = 0.f;
    int rc = check_shape(shape, &G, &c);              if (rc) return rc;
    rc = check_pool(pool, shape);                     if (rc) return rc;
    rc = check_rows(q, shape);                        if (rc) return rc;
    rc = check_rows(out, shape);                      if (rc) return rc;
    rc = check_lse(lse);                              if (rc) return rc;
    if (!reqs || n_req <= 0 || out->n_rows < q->n_rows) return APE_ERR_INVALID_ARG;
    int64_t max_extra = INT64_MAX;
    std::vector<ape_span_t> shared_ctx;
    for (int r = 0; r < n_req; ++r) {
        const ape_request_t& rq = reqs[r];
        if (rq.q_len != 1 || rq.q_start != reqs[0].q_start + r || rq.q_start < 0 || rq.q_start + 1 > q->n_rows) return APE_ERR_INVALID_ARG;
        if (rq.n_ctx < 0 || (rq.n_ctx > 0 && !rq.ctx)) return APE_ERR_INVALID_ARG;
        if (!span_ok(rq.prefix, pool->n_tokens) || !span_ok(rq.query_kv, pool->n_tokens)) return APE_ERR_INVALID_ARG;
        for (int i = 0; i < rq.n_ctx; ++i) if (!span_ok(rq.ctx[i], pool->n_tokens)) return APE_ERR_INVALID_ARG;
        if (rq.query_kv.len < 1) return APE_ERR_INVALID_ARG;
        if (rq.query_kv_capacity < rq.query_kv.len || rq.query_kv.start + rq.query_kv_capacity > pool->n_tokens) return APE_ERR_INVALID_ARG;
        max_extra = std::min(max_extra, rq.query_kv_capacity - rq.query_kv.len);
        // the same context tokens for every request (Eq. 5 does not care how they are cut into contexts, or in which order)
        std::vector<ape_span_t> mine = fuse_spans(rq.ctx, rq.n_ctx);
        if (r == 0) shared_ctx = mine;
        else {
            if (mine.size() != shared_ctx.size()) return APE_ERR_INVALID_ARG;
            for (size_t i = 0; i < mine.size(); ++i)
                if (mine[i].start != shared_ctx[i].start || mine[i].len != shared_ctx[i].len) return APE_ERR_INVALID_ARG;
        }
    }
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    const int D = shape->head_dim, H_kv = shape->n_kv_heads;

    auto new_plan = [&](PlanKind kind) {
        ape_plan_t p = new (std::nothrow) ape_plan_s();
        if (p) { p->h = h; p->kind = kind; p->shape = *shape; p->c = c; p->G = G; p->pool = *pool; p->q = *q; p->out = *out; p->lse = lse; }
        return p;
    };
    ape_plan_t p = new_plan(PLAN_SHARED);
    if (!p) return APE_ERR_NOMEM;
    p->max_kv_extra = max_extra;
    p->child_ctx = new_plan(PLAN_PREFILL);
    p->child_oth = new_plan(PLAN_DECODE);
    if (!p->child_ctx || !p->child_oth) { ape_plan_destroy(p); return APE_ERR_NOMEM; }
    try {
        // ---- context pass: the requests' query rows are the "tokens" of one row-block sequence ------------------------
        ape_plan_t a = p->child_ctx;
        HostMeta ma;
        std::vector<Run> runs_a;
        // With at most 128 query rows in the batch a 256-row block would be half empty: the row block then has 128 rows,
        // both halves of a CTA hold them and take alternate tiles (two partials of 128 rows per slot).
        a->alt_halves = n_req * G <= kAttnRows / 2;
        const int TB = (a->alt_halves ? kAttnRows / 2 : kAttnRows) / G;
        const int RB = (n_req + TB - 1) / TB;
        a->n_sib = std::max(1, std::min({4, RB, h->n_sm}));
        const int n_groups = std::max(1, h->n_sm / a->n_sib);
        ma.reqs.push_back(DevReq{static_cast<int32_t>(reqs[0].q_start), n_req, n_req, 0});
        const int t0 = 0;
        for (const auto& sp : shared_ctx) add_span_tiles(ma.tiles, sp.start, sp.len, kAttnTileN, 0, 0);
        const int t1 = static_cast<int>(ma.tiles.size());
        for (int hh = 0; hh < H_kv; ++hh)
            for (int rb0 = 0; rb0 < RB; rb0 += a->n_sib) {
                const int live = std::min(a->n_sib, RB - rb0);
                const int mi = static_cast<int>(ma.merge.size());
                for (int sb = 0; sb < live; ++sb) ma.merge.push_back(DevMerge{0, hh, rb0 + sb, 0, 0, 0, 0, 1});
                if (t1 > t0) runs_a.push_back(Run{0, hh, rb0, live, SEG_CTX, t0, t1, mi});
            }
        assign_stream(runs_a, n_groups, a->n_sib, ma);
        a->n_cta = n_groups * a->n_sib;
        a->n_slots = static_cast<int>(ma.items.size()) * a->n_sib;
        a->smem_bytes = attn_smem_bytes(D, a->alt_halves ? kAttnAlt : kAttnPrefill);
        rc = make_map(h, &a->tm_k, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, kAttnTileN);
        if (!rc) rc = make_map(h, &a->tm_v, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, kAttnTileN);
        if (!rc) rc = make_map(h, &a->tm_q, q->data, D, shape->n_q_heads, q->n_rows, q->head_stride, q->token_stride, G, 128 / G);
        if (!rc && attn_set_smem_attr(D, a->alt_halves ? kAttnAlt : kAttnPrefill, a->smem_bytes) != cudaSuccess) rc = APE_ERR_CUDA;
        if (!rc) { finish_items(ma); rc = upload(a, ma); }

        // ---- the rest, per request: prefix + the request's own (growing) query segment ------------------------------
        ape_plan_t b = p->child_oth;
        HostMeta mb;
        std::vector<Run> runs_b;
        for (int r = 0; r < n_req && !rc; ++r) {
            const ape_request_t& rq = reqs[r];
            mb.reqs.push_back(DevReq{static_cast<int32_t>(rq.q_start), 1, static_cast<int32_t>(rq.query_kv.len), 0});
            const int o0 = static_cast<int>(mb.tiles.size());
            add_span_tiles(mb.tiles, rq.prefix.start, rq.prefix.len, kDecodeTile, 0, 0);
            add_span_tiles(mb.tiles, rq.query_kv.start, rq.query_kv.len, kDecodeTile, TILE_GROWS, rq.query_kv_capacity);
            const int o1 = static_cast<int>(mb.tiles.size());
            for (int hh = 0; hh < H_kv; ++hh) {
                const int mi = static_cast<int>(mb.merge.size());
                mb.merge.push_back(DevMerge{r, hh, 0, 0, 0, 0, 0, 1});
                runs_b.push_back(Run{r, hh, 0, 1, SEG_OTHER, o0, o1, mi});
            }
        }
        if (!rc) {
            b->n_sib = 1; b->n_cta = h->n_sm;
            assign_stream(runs_b, b->n_cta, 1, mb);
            b->n_slots = static_cast<int>(mb.items.size());
            b->n_stages = decode_pick_stages(D, G, h->smem_optin - 2048);
            if (b->n_stages < 2) rc = APE_ERR_SHAPE;
        }
        if (!rc) {
            b->smem_bytes = decode_smem_bytes(D, G, b->n_stages);
            rc = make_map(h, &b->tm_k, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, kDecodeTile);
            if (!rc) rc = make_map(h, &b->tm_v, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, kDecodeTile);
            if (!rc && decode_set_smem_attr(D, b->smem_bytes) != cudaSuccess) rc = APE_ERR_CUDA;
            if (!rc) { finish_items(mb); rc = upload(b, mb); }
        }

        // ---- merge records of the whole plan: context partials from the first pass, the rest from the second -----------
        if (!rc) {
            HostMeta mp;
            mp.reqs = mb.reqs;
            for (int r = 0; r < n_req; ++r)
                for (int hh = 0; hh < H_kv; ++hh) {
                    const DevMerge& ga = ma.merge[static_cast<size_t>(hh) * RB + r / TB];
                    const DevMerge& gb = mb.merge[static_cast<size_t>(r) * H_kv + hh];
                    DevMerge g{r, hh, 0, ga.ctx_slot0, ga.ctx_n, gb.oth_slot0, gb.oth_n, std::max(1, gb.slot_stride)};
                    g.ctx_row_off = (r % TB) * G;
                    g.ctx_stride = ga.ctx_stride;
                    if (a->alt_halves) {
                        // one row block, one sibling: the items' slots are consecutive, and in units of 128 rows the two
                        // partials of slot s are 2 s (half 0) and 2 s + 1 (half 1)
                        g.ctx_slot0 = 2 * ga.ctx_slot0; g.ctx_n = 2 * ga.ctx_n; g.ctx_stride = 1;
                    }
                    mp.merge.push_back(g);
                }
            rc = upload(p, mp);
            if (!rc) rc = setup_decode_step(p, reqs, n_req);
            auto rnd = [](size_t x) { return (x + 255) & ~size_t(255); };
            const size_t rows_a = static_cast<size_t>(a->n_slots) * kAttnRows, rows_b = static_cast<size_t>(b->n_slots) * G;
            a->ws_bytes = rnd(rows_a * D * 4) + rnd(rows_a * 2 * 4);
            b->ws_bytes = rnd(rows_b * D * 4) + rnd(rows_b * 2 * 4);
            p->ws_bytes = a->ws_bytes + b->ws_bytes;
        }
    } catch (const std::bad_alloc&) {
        rc = APE_ERR_NOMEM;
    }
    if (rc) { ape_plan_destroy(p); return rc; }
    *plan_out = p;
    return APE_OK;
}

int ape_encode_plan(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                    const ape_rows_t* out, float* lse, const ape_span_t* prefix, const ape_span_t* ctx, int32_t n_ctx,
                    ape_plan_t* plan_out)
{
    if (!h || !plan_out) return APE_ERR_INVALID_ARG;
    *plan_out = nullptr;
    int G = 1; float c = 0.f;
    int rc = check_shape(shape, &G, &c);              if (rc) return rc;
    rc = check_pool(pool, shape);                     if (rc) return rc;
    rc = check_rows(q, shape);                        if (rc) return rc;
    rc = check_rows(out, shape);                      if (rc) return rc;
    rc = check_lse(lse);                              if (rc) return rc;
    if (!prefix || n_ctx < 0 || (n_ctx > 0 && !ctx)) return APE_ERR_INVALID_ARG;
    if (!span_ok(*prefix, pool->n_tokens)) return APE_ERR_INVALID_ARG;
    for (int i = 0; i < n_ctx; ++i) {
        if (!span_ok(ctx[i], pool->n_tokens)) return APE_ERR_INVALID_ARG;
        if (ctx[i].start + ctx[i].len > q->n_rows || ctx[i].start + ctx[i].len > out->n_rows) return APE_ERR_INVALID_ARG;
    }
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;

    ape_plan_t p = new (std::nothrow) ape_plan_s();
    if (!p) return APE_ERR_NOMEM;
    p->h = h; p->kind = PLAN_ENCODE; p->shape = *shape; p->c = c; p->G = G; p->pool = *pool; p->q = *q; p->out = *out; p->lse = lse;
    p->n_sib = 1;
    const int D = shape->head_dim, H_kv = shape->n_kv_heads, tile = kAttnTileN, TB = kAttnRows / G;

    // A prefix that ends inside a tile shares that tile with the head of each context (when the tail is a multiple of 8 rows,
    // which the 128-byte swizzle of the copy engine asks for): with a 64-token prefix and 256-token contexts that is 8
    // tiles per context instead of 10.
    const int split_r = (prefix->len % tile != 0 && (prefix->len % tile) % 8 == 0 && n_ctx > 0) ? static_cast<int>(prefix->len % tile) : 0;
    p->split_r = split_r;
    HostMeta m;
    try {
        // The row blocks of one (context, KV head) read the same K/V tiles: a pair's row blocks go to ONE CTA, back to back
        // (the longest, which touches every tile of the context, first), so the tiles come from HBM once and from L2 for the
        // other row blocks.  Whole pairs are dealt out while every CTA gets the same number; the rest goes item by item.
        struct Work { DevItem it; long long cost; };
        struct Pair { std::vector<Work> rows; long long cost; };
        std::vector<Pair> pairs;
        for (int i = 0; i < n_ctx; ++i) {
            DevReq dr{static_cast<int32_t>(ctx[i].start), static_cast<int32_t>(ctx[i].len), static_cast<int32_t>(ctx[i].len), 0};
            m.reqs.push_back(dr);
            if (ctx[i].len == 0) continue;
            const int t0 = static_cast<int>(m.tiles.size());
            int n_pref, head = 0;                     // head: context tokens that share a tile with the prefix tail
            if (split_r > 0) {
                // whole prefix tiles, then ONE tile = [prefix tail | first 128 - split_r context tokens], then the rest of
                // the context in whole tiles: no tile slot is spent on padding between prefix and context
                add_span_tiles(m.tiles, prefix->start, prefix->len - split_r, tile, 0, 0);
                head = static_cast<int>(std::min<int64_t>(tile - split_r, ctx[i].len));
                DevTile mt;
                mt.tok = static_cast<int32_t>(prefix->start + prefix->len - split_r);
                mt.n_valid = split_r + head; mt.key_base = -split_r; mt.flags = TILE_CAUSAL | TILE_SPLIT;
                m.tiles.push_back(mt);
                n_pref = static_cast<int>(m.tiles.size()) - t0;
                for (int64_t off = tile - split_r; off < ctx[i].len; off += tile) {
                    DevTile t;
                    t.tok = static_cast<int32_t>(ctx[i].start + off);
                    t.n_valid = static_cast<int32_t>(std::min<int64_t>(tile, ctx[i].len - off));
                    t.key_base = static_cast<int32_t>(off); t.flags = TILE_CAUSAL;
                    m.tiles.push_back(t);
                }
            } else {
                add_span_tiles(m.tiles, prefix->start, prefix->len, tile, 0, 0);
                n_pref = static_cast<int>(m.tiles.size()) - t0;
                add_span_tiles(m.tiles, ctx[i].start, ctx[i].len, tile, TILE_CAUSAL, 0);
            }
            const int t1 = static_cast<int>(m.tiles.size());
            const int RB = static_cast<int>((ctx[i].len + TB - 1) / TB);
            for (int hh = 0; hh < H_kv; ++hh) {
                Pair pr; pr.cost = 0;
                for (int rb = RB - 1; rb >= 0; --rb) {
                    const int64_t last_tok = std::min<int64_t>(ctx[i].len, static_cast<int64_t>(rb + 1) * TB) - 1;
                    // tiles this row block can see: the prefix tiles and every context tile whose first key is not past last_tok
                    const int vis = (split_r > 0)
                        ? n_pref + ((last_tok >= tile - split_r) ? static_cast<int>((last_tok - (tile - split_r)) / tile) + 1 : 0)
                        : n_pref + static_cast<int>(last_tok / tile) + 1;
                    DevItem it{};
                    it.req = i; it.kv_head = hh; it.row_block = rb; it.tile_begin = t0; it.tile_end = std::min(t1, t0 + vis);
                    it.slot = 0; it.seg = SEG_FINAL; it.n_sib = 1;
                    pr.rows.push_back(Work{it, vis}); pr.cost += vis;
                }
                pairs.push_back(std::move(pr));
            }
        }
        size_t n_items = 0;
        for (auto& pr : pairs) n_items += pr.rows.size();
        p->n_cta = std::max(1, std::min<int>(h->n_sm, static_cast<int>(n_items)));
        std::vector<std::vector<DevItem>> bins(p->n_cta);
        std::vector<long long> load(p->n_cta, 0);
        auto least = [&]() { return static_cast<int>(std::min_element(load.begin(), load.end()) - load.begin()); };
        std::stable_sort(pairs.begin(), pairs.end(), [](const Pair& a, const Pair& b) { return a.cost > b.cost; });
        const size_t whole = pairs.size() / p->n_cta * p->n_cta;      // pairs dealt out whole, longest first
        for (size_t i = 0; i < whole; ++i) {
            const int b = least();
            for (auto& w : pairs[i].rows) bins[b].push_back(w.it);
            load[b] += pairs[i].cost;
        }
        std::vector<Work> rest;
        for (size_t i = whole; i < pairs.size(); ++i) for (auto& w : pairs[i].rows) rest.push_back(w);
        std::stable_sort(rest.begin(), rest.end(), [](const Work& a, const Work& b) { return a.cost > b.cost; });
        for (auto& w : rest) { const int b = least(); bins[b].push_back(w.it); load[b] += w.cost; }
        m.cta_begin.push_back(0);
        for (auto& b : bins) { for (auto& it : b) m.items.push_back(it); m.cta_begin.push_back(static_cast<int32_t>(m.items.size())); }
        p->n_slots = 0;
        p->ws_bytes = 0;
        p->smem_bytes = attn_smem_bytes(D, kAttnEncode);
        rc = make_map(h, &p->tm_k, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
        if (!rc) rc = make_map(h, &p->tm_v, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
        if (!rc) rc = make_map(h, &p->tm_q, q->data, D, shape->n_q_heads, q->n_rows, q->head_stride, q->token_stride, G, 128 / G);
        if (!rc && split_r > 0) {
            rc = make_map(h, &p->tm_split.ka, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, split_r);
            if (!rc) rc = make_map(h, &p->tm_split.kb, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile - split_r);
            if (!rc) rc = make_map(h, &p->tm_split.va, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, split_r);
            if (!rc) rc = make_map(h, &p->tm_split.vb, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile - split_r);
        }
        // Every item of this plan has a row block of its own, so a finished row block may leave through its Q buffer.
        if (!rc) p->o_via_tma = make_map(h, &p->tm_o, out->data, D, shape->n_q_heads, out->n_rows, out->head_stride, out->token_stride,
                                         G, 128 / G) == APE_OK;
        if (!rc && attn_set_smem_attr(D, kAttnEncode, p->smem_bytes) != cudaSuccess) rc = APE_ERR_CUDA;
        if (!rc) { finish_items(m); rc = upload(p, m); }
    } catch (const std::bad_alloc&) {
        rc = APE_ERR_NOMEM;
    }
    if (rc) { ape_plan_destroy(p); return rc; }
    *plan_out = p;
    return APE_OK;
}

int ape_rope_runs_for_request(const ape_request_t* rq, int64_t src_start, ape_rope_run_t* runs, int32_t capacity, int32_t* n_runs) {
    if (!rq || !runs || !n_runs || src_start < 0 || rq->n_ctx < 0 || (rq->n_ctx > 0 && !rq->ctx)) return APE_ERR_INVALID_ARG;
    if (capacity < rq->n_ctx + 2) return APE_ERR_INVALID_ARG;
    if (rq->prefix.len < 0 || rq->prefix.start < 0 || rq->query_kv.len < 0 || rq->query_kv.start < 0) return APE_ERR_INVALID_ARG;
    int64_t src = src_start, longest = 0;
    int n = 0;
    runs[n++] = ape_rope_run_t{src, rq->prefix.start, rq->prefix.len, 0};
    src += rq->prefix.len;
    for (int i = 0; i < rq->n_ctx; ++i) {
        if (rq->ctx[i].len < 0 || rq->ctx[i].start < 0) return APE_ERR_INVALID_ARG;
        runs[n++] = ape_rope_run_t{src, rq->ctx[i].start, rq->ctx[i].len, rq->prefix.len};   // every context starts after the prefix
        src += rq->ctx[i].len;
        longest = std::max(longest, rq->ctx[i].len);
    }
    runs[n++] = ape_rope_run_t{src, rq->query_kv.start, rq->query_kv.len, rq->prefix.len + longest};
    *n_runs = n;
    return APE_OK;
}

int ape_rope_plan(ape_handle_t h, int32_t head_dim, double theta, const ape_rope_run_t* runs, int32_t n_runs, ape_plan_t* plan_out) {
    if (!h || !plan_out || n_runs < 0 || (n_runs > 0 && !runs)) return APE_ERR_INVALID_ARG;
    *plan_out = nullptr;
    if (head_dim != 64 && head_dim != 128) return APE_ERR_SHAPE;
    if (!(theta > 1.0) || !std::isfinite(theta)) return APE_ERR_RANGE;
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    int rc = APE_OK;
    ape_plan_t p = new (std::nothrow) ape_plan_s();
    if (!p) return APE_ERR_NOMEM;
    p->h = h; p->kind = PLAN_ROPE; p->shape.head_dim = head_dim; p->rope_log2_theta = std::log2(theta);
    try {
        std::vector<RopeChunk> chunks;
        constexpr int64_t kMaxRow = (1ll << 31) - 1;
        for (int r = 0; r < n_runs && !rc; ++r) {
            const ape_rope_run_t& run = runs[r];
            if (run.len < 0 || run.src_start < 0 || run.dst_start < 0 || run.pos0 < 0) { rc = APE_ERR_INVALID_ARG; break; }
            if (run.src_start + run.len > kMaxRow || run.dst_start + run.len > kMaxRow || run.pos0 + run.len > kMaxRow) { rc = APE_ERR_LAYOUT; break; }
            p->rope_src_rows = std::max(p->rope_src_rows, run.len ? run.src_start + run.len : 0);
            p->rope_dst_rows = std::max(p->rope_dst_rows, run.len ? run.dst_start + run.len : 0);
            for (int64_t off = 0; off < run.len; off += kRopeChunkTokens) {
                RopeChunk c;
                c.src_tok = static_cast<int32_t>(run.src_start + off); c.dst_tok = static_cast<int32_t>(run.dst_start + off);
                c.n_tok = static_cast<int32_t>(std::min<int64_t>(kRopeChunkTokens, run.len - off));
                c.pos0 = static_cast<int32_t>(run.pos0 + off);
                chunks.push_back(c);
            }
        }
        p->n_rope_chunks = static_cast<int>(chunks.size());
        if (!rc && !chunks.empty()) {
            if (cudaMalloc(&p->d_blob, chunks.size() * sizeof(RopeChunk)) != cudaSuccess) rc = APE_ERR_NOMEM;
            else if (cudaMemcpy(p->d_blob, chunks.data(), chunks.size() * sizeof(RopeChunk), cudaMemcpyHostToDevice) != cudaSuccess) rc = APE_ERR_CUDA;
            p->d_rope_chunks = static_cast<RopeChunk*>(p->d_blob);
        }
    } catch (const std::bad_alloc&) {
        rc = APE_ERR_NOMEM;
    }
    if (rc) { ape_plan_destroy(p); return rc; }
    *plan_out = p;
    return APE_OK;
}

int ape_rope_write(ape_plan_t p, const ape_rows_t* src, const ape_rows_t* dst, int32_t n_heads, int32_t rotate, void* stream_v) {
    if (!p || !src || !dst || !src->data || !dst->data || n_heads <= 0) return APE_ERR_INVALID_ARG;
    if (p->kind != PLAN_ROPE) return APE_ERR_MODE;
    const int D = p->shape.head_dim;
    for (const ape_rows_t* r : {src, dst}) {
        if (!aligned16(r->data) || r->head_stride % 8 || r->token_stride % 8) return APE_ERR_ALIGN;
        if (r->head_stride < D || r->token_stride < static_cast<int64_t>(n_heads - 1) * r->head_stride + D) return APE_ERR_INVALID_ARG;
    }
    if (p->rope_src_rows > src->n_rows || p->rope_dst_rows > dst->n_rows) return APE_ERR_INVALID_ARG;
    DeviceGuard guard(p->h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    p->last_launches = 0;
    if (p->n_rope_chunks == 0) return APE_OK;
    RopeParams rp;
    rp.chunks = p->d_rope_chunks; rp.n_chunks = p->n_rope_chunks;
    rp.src.data = static_cast<const __nv_bfloat16*>(src->data); rp.src.token_stride = src->token_stride; rp.src.head_stride = src->head_stride;
    rp.dst = rows_desc(*dst);
    rp.n_heads = n_heads; rp.rotate = rotate ? 1 : 0; rp.log2_theta = p->rope_log2_theta;
    const int n_cta = std::max(1, std::min(p->n_rope_chunks, p->h->n_sm * 8));
    if (launch_rope(D, rp, n_cta, static_cast<cudaStream_t>(stream_v)) != cudaSuccess) return APE_ERR_CUDA;
    p->last_launches = 1;
    return APE_OK;
}

int ape_plan_workspace_bytes(ape_plan_t p, size_t* bytes) {
    if (!p || !bytes) return APE_ERR_INVALID_ARG;
    *bytes = p->ws_bytes;
    return APE_OK;
}

int ape_plan_last_launches(ape_plan_t p, int32_t* n) {
    if (!p || !n) return APE_ERR_INVALID_ARG;
    *n = p->last_launches;
    return APE_OK;
}

static int attend_impl(ape_plan_t p, float T, float S, int64_t kv_extra, void* workspace, size_t ws_bytes, void* stream_v,
                       const ape_partials_t* part) {
    if (!p) return APE_ERR_INVALID_ARG;
    if (part && (!part->o_ctx || !part->lse_ctx || !part->o_oth || !part->lse_oth)) return APE_ERR_INVALID_ARG;
    if (part && p->per_context) return APE_ERR_MODE;
    if (p->kind != PLAN_PREFILL && p->kind != PLAN_DECODE && p->kind != PLAN_SHARED) return APE_ERR_MODE;
    if (!(T > 0.f) || !(S > 0.f) || !std::isfinite(T) || !std::isfinite(S)) return APE_ERR_RANGE;
    if (kv_extra < 0 || kv_extra > p->max_kv_extra) return APE_ERR_RANGE;
    if (p->ws_bytes > 0 && (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || ws_bytes < p->ws_bytes)) return APE_ERR_WORKSPACE;
    DeviceGuard guard(p->h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int D = p->shape.head_dim, G = p->G;
    constexpr float kLog2e = 1.4426950408889634f;
    if (p->kind == PLAN_SHARED) {
        // context pass of all requests at once, the per-request rest, then one merge that reads both sets of partials
        ape_plan_t a = p->child_ctx, b = p->child_oth;
        auto rnd = [](size_t x) { return (x + 255) & ~size_t(255); };
        const size_t rows_a = static_cast<size_t>(a->n_slots) * kAttnRows, rows_b = static_cast<size_t>(b->n_slots) * G;
        uint8_t* base = static_cast<uint8_t*>(workspace);
        float* a_o = reinterpret_cast<float*>(base);
        float* a_ml = reinterpret_cast<float*>(base + rnd(rows_a * D * 4));
        float* b_o = reinterpret_cast<float*>(base + a->ws_bytes);
        float* b_ml = reinterpret_cast<float*>(base + a->ws_bytes + rnd(rows_b * D * 4));
        p->last_launches = 0;
        if (a->n_items > 0) {
            AttnParams ap;
            ap.tiles = a->d_tiles; ap.items = a->d_items; ap.cta_item_begin = a->d_cta_begin; ap.reqs = a->d_reqs;
            ap.out = rows_desc(p->out); ap.lse_out = nullptr; ap.ws_o = a_o; ap.ws_ml = a_ml;
            ap.scale_oth_log2 = p->c * kLog2e; ap.scale_ctx_log2 = p->c / T * kLog2e;
            ap.G = G; ap.H_q = p->shape.n_q_heads; ap.n_sib = a->n_sib; ap.mode = kAttnPrefill; ap.q_rows_are_pool = 0; ap.status = p->h->d_status;
            ap.o_via_tma = 0; ap.split_r = 0; ap.stats = nullptr; ap.bias = nullptr; ap.stat_rows = 0; if (a->alt_halves) ap.mode = kAttnAlt;
            if (launch_attn(D, a->tm_q, a->tm_k, a->tm_v, a->tm_q, a->tm_split, ap, a->n_cta, a->smem_bytes, stream) != cudaSuccess) return APE_ERR_CUDA;
            p->last_launches++;
        }
        DecodeParams dp;
        dp.tiles = b->d_tiles; dp.items = b->d_items; dp.cta_item_begin = b->d_cta_begin; dp.reqs = b->d_reqs;
        dp.q = rows_desc(p->q); dp.ws_o = b_o; dp.ws_ml = b_ml;
        dp.scale_oth_log2 = p->c * kLog2e; dp.scale_ctx_log2 = p->c / T * kLog2e;
        dp.kv_extra = static_cast<int32_t>(kv_extra); dp.G = G; dp.n_stages = b->n_stages; dp.status = p->h->d_status;
        if (launch_decode(D, b->tm_k, b->tm_v, dp, b->n_cta, b->smem_bytes, stream) != cudaSuccess) return APE_ERR_CUDA;
        p->last_launches++;
        MergeParams mp;
        mp.groups = p->d_merge; mp.reqs = p->d_reqs; mp.items = nullptr; mp.per_context = 0; mp.nodes = nullptr; mp.n_groups = p->n_merge;
        mp.rows_per_slot = G; mp.tokens_per_block = 1; mp.ws_o = b_o; mp.ws_ml = b_ml;
        mp.ws_o_ctx = a_o; mp.ws_ml_ctx = a_ml; mp.rows_per_slot_ctx = a->alt_halves ? kAttnRows / 2 : kAttnRows;
        mp.out = rows_desc(p->out); mp.lse_out = p->lse; mp.S = S; mp.G = G; mp.H_q = p->shape.n_q_heads; mp.D = D;
        mp.part_o_ctx = part ? part->o_ctx : nullptr; mp.part_lse_ctx = part ? part->lse_ctx : nullptr;
        mp.part_o_oth = part ? part->o_oth : nullptr; mp.part_lse_oth = part ? part->lse_oth : nullptr;
        if (launch_merge(mp, stream) != cudaSuccess) return APE_ERR_CUDA;
        p->last_launches++;
        return APE_OK;
    }
    const int rows_per_slot = (p->kind == PLAN_DECODE) ? G : kAttnRows;
    const size_t rows = static_cast<size_t>(p->n_slots) * rows_per_slot;
    float* ws_o = static_cast<float*>(workspace);
    float* ws_ml = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + ((rows * D * 4 + 255) & ~size_t(255)));
    p->last_launches = 0;

    if (p->kind == PLAN_DECODE) {
        DecodeParams dp;
        dp.tiles = p->d_tiles; dp.items = p->d_items; dp.cta_item_begin = p->d_cta_begin; dp.reqs = p->d_reqs;
        dp.q = rows_desc(p->q); dp.ws_o = ws_o; dp.ws_ml = ws_ml;
        dp.scale_oth_log2 = p->c * kLog2e; dp.scale_ctx_log2 = p->c / T * kLog2e;
        dp.kv_extra = static_cast<int32_t>(kv_extra); dp.G = G; dp.n_stages = p->n_stages; dp.status = p->h->d_status;
        if (launch_decode(D, p->tm_k, p->tm_v, dp, p->n_cta, p->smem_bytes, stream) != cudaSuccess) return APE_ERR_CUDA;
    } else {
        AttnParams ap;
        ap.tiles = p->d_tiles; ap.items = p->d_items; ap.cta_item_begin = p->d_cta_begin; ap.reqs = p->d_reqs;
        ap.out = rows_desc(p->out); ap.lse_out = nullptr; ap.ws_o = ws_o; ap.ws_ml = ws_ml;
        ap.scale_oth_log2 = p->c * kLog2e; ap.scale_ctx_log2 = p->c / T * kLog2e;
        ap.G = G; ap.H_q = p->shape.n_q_heads; ap.n_sib = p->n_sib; ap.mode = kAttnPrefill; ap.q_rows_are_pool = 0; ap.status = p->h->d_status;
        ap.o_via_tma = 0; ap.split_r = 0; ap.stats = nullptr; ap.bias = nullptr; ap.stat_rows = 0;
        if (p->two_pass) {
            // per-context form / context trees: (1) every node's own (maximum, sum) per row, (2) per-row, per-node biases
            // from them and S, (3) the prefill with the biases on the context logits; the merge below then sees an
            // ordinary context segment whose scaling has been applied already
            uint8_t* base = static_cast<uint8_t*>(workspace);
            ap.stat_rows = p->stat_rows;
            ap.mode = kAttnStats; ap.stats = reinterpret_cast<float2*>(base + p->off_stats);
            if (launch_attn(D, p->tm_q, p->tm_k, p->tm_v, p->tm_q, p->tm_split, ap, p->n_cta, p->smem_bytes, stream) != cudaSuccess) return APE_ERR_CUDA;
            NodeBiasParams nb;
            nb.nodes = p->d_nodes; nb.reqs = p->d_reqs; nb.req_node0 = p->d_req_node0; nb.n_req = static_cast<int32_t>(p->n_req);
            nb.stats = ap.stats; nb.mass = reinterpret_cast<float*>(base + p->off_mass); nb.bias = reinterpret_cast<float*>(base + p->off_bias);
            nb.stat_rows = p->stat_rows; nb.S = S; nb.H_q = p->shape.n_q_heads; nb.max_rows = p->max_rows;
            nb.max_nodes = p->max_nodes; nb.smem_limit = p->h->smem_optin;
            if (launch_node_bias(nb, stream) != cudaSuccess) return APE_ERR_CUDA;
            ap.mode = kAttnBias; ap.stats = nullptr; ap.bias = nb.bias;
            p->last_launches += 2;
        }
        if (launch_attn(D, p->tm_q, p->tm_k, p->tm_v, p->tm_q, p->tm_split, ap, p->n_cta, p->smem_bytes, stream) != cudaSuccess) return APE_ERR_CUDA;
    }
    p->last_launches++;

    MergeParams mp;
    mp.groups = p->d_merge; mp.reqs = p->d_reqs; mp.items = p->d_items; mp.per_context = p->two_pass ? 0 : p->per_context; mp.nodes = p->d_nodes; mp.n_groups = p->n_merge; mp.rows_per_slot = rows_per_slot;
    mp.tokens_per_block = rows_per_slot / G; mp.ws_o = ws_o; mp.ws_ml = ws_ml; mp.out = rows_desc(p->out); mp.lse_out = p->lse;
    mp.ws_o_ctx = ws_o; mp.ws_ml_ctx = ws_ml; mp.rows_per_slot_ctx = rows_per_slot;
    mp.S = p->two_pass ? 1.f : S; mp.G = G; mp.H_q = p->shape.n_q_heads; mp.D = D;
    mp.part_o_ctx = part ? part->o_ctx : nullptr; mp.part_lse_ctx = part ? part->lse_ctx : nullptr;
    mp.part_o_oth = part ? part->o_oth : nullptr; mp.part_lse_oth = part ? part->lse_oth : nullptr;
    if (launch_merge(mp, stream) != cudaSuccess) return APE_ERR_CUDA;
    p->last_launches++;
    return APE_OK;
}

int ape_attend(ape_plan_t p, float T, float S, int64_t kv_extra, void* workspace, size_t ws_bytes, void* stream_v) {
    return attend_impl(p, T, S, kv_extra, workspace, ws_bytes, stream_v, nullptr);
}

int ape_attend_once(ape_handle_t h, const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q,
                    const ape_rows_t* out, float* lse, const ape_request_t* reqs, int32_t n_req, ape_mode_t mode, float T, float S,
                    void* stream_v) {
    ape_plan_t plan = nullptr;
    int rc = ape_attend_plan(h, shape, pool, q, out, lse, reqs, n_req, mode, &plan);
    if (rc) return rc;
    DeviceGuard guard(h->device);
    void* ws = nullptr;
    if (!guard.ok) rc = APE_ERR_CUDA;
    if (!rc && plan->ws_bytes > 0 && cudaMalloc(&ws, plan->ws_bytes) != cudaSuccess) { ws = nullptr; rc = APE_ERR_NOMEM; }
    if (!rc) rc = ape_attend(plan, T, S, 0, ws, plan->ws_bytes, stream_v);
    if (!rc && cudaStreamSynchronize(static_cast<cudaStream_t>(stream_v)) != cudaSuccess) rc = APE_ERR_CUDA;
    if (ws) cudaFree(ws);
    ape_plan_destroy(plan);
    return rc;
}

int ape_attend_partial(ape_plan_t p, float T, int64_t kv_extra, void* workspace, size_t ws_bytes, const ape_partials_t* part,
                       void* stream_v) {
    if (!part) return APE_ERR_INVALID_ARG;
    return attend_impl(p, T, 1.0f, kv_extra, workspace, ws_bytes, stream_v, part);
}

int ape_merge_shards(ape_handle_t h, const ape_shape_t* shape, int64_t n_rows, int32_t n_shards, const float* o_ctx_all,
                     const float* lse_ctx_all, const float* o_oth, const float* lse_oth, float S, const ape_rows_t* out,
                     float* lse, void* stream_v) {
    if (!h || !o_ctx_all || !lse_ctx_all || !o_oth || !lse_oth || n_rows <= 0 || n_shards <= 0) return APE_ERR_INVALID_ARG;
    int G = 1; float c = 0.f;
    int rc = check_shape(shape, &G, &c);              if (rc) return rc;
    rc = check_rows(out, shape);                      if (rc) return rc;
    if (out->n_rows < n_rows) return APE_ERR_INVALID_ARG;
    rc = check_lse(lse);                              if (rc) return rc;
    if (!(S > 0.f) || !std::isfinite(S)) return APE_ERR_RANGE;
    for (const void* ptr : {static_cast<const void*>(o_ctx_all), static_cast<const void*>(o_oth)}) if (!aligned16(ptr)) return APE_ERR_ALIGN;
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    ShardMergeParams sp;
    sp.o_ctx = o_ctx_all; sp.lse_ctx = lse_ctx_all; sp.o_oth = o_oth; sp.lse_oth = lse_oth; sp.n_shards = n_shards; sp.n_rows = n_rows;
    sp.out = rows_desc(*out); sp.lse_out = lse; sp.S = S; sp.H_q = shape->n_q_heads; sp.D = shape->head_dim;
    return launch_shard_merge(sp, static_cast<cudaStream_t>(stream_v)) == cudaSuccess ? APE_OK : APE_ERR_CUDA;
}

int ape_encode_contexts(ape_plan_t p, void* workspace, size_t ws_bytes, void* stream_v) {
    (void)workspace; (void)ws_bytes;
    if (!p) return APE_ERR_INVALID_ARG;
    if (p->kind != PLAN_ENCODE) return APE_ERR_MODE;
    DeviceGuard guard(p->h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    p->last_launches = 0;
    if (p->n_items == 0) return APE_OK;
    constexpr float kLog2e = 1.4426950408889634f;
    AttnParams ap;
    ap.tiles = p->d_tiles; ap.items = p->d_items; ap.cta_item_begin = p->d_cta_begin; ap.reqs = p->d_reqs;
    ap.out = rows_desc(p->out); ap.lse_out = p->lse; ap.ws_o = nullptr; ap.ws_ml = nullptr;
    ap.scale_oth_log2 = p->c * kLog2e; ap.scale_ctx_log2 = p->c * kLog2e;
    ap.G = p->G; ap.H_q = p->shape.n_q_heads; ap.n_sib = 1; ap.mode = kAttnEncode; ap.q_rows_are_pool = 1; ap.status = p->h->d_status;
    ap.o_via_tma = p->o_via_tma ? 1 : 0; ap.split_r = p->split_r; ap.stats = nullptr; ap.bias = nullptr; ap.stat_rows = 0;
    if (launch_attn(p->shape.head_dim, p->tm_q, p->tm_k, p->tm_v, p->tm_o, p->tm_split, ap, p->n_cta, p->smem_bytes,
                    static_cast<cudaStream_t>(stream_v)) != cudaSuccess) return APE_ERR_CUDA;
    p->last_launches = 1;
    return APE_OK;
}

int ape_attend_host(ape_plan_t p, float T, float S, int64_t kv_extra, void* workspace, size_t ws_bytes,
                    const void* h_q, const void* h_k, const void* h_v, void* h_out,
                    size_t* h2d_bytes, size_t* d2h_bytes, void* stream_v) {
    if (!p || !h_q || !h_k || !h_v || !h_out) return APE_ERR_INVALID_ARG;
    if (p->kind != PLAN_PREFILL && p->kind != PLAN_DECODE) return APE_ERR_MODE;
    DeviceGuard guard(p->h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    int rc = APE_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t qb = static_cast<size_t>(p->q.n_rows) * p->q.token_stride * 2;
    const size_t kb = static_cast<size_t>(p->pool.n_tokens) * p->pool.token_stride * 2;
    const size_t ob = static_cast<size_t>(p->q.n_rows) * p->out.token_stride * 2;
    if (cudaMemcpyAsync(p->q.data, h_q, qb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
    if (cudaMemcpyAsync(const_cast<void*>(p->pool.k), h_k, kb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
    if (cudaMemcpyAsync(const_cast<void*>(p->pool.v), h_v, kb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
    rc = ape_attend(p, T, S, kv_extra, workspace, ws_bytes, stream_v);
    if (rc) return rc;
    if (cudaMemcpyAsync(h_out, p->out.data, ob, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return APE_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return APE_ERR_CUDA;
    if (h2d_bytes) *h2d_bytes = qb + 2 * kb;
    if (d2h_bytes) *d2h_bytes = ob;
    return APE_OK;
}

int ape_decode_step_host(ape_plan_t p, float T, float S, int64_t kv_extra, void* workspace, size_t ws_bytes,
                         const void* h_q, const void* h_k_new, const void* h_v_new, void* h_out,
                         size_t* h2d_bytes, size_t* d2h_bytes, void* stream_v) {
    if (!p || !h_q || !h_out || (!h_k_new) != (!h_v_new)) return APE_ERR_INVALID_ARG;
    if ((p->kind != PLAN_DECODE && p->kind != PLAN_SHARED) || !p->d_step) return APE_ERR_MODE;
    if (kv_extra < 0 || kv_extra > p->max_kv_extra) return APE_ERR_RANGE;
    DeviceGuard guard(p->h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int n = p->n_req, H_q = p->shape.n_q_heads, H_kv = p->shape.n_kv_heads, D = p->shape.head_dim;
    const size_t q_row_bytes = static_cast<size_t>(H_q) * D * 2, kv_row_bytes = static_cast<size_t>(H_kv) * D * 2;
    // Q rows: one copy when the requests' rows are consecutive and dense, else one strided copy per request
    bool q_dense = p->q.head_stride == D && p->q.token_stride == static_cast<int64_t>(H_q) * D
                && p->out.head_stride == D && p->out.token_stride == static_cast<int64_t>(H_q) * D;
    for (int r = 1; r < n && q_dense; ++r) q_dense = p->q_rows[r] == p->q_rows[0] + r;
    auto q_ptr = [&](const ape_rows_t& t, int r) { return static_cast<uint8_t*>(t.data) + static_cast<size_t>(p->q_rows[r]) * t.token_stride * 2; };
    if (q_dense) {
        if (cudaMemcpyAsync(q_ptr(p->q, 0), h_q, n * q_row_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
    } else {
        for (int r = 0; r < n; ++r)
            if (cudaMemcpy2DAsync(q_ptr(p->q, r), static_cast<size_t>(p->q.head_stride) * 2, static_cast<const uint8_t*>(h_q) + r * q_row_bytes,
                                  static_cast<size_t>(D) * 2, static_cast<size_t>(D) * 2, H_q, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
    }
    size_t up = n * q_row_bytes;
    if (h_k_new) {
        // D0: the new token's K and V rows land densely in the plan's staging area and one small kernel puts them at the
        // rows the query segments have reached (row of the newest token at planning time + kv_extra)
        uint8_t* base = static_cast<uint8_t*>(p->d_step);
        const size_t b_rows = (static_cast<size_t>(n) * 8 + 255) & ~size_t(255);
        uint8_t* k_stage = base + b_rows;
        uint8_t* v_stage = k_stage + n * kv_row_bytes;
        if (cudaMemcpyAsync(k_stage, h_k_new, n * kv_row_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
        if (cudaMemcpyAsync(v_stage, h_v_new, n * kv_row_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return APE_ERR_CUDA;
        AppendParams ap;
        ap.k_new = reinterpret_cast<const __nv_bfloat16*>(k_stage); ap.v_new = reinterpret_cast<const __nv_bfloat16*>(v_stage);
        ap.k_pool = static_cast<__nv_bfloat16*>(const_cast<void*>(p->pool.k)); ap.v_pool = static_cast<__nv_bfloat16*>(const_cast<void*>(p->pool.v));
        ap.rows = reinterpret_cast<const int64_t*>(base); ap.kv_extra = kv_extra;
        ap.token_stride = p->pool.token_stride; ap.head_stride = p->pool.head_stride; ap.n_req = n; ap.H_kv = H_kv; ap.D = D;
        if (launch_append(ap, stream) != cudaSuccess) return APE_ERR_CUDA;
        up += 2 * n * kv_row_bytes;
    }
    int rc = ape_attend(p, T, S, kv_extra, workspace, ws_bytes, stream_v);
    if (rc) return rc;
    if (h_k_new) p->last_launches++;
    if (q_dense) {
        if (cudaMemcpyAsync(h_out, q_ptr(p->out, 0), n * q_row_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return APE_ERR_CUDA;
    } else {
        for (int r = 0; r < n; ++r)
            if (cudaMemcpy2DAsync(static_cast<uint8_t*>(h_out) + r * q_row_bytes, static_cast<size_t>(D) * 2, q_ptr(p->out, r),
                                  static_cast<size_t>(p->out.head_stride) * 2, static_cast<size_t>(D) * 2, H_q, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return APE_ERR_CUDA;
    }
    if (cudaStreamSynchronize(stream) != cudaSuccess) return APE_ERR_CUDA;
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = n * q_row_bytes;
    return APE_OK;
}

int ape_get_status(ape_handle_t h, int32_t* device_status) {
    if (!h || !device_status) return APE_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return APE_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, h->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return APE_ERR_CUDA;
    if (v != 0 && cudaMemset(h->d_status, 0, sizeof(int)) != cudaSuccess) return APE_ERR_CUDA;
    *device_status = v;
    return APE_OK;
}

int ape_get_status_stream(ape_handle_t h, void* stream_v, int32_t* device_status) {
    if (!h || !device_status) return APE_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) return APE_ERR_CUDA;
    if (cap != cudaStreamCaptureStatusNone) return APE_ERR_MODE;      // a read-back cannot be part of a capture
    int v = 0;
    if (cudaMemcpyAsync(&v, h->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return APE_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return APE_ERR_CUDA;
    // cleared only after it has been copied out, and on the same stream, so a later launch there starts from zero
    if (v != 0 && cudaMemsetAsync(h->d_status, 0, sizeof(int), stream) != cudaSuccess) return APE_ERR_CUDA;
    *device_status = v;
    return APE_OK;
}

int ape_set_sm_budget(ape_handle_t h, int32_t n_sm) {
    if (!h || n_sm < 0 || n_sm > h->n_sm_device) return APE_ERR_INVALID_ARG;
    h->n_sm = (n_sm == 0) ? h->n_sm_device : n_sm;
    return APE_OK;
}

namespace {
// One warp waits, with the library's bounded wait, on a barrier that nothing ever completes: after the bound (about a second)
// the wait gives up, raises the status word and the kernel returns normally.
__global__ void ape_wait_probe_kernel(int* status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { ape::mbar_init(ape::smem_u32(&bar), 1); abort_flag = 0; ape::mbar_fence_init(); }
    __syncwarp();
    ape::mbar_wait(ape::smem_u32(&bar), 0, &abort_flag, status);
}
}  // namespace

int ape_selftest_timeout(ape_handle_t h, void* stream_v) {
    if (!h) return APE_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return APE_ERR_CUDA;
    ape_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream_v)>>>(h->d_status);
    return cudaGetLastError() == cudaSuccess ? APE_OK : APE_ERR_CUDA;
}

const char* ape_status_string(int s) {
    switch (s) {
        case APE_OK: return "ok";
        case APE_ERR_INVALID_ARG: return "invalid argument";
        case APE_ERR_SHAPE: return "unsupported head shape";
        case APE_ERR_ALIGN: return "pointer or stride not aligned";
        case APE_ERR_RANGE: return "value out of range";
        case APE_ERR_LAYOUT: return "tensor layout cannot be described to the copy engine";
        case APE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case APE_ERR_CUDA: return "CUDA call failed";
        case APE_ERR_TIMEOUT: return "a kernel gave up on a bounded wait";
        case APE_ERR_NOMEM: return "out of memory";
        case APE_ERR_MODE: return "plan used with the wrong entry point";
        default: return "unknown status";
    }
}

}  // extern "C"

// ---- allocation-free decode ------------------------------------------------------------------------------------------
// A decode step for callers that must not allocate device memory (see include/ape.h).  Everything a plan would put
// into cudaMalloc'ed memory or into the caller's workspace lives in one fixed device array of the library image.

namespace {

constexpr size_t kNoAllocBytes = 8u << 20;        // whole array
constexpr size_t kNoAllocMetaBytes = 4u << 20;    // [0, 256): status word; then tiles, items, CTA ranges, requests, merge groups
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

struct NoAllocDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;             // DEVICE address of g_noalloc_scratch on this device
    ape_handle_s h;                               // host-side record only (no device allocation behind it)
};
constexpr int kMaxDevices = 64;
NoAllocDevice g_noalloc_dev[kMaxDevices];
std::mutex g_noalloc_mutex;

// Once per device, with that device current: the array's name is a host-side stand-in here, so ask the runtime for
// the address the kernels must be given.
int noalloc_setup(int device, NoAllocDevice** out) {
    if (device < 0 || device >= kMaxDevices) return APE_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& d = g_noalloc_dev[device];
    DeviceGuard guard(device);
    if (!guard.ok) return APE_ERR_CUDA;
    if (!d.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return APE_ERR_CUDA;
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return APE_ERR_CUDA;
        if (prop.major != 10) return APE_ERR_CUDA;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) return APE_ERR_CUDA;
        d.scratch = static_cast<unsigned char*>(ptr);
        d.h.device = device; d.h.n_sm = prop.multiProcessorCount; d.h.smem_optin = prop.sharedMemPerBlockOptin;
        d.h.d_status = reinterpret_cast<int*>(d.scratch);
        d.h.encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
        d.ready = true;
    }
    *out = &d;
    return APE_OK;
}

}  // namespace

extern "C" {

int ape_decode_noalloc(const ape_shape_t* shape, const ape_kv_pool_t* pool, const ape_rows_t* q, const ape_rows_t* out,
                       float* lse, const ape_request_t* reqs, int32_t n_req, float T, float S, int64_t kv_extra,
                       int device, void* stream_v, int32_t* device_status)
{
    int G = 1; float c = 0.f;
    int rc = check_shape(shape, &G, &c);              if (rc) return rc;
    rc = check_pool(pool, shape);                     if (rc) return rc;
    rc = check_rows(q, shape);                        if (rc) return rc;
    rc = check_rows(out, shape);                      if (rc) return rc;
    rc = check_lse(lse);                              if (rc) return rc;
    if (!reqs || n_req <= 0 || out->n_rows < q->n_rows) return APE_ERR_INVALID_ARG;
    if (!(T > 0.f) || !(S > 0.f) || !std::isfinite(T) || !std::isfinite(S)) return APE_ERR_RANGE;
    int64_t max_extra = INT64_MAX, total_tiles = 0;
    try {
        for (int r = 0; r < n_req; ++r) {
            const ape_request_t& rq = reqs[r];
            if (rq.q_len != 1 || rq.q_start < 0 || rq.q_start + 1 > q->n_rows) return APE_ERR_INVALID_ARG;
            if (rq.n_ctx < 0 || (rq.n_ctx > 0 && !rq.ctx)) return APE_ERR_INVALID_ARG;
            if (!span_ok(rq.prefix, pool->n_tokens) || !span_ok(rq.query_kv, pool->n_tokens)) return APE_ERR_INVALID_ARG;
            if (rq.query_kv.len < 1) return APE_ERR_INVALID_ARG;
            if (rq.query_kv_capacity < rq.query_kv.len || rq.query_kv.start + rq.query_kv_capacity > pool->n_tokens) return APE_ERR_INVALID_ARG;
            total_tiles += (rq.prefix.len + kDecodeTile - 1) / kDecodeTile + (rq.query_kv_capacity + kDecodeTile - 1) / kDecodeTile;
            for (int i = 0; i < rq.n_ctx; ++i) if (!span_ok(rq.ctx[i], pool->n_tokens)) return APE_ERR_INVALID_ARG;
            // tiles are cut from the fused spans (touching contexts form one span), exactly as the tile list below is
            for (const auto& sp : fuse_spans(rq.ctx, rq.n_ctx)) total_tiles += (sp.len + kDecodeTile - 1) / kDecodeTile;
            max_extra = std::min(max_extra, rq.query_kv_capacity - rq.query_kv.len);
        }
    } catch (const std::bad_alloc&) {
        return APE_ERR_NOMEM;
    }
    if (kv_extra < 0 || kv_extra > max_extra) return APE_ERR_RANGE;
    // size gate, before the tile list is built and before anything touches the device
    if (static_cast<size_t>(total_tiles) * sizeof(DevTile) > kNoAllocMetaBytes) return APE_ERR_WORKSPACE;

    NoAllocDevice* dv = nullptr;
    rc = noalloc_setup(device, &dv);                  if (rc) return rc;
    DeviceGuard guard(device);
    if (!guard.ok) return APE_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    {
        // Never part of a stream capture: the metadata is rebuilt from the caller's host arrays on every call and uploaded
        // from a buffer that dies with the call, so a replayed graph would read freed host memory and feed the kernels
        // stale item records.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) return APE_ERR_CUDA;
        if (cap != cudaStreamCaptureStatusNone) return APE_ERR_MODE;
    }
    const int D = shape->head_dim, H_kv = shape->n_kv_heads, tile = kDecodeTile;
    const int n_cta = dv->h.n_sm;

    HostMeta m;
    std::vector<uint8_t> blob;
    size_t o_tiles = 0, o_items = 0, o_cta = 0, o_reqs = 0, o_merge = 0;
    try {
        std::vector<Run> runs;
        for (int r = 0; r < n_req; ++r) {
            const ape_request_t& rq = reqs[r];
            m.reqs.push_back(DevReq{static_cast<int32_t>(rq.q_start), 1, static_cast<int32_t>(rq.query_kv.len), 0});
            const int o0 = static_cast<int>(m.tiles.size());
            add_span_tiles(m.tiles, rq.prefix.start, rq.prefix.len, tile, 0, 0);
            add_span_tiles(m.tiles, rq.query_kv.start, rq.query_kv.len, tile, TILE_GROWS, rq.query_kv_capacity);
            const int o1 = static_cast<int>(m.tiles.size());
            const auto ctx_ranges = add_context_tiles(m.tiles, rq.ctx, rq.n_ctx, tile, false);
            for (int hh = 0; hh < H_kv; ++hh) {
                const int mi = static_cast<int>(m.merge.size());
                m.merge.push_back(DevMerge{r, hh, 0, 0, 0, 0, 0, 1});
                runs.push_back(Run{r, hh, 0, 1, SEG_OTHER, o0, o1, mi});
                for (const auto& cr : ctx_ranges) runs.push_back(Run{r, hh, 0, 1, SEG_CTX, cr.t0, cr.t1, mi});
            }
        }
        assign_stream(runs, n_cta, 1, m);
        finish_items(m);
        auto rnd = [](size_t x) { return (x + 255) & ~size_t(255); };
        o_tiles = 256;                                                     // after the status word
        o_items = o_tiles + rnd(m.tiles.size() * sizeof(DevTile));
        o_cta = o_items + rnd(m.items.size() * sizeof(DevItem));
        o_reqs = o_cta + rnd(m.cta_begin.size() * 4);
        o_merge = o_reqs + rnd(m.reqs.size() * sizeof(DevReq));
        const size_t meta_end = o_merge + rnd(m.merge.size() * sizeof(DevMerge));
        const size_t rows = m.items.size() * static_cast<size_t>(G);
        const size_t part_bytes = rnd(rows * D * 4) + rnd(rows * 2 * 4);
        if (meta_end > kNoAllocMetaBytes || part_bytes > kNoAllocBytes - kNoAllocMetaBytes) return APE_ERR_WORKSPACE;
        blob.assign(meta_end, 0);                                          // byte 0..255 stand for the status word: not uploaded
        std::memcpy(blob.data() + o_tiles, m.tiles.data(), m.tiles.size() * sizeof(DevTile));
        std::memcpy(blob.data() + o_items, m.items.data(), m.items.size() * sizeof(DevItem));
        std::memcpy(blob.data() + o_cta, m.cta_begin.data(), m.cta_begin.size() * 4);
        std::memcpy(blob.data() + o_reqs, m.reqs.data(), m.reqs.size() * sizeof(DevReq));
        std::memcpy(blob.data() + o_merge, m.merge.data(), m.merge.size() * sizeof(DevMerge));
    } catch (const std::bad_alloc&) {
        return APE_ERR_NOMEM;
    }

    const int n_stages = decode_pick_stages(D, G, dv->h.smem_optin - 2048);
    if (n_stages < 2) return APE_ERR_SHAPE;
    const size_t smem_bytes = decode_smem_bytes(D, G, n_stages);
    if (decode_set_smem_attr(D, smem_bytes) != cudaSuccess) return APE_ERR_CUDA;
    CUtensorMap tm_k, tm_v;
    rc = make_map(&dv->h, &tm_k, pool->k, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
    if (!rc) rc = make_map(&dv->h, &tm_v, pool->v, D, H_kv, pool->n_tokens, pool->head_stride, pool->token_stride, 1, tile);
    if (rc) return rc;

    unsigned char* base = dv->scratch;
    // The array still holds the previous call's status word, metadata and partials.  The copy below rewrites all
    // metadata this call uses; partial slots are fully written by the decode kernel before the merge kernel reads
    // them, so they need no clearing.  The status word (first 256 bytes) is NOT rewritten: it is zero when the library
    // image is loaded, a kernel that gives up on a bounded wait sets it, and it stays set -- across later calls too --
    // until a call hands it out through `device_status` and clears it.  The source of the copy is pageable host memory:
    // the runtime waits for earlier work on the stream, stages the bytes, and has taken its copy when the call returns.
    if (cudaMemcpyAsync(base + o_tiles, blob.data() + o_tiles, blob.size() - o_tiles, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return APE_ERR_CUDA;

    constexpr float kLog2e = 1.4426950408889634f;
    const size_t rows = m.items.size() * static_cast<size_t>(G);
    float* ws_o = reinterpret_cast<float*>(base + kNoAllocMetaBytes);
    float* ws_ml = reinterpret_cast<float*>(base + kNoAllocMetaBytes + ((rows * D * 4 + 255) & ~size_t(255)));
    DecodeParams dp;
    dp.tiles = reinterpret_cast<const DevTile*>(base + o_tiles); dp.items = reinterpret_cast<const DevItem*>(base + o_items);
    dp.cta_item_begin = reinterpret_cast<const int32_t*>(base + o_cta); dp.reqs = reinterpret_cast<const DevReq*>(base + o_reqs);
    dp.q = rows_desc(*q); dp.ws_o = ws_o; dp.ws_ml = ws_ml;
    dp.scale_oth_log2 = c * kLog2e; dp.scale_ctx_log2 = c / T * kLog2e;
    dp.kv_extra = static_cast<int32_t>(kv_extra); dp.G = G; dp.n_stages = n_stages; dp.status = reinterpret_cast<int*>(base);
    if (launch_decode(D, tm_k, tm_v, dp, n_cta, smem_bytes, stream) != cudaSuccess) return APE_ERR_CUDA;
    MergeParams mp;
    mp.groups = reinterpret_cast<const DevMerge*>(base + o_merge); mp.reqs = dp.reqs; mp.items = dp.items; mp.per_context = 0; mp.nodes = nullptr; mp.n_groups = static_cast<int32_t>(m.merge.size());
    mp.rows_per_slot = G; mp.tokens_per_block = 1; mp.ws_o = ws_o; mp.ws_ml = ws_ml; mp.out = rows_desc(*out); mp.lse_out = lse;
    mp.ws_o_ctx = ws_o; mp.ws_ml_ctx = ws_ml; mp.rows_per_slot_ctx = G;
    mp.part_o_ctx = nullptr; mp.part_lse_ctx = nullptr; mp.part_o_oth = nullptr; mp.part_lse_oth = nullptr;
    mp.S = S; mp.G = G; mp.H_q = shape->n_q_heads; mp.D = D;
    if (launch_merge(mp, stream) != cudaSuccess) return APE_ERR_CUDA;
    if (device_status != nullptr) {
        // the caller asked for the status word: this makes the call synchronous; a word that was set is cleared once read
        int v = 0;
        if (cudaMemcpyAsync(&v, base, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return APE_ERR_CUDA;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return APE_ERR_CUDA;
        if (v != 0 && cudaMemsetAsync(base, 0, sizeof(int), stream) != cudaSuccess) return APE_ERR_CUDA;
        *device_status = v;
    }
    return APE_OK;
}

int ape_selftest_timeout_noalloc(int device, void* stream_v) {
    NoAllocDevice* dv = nullptr;
    int rc = noalloc_setup(device, &dv);              if (rc) return rc;
    DeviceGuard guard(device);
    if (!guard.ok) return APE_ERR_CUDA;
    ape_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream_v)>>>(reinterpret_cast<int*>(dv->scratch));
    return cudaGetLastError() == cudaSuccess ? APE_OK : APE_ERR_CUDA;
}

}  // extern "C"
