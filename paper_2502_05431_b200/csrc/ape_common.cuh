// Shared device-side declarations of libape: plan metadata records and thin PTX wrappers
// (mbarrier, bulk tensor copy, bounded waits).  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ape {

// ---- plan metadata (host-built, device-resident) ---------------------------------------------------------------

// One tile of consecutive pool tokens that belong to one segment of one request.
struct DevTile {
    int32_t tok;       // first pool token of the tile (copy-engine coordinate)
    int32_t n_valid;   // keys of the tile that belong to the span (static tiles)
    int32_t key_base;  // index of the tile's first key inside the query segment / context (causal, growing tiles)
    int32_t flags;     // TILE_CAUSAL: apply the causal rule; TILE_GROWS: n_valid follows the segment's current length
};
enum : int32_t { TILE_CAUSAL = 1, TILE_GROWS = 2, TILE_SPLIT = 4, TILE_CTX_END = 8 };
// TILE_SPLIT (encode plans): the tile's first split_r rows are the tail of the shared prefix (from `tok`), the rest are the
// first tokens of the item's context; key_base is -split_r, so the causal rule sees the prefix keys as "before the context".
// TILE_CTX_END (two-pass plans): the last tile of a context node's own tokens; such plans keep the node's index in key_base
// of their context tiles (which are not causal and need no key index).

// A run of tiles of one segment for one (request, KV head, row block): yields one partial (m, l, O~).
struct DevItem {
    int32_t req;         // request index (attend) or context index (encode)
    int32_t kv_head;
    int32_t row_block;   // first row block of the sibling group; sibling s handles row_block + s
    int32_t tile_begin;  // [tile_begin, tile_end) in the tile list
    int32_t tile_end;
    int32_t slot;        // partial slot of sibling 0; sibling s writes slot + s
    int32_t seg;         // SEG_OTHER (prefix + query segment), SEG_CTX, or SEG_FINAL (encode: write O directly)
    int32_t n_sib;       // live siblings of this item (row blocks that exist)
    // copies of the request geometry and of the first tile record, so that an item is ONE 64-byte load that the
    // tensor-core kernel fetches an item ahead (no dependent loads when it moves to the next item)
    int32_t q_row0;      // first row of Q / O of the request (encode: context start)
    int32_t q_len;       // query rows of the request
    int32_t l_k;         // keys in the query segment at planning time (encode: context length)
    int32_t ctx_id;      // SEG_CTX items: ordinal of the context (per-context plans) or index of the tree node (tree plans)
                         // the tiles belong to, else 0
    DevTile first_tile;  // tiles[tile_begin]
};
static_assert(sizeof(DevItem) == 64, "DevItem is one 64-byte record");
enum : int32_t { SEG_OTHER = 0, SEG_CTX = 1, SEG_FINAL = 2 };

// Per request (attend) / per context (encode) row geometry.
struct DevReq {
    int32_t q_row0;      // first row of Q / O
    int32_t q_len;       // query rows
    int32_t l_k;         // keys in the query segment at planning time (encode: context length)
    int32_t pad;
};

// What the merge kernel needs per (request, KV head, row block): where its partials are.
struct DevMerge {
    int32_t req;
    int32_t kv_head;
    int32_t row_block;
    int32_t ctx_slot0;   // first context slot, stride slot_stride between consecutive partials
    int32_t ctx_n;
    int32_t oth_slot0;
    int32_t oth_n;
    int32_t slot_stride; // between consecutive non-context partials (and context partials of ordinary plans)
    int32_t ctx_row_off; // added to the row when a context partial is read: shared-context plans keep the context
                         // partials of many requests in one slot, one group of rows per request
    int32_t ctx_stride;  // between consecutive context partials
};

// One node of a context tree (tree plans): a SEG_CTX item's ctx_id is the index of the node its tiles belong to.
struct DevNode {
    int32_t parent;      // index of the parent node in the same array, -1 for a top-level node
    int32_t depth;       // 0 for a top-level node
    int32_t scaled;      // != 0: the node hands S * log-sum-exp to its parent (Eq. 11), else its plain log-sum-exp
    int32_t pad;
};
constexpr int kMaxTreeDepth = 16;   // levels of nodes below the final merge

struct RowsDesc {        // Q or O rows: element (r, h, e) at data[r*token_stride + h*head_stride + e]
    __nv_bfloat16* data;
    int64_t token_stride;
    int64_t head_stride;
};

constexpr int32_t kStatusTimeout = -8;   // APE_ERR_TIMEOUT

// ---- PTX wrappers ----------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Every wait in the library is bounded: after about a second (2^31 SM cycles) the waiter raises the CTA's
// abort flag and the device status word, and every role of the CTA leaves its loop.  Returns false on abort.
constexpr long long kWaitCycles = 1ll << 31;

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = 0;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitCycles) {
                *abort_flag = 1;
                atomicExch(status, kStatusTimeout);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// 3-D tiled bulk tensor copy global -> shared of this CTA; completion is counted in bytes on `bar`.
// The innermost coordinate x must make x * sizeof(element) a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap* tmap, uint32_t bar,
                                            int32_t x, int32_t y, int32_t z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
// 3-D tiled bulk tensor copy shared -> global (same alignment rule for x; every coordinate non-negative).  The copy joins
// the issuing thread's current bulk group.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tmap, uint32_t smem_src, int32_t x, int32_t y, int32_t z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_src), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Returns once every bulk group of this thread has finished READING its shared-memory source.
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 32-byte store to global memory (address 32-byte aligned): one full sector per instruction
__device__ __forceinline__ void st_global_v8(void* ptr, uint32_t a, uint32_t b, uint32_t c, uint32_t d,
                                             uint32_t e, uint32_t f, uint32_t g, uint32_t h) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(ptr), "r"(a), "r"(b), "r"(c), "r"(d), "r"(e), "r"(f), "r"(g), "r"(h) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace ape
