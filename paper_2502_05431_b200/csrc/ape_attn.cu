// Tensor-core attention kernel of libape, shared by query prefill (ape_attend) and context encoding
// (ape_encode_contexts).  One persistent CTA owns a block of 256 packed query rows (row = token * G + head-in-group,
// so the G query heads of a KV head share every K/V tile) as two 128-row halves, and walks its list of work items.
// Every item is a run of 128-key tiles of ONE segment, so a plain online softmax per item is exact; the scaling
// factor S of Eq. 5 acts on whole-segment log-sum-exps and is applied by the merge kernel afterwards.
//
// Roles (warp-specialised, 384 threads):
//   warps 0-3 / 4-7  softmax of half 0 / half 1: one thread per row; S is read from TMEM, P = 2^(s - m) goes back
//                    to TMEM as bf16 over the S columns, the running sum stays in a register; also the epilogue
//                    (partials to the workspace, final rows to global memory or, for encode, into the item's Q buffer)
//   warp 8           producer: bulk tensor copies of K and V tiles (and of Q with one Q buffer) into 128-byte-swizzled
//                    shared memory
//   warps 9, 10      MMA issuers of half 0 / half 1: S = Q K^T (both operands in shared memory) and O += P V (P from
//                    TMEM) with tcgen05.mma, accumulators in TMEM; warp 9 owns the TMEM allocation
//   warp 11          with two Q buffers (encode): loads Q one row block ahead and hands finished O tiles to the bulk
//                    tensor store; idle otherwise
// The two halves run one tile apart, so that the tensor pipe works on one half while the other does its exponentials.
// When a row block has at most 128 live rows (a decode batch that shares its contexts), the plan can ask for the
// alternating form instead (ALT): both halves read the SAME 128 rows of Q and take every other tile, each with an online
// softmax and a partial of its own, so no half works on rows that do not exist; the Q half that is not needed pays for a
// third stage of K and of V, which a half that sees only every other tile needs to have its next tile under way.
#include "ape_common.cuh"
#include "ape_kernels.h"
#include "ape_tcgen05.cuh"

namespace ape {

namespace {

constexpr int kTileN = kAttnTileN;            // 128 keys per tile
constexpr int kHalfRows = 128;
constexpr int kThreads = 384;               // three warpgroups: two of softmax warps, one of producer / issuers / Q loader
constexpr int kRegsSoftmax = 216;            // registers per thread after the hand-over (two softmax warpgroups)
constexpr int kRegsOther = 72;               // producer / MMA warpgroup
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr int kSlabBytes = 128 * 128;         // 128 rows x 64 bf16
constexpr float kRescaleThreshold = 8.0f;     // base-2 units: O is rescaled only when the row maximum grew by more
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// packed pairs of floats in one 64-bit register (fma.rn.f32x2 / add.rn.f32x2)
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ void prefetch_l1(const void* ptr) {
    asm volatile("prefetch.global.L1 [%0];" ::"l"(ptr));
}

struct ItemGeom {
    int rb;          // row block of this CTA for the item
    int last_tok;    // last live query token of the row block
    int off;         // l_k - q_len: causal offset
};

__device__ __forceinline__ bool tile_visible(const DevTile& t, const ItemGeom& g) {
    if (t.n_valid <= 0) return false;
    if ((t.flags & TILE_CAUSAL) && t.key_base > g.last_tok + g.off) return false;
    return true;
}

}  // namespace

// QBUF: number of Q buffers.  Plans with long items (prefill) use one Q buffer and two stages each of K and V; plans
// with many short items (encode) use two Q buffers, so that the next row block's Q arrives while the current one is
// in use, and pay for them with a single V stage.
// MODE selects the configuration (ape_kernels.h): kAttnPrefill, kAttnEncode (two Q buffers), kAttnAlt (alternating halves),
// and the two passes of the plans that scale parts of the context segment separately (per-context form, context trees):
// kAttnStats computes, per row, the (maximum, sum) of every node's own tokens (S = Q K^T and the softmax sums only: no P,
// no V, no O); kAttnBias is the prefill pass with a per-row, per-node bias added to the context logits.
template <int D, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
ape_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                const __grid_constant__ SplitMaps tm_split, const AttnParams p)
{
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kSlabs * kSlabBytes;            // one K or V tile, also one Q half
    constexpr int QBUF = (MODE == kAttnEncode) ? 2 : 1;
    constexpr bool ALT = MODE == kAttnAlt, STATS = MODE == kAttnStats, BIAS = MODE == kAttnBias;
    constexpr int kQBytes = (ALT ? 1 : 2) * kTileBytes;        // both halves of a row block (ALT: the one half both read)
    constexpr int kNK = ALT ? 3 : 2;                           // K stages
    constexpr int kNV = ALT ? 3 : (QBUF == 2) ? 1 : 2;         // V stages
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 256 + D;
    constexpr uint32_t kIdescQK = idesc_bf16_f32(128, kTileN, 0, 0);
    constexpr uint32_t kIdescPV = idesc_bf16_f32(128, D, 0, 1);

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* q_smem = smem;                                    // QBUF buffers x 2 halves
    uint8_t* k_smem = q_smem + QBUF * kQBytes;                 // kNK stages
    uint8_t* v_smem = k_smem + kNK * kTileBytes;               // kNV stages
    uint64_t* bars = reinterpret_cast<uint64_t*>(v_smem + kNV * kTileBytes);
    // barrier map
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t bar_q_full = bar0, bar_q_empty = bar0 + 16;             // [QBUF] each
    const uint32_t bar_k_full = bar0 + 32, bar_k_empty = bar_k_full + 8 * kNK;
    const uint32_t bar_v_full = bar_k_empty + 8 * kNK, bar_v_empty = bar_v_full + 8 * kNV;
    const uint32_t bar_s_full = bar_v_empty + 8 * kNV;         // [2]
    const uint32_t bar_p_full = bar_s_full + 16;               // [2 halves][4 key quarters]: P columns of 32 keys written
    const uint32_t bar_o_full = bar_p_full + 64;               // [2]
    const uint32_t bar_done = bar_o_full + 16;
    const uint32_t bar_tok = bar_done + 8;                     // [2]: turn-taking of the two halves' exponential phases
    const uint32_t bar_o_staged = bar_tok + 16;                // [2]: a half's O tile sits in shared memory, ready for its bulk store
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int b = 0; b < QBUF; ++b) { mbar_init(bar_q_full + 8 * b, 1); mbar_init(bar_q_empty + 8 * b, 2); }   // released by both MMA issuers
        for (int s = 0; s < kNK; ++s) { mbar_init(bar_k_full + 8 * s, 1); mbar_init(bar_k_empty + 8 * s, 2); }   // released by both issuers
        for (int s = 0; s < kNV; ++s) { mbar_init(bar_v_full + 8 * s, 1); mbar_init(bar_v_empty + 8 * s, 2); }
        for (int w = 0; w < 2; ++w) {
            mbar_init(bar_s_full + 8 * w, 1);
            for (int qq = 0; qq < 4; ++qq) mbar_init(bar_p_full + 32 * w + 8 * qq, 4);   // one arrival per softmax warp
            mbar_init(bar_o_full + 8 * w, 1);
        }
        mbar_init(bar_done, 2);
        mbar_init(bar_tok, 4); mbar_init(bar_tok + 8, 4);          // one arrival per softmax warp of the other half
        mbar_init(bar_o_staged, 4); mbar_init(bar_o_staged + 8, 4);  // one arrival per softmax warp of the half
        mbar_fence_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&tmem_base_smem), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_smem;

    const int n_sib = p.n_sib;
    const int group = blockIdx.x / n_sib, sib = blockIdx.x - group * n_sib;
    const int item_begin = p.cta_item_begin[group], item_end = p.cta_item_begin[group + 1];
    const int G = p.G;
    constexpr bool alt = ALT;                // both halves read the same 128 rows and take alternate tiles
    const int TB = (alt ? kHalfRows : kAttnRows) / G;            // query tokens per row block

    auto geom = [&](const DevItem& item, const DevReq& rq) {
        ItemGeom g;
        g.rb = item.row_block + sib;
        g.last_tok = min(rq.q_len, (g.rb + 1) * TB) - 1;
        g.off = rq.l_k - rq.q_len;
        return g;
    };

    // A half whose 128 rows are all live query rows can leave as one tile (bulk store); ragged halves are written row by row.
    auto half_is_full = [&](const DevReq& rq, const ItemGeom& g, int w) {
        return g.rb * TB + (w + 1) * (kHalfRows / G) <= rq.q_len;
    };
    const bool o_via_tma = (QBUF == 2) && p.o_via_tma != 0;

    // Register hand-over at the head of every role: the softmax threads hold a whole 128-column row of S in registers,
    // the third warpgroup (producer, MMA issuers, Q loader) gives its share up.
    // Q of one row block (both halves) into buffer n % QBUF, once the MMAs that read that buffer last are done.
    auto load_q = [&](const DevItem& item, const DevReq& rq, const ItemGeom& g, uint32_t n) {
        const uint32_t qb = n % QBUF, q_use = n / QBUF;
        if (q_use > 0 && !mbar_wait(bar_q_empty + 8 * qb, (q_use - 1) & 1, &abort_flag, p.status)) return false;
        mbar_expect_tx(bar_q_full + 8 * qb, kQBytes);
        #pragma unroll
        for (int w = 0; w < (ALT ? 1 : 2); ++w) {
            const int tok0 = rq.q_row0 + g.rb * TB + w * (kHalfRows / G);
            #pragma unroll
            for (int sl = 0; sl < kSlabs; ++sl)
                tma_load_3d(smem_u32(q_smem + qb * kQBytes + w * kTileBytes + sl * kSlabBytes), &tm_q, bar_q_full + 8 * qb,
                            sl * 64, item.kv_head * G, tok0);
        }
        return true;
    };

    if (warp == kProducerWarp) {
        // =============================== producer ====================================================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
        if (lane == 0) {
            tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
            uint32_t kcnt = 0, vcnt = 0, q_loads = 0;
            int last_req = -1, last_head = -1, last_rb = -1;
            bool ok = true;
            for (int it = item_begin; it < item_end && ok; ++it) {
                const DevItem item = p.items[it];
                if (it + 1 < item_end) prefetch_l1(&p.items[it + 1]);   // the next item's record is in cache when its turn comes
                if (sib >= item.n_sib) continue;
                if (STATS && item.seg != SEG_CTX) continue;             // the statistics pass is about context nodes only
                const DevReq rq{item.q_row0, item.q_len, item.l_k, 0};
                const ItemGeom g = geom(item, rq);
                if (QBUF == 1 && !(item.req == last_req && item.kv_head == last_head && g.rb == last_rb)) {
                    if (!load_q(item, rq, g, q_loads)) { ok = false; break; }
                    ++q_loads; last_req = item.req; last_head = item.kv_head; last_rb = g.rb;
                }
                DevTile next_tile = item.first_tile;
                for (int t = item.tile_begin; t < item.tile_end; ++t) {
                    const DevTile tile = next_tile;
                    if (t + 1 < item.tile_end) next_tile = p.tiles[t + 1];
                    if (!tile_visible(tile, g)) continue;
                    {
                        const int s = kcnt % kNK; const uint32_t use = kcnt / kNK;
                        if (!mbar_wait(bar_k_empty + 8 * s, (use & 1) ^ 1, &abort_flag, p.status)) { ok = false; break; }
                        mbar_expect_tx(bar_k_full + 8 * s, kTileBytes);
                        if (tile.flags & TILE_SPLIT) {
                            // prefix tail in the first split_r rows, the context's first tokens behind it: two boxes that
                            // together fill the tile (same byte count), so no key slot of the tile is wasted on padding
                            #pragma unroll
                            for (int sl = 0; sl < kSlabs; ++sl) {
                                const uint32_t dst = smem_u32(k_smem + s * kTileBytes + sl * kSlabBytes);
                                tma_load_3d(dst, &tm_split.ka, bar_k_full + 8 * s, sl * 64, item.kv_head, tile.tok);
                                tma_load_3d(dst + p.split_r * 128, &tm_split.kb, bar_k_full + 8 * s, sl * 64, item.kv_head, item.q_row0);
                            }
                        } else
                        #pragma unroll
                        for (int sl = 0; sl < kSlabs; ++sl)
                            tma_load_3d(smem_u32(k_smem + s * kTileBytes + sl * kSlabBytes), &tm_k, bar_k_full + 8 * s,
                                        sl * 64, item.kv_head, tile.tok);
                        ++kcnt;
                    }
                    if (!STATS) {
                        const int s = vcnt % kNV; const uint32_t use = vcnt / kNV;
                        if (!mbar_wait(bar_v_empty + 8 * s, (use & 1) ^ 1, &abort_flag, p.status)) { ok = false; break; }
                        mbar_expect_tx(bar_v_full + 8 * s, kTileBytes);
                        if (tile.flags & TILE_SPLIT) {
                            #pragma unroll
                            for (int sl = 0; sl < kSlabs; ++sl) {
                                const uint32_t dst = smem_u32(v_smem + s * kTileBytes + sl * kSlabBytes);
                                tma_load_3d(dst, &tm_split.va, bar_v_full + 8 * s, sl * 64, item.kv_head, tile.tok);
                                tma_load_3d(dst + p.split_r * 128, &tm_split.vb, bar_v_full + 8 * s, sl * 64, item.kv_head, item.q_row0);
                            }
                        } else
                        #pragma unroll
                        for (int sl = 0; sl < kSlabs; ++sl)
                            tma_load_3d(smem_u32(v_smem + s * kTileBytes + sl * kSlabBytes), &tm_v, bar_v_full + 8 * s,
                                        sl * 64, item.kv_head, tile.tok);
                        ++vcnt;
                    }
                }
            }
            if (!ok) {
                // wait (bounded) for copies that were issued but whose barrier nobody may consume any more
                const long long t0 = clock64();
                for (int s = 0; s < kNK; ++s) {
                    const uint32_t issued = (kcnt > static_cast<uint32_t>(s)) ? (kcnt - 1 - s) / kNK + 1 : 0;
                    while (issued && !mbar_try_wait(bar_k_full + 8 * s, (issued - 1) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
                for (int s = 0; s < kNV; ++s) {
                    const uint32_t issued = (vcnt > static_cast<uint32_t>(s)) ? (vcnt - 1 - s) / kNV + 1 : 0;
                    while (issued && !mbar_try_wait(bar_v_full + 8 * s, (issued - 1) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
                for (uint32_t b = 0; b < QBUF; ++b) {
                    const uint32_t issued = (q_loads > b) ? (q_loads - 1 - b) / QBUF + 1 : 0;
                    while (QBUF == 1 && issued && !mbar_try_wait(bar_q_full + 8 * b, (issued - 1) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
        // =============================== MMA issuers: one warp per 128-row half =========================================
        // Each half has its own issuing warp so that neither half ever queues behind the other's waits.  All 32 lanes
        // walk the loop and take part in the waits; lane 0 issues the tensor-core instructions.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
        const int w = warp - kMmaWarp;
        uint32_t kcnt = 0, vcnt = 0, q_loads = 0, pcnt = 0;
        int last_req = -1, last_head = -1, last_rb = -1;
        bool ok = true;
        const uint32_t tS = tmem_base + (w ? kColS1 : kColS0);
        const uint32_t tO = tmem_base + (w ? kColO1 : kColO0);
        const uint32_t my_s_full = bar_s_full + 8 * w, my_p_full = bar_p_full + 32 * w, my_o_full = bar_o_full + 8 * w;
        const uint32_t leader = (lane == 0) ? 1u : 0u;
        auto wait_all = [&](uint32_t bar, uint32_t parity) {
            return __all_sync(0xffffffffu, mbar_wait(bar, parity, &abort_flag, p.status)) != 0;
        };
        // Descriptors differ from their tile's base descriptor only in the 14-bit start-address field (units of 16 B),
        // so every MMA costs one add per operand instead of a descriptor build: the issuing lane shares its scheduler
        // with two softmax warps and must stay lean.
        uint64_t q_desc0 = smem_desc_sw128(smem_u32(q_smem + (ALT ? 0 : w) * kTileBytes), 16, 1024);
        auto issue_qk = [&](uint32_t k_base) {
            const uint64_t k_desc0 = smem_desc_sw128(k_base, 16, 1024);
            #pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint64_t o = static_cast<uint64_t>(((ks >> 2) * kSlabBytes + (ks & 3) * 32) >> 4);
                mma_ss_elect(leader, tS, q_desc0 + o, k_desc0 + o, kIdescQK, ks > 0);
            }
        };
        // P is zero past the last key that any row of the block may see, so the product stops there (rounded up to 16).
        auto issue_pv = [&](uint64_t v_desc0, bool accumulate, int key_quarter) {   // keys 32*key_quarter .. +32
            #pragma unroll
            for (int k2 = 0; k2 < 2; ++k2) {
                const int ks = key_quarter * 2 + k2;
                mma_ts_elect(leader, tO, tS + ks * 8, v_desc0 + static_cast<uint64_t>((ks * 2048) >> 4), kIdescPV,
                       (accumulate || ks > 0) ? 1u : 0u);
            }
        };
        auto issue_pv_cut = [&](uint64_t v_desc0, bool accumulate, int key_quarter, int n16) {   // same, stopping at key n16
            #pragma unroll
            for (int k2 = 0; k2 < 2; ++k2) {
                const int ks = key_quarter * 2 + k2;
                if (ks * 16 < n16) mma_ts_elect(leader, tO, tS + ks * 8, v_desc0 + static_cast<uint64_t>((ks * 2048) >> 4), kIdescPV,
                       (accumulate || ks > 0) ? 1u : 0u);
            }
        };
        // V rows past the span may hold anything (even NaN bit patterns); P is 0 there, and 0 * NaN must stay 0.
        // Both issuing warps clear the same rows with the same zeros before their own products: a benign overlap.
        // Only rows that the product reads are cleared: [n_valid, n16).
        auto scrub_v = [&](uint8_t* v_tile, int n_valid, int n16) {
            const int per_slab = (n16 - n_valid) * 8;                 // 16-byte chunks to clear in each slab (fewer than 128)
            #pragma unroll
            for (int sl = 0; sl < kSlabs; ++sl)
                for (int i = lane; i < per_slab; i += 32)
                    *reinterpret_cast<uint4*>(v_tile + sl * kSlabBytes + (n_valid + (i >> 3)) * 128 + (i & 7) * 16) = make_uint4(0, 0, 0, 0);
            fence_proxy_async_smem();
            __syncwarp();
        };
        // O += P V for the previous tile of this half, in two key halves as P is published
        uint32_t prev_v_release = 0, pending_q_release = 0;
        bool s_pending = false;                                   // statistics pass: an S tile that has not been read yet
        auto pv_prev = [&](uint32_t prev_vs, uint32_t prev_vphase, int prev_valid, int prev_n16, bool o_started) {
            if (!wait_all(bar_v_full + 8 * prev_vs, prev_vphase)) return false;
            uint8_t* v_tile = v_smem + prev_vs * kTileBytes;
            if (prev_valid < prev_n16) scrub_v(v_tile, prev_valid, prev_n16);
            const uint32_t v_base = smem_u32(v_tile);
            const uint64_t v_desc0 = smem_desc_sw128(v_base, kSlabBytes, 1024);
            if (prev_n16 == kTileN) {
                #pragma unroll
                for (int qq = 0; qq < 4; ++qq) {                  // P arrives in quarters of 32 keys
                    if (!wait_all(my_p_full + 8 * qq, pcnt & 1)) return false;
                    tc_fence_after();
                    issue_pv(v_desc0, o_started, qq);
                }
            } else {
                #pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    if (!wait_all(my_p_full + 8 * qq, pcnt & 1)) return false;
                    tc_fence_after();
                    issue_pv_cut(v_desc0, o_started, qq, prev_n16);
                }
            }
            if (kNV == 1) {                                       // single V stage: free it at once, the next V load is waiting
                mma_commit_elect(leader, bar_v_empty + 8 * prev_vs);
            } else {
                prev_v_release = bar_v_empty + 8 * prev_vs;       // committed after the next S = Q K^T has been issued
            }
            ++pcnt;
            return true;
        };

        for (int it = item_begin; it < item_end && ok; ++it) {
            const DevItem item = p.items[it];
            if (it + 1 < item_end) prefetch_l1(&p.items[it + 1]);       // the next item's record is in cache when its turn comes
            if (sib >= item.n_sib) continue;
            if (STATS && item.seg != SEG_CTX) continue;
            const DevReq rq{item.q_row0, item.q_len, item.l_k, 0};
            const ItemGeom g = geom(item, rq);
            if (!(item.req == last_req && item.kv_head == last_head && g.rb == last_rb)) {
                // The Q buffer just used may be refilled once both halves' MMAs issued so far are done.  A commit that
                // follows another commit holds the issuing thread until the tensor pipe has drained, so with two Q
                // buffers this one is put off until the next S = Q K^T is on its way (with one buffer that product waits
                // for the refill, so the commit cannot wait for it).
                if (q_loads > 0) {
                    if (QBUF == 1) mma_commit_elect(leader, bar_q_empty);
                    else pending_q_release = bar_q_empty + 8 * ((q_loads - 1) % QBUF);
                }
                const uint32_t qb = q_loads % QBUF;
                if (!wait_all(bar_q_full + 8 * qb, (q_loads / QBUF) & 1)) { ok = false; break; }
                if (QBUF > 1) q_desc0 = smem_desc_sw128(smem_u32(q_smem + qb * kQBytes + (ALT ? 0 : w) * kTileBytes), 16, 1024);
                ++q_loads; last_req = item.req; last_head = item.kv_head; last_rb = g.rb;
            }
            bool have_prev = false, o_started = false;
            int prev_valid = kTileN, prev_n16 = kTileN;
            uint32_t prev_vs = 0, prev_vphase = 0;
            DevTile next_tile = item.first_tile;
            for (int t = item.tile_begin; t < item.tile_end; ++t) {
                const DevTile tile = next_tile;
                if (t + 1 < item.tile_end) next_tile = p.tiles[t + 1];
                if (!tile_visible(tile, g)) continue;
                const int ksn = kcnt % kNK;
                const uint32_t kphase = (kcnt / kNK) & 1;
                const uint32_t vs = vcnt % kNV, vphase = (vcnt / kNV) & 1;
                const uint32_t tile_no = kcnt;                     // visible tiles of the CTA before this one
                ++kcnt; ++vcnt;
                if (alt && (tile_no & 1u) != static_cast<uint32_t>(w)) {
                    // the other half's tile: this half only lets go of the stages, once they have been filled (an arrival
                    // before that could be counted for the stage's previous tile)
                    if (!wait_all(bar_k_full + 8 * ksn, kphase)) { ok = false; break; }
                    if (lane == 0) mbar_arrive(bar_k_empty + 8 * ksn);
                    if (!wait_all(bar_v_full + 8 * vs, vphase)) { ok = false; break; }
                    if (lane == 0) mbar_arrive(bar_v_empty + 8 * vs);
                    continue;
                }
                if (!wait_all(bar_k_full + 8 * ksn, kphase)) { ok = false; break; }
                const uint32_t k_base = smem_u32(k_smem + ksn * kTileBytes);
                if (STATS) {
                    // no product with V in this pass: the next S may be written once the softmax threads have read the
                    // previous one into registers (they say so on the first of the P barriers), also across items
                    if (s_pending) {
                        if (!wait_all(my_p_full, pcnt & 1)) { ok = false; break; }
                        ++pcnt;
                    }
                    tc_fence_after();
                    issue_qk(k_base);
                    mma_commit_elect(leader, my_s_full);
                    mma_commit_elect(leader, bar_k_empty + 8 * ksn);
                    s_pending = true;
                    continue;
                }
                if (have_prev) {
                    if (!pv_prev(prev_vs, prev_vphase, prev_valid, prev_n16, o_started)) { ok = false; break; }
                    o_started = true;
                }
                tc_fence_after();
                issue_qk(k_base);
                mma_commit_elect(leader, my_s_full);               // first: the softmax threads wait on this one
                mma_commit_elect(leader, bar_k_empty + 8 * ksn);
                if (prev_v_release) mma_commit_elect(leader, prev_v_release);
                if (pending_q_release) mma_commit_elect(leader, pending_q_release);
                prev_v_release = 0; pending_q_release = 0;
                {
                    int n_keys = tile.n_valid;                     // keys any row of the block may see
                    if (tile.flags & TILE_CAUSAL) n_keys = min(n_keys, g.last_tok + g.off - tile.key_base + 1);
                    prev_n16 = (n_keys + 15) & ~15;
                }
                have_prev = true; prev_valid = min(tile.n_valid, prev_n16); prev_vs = vs; prev_vphase = vphase;
            }
            if (ok && have_prev) {
                // drain: the last tile's O += P V; o_full tells the softmax threads that O is final
                if (!pv_prev(prev_vs, prev_vphase, prev_valid, prev_n16, o_started)) { ok = false; break; }
                // o_full only: the stage release waits for the next item's first product (nobody needs it sooner than that,
                // and after the last item nobody needs it at all)
                mma_commit_elect(leader, my_o_full);
            }
        }
        if (!ok) {
            // let the tensor pipe drain (bounded) before the tensor memory is released
            if (lane == 0) mma_commit(bar_done);
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_done, 0) && clock64() - t0 < (1ll << 24)) {}
        }
    } else if (warp < 8) {
        // =============================== softmax + epilogue ==========================================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        const int w = warp >> 2;
        const int r_local = (warp & 3) * 32 + lane;
        const int R = w * kHalfRows + r_local;                      // row inside the 256-row block
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_base + (w ? kColS1 : kColS0);
        const uint32_t tO = tmem_base + lane_base + (w ? kColO1 : kColO0);
        const uint32_t my_s_full = bar_s_full + 8 * w, my_p_full = bar_p_full + 32 * w, my_o_full = bar_o_full + 8 * w;
        uint32_t scnt = 0, ocnt = 0, q_loads = 0, tcnt = 0;         // tcnt: visible tiles of the CTA so far (either half's)
        int last_req = -1, last_head = -1, last_rb = -1;
        bool ok = true;

        for (int it = item_begin; it < item_end && ok; ++it) {
            const DevItem item = p.items[it];
            if (it + 1 < item_end) prefetch_l1(&p.items[it + 1]);       // the next item's record is in cache when its turn comes
            if (sib >= item.n_sib) continue;
            if (STATS && item.seg != SEG_CTX) continue;
            const DevReq rq{item.q_row0, item.q_len, item.l_k, 0};
            const ItemGeom g = geom(item, rq);
            if (!(item.req == last_req && item.kv_head == last_head && g.rb == last_rb)) {
                ++q_loads; last_req = item.req; last_head = item.kv_head; last_rb = g.rb;
            }
            const int Rq = alt ? r_local : R;                       // row of the block whose query this thread holds
            const int tok = g.rb * TB + Rq / G;
            const int hg = Rq % G;
            const bool live = tok < rq.q_len;
            const float scale = (item.seg == SEG_CTX) ? p.scale_ctx_log2 : p.scale_oth_log2;
            float m = -INFINITY, l = 0.f;
            int n_local = 0;
            // two-pass plans: this thread's row among all query rows of the plan, and the bias of the tile's node for it
            const bool node_tiles = (STATS || BIAS) && item.seg == SEG_CTX;
            const int64_t stat_row = node_tiles ? (static_cast<int64_t>(item.ctx_id) + (live ? tok : 0)) * p.H_q + item.kv_head * G + hg : 0;
            float b_cur = 0.f, b_next = 0.f;
            if (BIAS && node_tiles) b_next = p.bias[static_cast<int64_t>(item.first_tile.key_base) * p.stat_rows + stat_row];

            DevTile next_tile = item.first_tile;
            for (int t = item.tile_begin; t < item.tile_end; ++t) {
                const DevTile tile = next_tile;
                if (t + 1 < item.tile_end) next_tile = p.tiles[t + 1];      // in flight while this tile is processed
                if (!tile_visible(tile, g)) continue;
                if (alt && (tcnt++ & 1u) != static_cast<uint32_t>(w)) continue;   // the other half's tile
                if (BIAS) {
                    // the next tile's record has had a whole tile to arrive: ask for its node's bias now, use it next time
                    b_cur = b_next;
                    if (node_tiles && t + 1 < item.tile_end)
                        b_next = p.bias[static_cast<int64_t>(next_tile.key_base) * p.stat_rows + stat_row];
                }
                if (!__all_sync(0xffffffffu, mbar_wait(my_s_full, scnt & 1, &abort_flag, p.status))) { ok = false; break; }
                ++scnt;
                tc_fence_after();
                float s[kTileN];
                {
                    uint32_t (*sr)[32] = reinterpret_cast<uint32_t (*)[32]>(s);
                    #pragma unroll
                    for (int c = 0; c < kTileN / 32; ++c) tmem_ld32(tS + c * 32, sr[c]);
                    tmem_ld_wait();
                }
                if (STATS) {                                           // S is in registers: the next product may overwrite it
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(my_p_full);
                }
                int limit = tile.n_valid;
                if (tile.flags & TILE_CAUSAL) limit = min(limit, tok + g.off - tile.key_base + 1);
                if (limit < kTileN) {
                    #pragma unroll
                    for (int i = 0; i < kTileN; ++i) s[i] = (i < limit) ? s[i] : -INFINITY;
                }
                // eight independent running maxima (3-input max) keep the dependency chain short
                float mxa[8];
                #pragma unroll
                for (int k = 0; k < 8; ++k) mxa[k] = max3(s[k], s[8 + k], s[16 + k]);
                #pragma unroll
                for (int i = 24; i < kTileN - 8; i += 16) {
                    #pragma unroll
                    for (int k = 0; k < 8; ++k) mxa[k] = max3(mxa[k], s[i + k], s[i + 8 + k]);
                }
                #pragma unroll
                for (int k = 0; k < 8; ++k) mxa[k] = fmaxf(mxa[k], s[kTileN - 8 + k]);
                const float mx = fmaxf(max3(mxa[0], mxa[1], mxa[2]), fmaxf(max3(mxa[3], mxa[4], mxa[5]), fmaxf(mxa[6], mxa[7])));
                const float m_new = fmaxf(m, BIAS ? mx * scale + b_cur : mx * scale);
                if (STATS) {
                    // no accumulator to keep consistent: the running sum simply follows the maximum
                    l *= (m == -INFINITY) ? 0.f : fast_exp2(m - m_new);
                    m = m_new;
                } else if (n_local == 0) {
                    m = m_new;
                } else {
                    const bool grow = m_new > m + kRescaleThreshold;
                    if (__any_sync(0xffffffffu, grow)) {
                        // S of this tile is complete, so every earlier O += P V of this half is complete too, and the
                        // next one cannot start before this thread has published P: O is quiescent here.
                        const float f = grow ? fast_exp2(m - m_new) : 1.f;
                        l *= f;
                        #pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tO + c * 32, o);
                            tmem_ld_wait();
                            #pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                            tmem_st32(tO + c * 32, o);
                        }
                        tmem_st_wait();
                        if (grow) m = m_new;
                    }
                }
                const float m_use = (m == -INFINITY) ? 0.f : m;
                // The two halves take turns in the exponential phase: the special-function unit is the scarcest pipe, and
                // alternating keeps one half in its exponentials while the other half's MMAs run.  Phase n of half 0 follows
                // phase n-1 of half 1; phase n of half 1 follows phase n of half 0 (both halves see the same tiles).
                // (Alternating halves work on different tiles, with different numbers of them: no turns there.)
                if (!alt) {
                    const uint32_t n = scnt - 1;
                    bool turn = true;
                    if (w == 0) { if (n > 0) turn = mbar_wait(bar_tok, (n - 1) & 1, &abort_flag, p.status); }
                    else turn = mbar_wait(bar_tok + 8, n & 1, &abort_flag, p.status);
                    if (!__all_sync(0xffffffffu, turn)) { ok = false; break; }
                }
                // p = 2^(s * scale - m): the multiply-subtract and the row sum run as packed two-float operations
                const uint64_t scale2 = pack2(scale, scale), negm2 = BIAS ? pack2(b_cur - m_use, b_cur - m_use) : pack2(-m_use, -m_use);
                uint64_t sum2[2] = {0ull, 0ull};
                // P is computed and published in quarters of 32 keys (16 packed registers): the PV product over a quarter
                // runs while the next quarter's exponentials are computed, and only the last quarter's product plus the
                // next S = Q K^T remain on this half's critical path.
                #pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    if constexpr (STATS) {                                 // the sums only: nothing goes back to tensor memory
                        #pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float x0, x1;
                            unpack2(fma2(pack2(s[qq * 32 + 2 * i], s[qq * 32 + 2 * i + 1]), scale2, negm2), x0, x1);
                            sum2[i & 1] = add2(sum2[i & 1], pack2(fast_exp2(x0), fast_exp2(x1)));
                        }
                        if (qq == 3) {
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_tok + 8 * (1 - w));
                        }
                    } else {
                        uint32_t pk[16];
                        #pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float x0, x1;
                            unpack2(fma2(pack2(s[qq * 32 + 2 * i], s[qq * 32 + 2 * i + 1]), scale2, negm2), x0, x1);
                            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                            sum2[i & 1] = add2(sum2[i & 1], pack2(p0, p1));
                            pk[i] = pack_bf16x2(p0, p1);
                        }
                        if (qq == 3 && !alt) {                             // exponentials issued: the other half's turn
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_tok + 8 * (1 - w));
                        }
                        tmem_st16(tS + qq * 16, pk);
                        tmem_st_wait();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(my_p_full + 8 * qq);
                    }
                }
                float sum[4];
                unpack2(sum2[0], sum[0], sum[1]);
                unpack2(sum2[1], sum[2], sum[3]);
                l += (sum[0] + sum[1]) + (sum[2] + sum[3]);
                ++n_local;
                if (STATS && (tile.flags & TILE_CTX_END)) {
                    // the node's own tokens end here: its (maximum, sum) for this row, and a fresh start for the next node
                    if (live) p.stats[static_cast<int64_t>(tile.key_base) * p.stat_rows + stat_row] = make_float2(m, l);
                    m = -INFINITY; l = 0.f; n_local = 0;
                }
            }
            if (!ok) break;
            if (STATS) continue;                                        // no output in the statistics pass

            // ---- epilogue of the item -------------------------------------------------------------------------------
            if (n_local > 0) {
                if (!__all_sync(0xffffffffu, mbar_wait(my_o_full, ocnt & 1, &abort_flag, p.status))) { ok = false; break; }
                ++ocnt;
                tc_fence_after();
            }
            if (item.seg == SEG_FINAL) {
                const float inv = (l > 0.f) ? 1.f / l : 0.f;
                const int h = item.kv_head * G + hg;
                __nv_bfloat16* dst = p.out.data + static_cast<int64_t>(rq.q_row0 + tok) * p.out.token_stride
                                     + static_cast<int64_t>(h) * p.out.head_stride;
                const bool wide_ok = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
                if (o_via_tma && half_is_full(rq, g, w)) {
                    // The item's Q buffer is free (O is final, so every S = Q K^T that read it is done) and has the layout
                    // the bulk store wants: row r of the half, 16-byte chunk j of a 128-byte line at chunk j ^ (r mod 8).
                    uint8_t* stage = q_smem + ((q_loads - 1) % QBUF) * kQBytes + w * kTileBytes + r_local * 128;
                    #pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tO + c * 32, o);
                        tmem_ld_wait();
                        #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(o[8 * j + 0]) * inv, __uint_as_float(o[8 * j + 1]) * inv);
                            v.y = pack_bf16x2(__uint_as_float(o[8 * j + 2]) * inv, __uint_as_float(o[8 * j + 3]) * inv);
                            v.z = pack_bf16x2(__uint_as_float(o[8 * j + 4]) * inv, __uint_as_float(o[8 * j + 5]) * inv);
                            v.w = pack_bf16x2(__uint_as_float(o[8 * j + 6]) * inv, __uint_as_float(o[8 * j + 7]) * inv);
                            const int chunk = (c & 1) * 4 + j;
                            *reinterpret_cast<uint4*>(stage + (c >> 1) * kSlabBytes + ((chunk ^ (r_local & 7)) << 4)) = v;
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_o_staged + 8 * w);
                } else
                #pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_ld_wait();
                    if (live) {
                        uint32_t pk[16];
                        #pragma unroll
                        for (int i = 0; i < 16; ++i)
                            pk[i] = pack_bf16x2(__uint_as_float(o[2 * i]) * inv, __uint_as_float(o[2 * i + 1]) * inv);
                        if (wide_ok) {                 // 32-byte stores: one full sector per instruction
                            st_global_v8(dst + c * 32, pk[0], pk[1], pk[2], pk[3], pk[4], pk[5], pk[6], pk[7]);
                            st_global_v8(dst + c * 32 + 16, pk[8], pk[9], pk[10], pk[11], pk[12], pk[13], pk[14], pk[15]);
                        } else {
                            #pragma unroll
                            for (int i = 0; i < 4; ++i)
                                *reinterpret_cast<uint4*>(dst + c * 32 + i * 8) = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                        }
                    }
                }
                if (live && p.lse_out != nullptr)
                    p.lse_out[static_cast<int64_t>(rq.q_row0 + tok) * p.H_q + h] = (l > 0.f) ? (m + fast_log2(l)) * kLn2 : -INFINITY;
            } else {
                const size_t row = static_cast<size_t>(item.slot + sib) * kAttnRows + R;
                if (n_local > 0) {
                    float* dst = p.ws_o + row * D;
                    #pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tO + c * 32, o);
                        tmem_ld_wait();
                        if (live) {                        // workspace rows are 256-byte aligned
                            #pragma unroll
                            for (int i = 0; i < 4; ++i)
                                st_global_v8(dst + c * 32 + i * 8, o[8 * i], o[8 * i + 1], o[8 * i + 2], o[8 * i + 3],
                                             o[8 * i + 4], o[8 * i + 5], o[8 * i + 6], o[8 * i + 7]);
                        }
                    }
                }
                if (live) *reinterpret_cast<float2*>(p.ws_ml + row * 2) = make_float2(m, (n_local > 0) ? l : 0.f);
            }
        }
    }

    else {
        // =============================== warp 11: Q producer of the double-buffered configuration ==========================
        // With two Q buffers the loads of Q run in their own thread, one row block ahead of the MMAs, instead of queueing
        // behind the K/V loads of the current item.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
        if (QBUF == 2 && lane == 0) {
            tma_prefetch_desc(&tm_q);
            if (o_via_tma) tma_prefetch_desc(&tm_o);
            uint32_t q_loads = 0, staged[2] = {0, 0};
            int last_req = -1, last_head = -1, last_rb = -1;
            bool ok = true;
            // what the bulk store of a row block needs, kept for the two row blocks whose buffers are in use
            struct Pending { int head0, tok0; bool full[2]; } pend[2] = {{0, 0, {false, false}}, {0, 0, {false, false}}};
            // O of the row block that used buffer qb: wait for each staged half, send it, and return once the copies have
            // read the buffer (it is about to be refilled with the next Q).
            auto drain = [&](uint32_t qb) {
                bool any = false;
                #pragma unroll
                for (int w = 0; w < 2; ++w) {
                    if (!pend[qb].full[w]) continue;
                    if (!mbar_wait(bar_o_staged + 8 * w, staged[w] & 1, &abort_flag, p.status)) return false;
                    ++staged[w];
                    #pragma unroll
                    for (int sl = 0; sl < kSlabs; ++sl)
                        tma_store_3d(&tm_o, smem_u32(q_smem + qb * kQBytes + w * kTileBytes + sl * kSlabBytes),
                                     sl * 64, pend[qb].head0, pend[qb].tok0 + w * (kHalfRows / G));
                    any = true;
                }
                if (any) { bulk_commit_group(); bulk_wait_read_all(); }
                pend[qb].full[0] = pend[qb].full[1] = false;
                return true;
            };
            for (int it = item_begin; it < item_end && ok; ++it) {
                const DevItem item = p.items[it];
                if (it + 1 < item_end) prefetch_l1(&p.items[it + 1]);   // the next item's record is in cache when its turn comes
                if (sib >= item.n_sib) continue;
                const DevReq rq{item.q_row0, item.q_len, item.l_k, 0};
                const ItemGeom g = geom(item, rq);
                if (item.req == last_req && item.kv_head == last_head && g.rb == last_rb) continue;
                const uint32_t qb = q_loads % QBUF;
                if (o_via_tma && !drain(qb)) { ok = false; break; }
                if (!load_q(item, rq, g, q_loads)) { ok = false; break; }
                if (o_via_tma && item.seg == SEG_FINAL) {
                    pend[qb].head0 = item.kv_head * G; pend[qb].tok0 = rq.q_row0 + g.rb * TB;
                    pend[qb].full[0] = half_is_full(rq, g, 0); pend[qb].full[1] = half_is_full(rq, g, 1);
                }
                ++q_loads; last_req = item.req; last_head = item.kv_head; last_rb = g.rb;
            }
            if (ok && o_via_tma) {                                  // the last two row blocks, oldest first
                ok = drain(q_loads % QBUF) && drain((q_loads + 1) % QBUF);
            }
            if (!ok) {
                const long long t0 = clock64();
                for (uint32_t b = 0; b < 2; ++b) {
                    const uint32_t issued = (q_loads > b) ? (q_loads - 1 - b) / 2 + 1 : 0;
                    while (issued && !mbar_try_wait(bar_q_full + 8 * b, (issued - 1) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    }

    // ---- teardown: every role has left its loop (normally or on an abort) ----------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

size_t attn_smem_bytes(int D, int mode) {
    const size_t tile = static_cast<size_t>(D / 64) * kSlabBytes;
    // Q halves + K stages + V stages
    const int tiles = (mode == kAttnAlt) ? (1 + 3 + 3) : (mode == kAttnEncode) ? (4 + 2 + 1) : (2 + 2 + 2);
    return 1024 + tiles * tile + 512;
}

// The register hand-over only works if the registers that the third warpgroup gives up cover what the two softmax
// warpgroups ask for: setmaxnreg.inc waits, without a bound, until they are there.  The launch-time register count is
// the compiler's choice, so it is checked here, on the host, before the kernel is ever launched.
template <typename K>
static cudaError_t check_register_handover(K kernel) {
    cudaFuncAttributes attr;
    const cudaError_t e = cudaFuncGetAttributes(&attr, kernel);
    if (e != cudaSuccess) return e;
    const int freed = (attr.numRegs - kRegsOther) * 128;
    const int wanted = (kRegsSoftmax - attr.numRegs) * 256;
    return (attr.numRegs >= kRegsOther && attr.numRegs <= kRegsSoftmax && freed >= wanted) ? cudaSuccess : cudaErrorLaunchOutOfResources;
}

template <typename K>
static cudaError_t prepare_kernel(K kernel, int smem_bytes) {
    const cudaError_t e = check_register_handover(kernel);
    return e != cudaSuccess ? e : cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
}

template <int D>
static cudaError_t prepare_mode(int mode, int n) {
    switch (mode) {
        case kAttnPrefill: return prepare_kernel(ape_attn_kernel<D, kAttnPrefill>, n);
        case kAttnEncode:  return prepare_kernel(ape_attn_kernel<D, kAttnEncode>, n);
        case kAttnAlt:     return prepare_kernel(ape_attn_kernel<D, kAttnAlt>, n);
        case kAttnStats:   return prepare_kernel(ape_attn_kernel<D, kAttnStats>, n);
        case kAttnBias:    return prepare_kernel(ape_attn_kernel<D, kAttnBias>, n);
    }
    return cudaErrorInvalidValue;
}

cudaError_t attn_set_smem_attr(int D, int mode, size_t smem_bytes) {
    const int n = static_cast<int>(smem_bytes);
    return D == 128 ? prepare_mode<128>(mode, n) : prepare_mode<64>(mode, n);
}

template <int D>
static void launch_mode(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const CUtensorMap& tm_o,
                        const SplitMaps& split, const AttnParams& p, int n_cta, size_t smem_bytes, cudaStream_t stream) {
    switch (p.mode) {
        case kAttnPrefill: ape_attn_kernel<D, kAttnPrefill><<<n_cta, kThreads, smem_bytes, stream>>>(tm_q, tm_k, tm_v, tm_o, split, p); break;
        case kAttnEncode:  ape_attn_kernel<D, kAttnEncode><<<n_cta, kThreads, smem_bytes, stream>>>(tm_q, tm_k, tm_v, tm_o, split, p); break;
        case kAttnAlt:     ape_attn_kernel<D, kAttnAlt><<<n_cta, kThreads, smem_bytes, stream>>>(tm_q, tm_k, tm_v, tm_o, split, p); break;
        case kAttnStats:   ape_attn_kernel<D, kAttnStats><<<n_cta, kThreads, smem_bytes, stream>>>(tm_q, tm_k, tm_v, tm_o, split, p); break;
        case kAttnBias:    ape_attn_kernel<D, kAttnBias><<<n_cta, kThreads, smem_bytes, stream>>>(tm_q, tm_k, tm_v, tm_o, split, p); break;
        default: break;
    }
}

cudaError_t launch_attn(int D, const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const CUtensorMap& tm_o,
                        const SplitMaps& split, const AttnParams& p, int n_cta, size_t smem_bytes, cudaStream_t stream)
{
    if (p.mode < kAttnPrefill || p.mode > kAttnBias) return cudaErrorInvalidValue;
    if (D == 128) launch_mode<128>(tm_q, tm_k, tm_v, tm_o, split, p, n_cta, smem_bytes, stream);
    else launch_mode<64>(tm_q, tm_k, tm_v, tm_o, split, p, n_cta, smem_bytes, stream);
    return cudaGetLastError();
}

}  // namespace ape
