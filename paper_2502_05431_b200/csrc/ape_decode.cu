// Split-KV decode kernel of APE attention: one new query token per request streams the whole cached
// sequence [prefix | contexts | query segment] once.  HBM-bound: K/V tiles are brought in by the bulk
// tensor copy engine through a multi-stage shared-memory ring; the small (G rows) x (16 tokens) products run on
// warp-level mma so that arithmetic never limits the stream.  Each work item covers tiles of ONE segment
// (context, or prefix + query segment) and emits one partial (m, l, O~) in base-2 units; the merge kernel
// applies the hierarchical softmax identity and Eq. 5's S afterwards.
#include "ape_common.cuh"
#include "ape_kernels.h"

namespace ape {

namespace {

constexpr int kTile = kDecodeTile;          // tokens per stage
constexpr int kConsumerWarps = 8;           // two groups of four; group w/4 takes every other tile
constexpr int kThreads = (kConsumerWarps + 1) * 32;

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of token row `row` inside a K or V stage that the copy engine
// wrote as D/64 slabs of [kTile rows][128 B] with the 128-byte swizzle.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return static_cast<uint32_t>((chunk >> 3) * (kTile * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
ape_decode_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const DecodeParams p)
{
    constexpr int kSlabs = D / 64;
    constexpr int kStageBytes = 2 * kTile * D * 2;      // K + V
    constexpr int kKSteps = D / 16;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int n_stages = p.n_stages;
    uint8_t* stage_base = smem;
    float* red = reinterpret_cast<float*>(smem + static_cast<size_t>(n_stages) * kStageBytes);  // [8][G][D], [8][16] m, [8][16] l
    float* red_m = red + kConsumerWarps * p.G * D;
    float* red_l = red_m + kConsumerWarps * 16;
    uint64_t* bars = reinterpret_cast<uint64_t*>(red_l + kConsumerWarps * 16);   // full[n_stages], empty[n_stages]
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + n_stages);

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 4);       // one arrival per warp of the group that consumed the stage
        }
        mbar_fence_init();
    }
    __syncthreads();

    const int item_begin = p.cta_item_begin[blockIdx.x], item_end = p.cta_item_begin[blockIdx.x + 1];

    if (warp == kConsumerWarps) {
        // ---------------- producer: one lane feeds the ring --------------------------------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&tm_k);
            tma_prefetch_desc(&tm_v);
            uint32_t cnt = 0;
            bool ok = true;
            for (int it = item_begin; it < item_end && ok; ++it) {
                const DevItem item = p.items[it];
                for (int t = item.tile_begin; t < item.tile_end; ++t, ++cnt) {
                    const int s = cnt % n_stages;
                    const uint32_t use = cnt / n_stages;
                    if (!mbar_wait(bar_empty + 8 * s, (use & 1) ^ 1, &abort_flag, p.status)) { ok = false; break; }
                    const int tok = p.tiles[t].tok;
                    const uint32_t dst = smem_u32(stage_base + static_cast<size_t>(s) * kStageBytes);
                    mbar_expect_tx(bar_full + 8 * s, kStageBytes);
                    #pragma unroll
                    for (int sl = 0; sl < kSlabs; ++sl) {
                        tma_load_3d(dst + sl * (kTile * 128), &tm_k, bar_full + 8 * s, sl * 64, item.kv_head, tok);
                        tma_load_3d(dst + kTile * D * 2 + sl * (kTile * 128), &tm_v, bar_full + 8 * s, sl * 64, item.kv_head, tok);
                    }
                }
            }
            // Nothing may still be landing in shared memory when the CTA exits: on an abort, wait (bounded) for the
            // copies already issued.  In the normal case the consumers have waited on every stage already.
            if (!ok) {
                for (int s = 0; s < n_stages; ++s) {
                    const long long t0 = clock64();
                    const uint32_t issued = (cnt > static_cast<uint32_t>(s)) ? (cnt - 1 - s) / n_stages + 1 : 0;
                    if (issued == 0) continue;
                    while (!mbar_try_wait(bar_full + 8 * s, (issued - 1) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else {
        // ---------------- consumers ----------------------------------------------------------------------------------
        const int grp = warp >> 2;            // which half of the tiles
        const int w4 = warp & 3;              // 16-token slice inside a tile
        const int G = p.G;
        const int qr = lane >> 2, qc = lane & 3;
        uint32_t cnt = 0;

        for (int it = item_begin; it < item_end; ++it) {
            const DevItem item = p.items[it];
            const DevReq rq = p.reqs[item.req];
            const float scale = (item.seg == SEG_CTX) ? p.scale_ctx_log2 : p.scale_oth_log2;
            const int l_k_now = rq.l_k + p.kv_extra;

            // Q fragments (A operand, 16 x D, rows >= G are zero)
            uint32_t qa[kKSteps][4];
            {
                const __nv_bfloat16* qbase = p.q.data + static_cast<int64_t>(rq.q_row0) * p.q.token_stride
                                             + static_cast<int64_t>(item.kv_head) * G * p.q.head_stride;
                #pragma unroll
                for (int ks = 0; ks < kKSteps; ++ks) {
                    const int col = ks * 16 + 2 * qc;
                    const uint32_t* r_lo = reinterpret_cast<const uint32_t*>(qbase + static_cast<int64_t>(qr) * p.q.head_stride + col);
                    const uint32_t* r_hi = reinterpret_cast<const uint32_t*>(qbase + static_cast<int64_t>(qr + 8) * p.q.head_stride + col);
                    qa[ks][0] = (qr < G) ? __ldg(r_lo) : 0u;
                    qa[ks][1] = (qr + 8 < G) ? __ldg(r_hi) : 0u;
                    qa[ks][2] = (qr < G) ? __ldg(r_lo + 4) : 0u;
                    qa[ks][3] = (qr + 8 < G) ? __ldg(r_hi + 4) : 0u;
                }
            }

            float o[D / 8][4];
            #pragma unroll
            for (int j = 0; j < D / 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
            float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

            for (int t = item.tile_begin; t < item.tile_end; ++t, ++cnt) {
                if ((cnt & 1u) != static_cast<uint32_t>(grp)) continue;
                const int s = cnt % n_stages;
                const uint32_t use = cnt / n_stages;
                const DevTile tile = p.tiles[t];
                int n_valid = tile.n_valid;
                if (tile.flags & TILE_GROWS) n_valid = min(max(l_k_now - tile.key_base, 0), kTile);
                if (!mbar_wait(bar_full + 8 * s, use & 1, &abort_flag, p.status)) break;

                const int tok0 = w4 * 16;
                if (tok0 < n_valid) {
                    const uint32_t k_s = smem_u32(stage_base + static_cast<size_t>(s) * kStageBytes);
                    const uint32_t v_s = k_s + kTile * D * 2;

                    if (n_valid < tok0 + 16) {
                        // ragged tile: V rows past the span may hold anything (even NaN); zero them so that 0 * v stays 0
                        const int row = tok0 + (lane >> 1);
                        if (row >= n_valid) {
                            uint8_t* vrow = stage_base + static_cast<size_t>(s) * kStageBytes + kTile * D * 2;
                            #pragma unroll
                            for (int sl = 0; sl < kSlabs; ++sl) {
                                uint4* dst = reinterpret_cast<uint4*>(vrow + sl * (kTile * 128) + row * 128 + (lane & 1) * 64);
                                dst[0] = dst[1] = dst[2] = dst[3] = make_uint4(0, 0, 0, 0);
                            }
                            fence_proxy_async_smem();   // these generic writes precede the next bulk copy into the stage
                        }
                        __syncwarp();
                    }

                    // S = Q K^T for 16 tokens: two n-tiles of 8 tokens
                    float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                    {
                        const int row = tok0 + ((lane >> 4) << 3) + (lane & 7);
                        const int chunk_sel = (lane >> 3) & 1;
                        #pragma unroll
                        for (int ks = 0; ks < kKSteps; ++ks) {
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4(k_s + swz(row, 2 * ks + chunk_sel), b0, b1, b2, b3);
                            mma_bf16_16816(sc[0], qa[ks], b0, b1);
                            mma_bf16_16816(sc[1], qa[ks], b2, b3);
                        }
                    }
                    // base-2 logits, validity mask
                    #pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        const int c0 = tok0 + nt * 8 + 2 * qc;
                        const bool v0 = c0 < n_valid, v1 = c0 + 1 < n_valid;
                        sc[nt][0] = v0 ? sc[nt][0] * scale : -INFINITY;
                        sc[nt][1] = v1 ? sc[nt][1] * scale : -INFINITY;
                        sc[nt][2] = v0 ? sc[nt][2] * scale : -INFINITY;
                        sc[nt][3] = v1 ? sc[nt][3] * scale : -INFINITY;
                    }
                    float mx_lo = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
                    float mx_hi = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
                    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);   // finite: the slice holds a valid key
                    if (__any_sync(0xffffffffu, (mn_lo > m_lo) | (mn_hi > m_hi))) {
                        const float f_lo = fast_exp2(m_lo - mn_lo), f_hi = fast_exp2(m_hi - mn_hi);
                        l_lo *= f_lo; l_hi *= f_hi;
                        #pragma unroll
                        for (int j = 0; j < D / 8; ++j) { o[j][0] *= f_lo; o[j][1] *= f_lo; o[j][2] *= f_hi; o[j][3] *= f_hi; }
                        m_lo = mn_lo; m_hi = mn_hi;
                    }
                    uint32_t pa[4];
                    {
                        const float p00 = fast_exp2(sc[0][0] - m_lo), p01 = fast_exp2(sc[0][1] - m_lo);
                        const float p02 = fast_exp2(sc[0][2] - m_hi), p03 = fast_exp2(sc[0][3] - m_hi);
                        const float p10 = fast_exp2(sc[1][0] - m_lo), p11 = fast_exp2(sc[1][1] - m_lo);
                        const float p12 = fast_exp2(sc[1][2] - m_hi), p13 = fast_exp2(sc[1][3] - m_hi);
                        l_lo += (p00 + p01) + (p10 + p11);
                        l_hi += (p02 + p03) + (p12 + p13);
                        pa[0] = pack_bf16x2(p00, p01); pa[1] = pack_bf16x2(p02, p03);
                        pa[2] = pack_bf16x2(p10, p11); pa[3] = pack_bf16x2(p12, p13);
                    }
                    // O += P V
                    {
                        const int row = tok0 + (((lane >> 3) & 1) << 3) + (lane & 7);
                        const int chunk_sel = lane >> 4;
                        #pragma unroll
                        for (int j = 0; j < D / 16; ++j) {
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4_trans(v_s + swz(row, 2 * j + chunk_sel), b0, b1, b2, b3);
                            mma_bf16_16816(o[2 * j], pa, b0, b1);
                            mma_bf16_16816(o[2 * j + 1], pa, b2, b3);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty + 8 * s);
            }

            // ---- combine the eight warps' partials of this item and write one (m, l, O~) to the workspace ------------
            l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
            l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
            if (qc == 0) {
                red_m[warp * 16 + qr] = m_lo; red_m[warp * 16 + qr + 8] = m_hi;
                red_l[warp * 16 + qr] = l_lo; red_l[warp * 16 + qr + 8] = l_hi;
            }
            #pragma unroll
            for (int j = 0; j < D / 8; ++j) {
                const int e = j * 8 + 2 * qc;
                if (qr < G) *reinterpret_cast<float2*>(&red[(warp * G + qr) * D + e]) = make_float2(o[j][0], o[j][1]);
                if (qr + 8 < G) *reinterpret_cast<float2*>(&red[(warp * G + qr + 8) * D + e]) = make_float2(o[j][2], o[j][3]);
            }
            // Every consumer warp reaches this barrier, also one that gave up on a wait, so the decision to stop is
            // taken by all of them together.
            named_bar_sync(1, kConsumerWarps * 32);
            if (abort_flag) break;
            {
                float* ws_o = p.ws_o + static_cast<size_t>(item.slot) * G * D;
                float* ws_ml = p.ws_ml + static_cast<size_t>(item.slot) * G * 2;
                const int tid = threadIdx.x;
                for (int idx = tid; idx < G * D; idx += kConsumerWarps * 32) {
                    const int row = idx / D, e = idx - row * D;
                    float M = -INFINITY;
                    #pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, red_m[w * 16 + row]);
                    const float Ms = (M == -INFINITY) ? 0.f : M;
                    float acc = 0.f, L = 0.f;
                    #pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const float f = fast_exp2(red_m[w * 16 + row] - Ms);
                        acc += f * red[(w * G + row) * D + e];
                        L += f * red_l[w * 16 + row];
                    }
                    ws_o[idx] = acc;
                    if (e == 0) { ws_ml[row * 2] = M; ws_ml[row * 2 + 1] = L; }
                }
            }
            named_bar_sync(1, kConsumerWarps * 32);
        }
    }
}

size_t decode_smem_bytes(int D, int G, int n_stages) {
    return 1024 + static_cast<size_t>(n_stages) * (2 * kTile * D * 2)
           + sizeof(float) * (kConsumerWarps * G * D + 2 * kConsumerWarps * 16) + 16 * n_stages + 64;
}

int decode_pick_stages(int D, int G, size_t smem_limit) {
    int n = 8;
    while (n > 2 && decode_smem_bytes(D, G, n) > smem_limit) --n;
    return decode_smem_bytes(D, G, n) <= smem_limit ? n : 0;
}

cudaError_t launch_decode(int D, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const DecodeParams& p,
                          int n_cta, size_t smem_bytes, cudaStream_t stream)
{
    if (D == 128) {
        ape_decode_kernel<128><<<n_cta, kThreads, smem_bytes, stream>>>(tm_k, tm_v, p);
    } else {
        ape_decode_kernel<64><<<n_cta, kThreads, smem_bytes, stream>>>(tm_k, tm_v, p);
    }
    return cudaGetLastError();
}

cudaError_t decode_set_smem_attr(int D, size_t smem_bytes) {
    if (D == 128)
        return cudaFuncSetAttribute(ape_decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes));
    return cudaFuncSetAttribute(ape_decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes));
}

}  // namespace ape
