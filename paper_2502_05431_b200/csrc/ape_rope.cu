// Rotary position embedding with position re-use, fused with the write into its destination (the KV pool for K and V,
// a query buffer for Q).  Memory-bound: every element is read once and written once; the cosines and sines of a token
// are computed once per token and shared by all its heads through shared memory.
//
// Rotation (Su et al., the embedding named in the paper's Section 2 "Position Embedding"; half-split pairing of the
// Llama family): component i of a head is paired with component i + d/2,
//     out[i]       = x[i] cos(phi_i) - x[i + d/2] sin(phi_i)
//     out[i + d/2] = x[i + d/2] cos(phi_i) + x[i] sin(phi_i),      phi_i = pos * theta^(-2i/d).
// Positions reach 2^17 and beyond, so phi_i is formed and reduced to [-pi, pi] in double precision (a float angle of
// 10^5 radians is only good to 10^-2); the sine and cosine of the reduced angle and the rotation itself are fp32.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ape_kernels.h"

namespace ape {

namespace {

constexpr int kRopeThreads = 256;

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_rn(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D>
__global__ void __launch_bounds__(kRopeThreads)
ape_rope_kernel(const RopeParams p)
{
    constexpr int kHalf = D / 2;               // pairs per head
    constexpr int kVec = D / 16;               // 16-byte vectors per half head
    __shared__ __align__(16) float2 table[2][kRopeChunkTokens][kHalf];       // (cos, sin) of the chunk's tokens, double-buffered

    const int tid = threadIdx.x;
    // kRopeThreads is a multiple of kHalf: a thread always fills the same pair index of the table
    const int my_i = tid % kHalf;
    const double inv_freq = exp2(-(2.0 * my_i / D) * p.log2_theta);
    constexpr double kInv2Pi = 0.15915494309189535;
    constexpr double k2PiHi = 6.283185307179586, k2PiLo = 2.4492935982947064e-16;

    int buf = 0;
    for (int c = blockIdx.x; c < p.n_chunks; c += gridDim.x, buf ^= 1) {
        const RopeChunk ch = p.chunks[c];
        if (p.rotate) {
            for (int e = tid; e < ch.n_tok * kHalf; e += kRopeThreads) {
                const int t = e / kHalf;
                const double ang = static_cast<double>(ch.pos0 + t) * inv_freq;
                const double k = rint(ang * kInv2Pi);
                double r = fma(-k, k2PiHi, ang);
                r = fma(-k, k2PiLo, r);
                float sn, cs;
                __sincosf(static_cast<float>(r), &sn, &cs);       // |r| <= pi: the fast form is good to a few 1e-7 there
                table[buf][t][my_i] = make_float2(cs, sn);
            }
            // One barrier per chunk is enough with two tables: a thread can only reach the fill of this buffer's next
            // use after passing the barrier of the chunk in between, which every thread reaches after its last read here.
            __syncthreads();
        }
        const int n_items = ch.n_tok * p.n_heads * kVec;
        #pragma unroll 4
        for (int it = tid; it < n_items; it += kRopeThreads) {
            const int v = it % kVec;
            const int h = (it / kVec) % p.n_heads;
            const int t = it / (kVec * p.n_heads);
            const __nv_bfloat16* src = p.src.data + static_cast<int64_t>(ch.src_tok + t) * p.src.token_stride
                                       + static_cast<int64_t>(h) * p.src.head_stride + v * 8;
            __nv_bfloat16* dst = p.dst.data + static_cast<int64_t>(ch.dst_tok + t) * p.dst.token_stride
                                 + static_cast<int64_t>(h) * p.dst.head_stride + v * 8;
            const uint4 a = *reinterpret_cast<const uint4*>(src);
            const uint4 b = *reinterpret_cast<const uint4*>(src + kHalf);
            if (!p.rotate) {
                *reinterpret_cast<uint4*>(dst) = a;
                *reinterpret_cast<uint4*>(dst + kHalf) = b;
                continue;
            }
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
            uint32_t lo[4], hi[4];
            // the thread's eight (cos, sin) pairs are 64 contiguous bytes: four 16-byte reads, free of bank conflicts
            const float4* tb = reinterpret_cast<const float4*>(&table[buf][t][v * 8]);
            #pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float4 cs = tb[j];                           // (cos, sin) of pair 2j and of pair 2j + 1
                const float a0 = bf16_lo(aw[j]), a1 = bf16_hi(aw[j]), b0 = bf16_lo(bw[j]), b1 = bf16_hi(bw[j]);
                lo[j] = pack_rn(fmaf(a0, cs.x, -b0 * cs.y), fmaf(a1, cs.z, -b1 * cs.w));
                hi[j] = pack_rn(fmaf(b0, cs.x, a0 * cs.y), fmaf(b1, cs.z, a1 * cs.w));
            }
            *reinterpret_cast<uint4*>(dst) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            *reinterpret_cast<uint4*>(dst + kHalf) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        }
    }
}

// D0 of the decode path: the new token's K and V rows of every request (staged densely, [n_req][H_kv][D]) go to the
// pool row that the request's query segment has reached.  One thread block per request, 16 bytes per thread and turn.
__global__ void __launch_bounds__(128) ape_append_kernel(const AppendParams p)
{
    const int r = blockIdx.x;
    const int64_t row = p.rows[r] + p.kv_extra;
    const int vec_per_head = p.D / 8, n_vec = p.H_kv * vec_per_head;
    for (int i = threadIdx.x; i < 2 * n_vec; i += blockDim.x) {
        const int which = i / n_vec, j = i - which * n_vec;
        const int h = j / vec_per_head, v = j - h * vec_per_head;
        const __nv_bfloat16* src = (which ? p.v_new : p.k_new) + (static_cast<int64_t>(r) * p.H_kv + h) * p.D + v * 8;
        __nv_bfloat16* dst = (which ? p.v_pool : p.k_pool) + row * p.token_stride + static_cast<int64_t>(h) * p.head_stride + v * 8;
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    }
}

}  // namespace

cudaError_t launch_append(const AppendParams& p, cudaStream_t stream) {
    if (p.n_req <= 0) return cudaSuccess;
    ape_append_kernel<<<p.n_req, 128, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_rope(int D, const RopeParams& p, int n_cta, cudaStream_t stream) {
    if (D == 128) ape_rope_kernel<128><<<n_cta, kRopeThreads, 0, stream>>>(p);
    else ape_rope_kernel<64><<<n_cta, kRopeThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace ape
