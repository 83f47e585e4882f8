// Rotary position encoding fused into the KV append, and the same rotation for the query rows.
//
// The decoder layers of the paper's models (Vicuna-7B/13B, Sec. 4.1) rotate query and key rows by their token position
// before the attention of Sec. 2.1, and the cache stores the rotated keys.  Row i of request r has position
// p = prefix_len[r] + i; pair c of a head (c = 0 .. d/2 - 1) turns by p * theta^(-2c/d).  Pairs are (x[c], x[c + d/2])
// or, interleaved, (x[2c], x[2c + 1]).  The angle is formed and reduced to [-pi, pi] in double (at position 8000 an fp32
// angle is already off by more than the 16-bit result resolves), sine, cosine and the rotation run in fp32, and the
// result is rounded to the 16-bit type once.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cmath>

#include "hat_internal.h"

namespace hat {
namespace {

template <bool BF16>
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    if constexpr (BF16) return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    else {
        const __half2 h = *reinterpret_cast<const __half2*>(&w);
        return __half22float2(h);
    }
}

// One thread: for one packed row, one 16-byte vector of the low half of a head and its partner in the high half (or,
// interleaved, two neighbouring vectors) = 8 pairs, for kHeadsPerThread heads in turn: the 8 sines and cosines depend on
// the row and the pair only and are computed once for them.  `to_cache`: rows are K rows and go to their slot of the pool, with the matching
// V vectors copied as they come; otherwise rows are written to `dst` at their packed position (query rows).
template <bool BF16, int kHeadsPerThread>
__global__ void __launch_bounds__(256)
rope_kernel(DevicePlan plan, int heads, int d, const __grid_constant__ InvFreq fr, int interleaved, const uint4* __restrict__ src,
            uint4* __restrict__ dst, int to_cache, int64_t stride_page, int64_t stride_token, int64_t stride_head,
            uint4* __restrict__ k_pool, uint4* __restrict__ v_pool, const uint4* __restrict__ v_new, int64_t total) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int vec_per_head = d / 8, pairs_vec = vec_per_head / 2;        // vectors per head, vector pairs per head
    const int groups = (heads + kHeadsPerThread - 1) / kHeadsPerThread;
    const int t = (int)(idx / ((int64_t)groups * pairs_vec));
    const int within = (int)(idx - (int64_t)t * groups * pairs_vec);
    const int hg = within / pairs_vec, pv = within - hg * pairs_vec;
    const int r = plan.row_req[t];
    const int p = plan.prefix_len[r] + (t - plan.cu_chunk[r]);

    const int va = interleaved ? 2 * pv : pv;                            // the two vectors this thread owns in a head
    const int vb = interleaved ? 2 * pv + 1 : pv + pairs_vec;
    float sn[8], cs[8];                                                  // pair 8 pv + k of every head
#pragma unroll
    for (int k = 0; k < 8; ++k) rope_sincos(p, fr.f[8 * pv + k], &sn[k], &cs[k]);

    int64_t pool_base = 0;
    if (to_cache) {
        const int page = plan.block_table[(int64_t)r * plan.max_pages + p / kPageSize];
        pool_base = ((int64_t)page * stride_page + (int64_t)(p % kPageSize) * stride_token) / 8;
    }
    const int h_end = min(heads, (hg + 1) * kHeadsPerThread);
#pragma unroll 2
    for (int h = hg * kHeadsPerThread; h < h_end; ++h) {
        const int64_t row_vec = ((int64_t)t * heads + h) * vec_per_head;
        uint4 a = __ldg(src + row_vec + va), b = __ldg(src + row_vec + vb);
        uint32_t* aw = reinterpret_cast<uint32_t*>(&a);
        uint32_t* bw = reinterpret_cast<uint32_t*>(&b);
        if (interleaved) {
            // each 32-bit word is one pair: words of a are pairs 8 pv .. +3, words of b pairs 8 pv + 4 .. +7
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 x = unpack2<BF16>(aw[k]), y = unpack2<BF16>(bw[k]);
                aw[k] = pack_out16(x.x * cs[k] - x.y * sn[k], x.y * cs[k] + x.x * sn[k], BF16);
                bw[k] = pack_out16(y.x * cs[k + 4] - y.y * sn[k + 4], y.y * cs[k + 4] + y.x * sn[k + 4], BF16);
            }
        } else {
            // element e of a pairs with element e of b: pair 8 pv + e
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 x = unpack2<BF16>(aw[k]), y = unpack2<BF16>(bw[k]);
                aw[k] = pack_out16(x.x * cs[2 * k] - y.x * sn[2 * k], x.y * cs[2 * k + 1] - y.y * sn[2 * k + 1], BF16);
                bw[k] = pack_out16(y.x * cs[2 * k] + x.x * sn[2 * k], y.y * cs[2 * k + 1] + x.y * sn[2 * k + 1], BF16);
            }
        }
        if (to_cache) {
            const int64_t base = pool_base + (int64_t)h * stride_head / 8;
            k_pool[base + va] = a;
            k_pool[base + vb] = b;
            v_pool[base + va] = __ldg(v_new + row_vec + va);
            v_pool[base + vb] = __ldg(v_new + row_vec + vb);
        } else {
            dst[row_vec + va] = a;
            dst[row_vec + vb] = b;
        }
    }
}

}  // namespace

cudaError_t launch_rope(const hat_plan* plan, int heads, float theta, int interleaved, const void* src, void* dst,
                        const CacheView* cache, void* k_pool, void* v_pool, const void* v_new, cudaStream_t stream) {
    const int d = plan->head_dim;
    // measured: the append (K and V traffic per thread) is fastest with one head per thread, the query rotation with four
    const int hpt = cache != nullptr ? 1 : 4;
    const int64_t total = (int64_t)plan->total_rows * ((heads + hpt - 1) / hpt) * (d / 16);
    if (total == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    InvFreq fr;
    for (int c = 0; c < d / 2; ++c) fr.f[c] = std::pow((double)theta, -2.0 * c / d);
    const int to_cache = cache != nullptr;
    const int64_t sp = to_cache ? cache->stride_page : 0, st = to_cache ? cache->stride_token : 0,
                  sh = to_cache ? cache->stride_head : 0;
    auto launch = [&](auto kern) {
        kern<<<blocks, 256, 0, stream>>>(plan->dev, heads, d, fr, interleaved, static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                         to_cache, sp, st, sh, static_cast<uint4*>(k_pool), static_cast<uint4*>(v_pool),
                                         static_cast<const uint4*>(v_new), total);
    };
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    if (to_cache) { if (bf16) launch(rope_kernel<true, 1>); else launch(rope_kernel<false, 1>); }
    else { if (bf16) launch(rope_kernel<true, 4>); else launch(rope_kernel<false, 4>); }
    count_launch();
    return cudaGetLastError();
}

}  // namespace hat
