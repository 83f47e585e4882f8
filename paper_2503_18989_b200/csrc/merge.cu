// Split-KV merge: combine the partial (out, lse) rows of one query row computed over disjoint key
// ranges.  One warp per (row, head): lane s holds lse_s, the maximum and the sum of exp are
// warp-shuffle reductions, and each lane then accumulates its slice of head_dim over the parts.
#include "hat_internal.h"

namespace hat {

template <int D>
__global__ void __launch_bounds__(128)
merge_kernel(const MergeRow* __restrict__ rows, int num_rows, int H,
             const float* __restrict__ part_out, const float* __restrict__ part_lse,
             float* __restrict__ out, float* __restrict__ lse, void* __restrict__ out16, int out16_bf16) {
    const int lane = threadIdx.x & 31;
    const int64_t unit = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);     // (row, head) pair
    if (unit >= (int64_t)num_rows * H) return;
    const MergeRow mr = rows[unit / H];
    const int h = (int)(unit % H);

    float my = -INFINITY;
    if (lane < mr.nsplit) my = part_lse[((int64_t)mr.part0 + (int64_t)lane * mr.stride) * H + h];
    float mx = my;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float ms = (mx == -INFINITY) ? 0.f : mx;
    float w = expf(my - ms);                                             // 0 for empty parts and idle lanes
    float sum = w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = sum > 0.f ? 1.f / sum : 0.f;
    w *= inv;

    constexpr int V = D / 32;                                              // floats per lane
    float acc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) acc[k] = 0.f;
    for (int s = 0; s < mr.nsplit; ++s) {
        const float ws = __shfl_sync(0xffffffffu, w, s);
        const float* src = part_out + (((int64_t)mr.part0 + (int64_t)s * mr.stride) * H + h) * D + lane * V;
        if constexpr (V == 4) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(src));
            acc[0] += ws * v.x; acc[1] += ws * v.y; acc[2] += ws * v.z; acc[3] += ws * v.w;
        } else {
            const float2 v = __ldg(reinterpret_cast<const float2*>(src));
            acc[0] += ws * v.x; acc[1] += ws * v.y;
        }
    }
    const int64_t at = ((int64_t)mr.row * H + h) * D + lane * V;
    if (out16 != nullptr) {
        uint16_t* dst = static_cast<uint16_t*>(out16) + at;
        if constexpr (V == 4)
            *reinterpret_cast<uint2*>(dst) = make_uint2(pack_out16(acc[0], acc[1], out16_bf16), pack_out16(acc[2], acc[3], out16_bf16));
        else
            *reinterpret_cast<uint32_t*>(dst) = pack_out16(acc[0], acc[1], out16_bf16);
    } else if constexpr (V == 4) {
        *reinterpret_cast<float4*>(out + at) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    } else {
        *reinterpret_cast<float2*>(out + at) = make_float2(acc[0], acc[1]);
    }
    if (lane == 0) lse[(int64_t)mr.row * H + h] = sum > 0.f ? ms + logf(sum) : -INFINITY;
}

cudaError_t launch_merge(const hat_plan* plan, const AttnArgs& args, int first_row, int num_rows, cudaStream_t stream) {
    const int n = num_rows;
    if (n <= 0) return cudaSuccess;
    const int H = plan->num_heads;
    const int64_t units = (int64_t)n * H;
    const unsigned blocks = (unsigned)((units + 3) / 4);
    if (plan->head_dim == 128)
        merge_kernel<128><<<blocks, 128, 0, stream>>>(plan->dev.merge_rows + first_row, n, H, args.part_out, args.part_lse,
                                                      args.out, args.lse, args.out16, args.out16_bf16);
    else
        merge_kernel<64><<<blocks, 128, 0, stream>>>(plan->dev.merge_rows + first_row, n, H, args.part_out, args.part_lse,
                                                     args.out, args.lse, args.out16, args.out16_bf16);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hat
