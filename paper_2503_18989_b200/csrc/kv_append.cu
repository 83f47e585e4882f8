// KV append: scatter the chunk's new K/V rows into the paged pools (bit-exact 16-byte copies).
#include "hat_internal.h"

namespace hat {

// A warp moves 128 consecutive 16-byte vectors of K and the matching 128 of V: vector 32 i + lane in its i-th
// round, so every load and store instruction covers 512 contiguous bytes, and all eight loads of a thread are in
// flight before the page lookups (a chain of dependent loads) and the stores.
// vec_per_row = H * d / 8; vector index -> (packed row t, head, vector within the head).
constexpr int kVecsPerThread = 4;
__global__ void __launch_bounds__(256)
kv_append_kernel(DevicePlan plan, int64_t stride_page, int64_t stride_token, int64_t stride_head,
                 uint4* __restrict__ k_pool, uint4* __restrict__ v_pool,
                 const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                 int vec_per_head, int64_t total_vecs) {
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t first = warp * (32 * kVecsPerThread) + (threadIdx.x & 31);
    uint4 kv[kVecsPerThread], vv[kVecsPerThread];
#pragma unroll
    for (int i = 0; i < kVecsPerThread; ++i)
        if (first + 32 * i < total_vecs) kv[i] = __ldg(k_new + first + 32 * i);
#pragma unroll
    for (int i = 0; i < kVecsPerThread; ++i)
        if (first + 32 * i < total_vecs) vv[i] = __ldg(v_new + first + 32 * i);

    const int vec_per_row = vec_per_head * plan.num_kv_heads;
#pragma unroll
    for (int i = 0; i < kVecsPerThread; ++i) {
        const int64_t idx = first + 32 * i;
        if (idx >= total_vecs) break;
        const int t = (int)(idx / vec_per_row);
        const int within = (int)(idx - (int64_t)t * vec_per_row);
        const int h = within / vec_per_head;
        const int c = within - h * vec_per_head;
        const int r = plan.row_req[HAT_IN_RANGE(t, plan.total_rows, plan.status)];
        const int pos = plan.prefix_len[r] + (t - plan.cu_chunk[r]);     // logical token index
        const int page = HAT_IN_RANGE(plan.block_table[(int64_t)r * plan.max_pages + HAT_IN_RANGE(pos / kPageSize, plan.max_pages, plan.status)],
                                      plan.num_pages, plan.status);
        const int slot = pos % kPageSize;
        // strides are multiples of 8 elements, so the offset in 16-byte vectors is exact
        const int64_t dst = ((int64_t)page * stride_page + (int64_t)slot * stride_token + (int64_t)h * stride_head) / 8 + c;
        k_pool[dst] = kv[i];
        v_pool[dst] = vv[i];
    }
}

cudaError_t launch_kv_append(const hat_plan* plan, const CacheView& cache, void* k_pool, void* v_pool,
                             const void* k_new, const void* v_new, cudaStream_t stream) {
    const int vec_per_head = plan->head_dim / 8;
    const int64_t total = (int64_t)plan->total_rows * plan->num_kv_heads * vec_per_head;
    if (total == 0) return cudaSuccess;
    const int threads = 256;
    const int64_t per_block = (int64_t)threads * kVecsPerThread;
    const int64_t blocks = (total + per_block - 1) / per_block;
    kv_append_kernel<<<(unsigned)blocks, threads, 0, stream>>>(
        plan->dev, cache.stride_page, cache.stride_token, cache.stride_head,
        static_cast<uint4*>(k_pool), static_cast<uint4*>(v_pool),
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), vec_per_head, total);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hat
