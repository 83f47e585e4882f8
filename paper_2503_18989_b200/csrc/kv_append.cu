// KV append: scatter the chunk's new K/V rows into the paged pools (bit-exact 16-byte copies).
#include "hat_internal.h"

namespace hat {

// One thread moves one 16-byte vector of K and the matching vector of V.
// vectors_per_row = H * d / 8; thread index -> (packed row t, vector within the row).
__global__ void __launch_bounds__(256)
kv_append_kernel(DevicePlan plan, int64_t stride_page, int64_t stride_token, int64_t stride_head,
                 uint4* __restrict__ k_pool, uint4* __restrict__ v_pool,
                 const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                 int vec_per_head, int64_t total_vecs) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_vecs) return;
    const int vec_per_row = vec_per_head * plan.num_kv_heads;
    const int t = (int)(idx / vec_per_row);
    const int within = (int)(idx - (int64_t)t * vec_per_row);
    const int h = within / vec_per_head;
    const int c = within - h * vec_per_head;

    const int r = plan.row_req[t];
    const int pos = plan.prefix_len[r] + (t - plan.cu_chunk[r]);     // logical token index
    const int page = plan.block_table[(int64_t)r * plan.max_pages + pos / kPageSize];
    const int slot = pos % kPageSize;
    // strides are multiples of 8 elements, so the offset in 16-byte vectors is exact
    const int64_t dst = ((int64_t)page * stride_page + (int64_t)slot * stride_token + (int64_t)h * stride_head) / 8 + c;

    const uint4 kv = __ldg(k_new + idx);
    const uint4 vv = __ldg(v_new + idx);
    k_pool[dst] = kv;
    v_pool[dst] = vv;
}

cudaError_t launch_kv_append(const hat_plan* plan, const CacheView& cache, void* k_pool, void* v_pool,
                             const void* k_new, const void* v_new, cudaStream_t stream) {
    const int vec_per_head = plan->head_dim / 8;
    const int64_t total = (int64_t)plan->total_rows * plan->num_kv_heads * vec_per_head;
    if (total == 0) return cudaSuccess;
    const int threads = 256;
    const int64_t blocks = (total + threads - 1) / threads;
    kv_append_kernel<<<(unsigned)blocks, threads, 0, stream>>>(
        plan->dev, cache.stride_page, cache.stride_token, cache.stride_head,
        static_cast<uint4*>(k_pool), static_cast<uint4*>(v_pool),
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), vec_per_head, total);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hat
