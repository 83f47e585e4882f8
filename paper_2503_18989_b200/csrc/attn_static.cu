// Streaming (verify-class) chunk attention for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a CUDA-graph capture or
// a latency-critical serving loop whose memory was carved up at start-up, or under a framework that
// owns the whole device heap.  hat_chunk_attention needs a plan (one cudaMalloc) and a caller-provided
// workspace for its split-KV partial results.  The entry point in this file needs neither: the batch
// descriptor arrays are read straight from device memory, every request is cut into a fixed number of
// key ranges computed from its length inside the kernel, and the partial results live in a file-scope
// __device__ array that is part of the loaded module (HAT_STATIC_SCRATCH_BYTES on every GPU that loads
// the library, until the process exits).
//
// The kernels are a self-contained variant of the streaming kernel (one warp per key group, mma.sync
// m16n8k16, cp.async ring), followed by a merge over the fixed number of ranges.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cmath>

#include "hat_internal.h"

namespace {

constexpr int kSplits = HAT_STATIC_SPLITS;
constexpr int kMaxDevices = 64;

// Partial results of the last call: [request][range][row][head][d] floats followed by
// [request][range][row][head] log-sum-exps.  Shared by every call on this GPU.
static __device__ __align__(256) unsigned char g_scratch[HAT_STATIC_SCRATCH_BYTES];

// Device address of g_scratch per device ordinal, resolved on first use.  In host code the name
// g_scratch is only a handle for the runtime; the address a kernel can use comes from
// cudaGetSymbolAddress.
static void* g_scratch_addr[kMaxDevices] = {nullptr};

struct StaticArgs {
    const void* k_pool;
    const void* v_pool;
    int64_t stride_page, stride_token, stride_head;
    const int32_t* cu_chunk;
    const int32_t* prefix_len;
    const int32_t* chunk_len;
    const int32_t* block_table;
    const void* q;
    float* out;
    float* lse;
    float* part_out;
    float* part_lse;
    float scale_log2;
    int32_t num_pages, max_pages, num_heads, max_rows;
};

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
template <bool BF16>
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if constexpr (BF16) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    } else {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
}
template <bool BF16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    if constexpr (BF16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}
template <int D>
__device__ __forceinline__ uint32_t sw(int row, int c) { return (uint32_t)(row * (D * 2) + ((c ^ (row & 7)) << 4)); }

// grid (heads, requests * kSplits); 4 warps, warp w streams pages w, w+4, ... of the CTA's key range.
template <bool BF16, int D>
__global__ void __launch_bounds__(128) static_stream_kernel(StaticArgs a) {
    using T = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    constexpr int CH = D / 8, PAGE_BYTES = 16 * D * 2, STAGES = 3, ON = D / 8, WN = 4;
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t sbase = s_u32(smem);
    const int h = blockIdx.x, r = blockIdx.y / kSplits, sp = blockIdx.y % kSplits;
    const int H = a.num_heads;
    // lengths come from device memory nobody validated: clamp them so that no lookup leaves the block table
    const hat::StaticRange rg = hat::static_key_range(a.prefix_len[r], a.chunk_len[r], a.max_rows, a.max_pages, sp);
    const int P = rg.prefix, C = rg.rows;
    if (C <= 0) return;
    const int kv_begin = rg.kv_begin, kv_end = rg.kv_end;
    const int row_base = a.cu_chunk[r];
    const int32_t* __restrict__ table = a.block_table + (int64_t)r * a.max_pages;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const T* __restrict__ kpool = static_cast<const T*>(a.k_pool);
    const T* __restrict__ vpool = static_cast<const T*>(a.v_pool);
    const int64_t head_off = (int64_t)h * a.stride_head;

    float o[ON][4];
#pragma unroll
    for (int n = 0; n < ON; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    const int n_pages = kv_end > kv_begin ? (kv_end - kv_begin + 15) / 16 : 0;
    const int n_my = n_pages > warp ? (n_pages - warp + WN - 1) / WN : 0;
    const uint32_t ring = sbase + 16 * D * 2 + warp * (STAGES * 2 * PAGE_BYTES);
    auto issue = [&](int ti, int slot) {
        const int kb = kv_begin + ti * 16;
        const uint32_t kdst = ring + slot * (2 * PAGE_BYTES), vdst = kdst + PAGE_BYTES;
        int page = __ldg(table + min(kb / 16, a.max_pages - 1));            // never leave the request's table row
        page = min(max(page, 0), a.num_pages - 1);                          // nor the pool
#pragma unroll
        for (int idx = lane; idx < 16 * CH; idx += 32) {
            const int row = idx / CH, c = idx % CH;
            const uint32_t off = sw<D>(row, c);
            if (kb + row < kv_end) {
                const int64_t e = (int64_t)page * a.stride_page + (int64_t)row * a.stride_token + head_off + c * 8;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(kdst + off), "l"(kpool + e));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(vdst + off), "l"(vpool + e));
            } else {
                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(kdst + off), "r"(0));
                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(vdst + off), "r"(0));
            }
        }
    };
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < n_my) issue(warp + s * WN, s);
        asm volatile("cp.async.commit_group;\n" ::);
    }
    {
        const T* __restrict__ q = static_cast<const T*>(a.q);
        for (int idx = tid; idx < 16 * CH; idx += 128) {
            const int row = idx / CH, c = idx % CH;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (row < C) v = __ldg(reinterpret_cast<const uint4*>(q + ((int64_t)(row_base + row) * H + h) * D) + c);
            *reinterpret_cast<uint4*>(smem + sw<D>(row, c)) = v;
        }
    }
    __syncthreads();
    uint32_t qf[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const int mi = lane >> 3;
        ldsm4(qf[ks], sbase + sw<D>((mi & 1) * 8 + (lane & 7), ks * 2 + (mi >> 1)));
    }
    const int lim0 = P + g, lim1 = lim0 + 8;
    for (int it = 0; it < n_my; ++it) {
        asm volatile("cp.async.wait_group %0;\n" ::"n"(STAGES - 2));
        __syncwarp();
        if (it + STAGES - 1 < n_my) issue(warp + (it + STAGES - 1) * WN, (it + STAGES - 1) % STAGES);
        asm volatile("cp.async.commit_group;\n" ::);
        const int kb = kv_begin + (warp + it * WN) * 16;
        const uint32_t kst = ring + (it % STAGES) * (2 * PAGE_BYTES), vst = kst + PAGE_BYTES;
        float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const int mi = lane >> 3;
            uint32_t b[4];
            ldsm4(b, kst + sw<D>((mi >> 1) * 8 + (lane & 7), ks * 2 + (mi & 1)));
            mma16816<BF16>(s[0], qf[ks], b[0], b[1]);
            mma16816<BF16>(s[1], qf[ks], b[2], b[3]);
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            const int j = kb + n * 8 + 2 * t4;
            s[n][0] = (j <= lim0 && j < kv_end) ? s[n][0] * a.scale_log2 : -INFINITY;
            s[n][1] = (j + 1 <= lim0 && j + 1 < kv_end) ? s[n][1] * a.scale_log2 : -INFINITY;
            s[n][2] = (j <= lim1 && j < kv_end) ? s[n][2] * a.scale_log2 : -INFINITY;
            s[n][3] = (j + 1 <= lim1 && j + 1 < kv_end) ? s[n][3] * a.scale_log2 : -INFINITY;
            mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
            mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float al0 = exp2f(m0 - ms0), al1 = exp2f(m1 - ms1);
        m0 = mn0; m1 = mn1;
        float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            s[n][0] = exp2f(s[n][0] - ms0); s[n][1] = exp2f(s[n][1] - ms0);
            s[n][2] = exp2f(s[n][2] - ms1); s[n][3] = exp2f(s[n][3] - ms1);
            rs0 += s[n][0] + s[n][1]; rs1 += s[n][2] + s[n][3];
        }
        l0 = l0 * al0 + rs0; l1 = l1 * al1 + rs1;
#pragma unroll
        for (int n = 0; n < ON; ++n) { o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1; }
        uint32_t pa[4], pl[4];
        pa[0] = pack2<BF16>(s[0][0], s[0][1]); pa[1] = pack2<BF16>(s[0][2], s[0][3]);
        pa[2] = pack2<BF16>(s[1][0], s[1][1]); pa[3] = pack2<BF16>(s[1][2], s[1][3]);
        if constexpr (BF16) {
            // second operand with what the 8-bit rounding of P dropped
            const float* sf = &s[0][0];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float lo = __uint_as_float(pa[k] << 16), hi = __uint_as_float(pa[k] & 0xffff0000u);
                pl[k] = pack2<BF16>(sf[2 * k] - lo, sf[2 * k + 1] - hi);
            }
        }
#pragma unroll
        for (int dn = 0; dn < D / 16; ++dn) {
            const int mi = lane >> 3;
            uint32_t b[4];
            ldsm4t(b, vst + sw<D>((mi & 1) * 8 + (lane & 7), dn * 2 + (mi >> 1)));
            mma16816<BF16>(o[2 * dn], pa, b[0], b[1]);
            mma16816<BF16>(o[2 * dn + 1], pa, b[2], b[3]);
            if constexpr (BF16) {
                mma16816<BF16>(o[2 * dn], pl, b[0], b[1]);
                mma16816<BF16>(o[2 * dn + 1], pl, b[2], b[3]);
            }
        }
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // combine the four warps (same fragment positions in each)
    constexpr int VALS = ON * 4 + 4;
    asm volatile("cp.async.wait_group 0;\n" ::);
    __syncthreads();
    float* xbuf = reinterpret_cast<float*>(smem + 16 * D * 2);
    if (warp > 0) {
        float* dst = xbuf + (warp - 1) * (VALS * 32) + lane;
#pragma unroll
        for (int n = 0; n < ON; ++n)
#pragma unroll
            for (int k = 0; k < 4; ++k) dst[(n * 4 + k) * 32] = o[n][k];
        dst[(ON * 4 + 0) * 32] = m0; dst[(ON * 4 + 1) * 32] = m1;
        dst[(ON * 4 + 2) * 32] = l0; dst[(ON * 4 + 3) * 32] = l1;
    }
    __syncthreads();
    if (warp > 0) return;
    float mt0 = m0, mt1 = m1;
#pragma unroll
    for (int k = 1; k < WN; ++k) {
        const float* src = xbuf + (k - 1) * (VALS * 32) + lane;
        mt0 = fmaxf(mt0, src[(ON * 4 + 0) * 32]);
        mt1 = fmaxf(mt1, src[(ON * 4 + 1) * 32]);
    }
    const float ms0 = (mt0 == -INFINITY) ? 0.f : mt0, ms1 = (mt1 == -INFINITY) ? 0.f : mt1;
    {
        const float w0 = exp2f(m0 - ms0), w1 = exp2f(m1 - ms1);
        l0 *= w0; l1 *= w1;
#pragma unroll
        for (int n = 0; n < ON; ++n) { o[n][0] *= w0; o[n][1] *= w0; o[n][2] *= w1; o[n][3] *= w1; }
    }
#pragma unroll
    for (int k = 1; k < WN; ++k) {
        const float* src = xbuf + (k - 1) * (VALS * 32) + lane;
        const float w0 = exp2f(src[(ON * 4 + 0) * 32] - ms0), w1 = exp2f(src[(ON * 4 + 1) * 32] - ms1);
        l0 += w0 * src[(ON * 4 + 2) * 32];
        l1 += w1 * src[(ON * 4 + 3) * 32];
#pragma unroll
        for (int n = 0; n < ON; ++n) {
            o[n][0] += w0 * src[(n * 4 + 0) * 32]; o[n][1] += w0 * src[(n * 4 + 1) * 32];
            o[n][2] += w1 * src[(n * 4 + 2) * 32]; o[n][3] += w1 * src[(n * 4 + 3) * 32];
        }
    }
    // every (range, row < C) slot is written on every call, an empty range as (0, -inf): the merge
    // never reads anything left over from an earlier call, so nothing needs clearing beforehand
    const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
    constexpr float kLn2 = 0.6931471805599453f;
    const float lse0 = l0 > 0.f ? (mt0 + log2f(l0)) * kLn2 : -INFINITY;
    const float lse1 = l1 > 0.f ? (mt1 + log2f(l1)) * kLn2 : -INFINITY;
    const int64_t slot = ((int64_t)r * kSplits + sp) * a.max_rows;
    if (g < C) {
        float* dst = a.part_out + ((slot + g) * H + h) * D + 2 * t4;
#pragma unroll
        for (int n = 0; n < ON; ++n) *reinterpret_cast<float2*>(dst + n * 8) = make_float2(o[n][0] * inv0, o[n][1] * inv0);
        if (t4 == 0) a.part_lse[(slot + g) * H + h] = lse0;
    }
    if (g + 8 < C) {
        float* dst = a.part_out + ((slot + g + 8) * H + h) * D + 2 * t4;
#pragma unroll
        for (int n = 0; n < ON; ++n) *reinterpret_cast<float2*>(dst + n * 8) = make_float2(o[n][2] * inv1, o[n][3] * inv1);
        if (t4 == 0) a.part_lse[(slot + g + 8) * H + h] = lse1;
    }
}

// One warp per (request, row slot, head): merge the kSplits partial rows.
template <int D>
__global__ void __launch_bounds__(128) static_merge_kernel(StaticArgs a, int num_requests) {
    const int lane = threadIdx.x & 31;
    const int64_t unit = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int H = a.num_heads;
    if (unit >= (int64_t)num_requests * a.max_rows * H) return;
    const int h = (int)(unit % H);
    const int i = (int)((unit / H) % a.max_rows);
    const int r = (int)(unit / ((int64_t)H * a.max_rows));
    if (i >= hat::static_key_range(a.prefix_len[r], a.chunk_len[r], a.max_rows, a.max_pages, 0).rows) return;
    float my = -INFINITY;
    if (lane < kSplits) my = a.part_lse[(((int64_t)r * kSplits + lane) * a.max_rows + i) * H + h];
    float mx = my;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float ms = (mx == -INFINITY) ? 0.f : mx;
    float w = expf(my - ms);
    float sum = w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    w *= sum > 0.f ? 1.f / sum : 0.f;
    constexpr int V = D / 32;
    float acc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) acc[k] = 0.f;
    for (int s = 0; s < kSplits; ++s) {
        const float ws = __shfl_sync(0xffffffffu, w, s);
        const float* src = a.part_out + ((((int64_t)r * kSplits + s) * a.max_rows + i) * H + h) * D + lane * V;
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] += ws * src[k];
    }
    const int64_t row = a.cu_chunk[r] + i;
    float* dst = a.out + (row * H + h) * D + lane * V;
#pragma unroll
    for (int k = 0; k < V; ++k) dst[k] = acc[k];
    if (lane == 0) a.lse[row * H + h] = sum > 0.f ? ms + logf(sum) : -INFINITY;
}

template <bool BF16, int D>
cudaError_t launch_static(const StaticArgs& a, int R, cudaStream_t s) {
    constexpr int smem = 16 * D * 2 + 4 * 3 * 2 * (16 * D * 2);
    auto kern = static_stream_kernel<BF16, D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<dim3(a.num_heads, R * kSplits), 128, smem, s>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const int64_t units = (int64_t)R * a.max_rows * a.num_heads;
    static_merge_kernel<D><<<(unsigned)((units + 3) / 4), 128, 0, s>>>(a, R);
    hat::count_launch(2);
    return cudaGetLastError();
}

}  // namespace

extern "C" int hat_verify_attention_static(const hat_cache_desc* cache, int num_requests, int num_q_heads,
                                           int max_chunk_len, int max_pages, const int32_t* cu_chunk,
                                           const int32_t* prefix_len, const int32_t* chunk_len,
                                           const int32_t* block_table, const void* q, float* out, float* lse,
                                           float sm_scale, void* stream) {
    if (!cache || !cache->k_pool || !cache->v_pool) return HAT_ERR_INVALID_ARG;
    if (cache->dtype != HAT_DTYPE_FP16 && cache->dtype != HAT_DTYPE_BF16) return HAT_ERR_UNSUPPORTED;
    if (cache->page_size != 16 || (cache->head_dim != 64 && cache->head_dim != 128)) return HAT_ERR_UNSUPPORTED;
    if (num_q_heads <= 0 || num_q_heads != cache->num_kv_heads) return HAT_ERR_UNSUPPORTED;
    if (cache->stride_page <= 0 || cache->stride_token <= 0 || cache->stride_head <= 0 ||
        cache->stride_page % 8 || cache->stride_token % 8 || cache->stride_head % 8)
        return HAT_ERR_UNSUPPORTED;
    if (num_requests < 0 || max_pages <= 0 || cache->num_pages <= 0) return HAT_ERR_INVALID_ARG;
    if (max_chunk_len < 1 || max_chunk_len > 16) return HAT_ERR_INVALID_ARG;
    if (num_requests == 0) return HAT_OK;
    if (!cu_chunk || !prefix_len || !chunk_len || !block_table || !q || !out || !lse) return HAT_ERR_INVALID_ARG;
    if ((int64_t)num_requests * HAT_STATIC_SPLITS > 65535) return HAT_ERR_TOO_LARGE;
    const int64_t H = num_q_heads, d = cache->head_dim;
    const int64_t slots = (int64_t)num_requests * HAT_STATIC_SPLITS * max_chunk_len;
    const int64_t out_bytes = (slots * H * d * 4 + 255) / 256 * 256;
    const int64_t lse_bytes = slots * H * 4;
    if (out_bytes + lse_bytes > (int64_t)HAT_STATIC_SCRATCH_BYTES) return HAT_ERR_TOO_LARGE;

    // first call on a device: resolve the device address of the scratch array (no allocation)
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) { hat::set_last_cuda_error((int)e); return HAT_ERR_CUDA; }
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess || !p) { hat::set_last_cuda_error((int)e); return HAT_ERR_CUDA; }
        g_scratch_addr[dev] = p;
    }
    if (!(sm_scale > 0.f) || !std::isfinite(sm_scale)) sm_scale = 1.0f / std::sqrt((float)d);

    StaticArgs a;
    a.k_pool = cache->k_pool; a.v_pool = cache->v_pool;
    a.stride_page = cache->stride_page; a.stride_token = cache->stride_token; a.stride_head = cache->stride_head;
    a.cu_chunk = cu_chunk; a.prefix_len = prefix_len; a.chunk_len = chunk_len; a.block_table = block_table;
    a.q = q; a.out = out; a.lse = lse;
    a.part_out = static_cast<float*>(g_scratch_addr[dev]);
    a.part_lse = reinterpret_cast<float*>(static_cast<char*>(g_scratch_addr[dev]) + out_bytes);
    a.scale_log2 = sm_scale * 1.4426950408889634f;
    a.num_pages = cache->num_pages; a.max_pages = max_pages; a.num_heads = num_q_heads; a.max_rows = max_chunk_len;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool bf16 = cache->dtype == HAT_DTYPE_BF16;
    if (d == 128) e = bf16 ? launch_static<true, 128>(a, num_requests, s) : launch_static<false, 128>(a, num_requests, s);
    else e = bf16 ? launch_static<true, 64>(a, num_requests, s) : launch_static<false, 64>(a, num_requests, s);
    if (e != cudaSuccess) hat::set_last_cuda_error((int)e);
    return e == cudaSuccess ? HAT_OK : HAT_ERR_CUDA;
}

extern "C" int hat_static_key_range(int prefix_len, int chunk_len, int max_chunk_len, int max_pages, int split,
                                    int* prefix, int* rows, int* kv_begin, int* kv_end) {
    if (max_chunk_len < 1 || max_chunk_len > 16 || max_pages <= 0 || split < 0 || split >= HAT_STATIC_SPLITS)
        return HAT_ERR_INVALID_ARG;
    const hat::StaticRange rg = hat::static_key_range(prefix_len, chunk_len, max_chunk_len, max_pages, split);
    if (prefix) *prefix = rg.prefix;
    if (rows) *rows = rg.rows;
    if (kv_begin) *kv_begin = rg.kv_begin;
    if (kv_end) *kv_end = rg.kv_end;
    return HAT_OK;
}
