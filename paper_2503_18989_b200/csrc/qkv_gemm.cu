// The step in front of the attention module (paper Sec. 2.1: Q = X W_Q, K = X W_K, V = X W_V) as one tcgen05 GEMM whose
// epilogue rotates the query and key rows by their token position and writes K and V straight into the paged cache:
// the projected rows never make a round trip through HBM in front of the attention kernels.
//
//   y[t][f] = sum_j x[t][j] w[f][j]        x [T][hidden], w [(Hq + 2 Hkv) d][hidden] (one row per output feature),
//                                          features ordered q heads | k heads | v heads
// Persistent kernel, one CTA per SM, output tiles of 128 rows x 256 features (two heads of 128 or four of 64), drawn
// in a fixed order with the row tile running fastest: the CTAs of one round share a strip of w, which then crosses
// HBM once, and x (much smaller) stays in L2.  Roles:
//   warp 0      TMA producer: per 64 columns of the hidden dimension one box of x (128 rows) and one of w (256 rows),
//               128-byte swizzle, into a four-stage ring
//   warp 1      one thread issues tcgen05.mma (M 128, N 256, K 16; four per stage) into one of two 256-column
//               accumulators in TMEM; tcgen05.commit frees the stage and, after the last stage of a tile, hands the
//               accumulator to the epilogue.  Owns the TMEM allocation
//   warps 2-5   epilogue, thread = output row = TMEM lane: reads the accumulator 32 columns at a time, rotates q and k
//               heads with the (cos, sin) pairs of the row's position (a table filled by a small kernel in front, the
//               same double-precision angle reduction as the rotating append), rounds to the 16-bit type once and
//               stores q rows packed and k / v rows at their slot of the pools; the other accumulator is being
//               filled meanwhile
// Every wait is bounded; a wait that gives up sets bit 0 of the plan's status word and the CTA winds down normally.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>

#include "hat_internal.h"
#include "tma_desc.h"
#include "tc5_ptx.cuh"

namespace hat {
namespace {
using namespace tc5;

constexpr int kTileM = 128, kTileN = 256, kTileK = 64;
constexpr int kStages = 4;
constexpr uint32_t kABytes = kTileM * kTileK * 2;        // 16 KiB
constexpr uint32_t kBBytes = kTileN * kTileK * 2;        // 32 KiB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr int kThreads = 192;

struct __align__(8) Barriers {
    uint64_t full[kStages], empty[kStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t drain;
    long long wait_cycles;
    uint32_t tmem_base;
    volatile int abort_flag;
};
constexpr uint32_t kSmemBytes = 1024 + kStages * kStageBytes + sizeof(Barriers);
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");

struct QkvArgs {
    DevicePlan plan;
    CacheView cache;
    void* k_pool;
    void* v_pool;
    void* q_out;              // [T][Hq][d]
    const float2* trig;       // [T][d/2] (cos, sin), or null: no rotation
    int hidden, head_dim, interleaved;
    int m_tiles, n_tiles;
    long long wait_cycles;
};

__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Barriers* b, int32_t* status) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try(bar, parity)) {
        if (b->abort_flag) return false;
        if (clock64() - t0 > b->wait_cycles) {
            b->abort_flag = 1;
            atomicOr(status, 1);
            return false;
        }
    }
    return true;
}

// 32 fp32 values rounded into 64 bytes at dst (16-byte aligned)
template <bool BF16>
__device__ __forceinline__ void store32(unsigned char* dst, const float* v) {
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint4 o;
        o.x = pack2<BF16>(v[8 * g + 0], v[8 * g + 1]);
        o.y = pack2<BF16>(v[8 * g + 2], v[8 * g + 3]);
        o.z = pack2<BF16>(v[8 * g + 4], v[8 * g + 5]);
        o.w = pack2<BF16>(v[8 * g + 6], v[8 * g + 7]);
        *reinterpret_cast<uint4*>(dst + 16 * g) = o;
    }
}

// (cos, sin) of every row and pair: trig[t][c], position of row t = prefix_len[r] + (t - cu_chunk[r])
__global__ void __launch_bounds__(256) rope_table_kernel(DevicePlan plan, int half, const __grid_constant__ InvFreq fr,
                                                         float2* __restrict__ trig) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)plan.total_rows * half) return;
    const int t = (int)(idx / half), c = (int)(idx - (int64_t)t * half);
    const int r = plan.row_req[t];
    const int p = plan.prefix_len[r] + (t - plan.cu_chunk[r]);
    float s, co;
    rope_sincos(p, fr.f[c], &s, &co);
    trig[idx] = make_float2(co, s);
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads, 1)
qkv_gemm_kernel(const __grid_constant__ QkvArgs a, const __grid_constant__ CUtensorMap map_x,
                const __grid_constant__ CUtensorMap map_w) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t* status = a.plan.status;
    const int k_steps = a.hidden / kTileK;
    const int total_tiles = a.m_tiles * a.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->acc_full[s], 1); mbar_init(&bars->acc_empty[s], 4); }
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        bars->wait_cycles = a.wait_cycles;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            bool ok = true;
            int it = 0;                                        // stages issued so far, over all tiles
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int m = tile % a.m_tiles, n = tile / a.m_tiles;
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % kStages;
                    if (it >= kStages) ok = mbar_wait(&bars->empty[s], ((it / kStages) & 1) ^ 1, bars, status);
                    if (!ok) break;
                    const uint32_t dst = smem_u32(smem) + s * kStageBytes;
                    mbar_expect_tx(&bars->full[s], kStageBytes);
                    tma_load_2d(dst, &map_x, ks * kTileK, m * kTileM, &bars->full[s]);
                    tma_load_2d(dst + kABytes, &map_w, ks * kTileK, n * kTileN, &bars->full[s]);
                }
            }
            if (!ok) {
                // give copies already in flight a bounded chance to land before the CTA's shared memory is released
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) { }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BF16 ? 1u : 0u, 0, kTileM, kTileN);     // x (K-major) x w (K-major)
            const uint64_t a_desc0 = smem_desc(smem_u32(smem), 16, 1024);
            const uint64_t b_desc0 = smem_desc(smem_u32(smem) + kABytes, 16, 1024);
            bool ok = true;
            int it = 0, n_done = 0;                            // stages consumed, tiles issued
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++n_done) {
                const int buf = n_done & 1;
                if (n_done >= 2) {
                    // the epilogue has read the tile before last out of this accumulator
                    ok = mbar_wait(&bars->acc_empty[buf], ((n_done >> 1) & 1) ^ 1, bars, status);
                    if (!ok) break;
                    tc_fence_after();
                }
                const uint32_t d_tmem = tmem + buf * kTileN;
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(&bars->full[s], (it / kStages) & 1, bars, status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t off = (uint64_t)((s * kStageBytes) >> 4);
#pragma unroll
                    for (int kk = 0; kk < kTileK / 16; ++kk)   // 16 columns = 32 bytes inside a 128-byte row
                        mma_ss(d_tmem, a_desc0 + off + 2 * kk, b_desc0 + off + 2 * kk, idesc, (ks | kk) != 0);
                    tc_commit(&bars->empty[s]);
                }
                if (ok) tc_commit(&bars->acc_full[buf]);
            }
            if (!ok) {
                tc_commit(&bars->drain);
                const long long t0 = clock64();
                while (!mbar_try(&bars->drain, 0) && clock64() - t0 < bars->wait_cycles) { }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue: thread = output row
        const int quarter = warp & 3;                          // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const int d = a.head_dim, half = d / 2;
        const int Hq = a.plan.num_heads, Hkv = a.plan.num_kv_heads;
        const int heads_total = Hq + 2 * Hkv;
        const bool rotate = a.trig != nullptr;
        bool ok = true;
        int n_done = 0;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++n_done) {
            const int m = tile % a.m_tiles, n = tile / a.m_tiles;
            const int buf = n_done & 1;
            const int t = m * kTileM + row;
            const bool valid = t < a.plan.total_rows;
            int64_t pool_off = 0;                              // element offset of (page, slot) in the pools
            const float2* trig = nullptr;
            if (valid) {
                const int r = a.plan.row_req[t];
                const int p = a.plan.prefix_len[r] + (t - a.plan.cu_chunk[r]);
                const int page = HAT_IN_RANGE(__ldg(a.plan.block_table + (int64_t)r * a.plan.max_pages +
                                                    HAT_IN_RANGE(p / kPageSize, a.plan.max_pages, status)),
                                              a.plan.num_pages, status);
                pool_off = (int64_t)page * a.cache.stride_page + (int64_t)(p % kPageSize) * a.cache.stride_token;
                if (rotate) trig = a.trig + (int64_t)t * half;
            }
            ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], (n_done >> 1) & 1, bars, status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t acc = tmem + buf * kTileN + lane_sel;

            for (int hb = 0; hb < kTileN; hb += d) {           // heads of this tile, by their first column in it
                const int hh = (n * kTileN + hb) / d;
                if (hh >= heads_total) break;                  // uniform: the feature count does not fill the last tile
                // where the head's d values go
                unsigned char* dst;
                bool rot = rotate;
                if (hh < Hq) {
                    dst = static_cast<unsigned char*>(a.q_out) + ((int64_t)t * Hq + hh) * d * 2;
                } else if (hh < Hq + Hkv) {
                    dst = static_cast<unsigned char*>(a.k_pool) + (pool_off + (int64_t)(hh - Hq) * a.cache.stride_head) * 2;
                } else {
                    dst = static_cast<unsigned char*>(a.v_pool) + (pool_off + (int64_t)(hh - Hq - Hkv) * a.cache.stride_head) * 2;
                    rot = false;
                }
                if (!rot) {
                    for (int c0 = 0; c0 < d; c0 += 32) {
                        float v[32];
                        tmem_ld32(acc + hb + c0, reinterpret_cast<uint32_t*>(v));
                        tmem_ld_wait();
                        if (valid) store32<BF16>(dst + c0 * 2, v);
                    }
                } else if (a.interleaved) {
                    // pairs (x[2c], x[2c+1]): 32 columns hold pairs c0/2 .. c0/2 + 15
                    for (int c0 = 0; c0 < d; c0 += 32) {
                        float v[32];
                        tmem_ld32(acc + hb + c0, reinterpret_cast<uint32_t*>(v));
                        tmem_ld_wait();
                        if (valid) {
#pragma unroll
                            for (int i = 0; i < 16; i += 2) {
                                const float4 cs = __ldg(reinterpret_cast<const float4*>(trig + c0 / 2 + i));   // two (cos, sin)
                                const float lo0 = v[2 * i], hi0 = v[2 * i + 1], lo1 = v[2 * i + 2], hi1 = v[2 * i + 3];
                                v[2 * i] = lo0 * cs.x - hi0 * cs.y;
                                v[2 * i + 1] = hi0 * cs.x + lo0 * cs.y;
                                v[2 * i + 2] = lo1 * cs.z - hi1 * cs.w;
                                v[2 * i + 3] = hi1 * cs.z + lo1 * cs.w;
                            }
                            store32<BF16>(dst + c0 * 2, v);
                        }
                    }
                } else {
                    // pairs (x[c], x[c + d/2]): 32 columns of the low half with their partners of the high half
                    for (int c0 = 0; c0 < half; c0 += 32) {
                        float lo[32], hi[32];
                        tmem_ld32(acc + hb + c0, reinterpret_cast<uint32_t*>(lo));
                        tmem_ld32(acc + hb + half + c0, reinterpret_cast<uint32_t*>(hi));
                        tmem_ld_wait();
                        if (valid) {
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                const float4 cs = __ldg(reinterpret_cast<const float4*>(trig + c0 + i));
                                const float l0 = lo[i], h0 = hi[i], l1 = lo[i + 1], h1 = hi[i + 1];
                                lo[i] = l0 * cs.x - h0 * cs.y;
                                hi[i] = h0 * cs.x + l0 * cs.y;
                                lo[i + 1] = l1 * cs.z - h1 * cs.w;
                                hi[i + 1] = h1 * cs.z + l1 * cs.w;
                            }
                            store32<BF16>(dst + c0 * 2, lo);
                            store32<BF16>(dst + (half + c0) * 2, hi);
                        }
                    }
                }
            }
            // every value of this accumulator is in registers or stored: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_empty[buf]);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
    }
}

}  // namespace

size_t qkv_workspace_bytes(const hat_plan* plan) {
    return (size_t)plan->total_rows * (plan->head_dim / 2) * sizeof(float2);
}

cudaError_t launch_qkv_gemm(const hat_plan* plan, const CacheView& cache, void* k_pool, void* v_pool, const void* x,
                            int hidden, const void* w, void* q_out, float theta, int interleaved, void* workspace,
                            cudaStream_t stream) {
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    const int d = plan->head_dim, T = plan->total_rows;
    const int64_t features = (int64_t)(plan->num_heads + 2 * plan->num_kv_heads) * d;
    CUtensorMap mx, mw;
    if (!tma_encode_matrix_map(&mx, bf16, x, T, hidden, kTileM) || !tma_encode_matrix_map(&mw, bf16, w, features, hidden, kTileN))
        return cudaErrorInvalidValue;
    QkvArgs a;
    a.plan = plan->dev;
    a.cache = cache;
    a.k_pool = k_pool; a.v_pool = v_pool; a.q_out = q_out;
    a.trig = nullptr;
    a.hidden = hidden; a.head_dim = d; a.interleaved = interleaved;
    a.m_tiles = (T + kTileM - 1) / kTileM;
    a.n_tiles = (int)((features + kTileN - 1) / kTileN);
    a.wait_cycles = plan->wait_cycles;
    if (theta > 0.f) {
        InvFreq fr;
        for (int c = 0; c < d / 2; ++c) fr.f[c] = std::pow((double)theta, -2.0 * c / d);
        const int64_t total = (int64_t)T * (d / 2);
        rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(plan->dev, d / 2, fr, static_cast<float2*>(workspace));
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        a.trig = static_cast<const float2*>(workspace);
    }
    auto kern = bf16 ? qkv_gemm_kernel<true> : qkv_gemm_kernel<false>;
    cudaError_t e = smem_attr_once(reinterpret_cast<const void*>(kern), (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    const int ctas = std::min(plan->num_sms, a.m_tiles * a.n_tiles);
    kern<<<dim3((unsigned)ctas), kThreads, kSmemBytes, stream>>>(a, mx, mw);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hat
