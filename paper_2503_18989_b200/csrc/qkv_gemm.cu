// The step in front of the attention module (paper Sec. 2.1: Q = X W_Q, K = X W_K, V = X W_V) as one tcgen05 GEMM whose
// epilogue rotates the query and key rows by their token position and writes K and V straight into the paged cache:
// the projected rows never make a round trip through HBM in front of the attention kernels.
//
//   y[t][f] = sum_j x[t][j] w[f][j]        x [T][hidden], w [(Hq + 2 Hkv) d][hidden] (one row per output feature),
//                                          features ordered q heads | k heads | v heads
// Persistent kernel, output tiles of whole heads, drawn in a fixed order with the row tile running fastest: the CTAs of
// one round share a strip of w, which then crosses HBM once, and x (much smaller) stays in L2.  Two forms:
//   PAIR   clusters of two CTAs, tcgen05.mma.cta_group::2 with M = 256, tiles of 256 features (two heads of 128 or four
//          of 64): each CTA stages its own 128 rows of x and HALF of the 256 rows of w (32 KiB per 64 columns of the
//          hidden dimension and CTA, six stages).  What bounds this GEMM on 148 SMs is the path from L2 into shared
//          memory, and a pair moves 2/3 of the bytes per flop that two single CTAs with 128 x 256 tiles do
//   single batches of at most 128 rows (draft verification), which would leave half of a pair idle and are bound by
//          reading w once from HBM: one CTA per tile of 128 rows x 128 features, so that twice as many SMs pull on w
//          (120 tiles at the 13B shape: 47 us, where 256-feature tiles gave 60 tiles and 57 us)
// Roles (per CTA):
//   warp 0      TMA producer: per 64 columns of the hidden dimension one box of x and one of w, 128-byte swizzle
//   warp 1      CTA 0 of a pair (or the single CTA): one thread issues tcgen05.mma (four per stage) into one of two
//               accumulators (256 or 128 columns) in TMEM; tcgen05.commit frees the stage (in both CTAs) and, after the last
//               stage of a tile, hands the accumulator to the epilogue warps.  CTA 1: one thread forwards "my half of
//               this stage has landed" to CTA 0's barrier.  The warp owns the TMEM allocation
//   warps 2-5   epilogue, thread = output row = TMEM lane: reads the accumulator 32 columns at a time, rotates q and k
//               heads with the (cos, sin) of the row's position (a table kept with the plan, filled once per plan and
//               base by a small kernel with the same double-precision angle reduction as the rotating append), rounds
//               to the 16-bit type once and stores q rows packed and k / v rows at their slot of the pools; the other
//               accumulator is being filled meanwhile
// Every wait is bounded; a wait that gives up sets bit 0 of the plan's status word, tells the other CTA of the pair, and
// the CTA winds down normally.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>

#include "hat_internal.h"
#include "tma_desc.h"
#include "tc5_ptx.cuh"

namespace hat {
namespace {
using namespace tc5;

constexpr int kTileM = 128, kTileK = 64;
constexpr uint32_t kABytes = kTileM * kTileK * 2;        // 16 KiB: 128 rows of x
constexpr int kThreads = 192;
constexpr int kMaxStages = 6;

template <bool PAIR> struct Geo {
    static constexpr int kStages = 6;
    static constexpr int kTileN = PAIR ? 256 : 128;                      // features per output tile
    static constexpr int kBRows = 128;                                   // rows of w one CTA stages (half a tile for pairs)
    static constexpr uint32_t kBBytes = kBRows * kTileK * 2;
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
};

struct __align__(8) Barriers {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t drain;
    long long wait_cycles;
    uint32_t tmem_base;
    volatile int abort_flag;
};
template <bool PAIR> constexpr uint32_t smem_bytes() { return 1024 + Geo<PAIR>::kStages * Geo<PAIR>::kStageBytes + sizeof(Barriers); }
static_assert(smem_bytes<true>() <= 227 * 1024 && smem_bytes<false>() <= 227 * 1024, "shared memory of one CTA");

struct QkvArgs {
    DevicePlan plan;
    CacheView cache;
    void* k_pool;
    void* v_pool;
    void* q_out;              // [T][Hq][d]
    const float2* trig;       // [T][d/2] (cos, sin), or null: q and k are stored as projected
    int hidden, head_dim, interleaved;
    int m_tiles, n_tiles;     // row tiles (of 256 rows for pairs, else 128) and feature tiles
    long long wait_cycles;
    int withhold;             // self test: the first stage of CTA 0 (of every pair) never arrives, so a wait runs out
};

struct Ctx {
    Barriers* bars;
    int32_t* status;
    uint32_t peer_abort;      // shared::cluster address of the other CTA's abort flag (pairs)
    bool pair;
};

__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const Ctx& cx) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try(bar, parity)) {
        if (cx.bars->abort_flag) return false;
        if (clock64() - t0 > cx.bars->wait_cycles) {
            cx.bars->abort_flag = 1;
            if (cx.pair) st_cluster_b32(cx.peer_abort, 1u);
            atomicOr(cx.status, 1);
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

// One output row of one tile: the thread's TMEM lane of the accumulator at `acc`, packed row t, feature tile n.
template <bool BF16, int kTileN>
__device__ __forceinline__ void epilogue_row(const QkvArgs& a, uint32_t acc, int t, int n, int32_t* status) {
    const int d = a.head_dim, half = d / 2;
    const int Hq = a.plan.num_heads, Hkv = a.plan.num_kv_heads;
    const bool valid = t < a.plan.total_rows;
    int64_t pool_off = 0;                                  // element offset of (page, slot) in the pools
    const float2* trig = nullptr;
    if (valid) {
        const int r = a.plan.row_req[t];
        const int p = a.plan.prefix_len[r] + (t - a.plan.cu_chunk[r]);
        const int page = HAT_IN_RANGE(__ldg(a.plan.block_table + (int64_t)r * a.plan.max_pages +
                                            HAT_IN_RANGE(p / kPageSize, a.plan.max_pages, status)),
                                      a.plan.num_pages, status);
        pool_off = (int64_t)page * a.cache.stride_page + (int64_t)(p % kPageSize) * a.cache.stride_token;
        if (a.trig) trig = a.trig + (int64_t)t * half;
    }
    const int h_first = (n * kTileN) / d;                  // first head of this tile
    const int h_count = min(kTileN / d, Hq + 2 * Hkv - h_first);
    for (int hi = 0; hi < h_count; ++hi) {
        const int hh = h_first + hi;
        // where the head's d values of this row go
        unsigned char* dst;
        bool rot = a.trig != nullptr;
        if (hh < Hq) {
            dst = static_cast<unsigned char*>(a.q_out) + ((int64_t)t * Hq + hh) * d * 2;
        } else if (hh < Hq + Hkv) {
            dst = static_cast<unsigned char*>(a.k_pool) + (pool_off + (int64_t)(hh - Hq) * a.cache.stride_head) * 2;
        } else {
            dst = static_cast<unsigned char*>(a.v_pool) + (pool_off + (int64_t)(hh - Hq - Hkv) * a.cache.stride_head) * 2;
            rot = false;
        }
        const uint32_t col = acc + hi * d;
        if (!rot) {
            for (int c0 = 0; c0 < d; c0 += 32) {
                float v[32];
                tmem_ld32(col + c0, reinterpret_cast<uint32_t*>(v));
                tmem_ld_wait();
                if (valid) store32<BF16>(dst + c0 * 2, v);
            }
        } else if (a.interleaved) {
            // pairs (x[2c], x[2c+1]): 32 columns hold pairs c0/2 .. c0/2 + 15
            for (int c0 = 0; c0 < d; c0 += 32) {
                float v[32];
                tmem_ld32(col + c0, reinterpret_cast<uint32_t*>(v));
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
                float lo[32], hv[32];
                tmem_ld32(col + c0, reinterpret_cast<uint32_t*>(lo));
                tmem_ld32(col + half + c0, reinterpret_cast<uint32_t*>(hv));
                tmem_ld_wait();
                if (valid) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float4 cs = __ldg(reinterpret_cast<const float4*>(trig + c0 + i));
                        const float l0 = lo[i], h0 = hv[i], l1 = lo[i + 1], h1 = hv[i + 1];
                        lo[i] = l0 * cs.x - h0 * cs.y;
                        hv[i] = h0 * cs.x + l0 * cs.y;
                        lo[i + 1] = l1 * cs.z - h1 * cs.w;
                        hv[i + 1] = h1 * cs.z + l1 * cs.w;
                    }
                    store32<BF16>(dst + c0 * 2, lo);
                    store32<BF16>(dst + (half + c0) * 2, hv);
                }
            }
        }
    }
}

template <bool BF16, bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
qkv_gemm_kernel(const __grid_constant__ QkvArgs a, const __grid_constant__ CUtensorMap map_x,
                const __grid_constant__ CUtensorMap map_w) {
    using G = Geo<PAIR>;
    constexpr int kStages = G::kStages;
    constexpr int kTileN = G::kTileN;
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the swizzle pattern; both CTAs of a pair get the same offsets (one descriptor serves both)
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kStages * G::kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t rank = 0;                                          // 0: the CTA whose thread issues the MMAs
    if constexpr (PAIR) rank = cluster_ctarank();
    Ctx cx;
    cx.bars = bars;
    cx.status = a.plan.status;
    cx.pair = PAIR;
    cx.peer_abort = 0;
    if constexpr (PAIR) cx.peer_abort = map_to_cta(smem_u32(const_cast<int*>(&bars->abort_flag)), rank ^ 1u);
    const int k_steps = a.hidden / kTileK;
    const int total_tiles = a.m_tiles * a.n_tiles;
    const int first_tile = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int tile_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        const uint32_t fwd = (PAIR && rank == 0) ? 2u : 1u;     // CTA 0's "full" barriers also take CTA 1's forwarded arrival
        for (int s = 0; s < kStages; ++s) { mbar_init(&bars->full[s], fwd); mbar_init(&bars->empty[s], 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->acc_full[s], 1);
            mbar_init(&bars->acc_empty[s], PAIR ? 8 : 4);       // one arrival per epilogue warp (of both CTAs)
        }
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        bars->wait_cycles = a.wait_cycles;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 1) {
        if constexpr (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) {
        // the other CTA's barriers must be initialised before anything arrives on them
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            bool ok = true;
            int it = 0;                                        // stages issued so far, over all tiles
            for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
                const int m = tile % a.m_tiles, n = tile / a.m_tiles;
                const int x_row = PAIR ? m * 2 * kTileM + (int)rank * kTileM : m * kTileM;
                const int w_row = n * kTileN + (int)rank * G::kBRows;
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % kStages;
                    if (it >= kStages) ok = mbar_wait(&bars->empty[s], ((it / kStages) & 1) ^ 1, cx);
                    if (!ok) break;
                    if (a.withhold && it == 0 && rank == 0) continue;      // self test: its consumers give up
                    const uint32_t dst = smem_u32(smem) + s * G::kStageBytes;
                    mbar_expect_tx(&bars->full[s], G::kStageBytes);
                    tma_load_2d(dst, &map_x, ks * kTileK, x_row, &bars->full[s]);
                    tma_load_2d(dst + kABytes, &map_w, ks * kTileK, w_row, &bars->full[s]);
                }
            }
            if (!ok) {
                // give copies already in flight a bounded chance to land before the CTA's shared memory is released
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) { }
            }
        }
        __syncwarp();
    } else if (warp == 1 && rank != 0) {
        // ------------------------------------------------------------------ CTA 1: forward "landed" to CTA 0's barriers
        if constexpr (PAIR) {
            if (lane == 0) {
                bool ok = true;
                int it = 0;
                for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
                    for (int ks = 0; ks < k_steps; ++ks, ++it) {
                        const int s = it % kStages;
                        ok = mbar_wait(&bars->full[s], (it / kStages) & 1, cx);
                        if (!ok) break;
                        mbar_arrive_remote(map_to_cta(smem_u32(&bars->full[s]), 0u));
                    }
                }
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BF16 ? 1u : 0u, 0, PAIR ? 2 * kTileM : kTileM, kTileN);   // x (K-major) x w (K-major)
            const uint64_t a_desc0 = smem_desc(smem_u32(smem), 16, 1024);
            const uint64_t b_desc0 = smem_desc(smem_u32(smem) + kABytes, 16, 1024);
            auto commit = [&](uint64_t* bar) { if constexpr (PAIR) tc_commit_pair(bar); else tc_commit(bar); };
            bool ok = true;
            int it = 0, n_done = 0;                            // stages consumed, tiles issued
            for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++n_done) {
                const int buf = n_done & 1;
                if (n_done >= 2) {
                    // the epilogue warps have read the tile before last out of this accumulator
                    ok = mbar_wait(&bars->acc_empty[buf], ((n_done >> 1) & 1) ^ 1, cx);
                    if (!ok) break;
                    tc_fence_after();
                }
                const uint32_t d_tmem = tmem + buf * kTileN;
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(&bars->full[s], (it / kStages) & 1, cx);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t off = (uint64_t)((s * G::kStageBytes) >> 4);
#pragma unroll
                    for (int kk = 0; kk < kTileK / 16; ++kk) { // 16 columns = 32 bytes inside a 128-byte row
                        if constexpr (PAIR) mma_ss_pair(d_tmem, a_desc0 + off + 2 * kk, b_desc0 + off + 2 * kk, idesc, (ks | kk) != 0);
                        else mma_ss(d_tmem, a_desc0 + off + 2 * kk, b_desc0 + off + 2 * kk, idesc, (ks | kk) != 0);
                    }
                    commit(&bars->empty[s]);
                }
                if (ok) commit(&bars->acc_full[buf]);
            }
            if (!ok) {
                // gave up: let the MMAs already issued finish (bounded) before TMEM is released
                commit(&bars->drain);
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
        uint32_t lead_empty[2] = {0, 0};                       // CTA 0's acc_empty barriers (pairs)
        if constexpr (PAIR) {
            lead_empty[0] = map_to_cta(smem_u32(&bars->acc_empty[0]), 0u);
            lead_empty[1] = map_to_cta(smem_u32(&bars->acc_empty[1]), 0u);
        }
        bool ok = true;
        int n_done = 0;
        for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++n_done) {
            const int m = tile % a.m_tiles, n = tile / a.m_tiles;
            const int buf = n_done & 1;
            const int t = (PAIR ? m * 2 * kTileM + (int)rank * kTileM : m * kTileM) + row;
            ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], (n_done >> 1) & 1, cx));
            if (!ok) break;
            tc_fence_after();
            epilogue_row<BF16, kTileN>(a, tmem + buf * kTileN + lane_sel, t, n, cx.status);
            // every value of this accumulator is in registers or stored: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_remote(lead_empty[buf]);
                else mbar_arrive(&bars->acc_empty[buf]);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) {
        // both CTAs are done with each other's barriers, and every MMA has finished, before tensor memory is freed
        cluster_arrive();
        cluster_wait();
    }
    if (warp == 1) {
        tc_fence_after();
        if constexpr (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
    }
}

template <bool BF16, bool PAIR>
cudaError_t launch_form(const QkvArgs& a, const CUtensorMap& mx, const CUtensorMap& mw, int num_sms, cudaStream_t stream) {
    auto kern = qkv_gemm_kernel<BF16, PAIR>;
    constexpr uint32_t smem = smem_bytes<PAIR>();
    cudaError_t e = smem_attr_once(reinterpret_cast<const void*>(kern), (int)smem);
    if (e != cudaSuccess) return e;
    const int tiles = a.m_tiles * a.n_tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    if (PAIR) {
        cfg.gridDim = dim3((unsigned)(2 * std::min(num_sms / 2, tiles)));
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    } else {
        cfg.gridDim = dim3((unsigned)std::min(num_sms, tiles));
    }
    e = cudaLaunchKernelEx(&cfg, kern, a, mx, mw);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_qkv_gemm(const hat_plan* plan, const CacheView& cache, void* k_pool, void* v_pool, const void* x,
                            int hidden, const void* w, void* q_out, float theta, int interleaved, cudaStream_t stream) {
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    const int d = plan->head_dim, T = plan->total_rows;
    const int64_t features = (int64_t)(plan->num_heads + 2 * plan->num_kv_heads) * d;
    // pairs of CTAs work on 256 rows at a time; a batch that fits one 128-row tile would leave the second CTA idle
    // (HAT_QKV_PAIR_ROWS overrides the row count above which pairs are used, for tuning)
    int pair_rows = kTileM;
    if (const char* v = std::getenv("HAT_QKV_PAIR_ROWS")) pair_rows = std::max(0, std::atoi(v));
    const bool pair = T > pair_rows;
    CUtensorMap mx, mw;
    if (!tma_encode_matrix_map(&mx, bf16, x, T, hidden, kTileM) ||
        !tma_encode_matrix_map(&mw, bf16, w, features, hidden, 128))
        return cudaErrorInvalidValue;
    QkvArgs a;
    a.plan = plan->dev;
    a.cache = cache;
    a.k_pool = k_pool; a.v_pool = v_pool; a.q_out = q_out;
    a.trig = nullptr;
    a.hidden = hidden; a.head_dim = d; a.interleaved = interleaved;
    a.m_tiles = pair ? (T + 2 * kTileM - 1) / (2 * kTileM) : (T + kTileM - 1) / kTileM;
    const int tile_n = pair ? Geo<true>::kTileN : Geo<false>::kTileN;
    a.n_tiles = (int)((features + tile_n - 1) / tile_n);
    a.wait_cycles = plan->wait_cycles;
    a.withhold = plan->withhold_next;
    const_cast<hat_plan*>(plan)->withhold_next = 0;
    cudaError_t e;
    if (theta > 0.f) {
        // the table of cosines and sines depends on the plan's positions and on the base only: every layer of a step
        // uses the one its first call filled
        hat_plan* mp = const_cast<hat_plan*>(plan);
        // Inside a stream capture nothing runs now: the fill becomes part of the captured graph (every replay refills the
        // table, which is harmless) and the plan does not take the table as filled.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if ((e = cudaStreamIsCapturing(stream, &cap)) != cudaSuccess) return e;
        const bool capturing = cap != cudaStreamCaptureStatusNone;
        if (capturing) {
            InvFreq fr;
            for (int c = 0; c < 64; ++c) fr.f[c] = c < d / 2 ? std::pow((double)theta, -2.0 * c / d) : 0.0;
            const int64_t total = (int64_t)T * (d / 2);
            rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(plan->dev, d / 2, fr, mp->rope_table);
            count_launch();
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
            mp->rope_theta = 0.f;                // whoever calls next outside a capture fills it for itself
        } else if (mp->rope_theta != theta) {
            InvFreq fr;
            for (int c = 0; c < 64; ++c) fr.f[c] = c < d / 2 ? std::pow((double)theta, -2.0 * c / d) : 0.0;
            const int64_t total = (int64_t)T * (d / 2);
            // a call with the previous base may still be reading the table that is about to be replaced (rare: one
            // model has one base)
            if (mp->rope_theta > 0.f && (e = cudaDeviceSynchronize()) != cudaSuccess) return e;
            rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(plan->dev, d / 2, fr, mp->rope_table);
            count_launch();
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
            if ((e = cudaEventRecord(mp->ev_table, stream)) != cudaSuccess) return e;
            mp->rope_theta = theta;
            mp->table_stream = stream;
        } else if (mp->table_stream != stream) {
            if ((e = cudaStreamWaitEvent(stream, mp->ev_table, 0)) != cudaSuccess) return e;
        }
        a.trig = mp->rope_table;
    }
    if (pair) e = bf16 ? launch_form<true, true>(a, mx, mw, plan->num_sms, stream) : launch_form<false, true>(a, mx, mw, plan->num_sms, stream);
    else e = bf16 ? launch_form<true, false>(a, mx, mw, plan->num_sms, stream) : launch_form<false, false>(a, mx, mw, plan->num_sms, stream);
    return e;
}

}  // namespace hat
