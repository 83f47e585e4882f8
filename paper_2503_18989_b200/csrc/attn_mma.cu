// Chunk attention on warp-level mma.sync (m16n8k16, fp32 accumulate) with an online softmax.
//
// One CTA handles one work item (a tile of query rows of one request and a range of its keys) for
// one head.  Warps are arranged as WM row groups x WN key groups: a row group owns 16 query rows, a
// key group owns every WN-th stage of the key range and streams it through its own cp.async ring
// of 16-byte vectors (swizzled in shared memory so ldmatrix is conflict free).  Key groups are
// combined through shared memory at the end.  Two instantiations are used:
//   streaming (verify-class, <= 16 rows):  WM=1, WN=4, one page per stage  -> HBM-bound K/V streaming
//   tile      (prefill-class, 64 rows):    WM=4, WN=1, four pages per stage
// Results are written either as final out/lse rows or as partial rows for the merge kernel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "hat_internal.h"

namespace hat {
namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

template <typename T>
struct Mma;
template <>
struct Mma<__half> {
    static __device__ __forceinline__ void run(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static constexpr bool kSplitP = false;
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
    static __device__ __forceinline__ uint32_t pack_residual(float, float, uint32_t) { return 0u; }
};
template <>
struct Mma<__nv_bfloat16> {
    static __device__ __forceinline__ void run(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static constexpr bool kSplitP = true;
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
    // what the rounding in pack() dropped: (lo, hi) minus the packed pair, itself rounded to bf16
    static __device__ __forceinline__ uint32_t pack_residual(float lo, float hi, uint32_t packed) {
        const float plo = __uint_as_float(packed << 16), phi = __uint_as_float(packed & 0xffff0000u);
        return pack(lo - plo, hi - phi);
    }
};

template <int WM>
__device__ __forceinline__ void group_barrier(int kg) {
    if constexpr (WM == 1) {
        __syncwarp();
    } else {
        asm volatile("bar.sync %0, %1;\n" ::"r"(kg + 1), "n"(WM * 32));
    }
}

// Byte offset of 16-byte vector `c` of row `row` inside a swizzled [rows][D] 16-bit tile.
template <int D>
__device__ __forceinline__ uint32_t swz(int row, int c) {
    return (uint32_t)(row * (D * 2) + ((c ^ (row & 7)) << 4));
}

template <typename T, int D, int WM, int WN, int PG, int STAGES>
__global__ void __launch_bounds__(WM * WN * 32)
attn_mma_kernel(AttnArgs a, const WorkItem* __restrict__ items) {
    constexpr int ROWS = 16 * WM;           // query rows per CTA
    constexpr int KB = kPageSize * PG;      // keys per stage
    constexpr int CH = D / 8;               // 16-byte vectors per row
    constexpr int NT = WM * WN * 32;
    constexpr int GT = WM * 32;             // threads of one key group
    constexpr int TILE_BYTES = KB * D * 2;  // one K (or V) stage
    constexpr int Q_BYTES = ROWS * D * 2;
    constexpr int ON = D / 8;               // output n-tiles per warp

    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t smem_base = smem_u32(smem);

    const WorkItem item = items[blockIdx.y];
    const int h = blockIdx.x;
    const int H = a.plan.num_heads;
    const int r = item.req;
    const int P = a.plan.prefix_len[r];
    const int C = a.plan.chunk_len[r];
    const int row_base = a.plan.cu_chunk[r];
    const int32_t* __restrict__ table = a.plan.block_table + (int64_t)r * a.plan.max_pages;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int kg = warp / WM, wm = warp % WM;
    const int g = lane >> 2, t4 = lane & 3;
    const int tid_g = tid - kg * GT;

    const T* __restrict__ kpool = static_cast<const T*>(a.cache.k_pool);
    const T* __restrict__ vpool = static_cast<const T*>(a.cache.v_pool);
    const int64_t head_off = (int64_t)(h / a.plan.group) * a.cache.stride_head;   // query head h reads K/V head h / G

    // ---- stage loader for this key group: tile index ti -> keys [kv_begin + ti*KB, +KB)
    const uint32_t stage_base = smem_base + Q_BYTES + kg * (STAGES * 2 * TILE_BYTES);
    auto issue_load = [&](int ti, int slot) {
        const int kb = item.kv_begin + ti * KB;
        const uint32_t kdst = stage_base + slot * (2 * TILE_BYTES);
        const uint32_t vdst = kdst + TILE_BYTES;
#pragma unroll
        for (int idx = tid_g; idx < KB * CH; idx += GT) {
            const int row = idx / CH, c = idx % CH;
            const int key = kb + row;
            const uint32_t off = swz<D>(row, c);
            if (key < item.kv_end) {
                const int page = HAT_IN_RANGE(__ldg(table + HAT_IN_RANGE(key / kPageSize, a.plan.max_pages, a.plan.status)), a.plan.num_pages, a.plan.status);
                const int64_t e = (int64_t)page * a.cache.stride_page + (int64_t)(key % kPageSize) * a.cache.stride_token +
                                  head_off + c * 8;
                cp_async16(kdst + off, kpool + e);
                cp_async16(vdst + off, vpool + e);
            } else {
                // beyond the key range: never dereference the table; zero rows keep P*V finite
                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(kdst + off), "r"(0));
                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(vdst + off), "r"(0));
            }
        }
    };

    const int n_tiles = (item.kv_end - item.kv_begin + KB - 1) / KB;
    const int n_my = n_tiles > kg ? (n_tiles - kg + WN - 1) / WN : 0;

    // ---- prologue: start the ring, then bring Q in while the first stages fly
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < n_my) issue_load(kg + s * WN, s);
        cp_async_commit();
    }
    {
        const T* __restrict__ q = static_cast<const T*>(a.q);
        for (int idx = tid; idx < ROWS * CH; idx += NT) {
            const int row = idx / CH, c = idx % CH;
            const int i = item.row0 + row;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (i < C) v = __ldg(reinterpret_cast<const uint4*>(q + ((int64_t)(row_base + i) * H + h) * D) + c);
            *reinterpret_cast<uint4*>(smem + swz<D>(row, c)) = v;
        }
    }
    __syncthreads();
    uint32_t qf[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const int mi = lane >> 3;
        const int row = wm * 16 + (mi & 1) * 8 + (lane & 7);
        ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], smem_base + swz<D>(row, ks * 2 + (mi >> 1)));
    }

    float o[ON][4];
#pragma unroll
    for (int n = 0; n < ON; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows g and g+8 (log2 domain)
    const int lim0 = P + item.row0 + wm * 16 + g;                // last visible key of row g
    const int lim1 = lim0 + 8;
    // token tree (short chunks only): the words say which chunk positions rows g and g+8 see
    const bool tree = a.plan.tree_mask != nullptr && C <= 16;
    uint32_t bits0 = 0, bits1 = 0;
    if (tree) {
        const int i0 = item.row0 + wm * 16 + g;
        if (i0 < C) bits0 = __ldg(a.plan.tree_mask + row_base + i0);
        if (i0 + 8 < C) bits1 = __ldg(a.plan.tree_mask + row_base + i0 + 8);
    }
    const int warp_last_visible = tree ? P + C - 1 : P + item.row0 + wm * 16 + 15;

    for (int it = 0; it < n_my; ++it) {
        cp_async_wait<STAGES - 2>();
        group_barrier<WM>(kg);
        {
            const int nx = it + STAGES - 1;
            if (nx < n_my) issue_load(kg + nx * WN, nx % STAGES);
            cp_async_commit();
        }
        const int kb = item.kv_begin + (kg + it * WN) * KB;
        if (kb > warp_last_visible) continue;                    // nothing in this stage is visible to this warp
        const uint32_t kst = stage_base + (it % STAGES) * (2 * TILE_BYTES);
        const uint32_t vst = kst + TILE_BYTES;

        // S = Q K^T
        float s[KB / 8][4];
#pragma unroll
        for (int n = 0; n < KB / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < KB / 16; ++np) {
                const int mi = lane >> 3;
                const int key = np * 16 + (mi >> 1) * 8 + (lane & 7);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, kst + swz<D>(key, ks * 2 + (mi & 1)));
                Mma<T>::run(s[2 * np], qf[ks], b0, b1);
                Mma<T>::run(s[2 * np + 1], qf[ks], b2, b3);
            }
        }

        // scale, mask, running max
        const int kend = item.kv_end;
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < KB / 8; ++n) {
            const int j = kb + n * 8 + 2 * t4;
            bool a0 = j <= lim0, a1 = j + 1 <= lim0, b0 = j <= lim1, b1 = j + 1 <= lim1;
            if (tree) {
                const uint32_t sh0 = (uint32_t)min(max(j - P, 0), 31), sh1 = (uint32_t)min(max(j + 1 - P, 0), 31);
                a0 = j < P || ((bits0 >> sh0) & 1u); a1 = j + 1 < P || ((bits0 >> sh1) & 1u);
                b0 = j < P || ((bits1 >> sh0) & 1u); b1 = j + 1 < P || ((bits1 >> sh1) & 1u);
            }
            s[n][0] = (a0 && j < kend) ? s[n][0] * a.scale_log2 : -INFINITY;
            s[n][1] = (a1 && j + 1 < kend) ? s[n][1] * a.scale_log2 : -INFINITY;
            s[n][2] = (b0 && j < kend) ? s[n][2] * a.scale_log2 : -INFINITY;
            s[n][3] = (b1 && j + 1 < kend) ? s[n][3] * a.scale_log2 : -INFINITY;
            mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
            mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0;        // all keys so far masked: keep exp2 finite
        const float ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float al0 = exp2f(m0 - ms0), al1 = exp2f(m1 - ms1);
        m0 = mn0; m1 = mn1;
        float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
        for (int n = 0; n < KB / 8; ++n) {
            s[n][0] = exp2f(s[n][0] - ms0);
            s[n][1] = exp2f(s[n][1] - ms0);
            s[n][2] = exp2f(s[n][2] - ms1);
            s[n][3] = exp2f(s[n][3] - ms1);
            rs0 += s[n][0] + s[n][1];
            rs1 += s[n][2] + s[n][3];
        }
        l0 = l0 * al0 + rs0;
        l1 = l1 * al1 + rs1;
#pragma unroll
        for (int n = 0; n < ON; ++n) {
            o[n][0] *= al0; o[n][1] *= al0;
            o[n][2] *= al1; o[n][3] *= al1;
        }

        // O += P V
#pragma unroll
        for (int kp = 0; kp < KB / 16; ++kp) {
            uint32_t pa[4], pl[4];
            pa[0] = Mma<T>::pack(s[2 * kp][0], s[2 * kp][1]);
            pa[1] = Mma<T>::pack(s[2 * kp][2], s[2 * kp][3]);
            pa[2] = Mma<T>::pack(s[2 * kp + 1][0], s[2 * kp + 1][1]);
            pa[3] = Mma<T>::pack(s[2 * kp + 1][2], s[2 * kp + 1][3]);
            if constexpr (Mma<T>::kSplitP) {
                // bf16 keeps 8 significant bits: carry the rounding remainder of P in a second operand
                pl[0] = Mma<T>::pack_residual(s[2 * kp][0], s[2 * kp][1], pa[0]);
                pl[1] = Mma<T>::pack_residual(s[2 * kp][2], s[2 * kp][3], pa[1]);
                pl[2] = Mma<T>::pack_residual(s[2 * kp + 1][0], s[2 * kp + 1][1], pa[2]);
                pl[3] = Mma<T>::pack_residual(s[2 * kp + 1][2], s[2 * kp + 1][3], pa[3]);
            }
#pragma unroll
            for (int dn = 0; dn < D / 16; ++dn) {
                const int mi = lane >> 3;
                const int key = kp * 16 + (mi & 1) * 8 + (lane & 7);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(b0, b1, b2, b3, vst + swz<D>(key, dn * 2 + (mi >> 1)));
                Mma<T>::run(o[2 * dn], pa, b0, b1);
                Mma<T>::run(o[2 * dn + 1], pa, b2, b3);
                if constexpr (Mma<T>::kSplitP) {
                    Mma<T>::run(o[2 * dn], pl, b0, b1);
                    Mma<T>::run(o[2 * dn + 1], pl, b2, b3);
                }
            }
        }
    }

    // row sums live spread over the four lanes of a quad
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- combine key groups through shared memory (fragment positions are identical across groups)
    if constexpr (WN > 1) {
        constexpr int VALS = ON * 4 + 4;
        cp_async_wait<0>();
        __syncthreads();                                         // every ring is idle: reuse it
        float* xbuf = reinterpret_cast<float*>(smem + Q_BYTES);
        if (kg > 0) {
            float* dst = xbuf + ((kg - 1) * WM + wm) * (VALS * 32) + lane;
#pragma unroll
            for (int n = 0; n < ON; ++n) {
#pragma unroll
                for (int k = 0; k < 4; ++k) dst[(n * 4 + k) * 32] = o[n][k];
            }
            dst[(ON * 4 + 0) * 32] = m0;
            dst[(ON * 4 + 1) * 32] = m1;
            dst[(ON * 4 + 2) * 32] = l0;
            dst[(ON * 4 + 3) * 32] = l1;
        }
        __syncthreads();
        if (kg > 0) return;
        float mt0 = m0, mt1 = m1;
#pragma unroll
        for (int k = 1; k < WN; ++k) {
            const float* src = xbuf + ((k - 1) * WM + wm) * (VALS * 32) + lane;
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
            const float* src = xbuf + ((k - 1) * WM + wm) * (VALS * 32) + lane;
            const float w0 = exp2f(src[(ON * 4 + 0) * 32] - ms0), w1 = exp2f(src[(ON * 4 + 1) * 32] - ms1);
            l0 += w0 * src[(ON * 4 + 2) * 32];
            l1 += w1 * src[(ON * 4 + 3) * 32];
#pragma unroll
            for (int n = 0; n < ON; ++n) {
                o[n][0] += w0 * src[(n * 4 + 0) * 32];
                o[n][1] += w0 * src[(n * 4 + 1) * 32];
                o[n][2] += w1 * src[(n * 4 + 2) * 32];
                o[n][3] += w1 * src[(n * 4 + 3) * 32];
            }
        }
        m0 = mt0; m1 = mt1;
    }

    // ---- normalise and store (final rows, or partial rows for the merge kernel)
    const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
    constexpr float kLn2 = 0.6931471805599453f;
    const float lse0 = l0 > 0.f ? (m0 + log2f(l0)) * kLn2 : -INFINITY;
    const float lse1 = l1 > 0.f ? (m1 + log2f(l1)) * kLn2 : -INFINITY;
    const int i0 = item.row0 + wm * 16 + g, i1 = i0 + 8;
    float* obase;
    float* lbase;
    int64_t r0, r1;
    if (item.part < 0) {
        obase = a.out; lbase = a.lse;
        r0 = row_base + i0; r1 = row_base + i1;
    } else {
        obase = a.part_out; lbase = a.part_lse;
        r0 = item.part + (i0 - item.row0); r1 = item.part + (i1 - item.row0);
    }
    const bool to16 = item.part < 0 && a.out16 != nullptr;      // final rows in the 16-bit output type
    if (i0 < C) {
        const int64_t at = (r0 * H + h) * D + 2 * t4;
#pragma unroll
        for (int n = 0; n < ON; ++n) {
            if (to16) *reinterpret_cast<uint32_t*>(static_cast<uint16_t*>(a.out16) + at + n * 8) = pack_out16(o[n][0] * inv0, o[n][1] * inv0, a.out16_bf16);
            else *reinterpret_cast<float2*>(obase + at + n * 8) = make_float2(o[n][0] * inv0, o[n][1] * inv0);
        }
        if (t4 == 0) lbase[r0 * H + h] = lse0;
    }
    if (i1 < C) {
        const int64_t at = (r1 * H + h) * D + 2 * t4;
#pragma unroll
        for (int n = 0; n < ON; ++n) {
            if (to16) *reinterpret_cast<uint32_t*>(static_cast<uint16_t*>(a.out16) + at + n * 8) = pack_out16(o[n][2] * inv1, o[n][3] * inv1, a.out16_bf16);
            else *reinterpret_cast<float2*>(obase + at + n * 8) = make_float2(o[n][2] * inv1, o[n][3] * inv1);
        }
        if (t4 == 0) lbase[r1 * H + h] = lse1;
    }
}

template <typename T, int D, int WM, int WN, int PG, int STAGES>
cudaError_t launch_one(const AttnArgs& args, const WorkItem* items, int num_items, int H, cudaStream_t stream) {
    constexpr int smem = 16 * WM * D * 2 + WN * STAGES * 2 * (kPageSize * PG * D * 2);
    static_assert((WN - 1) * WM * (D / 8 * 4 + 4) * 32 * 4 <= WN * STAGES * 2 * (kPageSize * PG * D * 2),
                  "key-group exchange buffer must fit in the stage rings");
    auto kern = attn_mma_kernel<T, D, WM, WN, PG, STAGES>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<dim3(H, num_items), WM * WN * 32, smem, stream>>>(args, items);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_typed(const hat_plan* plan, const AttnArgs& args, bool verify_class, cudaStream_t stream) {
    if (verify_class)
        return launch_one<T, D, 1, 4, 1, 3>(args, plan->dev.verify_items, (int)plan->verify_items.size(),
                                            plan->num_heads, stream);
    return launch_one<T, D, 4, 1, 4, 3>(args, plan->dev.prefill_items, (int)plan->prefill_items.size(),
                                        plan->num_heads, stream);
}

}  // namespace

cudaError_t launch_attn_mma(const hat_plan* plan, const AttnArgs& args, bool verify_class, cudaStream_t stream) {
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    if (plan->head_dim == 128)
        return bf16 ? launch_typed<__nv_bfloat16, 128>(plan, args, verify_class, stream)
                    : launch_typed<__half, 128>(plan, args, verify_class, stream);
    return bf16 ? launch_typed<__nv_bfloat16, 64>(plan, args, verify_class, stream)
                : launch_typed<__half, 64>(plan, args, verify_class, stream);
}

}  // namespace hat
