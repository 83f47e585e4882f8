// Streaming (verify-class) chunk attention: up to 16 query rows of one request against a long key range, bound by
// HBM bandwidth.  One CTA = one work item (request, key range) x one head, four warps; warp w owns pages
// w, w+4, ... of the range and streams them through its own three-slot shared-memory ring.  A page of one head is
// fetched by TMA as 2 KiB boxes (64 columns x 16 tokens, 128-byte swizzle) whose arrival is counted on the slot's
// mbarrier, so a page costs the warp a handful of instructions instead of address arithmetic for 32 vector loads.
// The math is warp-level mma.sync m16n8k16 (queries padded to 16 rows, fp32 accumulate) with an online softmax whose
// reference maximum only moves when it grows by more than 2^8, so the output accumulator is rarely rescaled.
// The four warps are combined through shared memory; the result goes to out/lse or, for a cut request, to the
// partial rows the merge kernel reads.  Waits on the mbarriers are bounded and report through the plan's status word.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "hat_internal.h"
#include "tma_desc.h"

namespace hat {
namespace {

constexpr int kWarps = 4;
constexpr int kSlots = 3;
constexpr float kMoveThreshold = 8.0f;      // log2 units

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
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Byte offset of 16-byte vector c of token row `row` in a page as TMA lays it down: two 2 KiB column halves,
// rows of 128 bytes, the vector index XORed with the row (128-byte swizzle).
template <int D>
__device__ __forceinline__ uint32_t page_off(int row, int c) {
    if constexpr (D == 128) return (uint32_t)((c >> 3) * 2048 + row * 128 + (((c & 7) ^ (row & 7)) << 4));
    else return (uint32_t)(row * 128 + ((c ^ (row & 7)) << 4));
}
// The Q tile is written by ordinary stores: rows of D*2 bytes, vector index XORed with the row.
template <int D>
__device__ __forceinline__ uint32_t q_off(int row, int c) { return (uint32_t)(row * (D * 2) + ((c ^ (row & 7)) << 4)); }

template <bool BF16, int D>
__global__ void __launch_bounds__(kWarps * 32)
attn_stream_kernel(AttnArgs a, const WorkItem* __restrict__ items, int n_sub, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v) {
    using T = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    constexpr int CH = D / 8, ON = D / 8, HALVES = D / 64;
    constexpr uint32_t PAGE_BYTES = 16 * D * 2;              // K (or V) of one page of one head
    constexpr uint32_t SLOT_BYTES = 2 * PAGE_BYTES;          // K then V
    constexpr uint32_t Q_BYTES = 16 * D * 2;                 // multiple of 1024 for D = 64 and 128

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Q_BYTES + kWarps * kSlots * SLOT_BYTES);
    const uint32_t sbase = s_u32(smem);

    // A CTA serves one K/V head and 16 of the request's (chunk row i, query head gq of the head's group) pairs:
    // MMA row m of slab `sub` is pair number sub * 16 + m = i * G + gq, so K/V are read once for the whole group.
    const WorkItem item = items[blockIdx.y];
    const int h = blockIdx.x / n_sub, sub = blockIdx.x % n_sub;
    const int H = a.plan.num_heads, G = a.plan.group;
    const int r = item.req;
    const int P = a.plan.prefix_len[r];
    const int C = a.plan.chunk_len[r];
    if (sub * 16 >= C * G) return;                            // this request has fewer pairs
    const int row_base = a.plan.cu_chunk[r];
    const int32_t* __restrict__ table = a.plan.block_table + (int64_t)r * a.plan.max_pages;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;

    if (tid < kWarps * kSlots) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(s_u32(bars + tid)));
    if (tid == 0) {
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    // Q tile (rows >= C are zero)
    {
        const T* __restrict__ q = static_cast<const T*>(a.q);
        for (int idx = tid; idx < 16 * CH; idx += kWarps * 32) {
            const int row = idx / CH, c = idx % CH;
            uint4 v = make_uint4(0, 0, 0, 0);
            const int pair = sub * 16 + row, i = pair / G;
            if (i < C)
                v = __ldg(reinterpret_cast<const uint4*>(q + ((int64_t)(row_base + i) * H + h * G + pair % G) * D) + c);
            *reinterpret_cast<uint4*>(smem + q_off<D>(row, c)) = v;
        }
    }
    __syncthreads();

    // ---- this warp's pages and its ring
    const int n_pages = (item.kv_end - item.kv_begin + kPageSize - 1) / kPageSize;
    const int n_my = n_pages > warp ? (n_pages - warp + kWarps - 1) / kWarps : 0;
    const uint32_t ring = sbase + Q_BYTES + warp * (kSlots * SLOT_BYTES);
    const uint32_t bar0 = s_u32(bars + warp * kSlots);
    // lanes 0 .. 2*HALVES-1 each move one box: (K or V, column half)
    auto issue = [&](int ti, int slot) {
        const int kb = item.kv_begin + ti * kPageSize;
        const uint32_t bar = bar0 + slot * 8;
        if (lane == 0)
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(SLOT_BYTES) : "memory");
        __syncwarp();
        if (lane < 2 * HALVES) {
            const int is_v = lane / HALVES, half = lane % HALVES;
            const int page = HAT_IN_RANGE(__ldg(table + HAT_IN_RANGE(kb / kPageSize, a.plan.max_pages, a.plan.status)), a.plan.num_pages, a.plan.status);
            const uint32_t dst = ring + slot * SLOT_BYTES + is_v * PAGE_BYTES + half * 2048;
            const CUtensorMap* map = is_v ? &map_v : &map_k;
            asm volatile(
                "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
                ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(half * 64), "r"(0), "r"(h), "r"(page), "r"(bar)
                : "memory");
        }
    };
#pragma unroll
    for (int s = 0; s < kSlots - 1; ++s)
        if (s < n_my) issue(warp + s * kWarps, s);

    uint32_t qf[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const int mi = lane >> 3;
        ldsm4(qf[ks], sbase + q_off<D>((mi & 1) * 8 + (lane & 7), ks * 2 + (mi >> 1)));
    }

    float o[ON][4];
#pragma unroll
    for (int n = 0; n < ON; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // reference maxima (log2 units) and row sums, rows g and g+8
    // chunk rows of MMA rows g and g+8, and the chunk positions each may see: bit c <=> key P + c.  The causal rule
    // (Sec. 2.1 / 3.4: a linear draft sequence) is bits 0..i; a token tree supplies its own words
    const int i0 = (sub * 16 + g) / G, i1 = (sub * 16 + g + 8) / G;
    uint32_t bits0 = i0 < C ? (2u << i0) - 1u : 0u, bits1 = i1 < C ? (2u << i1) - 1u : 0u;
    if (a.plan.tree_mask != nullptr) {
        if (i0 < C) bits0 = __ldg(a.plan.tree_mask + row_base + i0);
        if (i1 < C) bits1 = __ldg(a.plan.tree_mask + row_base + i1);
    }
    const int kend = item.kv_end;
    bool ok = true;

    for (int it = 0; it < n_my; ++it) {
        const int slot = it % kSlots;
        // the slot that page it+2 goes to was read in the previous iteration: every lane is past those reads here
        __syncwarp();
        if (it + kSlots - 1 < n_my) issue(warp + (it + kSlots - 1) * kWarps, (it + kSlots - 1) % kSlots);
        {
            const uint32_t bar = bar0 + slot * 8, parity = (it / kSlots) & 1;
            if (!mbar_try(bar, parity)) {
                const long long t0 = clock64();
                while (!mbar_try(bar, parity)) {
                    if (clock64() - t0 > a.wait_cycles) { ok = false; break; }
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
        }
        const int kb = item.kv_begin + (warp + it * kWarps) * kPageSize;
        const uint32_t kst = ring + slot * SLOT_BYTES, vst = kst + PAGE_BYTES;
        if (kb + kPageSize > kend) {
            // the range ends inside this page: the slots past it hold stale tokens; zero their V rows so that
            // 0 * garbage cannot produce NaN (their scores are masked below)
            const int first = kend - kb;
            for (int idx = lane; idx < (kPageSize - first) * CH; idx += 32) {
                const int row = first + idx / CH, c = idx % CH;
                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(vst + page_off<D>(row, c)), "r"(0));
            }
            __syncwarp();
        }

        // S = Q K^T for the 16 keys of the page
        float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const int mi = lane >> 3;
            uint32_t b[4];
            ldsm4(b, kst + page_off<D>((mi >> 1) * 8 + (lane & 7), ks * 2 + (mi & 1)));
            mma16816<BF16>(s[0], qf[ks], b[0], b[1]);
            mma16816<BF16>(s[1], qf[ks], b[2], b[3]);
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
        if (kb + kPageSize > min(P, kend)) {                     // the page holds chunk positions or ends the range
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                const int j = kb + n * 8 + 2 * t4;
                // key j of the range: everything below P, bit j - P from there on (j < kend <= P + 16 bounds the shift)
                const bool in0 = j < kend, in1 = j + 1 < kend;
                const uint32_t sh0 = (uint32_t)min(max(j - P, 0), 31), sh1 = (uint32_t)min(max(j + 1 - P, 0), 31);
                const bool a0 = in0 && (j < P || ((bits0 >> sh0) & 1u));
                const bool a1 = in1 && (j + 1 < P || ((bits0 >> sh1) & 1u));
                const bool b0 = in0 && (j < P || ((bits1 >> sh0) & 1u));
                const bool b1 = in1 && (j + 1 < P || ((bits1 >> sh1) & 1u));
                s[n][0] = a0 ? s[n][0] * a.scale_log2 : -INFINITY;
                s[n][1] = a1 ? s[n][1] * a.scale_log2 : -INFINITY;
                s[n][2] = b0 ? s[n][2] * a.scale_log2 : -INFINITY;
                s[n][3] = b1 ? s[n][3] * a.scale_log2 : -INFINITY;
            }
        } else {
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                s[n][0] *= a.scale_log2; s[n][1] *= a.scale_log2; s[n][2] *= a.scale_log2; s[n][3] *= a.scale_log2;
            }
        }
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
            mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        // move a row's reference maximum only when the new maximum exceeds it by more than the threshold; weights
        // then stay below 2^8 and the accumulators are rescaled only on the (rare) iterations where some row moved
        const bool mv0 = mx0 > m0 + kMoveThreshold, mv1 = mx1 > m1 + kMoveThreshold;
        if (__any_sync(0xffffffffu, mv0 || mv1)) {
            const float al0 = mv0 ? ((m0 == -INFINITY) ? 0.f : exp2f(m0 - mx0)) : 1.f;
            const float al1 = mv1 ? ((m1 == -INFINITY) ? 0.f : exp2f(m1 - mx1)) : 1.f;
            if (mv0) m0 = mx0;
            if (mv1) m1 = mx1;
            l0 *= al0; l1 *= al1;
#pragma unroll
            for (int n = 0; n < ON; ++n) { o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1; }
        }
        const float r0 = (m0 == -INFINITY) ? 0.f : m0, r1 = (m1 == -INFINITY) ? 0.f : m1;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            s[n][0] = exp2f(s[n][0] - r0); s[n][1] = exp2f(s[n][1] - r0);
            s[n][2] = exp2f(s[n][2] - r1); s[n][3] = exp2f(s[n][3] - r1);
            l0 += s[n][0] + s[n][1];
            l1 += s[n][2] + s[n][3];
        }
        // O += P V
        uint32_t pa[4], pl[4];
        pa[0] = pack2<BF16>(s[0][0], s[0][1]); pa[1] = pack2<BF16>(s[0][2], s[0][3]);
        pa[2] = pack2<BF16>(s[1][0], s[1][1]); pa[3] = pack2<BF16>(s[1][2], s[1][3]);
        if constexpr (BF16) {
            // bf16 keeps 8 significant bits: a second operand carries what the rounding of P dropped
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
            ldsm4t(b, vst + page_off<D>((mi & 1) * 8 + (lane & 7), dn * 2 + (mi >> 1)));
            mma16816<BF16>(o[2 * dn], pa, b[0], b[1]);
            mma16816<BF16>(o[2 * dn + 1], pa, b[2], b[3]);
            if constexpr (BF16) {
                mma16816<BF16>(o[2 * dn], pl, b[0], b[1]);
                mma16816<BF16>(o[2 * dn + 1], pl, b[2], b[3]);
            }
        }
    }
    if (!ok) {
        // a transfer never arrived: report it, then give the copies still in flight a bounded time to land
        if (lane == 0) atomicExch(a.plan.status, 1);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
        for (int n = 0; n < ON; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
        l0 = l1 = 0.f;
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- combine the four warps through shared memory (fragment positions are identical in each)
    constexpr int VALS = ON * 4 + 4;
    static_assert((kWarps - 1) * VALS * 32 * 4 <= kWarps * kSlots * (int)SLOT_BYTES, "exchange buffer must fit in the rings");
    __syncthreads();                                             // every ring is idle: no load is outstanding
    float* xbuf = reinterpret_cast<float*>(smem + Q_BYTES);
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
    for (int k = 1; k < kWarps; ++k) {
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
    for (int k = 1; k < kWarps; ++k) {
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

    // ---- normalise and store (final rows, or partial rows for the merge kernel)
    const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
    constexpr float kLn2 = 0.6931471805599453f;
    const float lse0 = l0 > 0.f ? (mt0 + log2f(l0)) * kLn2 : -INFINITY;
    const float lse1 = l1 > 0.f ? (mt1 + log2f(l1)) * kLn2 : -INFINITY;
    const int hq0 = h * G + (sub * 16 + g) % G, hq1 = h * G + (sub * 16 + g + 8) % G;
    float* obase; float* lbase; int64_t r0, r1;
    if (item.part < 0) { obase = a.out; lbase = a.lse; r0 = row_base + i0; r1 = row_base + i1; }
    else { obase = a.part_out; lbase = a.part_lse; r0 = item.part + i0; r1 = item.part + i1; }
    const bool to16 = item.part < 0 && a.out16 != nullptr;      // final rows in the 16-bit output type
    if (i0 < C) {
        const int64_t at = (r0 * H + hq0) * D + 2 * t4;
        if (to16) {
#pragma unroll
            for (int n = 0; n < ON; ++n)
                *reinterpret_cast<uint32_t*>(static_cast<uint16_t*>(a.out16) + at + n * 8) = pack_out16(o[n][0] * inv0, o[n][1] * inv0, a.out16_bf16);
        } else {
#pragma unroll
            for (int n = 0; n < ON; ++n) *reinterpret_cast<float2*>(obase + at + n * 8) = make_float2(o[n][0] * inv0, o[n][1] * inv0);
        }
        if (t4 == 0) lbase[r0 * H + hq0] = lse0;
    }
    if (i1 < C) {
        const int64_t at = (r1 * H + hq1) * D + 2 * t4;
        if (to16) {
#pragma unroll
            for (int n = 0; n < ON; ++n)
                *reinterpret_cast<uint32_t*>(static_cast<uint16_t*>(a.out16) + at + n * 8) = pack_out16(o[n][2] * inv1, o[n][3] * inv1, a.out16_bf16);
        } else {
#pragma unroll
            for (int n = 0; n < ON; ++n) *reinterpret_cast<float2*>(obase + at + n * 8) = make_float2(o[n][2] * inv1, o[n][3] * inv1);
        }
        if (t4 == 0) lbase[r1 * H + hq1] = lse1;
    }
}

template <bool BF16, int D>
cudaError_t launch_one(const hat_plan* plan, const AttnArgs& args, const CUtensorMap& mk, const CUtensorMap& mv,
                       cudaStream_t stream) {
    constexpr int smem = 1024 + 16 * D * 2 + kWarps * kSlots * 2 * (16 * D * 2) + kWarps * kSlots * 8 + 64;
    auto kern = attn_stream_kernel<BF16, D>;
    cudaError_t e = smem_attr_once(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
    kern<<<dim3(plan->num_kv_heads * plan->verify_subtiles, (unsigned)plan->verify_items.size()), kWarps * 32, smem, stream>>>(
        args, plan->dev.verify_items, plan->verify_subtiles, mk, mv);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool stream_layout_supported(int dtype, int head_dim, int num_pages, int H, int64_t stride_page, int64_t stride_token,
                             int64_t stride_head) {
    CUtensorMap m;
    // the encoder checks alignment and ranges only; any 16-byte aligned address will do for the probe
    return tma_encode_pool_map(&m, dtype == HAT_DTYPE_BF16, reinterpret_cast<const void*>(uintptr_t(1) << 30), head_dim,
                               num_pages, H, stride_page, stride_token, stride_head);
}

cudaError_t launch_attn_stream(const hat_plan* plan, const AttnArgs& args, cudaStream_t stream) {
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    const CUtensorMap *mk = nullptr, *mv = nullptr;
    if (!plan_pool_maps(plan, args.cache, &mk, &mv)) return cudaErrorInvalidValue;
    if (plan->head_dim == 128)
        return bf16 ? launch_one<true, 128>(plan, args, *mk, *mv, stream) : launch_one<false, 128>(plan, args, *mk, *mv, stream);
    return bf16 ? launch_one<true, 64>(plan, args, *mk, *mv, stream) : launch_one<false, 64>(plan, args, *mk, *mv, stream);
}

}  // namespace hat
