// Prefill-chunk attention on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// Persistent kernel, one CTA per SM.  A work unit = up to 256 query rows (two 128-row query tiles) of one request x
// one head x one key range; CTAs draw units (longest first) from a global counter until none is left.  Both query
// tiles of a unit use the same K/V tiles in shared memory, and while one tile's softmax runs the tensor pipe works
// for the other.  Roles:
//   warp 0      draws the next unit and publishes it to the other roles; TMA producer: the unit's Q tiles, then K
//               and V tiles of 128 keys (8 pages x 2 halves of 64 columns, 128-byte swizzle) into a two-slot K ring
//               and a three-slot V ring, completion on mbarriers.  It runs ahead across units: the next unit's Q and
//               first K/V tiles are already landing while the current unit's last tiles and its output are processed
//   warp 1      one thread issues tcgen05.mma: S_t = Q_t K^T for query tile t, then O_t += P_t V with P read
//               from TMEM; tcgen05.commit signals the consumers and frees the ring slots.  Owns the TMEM allocation
//   warps 2-5, 6-9   one warpgroup per query tile, thread = query row = TMEM lane: tcgen05.ld of S, scale/mask/online
//               softmax in registers (reference maximum only moved when it grows by more than 2^8, so O is rarely
//               rescaled), P written back to TMEM as the 16-bit A operand; at the end of a unit O is pulled into
//               registers (which frees the accumulator for the next unit), divided by l and stored with the lse
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512).  P_t(j) overwrites S_t(j) in place (16-bit pairs in
// columns [0,64), the bf16 rounding remainder in [64,128)); S_t(j+1) is issued after P_t V(j) by the same thread, and
// tcgen05 executes one thread's MMAs in issue order, so no extra barrier guards the reuse.
// A unit of at most 128 rows uses both column pairs for the SAME query tile: two chains over alternating key tiles,
// merged by the first chain's warpgroup when the unit ends (see Unit::split).
// Every wait is bounded (about a second by default); a wait that gives up sets the plan's status word, raises a
// CTA-wide abort flag that all other waits observe, and the CTA still frees its TMEM and exits normally.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <type_traits>

#include "hat_internal.h"
#include "tma_desc.h"
#include "tc5_ptx.cuh"

namespace hat {
namespace {
using namespace tc5;

constexpr int kRows = 128;      // query rows per CTA (MMA M)
constexpr int kKeys = 128;      // keys per tile (MMA N of S, K extent of PV)
constexpr int kStagesK = 2;     // ring slots for K tiles
constexpr int kStagesV = 3;     // ring slots for V tiles (V is requested later in a step than K, so it gets the deeper ring)
// one K or V tile, or the Q tile: 128 rows of head_dim 16-bit values (32 KiB at head_dim 128, 16 KiB at 64), stored as
// head_dim / 64 slabs of 64 columns
template <int D> constexpr uint32_t tile_bytes() { return kKeys * D * 2; }
constexpr uint32_t kSlabBytes = kKeys * 64 * 2;          // 16 KiB: 64 columns of 128 rows
constexpr uint32_t kPageBoxBytes = 16 * 64 * 2;          // 2 KiB: one TMA box (16 tokens x 64 columns)
constexpr float kRescaleThreshold = 8.0f;                // log2 units

struct __align__(8) Barriers {
    uint64_t q_full, q_empty;
    uint64_t k_full[kStagesK], k_empty[kStagesK];
    uint64_t v_full[kStagesV], v_empty[kStagesV];
    uint64_t s_full[2], p_ready[2], o_done[2], o_free[2];   // per query tile
    uint64_t unit_full[2], unit_empty[2];                   // two-slot queue of work units, producer -> other roles
    uint64_t x_ready;                                       // split units: chain 1's (reference maximum, row sum) are in xchg
    uint64_t drain;
    long long wait_cycles;                                  // bound of every wait below
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile int unit_slot[2];                              // unit index, or -1 when the work has run out
    float2 xchg[kRows];                                     // split units: per row, chain 1's reference maximum and row sum
};
template <int D> constexpr uint32_t smem_bytes() { return 1024 /*alignment slack*/ + tile_bytes<D>() * (2 + kStagesK + kStagesV) + sizeof(Barriers); }
static_assert(smem_bytes<128>() <= 227 * 1024, "shared memory of one CTA");
constexpr int kThreads = 320;   // producer warp, MMA warp, two softmax warpgroups

// Bounded wait.  Returns false if the wait gave up or another role already did.
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

// What every role needs to know about a unit; all of them decode it the same way.
struct Unit {
    int h, hk, r, P, C, row_base, row0, kv_begin, kv_end, part;   // h: query head, hk = h / G: the K/V head it reads
    int nq;       // query tiles in use (1 or 2)
    int n_all;    // key tiles of the range
    int n_q0;     // key tiles query tile 0 can see (tile 0 does not see the keys past its own last row)
    // A unit with a single query tile would leave the second accumulator pair and warpgroup idle and the tensor
    // pipe waiting through every softmax.  It runs as two chains instead: chain t takes key tiles t, t+2, t+4, ... with
    // the same Q tile, and the two partial results (disjoint key sets) are merged when the unit ends.
    bool split;
    int n_t0, n_t1;   // key tiles of chain (or query tile) 0 and 1
    __device__ __forceinline__ int n_t(int t) const { return t == 0 ? n_t0 : n_t1; }
    // key tile of step s of chain t
    __device__ __forceinline__ int tile_of(int t, int s) const { return split ? 2 * s + t : s; }
};
__device__ __forceinline__ Unit decode_unit(const AttnArgs& a, const WorkItem* __restrict__ items, int unit) {
    const uint32_t e = __ldg(a.plan.tile_units + unit);      // item | head << 16
    const WorkItem it = items[e & 0xffffu];
    Unit u;
    u.h = (int)(e >> 16);
    u.hk = u.h / a.plan.group;
    u.r = it.req;
    u.P = a.plan.prefix_len[u.r];
    u.C = a.plan.chunk_len[u.r];
    u.row_base = a.plan.cu_chunk[u.r];
    u.row0 = it.row0; u.kv_begin = it.kv_begin; u.kv_end = it.kv_end; u.part = it.part;
    u.nq = (u.C - u.row0 > kRows) ? 2 : 1;
    u.n_all = (u.kv_end - u.kv_begin + kKeys - 1) / kKeys;
    const int end0 = min(u.kv_end, u.P + u.row0 + kRows);
    u.n_q0 = u.nq == 1 ? u.n_all : max(0, (end0 - u.kv_begin + kKeys - 1) / kKeys);
    u.split = u.nq == 1;
    u.n_t0 = u.split ? (u.n_all + 1) / 2 : u.n_q0;
    u.n_t1 = u.split ? u.n_all / 2 : (u.nq == 2 ? u.n_all : 0);
    return u;
}

template <bool BF16, int kD>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc5_kernel(AttnArgs a, const WorkItem* __restrict__ items, int total_units, int32_t* work_counter,
                const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v) {
    constexpr uint32_t kTileBytes = tile_bytes<kD>();
    constexpr int kHalves = kD / 64;                             // 64-column slabs (and TMA boxes per page) of a tile
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment: the swizzle pattern and the matrix descriptors assume it
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* q_tiles = smem;                               // 2 x 32 KiB
    unsigned char* k_ring = smem + 2 * kTileBytes;
    unsigned char* v_ring = k_ring + kStagesK * kTileBytes;
    Barriers* bars = reinterpret_cast<Barriers*>(v_ring + kStagesV * kTileBytes);

    const int H = a.plan.num_heads;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t* status = a.plan.status;

    if (threadIdx.x == 0) {
        mbar_init(&bars->q_full, 1); mbar_init(&bars->q_empty, 1);
        for (int s = 0; s < kStagesK; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], 1); }
        for (int s = 0; s < kStagesV; ++s) { mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->s_full[s], 1);
            mbar_init(&bars->p_ready[s], 4);                     // one arrival per softmax warp
            mbar_init(&bars->o_done[s], 1);
            mbar_init(&bars->o_free[s], 4);
            mbar_init(&bars->unit_full[s], 1);
            mbar_init(&bars->unit_empty[s], 1 + 8);              // the MMA thread and every softmax warp
        }
        mbar_init(&bars->x_ready, 4);
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
        // ------------------------------------------------------------------ unit fetch + TMA producer
        // lane l < 16 moves box (page l/2 of the tile, column half l%2)
        const int pg = lane / kHalves, half = lane % kHalves;
        int kt = 0;                                              // K/V tiles issued so far, over all units
        bool ok = true;
        for (int un = 0; ok; ++un) {
            const int slot = un & 1;
            if (un >= 2) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->unit_empty[slot], ((un >> 1) - 1) & 1, bars, status));
                if (!ok) break;
            }
            int unit = 0;
            if (lane == 0) {
                unit = atomicAdd(work_counter, 1);
                if (unit >= total_units) unit = -1;
                bars->unit_slot[slot] = unit;
                mbar_arrive(&bars->unit_full[slot]);             // release: the slot is written before the arrival
            }
            unit = __shfl_sync(0xffffffffu, unit, 0);
            if (unit < 0) break;
            const Unit u = decode_unit(a, items, unit);
            const int32_t* __restrict__ table = a.plan.block_table + (int64_t)u.r * a.plan.max_pages;
            // Q tiles: the previous unit's last S must have read the old ones
            if (un > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->q_empty, (un - 1) & 1, bars, status));
                if (!ok) break;
            }
            if (lane == 0) mbar_expect_tx(&bars->q_full, u.nq * kTileBytes);
            __syncwarp();
            if (lane < kHalves * u.nq)      // lane = kHalves * (query tile) + (column half)
                tma_load_3d(smem_u32(q_tiles) + (lane / kHalves) * kTileBytes + (lane % kHalves) * kSlabBytes, &map_q, (lane % kHalves) * 64, u.h,
                            u.row_base + u.row0 + (lane / kHalves) * kRows, &bars->q_full);
            for (int j = 0; j < u.n_all; ++j, ++kt) {
                const int sk = kt % kStagesK, sv = kt % kStagesV;
                const int kb = u.kv_begin + j * kKeys;
                const int npages = (min(u.kv_end, kb + kKeys) - kb + kPageSize - 1) / kPageSize;
                int page = 0;
                if (lane < 8 * kHalves && pg < npages)
                    page = HAT_IN_RANGE(__ldg(table + HAT_IN_RANGE(kb / kPageSize + pg, a.plan.max_pages, status)), a.plan.num_pages, status);
                HAT_CHECK(sk < kStagesK && sv < kStagesV, status);
                if (kt >= kStagesK) ok = mbar_wait(&bars->k_empty[sk], ((kt / kStagesK) & 1) ^ 1, bars, status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane == 0) mbar_expect_tx(&bars->k_full[sk], npages * kHalves * kPageBoxBytes);
                __syncwarp();
                if (lane < 8 * kHalves && pg < npages)
                    tma_load_4d(smem_u32(k_ring) + sk * kTileBytes + half * kSlabBytes + pg * kPageBoxBytes, &map_k, half * 64, 0,
                                u.hk, page, &bars->k_full[sk]);
                if (kt >= kStagesV) ok = mbar_wait(&bars->v_empty[sv], ((kt / kStagesV) & 1) ^ 1, bars, status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (a.withhold && kt == 0) continue;         // self test: this V tile never arrives, its consumers give up
                if (lane == 0) mbar_expect_tx(&bars->v_full[sv], npages * kHalves * kPageBoxBytes);
                __syncwarp();
                if (lane < 8 * kHalves && pg < npages)
                    tma_load_4d(smem_u32(v_ring) + sv * kTileBytes + half * kSlabBytes + pg * kPageBoxBytes, &map_v, half * 64, 0,
                                u.hk, page, &bars->v_full[sv]);
            }
        }
        if (!ok) {
            // give copies already in flight a bounded chance to land before the CTA's shared memory is released
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000) { }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t fmt = BF16 ? 1u : 0u;
            constexpr uint32_t idesc_s = make_idesc(fmt, 0, kRows, kKeys);   // Q (K-major) x K (K-major)
            constexpr uint32_t idesc_o = make_idesc(fmt, 1, kRows, kD);      // P (TMEM)    x V (MN-major)
            // matrix descriptors of Q tile 0 and of slot 0 of each ring, built once
            const uint64_t q_desc0 = smem_desc(smem_u32(q_tiles), 16, 1024);
            const uint64_t k_desc0 = smem_desc(smem_u32(k_ring), 16, 1024);
            const uint64_t v_desc0 = smem_desc(smem_u32(v_ring), kSlabBytes, 1024);
            bool ok = true;
            int kt_base = 0;                          // K/V tiles of the units before this one
            int p_cnt[2] = {0, 0};                    // completions of p_ready[t] consumed so far
            int f_cnt[2] = {0, 0};                    // completions of o_free[t] consumed so far
            bool o_busy[2] = {false, false};          // O_t holds a finished unit that its warpgroup may still be reading
            for (int un = 0; ok; ++un) {
                const int slot = un & 1;
                ok = mbar_wait(&bars->unit_full[slot], (un >> 1) & 1, bars, status);
                if (!ok) break;
                const int unit = bars->unit_slot[slot];
                mbar_arrive(&bars->unit_empty[slot]);
                if (unit < 0) break;
                const Unit u = decode_unit(a, items, unit);
                ok = mbar_wait(&bars->q_full, un & 1, bars, status);
                if (!ok) break;
                // the two kinds of unit get their own copy of the issue loop: every instruction of this thread counts
                auto run_unit = [&](auto split_tag) {
                    constexpr bool SPLIT = decltype(split_tag)::value;
                    int k_ready = -1, v_ready = -1;       // last K / V tile of this unit known to have landed
                    // S_t(s) = Q K(j)^T into TMEM columns [128 t, 128 t + 128), j = the key tile of step s of chain / tile t
                    auto issue_s = [&](int qt, int sidx) {
                        const int j = SPLIT ? 2 * sidx + qt : sidx;
                        const int kt = kt_base + j, st = kt % kStagesK;
                        if (k_ready < j) {
                            ok = mbar_wait(&bars->k_full[st], (kt / kStagesK) & 1, bars, status);
                            k_ready = j;
                            if (!ok) return;
                        }
                        // descriptors of the first 16 columns; the others differ in the address field only
                        const uint64_t qd = q_desc0 + (uint64_t)((SPLIT ? 0 : qt) * (kTileBytes >> 4));
                        const uint64_t kd = k_desc0 + (uint64_t)(st * (kTileBytes >> 4));
                        tc_fence_after();
#pragma unroll
                        for (int ks = 0; ks < kD / 16; ++ks) {
                            const uint32_t off = ((ks >> 2) * kSlabBytes + (ks & 3) * 32) >> 4;   // 16 columns = 32 bytes inside a slab row
                            mma_ss(tmem + qt * 128, qd + off, kd + off, idesc_s, ks > 0);
                        }
                        tc_commit(&bars->s_full[qt]);
                        if (SPLIT || qt == u.nq - 1) {
                            tc_commit(&bars->k_empty[st]);                       // the last reader of this K tile
                            if (j == u.n_all - 1) tc_commit(&bars->q_empty);     // and the unit's last read of the Q tiles
                        }
                    };
                    // O_t (+)= P_t V(j); P sits in the columns S_t was computed in
                    auto issue_pv = [&](int qt, int sidx) {
                        const int j = SPLIT ? 2 * sidx + qt : sidx;
                        const int kt = kt_base + j, st = kt % kStagesV;
                        if (v_ready < j) {
                            ok = mbar_wait(&bars->v_full[st], (kt / kStagesV) & 1, bars, status);
                            v_ready = j;
                            if (!ok) return;
                        }
                        if (sidx == 0 && o_busy[qt]) {
                            // the accumulator still holds the previous unit: wait until its rows are in registers
                            ok = mbar_wait(&bars->o_free[qt], f_cnt[qt] & 1, bars, status);
                            ++f_cnt[qt];
                            o_busy[qt] = false;
                            if (!ok) return;
                        }
                        ok = mbar_wait(&bars->p_ready[qt], p_cnt[qt] & 1, bars, status);
                        ++p_cnt[qt];
                        if (!ok) return;
                        tc_fence_after();
                        const uint64_t vd = v_desc0 + (uint64_t)(st * (kTileBytes >> 4));
                        const uint32_t tp = tmem + qt * 128, to = tmem + 256 + qt * 128;
                        HAT_CHECK((to & 0xffffu) + 128 <= 512 && (tp & 0xffffu) + 128 <= 256, status);
#pragma unroll
                        for (int ks = 0; ks < kKeys / 16; ++ks) {
                            // 16 keys = 2048 bytes of every 64-column slab; slabs 16 KiB apart (leading), 8-key groups 1 KiB apart
                            const uint64_t vdesc = vd + (uint64_t)((ks * 2048) >> 4);
                            mma_ts(to, tp + ks * 8, vdesc, idesc_o, (sidx > 0) || (ks > 0));
                            if constexpr (BF16) mma_ts(to, tp + 64 + ks * 8, vdesc, idesc_o, true);
                        }
                        tc_commit(&bars->o_done[qt]);
                        if (SPLIT || qt == u.nq - 1) tc_commit(&bars->v_empty[st]);
                    };
                    if (u.n_t0 > 0) issue_s(0, 0);
                    if (ok && u.n_t1 > 0) issue_s(1, 0);
                    for (int sidx = 0; sidx < max(u.n_t0, u.n_t1) && ok; ++sidx) {
                        // tile 0's P V, then at once its next S: the tensor pipe works on them while tile 1's softmax runs
                        if (sidx < u.n_t0) {
                            issue_pv(0, sidx);
                            if (ok && sidx + 1 < u.n_t0) issue_s(0, sidx + 1);
                        }
                        if (ok && sidx < u.n_t1) {
                            issue_pv(1, sidx);
                            if (ok && sidx + 1 < u.n_t1) issue_s(1, sidx + 1);
                        }
                    }
                };
                if (u.split) run_unit(std::true_type{}); else run_unit(std::false_type{});
                // a unit in which a tile had no keys leaves that tile's earlier hand-over pending
                if (u.n_t0 > 0) o_busy[0] = true;
                if (u.n_t1 > 0) o_busy[1] = true;
                kt_base += u.n_all;
            }
            if (!ok) {
                // gave up: let the MMAs already issued finish (bounded) before TMEM is released
                tc_commit(&bars->drain);
                const long long t0 = clock64();
                while (!mbar_try(&bars->drain, 0) && clock64() - t0 < bars->wait_cycles) { }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax / correction / output
        const int qt = (warp - 2) >> 2;                     // query tile of this warpgroup
        const int quarter = warp & 3;                       // TMEM lanes this warp may touch
        const int t = quarter * 32 + lane;                  // query row inside the tile = TMEM lane
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t tm_s = tmem + qt * 128 + lane_sel, tm_o = tmem + 256 + qt * 128 + lane_sel;
        const int wg_tid = (int)threadIdx.x - 64 - qt * 128;
        const float sc = a.scale_log2;
        // rows are 512 bytes apart at least, so a 32-byte aligned base keeps every 32-byte store aligned
        const bool wide_stores = ((reinterpret_cast<uintptr_t>(a.out) | reinterpret_cast<uintptr_t>(a.part_out)) & 31) == 0;
        int kt_base = 0;                                    // K/V tiles of the units before this one
        int s_cnt = 0, o_cnt = 0, x_cnt = 0;                // completions of s_full[qt] / o_done[qt] / x_ready consumed so far
        bool ok = true;
        for (int un = 0; ok; ++un) {
            const int slot = un & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(&bars->unit_full[slot], (un >> 1) & 1, bars, status));
            if (!ok) break;
            const int unit = bars->unit_slot[slot];
            __syncwarp();                                    // every lane has read the slot
            if (lane == 0) mbar_arrive(&bars->unit_empty[slot]);
            if (unit < 0) break;
            const Unit u = decode_unit(a, items, unit);
            if (qt < u.nq || u.split) {
                const int n_mine = u.n_t(qt);
                const int i_row = u.row0 + (u.split ? 0 : qt * kRows) + t;   // row inside the chunk
                const int last_key = min(u.P + i_row, u.kv_end - 1);
                float m_used = -INFINITY, l = 0.f;           // in units of scale_log2
                for (int sidx = 0; sidx < n_mine; ++sidx) {
                    const int j = u.tile_of(qt, sidx);       // key tile of this step
                    const int kb = u.kv_begin + j * kKeys;
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->s_full[qt], s_cnt & 1, bars, status));
                    ++s_cnt;
                    if (!ok) break;
                    tc_fence_after();
                    float s[kKeys];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(tm_s + c * 32, reinterpret_cast<uint32_t*>(s) + c * 32);
                    tmem_ld_wait();

                    // raw maximum (the scale is positive, so it commutes with max); four independent chains
                    const int lim = last_key - kb;          // keys 0..lim of this tile are visible to this row
                    if (lim < kKeys - 1) {
#pragma unroll
                        for (int k = 0; k < kKeys; ++k) s[k] = (k <= lim) ? s[k] : -INFINITY;
                    }
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int k = 0; k < kKeys; k += 8) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) mx4[v] = fmaxf(mx4[v], fmaxf(s[k + 2 * v], s[k + 2 * v + 1]));
                    }
                    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;
                    // move the reference maximum only when it grew by more than the threshold
                    float alpha = 1.f;
                    bool rescale = false;
                    if (mx > m_used + kRescaleThreshold) {
                        alpha = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - mx);
                        rescale = (m_used != -INFINITY);
                        m_used = mx;
                    }
                    const float neg_ref = (m_used == -INFINITY) ? 0.f : -m_used;
                    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t p[16];
                        uint32_t pl[16];
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            const float e0 = fast_exp2(fmaf(s[c * 32 + k], sc, neg_ref));
                            const float e1 = fast_exp2(fmaf(s[c * 32 + k + 1], sc, neg_ref));
                            sum4[(k >> 1) & 3] += e0 + e1;
                            p[k / 2] = pack2<BF16>(e0, e1);
                            if constexpr (BF16) {
                                const float r0 = e0 - __uint_as_float(p[k / 2] << 16);
                                const float r1 = e1 - __uint_as_float(p[k / 2] & 0xffff0000u);
                                pl[k / 2] = pack2<BF16>(r0, r1);
                            }
                        }
                        tmem_st16(tm_s + c * 16, p);
                        if constexpr (BF16) tmem_st16(tm_s + 64 + c * 16, pl);
                    }
                    l = l * alpha + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));

                    // O may only be rescaled once the previous P V product has finished; waiting here every tile (it
                    // has long completed by now) also keeps this thread's count of the barrier's phases exact
                    if (sidx > 0) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&bars->o_done[qt], o_cnt & 1, bars, status));
                        ++o_cnt;
                        if (!ok) break;
                        tc_fence_after();
                    }
                    if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
                        for (int c = 0; c < kD / 32; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tm_o + c * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                            tmem_st32(tm_o + c * 32, o);
                        }
                    }
                    tmem_st_wait();
                    // a range that ends inside this tile: V rows past the range were not loaded (or hold stale
                    // slots); zero them so that 0 * garbage cannot produce NaN (both warpgroups may do it: same zeros)
                    if (kb + kKeys > u.kv_end) {
                        const int kt = kt_base + j;
                        ok = __all_sync(0xffffffffu, mbar_wait(&bars->v_full[kt % kStagesV], (kt / kStagesV) & 1, bars, status));
                        if (!ok) break;
                        unsigned char* vt = v_ring + (kt % kStagesV) * kTileBytes;
                        const int first = u.kv_end - kb;
                        constexpr int kVecs = kD / 8;                              // 16-byte vectors per row
                        for (int idx = wg_tid; idx < (kKeys - first) * kVecs; idx += 128) {
                            const int row = first + idx / kVecs, part = idx % kVecs;
                            *reinterpret_cast<uint4*>(vt + (part >> 3) * kSlabBytes + row * 128 + (part & 7) * 16) = make_uint4(0, 0, 0, 0);
                        }
                        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    }
                    // one arrival per warp: every lane's P is in TMEM (wait::st) and fenced before the warp meets
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->p_ready[qt]);
                }
                if (!ok) break;
                // ---- output of the unit: pull O into registers, hand the accumulator back, then store
                float o[kD];
                if (n_mine > 0) {                            // uniform over the warpgroup
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->o_done[qt], o_cnt & 1, bars, status));
                    ++o_cnt;
                    if (!ok) break;
                    tc_fence_after();
                }
                if (u.split && qt == 1) {
                    // second chain of a split unit: its accumulator is complete; publish the row's reference maximum
                    // and sum, the first chain's warpgroup reads the accumulator itself (same TMEM lanes) and stores
                    if (n_mine > 0) {
                        bars->xchg[t] = make_float2(m_used, l);
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars->x_ready);
                    }
                } else {
                    if (n_mine > 0) {
#pragma unroll
                        for (int c = 0; c < kD / 32; ++c) tmem_ld32(tm_o + c * 32, reinterpret_cast<uint32_t*>(o) + c * 32);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int k = 0; k < kD; ++k) o[k] = 0.f;
                    }
                    if (u.split && u.n_t1 > 0) {
                        // merge the second chain (disjoint keys): weights 2^(m_t - m), sums and accumulators add up
                        ok = __all_sync(0xffffffffu, mbar_wait(&bars->x_ready, x_cnt & 1, bars, status));
                        ++x_cnt;
                        if (!ok) break;
                        tc_fence_after();
                        const float2 other = bars->xchg[t];
                        const float m_new = fmaxf(m_used, other.x);
                        const float w0 = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_new);
                        const float w1 = (other.x == -INFINITY) ? 0.f : fast_exp2(other.x - m_new);
                        l = l * w0 + other.y * w1;
                        m_used = m_new;
#pragma unroll
                        for (int c = 0; c < kD / 16; ++c) {
                            uint32_t o1[16];
                            tmem_ld16(tm_o + 128 + c * 16, o1);      // the second chain's accumulator: next 128 columns
                            tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 16; ++k) o[c * 16 + k] = o[c * 16 + k] * w0 + __uint_as_float(o1[k]) * w1;
                        }
                    }
                    if (n_mine > 0 || (u.split && u.n_t1 > 0)) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (n_mine > 0) mbar_arrive(&bars->o_free[qt]);
                            if (u.split && u.n_t1 > 0) mbar_arrive(&bars->o_free[1]);
                        }
                    }
                    if (i_row < u.C) {
                        const float inv = l > 0.f ? 1.f / l : 0.f;
                        float* obase; float* lbase; int64_t orow;
                        if (u.part < 0) { obase = a.out; lbase = a.lse; orow = u.row_base + i_row; }
                        else { obase = a.part_out; lbase = a.part_lse; orow = u.part + (i_row - u.row0); }
                        HAT_CHECK(orow >= 0 && orow < (u.part < 0 ? (int64_t)a.plan.total_rows : a.part_rows), status);
                        float* dst = obase + (orow * H + u.h) * kD;
                        if (u.part < 0 && a.out16 != nullptr) {
                            // final rows in the 16-bit output type: 256 bytes per row, eight 32-byte stores
                            uint16_t* dst16 = static_cast<uint16_t*>(a.out16) + (orow * H + u.h) * kD;
                            const bool wide16 = (reinterpret_cast<uintptr_t>(a.out16) & 31) == 0;
#pragma unroll
                            for (int k = 0; k < kD; k += 16) {
                                uint32_t w[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) w[e] = pack_out16(o[k + 2 * e] * inv, o[k + 2 * e + 1] * inv, a.out16_bf16);
                                if (wide16) {
                                    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n"
                                                 ::"l"(dst16 + k), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
                                } else {
                                    *reinterpret_cast<uint4*>(dst16 + k) = make_uint4(w[0], w[1], w[2], w[3]);
                                    *reinterpret_cast<uint4*>(dst16 + k + 8) = make_uint4(w[4], w[5], w[6], w[7]);
                                }
                            }
                        } else if (wide_stores) {
                            // a thread stores its whole row; 32-byte stores fill a sector each (half as many sector writes
                            // as 16-byte ones, and the sector rate is what bounds this part)
#pragma unroll
                            for (int k = 0; k < kD; k += 8)
                                st_global_v8(dst + k, o[k] * inv, o[k + 1] * inv, o[k + 2] * inv, o[k + 3] * inv, o[k + 4] * inv,
                                             o[k + 5] * inv, o[k + 6] * inv, o[k + 7] * inv);
                        } else {
#pragma unroll
                            for (int k = 0; k < kD; k += 4)
                                *reinterpret_cast<float4*>(dst + k) = make_float4(o[k] * inv, o[k + 1] * inv, o[k + 2] * inv, o[k + 3] * inv);
                        }
                        lbase[orow * H + u.h] = l > 0.f ? (m_used + log2f(l)) * 0.6931471805599453f : -INFINITY;
                    }
                }
            }
            kt_base += u.n_all;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
    }
    // The last CTA to get here (none draws units any more) leaves the unit counter at zero for the next call, which
    // then needs no memset in front of it.  work_counter[1] counts the CTAs that have finished.
    if (a.tail_reset && threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(work_counter + 1, 1) == (int)gridDim.x - 1) {
            work_counter[0] = 0;
            work_counter[1] = 0;
            __threadfence();
        }
    }
}

// ---------------------------------------------------------------------------------------------- host side
}  // namespace

bool tc5_layout_supported(int dtype, int head_dim, int num_pages, int H, int64_t stride_page, int64_t stride_token,
                          int64_t stride_head) {
    if ((head_dim != 64 && head_dim != 128) || num_pages <= 0) return false;
    CUtensorMap m;
    // the encoder checks alignment and ranges only; any 16-byte aligned address will do for the probe
    return tma_encode_pool_map(&m, dtype == HAT_DTYPE_BF16, reinterpret_cast<const void*>(uintptr_t(1) << 30), head_dim,
                               num_pages, H, stride_page, stride_token, stride_head);
}

cudaError_t launch_attn_tc5(const hat_plan* plan, const AttnArgs& args, cudaStream_t stream, int grid_limit,
                            bool reset_counter, int first_unit, int num_units, int counter_word) {
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    const CUtensorMap *mk = nullptr, *mv = nullptr;
    const CUtensorMap* mq = plan_q_map(plan, args.q);
    if (!mq || !plan_pool_maps(plan, args.cache, &mk, &mv)) return cudaErrorInvalidValue;
    // one CTA per SM draws units from a counter that is zero at this point: the previous call's last CTA cleared it
    // (reset_counter); a grid that joins another one on the same counter leaves it alone
    const int total_units = num_units >= 0 ? num_units : (int)plan->tile_units.size() - first_unit;
    if (total_units <= 0) return cudaSuccess;
    int32_t* counter = plan->dev.status + counter_word;
    AttnArgs a2 = args;
    a2.plan.tile_units = plan->dev.tile_units + first_unit;
    a2.tail_reset = reset_counter ? 1 : 0;
    int ctas = std::min(total_units, plan->num_sms);
    if (grid_limit > 0) ctas = std::min(ctas, grid_limit);
    const dim3 grid((unsigned)ctas);
    const bool d128 = plan->head_dim == 128;
    auto kern = d128 ? (bf16 ? attn_tc5_kernel<true, 128> : attn_tc5_kernel<false, 128>)
                     : (bf16 ? attn_tc5_kernel<true, 64> : attn_tc5_kernel<false, 64>);
    const uint32_t smem = d128 ? smem_bytes<128>() : smem_bytes<64>();
    cudaError_t e = smem_attr_once(reinterpret_cast<const void*>(kern), (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, smem, stream>>>(a2, plan->dev.prefill_items, total_units, counter, *mq, *mk, *mv);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hat
