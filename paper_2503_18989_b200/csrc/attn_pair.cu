// Prefill-chunk attention on tcgen05 / TMEM by pairs of CTAs (cta_group::2) with a ring of three score buffers.
//
// Persistent kernel launched as clusters of two CTAs, one cluster per pair of SMs.  A work unit = up to 256 query rows
// of one request x one head x one key range; CTA c of the pair owns rows [128 c, 128 c + 128) of it: its Q tile, its
// softmax warpgroups, its TMEM (score ring + accumulator) and its output rows.  The MMAs are issued by one thread of
// CTA 0 for both CTAs at once (M = 256): each CTA feeds HALF of every K tile (64 of the 128 keys) and HALF of every V
// tile (64 of the 128 columns) from its own shared memory, so a CTA loads, stores and re-reads half the K/V bytes per
// tile of a single-CTA kernel.  That is what lets one query tile per CTA keep three score tiles in flight within 512
// TMEM columns and still have the K/V rings cover the load latency.
//
// The key range is walked in tiles of 128 keys; the tiles of all units a pair processes form ONE sequence, numbered g,
// and every ring below is indexed by g, so the pipeline does not drain at a unit boundary.
//
// TMEM of each CTA (512 columns): score buffers S_b at columns [128 b, 128 b + 128), b = g % 3; accumulator O at
// [384, 512).  The softmax of tile g overwrites S_b with P (16-bit pairs in columns [0, 64) of the buffer; for bf16 the
// rounding remainder of P in [64, 128)), the A operand of the P V product straight from TMEM.
//
//   warp 0      CTA 0: draws units from a global counter (one ahead of the unit it loads) and publishes them to both
//               CTAs through four-slot queues.  Both CTAs: TMA producer of the own Q tile (two slots) and of the own
//               halves of the K tiles (ring); plain tile loads, completion on the CTA's own mbarriers
//   warp 11     TMA producer of the own halves of the V tiles (ring).  A warp of its own so that the two rings fill
//               independently and two warps feed the TMA unit (one 2 KiB box per page and column half is the largest
//               the paged layout allows, and the unit's rate of such boxes is what the rings have to hide)
//   warp 10     CTA 0: one thread issues S(g) = Q K(g)^T for every tile, up to three tiles ahead of the P V products
//   warp 1      CTA 0: one thread issues O (+)= P(g) V(g).  Two issuing threads because whatever a thread does between
//               two MMAs (a barrier poll above all) delays its next MMA: while one polls, the other's MMAs run.  MMAs of
//               different threads are unordered, so S(g+3), which lands in the buffer P(g) was read from, waits for the
//               commit of P V(g).  Commits are multicast to the barriers of both CTAs.
//               CTA 1: one thread forwards "my half has landed" of every Q and K load to CTA 0's barriers (the V halves
//               are checked by the softmax warpgroups before they hand P over).  Both CTAs: owns the TMEM allocation
//   warps 2-5   softmax warpgroup 0   (thread = query row = TMEM lane; the two warpgroups share the CTA's 128 rows)
//   warps 6-9   softmax warpgroup 1
//
// Both warpgroups of a CTA feed the same accumulator, so a row has ONE reference maximum.  It only moves when a tile's
// row maximum exceeds it by more than 2^8 (then O is rescaled in TMEM, after the previous P V has finished and before
// the tile's own is issued).  How a tile is shared depends on the type (measured, see the softmax role below):
//   fp16   the warpgroups take alternate tiles (even / odd g).  The reference passes from tile g to tile g+1 through
//          shared memory as soon as tile g's row maximum is known, i.e. before its exponentials: the only serial link
//          between consecutive tiles.  Each warpgroup keeps its own row sums; they are combined when the unit ends.
//   bf16   both warpgroups take every tile, 64 keys each: a row has two threads (the same lane of the two warps that
//          share a lane quarter).  They exchange the maxima of their halves through shared memory every tile and take
//          the same decisions from them; each keeps the row sum of its keys and rescales its half of O's columns.
// Either way each warpgroup stores one half of the output columns.
//
// Every wait is bounded; a wait that gives up sets the plan's status word and the abort flags of both CTAs, which every
// other wait observes; both CTAs then still meet at the cluster barrier, free their TMEM and exit normally.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cstdlib>

#include "hat_internal.h"
#include "tma_desc.h"
#include "tc5_ptx.cuh"

namespace hat {
namespace {
using namespace tc5;

constexpr int kRows = 128;      // query rows per CTA (the MMA spans both CTAs: M = 256)
constexpr int kKeys = 128;      // keys per tile (MMA N of S, K extent of P V)
constexpr int kD = 128;         // head_dim
constexpr int kSBuf = 3;        // score buffers in TMEM
constexpr int kStagesK = 4;     // ring slots for this CTA's halves of the K tiles
constexpr int kStagesV = 5;     // ring slots for this CTA's halves of the V tiles
constexpr int kUnitSlots = 4;   // queue of published units
constexpr uint32_t kTileBytes = kRows * kD * 2;          // 32 KiB: the Q tile of one CTA
constexpr uint32_t kSlabBytes = kRows * 64 * 2;          // 16 KiB: 64 columns of 128 rows
constexpr uint32_t kHalfBytes = kKeys * kD;              // 16 KiB: 64 keys x 128 columns of K, or 128 keys x 64 columns of V
constexpr uint32_t kKSlabBytes = 64 * 64 * 2;            // 8 KiB: 64 columns of the 64 keys of a K half
constexpr uint32_t kPageBoxBytes = 16 * 64 * 2;          // 2 KiB: one TMA box (16 tokens x 64 columns)
constexpr uint32_t kColO = 384;                          // first TMEM column of the accumulator
constexpr float kRescaleThreshold = 8.0f;                // log2 units

struct __align__(8) Barriers {
    // Barriers with the same name exist in both CTAs (same offsets).  "pair": the MMA thread's commit arrives on it in
    // both CTAs.  "CTA 0": only CTA 0's copy is used, CTA 1 arrives on it remotely.
    uint64_t q_full[2];                                     // own loads; CTA 0's copy also counts CTA 1's forwarded arrival
    uint64_t q_empty[2];                                    // pair
    uint64_t k_full[kStagesK];                              // as q_full
    uint64_t v_full[kStagesV];                              // own loads only: the tile's warpgroup checks it before it arrives on p_ready
    uint64_t k_empty[kStagesK], v_empty[kStagesV];          // pair (a commit costs the issuing thread nothing; a poll does)
    uint64_t s_full[kSBuf], pv_done[kSBuf];                 // pair
    uint64_t p_ready[kSBuf];                                // CTA 0: the softmax warps that work on the tile, of both CTAs
    uint64_t o_free;                                        // CTA 0: all sixteen softmax warps hold their part of O in registers
    uint64_t unit_full[kUnitSlots];                         // own queue, filled by CTA 0's producer
    uint64_t unit_empty[kUnitSlots];                        // CTA 0: every reader of the queue in both CTAs
    uint64_t pair_bar[4];                                   // bf16, own: the two warps that share lane quarter q (one of each warpgroup) meet here
    uint64_t m_ready[2][4];                                 // fp16, own: warpgroup w, lane quarter q published its tile's reference maximum
    uint64_t fin_ready[2][4];                               // fp16, own: the same for the row-sum hand-over at the end of a unit
    uint64_t drain, drain2;
    long long wait_cycles;                                  // bound of every wait below
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile int unit_slot[kUnitSlots];                     // unit index, or -1 when the work has run out
    float mx_x[2][2][kRows];                                // bf16, [tile parity][warpgroup][row]: maximum over the warpgroup's half of the tile's keys
    float lsum2[2][2][kRows];                               // bf16, [unit parity][warpgroup][row]: row sum over the warpgroup's keys of the unit
    float mref[kRows];                                      // fp16, per row: the reference maximum the latest tile left behind
    float lsum[2][kRows];                                   // fp16, [unit parity][row]: row-sum hand-over at the end of a unit
};
constexpr uint32_t kSmemBytes = 1024 /*alignment slack*/ + kTileBytes * 2 + kHalfBytes * (kStagesK + kStagesV) + sizeof(Barriers);
static_assert(kSmemBytes <= 227 * 1024, "shared memory of one CTA");
constexpr int kThreads = 384;   // K producer, P V issuer / forwarder, two softmax warpgroups, S issuer, V producer
constexpr int kQueueReaders0 = 2 + 8 + 1;    // CTA 0: the two MMA threads, softmax warps, V producer (the K producer drew the unit itself)
constexpr int kQueueReaders1 = 2 + 1 + 8;    // CTA 1: both producer warps, forwarding thread, softmax warps

#ifdef HAT_PHASE_TIMERS
// Diagnostic build only: cycles spent per phase, summed over all CTAs (clock64 stamps around the phases).
__device__ unsigned long long g_phase[80];
#define PH_T0(v) long long v = clock64()
#define PH_ADD(slot, v) do { const long long now_ = clock64(); ph[slot] += now_ - v; v = now_; } while (0)
#define PH_DECL(n) long long ph[n] = {0}
#define PH_FLUSH(base, n) do { for (int i_ = 0; i_ < n; ++i_) atomicAdd(&g_phase[base + i_], (unsigned long long)ph[i_]); } while (0)
#else
#define PH_T0(v)
#define PH_ADD(slot, v)
#define PH_DECL(n)
#define PH_FLUSH(base, n)
#endif

struct Ctx {
    Barriers* bars;
    int32_t* status;
    uint32_t peer_abort;     // shared::cluster address of the other CTA's abort flag
};

// Bounded wait.  Returns false if the wait gave up or another role, here or in the other CTA, already did.
// CLUSTER: acquire at cluster scope (needed where the arrival announces plain stores made by the other CTA).
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const Ctx& cx) {
    auto poll = [&]() { return CLUSTER ? mbar_try_cluster(bar, parity) : mbar_try(bar, parity); };
    if (poll()) return true;
    const long long t0 = clock64();
    while (!poll()) {
        if (cx.bars->abort_flag) return false;
        if (clock64() - t0 > cx.bars->wait_cycles) {
            cx.bars->abort_flag = 1;
            st_cluster_b32(cx.peer_abort, 1u);
            atomicOr(cx.status, 1);
            return false;
        }
    }
    return true;
}

// What every role needs to know about a unit; all of them decode it the same way.
struct Unit {
    int h, hk, r, P, C, row_base, row0, kv_begin, kv_end, part;   // h: query head, hk = h / G: the K/V head it reads
    int n;                                                        // key tiles of the range (at least 1)
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
    u.n = max(1, (u.kv_end - u.kv_begin + kKeys - 1) / kKeys);
    return u;
}

template <bool BF16>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attn_pair_kernel(AttnArgs a, const WorkItem* __restrict__ items, int total_units, int32_t* work_counter,
                 const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment: the swizzle pattern and the matrix descriptors assume it.  Both CTAs of a pair must end up
    // with the same offsets (the MMA applies one descriptor to both); the dynamic shared memory of a kernel starts at
    // the same address in every CTA, so the same rounding gives the same layout.
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* q_tiles = smem;                               // 2 x 32 KiB
    unsigned char* k_ring = smem + 2 * kTileBytes;               // kStagesK x 16 KiB
    unsigned char* v_ring = k_ring + kStagesK * kHalfBytes;      // kStagesV x 16 KiB
    Barriers* bars = reinterpret_cast<Barriers*>(v_ring + kStagesV * kHalfBytes);

    const int H = a.plan.num_heads;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                     // 0: the CTA whose thread issues the MMAs
    Ctx cx;
    cx.bars = bars;
    cx.status = a.plan.status;
    cx.peer_abort = map_to_cta(smem_u32(const_cast<int*>(&bars->abort_flag)), rank ^ 1u);
    // shared::cluster address of CTA 0's copy of a barrier
    auto lead = [&](uint64_t* bar) -> uint32_t { return map_to_cta(smem_u32(bar), 0u); };

    if (threadIdx.x == 0) {
        const uint32_t fwd = rank == 0 ? 2u : 1u;                // CTA 0's "full" barriers also take CTA 1's forwarded arrival
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->q_full[s], fwd); mbar_init(&bars->q_empty[s], 1); }
        for (int s = 0; s < kStagesK; ++s) { mbar_init(&bars->k_full[s], fwd); mbar_init(&bars->k_empty[s], 1); }
        for (int s = 0; s < kStagesV; ++s) { mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], 1); }
        for (int s = 0; s < kSBuf; ++s) {
            mbar_init(&bars->s_full[s], 1);
            mbar_init(&bars->p_ready[s], BF16 ? 16 : 8);          // one arrival per softmax warp that works on the tile, both CTAs
            mbar_init(&bars->pv_done[s], 1);
        }
        mbar_init(&bars->o_free, 16);
        for (int s = 0; s < kUnitSlots; ++s) {
            mbar_init(&bars->unit_full[s], 1);
            mbar_init(&bars->unit_empty[s], kQueueReaders0 + kQueueReaders1);
        }
        for (int q = 0; q < 4; ++q) mbar_init(&bars->pair_bar[q], 2);
        for (int w = 0; w < 2; ++w)
            for (int q = 0; q < 4; ++q) { mbar_init(&bars->m_ready[w][q], 1); mbar_init(&bars->fin_ready[w][q], 1); }
        mbar_init(&bars->drain, 1);
        mbar_init(&bars->drain2, 1);
        bars->abort_flag = 0;
        bars->wait_cycles = a.wait_cycles;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 1) {
        // the same warp of both CTAs allocates (and later frees) the pair's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    // the other CTA's barriers must be initialised before anything arrives on them
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    // A consumer's read of the unit queue: the unit published as number `un` (-1: none left, -2: gave up).
    auto read_unit = [&](int un, bool whole_warp) -> int {
        const int slot = un % kUnitSlots;
        bool ok = mbar_wait<true>(&bars->unit_full[slot], (un / kUnitSlots) & 1, cx);   // the slot was stored by CTA 0
        if (whole_warp) ok = __all_sync(0xffffffffu, ok);
        if (!ok) return -2;
        const int unit = bars->unit_slot[slot];
        if (whole_warp) __syncwarp();                            // every lane has read the slot
        if (!whole_warp || lane == 0) mbar_arrive_remote(lead(&bars->unit_empty[slot]));
        return unit;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ unit fetch (CTA 0) + TMA producer (both)
        int g = 0;                                               // K/V tiles issued so far, over all units
        bool ok = true;
        PH_DECL(8);
        PH_T0(tq0);
        // CTA 0: draw a unit and publish it in slot un % 4 of both CTAs' queues (all lanes return it); the slot is free
        // once every reader in both CTAs has read the unit published four draws earlier
        auto publish = [&](int un) -> int {
            const int slot = un % kUnitSlots;
            if (un >= kUnitSlots) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->unit_empty[slot], ((un / kUnitSlots) - 1) & 1, cx));
                if (!ok) return -1;
            }
            int unit = 0;
            if (lane == 0) {
                unit = atomicAdd(work_counter, 1);
                if (unit >= total_units) unit = -1;
                bars->unit_slot[slot] = unit;
                mbar_arrive(&bars->unit_full[slot]);             // release: the slot is written before the arrival
                st_cluster_b32(map_to_cta(smem_u32(const_cast<int*>(&bars->unit_slot[slot])), 1u), (uint32_t)unit);
                mbar_arrive_cluster(map_to_cta(smem_u32(&bars->unit_full[slot]), 1u));
            }
            return __shfl_sync(0xffffffffu, unit, 0);
        };
        int next_unit = rank == 0 ? publish(0) : 0;
        for (int un = 0; ok; ++un) {
            int unit;
            if (rank == 0) {
                unit = next_unit;
                if (unit < 0) break;
                // the unit after this one is published before this one's tiles are requested, so that the MMA thread can
                // run its score tiles ahead across the unit boundary
                next_unit = publish(un + 1);
                if (!ok) break;
            } else {
                unit = read_unit(un, true);
                if (unit == -2) { ok = false; break; }
                if (unit < 0) break;
            }
            const Unit u = decode_unit(a, items, unit);
            const int32_t* __restrict__ table = a.plan.block_table + (int64_t)u.r * a.plan.max_pages + u.kv_begin / kPageSize;
            const int qs = un & 1;
            PH_ADD(0, tq0);
            if (un >= 2) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->q_empty[qs], ((un >> 1) - 1) & 1, cx));
                if (!ok) break;
            }
            if (lane == 0) mbar_expect_tx(&bars->q_full[qs], kTileBytes);
            __syncwarp();
            if (lane < 2)      // lane = column half; this CTA's 128 rows
                tma_load_3d(smem_u32(q_tiles) + qs * kTileBytes + lane * kSlabBytes, &map_q, lane * 64, u.h,
                            u.row_base + u.row0 + (int)rank * kRows, &bars->q_full[qs]);
            PH_ADD(1, tq0);
            // K: this CTA's 64 keys = pages 4 rank .. 4 rank + 3 of every tile, both column halves: lane = 2 * page + half.
            // The page id of the NEXT tile is fetched while this tile's boxes are issued.
            const int total_pages = (u.kv_end - u.kv_begin + kPageSize - 1) / kPageSize;
            const int kpg = 4 * (int)rank + (lane >> 1), khalf = lane & 1;
            HAT_CHECK(u.kv_begin / kPageSize + total_pages <= a.plan.max_pages, cx.status);
            int page = (lane < 8 && kpg < total_pages) ? HAT_IN_RANGE(__ldg(table + kpg), a.plan.num_pages, cx.status) : 0;
            for (int j = 0; j < u.n; ++j, ++g) {
                const int sk = g % kStagesK;
                const int npages = min(8, total_pages - 8 * j);                                   // pages of this tile: 1..8
                const int nk = max(0, min(4, npages - 4 * (int)rank));                            // K pages this CTA loads
                const int next_pg = 8 * (j + 1) + kpg;
                const int page_next = (lane < 8 && next_pg < total_pages) ? HAT_IN_RANGE(__ldg(table + next_pg), a.plan.num_pages, cx.status) : 0;
                HAT_CHECK(sk < kStagesK, cx.status);
                PH_ADD(2, tq0);
                if (g >= kStagesK) ok = mbar_wait(&bars->k_empty[sk], ((g / kStagesK) & 1) ^ 1, cx);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                PH_ADD(3, tq0);
                if (lane == 0) mbar_expect_tx(&bars->k_full[sk], nk * 2 * kPageBoxBytes);
                __syncwarp();
                if (lane < 8 && kpg < npages)
                    tma_load_4d(smem_u32(k_ring) + sk * kHalfBytes + khalf * kKSlabBytes + (lane >> 1) * kPageBoxBytes, &map_k,
                                khalf * 64, 0, u.hk, page, &bars->k_full[sk]);
                PH_ADD(4, tq0);
#ifdef HAT_PHASE_TIMERS
                ph[7] += 1;
#endif
                page = page_next;
            }
        }
#ifdef HAT_PHASE_TIMERS
        if (lane == 0) PH_FLUSH(48 + 8 * (int)rank, 8);
#endif
        if (!ok) {
            // give copies already in flight a bounded chance to land before the CTA's shared memory is released
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000) { }
        }
    } else if (warp == 11) {
        // ------------------------------------------------------------------ TMA producer of the V halves (both CTAs)
        // A warp of its own: the K and the V ring then fill independently (one warp doing both waits for a V slot
        // before it may request the next K tile), and two warps feed the TMA unit.
        // All 8 pages of every tile, this CTA's column half: lane = page.
        int g = 0;
        bool ok = true;
        for (int un = 0; ok; ++un) {
            const int unit = read_unit(un, true);
            if (unit == -2) { ok = false; break; }
            if (unit < 0) break;
            const Unit u = decode_unit(a, items, unit);
            const int32_t* __restrict__ table = a.plan.block_table + (int64_t)u.r * a.plan.max_pages + u.kv_begin / kPageSize;
            const int total_pages = (u.kv_end - u.kv_begin + kPageSize - 1) / kPageSize;
            HAT_CHECK(u.kv_begin / kPageSize + total_pages <= a.plan.max_pages, cx.status);
            int page = (lane < 8 && lane < total_pages) ? HAT_IN_RANGE(__ldg(table + lane), a.plan.num_pages, cx.status) : 0;
            for (int j = 0; j < u.n; ++j, ++g) {
                const int sv = g % kStagesV;
                const int npages = min(8, total_pages - 8 * j);
                const int next_pg = 8 * (j + 1) + lane;
                const int page_next = (lane < 8 && next_pg < total_pages) ? HAT_IN_RANGE(__ldg(table + next_pg), a.plan.num_pages, cx.status) : 0;
                HAT_CHECK(sv < kStagesV, cx.status);
                if (g >= kStagesV) ok = mbar_wait(&bars->v_empty[sv], ((g / kStagesV) & 1) ^ 1, cx);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (!(a.withhold && g == 0)) {               // self test: this V tile never arrives, its consumers give up
                    if (lane == 0) mbar_expect_tx(&bars->v_full[sv], npages * kPageBoxBytes);
                    __syncwarp();
                    if (lane < 8 && lane < npages)
                        tma_load_4d(smem_u32(v_ring) + sv * kHalfBytes + lane * kPageBoxBytes, &map_v, (int)rank * 64, 0, u.hk, page,
                                    &bars->v_full[sv]);
                }
                page = page_next;
            }
        }
        if (!ok) {
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000) { }
        }
    } else if (warp == 1 && rank != 0) {
        // ------------------------------------------------------------------ CTA 1: forward "landed" to CTA 0's barriers
        if (lane == 0) {
            int g = 0;
            bool ok = true;
            PH_DECL(8);
            PH_T0(tf0);
            for (int un = 0; ok; ++un) {
                const int unit = read_unit(un, false);
                PH_ADD(0, tf0);
                if (unit < 0) break;
                const Unit u = decode_unit(a, items, unit);
                const int qs = un & 1;
                ok = mbar_wait(&bars->q_full[qs], (un >> 1) & 1, cx);
                if (!ok) break;
                mbar_arrive_remote(lead(&bars->q_full[qs]));
                PH_ADD(1, tf0);
                for (int j = 0; j < u.n && ok; ++j, ++g) {
                    const int sk = g % kStagesK;
                    ok = mbar_wait(&bars->k_full[sk], (g / kStagesK) & 1, cx);
                    if (!ok) break;
                    PH_ADD(2, tf0);
                    mbar_arrive_remote(lead(&bars->k_full[sk]));
                    PH_ADD(3, tf0);
#ifdef HAT_PHASE_TIMERS
                    ph[7] += 1;
#endif
                }
            }
            PH_FLUSH(64, 8);
        }
        __syncwarp();
    } else if (warp == 1 || warp == 10) {
        // ------------------------------------------------------------------ CTA 0: the two MMA issuers (one thread each)
        // Whatever an issuing thread does between two MMAs (a barrier poll above all) delays its next MMA by that much:
        // the tensor pipe does not run far ahead of the thread that feeds it.  So the S products and the P V products
        // are issued by two threads of different warps: while one polls, the other's MMAs keep the pipe busy.  MMAs of
        // different threads are not ordered against each other, so the one dependency between the two streams is made
        // explicit: S(g+3) overwrites the buffer P(g) is read from, and waits for pv_done of tile g.
        // Ring positions, parities, barrier addresses and descriptors are carried along and stepped (no divisions).
        if (lane == 0 && rank == 0) {
            constexpr uint32_t fmt = BF16 ? 1u : 0u;
            constexpr uint32_t idesc_s = make_idesc(fmt, 0, 2 * kRows, kKeys);   // Q (K-major) x K (K-major), M = 256 over the pair
            constexpr uint32_t idesc_o = make_idesc(fmt, 1, 2 * kRows, kD);      // P (TMEM)    x V (MN-major)
            bool ok = true;
            auto wait_addr = [&](uint32_t bar_addr, uint32_t parity) -> bool {
                return mbar_wait(reinterpret_cast<uint64_t*>(__cvta_shared_to_generic(bar_addr)), parity, cx);
            };
            auto commit_addr = [&](uint32_t bar_addr) {
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n"
                             ::"r"(bar_addr), "h"((uint16_t)3) : "memory");
            };
            PH_DECL(16);
            PH_T0(tl0);
            if (warp == 10) {
                // ---- S = Q K^T of every tile, up to three tiles ahead of the P V products
                const uint64_t q_desc0 = smem_desc(smem_u32(q_tiles), 16, 1024);
                const uint64_t k_desc0 = smem_desc(smem_u32(k_ring), 16, 1024);
                uint32_t s_col = tmem, s_bar = smem_u32(&bars->s_full[0]), pv_bar = smem_u32(&bars->pv_done[0]), pv_par = 0;
                int s_buf = 0, k_slot = 0;
                bool wrapped = false;                       // the buffer about to be written has been used before
                uint64_t kd = k_desc0;
                uint32_t k_bar = smem_u32(&bars->k_full[0]), k_par = 0, ke_bar = smem_u32(&bars->k_empty[0]);
                for (int un = 0; ok; ++un) {
                    const int slot = un % kUnitSlots;
                    ok = mbar_wait(&bars->unit_full[slot], (un / kUnitSlots) & 1, cx);
                    if (!ok) break;
                    const int unit = bars->unit_slot[slot];
                    mbar_arrive(&bars->unit_empty[slot]);
                    if (unit < 0) break;
                    const WorkItem it = items[__ldg(a.plan.tile_units + unit) & 0xffffu];
                    const int n = max(1, (it.kv_end - it.kv_begin + kKeys - 1) / kKeys);
                    const int qs = un & 1;
                    const uint64_t qd = q_desc0 + (uint64_t)(qs * (kTileBytes >> 4));
                    ok = mbar_wait(&bars->q_full[qs], (un >> 1) & 1, cx);
                    for (int j = 0; j < n && ok; ++j) {
                        PH_T0(ts0);
                        ok = wait_addr(k_bar, k_par);
                        if (!ok) break;
                        PH_ADD(0, ts0);
                        if (wrapped) {                      // the P V product that read this buffer three tiles ago
                            ok = wait_addr(pv_bar, pv_par);
                            if (!ok) break;
                        }
                        PH_ADD(1, ts0);
                        tc_fence_after();
#pragma unroll
                        for (int ks = 0; ks < kD / 16; ++ks) {
                            // 16 columns = 32 bytes inside a row of a 64-column slab; Q slabs are 16 KiB, K-half slabs 8 KiB apart
                            const uint32_t qoff = ((ks >> 2) * kSlabBytes + (ks & 3) * 32) >> 4;
                            const uint32_t koff = ((ks >> 2) * kKSlabBytes + (ks & 3) * 32) >> 4;
                            mma_ss_pair(s_col, qd + qoff, kd + koff, idesc_s, ks > 0);
                        }
                        commit_addr(s_bar);
                        commit_addr(ke_bar);
                        if (j == n - 1) commit_addr(smem_u32(&bars->q_empty[qs]));
                        if (++s_buf == kSBuf) {
                            s_buf = 0; s_col = tmem; s_bar = smem_u32(&bars->s_full[0]); pv_bar = smem_u32(&bars->pv_done[0]);
                            if (wrapped) pv_par ^= 1;
                            wrapped = true;
                        } else { s_col += 128; s_bar += 8; pv_bar += 8; }
                        if (++k_slot == kStagesK) { k_slot = 0; kd = k_desc0; k_bar = smem_u32(&bars->k_full[0]); ke_bar = smem_u32(&bars->k_empty[0]); k_par ^= 1; }
                        else { kd += kHalfBytes >> 4; k_bar += 8; ke_bar += 8; }
                        PH_ADD(2, ts0);
#ifdef HAT_PHASE_TIMERS
                        ph[6] += 1;
#endif
                    }
                }
                PH_ADD(5, tl0);
#ifdef HAT_PHASE_TIMERS
                ph[7] = 1;
#endif
                PH_FLUSH(0, 8);
            } else {
                // ---- O (+)= P V of every tile
                const uint64_t v_desc0 = smem_desc(smem_u32(v_ring), kSlabBytes, 1024);
                uint32_t p_col = tmem, p_bar = smem_u32(&bars->p_ready[0]), pv_bar = smem_u32(&bars->pv_done[0]), p_par = 0;
                int p_buf = 0, v_slot = 0;
                uint64_t vd = v_desc0;
                uint32_t ve_bar = smem_u32(&bars->v_empty[0]);
                const uint32_t to = tmem + kColO;
                for (int un = 0; ok; ++un) {
                    const int slot = un % kUnitSlots;
                    ok = mbar_wait(&bars->unit_full[slot], (un / kUnitSlots) & 1, cx);
                    if (!ok) break;
                    const int unit = bars->unit_slot[slot];
                    mbar_arrive(&bars->unit_empty[slot]);
                    if (unit < 0) break;
                    const WorkItem it = items[__ldg(a.plan.tile_units + unit) & 0xffffu];
                    const int n = max(1, (it.kv_end - it.kv_begin + kKeys - 1) / kKeys);
                    // the accumulators still hold the previous unit until its rows are in registers
                    if (un > 0) ok = mbar_wait(&bars->o_free, (un - 1) & 1, cx);
                    for (int j = 0; j < n && ok; ++j) {
                        PH_T0(tp0);
                        ok = wait_addr(p_bar, p_par);
                        if (!ok) break;
                        PH_ADD(0, tp0);
                        tc_fence_after();
#pragma unroll
                        for (int ks = 0; ks < kKeys / 16; ++ks) {
                            // 16 keys = 2048 bytes of this CTA's 64-column slab, 8-key groups 1 KiB apart
                            const uint64_t vdesc = vd + (uint64_t)((ks * 2048) >> 4);
                            if (ks == 0) mma_ts_pair(to, p_col, vdesc, idesc_o, j > 0);
                            else mma_ts_pair(to, p_col + ks * 8, vdesc, idesc_o, true);
                            if constexpr (BF16) mma_ts_pair(to, p_col + 64 + ks * 8, vdesc, idesc_o, true);
                        }
                        commit_addr(pv_bar);
                        commit_addr(ve_bar);
                        if (++p_buf == kSBuf) { p_buf = 0; p_col = tmem; p_bar = smem_u32(&bars->p_ready[0]); pv_bar = smem_u32(&bars->pv_done[0]); p_par ^= 1; }
                        else { p_col += 128; p_bar += 8; pv_bar += 8; }
                        if (++v_slot == kStagesV) { v_slot = 0; vd = v_desc0; ve_bar = smem_u32(&bars->v_empty[0]); }
                        else { vd += kHalfBytes >> 4; ve_bar += 8; }
                        PH_ADD(2, tp0);
#ifdef HAT_PHASE_TIMERS
                        ph[6] += 1;
#endif
                    }
                }
                PH_ADD(5, tl0);
#ifdef HAT_PHASE_TIMERS
                ph[7] = 1;
#endif
                PH_FLUSH(8, 8);
            }
            if (!ok) {
                // gave up: let the MMAs this thread issued finish (bounded) before TMEM is released
                uint64_t* dr = warp == 1 ? &bars->drain : &bars->drain2;
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n"
                             ::"r"(smem_u32(dr)) : "memory");
                const long long t0 = clock64();
                while (!mbar_try(dr, 0) && clock64() - t0 < bars->wait_cycles) { }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax / correction / output
        // Two ways of sharing a tile between the CTA's two softmax warpgroups (thread = query row = TMEM lane in both):
        // bf16: every tile is taken by both warpgroups, 64 keys each, so that a row has two threads; the halves' maxima are
        // exchanged through shared memory every tile.  The work per key is higher (P and its rounding remainder), and this
        // form measured 9 % faster (mixed 13B-shaped batch, tile kernel 0.556 -> 0.506 ms).
        // fp16: the warpgroups take alternate tiles, a whole row per thread; the exponentials of one overlap the waits of the
        // other.  Measured 8 % faster than the split form for fp16 (8 chunks of 512 rows, 40 heads: 930 vs 858 TFLOP/s).
        if constexpr (BF16) {
            const int w = (warp - 2) >> 2;                      // warpgroup: takes keys [64 w, 64 w + 64) of every tile
            const int quarter = warp & 3;                       // TMEM lanes this warp may touch
            const int t = quarter * 32 + lane;                  // query row inside this CTA's tile = TMEM lane
            const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
            const uint32_t tm_o = tmem + kColO + lane_sel;
            const int wg_tid = (int)threadIdx.x - 64 - w * 128;
            const float sc = a.scale_log2;
            const bool wide_stores = ((reinterpret_cast<uintptr_t>(a.out) | reinterpret_cast<uintptr_t>(a.part_out)) & 31) == 0;
            const uint32_t lead_o_free = lead(&bars->o_free), lead_p_ready = lead(&bars->p_ready[0]);
            int g0 = 0;                                         // global index of the unit's first tile
            int px = 0;                                         // meetings of this warp with its partner so far
            bool ok = true;
            // The two threads of a row (same lane of the two warps that share a lane quarter) meet: what each wrote to shared
            // memory before is visible to the other afterwards.  A bounded mbarrier wait like every other wait of the kernel.
            auto pair_sync = [&]() -> bool {
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->pair_bar[quarter]);
                const bool met = __all_sync(0xffffffffu, mbar_wait(&bars->pair_bar[quarter], px & 1, cx));
                ++px;
                return met;
            };
            PH_DECL(16);
            PH_T0(tw0);
            for (int un = 0; ok; ++un) {
                const int unit = read_unit(un, true);
                PH_ADD(0, tw0);
                if (unit == -2) { ok = false; break; }
                if (unit < 0) break;
                const Unit u = decode_unit(a, items, unit);
                const int i_row = u.row0 + (int)rank * kRows + t;   // row inside the chunk
                const int last_key = min(u.P + i_row, u.kv_end - 1);
                float m_ref = -INFINITY;                         // the row's reference maximum (both threads of the row hold the same value)
                float l = 0.f;                                   // row sum over this thread's keys, in units of m_ref
                for (int j = 0; j < u.n; ++j) {
                    const int g = g0 + j, b = g % kSBuf;
                    const int kb = u.kv_begin + j * kKeys + w * 64;                  // first key of this thread's half
                    const uint32_t tm_s = tmem + b * 128 + lane_sel;
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->s_full[b], (g / kSBuf) & 1, cx));
                    if (!ok) break;
                    PH_ADD(1, tw0);
                    tc_fence_after();
                    float s[64];
#pragma unroll
                    for (int c = 0; c < 2; ++c) tmem_ld32(tm_s + w * 64 + c * 32, reinterpret_cast<uint32_t*>(s) + c * 32);
                    tmem_ld_wait();

                    // raw maximum (the scale is positive, so it commutes with max); four independent chains
                    const int lim = last_key - kb;              // keys 0..lim of this half are visible to this row
                    if (lim < 63) {
#pragma unroll
                        for (int k = 0; k < 64; ++k) s[k] = (k <= lim) ? s[k] : -INFINITY;
                    }
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int k = 0; k < 64; k += 8) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) mx4[v] = fmaxf(mx4[v], fmaxf(s[k + 2 * v], s[k + 2 * v + 1]));
                    }
                    const float mx_half = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                    PH_ADD(2, tw0);
                    // the other half's maximum.  After this meeting both threads also have their scores in registers, so P
                    // (which overwrites the score columns of BOTH halves) may be written
                    bars->mx_x[g & 1][w][t] = mx_half;
                    ok = pair_sync();
                    if (!ok) break;
                    const float mx = fmaxf(mx_half, bars->mx_x[g & 1][w ^ 1][t]) * sc;
                    PH_ADD(3, tw0);
                    // the reference moves only when this tile's maximum exceeds it by more than the threshold (same decision in
                    // both threads of the row: same inputs)
                    const float m_new = (mx > m_ref + kRescaleThreshold) ? mx : m_ref;
                    const bool rescale = (m_new != m_ref) && (m_ref != -INFINITY);
                    const float alpha = rescale ? fast_exp2(m_ref - m_new) : 1.f;
                    if (m_ref != m_new) l *= (m_ref == -INFINITY) ? 0.f : alpha;
                    m_ref = m_new;

                    const float neg_ref = (m_new == -INFINITY) ? 0.f : -m_new;
                    // packed fp32 arithmetic (two values per instruction) for the scale, the row sum and the remainder
                    const uint64_t sc2 = f2_pack(sc, sc), neg2 = f2_pack(neg_ref, neg_ref);
                    uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t p[16];
                        uint32_t pl[16];
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            float x0, x1;
                            f2_unpack(f2_fma(f2_pack(s[c * 32 + k], s[c * 32 + k + 1]), sc2, neg2), x0, x1);
                            const float e0 = fast_exp2(x0), e1 = fast_exp2(x1);
                            const uint64_t e2 = f2_pack(e0, e1);
                            sum2[(k >> 1) & 3] = f2_add(sum2[(k >> 1) & 3], e2);
                            p[k / 2] = pack2<true>(e0, e1);
                            float r0, r1;
                            f2_unpack(f2_sub(e2, f2_pack(__uint_as_float(p[k / 2] << 16), __uint_as_float(p[k / 2] & 0xffff0000u))), r0, r1);
                            pl[k / 2] = pack2<true>(r0, r1);
                        }
                        // keys 64 w + 32 c .. + 31 are words 32 w + 16 c .. + 15 of P (and of its remainder, 64 columns on)
                        tmem_st16(tm_s + w * 32 + c * 16, p);
                        tmem_st16(tm_s + 64 + w * 32 + c * 16, pl);
                    }
                    float sum4[4];
                    {
                        float a0, a1, b0, b1, c0, c1, d0, d1;
                        f2_unpack(sum2[0], a0, a1); f2_unpack(sum2[1], b0, b1); f2_unpack(sum2[2], c0, c1); f2_unpack(sum2[3], d0, d1);
                        sum4[0] = a0 + a1; sum4[1] = b0 + b1; sum4[2] = c0 + c1; sum4[3] = d0 + d1;
                    }
                    l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                    PH_ADD(4, tw0);

                    if (__any_sync(0xffffffffu, rescale)) {
                        // O holds the tiles before this one in units of the old reference; the previous tile's P V must have
                        // finished.  Each thread of the row rescales its half of the columns
                        ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[(g - 1) % kSBuf], ((g - 1) / kSBuf) & 1, cx));
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tm_o + w * 64 + c * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                            tmem_st32(tm_o + w * 64 + c * 32, o);
                        }
                    }
                    tmem_st_wait();
                    PH_ADD(5, tw0);
                    // this CTA's half of V tile g must have landed before the P V product may be issued (the MMA thread does
                    // not look at the V ring itself)
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->v_full[g % kStagesV], (g / kStagesV) & 1, cx));
                    if (!ok) break;
                    // a range that ends inside this tile: V rows past the range were not loaded (or hold stale slots); zero
                    // them in this CTA's column half so that 0 * garbage cannot produce NaN
                    if (u.kv_begin + (j + 1) * kKeys > u.kv_end) {
                        unsigned char* vt = v_ring + (g % kStagesV) * kHalfBytes;
                        const int first = u.kv_end - (u.kv_begin + j * kKeys);
                        for (int idx = wg_tid + w * 128; idx < (kKeys - first) * 8; idx += 256) {
                            const int row = first + idx / 8, part = idx % 8;       // 8 vectors of 16 bytes per 128-byte row
                            *reinterpret_cast<uint4*>(vt + row * 128 + part * 16) = make_uint4(0, 0, 0, 0);
                        }
                        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    }
                    // one arrival per warp: every lane's P is in TMEM (wait::st) and fenced before the warp meets
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(lead_p_ready + b * 8);
                    PH_ADD(6, tw0);
#ifdef HAT_PHASE_TIMERS
                    ph[15] += 1;
#endif
                }
                if (!ok) break;
                // ---- end of the unit: the two threads of a row add their row sums (both in units of the same reference),
                // and each stores its half of the columns
                const int up = un & 1;
                const int g_last = g0 + u.n - 1;
                bars->lsum2[up][w][t] = l;
                ok = pair_sync();
                if (!ok) break;
                const float l_tot = l + bars->lsum2[up][w ^ 1][t];
                const float m_fin = m_ref;
                PH_ADD(7, tw0);
                // the last P V of the unit
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[g_last % kSBuf], (g_last / kSBuf) & 1, cx));
                if (!ok) break;
                PH_ADD(8, tw0);
                tc_fence_after();
                float o[64];                                    // this warpgroup's half of the columns
#pragma unroll
                for (int c = 0; c < 2; ++c) tmem_ld32(tm_o + w * 64 + c * 32, reinterpret_cast<uint32_t*>(o) + c * 32);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(lead_o_free);
                if (i_row < u.C) {
                    const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
                    float* obase; float* lbase; int64_t orow;
                    if (u.part < 0) { obase = a.out; lbase = a.lse; orow = u.row_base + i_row; }
                    else { obase = a.part_out; lbase = a.part_lse; orow = u.part + (i_row - u.row0); }
                    HAT_CHECK(orow >= 0 && orow < (u.part < 0 ? (int64_t)a.plan.total_rows : a.part_rows), cx.status);
                    if (u.part < 0 && a.out16 != nullptr) {
                        // final rows in the 16-bit output type: 128 bytes per row and warpgroup
                        uint16_t* dst16 = static_cast<uint16_t*>(a.out16) + (orow * H + u.h) * kD + w * 64;
                        const bool wide16 = (reinterpret_cast<uintptr_t>(a.out16) & 31) == 0;
#pragma unroll
                        for (int k = 0; k < 64; k += 16) {
                            uint32_t wd[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) wd[e] = pack_out16(o[k + 2 * e] * inv, o[k + 2 * e + 1] * inv, a.out16_bf16);
                            if (wide16) {
                                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n"
                                             ::"l"(dst16 + k), "r"(wd[0]), "r"(wd[1]), "r"(wd[2]), "r"(wd[3]), "r"(wd[4]), "r"(wd[5]), "r"(wd[6]), "r"(wd[7]) : "memory");
                            } else {
                                *reinterpret_cast<uint4*>(dst16 + k) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                                *reinterpret_cast<uint4*>(dst16 + k + 8) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
                            }
                        }
                    } else {
                        float* dst = obase + (orow * H + u.h) * kD + w * 64;
                        if (wide_stores) {
#pragma unroll
                            for (int k = 0; k < 64; k += 8)
                                st_global_v8(dst + k, o[k] * inv, o[k + 1] * inv, o[k + 2] * inv, o[k + 3] * inv, o[k + 4] * inv,
                                             o[k + 5] * inv, o[k + 6] * inv, o[k + 7] * inv);
                        } else {
#pragma unroll
                            for (int k = 0; k < 64; k += 4)
                                *reinterpret_cast<float4*>(dst + k) = make_float4(o[k] * inv, o[k + 1] * inv, o[k + 2] * inv, o[k + 3] * inv);
                        }
                    }
                    if (w == 0) lbase[orow * H + u.h] = l_tot > 0.f ? (m_fin + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
                }
                g0 += u.n;
                PH_ADD(9, tw0);
#ifdef HAT_PHASE_TIMERS
                ph[14] += 1;
#endif
            }
#ifdef HAT_PHASE_TIMERS
            if (lane == 0 && quarter == 0) PH_FLUSH(16 + 16 * w, 16);
#endif
        } else {
            const int w = (warp - 2) >> 2;                      // warpgroup: takes the tiles with g % 2 == w
            const int quarter = warp & 3;                       // TMEM lanes this warp may touch
            const int t = quarter * 32 + lane;                  // query row inside this CTA's tile = TMEM lane
            const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
            const uint32_t tm_o = tmem + kColO + lane_sel;
            const int wg_tid = (int)threadIdx.x - 64 - w * 128;
            const float sc = a.scale_log2;
            const bool wide_stores = ((reinterpret_cast<uintptr_t>(a.out) | reinterpret_cast<uintptr_t>(a.part_out)) & 31) == 0;
            const uint32_t lead_o_free = lead(&bars->o_free), lead_p_ready = lead(&bars->p_ready[0]);
            int g0 = 0;                                         // global index of the unit's first tile
            bool ok = true;
            PH_DECL(16);
            PH_T0(tw0);
            for (int un = 0; ok; ++un) {
                const int unit = read_unit(un, true);
                PH_ADD(0, tw0);
                if (unit == -2) { ok = false; break; }
                if (unit < 0) break;
                const Unit u = decode_unit(a, items, unit);
                const int i_row = u.row0 + (int)rank * kRows + t;   // row inside the chunk
                const int last_key = min(u.P + i_row, u.kv_end - 1);
                float m_mine = -INFINITY, l = 0.f;               // reference this warpgroup's row sum is expressed in; the sum
                float m_other = -INFINITY;                       // reference the other warpgroup's latest tile of this unit left
                for (int j = (g0 & 1) == w ? 0 : 1; j < u.n; j += 2) {
                    const int g = g0 + j, b = g % kSBuf;
                    const int kb = u.kv_begin + j * kKeys;
                    const uint32_t tm_s = tmem + b * 128 + lane_sel;
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->s_full[b], (g / kSBuf) & 1, cx));
                    if (!ok) break;
                    PH_ADD(1, tw0);
                    tc_fence_after();
                    float s[kKeys];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(tm_s + c * 32, reinterpret_cast<uint32_t*>(s) + c * 32);
                    tmem_ld_wait();

                    // raw maximum (the scale is positive, so it commutes with max); four independent chains
                    const int lim = last_key - kb;              // keys 0..lim of this tile are visible to this row
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
                    PH_ADD(2, tw0);
                    // the reference the previous tile (the other warpgroup's) left behind
                    float m_prev = -INFINITY;
                    if (j > 0) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&bars->m_ready[w ^ 1][quarter], ((g - 1) >> 1) & 1, cx));
                        if (!ok) break;
                        m_prev = bars->mref[t];
                    }
                    PH_ADD(3, tw0);
                    // move it only when this tile's maximum exceeds it by more than the threshold
                    const float m_new = (mx > m_prev + kRescaleThreshold) ? mx : m_prev;
                    const bool rescale = (m_new != m_prev) && (m_prev != -INFINITY);
                    bars->mref[t] = m_new;                      // (this thread read the old value above: one array serves both directions)
                    m_other = m_prev;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->m_ready[w][quarter]);

                    const float neg_ref = (m_new == -INFINITY) ? 0.f : -m_new;
                    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t p[16];
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            const float e0 = fast_exp2(fmaf(s[c * 32 + k], sc, neg_ref));
                            const float e1 = fast_exp2(fmaf(s[c * 32 + k + 1], sc, neg_ref));
                            sum4[(k >> 1) & 3] += e0 + e1;
                            p[k / 2] = pack2<false>(e0, e1);
                        }
                        tmem_st16(tm_s + c * 16, p);
                    }
                    // this warpgroup's row sum, brought to the current reference first
                    if (m_mine != m_new) {
                        l *= (m_mine == -INFINITY) ? 0.f : fast_exp2(m_mine - m_new);
                        m_mine = m_new;
                    }
                    l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                    PH_ADD(4, tw0);

                    if (__any_sync(0xffffffffu, rescale)) {
                        // O holds the tiles before this one in units of m_prev; the previous tile's P V must have finished
                        ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[(g - 1) % kSBuf], ((g - 1) / kSBuf) & 1, cx));
                        if (!ok) break;
                        tc_fence_after();
                        const float alpha = rescale ? fast_exp2(m_prev - m_new) : 1.f;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tm_o + c * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                            tmem_st32(tm_o + c * 32, o);
                        }
                    }
                    tmem_st_wait();
                    PH_ADD(5, tw0);
                    // this CTA's half of V tile g must have landed before the P V product may be issued (the MMA thread does
                    // not look at the V ring itself)
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->v_full[g % kStagesV], (g / kStagesV) & 1, cx));
                    if (!ok) break;
                    // a range that ends inside this tile: V rows past the range were not loaded (or hold stale slots); zero
                    // them in this CTA's column half so that 0 * garbage cannot produce NaN
                    if (kb + kKeys > u.kv_end) {
                        unsigned char* vt = v_ring + (g % kStagesV) * kHalfBytes;
                        const int first = u.kv_end - kb;
                        for (int idx = wg_tid; idx < (kKeys - first) * 8; idx += 128) {
                            const int row = first + idx / 8, part = idx % 8;       // 8 vectors of 16 bytes per 128-byte row
                            *reinterpret_cast<uint4*>(vt + row * 128 + part * 16) = make_uint4(0, 0, 0, 0);
                        }
                        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    }
                    // one arrival per warp: every lane's P is in TMEM (wait::st) and fenced before the warp meets
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(lead_p_ready + b * 8);
                    PH_ADD(6, tw0);
#ifdef HAT_PHASE_TIMERS
                    ph[15] += 1;
#endif
                }
                if (!ok) break;
                // ---- end of the unit.  The warpgroup that did not take the last tile hands its row sum over (it is in units
                // of the reference the last tile read as m_prev); the other one adds its own, hands the total back and
                // writes the lse.  Each then stores its half of the columns.
                const int up = un & 1;
                const int g_last = g0 + u.n - 1;
                const bool took_last = (g_last & 1) == w;
                float l_tot, m_fin = m_mine;
                if (!took_last) {
                    bars->lsum[up][t] = l;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->fin_ready[w][quarter]);
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->fin_ready[w ^ 1][quarter], un & 1, cx));
                    if (!ok) break;
                    l_tot = bars->lsum[up][t];
                } else {
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->fin_ready[w ^ 1][quarter], un & 1, cx));
                    if (!ok) break;
                    const float l_other = bars->lsum[up][t];
                    l_tot = l;
                    if (u.n > 1 && m_other != -INFINITY) l_tot += l_other * fast_exp2(m_other - m_fin);
                    bars->lsum[up][t] = l_tot;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->fin_ready[w][quarter]);
                }
                PH_ADD(7, tw0);
                // the last P V of the unit
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[g_last % kSBuf], (g_last / kSBuf) & 1, cx));
                if (!ok) break;
                PH_ADD(8, tw0);
                tc_fence_after();
                float o[64];                                    // this warpgroup's half of the columns
#pragma unroll
                for (int c = 0; c < 2; ++c) tmem_ld32(tm_o + w * 64 + c * 32, reinterpret_cast<uint32_t*>(o) + c * 32);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(lead_o_free);
                if (i_row < u.C) {
                    const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
                    float* obase; float* lbase; int64_t orow;
                    if (u.part < 0) { obase = a.out; lbase = a.lse; orow = u.row_base + i_row; }
                    else { obase = a.part_out; lbase = a.part_lse; orow = u.part + (i_row - u.row0); }
                    HAT_CHECK(orow >= 0 && orow < (u.part < 0 ? (int64_t)a.plan.total_rows : a.part_rows), cx.status);
                    if (u.part < 0 && a.out16 != nullptr) {
                        // final rows in the 16-bit output type: 128 bytes per row and warpgroup
                        uint16_t* dst16 = static_cast<uint16_t*>(a.out16) + (orow * H + u.h) * kD + w * 64;
                        const bool wide16 = (reinterpret_cast<uintptr_t>(a.out16) & 31) == 0;
#pragma unroll
                        for (int k = 0; k < 64; k += 16) {
                            uint32_t wd[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) wd[e] = pack_out16(o[k + 2 * e] * inv, o[k + 2 * e + 1] * inv, a.out16_bf16);
                            if (wide16) {
                                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n"
                                             ::"l"(dst16 + k), "r"(wd[0]), "r"(wd[1]), "r"(wd[2]), "r"(wd[3]), "r"(wd[4]), "r"(wd[5]), "r"(wd[6]), "r"(wd[7]) : "memory");
                            } else {
                                *reinterpret_cast<uint4*>(dst16 + k) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                                *reinterpret_cast<uint4*>(dst16 + k + 8) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
                            }
                        }
                    } else {
                        float* dst = obase + (orow * H + u.h) * kD + w * 64;
                        if (wide_stores) {
#pragma unroll
                            for (int k = 0; k < 64; k += 8)
                                st_global_v8(dst + k, o[k] * inv, o[k + 1] * inv, o[k + 2] * inv, o[k + 3] * inv, o[k + 4] * inv,
                                             o[k + 5] * inv, o[k + 6] * inv, o[k + 7] * inv);
                        } else {
#pragma unroll
                            for (int k = 0; k < 64; k += 4)
                                *reinterpret_cast<float4*>(dst + k) = make_float4(o[k] * inv, o[k + 1] * inv, o[k + 2] * inv, o[k + 3] * inv);
                        }
                    }
                    if (took_last) lbase[orow * H + u.h] = l_tot > 0.f ? (m_fin + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
                }
                g0 += u.n;
                PH_ADD(9, tw0);
#ifdef HAT_PHASE_TIMERS
                ph[14] += 1;
#endif
            }
#ifdef HAT_PHASE_TIMERS
            if (lane == 0 && quarter == 0) PH_FLUSH(16 + 16 * w, 16);
#endif
        }
    }

    // both CTAs are done with each other's barriers, and every MMA has finished, before tensor memory is freed
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
    }
    // The last CTA to get here (none draws units any more) leaves the unit counter at zero for the next call, which
    // then needs no memset in front of it.  work_counter[1] counts the CTAs that have finished.
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(work_counter + 1, 1) == (int)gridDim.x - 1) {
            work_counter[0] = 0;
            work_counter[1] = 0;
            __threadfence();
        }
    }
}

}  // namespace

cudaError_t launch_attn_pair(const hat_plan* plan, const AttnArgs& args, cudaStream_t stream, int num_units) {
    const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
    const CUtensorMap *mk = nullptr, *mv = nullptr;
    const CUtensorMap* mq = plan_q_map(plan, args.q);
    if (!mq || !plan_pool_maps(plan, args.cache, &mk, &mv)) return cudaErrorInvalidValue;
    // the unit counter is zero at this point: the previous call's last CTA cleared it
    const int total_units = num_units >= 0 ? num_units : (int)plan->tile_units.size();
    if (total_units <= 0) return cudaSuccess;
    int32_t* counter = plan->dev.status + 1;
    // one cluster of two CTAs per pair of SMs, never more clusters than units
    int pairs = std::min(total_units, plan->num_sms / 2);
    if (const char* g = std::getenv("HAT_PAIR_GRID")) pairs = std::max(1, std::min(pairs, std::atoi(g)));
    const dim3 grid((unsigned)(2 * pairs));
    auto kern = bf16 ? attn_pair_kernel<true> : attn_pair_kernel<false>;
    cudaError_t e = smem_attr_once(reinterpret_cast<const void*>(kern), kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmemBytes, stream>>>(args, plan->dev.prefill_items, total_units, counter, *mq, *mk, *mv);
    count_launch();
    return cudaGetLastError();
}

#ifdef HAT_PHASE_TIMERS
extern "C" int hat_debug_phase_read(unsigned long long* out, int n, int clear) {
    if (n > 80) n = 80;
    cudaError_t e = cudaMemcpyFromSymbol(out, g_phase, sizeof(unsigned long long) * n);
    if (e == cudaSuccess && clear) {
        unsigned long long z[80] = {0};
        e = cudaMemcpyToSymbol(g_phase, z, sizeof z);
    }
    return e == cudaSuccess ? 0 : -1;
}
#endif

}  // namespace hat
