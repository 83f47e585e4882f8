// Internal declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <vector>

#include "../../include/hat.h"

namespace hat {

constexpr int kPageSize = 16;
constexpr int kMaxSplits = 32;     // a merged row combines at most this many key ranges (one lane each)

// One CTA's worth of attention work for one head: rows [row0, row0+tile_rows) of request `req`
// against keys [kv_begin, kv_end).  `part` < 0: the CTA writes the final out/lse rows; otherwise it
// writes partial results at partial-row index part + (row - 0) for later merging.
struct WorkItem {
    int32_t req;
    int32_t row0;
    int32_t kv_begin;
    int32_t kv_end;
    int32_t part;
    int32_t pad0, pad1, pad2;
};

// Rows whose result is merged from `nsplit` partial rows part0 + s*stride, s = 0..nsplit-1.
struct MergeRow {
    int32_t row;      // packed row index t
    int32_t part0;    // partial-row index of split 0
    int32_t stride;   // partial-row distance between consecutive splits
    int32_t nsplit;
};

// Device-resident view of a plan (all pointers device).
struct DevicePlan {
    const int32_t*  cu_chunk;
    const int32_t*  prefix_len;
    const int32_t*  chunk_len;
    const int32_t*  block_table;
    const int32_t*  row_req;        // [T] request of each packed row
    const WorkItem* verify_items;
    const WorkItem* prefill_items;
    const uint32_t* tile_units;     // tcgen05 tile kernels: unit -> prefill item (low 16 bits) | query head (high 16 bits), in draw order
    const MergeRow* merge_rows;
    const uint32_t* tree_mask;      // [T] or null: visible chunk positions of each row of a streaming-class request
    int32_t*        status;         // device status word (0 = ok)
    int32_t         max_pages;
    int32_t         num_heads;      // query heads (q, out, lse, partial results)
    int32_t         num_kv_heads;   // K/V heads (pools, k_new, v_new)
    int32_t         group;          // query heads per K/V head
    int32_t         total_rows;
    int32_t         num_pages;      // pages in the pools (index checks of the debug build)
};

struct CacheView {
    const void* k_pool;
    const void* v_pool;
    int64_t stride_page, stride_token, stride_head;
};

struct AttnArgs {
    DevicePlan  plan;
    CacheView   cache;
    const void* q;
    float*      out;          // [T][H][d]; unused when out16 is set
    void*       out16;        // [T][H][d] in the cache's 16-bit type, or null: final rows go here instead of `out`
    int         out16_bf16;   // type of out16: 0 = fp16, 1 = bf16
    float*      lse;          // [T][H]
    float*      part_out;     // [part_rows][H][d]
    float*      part_lse;     // [part_rows][H]
    int64_t     part_rows;    // partial rows the workspace holds (index checks of the debug build)
    float       scale_log2;   // sm_scale * log2(e)
    long long   wait_cycles;  // bound of every device-side wait, in SM clock cycles
    int         withhold;     // self test: the tile kernel's producer skips its first V tile so that a wait runs out
    int         tail_reset;   // the last CTA of the persistent tile kernel to finish clears the unit counter for the next call
};

// Key range of one split of the allocation-free streaming entry point, from lengths that nobody validated (they are
// read from device memory).  A negative prefix counts as 0, the chunk is cut to [0, max_rows], and prefix + chunk is
// cut to the max_pages * 16 tokens one row of the block table can address: wrong lengths then give wrong rows, never a
// lookup outside the table.  Ranges are whole pages, HAT_STATIC_SPLITS of equal length; trailing ranges may be empty.
struct StaticRange { int prefix, rows, kv_begin, kv_end; };
#ifdef __CUDACC__
__host__ __device__
#endif
inline StaticRange static_key_range(int prefix_len, int chunk_len, int max_rows, int max_pages, int split) {
    const long long cap = (long long)max_pages * kPageSize;
    long long P = prefix_len < 0 ? 0 : prefix_len;
    long long C = chunk_len < 0 ? 0 : (chunk_len > max_rows ? max_rows : chunk_len);
    if (P > cap) P = cap;
    if (P + C > cap) C = cap - P;
    const long long N = P + C;
    const long long per = ((N + HAT_STATIC_SPLITS - 1) / HAT_STATIC_SPLITS + kPageSize - 1) / kPageSize * kPageSize;
    long long b = (long long)split * per, e = b + per;
    if (b > N) b = N;
    if (e > N) e = N;
    return StaticRange{(int)P, (int)C, (int)b, (int)e};
}

// Debug build (-DHAT_DEBUG_BOUNDS): indices that the release build trusts (they were validated on the host, or follow
// from the kernel's own arithmetic) are range-checked on the device; a violation raises bit 1 of the plan's status
// word (hat_last_device_status then reports HAT_ERR_DEVICE_BOUNDS) and never traps.  HAT_IN_RANGE returns the index
// clamped into [0, n) so that the access that follows stays inside the array either way.
#if defined(__CUDACC__) && defined(HAT_DEBUG_BOUNDS)
__device__ __forceinline__ int hat_in_range(int i, int n, int32_t* status) {
    if (i < 0 || i >= n) { atomicOr(status, 2); return i < 0 ? 0 : (n > 0 ? n - 1 : 0); }
    return i;
}
#define HAT_IN_RANGE(i, n, status) hat_in_range((i), (n), (status))
#define HAT_CHECK(cond, status) do { if (!(cond)) atomicOr((status), 2); } while (0)
#else
#define HAT_IN_RANGE(i, n, status) (i)
#define HAT_CHECK(cond, status) do { } while (0)
#endif

// Rotary position encoding: theta^(-2c/d) for c = 0 .. d/2 - 1, computed on the host in double and passed by value
struct InvFreq { double f[64]; };
#ifdef __CUDACC__
// sine and cosine of position p times one of those factors: the angle is formed and reduced to [-pi, pi] in double,
// the functions themselves are fp32
__device__ __forceinline__ void rope_sincos(int p, double inv_freq, float* s, float* c) {
    const double ang = (double)p * inv_freq;
    const double turns = rint(ang * 0.15915494309189535);                  // 1 / (2 pi)
    const double red = fma(-turns, 6.283185307179586, ang) - turns * 2.4492935982947064e-16;
    sincosf((float)red, s, c);
}
#endif

#ifdef __CUDACC__
// Two fp32 values rounded to nearest into one 32-bit word of the 16-bit output type (low half = first value).
__device__ __forceinline__ uint32_t pack_out16(float lo, float hi, int bf16) {
    uint32_t w;
    if (bf16) asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(w) : "f"(hi), "f"(lo));
    else asm("cvt.rn.f16x2.f32 %0, %1, %2;\n" : "=r"(w) : "f"(hi), "f"(lo));
    return w;
}
#endif

}  // namespace hat

namespace hat {
// Event recorder for the optional per-kernel timing (a start and an end event per slot and recorded call).
struct Timing {
    std::vector<cudaEvent_t> events;
    std::vector<uint8_t> launched;   // [call][slot]
    int max_calls = 0;
    int next = 0;
};
}  // namespace hat

#include <cuda.h>
namespace hat {
// Tensor maps of the last call, kept with what they were encoded for: a plan is reused for every layer of a step (and
// by benchmarks for many steps) with the same pools and often the same q buffer, and encoding three maps per call is
// a large part of the host time of a launch-bound step.
struct MapCache {
    const void* q = nullptr; const void* k = nullptr; const void* v = nullptr;
    int64_t stride_page = 0, stride_token = 0, stride_head = 0;
    bool have_q = false, have_kv = false;
    CUtensorMap mq, mk, mv;
};
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device instead of once per launch
cudaError_t smem_attr_once(const void* kernel, int bytes);
}  // namespace hat

struct hat_plan {
    // geometry the plan was made for
    int32_t dtype, num_pages, num_heads, num_kv_heads, head_dim, max_pages, num_requests, total_rows;   // num_heads: query heads
    int32_t verify_subtiles;    // 16-row slabs of (row, query head of a group) pairs per streaming work item and K/V head
    std::vector<uint32_t> tree_mask;
    bool host_only;
    int device;
    int num_sms;
    std::vector<int32_t> cu_chunk, prefix_len, chunk_len, block_table, row_req;
    std::vector<hat::WorkItem> verify_items, prefill_items;
    std::vector<uint32_t> tile_units;   // (item, head) of every unit of the tcgen05 tile kernels, in the order they are drawn
    bool pair_takes_all;                // HAT_PREFILL_KERNEL=pair: every unit goes to the CTA-pair kernel, narrow ones too (tests)
    int num_pair_units;                 // CTA-pair kernel in use: the first num_pair_units units are its (more than 128 rows each), the rest go to the one-CTA kernel
    std::vector<hat::MergeRow> merge_rows;
    int64_t part_rows;          // partial rows in the workspace
    hat_plan_info info;
    hat::Timing* timing;        // null unless hat_plan_enable_timing was called
    int num_verify_merge_rows;  // merge rows of streaming-class requests; they come first in merge_rows
    cudaEvent_t ev_verify;      // recorded in every attention call once the streaming-class rows are final
    cudaEvent_t ev_done;        // recorded at the end of every attention call: the next call on another stream waits for it
    cudaStream_t last_stream;   // stream of the previous attention call
    bool has_last;
    // mixed batches: the tile kernel starts on side_sms fewer SMs on a stream of its own while the streaming kernel
    // (bound by HBM, which far fewer than all SMs saturate) runs on the caller's stream; a second tile grid joins
    // on the freed SMs
    int side_sms;
    cudaStream_t aux_stream;
    cudaEvent_t ev_fork, ev_join;
    long long wait_cycles;      // bound of device-side waits (default: about a second)
    int withhold_next;          // self test of the bounded waits: applies to the next attention call only
    hat::MapCache maps;         // see MapCache (updated through const_cast by the launchers: one call at a time per plan)
    // rotary position encoding in the projection epilogue: (cos, sin) of every row and pair for base rope_theta
    // (0: not filled yet), inside dev_blob; ev_table orders calls on other streams behind the kernel that filled it
    float2* rope_table;
    float rope_theta;
    cudaStream_t table_stream;
    cudaEvent_t ev_table;
    void* dev_blob;             // one allocation holding every device array
    hat::DevicePlan dev;
};

namespace hat {
// kernel launchers (each returns a cudaError_t from the launch)
cudaError_t launch_kv_append(const hat_plan* plan, const CacheView& cache, void* k_pool, void* v_pool,
                             const void* k_new, const void* v_new, cudaStream_t stream);
cudaError_t launch_attn_mma(const hat_plan* plan, const AttnArgs& args, bool verify_class, cudaStream_t stream);
// rotary position encoding: of rows `src` ([T][heads][d]) into `dst`, or (cache != null) of K rows into the pools with
// the V rows copied beside them
cudaError_t launch_rope(const hat_plan* plan, int heads, float theta, int interleaved, const void* src, void* dst,
                        const CacheView* cache, void* k_pool, void* v_pool, const void* v_new, cudaStream_t stream);
cudaError_t launch_merge(const hat_plan* plan, const AttnArgs& args, int first_row, int num_rows, cudaStream_t stream);
// tcgen05 tile kernel (head_dim 64 or 128): whether a TMA descriptor can be built for this pool layout, and the launcher
bool tc5_layout_supported(int dtype, int head_dim, int num_pages, int H, int64_t stride_page, int64_t stride_token,
                          int64_t stride_head);
// grid_limit > 0 caps the number of CTAs; reset_counter = false joins a grid that is already drawing units
// first_unit / num_units (num_units < 0: all) select a part of the plan's unit list; counter_word: which pair of the
// plan's status words (unit counter, finished CTAs) the grid uses
cudaError_t launch_attn_tc5(const hat_plan* plan, const AttnArgs& args, cudaStream_t stream, int grid_limit = 0,
                            bool reset_counter = true, int first_unit = 0, int num_units = -1, int counter_word = 1);
// tcgen05 tile kernel with 256-row units processed by clusters of two CTAs (cta_group::2), same layout requirements
cudaError_t launch_attn_pair(const hat_plan* plan, const AttnArgs& args, cudaStream_t stream, int num_units = -1);   // the first num_units units
// TMA-fed streaming kernel: whether a TMA descriptor can be built for this pool layout, and the launcher
bool stream_layout_supported(int dtype, int head_dim, int num_pages, int H, int64_t stride_page, int64_t stride_token,
                             int64_t stride_head);
cudaError_t launch_attn_stream(const hat_plan* plan, const AttnArgs& args, cudaStream_t stream);
// Q/K/V projection with the rotation and the cache write in its epilogue (tcgen05); theta <= 0: no rotation
cudaError_t launch_qkv_gemm(const hat_plan* plan, const CacheView& cache, void* k_pool, void* v_pool, const void* x,
                            int hidden, const void* w, void* q_out, float theta, int interleaved, cudaStream_t stream);
void count_launch(int n = 1);
void set_last_cuda_error(int e);   // what hat_last_cuda_error() returns on this thread
}  // namespace hat

namespace hat {
// The plan's cached tensor maps for these pools / this q buffer, encoded again only when a pointer or a stride changed.
// Return null when no map can be built.  (Defined in hat_api.cu.)
bool plan_pool_maps(const hat_plan* plan, const CacheView& cache, const CUtensorMap** mk, const CUtensorMap** mv);
const CUtensorMap* plan_q_map(const hat_plan* plan, const void* q);
}  // namespace hat
