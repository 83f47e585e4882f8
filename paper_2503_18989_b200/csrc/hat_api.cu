// C ABI of the library: status strings, host-side validation and scheduling (the plan), and the
// entry points that enqueue the kernels.  Declarations and argument contracts are in include/hat.h.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>
#include <queue>

#include "hat_internal.h"
#include "tma_desc.h"

namespace hat {

static thread_local int g_last_cuda_error = 0;
static std::atomic<int64_t> g_launches{0};

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

cudaError_t smem_attr_once(const void* kernel, int bytes) {
    struct Done { const void* kernel; int device; };
    static std::mutex mu;
    static std::vector<Done> done;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (const Done& d : done)
        if (d.kernel == kernel && d.device == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done.push_back(Done{kernel, dev});
    return e;
}

bool plan_pool_maps(const hat_plan* plan, const CacheView& c, const CUtensorMap** mk, const CUtensorMap** mv) {
    MapCache& m = const_cast<hat_plan*>(plan)->maps;
    if (!m.have_kv || m.k != c.k_pool || m.v != c.v_pool || m.stride_page != c.stride_page ||
        m.stride_token != c.stride_token || m.stride_head != c.stride_head) {
        const bool bf16 = plan->dtype == HAT_DTYPE_BF16;
        m.have_kv = false;
        if (!tma_encode_pool_map(&m.mk, bf16, c.k_pool, plan->head_dim, plan->num_pages, plan->num_kv_heads, c.stride_page,
                                 c.stride_token, c.stride_head) ||
            !tma_encode_pool_map(&m.mv, bf16, c.v_pool, plan->head_dim, plan->num_pages, plan->num_kv_heads, c.stride_page,
                                 c.stride_token, c.stride_head))
            return false;
        m.k = c.k_pool; m.v = c.v_pool;
        m.stride_page = c.stride_page; m.stride_token = c.stride_token; m.stride_head = c.stride_head;
        m.have_kv = true;
    }
    *mk = &m.mk; *mv = &m.mv;
    return true;
}

const CUtensorMap* plan_q_map(const hat_plan* plan, const void* q) {
    MapCache& m = const_cast<hat_plan*>(plan)->maps;
    if (!m.have_q || m.q != q) {
        m.have_q = false;
        if (!tma_encode_q_map(&m.mq, plan->dtype == HAT_DTYPE_BF16, q, plan->total_rows, plan->num_heads, plan->head_dim)) return nullptr;
        m.q = q;
        m.have_q = true;
    }
    return &m.mq;
}

static int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return HAT_ERR_CUDA;
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    char* end = nullptr;
    long v = std::strtol(s, &end, 10);
    return (end && *end == 0) ? (int)v : dflt;
}

static inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
static inline int ceil_div(int x, int m) { return (x + m - 1) / m; }

static int check_cache_geometry(const hat_cache_desc* c) {
    if (!c) return HAT_ERR_INVALID_ARG;
    if (c->num_pages < 0) return HAT_ERR_INVALID_ARG;
    if (c->dtype != HAT_DTYPE_FP16 && c->dtype != HAT_DTYPE_BF16) return HAT_ERR_UNSUPPORTED;
    if (c->page_size != kPageSize) return HAT_ERR_UNSUPPORTED;
    if (c->head_dim != 64 && c->head_dim != 128) return HAT_ERR_UNSUPPORTED;
    if (c->num_kv_heads <= 0) return HAT_ERR_INVALID_ARG;
    if (c->stride_page <= 0 || c->stride_token <= 0 || c->stride_head <= 0) return HAT_ERR_INVALID_ARG;
    if (c->stride_page % 8 || c->stride_token % 8 || c->stride_head % 8) return HAT_ERR_UNSUPPORTED;
    return HAT_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Cut the key range [0, kv_end) of one tile into pieces of `split_len` keys (the last piece takes the
// remainder) and emit one work item per piece.
static void emit_tile(hat_plan* p, std::vector<WorkItem>& items, int req, int row0, int rows_valid,
                      int kv_end, int split_len) {
    int nsplit = (split_len > 0) ? ceil_div(kv_end, split_len) : 1;
    if (nsplit <= 1) {
        items.push_back(WorkItem{req, row0, 0, kv_end, -1, 0, 0, 0});
        return;
    }
    int64_t base = p->part_rows;
    for (int s = 0; s < nsplit; ++s) {
        int b = s * split_len, e = std::min(kv_end, b + split_len);
        items.push_back(WorkItem{req, row0, b, e, (int32_t)(base + (int64_t)s * rows_valid), 0, 0, 0});
    }
    int row_base = p->cu_chunk[req] + row0;
    for (int i = 0; i < rows_valid; ++i)
        p->merge_rows.push_back(MergeRow{row_base + i, (int32_t)(base + i), rows_valid, nsplit});
    p->part_rows += (int64_t)nsplit * rows_valid;
    p->info.max_splits = std::max(p->info.max_splits, nsplit);
}

static int split_len_for(int kv_end, int wanted, int granule) {
    // at most kMaxSplits pieces per tile
    int least = round_up(ceil_div(kv_end, kMaxSplits), granule);
    return std::max(wanted, least);
}

// Key-range length for the tile-class requests of a batch that is too small to fill the persistent tcgen05 kernel.
// Every candidate length is priced with a small model of that kernel, in SM clock cycles measured on B200: a 128-key
// step of a 256-row unit (two query tiles) or of a unit of at most 128 rows (two chains share it), the fixed cost of a
// unit (its Q tiles, refilling the rings, storing its rows), and the merge pass (its launch plus reading every partial
// row).  Units go to the CTAs longest first, as the kernel draws them.  Returns 0 for "leave every request whole".
static int pick_prefill_split(const hat_plan* p, int num_sms, int tile_rows, int key_granule) {
    constexpr int64_t kStepWide = 4000, kStepNarrow = 2200, kUnit = 10000, kMergeLaunch = 5700;
    constexpr int64_t kMergeBytesPerCycle = 3000;
    struct Tile { int keys, rows; };
    std::vector<Tile> tiles;
    int max_keys = 0;
    for (int r = 0; r < p->num_requests; ++r) {
        const int C = p->chunk_len[r];
        if (C <= 16) continue;
        for (int row0 = 0; row0 < C; row0 += tile_rows) {
            const int rows = std::min(tile_rows, C - row0);
            tiles.push_back(Tile{p->prefix_len[r] + row0 + rows, rows});
            max_keys = std::max(max_keys, tiles.back().keys);
        }
    }
    const int H = p->num_heads;
    std::vector<int64_t> units;
    auto price = [&](int len) -> int64_t {
        units.clear();
        int64_t part_rows = 0;
        for (const Tile& t : tiles) {
            const int sl = len > 0 ? split_len_for(t.keys, len, key_granule) : t.keys;
            const int n = ceil_div(t.keys, sl);
            if (n > 1) part_rows += (int64_t)n * t.rows;
            for (int s = 0; s < n; ++s) {
                const int keys = std::min(t.keys, (s + 1) * sl) - s * sl;
                units.push_back(ceil_div(keys, 128) * (t.rows > 128 ? kStepWide : kStepNarrow) + kUnit);
            }
        }
        std::sort(units.begin(), units.end(), std::greater<int64_t>());
        std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>> sms;
        for (int i = 0; i < num_sms; ++i) sms.push(0);
        int64_t makespan = 0;
        for (int h = 0; h < H; ++h) {
            for (int64_t u : units) {
                const int64_t t = sms.top() + u;
                sms.pop();
                sms.push(t);
                makespan = std::max(makespan, t);
            }
        }
        if (part_rows > 0) makespan += kMergeLaunch + part_rows * H * (p->head_dim + 1) * 4 / kMergeBytesPerCycle;
        return makespan;
    };
    int best = 0;
    int64_t best_cost = price(0);
    for (int len = 256; len < max_keys; len += (len < 1024 ? 128 : len < 4096 ? 512 : 2048)) {
        const int64_t c = price(len);
        if (c < best_cost) { best_cost = c; best = len; }
    }
    return best;
}

// tile_kernel: 0 = mma.sync, 1 = tcgen05 with two query tiles per CTA, 3 = tcgen05 by pairs of CTAs (cta_group::2) with a
// ring of three score buffers; both tcgen05 kernels take 256-row units
static void schedule(hat_plan* p, int num_sms, int tile_kernel) {
    const bool use_tc5 = tile_kernel != 0;
    const int H = p->num_heads;
    const int R = p->num_requests;
    hat_plan_info& info = p->info;

    const int verify_max_rows = 16;
    // tile kernel: tcgen05 with 256-row tiles (two 128-row MMA tiles) and 128-key steps, or mma.sync with 4 warps x 16 rows and 64-key steps
    const int tile_rows = use_tc5 ? 256 : 64;
    const int key_granule = use_tc5 ? 128 : 64;
    info.prefill_tile_rows = tile_rows;
    info.prefill_kernel = tile_kernel;

    // ---- streaming (verify-class) requests: fixed-length key ranges, shortened until the SMs are covered.
    // A CTA of the streaming kernel serves one K/V head and 16 (row, query head of the group) pairs.
    const int group = H / p->num_kv_heads;
    int max_verify_rows = 0;
    for (int r = 0; r < R; ++r) {
        int C = p->chunk_len[r];
        if (C >= 1 && C <= verify_max_rows) {
            info.num_verify_requests++;
            max_verify_rows = std::max(max_verify_rows, C);
        } else if (C > verify_max_rows) {
            info.num_prefill_requests++;
        }
    }
    p->verify_subtiles = std::max(1, ceil_div(max_verify_rows * group, 16));
    int vsplit = env_int("HAT_VERIFY_SPLIT_LEN", 0);
    if (vsplit <= 0) {
        // Long ranges stream best (a CTA's pipeline ramp and its cross-warp merge are paid once per range, and an
        // unsplit request needs no merge pass): start unsplit and halve the range only while the grid would not
        // give every SM about three rounds of two resident CTAs.
        vsplit = 16384;
        const int64_t want_ctas = (int64_t)num_sms * 6;
        auto ctas_at = [&](int len) {
            int64_t n = 0;
            for (int r = 0; r < R; ++r) {
                const int C = p->chunk_len[r];
                if (C >= 1 && C <= verify_max_rows) n += ceil_div(p->prefix_len[r] + C, len);
            }
            return n * p->num_kv_heads * p->verify_subtiles;
        };
        while (vsplit > 256 && ctas_at(vsplit) < want_ctas) vsplit /= 2;
    }
    vsplit = std::max(kPageSize, round_up(vsplit, kPageSize));
    info.verify_split_len = vsplit;

    // ---- tile (prefill-class) requests: cut keys only when there are too few tiles to cover the SMs
    int64_t tiles = 0, tile_keys = 0;
    for (int r = 0; r < R; ++r) {
        int C = p->chunk_len[r];
        if (C <= verify_max_rows) continue;
        for (int row0 = 0; row0 < C; row0 += tile_rows) {
            tiles++;
            tile_keys += p->prefix_len[r] + std::min(C, row0 + tile_rows);
        }
    }
    int psplit = env_int("HAT_PREFILL_SPLIT_LEN", -1);
    if (psplit < 0) {
        psplit = 0;
        const int64_t want_ctas = (int64_t)num_sms * 2;
        if (tiles > 0 && tiles * H < want_ctas && use_tc5) {
            psplit = pick_prefill_split(p, num_sms, tile_rows, key_granule);
        } else if (tiles > 0 && tiles * H < want_ctas) {
            // aim for want_ctas pieces of equal length, not shorter than 256 keys
            const int pieces = ceil_div((int)want_ctas, H);
            psplit = std::max(256, round_up((int)((tile_keys + pieces - 1) / pieces), key_granule));
        }
    }
    if (psplit > 0) psplit = round_up(psplit, key_granule);
    info.prefill_split_len = psplit;

    // streaming-class requests first: their merge rows form the head of merge_rows, so that they can be merged (and
    // announced through the plan's event) before the tile kernel runs
    for (int r = 0; r < R; ++r) {
        const int C = p->chunk_len[r], P = p->prefix_len[r];
        if (C <= 0 || C > verify_max_rows) continue;
        const int kv_end = P + C;
        emit_tile(p, p->verify_items, r, 0, C, kv_end, split_len_for(kv_end, vsplit, kPageSize));
    }
    p->num_verify_merge_rows = (int)p->merge_rows.size();
    for (int r = 0; r < R; ++r) {
        const int C = p->chunk_len[r], P = p->prefix_len[r];
        if (C <= verify_max_rows) continue;
        for (int row0 = 0; row0 < C; row0 += tile_rows) {
            const int rows_valid = std::min(tile_rows, C - row0);
            const int kv_end = P + row0 + rows_valid;
            const int sl = psplit > 0 ? split_len_for(kv_end, psplit, key_granule) : 0;
            emit_tile(p, p->prefill_items, r, row0, rows_valid, kv_end, sl);
        }
    }
    // longest pieces first so the tail of the grid is made of short ones
    auto longer = [](const WorkItem& a, const WorkItem& b) {
        return (a.kv_end - a.kv_begin) > (b.kv_end - b.kv_begin);
    };
    std::stable_sort(p->verify_items.begin(), p->verify_items.end(), longer);
    std::stable_sort(p->prefill_items.begin(), p->prefill_items.end(), longer);

    // Units of the persistent tcgen05 kernels, in the order the CTAs draw them: requests by their longest item first;
    // inside a request head by head, and for each head all items of the request one after the other, so that the row
    // blocks of one chunk (which read the same K/V of that head) run at the same time on neighbouring CTAs and meet in L2.
    p->tile_units.clear();
    p->num_pair_units = 0;
    if (use_tc5) {
        std::vector<int> first_of_req(R, -1);
        std::vector<std::vector<int>> group;
        for (int i = 0; i < (int)p->prefill_items.size(); ++i) {
            const int r = p->prefill_items[i].req;
            if (first_of_req[r] < 0) { first_of_req[r] = (int)group.size(); group.emplace_back(); }
            group[first_of_req[r]].push_back(i);
        }
        // With the CTA-pair kernel in use, units of more than 128 rows come first (they are its); units that would leave
        // half of a pair idle follow and go to the one-CTA kernel.
        auto rows_of = [&](int i) { return std::min(tile_rows, p->chunk_len[p->prefill_items[i].req] - p->prefill_items[i].row0); };
        for (int pass = 0; pass < (tile_kernel == 3 ? 2 : 1); ++pass) {
            for (const std::vector<int>& g : group)      // items are sorted longest first, so groups are too
                for (int h = 0; h < H; ++h)
                    for (int i : g) {
                        if (tile_kernel == 3 && ((rows_of(i) > 128 || p->pair_takes_all) != (pass == 0))) continue;
                        p->tile_units.push_back((uint32_t)i | ((uint32_t)h << 16));
                    }
            if (pass == 0) p->num_pair_units = tile_kernel == 3 ? (int)p->tile_units.size() : 0;
        }
    }

    info.num_verify_items = (int32_t)p->verify_items.size();
    info.num_prefill_items = (int32_t)p->prefill_items.size();
    info.num_merge_rows = (int32_t)p->merge_rows.size();
    const int64_t d = p->head_dim;
    int64_t part_out_bytes = p->part_rows * H * d * 4;
    part_out_bytes = (part_out_bytes + 255) / 256 * 256;
    info.workspace_bytes = p->part_rows ? part_out_bytes + ((p->part_rows * H * 4 + 255) / 256 * 256) : 0;
}

template <typename T>
static size_t blob_append(std::vector<char>& blob, const std::vector<T>& v) {
    size_t off = (blob.size() + 255) / 256 * 256;
    blob.resize(off + std::max<size_t>(v.size() * sizeof(T), 16));
    if (!v.empty()) std::memcpy(blob.data() + off, v.data(), v.size() * sizeof(T));
    return off;
}

static int upload(hat_plan* p) {
    std::vector<char> blob;
    size_t o_cu = blob_append(blob, p->cu_chunk);
    size_t o_pl = blob_append(blob, p->prefix_len);
    size_t o_cl = blob_append(blob, p->chunk_len);
    size_t o_bt = blob_append(blob, p->block_table);
    size_t o_rr = blob_append(blob, p->row_req);
    size_t o_vi = blob_append(blob, p->verify_items);
    size_t o_pi = blob_append(blob, p->prefill_items);
    size_t o_mr = blob_append(blob, p->merge_rows);
    size_t o_tu = blob_append(blob, p->tile_units);
    size_t o_tm = blob_append(blob, p->tree_mask);
    std::vector<int32_t> status(8, 0);     // status word; (unit counter, finished CTAs) of the tile kernel; the same for a second tile grid; spare
    size_t o_st = blob_append(blob, status);

    cudaError_t e = cudaGetDevice(&p->device);
    if (e != cudaSuccess) return cuda_fail(e);
    // behind the arrays: room for the (cos, sin) table of the projection epilogue, filled on the device when first used
    const size_t o_table = (blob.size() + 255) / 256 * 256;
    const size_t table_bytes = (size_t)p->total_rows * (p->head_dim / 2) * sizeof(float2);
    e = cudaMalloc(&p->dev_blob, o_table + std::max<size_t>(table_bytes, 16));
    if (e != cudaSuccess) { p->dev_blob = nullptr; return cuda_fail(e); }
    e = cudaMemcpy(p->dev_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return cuda_fail(e);
    char* base = static_cast<char*>(p->dev_blob);
    p->rope_table = reinterpret_cast<float2*>(base + o_table);
    DevicePlan& d = p->dev;
    d.cu_chunk = reinterpret_cast<const int32_t*>(base + o_cu);
    d.prefix_len = reinterpret_cast<const int32_t*>(base + o_pl);
    d.chunk_len = reinterpret_cast<const int32_t*>(base + o_cl);
    d.block_table = reinterpret_cast<const int32_t*>(base + o_bt);
    d.row_req = reinterpret_cast<const int32_t*>(base + o_rr);
    d.verify_items = reinterpret_cast<const WorkItem*>(base + o_vi);
    d.prefill_items = reinterpret_cast<const WorkItem*>(base + o_pi);
    d.merge_rows = reinterpret_cast<const MergeRow*>(base + o_mr);
    d.tile_units = reinterpret_cast<const uint32_t*>(base + o_tu);
    d.status = reinterpret_cast<int32_t*>(base + o_st);
    d.max_pages = p->max_pages;
    d.tree_mask = p->tree_mask.empty() ? nullptr : reinterpret_cast<const uint32_t*>(base + o_tm);
    d.num_heads = p->num_heads;
    d.num_kv_heads = p->num_kv_heads;
    d.group = p->num_heads / p->num_kv_heads;
    d.total_rows = p->total_rows;
    d.num_pages = p->num_pages;
    return HAT_OK;
}

static int check_call(const hat_cache_desc* cache, const hat_plan* plan) {
    if (!cache || !plan) return HAT_ERR_INVALID_ARG;
    if (plan->host_only) return HAT_ERR_INVALID_ARG;
    int st = check_cache_geometry(cache);
    if (st != HAT_OK) return st;
    if (cache->dtype != plan->dtype || cache->num_pages != plan->num_pages ||
        cache->num_kv_heads != plan->num_kv_heads || cache->head_dim != plan->head_dim)
        return HAT_ERR_INVALID_ARG;
    if (!cache->k_pool || !cache->v_pool) return HAT_ERR_INVALID_ARG;
    if (!aligned(cache->k_pool, 16) || !aligned(cache->v_pool, 16)) return HAT_ERR_INVALID_ARG;
    return HAT_OK;
}

static CacheView view_of(const hat_cache_desc* c) {
    return CacheView{c->k_pool, c->v_pool, c->stride_page, c->stride_token, c->stride_head};
}

}  // namespace hat

using namespace hat;

extern "C" {

const char* hat_status_string(int status) {
    switch (status) {
        case HAT_OK: return "ok";
        case HAT_ERR_INVALID_ARG: return "invalid argument";
        case HAT_ERR_UNSUPPORTED: return "unsupported configuration";
        case HAT_ERR_OUT_OF_RANGE: return "index out of range";
        case HAT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case HAT_ERR_CUDA: return "CUDA error";
        case HAT_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case HAT_ERR_TOO_LARGE: return "size exceeds a fixed maximum";
        case HAT_ERR_DEVICE_BOUNDS: return "device-side index check failed (debug build)";
        default: return "unknown status";
    }
}

int hat_version(void) { return HAT_VERSION; }
int hat_last_cuda_error(void) { return g_last_cuda_error; }
int64_t hat_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int hat_plan_create(const hat_cache_desc* cache, const hat_batch_desc* batch, hat_plan** out) {
    if (!out) return HAT_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cache || !batch) return HAT_ERR_INVALID_ARG;
    int st = check_cache_geometry(cache);
    if (st != HAT_OK) return st;
    const int R = batch->num_requests;
    if (R < 0 || batch->max_pages < 0 || batch->num_q_heads <= 0) return HAT_ERR_INVALID_ARG;
    if (batch->num_q_heads % cache->num_kv_heads != 0) return HAT_ERR_UNSUPPORTED;
    if (!batch->cu_chunk) return HAT_ERR_INVALID_ARG;
    if (R > 0 && (!batch->prefix_len || !batch->chunk_len)) return HAT_ERR_INVALID_ARG;
    if (batch->cu_chunk[0] != 0) return HAT_ERR_INVALID_ARG;

    // shapes
    int64_t total = 0;
    for (int r = 0; r < R; ++r) {
        if (batch->prefix_len[r] < 0 || batch->chunk_len[r] < 0) return HAT_ERR_INVALID_ARG;
        total += batch->chunk_len[r];
        if (batch->cu_chunk[r + 1] != total) return HAT_ERR_INVALID_ARG;
        if ((int64_t)batch->prefix_len[r] + batch->chunk_len[r] > (int64_t)INT32_MAX / 2) return HAT_ERR_TOO_LARGE;
    }
    if (total > INT32_MAX / 2) return HAT_ERR_TOO_LARGE;

    // block tables: long enough, inside the pool, and no page written by two requests
    std::vector<uint8_t> written(cache->num_pages > 0 ? cache->num_pages : 0, 0);
    for (int r = 0; r < R; ++r) {
        const int C = batch->chunk_len[r];
        if (C == 0) continue;
        const int N = batch->prefix_len[r] + C;
        const int need = (N + kPageSize - 1) / kPageSize;
        if (need > batch->max_pages) return HAT_ERR_OUT_OF_RANGE;
        if (!batch->block_table) return HAT_ERR_INVALID_ARG;
        const int32_t* row = batch->block_table + (int64_t)r * batch->max_pages;
        for (int j = 0; j < need; ++j)
            if (row[j] < 0 || row[j] >= cache->num_pages) return HAT_ERR_OUT_OF_RANGE;
        for (int j = batch->prefix_len[r] / kPageSize; j < need; ++j) {
            if (written[row[j]]) return HAT_ERR_OUT_OF_RANGE;
            written[row[j]] = 1;
        }
    }

    hat_plan* p = new (std::nothrow) hat_plan();
    if (!p) return HAT_ERR_INVALID_ARG;
    p->dtype = cache->dtype;
    p->num_pages = cache->num_pages;
    p->num_heads = batch->num_q_heads;
    p->num_kv_heads = cache->num_kv_heads;
    p->head_dim = cache->head_dim;
    p->max_pages = batch->max_pages;
    p->num_requests = R;
    p->total_rows = (int32_t)total;
    p->host_only = (batch->flags & HAT_PLAN_HOST_ONLY) != 0;
    p->device = -1;
    p->part_rows = 0;
    p->dev_blob = nullptr;
    p->timing = nullptr;
    p->num_verify_merge_rows = 0;
    p->ev_verify = nullptr;
    p->ev_done = nullptr;
    p->ev_table = nullptr;
    p->rope_table = nullptr;
    p->rope_theta = 0.f;
    p->table_stream = nullptr;
    p->last_stream = nullptr;
    p->has_last = false;
    p->side_sms = 0;
    p->aux_stream = nullptr;
    p->ev_fork = p->ev_join = nullptr;
    p->wait_cycles = 2000000000LL;
    p->withhold_next = 0;
    std::memset(&p->info, 0, sizeof p->info);
    std::memset(&p->dev, 0, sizeof p->dev);
    p->cu_chunk.assign(batch->cu_chunk, batch->cu_chunk + R + 1);
    p->prefix_len.assign(batch->prefix_len, batch->prefix_len + R);
    p->chunk_len.assign(batch->chunk_len, batch->chunk_len + R);
    if (batch->block_table && batch->max_pages > 0)
        p->block_table.assign(batch->block_table, batch->block_table + (int64_t)R * batch->max_pages);
    if (batch->tree_mask) p->tree_mask.assign(batch->tree_mask, batch->tree_mask + total);
    p->row_req.resize(total);
    for (int r = 0; r < R; ++r)
        for (int t = p->cu_chunk[r]; t < p->cu_chunk[r + 1]; ++t) p->row_req[t] = r;

    p->info.num_requests = R;
    p->info.total_rows = (int32_t)total;
    const int64_t d = p->head_dim, H = p->num_heads;
    for (int r = 0; r < R; ++r) {
        const int64_t C = p->chunk_len[r], P = p->prefix_len[r];
        if (C == 0) continue;
        p->info.attn_flops += 4 * d * H * (C * P + C * (C + 1) / 2);
        p->info.kv_read_bytes += 2 * (P + C) * p->num_kv_heads * d * 2;
    }

    int num_sms = 148;
    if (!p->host_only) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) { delete p; return cuda_fail(e); }
    }
    // the tcgen05 tile kernels need a pool layout a TMA descriptor can express (the CTA-pair one also head_dim 128)
    bool use_tc5 = true;
    if (const char* k = std::getenv("HAT_PREFILL_KERNEL"))
        if (std::strcmp(k, "mma") == 0) use_tc5 = false;
    if (use_tc5 && !p->host_only)
        use_tc5 = tc5_layout_supported(p->dtype, p->head_dim, p->num_pages, p->num_kv_heads, cache->stride_page,
                                       cache->stride_token, cache->stride_head);
    p->num_sms = num_sms;
    // Which tcgen05 tile kernel: the CTA-pair kernel (cta_group::2) shares every K/V tile between the two 128-row halves
    // of a 256-row unit and is the faster one when every unit fills both halves (and, for fp16, the batch is not small);
    // batches with 64- or 128-row chunks (half of a pair would idle) keep the one-CTA kernel.
    // HAT_PREFILL_KERNEL = tc5 | pair | mma overrides.
    int tile_kernel = use_tc5 ? 1 : 0;
    if (use_tc5 && p->head_dim == 128) {
        bool all_wide = true;
        int64_t wide_tiles = 0, wide_keys = 0;
        for (int r = 0; r < R; ++r) {
            const int C = p->chunk_len[r];
            if (C <= 16) continue;
            if (C % 256 != 0 && C % 256 <= 128) all_wide = false;
            for (int row0 = 0; row0 < C; row0 += 256)
                if (C - row0 > 128) { ++wide_tiles; wide_keys += p->prefix_len[r] + std::min(C, row0 + 256); }
        }
        // measured (chunks of 512 and 256 rows, 40 heads): for bf16 the pair kernel is the faster one at every batch size
        // (1 to 8 chunks: 9 to 26 %), for fp16 from about 1.5 units per SM on (equal at 160 units, 2.5 % at 240, 16 % at 320)
        // bf16: the units of more than 128 rows go to the pairs even when the batch also has narrower ones (those run on
        // single CTAs behind them: a ragged bf16 batch measured 0.298 + 0.118 ms that way against 0.49 on either kernel alone)
        // fp16: pairs pay off only for long units (prefix 4000: +16 %; 8 chunks of 512 at prefix 2000: +4.5 %, at 1000: -2 %; a ragged batch's wide units, ~2300 keys on average with many short ones: -3 %)
        const bool bf16 = p->dtype == HAT_DTYPE_BF16;
        const int64_t least = bf16 ? 1 : 3 * (int64_t)num_sms / 2;
        const bool long_units = bf16 || (wide_tiles > 0 && wide_keys / wide_tiles >= 2500);
        if ((all_wide || bf16) && long_units && wide_tiles > 0 && wide_tiles * p->num_heads >= least) tile_kernel = 3;
    }
    p->pair_takes_all = false;
    if (const char* k = std::getenv("HAT_PREFILL_KERNEL")) {
        if (use_tc5 && p->head_dim == 128 && std::strcmp(k, "pair") == 0) { tile_kernel = 3; p->pair_takes_all = true; }
        else if (use_tc5 && std::strcmp(k, "tc5") == 0) tile_kernel = 1;
    }
    schedule(p, num_sms, tile_kernel);
    // the streaming kernel takes its pages by TMA when a descriptor can be built for the pool layout
    bool stream_tma = true;
    if (const char* k = std::getenv("HAT_STREAM_KERNEL"))
        if (std::strcmp(k, "mma") == 0) stream_tma = false;
    if (stream_tma && !p->host_only)
        stream_tma = stream_layout_supported(p->dtype, p->head_dim, p->num_pages, p->num_kv_heads, cache->stride_page,
                                             cache->stride_token, cache->stride_head);
    p->info.stream_kernel = stream_tma ? 1 : 0;
    // launch-geometry limits: work items index gridDim.y (65535), partial rows and units are 32-bit
    if (p->verify_items.size() > 65535 || p->prefill_items.size() > 65535 || p->num_heads > 65535 ||
        p->part_rows > INT32_MAX / 2 || (int64_t)p->prefill_items.size() * p->num_heads > INT32_MAX / 2) {
        delete p;
        return HAT_ERR_TOO_LARGE;
    }

    if (!p->host_only) {
        st = upload(p);
        if (st != HAT_OK) { hat_plan_destroy(p); return st; }
        cudaError_t ee = cudaEventCreateWithFlags(&p->ev_verify, cudaEventDisableTiming);
        if (ee != cudaSuccess) { p->ev_verify = nullptr; hat_plan_destroy(p); return cuda_fail(ee); }
        ee = cudaEventCreateWithFlags(&p->ev_done, cudaEventDisableTiming);
        if (ee != cudaSuccess) { p->ev_done = nullptr; hat_plan_destroy(p); return cuda_fail(ee); }
        ee = cudaEventCreateWithFlags(&p->ev_table, cudaEventDisableTiming);
        if (ee != cudaSuccess) { p->ev_table = nullptr; hat_plan_destroy(p); return cuda_fail(ee); }
        // Optional throughput mode for a mixed batch on the tcgen05 path (HAT_SIDE_SMS = n > 0): see the launch
        // sequence.  Off by default: it finishes the whole step sooner but the decode-phase rows later.  The side
        // stream has the highest priority so that the tile CTAs are placed before the streaming kernel's many small
        // CTAs fill the SMs.
        if (!p->verify_items.empty() && !p->prefill_items.empty() && p->info.prefill_kernel == 1) {
            int side = env_int("HAT_SIDE_SMS", 0);
            side = std::max(0, std::min(side, p->num_sms - 8));
            if (side > 0) {
                int lo = 0, hi = 0;
                ee = cudaDeviceGetStreamPriorityRange(&lo, &hi);
                if (ee == cudaSuccess) ee = cudaStreamCreateWithPriority(&p->aux_stream, cudaStreamNonBlocking, hi);
                if (ee == cudaSuccess) ee = cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming);
                if (ee == cudaSuccess) ee = cudaEventCreateWithFlags(&p->ev_join, cudaEventDisableTiming);
                if (ee != cudaSuccess) { hat_plan_destroy(p); return cuda_fail(ee); }
                p->side_sms = side;
            }
        }
    }
    *out = p;
    return HAT_OK;
}

int hat_plan_get_info(const hat_plan* plan, hat_plan_info* out) {
    if (!plan || !out) return HAT_ERR_INVALID_ARG;
    *out = plan->info;
    return HAT_OK;
}

int hat_plan_workspace_bytes(const hat_plan* plan, size_t* out) {
    if (!plan || !out) return HAT_ERR_INVALID_ARG;
    *out = (size_t)plan->info.workspace_bytes;
    return HAT_OK;
}

int hat_plan_destroy(hat_plan* plan) {
    if (!plan) return HAT_OK;
    int st = HAT_OK;
    if (plan->timing) {
        for (cudaEvent_t ev : plan->timing->events) cudaEventDestroy(ev);
        delete plan->timing;
    }
    if (plan->ev_verify) cudaEventDestroy(plan->ev_verify);
    if (plan->ev_done) cudaEventDestroy(plan->ev_done);
    if (plan->ev_table) cudaEventDestroy(plan->ev_table);
    if (plan->ev_fork) cudaEventDestroy(plan->ev_fork);
    if (plan->ev_join) cudaEventDestroy(plan->ev_join);
    if (plan->aux_stream) cudaStreamDestroy(plan->aux_stream);
    if (plan->dev_blob) {
        cudaError_t e = cudaFree(plan->dev_blob);
        if (e != cudaSuccess) st = cuda_fail(e);
    }
    delete plan;
    return st;
}

int hat_kv_append(const hat_cache_desc* cache, const hat_plan* plan, const void* k_new, const void* v_new,
                  void* stream) {
    int st = check_call(cache, plan);
    if (st != HAT_OK) return st;
    if (plan->total_rows == 0) return HAT_OK;
    if (!k_new || !v_new || !aligned(k_new, 16) || !aligned(v_new, 16)) return HAT_ERR_INVALID_ARG;
    cudaError_t e = launch_kv_append(plan, view_of(cache), cache->k_pool, cache->v_pool, k_new, v_new,
                                     static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? HAT_OK : cuda_fail(e);
}

int hat_kv_append_rope(const hat_cache_desc* cache, const hat_plan* plan, const void* k_new, const void* v_new,
                       float theta, int interleaved, void* stream) {
    int st = check_call(cache, plan);
    if (st != HAT_OK) return st;
    if (!(theta > 1.f) || !std::isfinite(theta)) return HAT_ERR_INVALID_ARG;
    if (plan->total_rows == 0) return HAT_OK;
    if (!k_new || !v_new || !aligned(k_new, 16) || !aligned(v_new, 16)) return HAT_ERR_INVALID_ARG;
    const CacheView view = view_of(cache);
    cudaError_t e = launch_rope(plan, plan->num_kv_heads, theta, interleaved != 0, k_new, nullptr, &view, cache->k_pool,
                                cache->v_pool, v_new, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? HAT_OK : cuda_fail(e);
}

int hat_rope_q(const hat_plan* plan, const void* q, void* q_out, float theta, int interleaved, void* stream) {
    if (!plan || plan->host_only) return HAT_ERR_INVALID_ARG;
    if (!(theta > 1.f) || !std::isfinite(theta)) return HAT_ERR_INVALID_ARG;
    if (plan->total_rows == 0) return HAT_OK;
    if (!q || !q_out || !aligned(q, 16) || !aligned(q_out, 16)) return HAT_ERR_INVALID_ARG;
    cudaError_t e = launch_rope(plan, plan->num_heads, theta, interleaved != 0, q, q_out, nullptr, nullptr, nullptr, nullptr,
                                static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? HAT_OK : cuda_fail(e);
}

int hat_qkv_rope_append(const hat_cache_desc* cache, const hat_plan* plan, const void* x, int hidden, const void* w_qkv,
                        void* q_out, float theta, int interleaved, void* stream) {
    int st = check_call(cache, plan);
    if (st != HAT_OK) return st;
    if (theta > 0.f && (!(theta > 1.f) || !std::isfinite(theta))) return HAT_ERR_INVALID_ARG;
    if (hidden <= 0) return HAT_ERR_INVALID_ARG;
    if (hidden % 64 != 0 || (plan->head_dim != 64 && plan->head_dim != 128)) return HAT_ERR_UNSUPPORTED;
    if (plan->total_rows == 0) return HAT_OK;
    if (!x || !w_qkv || !q_out || !aligned(x, 16) || !aligned(w_qkv, 16) || !aligned(q_out, 16)) return HAT_ERR_INVALID_ARG;
    cudaError_t e = launch_qkv_gemm(plan, view_of(cache), cache->k_pool, cache->v_pool, x, hidden, w_qkv, q_out, theta,
                                    interleaved != 0, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? HAT_OK : cuda_fail(e);
}

// One attention step; the final rows go to `out` (fp32) or, when out16 is given, to out16 in the cache's 16-bit type.
static int run_attention(const hat_cache_desc* cache, const hat_plan* plan, const void* q, const void* k_new,
                         const void* v_new, float* out, void* out16, float* lse, float sm_scale, void* workspace,
                         size_t workspace_bytes, void* stream) {
    int st = check_call(cache, plan);
    if (st != HAT_OK) return st;
    if ((k_new == nullptr) != (v_new == nullptr)) return HAT_ERR_INVALID_ARG;
    if (plan->total_rows == 0) return HAT_OK;
    const void* dst = out16 ? out16 : static_cast<const void*>(out);
    if (!q || !dst || !lse) return HAT_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(dst, 16) || !aligned(lse, 16)) return HAT_ERR_INVALID_ARG;
    if (k_new && (!aligned(k_new, 16) || !aligned(v_new, 16))) return HAT_ERR_INVALID_ARG;
    const size_t need = (size_t)plan->info.workspace_bytes;
    if (need > 0) {
        if (!workspace || !aligned(workspace, 256)) return HAT_ERR_INVALID_ARG;
        if (workspace_bytes < need) return HAT_ERR_WORKSPACE_TOO_SMALL;
    }
    if (!(sm_scale > 0.f) || !std::isfinite(sm_scale)) sm_scale = 1.0f / std::sqrt((float)plan->head_dim);

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    // The plan's device state (unit counter, status word) serves one call at a time: a call on another stream than the
    // previous one is ordered behind it.
    // A call that is being captured into a graph cannot wait for (or be waited for through) an event of the world outside
    // the capture: there the caller orders the capturing stream behind the plan's earlier work before the capture begins.
    hat_plan* mplan = const_cast<hat_plan*>(plan);
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if ((e = cudaStreamIsCapturing(s, &cap)) != cudaSuccess) return cuda_fail(e);
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    if (!capturing && plan->has_last && plan->last_stream != s && (e = cudaStreamWaitEvent(s, plan->ev_done, 0)) != cudaSuccess)
        return cuda_fail(e);
    struct Done {
        hat_plan* p; cudaStream_t s; bool record;
        ~Done() { if (record && p->ev_done && cudaEventRecord(p->ev_done, s) == cudaSuccess) { p->last_stream = s; p->has_last = true; } }
    } done{mplan, s, !capturing};
    // optional event recorder: a start and an end event per slot (append, tile, streaming, merge)
    Timing* tm = plan->timing;
    int call = -1;
    if (tm && tm->next < tm->max_calls) call = tm->next++;
    auto mark = [&](int slot, int end) {
        if (call >= 0) cudaEventRecord(tm->events[((size_t)call * HAT_TIMING_SLOTS + slot) * 2 + end], s);
        if (call >= 0 && end) tm->launched[(size_t)call * HAT_TIMING_SLOTS + slot] = 1;
    };
    if (k_new) {
        mark(0, 0);
        e = launch_kv_append(plan, view_of(cache), cache->k_pool, cache->v_pool, k_new, v_new, s);
        if (e != cudaSuccess) return cuda_fail(e);
        mark(0, 1);
    }
    AttnArgs a;
    a.plan = plan->dev;
    a.cache = view_of(cache);
    a.q = q;
    a.out = out;
    a.out16 = out16;
    a.out16_bf16 = plan->dtype == HAT_DTYPE_BF16 ? 1 : 0;
    a.lse = lse;
    a.part_out = static_cast<float*>(workspace);
    const int64_t H = plan->num_heads, d = plan->head_dim;
    const size_t part_out_bytes = ((size_t)plan->part_rows * H * d * 4 + 255) / 256 * 256;
    a.part_lse = need ? reinterpret_cast<float*>(static_cast<char*>(workspace) + part_out_bytes) : nullptr;
    a.part_rows = plan->part_rows;
    a.scale_log2 = sm_scale * 1.4426950408889634f;
    a.wait_cycles = plan->wait_cycles;
    a.withhold = plan->withhold_next;
    a.tail_reset = 0;
    const_cast<hat_plan*>(plan)->withhold_next = 0;

    // Decode-phase (draft verification) requests first: their rows are final, and announced through the plan's event,
    // before the prompt chunks of the same batch are computed, so that they are not held back by them.
    const int n_vm = plan->num_verify_merge_rows, n_m = (int)plan->merge_rows.size();
    // Mixed batch: the tile kernel starts at once on all but side_sms SMs (own stream), the streaming kernel takes the
    // rest, and when it is done a second tile grid joins on the SMs it frees; both grids draw from one unit counter.
    const bool side = plan->side_sms > 0;
    if (side) {
        if ((e = cudaMemsetAsync(plan->dev.status + 1, 0, sizeof(int32_t), s)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventRecord(plan->ev_fork, s)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(plan->aux_stream, plan->ev_fork, 0)) != cudaSuccess) return cuda_fail(e);
        mark(1, 0);
        e = launch_attn_tc5(plan, a, plan->aux_stream, plan->num_sms - plan->side_sms, /*reset_counter=*/false);
        if (e == cudaSuccess) e = cudaEventRecord(plan->ev_join, plan->aux_stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (!plan->verify_items.empty()) {
        mark(2, 0);
        e = plan->info.stream_kernel == 1 ? launch_attn_stream(plan, a, s)
                                          : launch_attn_mma(plan, a, /*verify_class=*/true, s);
        if (e == cudaSuccess && n_vm > 0) e = launch_merge(plan, a, 0, n_vm, s);
        if (e != cudaSuccess) return cuda_fail(e);
        mark(2, 1);
    }
    if (plan->ev_verify && (e = cudaEventRecord(plan->ev_verify, s)) != cudaSuccess) return cuda_fail(e);
    if (side) {
        e = launch_attn_tc5(plan, a, s, plan->side_sms, /*reset_counter=*/false);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, plan->ev_join, 0);
        if (e != cudaSuccess) return cuda_fail(e);
        mark(1, 1);
    } else if (!plan->prefill_items.empty()) {
        mark(1, 0);
        if (plan->info.prefill_kernel == 3) {
            // units of more than 128 rows on CTA pairs, the others (if any) on single CTAs behind them
            e = launch_attn_pair(plan, a, s, plan->num_pair_units);
            if (e == cudaSuccess)
                e = launch_attn_tc5(plan, a, s, 0, true, plan->num_pair_units, -1, /*counter_word=*/3);
        } else {
            e = plan->info.prefill_kernel == 1 ? launch_attn_tc5(plan, a, s)
                                               : launch_attn_mma(plan, a, /*verify_class=*/false, s);
        }
        if (e != cudaSuccess) return cuda_fail(e);
        mark(1, 1);
    }
    if (n_m > n_vm) {
        mark(3, 0);
        e = launch_merge(plan, a, n_vm, n_m - n_vm, s);
        if (e != cudaSuccess) return cuda_fail(e);
        mark(3, 1);
    }
    return HAT_OK;
}


int hat_chunk_attention(const hat_cache_desc* cache, const hat_plan* plan, const void* q, const void* k_new,
                        const void* v_new, float* out, float* lse, float sm_scale, void* workspace,
                        size_t workspace_bytes, void* stream) {
    if (!out && plan && plan->total_rows > 0) return HAT_ERR_INVALID_ARG;
    return run_attention(cache, plan, q, k_new, v_new, out, nullptr, lse, sm_scale, workspace, workspace_bytes, stream);
}

int hat_chunk_attention_out16(const hat_cache_desc* cache, const hat_plan* plan, const void* q, const void* k_new,
                              const void* v_new, void* out16, float* lse, float sm_scale, void* workspace,
                              size_t workspace_bytes, void* stream) {
    if (!out16 && plan && plan->total_rows > 0) return HAT_ERR_INVALID_ARG;
    return run_attention(cache, plan, q, k_new, v_new, nullptr, out16, lse, sm_scale, workspace, workspace_bytes, stream);
}

int hat_plan_verify_event(const hat_plan* plan, void** event_out) {
    if (!plan || !event_out || plan->host_only) return HAT_ERR_INVALID_ARG;
    *event_out = plan->ev_verify;
    return HAT_OK;
}

int hat_plan_wait_verify(const hat_plan* plan) {
    if (!plan || plan->host_only || !plan->ev_verify) return HAT_ERR_INVALID_ARG;
    cudaError_t e = cudaEventSynchronize(plan->ev_verify);
    return e == cudaSuccess ? HAT_OK : cuda_fail(e);
}

int hat_plan_enable_timing(hat_plan* plan, int max_calls) {
    if (!plan || plan->host_only || max_calls <= 0 || max_calls > (1 << 20)) return HAT_ERR_INVALID_ARG;
    if (plan->timing) {
        for (cudaEvent_t ev : plan->timing->events) cudaEventDestroy(ev);
        delete plan->timing;
        plan->timing = nullptr;
    }
    Timing* tm = new (std::nothrow) Timing();
    if (!tm) return HAT_ERR_INVALID_ARG;
    tm->events.resize((size_t)max_calls * HAT_TIMING_SLOTS * 2);
    for (size_t i = 0; i < tm->events.size(); ++i) {
        cudaError_t e = cudaEventCreate(&tm->events[i]);
        if (e != cudaSuccess) {
            for (size_t j = 0; j < i; ++j) cudaEventDestroy(tm->events[j]);
            delete tm;
            return cuda_fail(e);
        }
    }
    tm->launched.assign((size_t)max_calls * HAT_TIMING_SLOTS, 0);
    tm->max_calls = max_calls;
    plan->timing = tm;
    return HAT_OK;
}

int hat_plan_read_timing(hat_plan* plan, float* ms, int capacity_calls, int* num_calls) {
    if (!plan || !ms || !num_calls || capacity_calls < 0 || !plan->timing) return HAT_ERR_INVALID_ARG;
    Timing* tm = plan->timing;
    const int n = std::min(tm->next, capacity_calls);
    for (int c = 0; c < n; ++c) {
        for (int sl = 0; sl < HAT_TIMING_SLOTS; ++sl) {
            float t = 0.f;
            if (tm->launched[(size_t)c * HAT_TIMING_SLOTS + sl]) {
                cudaEvent_t e0 = tm->events[((size_t)c * HAT_TIMING_SLOTS + sl) * 2];
                cudaEvent_t e1 = tm->events[((size_t)c * HAT_TIMING_SLOTS + sl) * 2 + 1];
                cudaError_t e = cudaEventSynchronize(e1);
                if (e == cudaSuccess) e = cudaEventElapsedTime(&t, e0, e1);
                if (e != cudaSuccess) return cuda_fail(e);
            }
            ms[(size_t)c * HAT_TIMING_SLOTS + sl] = t;
        }
    }
    *num_calls = n;
    tm->next = 0;
    std::fill(tm->launched.begin(), tm->launched.end(), 0);
    return HAT_OK;
}

int hat_plan_staging_bytes(const hat_plan* plan, size_t* out) {
    if (!plan || !out) return HAT_ERR_INVALID_ARG;
    const size_t T = plan->total_rows, H = plan->num_heads, Hkv = plan->num_kv_heads, d = plan->head_dim;
    const size_t q16 = (T * H * d * 2 + 255) / 256 * 256;
    const size_t kv16 = (T * Hkv * d * 2 + 255) / 256 * 256;
    const size_t out32 = (T * H * d * 4 + 255) / 256 * 256;
    const size_t lse32 = (T * H * 4 + 255) / 256 * 256;
    *out = q16 + 2 * kv16 + out32 + lse32;
    return HAT_OK;
}

int hat_chunk_attention_host(const hat_cache_desc* cache, const hat_plan* plan, const void* q_host,
                             const void* k_new_host, const void* v_new_host, float* out_host, float* lse_host,
                             float sm_scale, void* staging, size_t staging_bytes, void* workspace,
                             size_t workspace_bytes, void* stream) {
    int st = check_call(cache, plan);
    if (st != HAT_OK) return st;
    if (plan->total_rows == 0) return HAT_OK;
    if (!q_host || !k_new_host || !v_new_host || !out_host || !lse_host) return HAT_ERR_INVALID_ARG;
    size_t need = 0;
    hat_plan_staging_bytes(plan, &need);
    if (!staging || !aligned(staging, 256)) return HAT_ERR_INVALID_ARG;
    if (staging_bytes < need) return HAT_ERR_WORKSPACE_TOO_SMALL;
    const size_t T = plan->total_rows, H = plan->num_heads, Hkv = plan->num_kv_heads, d = plan->head_dim;
    const size_t act_bytes = T * H * d * 2, kv_bytes = T * Hkv * d * 2, out_bytes = T * H * d * 4, lse_bytes = T * H * 4;
    const size_t q16 = (act_bytes + 255) / 256 * 256, kv16 = (kv_bytes + 255) / 256 * 256, out32 = (out_bytes + 255) / 256 * 256;
    char* base = static_cast<char*>(staging);
    void* dq = base;
    void* dk = base + q16;
    void* dv = base + q16 + kv16;
    float* dout = reinterpret_cast<float*>(base + q16 + 2 * kv16);
    float* dlse = reinterpret_cast<float*>(base + q16 + 2 * kv16 + out32);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(dq, q_host, act_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(dk, k_new_host, kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(dv, v_new_host, kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e);
    st = hat_chunk_attention(cache, plan, dq, dk, dv, dout, dlse, sm_scale, workspace, workspace_bytes, stream);
    if (st != HAT_OK) return st;
    if ((e = cudaMemcpyAsync(out_host, dout, out_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(lse_host, dlse, lse_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    return HAT_OK;
}

int hat_last_device_status(const hat_plan* plan, void* stream, int* out) {
    if (!plan || !out || plan->host_only) return HAT_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, plan->dev.status, sizeof word, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(plan->dev.status, 0, 8 * sizeof word, s);     // status, unit counters, finished CTAs
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    *out = word == 0 ? HAT_OK : (word & 1) ? HAT_ERR_DEVICE_TIMEOUT : HAT_ERR_DEVICE_BOUNDS;
    return HAT_OK;
}

int hat_plan_set_wait_limit(hat_plan* plan, long long cycles, int withhold_next_call) {
    if (!plan || cycles < 0) return HAT_ERR_INVALID_ARG;
    plan->wait_cycles = cycles > 0 ? cycles : 2000000000LL;
    plan->withhold_next = withhold_next_call ? 1 : 0;
    return HAT_OK;
}

}  // extern "C"
