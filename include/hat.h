/*
 * hat.h -- C ABI of the HAT chunk-attention library (sm_100a).
 *
 * The library implements one step of a decoder layer of the cloud-side middle
 * submodel of HAT: for a ragged batch of requests coming from many end
 * devices, store the chunk's new keys/values in each request's paged KV cache
 * and compute causal attention of the chunk's query rows against that cache.
 * A chunk is either a prompt chunk (prompt chunking, Sec. 2.1 "Batched
 * Inference" and Sec. 3.3) or the short draft sequence sent up for
 * verification in a single inference step (Sec. 2.1 "Speculative Decoding",
 * Sec. 3.4).  Paging of the cache through a block table is what Sec. 4.1 calls
 * page attention.
 *
 * Conventions
 *   - Every function returns an int status: HAT_OK (0) or a negative error.
 *     No exception or abort crosses this boundary.
 *   - "host" / "device" on each pointer says where the memory must live.
 *   - The caller owns every buffer; the library owns only hat_plan objects.
 *   - hat_kv_append and hat_chunk_attention allocate nothing, never
 *     synchronise, and enqueue all work on the given CUDA stream
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - All argument errors are detected on the host before any launch.
 *   - Layout of packed activations (q, k_new, v_new, out): row-major
 *     [T][num_heads][head_dim], T = sum of chunk_len; request r owns rows
 *     cu_chunk[r] .. cu_chunk[r+1]-1.  lse is [T][num_heads].
 */
#ifndef HAT_H_
#define HAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HAT_VERSION 110   /* 110: hat_batch_desc gained tree_mask; grouped query heads; out16, rope entry points */

/* status codes */
#define HAT_OK                        0
#define HAT_ERR_INVALID_ARG          -1  /* null pointer, negative count, cu_chunk inconsistent with chunk_len */
#define HAT_ERR_UNSUPPORTED          -2  /* dtype, head_dim, page_size, head counts or strides outside what is built */
#define HAT_ERR_OUT_OF_RANGE         -3  /* page id outside the pool, table too short, page written by two requests */
#define HAT_ERR_WORKSPACE_TOO_SMALL  -4
#define HAT_ERR_CUDA                 -5  /* a CUDA runtime call failed; see hat_last_cuda_error */
#define HAT_ERR_DEVICE_TIMEOUT       -6  /* a bounded device-side wait gave up (reported by hat_last_device_status) */
#define HAT_ERR_TOO_LARGE            -7  /* a size exceeds a documented fixed maximum */
#define HAT_ERR_DEVICE_BOUNDS         -8  /* debug build only: a device-side index check failed (reported by hat_last_device_status) */

#define HAT_DTYPE_FP16 0
#define HAT_DTYPE_BF16 1

/* hat_batch_desc.flags */
#define HAT_PLAN_HOST_ONLY 1u   /* build and validate the plan but upload nothing (no CUDA call); such a plan
                                   can be inspected with hat_plan_get_info but not launched */

/*
 * Geometry of the KV cache (Sec. 2.1: keys and values of all previously
 * processed tokens; Sec. 4.1: paged).  Logical token p of a request lives in
 * page block_table[r][p / page_size], slot p % page_size.  Element (page, slot,
 * head, c) of a pool is at element offset
 *     page*stride_page + slot*stride_token + head*stride_head + c.
 * Strides are in elements and must be multiples of 8 (16-byte vectors);
 * head_dim is contiguous.  Two layouts are typical:
 *   paged      [page][head][slot][d]: stride_token=d, stride_head=page_size*d, stride_page=heads*page_size*d
 *   contiguous [token][head][d] with an identity block table:
 *              stride_token=heads*d, stride_head=d, stride_page=page_size*heads*d
 */
typedef struct hat_cache_desc {
    void*   k_pool;        /* device, 16-byte aligned; may be NULL for hat_plan_create */
    void*   v_pool;        /* device, 16-byte aligned; may be NULL for hat_plan_create */
    int32_t dtype;         /* HAT_DTYPE_FP16 | HAT_DTYPE_BF16 (q, k_new, v_new use the same type) */
    int32_t num_pages;     /* pages in each pool */
    int32_t page_size;     /* tokens per page; 16 is the only size built */
    int32_t num_kv_heads;  /* K/V heads; num_q_heads must be a multiple of it (equal in the paper's models, Sec. 4.1) */
    int32_t head_dim;      /* 64 or 128 */
    int32_t reserved;      /* 0 */
    int64_t stride_page;
    int64_t stride_token;
    int64_t stride_head;
} hat_cache_desc;

/*
 * One batch = one inference step over chunks from many devices (Sec. 2.1
 * continuous batching; Sec. 3.1).  All four arrays are HOST memory and are
 * copied by hat_plan_create (they may be freed afterwards).
 *   cu_chunk    [num_requests+1]  exclusive prefix sum of chunk_len, cu_chunk[0]=0
 *   prefix_len  [num_requests]    tokens already in the request's cache (>=0).  After a round in which
 *                                 drafts were rejected the caller simply passes the accepted length:
 *                                 stale slots beyond it are overwritten by the next append (Sec. 3.4)
 *   chunk_len   [num_requests]    rows of this chunk (>=0; 0 is a valid no-op)
 *   block_table [num_requests][max_pages] physical page ids; entries at or beyond
 *                                 ceil((prefix_len+chunk_len)/page_size) are ignored
 * Two optional extensions (the paper's models and HAT's own drafts need neither):
 *   num_q_heads = G * num_kv_heads   grouped query heads: query head h reads K/V head h / G; q, out and lse have
 *                                 num_q_heads heads, k_new, v_new and the pools num_kv_heads
 *   tree_mask   [T] or NULL       token-tree verification (the U-Medusa comparison system of Sec. 4.1; HAT's
 *                                 drafts are a linear sequence, Sec. 3.4 = NULL).  For a request with
 *                                 chunk_len <= 16, packed row t sees the whole cached prefix and chunk position c
 *                                 iff bit c of tree_mask[t] is set (bits at or above chunk_len are ignored; a row
 *                                 that sees nothing gets out = 0, lse = -inf).  Rows of longer chunks are prompt
 *                                 chunks: causal, their words are not read.
 */
typedef struct hat_batch_desc {
    int32_t        num_requests;
    int32_t        num_q_heads;
    int32_t        max_pages;
    uint32_t       flags;
    const int32_t* cu_chunk;
    const int32_t* prefix_len;
    const int32_t* chunk_len;
    const int32_t* block_table;
    const uint32_t* tree_mask;
} hat_batch_desc;

typedef struct hat_plan hat_plan;

/* What the host-side scheduler decided for a batch (for tests, tuning and reports). */
typedef struct hat_plan_info {
    int32_t num_requests;
    int32_t total_rows;          /* T */
    int32_t num_verify_requests; /* chunk_len in [1, 16]: split-KV streaming kernel */
    int32_t num_prefill_requests;/* chunk_len > 16: tile kernel */
    int32_t num_verify_items;    /* CTAs per head of the streaming kernel */
    int32_t num_prefill_items;   /* CTAs per head of the tile kernel */
    int32_t num_merge_rows;      /* rows whose result is merged from several key ranges */
    int32_t max_splits;          /* largest number of key ranges any request was cut into */
    int32_t verify_split_len;    /* tokens per key range, streaming kernel */
    int32_t prefill_split_len;   /* tokens per key range, tile kernel (0 = unsplit) */
    int32_t prefill_tile_rows;   /* query rows per CTA of the tile kernel */
    int32_t prefill_kernel;      /* 0 = mma.sync tile kernel, 1 = tcgen05 tile kernel (one CTA per unit), 3 = tcgen05 tile kernel by CTA pairs
                                    for the units of more than 128 rows (narrower units of the same batch: one CTA per unit) */
    int64_t workspace_bytes;
    int64_t attn_flops;          /* 4*d*H_q*sum_r [C_r*P_r + C_r*(C_r+1)/2] (causal count, also when a tree mask is given) */
    int64_t kv_read_bytes;       /* 2*sum_r (P_r+C_r)*H_kv*d*elem: every visible K and V row read once per K/V head */
    int32_t stream_kernel;       /* 0 = cp.async streaming kernel, 1 = TMA streaming kernel */
    int32_t reserved;
} hat_plan_info;

const char* hat_status_string(int status);
int         hat_version(void);

/* cudaError_t of the most recent failing CUDA call made by this library on the calling thread (0 if none). */
int         hat_last_cuda_error(void);

/* Number of kernels this library has launched in this process (all threads). */
int64_t     hat_launch_count(void);

/*
 * Validate a batch and schedule it (Sec. 2.1 "Batched Inference": the batch
 * mixes prefill chunks and decode-phase requests; cost follows the batched
 * token size).  Requests with chunk_len <= 16 take the split-KV streaming
 * path, longer chunks the tile path; long key ranges are cut so that every SM
 * has work, and rows cut into several ranges are merged afterwards.
 * Unless HAT_PLAN_HOST_ONLY is set the schedule is uploaded to the current
 * device (one cudaMalloc + one synchronous copy).  A plan can be reused for
 * every layer of the step and must be destroyed with hat_plan_destroy.
 * One call at a time per plan: the plan owns device state that an attention
 * call uses while it runs (the work counter of the persistent tile kernel, the
 * status word, the verify event, the timing recorder).  Calls that take the
 * same plan must therefore come from one host thread at a time, and the
 * library keeps them ordered on the device: a call given another stream than
 * the plan's previous call first makes that stream wait for the previous call
 * (cudaStreamWaitEvent on an event the plan owns).  To overlap two steps on
 * one GPU, create two plans.  A call that is captured into a CUDA graph
 * neither waits for nor records that event (a capture cannot depend on events
 * of the world outside it): the caller orders the capturing stream behind the
 * plan's earlier work before the capture begins, and replays of the graph
 * behind each other as for any graph.
 * Errors: INVALID_ARG, UNSUPPORTED, OUT_OF_RANGE, CUDA, TOO_LARGE (more than 65535 work items of one class,
 * i.e. key ranges or 256-row tiles, in one batch).  *out is NULL on error.
 */
int hat_plan_create(const hat_cache_desc* cache, const hat_batch_desc* batch, hat_plan** out);
int hat_plan_get_info(const hat_plan* plan, hat_plan_info* out);
int hat_plan_workspace_bytes(const hat_plan* plan, size_t* out);
int hat_plan_destroy(hat_plan* plan);   /* NULL is accepted */

/*
 * KV append (Sec. 2.1, KV cache).  For request r, chunk row i and head h the
 * 16-bit patterns k_new[cu_chunk[r]+i][h][:] and v_new[...] are stored,
 * bit-exactly, at logical token prefix_len[r]+i of the request's cache.  No
 * other slot of the pools is written.
 *   cache          geometry + device pools (both non-NULL)
 *   k_new, v_new   device, [T][heads][head_dim], 16-byte aligned
 */
int hat_kv_append(const hat_cache_desc* cache, const hat_plan* plan,
                  const void* k_new, const void* v_new, void* stream);

/*
 * Rotary position encoding fused into the append, and the same rotation for
 * the query rows.  The paper does not spell the position encoding out; its
 * models (Vicuna-7B/13B, Sec. 4.1) rotate query and key rows by their token
 * position in every decoder layer before the attention of Sec. 2.1 and cache
 * the rotated keys.  Chunk row i of request r has position p = prefix_len[r]+i;
 * pair c of a head (c = 0 .. head_dim/2-1) turns by the angle p * theta^(-2c/head_dim):
 *     (x_lo, x_hi) -> (x_lo cos - x_hi sin, x_hi cos + x_lo sin)
 * with (x_lo, x_hi) = (x[c], x[c+head_dim/2]), or (x[2c], x[2c+1]) when
 * `interleaved` is non-zero.  The rotation is computed in fp32 (the angle in
 * double) and rounded to the 16-bit type once.
 *   hat_kv_append_rope   k_new rows are rotated on their way into the K pool, v_new rows are stored as
 *                        they come: hat_kv_append with the rotation in between.  k_new, v_new as there.
 *   hat_rope_q           q_out[t][h][:] = rotated q[t][h][:] for all num_q_heads heads; q_out may be q.
 *                        Both device, [T][num_q_heads][head_dim], 16-byte aligned.
 *   theta                base of the angles (> 1; 10000 in the models of the paper)
 * hat_chunk_attention then takes q_out and no k_new/v_new.  Errors: INVALID_ARG, CUDA.
 */
int hat_kv_append_rope(const hat_cache_desc* cache, const hat_plan* plan, const void* k_new, const void* v_new,
                       float theta, int interleaved, void* stream);
int hat_rope_q(const hat_plan* plan, const void* q, void* q_out, float theta, int interleaved, void* stream);

/*
 * The projection in front of the attention module with the rotation and the
 * append in its epilogue (Sec. 2.1: Q = X W_Q, K = X W_K, V = X W_V, and the KV
 * cache keeps K and V of every token).  For packed row t and output feature f
 *     y[t][f] = sum_j x[t][j] * w_qkv[f][j]                 (fp32 accumulation)
 * with the features ordered  num_q_heads heads of q | num_kv_heads heads of k |
 * num_kv_heads heads of v, head_dim values each.  q and k heads are rotated by
 * the row's position exactly as hat_rope_q / hat_kv_append_rope do (theta <= 0:
 * no rotation), every value is rounded to the 16-bit type once, and
 *     q rows go to q_out[t][h][:]
 *     k and v rows go to logical token prefix_len[r]+i of request r's cache,
 *     as hat_kv_append would store them; no other slot of the pools is written.
 * hat_chunk_attention then takes q_out and no k_new/v_new.
 *   x          device, [T][hidden], the cache's 16-bit type, 16-byte aligned
 *   hidden     columns of x and of w_qkv; a multiple of 64
 *   w_qkv      device, [(num_q_heads + 2 num_kv_heads) * head_dim][hidden]: one
 *              row per output feature (the paper's W_Q | W_K | W_V, transposed)
 *   q_out      device, [T][num_q_heads][head_dim], 16-byte aligned
 * head_dim 64 or 128.  Nothing is owned or kept by the library.  Errors:
 * INVALID_ARG, UNSUPPORTED (hidden not a multiple of 64, other head_dim), CUDA;
 * a device-side wait that ran out shows in hat_last_device_status.  The table of
 * cosines and sines is kept with the plan and filled by the first call with a
 * given theta (one more small kernel in that call); a call captured into a CUDA
 * graph carries its own fill.  Like the attention calls, one call per plan at a time.
 */
int hat_qkv_rope_append(const hat_cache_desc* cache, const hat_plan* plan, const void* x, int hidden, const void* w_qkv,
                        void* q_out, float theta, int interleaved, void* stream);

/*
 * Chunk attention (Sec. 2.1 self-attention over the KV cache; Sec. 2.1 / 3.3
 * prompt chunks; Sec. 3.4 draft verification).  For packed row t = cu_chunk[r]+i
 * and head h, with g = prefix_len[r]+i and keys/values j = 0..g read through
 * the block table:
 *     s_j = sm_scale * <q[t][h], K_j[h]>
 *     out[t][h][:] = sum_j softmax(s)_j * V_j[h][:]        (fp32)
 *     lse[t][h]    = ln sum_j exp(s_j)                     (fp32, natural log)
 * The chunk's own K/V must be in the cache: either call hat_kv_append first, or
 * pass k_new/v_new here (both non-NULL), which performs the same append on
 * `stream` before attending.
 *   q                device [T][heads][head_dim], same dtype as the cache, 16-byte aligned
 *   out, lse         device fp32, 16-byte aligned
 *   sm_scale         <= 0 or NaN selects 1/sqrt(head_dim)
 *   workspace        device, 256-byte aligned, at least hat_plan_workspace_bytes; may be NULL if that is 0.
 *                    Calls on different plans that may overlap must use different workspaces (calls on one
 *                    plan never overlap, see hat_plan_create).
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, CUDA.
 */
int hat_chunk_attention(const hat_cache_desc* cache, const hat_plan* plan, const void* q,
                        const void* k_new, const void* v_new,
                        float* out, float* lse, float sm_scale,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same step with `out` in the cache's 16-bit type (what the output
 * projection of the decoder layer, Sec. 2.1, consumes): the fp32 result is
 * rounded to nearest once, when a final row is written; partial rows in the
 * workspace and lse stay fp32.  The paper fixes no output precision; this
 * entry point is an addition next to the fp32 one.
 *   out16            device [T][num_q_heads][head_dim], cache dtype, 16-byte aligned
 * All other arguments and errors as hat_chunk_attention.
 */
int hat_chunk_attention_out16(const hat_cache_desc* cache, const hat_plan* plan, const void* q,
                              const void* k_new, const void* v_new,
                              void* out16, float* lse, float sm_scale,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same step for a caller whose activations live in HOST memory (pinned
 * memory makes the copies asynchronous).  Copies q, k_new, v_new to `staging`,
 * appends, attends, copies out and lse back, all on `stream`, and returns
 * without synchronising: the host results are valid once the stream is.
 *   q_host, k_new_host, v_new_host   host [T][heads][head_dim] 16-bit
 *   out_host [T][heads][head_dim], lse_host [T][heads]   host fp32
 *   staging        device, 256-byte aligned, >= hat_plan_staging_bytes
 *   workspace      as for hat_chunk_attention
 */
int hat_plan_staging_bytes(const hat_plan* plan, size_t* out);
int hat_chunk_attention_host(const hat_cache_desc* cache, const hat_plan* plan,
                             const void* q_host, const void* k_new_host, const void* v_new_host,
                             float* out_host, float* lse_host, float sm_scale,
                             void* staging, size_t staging_bytes,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Optional per-kernel timing for benchmarks (not part of the method).  After
 * hat_plan_enable_timing, each of the next max_calls calls of
 * hat_chunk_attention / hat_chunk_attention_host on this plan records CUDA
 * events on its stream around each kernel it launches (this creates
 * 8*max_calls events once, here, not in the attention call).
 * hat_plan_read_timing waits for the recorded events and writes, per recorded
 * call, HAT_TIMING_SLOTS durations in milliseconds: [0] KV append, [1] tile
 * (prefill-class) attention, [2] streaming (verify-class) attention with the
 * merge of its rows, [3] merge of tile-class rows;
 * 0 where a kernel was not launched.  It then rewinds the recorder.
 *   ms          host, [capacity_calls][HAT_TIMING_SLOTS]
 *   num_calls   host, out: calls written
 */
#define HAT_TIMING_SLOTS 4
int hat_plan_enable_timing(hat_plan* plan, int max_calls);
int hat_plan_read_timing(hat_plan* plan, float* ms, int capacity_calls, int* num_calls);

/*
 * Decode-phase requests are not held back by prompt chunks (Sec. 2.1 "Batched
 * Inference": long prefills delay the decode requests of the same batch; Sec.
 * 3.3).  hat_chunk_attention computes the streaming-class chunks (draft
 * verification, chunk_len <= 16) first and records an event owned by the plan
 * as soon as their out/lse rows are final, before the tile kernel for the
 * prompt chunks of the same batch starts.
 *   hat_plan_verify_event   the cudaEvent_t (as void*), e.g. for cudaStreamWaitEvent on the caller's own stream
 *                           that returns those rows to the devices; it is re-recorded by every attention call
 *   hat_plan_wait_verify    blocks the host until the event of the latest call has occurred
 */
int hat_plan_verify_event(const hat_plan* plan, void** event_out);
int hat_plan_wait_verify(const hat_plan* plan);

/*
 * Read and clear the device-side status word of a plan (synchronises
 * `stream`).  *out is HAT_OK, HAT_ERR_DEVICE_BOUNDS (only a library built with
 * -DHAT_DEBUG_BOUNDS checks: a block-table column, page id, ring slot, TMEM column or output row was out of range;
 * the access was skipped or clamped, nothing trapped), or HAT_ERR_DEVICE_TIMEOUT if a bounded wait
 * inside a kernel gave up since the word was last read; the results of the
 * calls in between are then undefined, but the kernels have exited normally
 * and the context stays usable.
 */
int hat_last_device_status(const hat_plan* plan, void* stream, int* out);

/*
 * Failure detection of the tcgen05 kernels (tile attention, projection).
 * Every wait inside them (on a TMA transfer, on the tensor pipe, on another
 * warp or the other CTA of a pair) is bounded by `cycles` SM clock cycles (0
 * selects the default of 2e9, about a second); a wait that runs out sets the
 * status word above, tells the other warps of its CTA (and the other CTA of
 * its pair) to stop, and the CTA releases its tensor memory and exits.
 * withhold_next_call != 0 is a self test of that path: in the next
 * hat_chunk_attention or hat_qkv_rope_append call on this plan, whichever
 * comes first, every CTA that loads skips one of its own transfers, so that
 * a wait does run out within the bound; that call's results are undefined.
 * Nothing faults or hangs.
 */
int hat_plan_set_wait_limit(hat_plan* plan, long long cycles, int withhold_next_call);

/*
 * Cloud-side control plane (host only; no CUDA call).  It closes the loop the
 * paper describes around the attention step: per round the cloud records the
 * batched token size and the in-cloud computation delay, keeps moving
 * averages of them (Sec. 3.2, Eq. 1-2, alpha = 0.8 in the paper's
 * experiments), and from the predicted delay g(.) derives each device's
 * prompt chunk size (Sec. 3.3, Eq. 3) and its number of parallel-drafting
 * steps (Sec. 3.5, Eq. 6).
 *   g(.) is kept on a uniform grid of `num_bins` token sizes `bin_width` apart;
 *   an observation updates the grid point nearest to the smoothed token size;
 *   g is linear between observed points, continues with the outermost slope
 *   beyond them, is constant with one observed point and 0 with none.  The
 *   first observation of any moving average is taken as is.
 * hat_ctrl_observe(mu_hat, eta_hat)       Eq. 1 then Eq. 2 (tokens, seconds)
 * hat_ctrl_device_observe(i, gamma, beta_up, beta_down)   moving averages of device i's drafting delay per step
 *                                         (seconds) and up/down bandwidths (bytes per second)
 * hat_ctrl_chunk_size(i, A, P, x_min, x_max, &X)   smallest integer X in [x_min, x_max] with
 *                                         X*A/beta_up >= (g(mu) + g(mu + X)) / P   (A = bytes of hidden state per
 *                                         token, P = pipeline length); x_max if there is none
 * hat_ctrl_parallel_draft_steps(i, n, A, &lambda)  floor((n*A/beta_up + g(mu) + n*A/beta_down) / gamma) for a draft
 *                                         sequence of n tokens
 * Errors: INVALID_ARG (null, out-of-range device, device never observed, non-positive rates, alpha outside [0,1]).
 */
typedef struct hat_ctrl hat_ctrl;
int hat_ctrl_create(double alpha, double bin_width, int num_bins, int max_devices, hat_ctrl** out);
int hat_ctrl_destroy(hat_ctrl* ctrl);   /* NULL is accepted */
int hat_ctrl_observe(hat_ctrl* ctrl, double mu_hat, double eta_hat);
int hat_ctrl_mu(const hat_ctrl* ctrl, double* out);
int hat_ctrl_predict(const hat_ctrl* ctrl, double tokens, double* out);
int hat_ctrl_device_observe(hat_ctrl* ctrl, int device, double gamma_hat, double beta_up_hat, double beta_down_hat);
int hat_ctrl_device_state(const hat_ctrl* ctrl, int device, double* gamma, double* beta_up, double* beta_down);
int hat_ctrl_chunk_size(const hat_ctrl* ctrl, int device, double bytes_per_token, int pipeline_length,
                        int x_min, int x_max, int* out);
int hat_ctrl_parallel_draft_steps(const hat_ctrl* ctrl, int device, int draft_len, double bytes_per_token, int* out);

/*
 * Streaming attention for callers that must not allocate.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)
 *
 * Who needs it: a serving loop that runs under CUDA-graph capture or inside a
 * framework that has handed the whole device heap to its own allocator cannot
 * call cudaMalloc, so it can neither create a hat_plan nor obtain the workspace
 * hat_chunk_attention wants for its split-KV partial results.  This entry point
 * computes the same out/lse as hat_chunk_attention for short chunks
 * (chunk_len <= max_chunk_len <= 16, i.e. draft verification and decode) and
 * calls no cudaMalloc / cudaFree or any allocating routine.  Its partial
 * results go to a fixed array of HAT_STATIC_SCRATCH_BYTES that is part of the
 * library's device code: every GPU that loads the library holds that much
 * memory until the process exits.
 *
 * Differences from hat_chunk_attention:
 *   - cu_chunk, prefix_len, chunk_len, block_table are DEVICE arrays (same
 *     shapes and meaning as in hat_batch_desc); the host cannot inspect them,
 *     so they are not validated.  Instead every lookup is clamped: a negative
 *     prefix_len counts as 0, chunk_len is cut to [0, max_chunk_len] (rows at or
 *     beyond max_chunk_len are not computed and keep what out/lse held),
 *     prefix_len + chunk_len is cut to max_pages * 16, block-table columns stay
 *     inside the request's row and page ids inside the pool: wrong descriptor
 *     values give wrong rows, not reads outside the arrays.  cu_chunk is
 *     trusted: it addresses q, out and lse.  hat_static_key_range (a pure host
 *     function) returns the clamped lengths and the key range of each split.
 *   - No append: the chunk's K/V must already be in the cache.
 *   - Every request is cut into HAT_STATIC_SPLITS key ranges of equal length.
 *   - Limit: num_requests * HAT_STATIC_SPLITS * max_chunk_len * heads * (head_dim+1) * 4 bytes
 *     (rounded up to 256) must fit in HAT_STATIC_SCRATCH_BYTES, and
 *     num_requests * HAT_STATIC_SPLITS <= 65535; otherwise HAT_ERR_TOO_LARGE
 *     and nothing is launched.
 *   - The first call on each device looks up the device address of the scratch
 *     array (cudaGetSymbolAddress, with that device current); make that first
 *     call outside any stream capture.
 *   - All calls on one GPU share the scratch array, which keeps the previous
 *     call's partial results; each call overwrites every slot it later reads,
 *     so nothing has to be cleared, but two calls that overlap in time on the
 *     same GPU (different streams) race on it.  Serialise them.
 * Errors: INVALID_ARG, UNSUPPORTED, TOO_LARGE, CUDA (the cudaError_t is then
 * available from hat_last_cuda_error on the calling thread).
 */
#define HAT_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
#define HAT_STATIC_SPLITS 8
int hat_verify_attention_static(const hat_cache_desc* cache, int num_requests, int num_q_heads,
                                int max_chunk_len, int max_pages,
                                const int32_t* cu_chunk, const int32_t* prefix_len,      /* device */
                                const int32_t* chunk_len, const int32_t* block_table,    /* device */
                                const void* q, float* out, float* lse,                   /* device */
                                float sm_scale, void* stream);
/* Host only, no CUDA call: what split `split` (0 .. HAT_STATIC_SPLITS-1) of a request with these (unvalidated)
 * lengths computes in hat_verify_attention_static: the clamped prefix, the rows computed and the keys
 * [kv_begin, kv_end) of the split.  Null outputs are skipped.  INVALID_ARG for max_chunk_len outside 1..16,
 * max_pages <= 0 or a split outside the range.  (No counterpart in the paper.) */
int hat_static_key_range(int prefix_len, int chunk_len, int max_chunk_len, int max_pages, int split,
                         int* prefix, int* rows, int* kv_begin, int* kv_end);

#ifdef __cplusplus
}
#endif
#endif /* HAT_H_ */
