/*
 * tokenscale.h -- C ABI of the mixed paged-attention step of a Convertible Decoder.
 *
 * TokenScale (arXiv 2512.03416) lets a decoder GPU absorb the prefill of burst requests:
 * every iteration the decoder runs a batch made of its ongoing single-token decode
 * requests plus (a chunk of) one prefill task, bounded by a profiled "chunk size"
 * (Sec. 3.4 "Convertible Decoder", Sec. 4.4 "SLO-aware restricted chunked prefill", Eq. 5).
 * This library is the attention part of that iteration: grouped-query attention over a
 * paged KV cache (Sec. 2.1: prefill builds the KV cache of all input tokens, decode reuses
 * it and adds one token per iteration), the append of the step's new K/V into cache pages,
 * the page bookkeeping, and the per-step token counts that feed Token Velocity (Sec. 3.2, Eq. 1).
 *
 * All kernels are CUDA for sm_100a. There is no CPU fallback: a call that has to launch
 * work returns TS_ERR_CUDA when no usable device is present.
 *
 * ---------------------------------------------------------------------------------------
 * Data layout (frozen; everything is little endian, bf16 = upper 16 bits of an IEEE fp32)
 *
 *   KV pool (device, owned by the caller), bf16, index order
 *        pool[page][kv][head][slot][d]
 *        page in [0, n_pages), kv in {0 = K, 1 = V}, head in [0, n_kv_heads),
 *        slot in [0, page_size), d in [0, head_dim)
 *   element offset = (((page*2 + kv)*n_kv_heads + head)*page_size + slot)*head_dim + d
 *   One page therefore holds page_size tokens of every KV head, K and V together;
 *   a (page, kv, head) tile is page_size*head_dim contiguous elements.
 *
 *   Token t (0-based position in its request) lives in page block_table[t / page_size],
 *   slot t % page_size. Slots that hold no token yet are never read or written.
 *
 *   Step tensors (device): q and out are [N, n_q_heads, head_dim] bf16, k_new and v_new are
 *   [N, n_kv_heads, head_dim] bf16, where N = sum of q_len over the rows of the step and the
 *   rows' tokens are concatenated in row order. Query head h uses KV head h / (n_q_heads / n_kv_heads).
 *
 * What a step computes. For row r with ctx = ctx_len[r] cached tokens and q_len[r] new tokens,
 * new token i (0 <= i < q_len[r]) is appended at position ctx + i and then attends to the
 * positions 0 .. ctx + i of its own request (all cached context, plus the causal part of the chunk):
 *        s_j = scale * <q, K_j>,   p_j = exp(s_j - max_j s_j),   out = sum_j p_j V_j / sum_j p_j
 * with fp32 accumulation and a bf16 (round-to-nearest-even) result.
 * ---------------------------------------------------------------------------------------
 */
#ifndef TOKENSCALE_H_
#define TOKENSCALE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Return codes. Every entry point returns one of these; nothing throws across the ABI. */
enum {
  TS_OK = 0,
  TS_ERR_INVALID = -1,        /* null pointer, bad handle, bad slot, inconsistent lengths     */
  TS_ERR_NO_PAGES = -2,       /* the free list cannot cover the request (nothing was taken)   */
  TS_ERR_NO_SLOT = -3,        /* max_requests requests are already live                       */
  TS_ERR_TABLE_SHORT = -4,    /* a row's block table does not cover ctx_len + q_len tokens    */
  TS_ERR_BUDGET = -5,         /* prefill tokens + decode rows of the step exceed chunk_size   */
  TS_ERR_CUDA = -6,           /* a CUDA runtime call failed (ts_last_cuda_error has the code) */
  TS_ERR_DEVICE_TIMEOUT = -7, /* a bounded wait inside a kernel ran out                       */
  TS_ERR_UNSUPPORTED = -8,    /* shape outside what the kernels are built for                 */
  TS_ERR_WORKSPACE = -9       /* kv_pool or workspace smaller than ts_pool_bytes/ts_workspace_bytes */
};

typedef struct ts_ctx ts_ctx; /* opaque; host memory; one thread and one stream at a time */

/*
 * Static description of one decoder instance's attention layer and KV pool.
 * Supported shapes: head_dim in {64, 128}; page_size == 16; n_q_heads a multiple of
 * n_kv_heads with a group size n_q_heads / n_kv_heads <= 16.
 */
typedef struct {
  int32_t n_q_heads;          /* Hq                                                            */
  int32_t n_kv_heads;         /* Hkv                                                           */
  int32_t head_dim;           /* D                                                             */
  int32_t page_size;          /* tokens per page; 16                                           */
  int32_t n_pages;            /* pages in the pool                                             */
  int32_t max_requests;       /* request slots (rows of the block table)                       */
  int32_t max_pages_per_req;  /* columns of the block table                                    */
  int32_t chunk_size;         /* Sec. 4.4: largest allowed (prefill tokens + decode batch size)
                                 of one step; 0 disables the check                             */
  int32_t reserved_pages;     /* Eq. 6: pages only ts_alloc_pages(..., for_prefill=1) may take */
  int32_t decode_split_tokens;/* keys per split of a decode row; 0 = library default; rounded
                                 up to a multiple of 64                                        */
  int32_t mixed_prefill_ctas; /* CTAs of the mixed attention kernel that only take prefill tiles
                                 while the other CTAs stream the decode rows first (Sec. 3.4:
                                 the decoder absorbs prefill work next to its decode batch);
                                 0 = the library's cost model decides per step; < 0 = prefill
                                 tiles and decode rows run as two launches, one after the other */
  float softmax_scale;        /* 0 => 1/sqrt(head_dim)                                         */
  int32_t device;             /* CUDA device ordinal that owns kv_pool and workspace           */
  uint64_t alloc_shuffle_seed;/* 0: free list hands out pages 0,1,2,...; otherwise the initial
                                 free list is a seeded permutation (scattered pages)           */
  void* kv_pool;              /* DEVICE, ts_pool_bytes() bytes, caller-owned, 256-byte aligned */
  size_t kv_pool_bytes;
  void* workspace;            /* DEVICE scratch, ts_workspace_bytes() bytes, caller-owned,
                                 256-byte aligned; holds the device block table, the step
                                 metadata, split partials and the host-buffer staging area     */
  size_t workspace_bytes;
  int64_t wait_limit_cycles;  /* limit of every bounded wait inside the kernels, in GPU clock
                                 cycles; 0 = the library's default (about one second)          */
  int32_t debug_flags;        /* 0, or TS_DEBUG_* bits (testing the failure path, see below)   */
} ts_config;

/*
 * Debug flags (the paper has no counterpart). TS_DEBUG_LOSE_APPEND_ARRIVAL makes the launch-wide
 * barrier after the KV append of a step with prefill rows wait for one thread block more than the
 * launch has, so that this wait runs out: every block then raises TS_DEV_TIMEOUT after
 * wait_limit_cycles and carries on (all blocks did arrive, so the step's output is still valid).
 * It exists so that the time-out path can be exercised without a fault: ts_create refuses it
 * (TS_ERR_INVALID) unless 0 < wait_limit_cycles <= 50,000,000 (about 25 ms), so it can never spin
 * for the default second.
 */
enum { TS_DEBUG_LOSE_APPEND_ARRIVAL = 1 };

/* Sizes the caller must allocate. Only the shape fields of cfg are read. 0 on a bad shape. */
size_t ts_pool_bytes(const ts_config* cfg);
size_t ts_workspace_bytes(const ts_config* cfg);

/*
 * ts_create: builds the host bookkeeping (free list, block tables, counters). Makes no CUDA
 * call; kv_pool/workspace may be NULL for host-only use (allocator, planning), in which case
 * calls that launch return TS_ERR_CUDA. The pool contents are not touched.
 * ts_destroy: frees host memory and the library's pinned staging buffers; never the pool.
 */
int ts_create(const ts_config* cfg, ts_ctx** out);
int ts_destroy(ts_ctx* ctx);

/*
 * Requests (Sec. 4.1: the gateway records each request's input length and a predicted
 * output length). ts_request_add takes a free slot (TS_ERR_NO_SLOT if none) and records the
 * lengths; no pages are taken yet. expected_output_len is informational (<= 0 if unknown).
 */
int ts_request_add(ts_ctx* ctx, int64_t req_id, int32_t prompt_len, int32_t expected_output_len,
                   int32_t* slot_out);

/*
 * ts_alloc_pages: grow the slot's block table so that it covers total_tokens tokens
 * (ceil(total_tokens / page_size) pages). All or nothing: on TS_ERR_NO_PAGES or
 * TS_ERR_TABLE_SHORT (more than max_pages_per_req) the table is unchanged. for_prefill != 0
 * may dip into the reserved_pages held back for absorbed prefill work (Eq. 6).
 * Never shrinks. Host only; the device copy of the table is refreshed by the next step.
 */
int ts_alloc_pages(ts_ctx* ctx, int32_t slot, int32_t total_tokens, int32_t for_prefill);

/*
 * ts_block_table: borrowed, read-only host view of a slot's page list, its page count and the
 * number of tokens currently cached. Valid until the next call that changes this slot.
 * Any of the out pointers may be NULL.
 */
int ts_block_table(ts_ctx* ctx, int32_t slot, const int32_t** pages_out, int32_t* n_pages_out,
                   int32_t* n_tokens_out);

/*
 * ts_block_table_set: replace a slot's page list by the given pages (each in [0, n_pages),
 * not owned by another slot, no duplicates; pages previously held by the slot return to the
 * free list first). Lets a caller or a test lay a request out on chosen pages.
 */
int ts_block_table_set(ts_ctx* ctx, int32_t slot, const int32_t* pages, int32_t n_pages);

/*
 * ts_request_free: the request completed. Its pages return to the free list and its length
 * L_r (tokens cached = prompt + generated) is added to released_tokens: Eq. 1 counts Decode
 * Velocity as tokens *released* per unit time. The slot becomes reusable.
 */
int ts_request_free(ts_ctx* ctx, int32_t slot);

/* ts_request_set_len: overwrite the slot's cached-token count (<= tokens its table covers).
 * Used to declare context that was written into the pool by other means, or to rewind. */
int ts_request_set_len(ts_ctx* ctx, int32_t slot, int32_t n_tokens);

/* Step flags */
enum {
  TS_STEP_KEEP_LEN = 1,  /* do not advance the slots' cached lengths: the same step can be
                            issued again and rewrites the same bytes (used for timing)       */
  TS_STEP_HOST_ASYNC = 2 /* ts_mixed_step_host only: return once everything is enqueued      */
};

/*
 * One iteration's batch (Sec. 4.4): rows with q_len == 1 are decode requests, rows with
 * q_len > 1 are prefill chunks. ctx_len[r] must equal the library's cached length of slot[r]
 * and the slot's table must already cover ctx_len + q_len tokens (ts_alloc_pages), otherwise
 * the call fails on the host and launches nothing. A slot may appear once per step.
 * q/k_new/v_new/out: see "Step tensors" above; 16-byte aligned.
 */
typedef struct {
  int32_t n_rows;
  int32_t flags;
  const int32_t* slot;    /* HOST [n_rows] */
  const int32_t* q_len;   /* HOST [n_rows], >= 1 */
  const int32_t* ctx_len; /* HOST [n_rows], >= 0 */
  const void* q;          /* DEVICE bf16 [N, Hq, D]  (ts_mixed_step_host: HOST) */
  const void* k_new;      /* DEVICE bf16 [N, Hkv, D] (ts_mixed_step_host: HOST) */
  const void* v_new;      /* DEVICE bf16 [N, Hkv, D] (ts_mixed_step_host: HOST) */
  void* out;              /* DEVICE bf16 [N, Hq, D]  (ts_mixed_step_host: HOST) */
} ts_step;

/*
 * ts_alloc_step: ts_alloc_pages for every row of a step in one call -- grows slot[r]'s table to
 * ctx_len[r] + q_len[r] tokens (rows with q_len > 1 count as prefill work and may use the reserved
 * pages). Stops at the first row that cannot be served and returns its error; rows before it
 * keep their new pages. Only slot, q_len and ctx_len of the step are read.
 */
int ts_alloc_step(ts_ctx* ctx, const ts_step* step);

/*
 * ts_kv_append: write the step's new K/V into the rows' pages (Sec. 2.1) and, unless
 * TS_STEP_KEEP_LEN, advance the cached lengths. q and out are ignored. Asynchronous on
 * cuda_stream (a cudaStream_t passed as void*; NULL = legacy default stream). Also the way
 * to load pre-existing context: one row with ctx_len = 0 and q_len = the context length.
 * Not subject to chunk_size and not counted as a step.
 */
int ts_kv_append(ts_ctx* ctx, const ts_step* step, void* cuda_stream);

/*
 * ts_mixed_step: the decoder iteration. Appends, then runs split-KV decode attention for the
 * 1-token rows and tiled causal attention for the prefill-chunk rows, merges the splits, and
 * writes out. Everything is enqueued on cuda_stream; the call does not synchronise.
 * Enforces Sec. 4.4's budget: (prefill tokens + decode rows) <= chunk_size, else TS_ERR_BUDGET.
 * Updates the Token Velocity counters. An empty step (n_rows == 0) is TS_OK and launches nothing.
 * A step with prefill rows runs as one kernel that fills every SM and whose thread blocks wait
 * for one another (bounded waits): steps of different contexts on the same device must not
 * overlap on the GPU -- issue them to one stream, or order the streams with events. If they do
 * overlap, the waits run out, the step's output is wrong and ts_last_device_status reports
 * TS_DEV_TIMEOUT; nothing hangs.
 */
int ts_mixed_step(ts_ctx* ctx, const ts_step* step, void* cuda_stream);

/*
 * ts_mixed_step_host: same step with q, k_new, v_new, out in HOST memory (pinned memory makes
 * the copies asynchronous). Copies the inputs into a staging set of the workspace on the
 * context's own upload stream, runs the step on cuda_stream, copies out back on the context's
 * download stream, makes cuda_stream wait for that copy, and waits for cuda_stream: on return
 * out is valid. N <= chunk_size required (the staging sets are sized by chunk_size; chunk_size
 * must be > 0). The paper's decoder receives its inputs from the layers before attention, on the
 * device; this entry point serves callers and measurements that start from host memory.
 * With TS_STEP_HOST_ASYNC the call returns once everything is enqueued and cuda_stream does not
 * wait for the download either. The inputs are read at any time from the call on, so they must
 * be final when it is made and stay unchanged, and out untouched, until cuda_stream has passed
 * a ts_host_fence issued after the call (then synchronise the stream or record an event), or
 * until a later ts_mixed_step_host without the flag has returned. Three staging sets take
 * turns: the uploads and kernels of the following steps overlap this step's download, so a
 * sequence of such calls is bound by the slowest of upload, kernels and download instead of by
 * their sum. A failed call has enqueued nothing that writes out.
 */
int ts_mixed_step_host(ts_ctx* ctx, const ts_step* step, void* cuda_stream);

/*
 * ts_host_fence (the paper has no counterpart): makes cuda_stream wait, on the device, for the
 * downloads of every ts_mixed_step_host call issued so far; the call itself does not block.
 * TS_OK when no host step has been issued.
 */
int ts_host_fence(ts_ctx* ctx, void* cuda_stream);

/*
 * Token Velocity counters (Sec. 3.2). Cumulative since ts_create; a monitor divides deltas by
 * its window: prefill velocity = d(prefill_tokens)/dt, generation throughput =
 * d(decode_tokens)/dt, Decode Velocity (Eq. 1) = d(released_tokens)/dt.
 * busy_seconds is the sum of caller-reported step times (ts_report_step_time).
 */
typedef struct {
  uint64_t steps;
  uint64_t prefill_tokens;     /* sum of q_len over rows with q_len > 1                      */
  uint64_t decode_tokens;      /* number of rows with q_len == 1                             */
  uint64_t released_tokens;    /* sum of L_r over freed requests (Eq. 1 numerator)           */
  uint64_t released_requests;
  uint64_t pages_in_use;
  uint64_t pages_free;
  uint64_t kernel_launches;    /* kernels this context has enqueued                          */
  double busy_seconds;
} ts_velocity_counters;
int ts_velocity(ts_ctx* ctx, ts_velocity_counters* out);
int ts_report_step_time(ts_ctx* ctx, double seconds);

/*
 * Per-kernel device timing, for benchmarks. While enabled, every ts_mixed_step records CUDA
 * events around its kernels on the step's stream. ts_profile_read waits for the stream, returns
 * the milliseconds accumulated per kernel over the steps recorded since the last read, and
 * clears them. Not meant for production steps (each event costs a little stream time).
 */
typedef struct {
  double append_ms;     /* table update + KV append kernels                  */
  double prefill_ms;    /* attention kernel of steps whose launch held prefill tiles only */
  double decode_ms;     /* stand-alone split-KV decode attention kernel      */
  double combine_ms;    /* split-combine kernel                              */
  int64_t steps;
  double mixed_ms;      /* attention kernel of steps where one launch ran the prefill tiles
                           and the decode rows together                       */
  int64_t mixed_steps;  /* how many of `steps` those were                     */
} ts_profile;
int ts_profile_enable(ts_ctx* ctx, int enable);
int ts_profile_read(ts_ctx* ctx, void* cuda_stream, ts_profile* out);

/*
 * ts_prefill_budget: Eq. 5 per iteration -- the prefill tokens a Convertible Decoder may take
 * next to decode_batch_size decode rows: max(chunk_size - decode_batch_size, 0).
 * Dividing by the TPOT SLO gives V_D^{P'}.
 */
int32_t ts_prefill_budget(const ts_ctx* ctx, int32_t decode_batch_size);

/*
 * Configuring a Convertible Decoder (Sec. 4.4). Host-only arithmetic, no context needed.
 *
 * ts_pick_chunk_size: the chunk size is found by profiling the iteration time while the prefill
 * chunk grows, until the TPOT SLO is violated; the largest chunk size before that is taken.
 * prefill_tokens[i] (ascending, > 0) are the profiled prefill sizes at a fixed decode batch,
 * iteration_seconds[i] the caller's iteration time at each (e.g. the measured ts_mixed_step
 * time times the number of layers). Returns prefill_tokens[last point within the SLO before the
 * first violation] + decode_batch_size -- chunk size is defined as prefill tokens + decode batch
 * size -- or 0 when the first point already violates it, or TS_ERR_INVALID (negative) for null
 * arrays, n <= 0, sizes that are not ascending, a negative batch size or a non-positive SLO.
 *
 * ts_convertible_prefill_velocity: Eq. 5, V_D^{P'} = (chunk_size - batch_size) / TPOT_SLO in
 * tokens/s, with the average decode batch size as a real number; 0 when the batch fills the chunk
 * or the SLO is not positive.
 *
 * ts_reserved_memory: Eq. 6, Mem_Reserved = V_D^{P'} * Mem_T * TTFT_SLO in the unit of
 * mem_per_token. ts_reserved_pages: the same in whole KV pages of page_size tokens (Mem_T cancels:
 * V_D^{P'} * TTFT_SLO tokens, rounded up) -- the value for ts_config.reserved_pages. Both return
 * 0 for non-positive arguments.
 */
int32_t ts_pick_chunk_size(const int32_t* prefill_tokens, const double* iteration_seconds, int32_t n,
                           int32_t decode_batch_size, double tpot_slo_s);
double ts_convertible_prefill_velocity(int32_t chunk_size, double decode_batch_size, double tpot_slo_s);
double ts_reserved_memory(double prefill_velocity, double mem_per_token, double ttft_slo_s);
int32_t ts_reserved_pages(double prefill_velocity, double ttft_slo_s, int32_t page_size);

/*
 * The Token Velocity policy around the step (Sec. 4.3, Sec. 4.5.1). Host-only arithmetic fed by
 * rates the caller measures and by velocities profiled with ts_velocity / ts_report_step_time.
 *
 * ts_prefiller_instances: Eq. 2, I^P = lambda / min(V_P, V_BW), as the minimum whole number of
 * instances whose velocity covers the input token rate (rounded up). 0 for a non-positive rate,
 * TS_ERR_INVALID (negative) for a non-positive velocity.
 * ts_decoder_demand: Eq. 3, I^D = sum over the n_buckets request buckets of
 * token_rate[b] / velocity[b], as a real number (the paper compares 3.2 against 3 provisioned);
 * -1.0 for null arrays, n_buckets <= 0, a negative rate or a non-positive velocity.
 * ts_regular_decoders: Eq. 4, I^D_r = max(ceil(I^D) - I^D_c, 0), the Convertible Decoders being a
 * fixed pool that is never scaled.
 *
 * ts_route_prefill: Algorithm 1. The request goes to the first of the n_prefillers prefillers
 * whose estimated waiting time inflight_tokens / velocity is <= slo_s; failing that to the first
 * of the n_convertible Convertible Decoders that passes the same test with its prefill velocity
 * V_D^{P'} (Eq. 5); failing that it is queued. *kind_out: TS_ROUTE_PREFILLER, TS_ROUTE_CONVERTIBLE
 * or TS_ROUTE_QUEUE; returns the chosen index (0 when queued) or TS_ERR_INVALID for a null
 * kind_out, a null array with a positive count, a negative in-flight count or a non-positive
 * velocity. Arrays are HOST memory and only read.
 */
enum { TS_ROUTE_PREFILLER = 0, TS_ROUTE_CONVERTIBLE = 1, TS_ROUTE_QUEUE = 2 };
int32_t ts_prefiller_instances(double token_rate, double prefill_velocity, double network_velocity);
double ts_decoder_demand(const double* token_rate, const double* velocity, int32_t n_buckets);
int32_t ts_regular_decoders(double decoder_demand, int32_t convertible_decoders);
int32_t ts_route_prefill(const double* prefiller_inflight_tokens, const double* prefiller_velocity,
                         int32_t n_prefillers, const double* convertible_inflight_tokens,
                         const double* convertible_prefill_velocity, int32_t n_convertible, double slo_s,
                         int32_t* kind_out);

/*
 * ts_plan_step: host-only. Validates the step exactly as ts_mixed_step does and writes the
 * work list it would launch: one record of 8 int32 per work item
 *   {row, kind (0 decode split, 1 prefill tile), q_begin, q_count, k_begin, k_end,
 *    partial_slot (-1: writes out directly), reserved}
 * q_begin/q_count: the new tokens of the row the item covers (a decode split: 0, 1; a prefill
 * tile: 2*(128/G) tokens at most for head_dim 128, 64/G for head_dim 64); the item attends keys
 * [k_begin, k_end), each token only up to its own position.
 * (token and key positions are relative to the row's request). items may be NULL to query the
 * count. Returns TS_OK or the validation error; *n_items_out receives the number of items.
 */
int ts_plan_step(ts_ctx* ctx, const ts_step* step, int32_t* items, int32_t items_capacity,
                 int32_t* n_items_out);

/*
 * ts_last_device_status: waits for cuda_stream, then reads and clears the device status word:
 * 0, or a bit set of TS_DEV_* flags raised by kernels (they skip the offending access
 * instead of faulting).
 */
enum { TS_DEV_BAD_PAGE = 1, TS_DEV_TIMEOUT = 2, TS_DEV_BAD_INDEX = 4 };
int ts_last_device_status(ts_ctx* ctx, void* cuda_stream, int32_t* status_out);

/*
 * ts_decode_attention_static: decode attention (one query token per row) that allocates
 * nothing and needs no workspace. (The paper has no counterpart; this is a packaging variant
 * of the split-KV decode path of ts_mixed_step.)
 *
 * Who it is for: code that must not, or cannot, obtain device memory at the point where it
 * needs attention -- for example a serving process whose framework has already claimed all
 * of HBM for its own KV pool, so that a further cudaMalloc would fail; a plug-in that is only
 * handed tensors and is not allowed to own memory; or a latency-critical loop that cannot
 * afford the device-wide synchronisation an allocation may imply. Such a caller cannot supply
 * the workspace ts_create asks for. Here the split partials and the work list live in a
 * fixed array inside the library (about 8.4 MiB, present on every GPU that loads the
 * library, until the process ends). The call makes no cudaMalloc/cudaFree and uses no
 * allocating routine.
 *
 * Arguments (all tensors DEVICE memory of `device`, owned by the caller):
 *   kv_pool       the pool in the layout documented above; the K/V of every attended token,
 *                 the newest one included, must already be in it (this call appends nothing)
 *   block_tables  int32 [n_rows][table_width]: page ids of row r in its first
 *                 ceil(kv_len[r]/16) entries. A page id outside [0, n_pages) is not followed:
 *                 its 16 keys count as absent (zero-filled K/V), the row's output is then wrong
 *                 but finite, and NO error is reported -- this entry point has no status word
 *                 the host can read, so the caller must pass valid tables
 *   kv_len        int32 [n_rows]: tokens row r attends to, 1 <= kv_len[r] <= 16*table_width
 *                 (a row outside this range is not processed and its output is NaN)
 *   q, out        bf16 [n_rows, n_q_heads, head_dim], 16-byte aligned
 *   n_splits      keys of each row are cut into at most this many splits (1..16)
 *   softmax_scale 0 => 1/sqrt(head_dim)
 * Limits of the built-in scratch: n_rows <= 256, n_splits <= 16 and
 * n_rows * n_splits * n_q_heads * head_dim <= 2^21; beyond them the call returns
 * TS_ERR_WORKSPACE and launches nothing. Shapes as for ts_config, else TS_ERR_UNSUPPORTED.
 *
 * The work is enqueued on cuda_stream and the call returns without waiting. The first call on
 * a device looks up the device address of the built-in array (it makes `device` current, as
 * every call does); make that first call outside any stream capture.
 * All calls in the process share the one array and it keeps the previous call's contents
 * (each call rewrites every entry it later reads, so nothing needs clearing by the caller):
 * two calls whose kernels can overlap on the GPU -- different streams, or different host
 * threads -- race on it. Keep calls on one stream, or order them with events.
 */
int ts_decode_attention_static(int32_t device, int32_t n_q_heads, int32_t n_kv_heads,
                               int32_t head_dim, int32_t n_pages, const void* kv_pool,
                               const int32_t* block_tables, int32_t table_width,
                               const int32_t* kv_len, int32_t n_rows, int32_t n_splits,
                               float softmax_scale, const void* q, void* out, void* cuda_stream);

/*
 * The decoder layer around the attention step. The paper's velocities are rates of whole model
 * iterations (prefill velocity, Sec. 3.2: the maximum speed at which input tokens are processed,
 * bound by GPU compute; Sec. 4.4 profiles the iteration time of a Convertible Decoder against the
 * TPOT SLO); an iteration runs, for every layer, the projections in front of attention, attention
 * over the paged KV cache with the append of the new K/V (Sec. 2.1), the output projection and the
 * MLP. The paper runs Llama-3.1-8B and Qwen-2.5-32B (Sec. 6.1) and describes none of this; the
 * layer here is the pre-norm block those models share:
 *      h = rmsnorm(x; w_norm1)            q, k, v = split(h . W_qkv^T); q, k = rope(q, k; position)
 *      a = ts_mixed_step(q, k, v)         y = x + a . W_o^T
 *      h2 = rmsnorm(y; w_norm2)           out = y + (silu(h2 . W_gate^T) * (h2 . W_up^T)) . W_down^T
 * rmsnorm(x; w) = x / sqrt(mean(x^2) + rms_eps) * w per token; rope rotates the pairs (i, i + D/2)
 * of every query and key head by the angle position * rope_theta^(-2i/D), position = ctx_len + i
 * for the row's i-th new token; silu(t) = t / (1 + exp(-t)). All tensors are bf16 (the serving
 * precision, Sec. 6.1): every tensor named above is rounded to bf16 (nearest even) where it is
 * produced, sums are accumulated in fp32. Weights are [out features][in features], row-major.
 * head_dim must be 128, hidden a multiple of 64, intermediate a multiple of 128, and the context's
 * chunk_size > 0 (it sizes the activations).
 */
typedef struct ts_layer ts_layer; /* opaque; host memory; used with its ts_ctx, one thread and stream at a time */
typedef struct {
  int32_t hidden;           /* model width: columns of x                                        */
  int32_t intermediate;     /* MLP width                                                        */
  int32_t max_position;     /* rows of the rotary table: ctx_len + q_len of a row must not exceed it */
  float rms_eps;            /* 0 => 1e-5                                                        */
  float rope_theta;         /* 0 => 500000                                                      */
  const void* w_norm1;      /* DEVICE bf16 [hidden]                                             */
  const void* w_qkv;        /* DEVICE bf16 [(Hq + 2 Hkv) D][hidden]: query heads, key heads, value heads */
  const void* w_o;          /* DEVICE bf16 [hidden][Hq D]                                       */
  const void* w_norm2;      /* DEVICE bf16 [hidden]                                             */
  const void* w_gate_up;    /* DEVICE bf16 [2 intermediate][hidden] in the order ts_pack_gate_up writes */
  const void* w_down;       /* DEVICE bf16 [hidden][intermediate]                               */
  void* workspace;          /* DEVICE, ts_layer_workspace_bytes() bytes, 256-byte aligned, caller-owned: the
                               rotary table and the layer's activations                         */
  size_t workspace_bytes;
} ts_layer_config;          /* all weight pointers 16-byte aligned, caller-owned, only read     */

/* 0 on an unsupported shape. Reads the shape fields of both structs and cfg->chunk_size. */
size_t ts_layer_workspace_bytes(const ts_config* cfg, const ts_layer_config* layer);

/*
 * ts_pack_gate_up: writes the gate and up projection weights (DEVICE bf16 [intermediate][hidden]
 * each) interleaved in blocks of 128 rows -- rows [256 b, 256 b + 128) of the result are gate rows
 * [128 b, 128 b + 128), the next 128 rows the up rows of the same features -- so that one GEMM
 * tile holds both halves of a feature and can apply the SiLU gate itself. Asynchronous on
 * cuda_stream. TS_ERR_INVALID unless intermediate % 128 == 0 and hidden % 8 == 0.
 */
int ts_pack_gate_up(const void* w_gate, const void* w_up, void* w_gate_up, int32_t intermediate, int32_t hidden,
                    void* cuda_stream);

/*
 * ts_layer_create: binds the weights to a context (the layer's attention runs on the context's
 * pool and block tables) and enqueues the rotary table's computation on cuda_stream.
 * TS_ERR_UNSUPPORTED for a shape outside the limits above, TS_ERR_WORKSPACE for a short workspace.
 * ts_layer_destroy frees host memory only; destroy the layer before its context.
 */
int ts_layer_create(ts_ctx* ctx, const ts_layer_config* cfg, void* cuda_stream, ts_layer** out);
int ts_layer_destroy(ts_layer* layer);

/*
 * ts_layer_step: one iteration of the layer over the step's rows (slot, q_len, ctx_len as for
 * ts_mixed_step, which it calls; q, k_new, v_new, out of `step` are ignored). x_in, x_out: DEVICE
 * bf16 [N][hidden], 16-byte aligned, may not alias. Everything is enqueued on cuda_stream; the
 * call does not synchronise. Validation is the step's own (nothing is launched on failure), plus
 * TS_ERR_INVALID when a row reaches past max_position. Updates the context's counters as
 * ts_mixed_step does.
 */
int ts_layer_step(ts_layer* layer, const ts_step* step, const void* x_in, void* x_out, void* cuda_stream);
int ts_layer_last_cuda_error(const ts_layer* layer);

/*
 * ts_gemm_bf16: the layer's projection kernel by itself (for measurements and tests):
 * C[M][N] = (R ? R : 0) + A[M][K] . B[N][K]^T, all DEVICE bf16 row-major and 16-byte aligned, fp32
 * accumulation, bf16 result. N and K multiples of 8. tile_m: rows of an output tile per thread
 * block, 128 or 256, 0 = chosen from the shape. device_status: DEVICE int32 the caller has zeroed;
 * a bounded wait that runs out sets TS_DEV_TIMEOUT there. Asynchronous on cuda_stream.
 */
int ts_gemm_bf16(int32_t device, int32_t M, int32_t N, int32_t K, const void* A, const void* B, const void* R,
                 void* C, int32_t tile_m, int32_t* device_status, void* cuda_stream);

/* The cudaError_t of the most recent failed CUDA call of this context (0 if none). */
int ts_last_cuda_error(const ts_ctx* ctx);

const char* ts_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* TOKENSCALE_H_ */
