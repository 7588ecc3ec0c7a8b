// Host side of the mixed paged-attention step: page allocator, per-request block tables,
// step validation, work-list planning, metadata upload and kernel launches, Token Velocity
// counters. The public ABI is documented in include/tokenscale.h.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/tokenscale.h"
#include "ts_internal.h"

namespace {

using ts::CombineItem;
using ts::TableDelta;
using ts::WorkItem;

constexpr int kRing = 4;                  // pinned metadata buffers in flight
constexpr int kDeltaCapacity = 32768;     // table entries per upload batch (bulk loads)
constexpr int kSlotDeltas = 4096;         // table entries that ride along with a step's metadata
constexpr int kDefaultSplit = 4096;       // keys per decode split (measured: 2048 and 8192 are both a few percent slower)
constexpr int kDefaultMaxTokens = 16384;  // step size bound when chunk_size == 0
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

constexpr int kStageSets = 3;   // staging sets of ts_mixed_step_host: one step uploads while another runs
                                // and a third one's result goes down

struct Layout {
  int max_tokens, max_partials, max_items;
  size_t off_status, off_table, off_meta, off_delta, off_part_acc, off_part_ml, off_stage;
  size_t meta_bytes, slot_bytes, delta_bytes, stage_q_bytes, stage_kv_bytes, stage_set_bytes, total;
  // int32 offsets inside the meta area
  size_t m_row_slot, m_row_ctx, m_row_qlen, m_row_tok0, m_items, m_combines, m_end;
};

bool shape_ok(const ts_config* c) {
  if (!c) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->page_size != ts::kPageSize) return false;
  if (c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->n_q_heads % c->n_kv_heads) return false;
  if (c->n_q_heads / c->n_kv_heads > ts::kMaxGroup) return false;
  if (c->n_pages <= 0 || c->max_requests <= 0 || c->max_pages_per_req <= 0) return false;
  if (c->chunk_size < 0 || c->reserved_pages < 0 || c->decode_split_tokens < 0) return false;
  if (c->wait_limit_cycles < 0) return false;
  return true;
}

void compute_layout(const ts_config* c, Layout* L) {
  const int G = c->n_q_heads / c->n_kv_heads;
  const int R = c->max_requests;
  L->max_tokens = c->chunk_size > 0 ? c->chunk_size : kDefaultMaxTokens;
  L->max_partials = 2048 + 2 * R;
  L->max_items = L->max_partials + R + ceil_div(L->max_tokens, std::max(1, ts::kPackedRowsPerTile / G)) + R;
  size_t m = 0;
  L->m_row_slot = m; m += R;
  L->m_row_ctx = m; m += R;
  L->m_row_qlen = m; m += R;
  L->m_row_tok0 = m; m += R + 1;
  m = (m + 7) / 8 * 8;                       // items start 32-byte aligned
  L->m_items = m; m += (size_t)L->max_items * 8;
  L->m_combines = m; m += (size_t)R * 4;
  L->m_end = m;
  L->meta_bytes = align_up(m * sizeof(int32_t));
  L->delta_bytes = align_up((size_t)kDeltaCapacity * sizeof(TableDelta));
  size_t off = 0;
  L->off_status = off; off += kAlign;
  L->off_table = off; off += align_up((size_t)R * c->max_pages_per_req * sizeof(int32_t));
  // one slot per step in flight: the step's metadata, then up to kSlotDeltas block-table entries
  L->slot_bytes = L->meta_bytes + align_up((size_t)kSlotDeltas * sizeof(TableDelta));
  L->off_meta = off; off += kRing * L->slot_bytes;
  L->off_delta = off; off += L->delta_bytes;
  L->off_part_acc = off;
  off += align_up((size_t)L->max_partials * c->n_q_heads * c->head_dim * sizeof(float));
  L->off_part_ml = off; off += align_up((size_t)L->max_partials * c->n_q_heads * 2 * sizeof(float));
  L->stage_q_bytes = align_up((size_t)L->max_tokens * c->n_q_heads * c->head_dim * 2);
  L->stage_kv_bytes = align_up((size_t)L->max_tokens * c->n_kv_heads * c->head_dim * 2);
  L->stage_set_bytes = 2 * L->stage_q_bytes + 2 * L->stage_kv_bytes;     // q, out, k_new, v_new
  L->off_stage = off; off += kStageSets * L->stage_set_bytes;
  L->total = off;
}

struct Slot {
  bool live = false;
  int64_t req_id = 0;
  int32_t prompt_len = 0, expected_output_len = 0;
  int32_t n_pages = 0;       // table entries in use
  int32_t n_tokens = 0;      // tokens cached
  int32_t synced_pages = 0;  // leading entries the device copy already holds
  uint32_t stamp = 0;        // duplicate detection within a step
};

struct RingBuf {
  void* host = nullptr;
  cudaEvent_t ev = nullptr;
  bool in_flight = false;
};

// One slot of step metadata: a pinned host buffer, its device copy in the workspace, and the
// two events that order them. The upload runs on the context's own copy stream, next to the
// previous step's kernels instead of between them.
struct MetaSlot {
  void* host = nullptr;
  cudaEvent_t copied = nullptr;     // copy stream: the slot's upload has finished
  cudaEvent_t consumed = nullptr;   // caller's stream: the step that read the slot is done
  bool copy_in_flight = false;
  bool read_in_flight = false;
};

uint64_t splitmix64(uint64_t& s) {
  uint64_t z = (s += 0x9E3779B97F4A7C15ull);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

}  // namespace

struct ts_ctx {
  ts_config cfg;
  Layout L;
  int G = 1;
  float scale = 0.f;
  std::vector<int32_t> table;       // [max_requests][max_pages_per_req]
  std::vector<Slot> slots;
  std::vector<int32_t> free_pages;  // stack, next page at the back
  std::vector<int32_t> page_owner;  // -1 = free
  std::vector<int32_t> free_slots;  // stack
  ts_velocity_counters cnt;
  RingBuf ring[kRing];              // block-table deltas
  int ring_next = 0;
  size_t ring_bytes = 0;
  MetaSlot meta[kRing];             // step metadata
  int meta_next = 0;
  int meta_cur = 0;                 // slot of the step being issued
  cudaStream_t copy_stream = nullptr;
  // ts_mixed_step_host: inputs go up on up_stream, results come down on down_stream, the step
  // itself runs on the caller's stream; the events order the three per staging set
  cudaStream_t up_stream = nullptr, down_stream = nullptr;
  cudaEvent_t up_done[kStageSets] = {}, step_done[kStageSets] = {}, down_done[kStageSets] = {};
  bool stage_used[kStageSets] = {};
  uint64_t host_steps = 0;
  bool cuda_ready = false;
  CUtensorMap kv_map;               // TMA view of the pool, box = K and V of one (page, head) half
  CUtensorMap kv_tile_map;          // same view, box = K or V of one (page, head) half
  void* encode_fn = nullptr;        // cuTensorMapEncodeTiled
  int n_sms = 0;
  int n_prefill_items = 0;          // of the current plan
  bool status_cleared = false;
  int last_cuda_error = 0;
  uint32_t stamp = 0;
  // scratch reused across steps
  std::vector<WorkItem> items;
  std::vector<CombineItem> combines;
  std::vector<int32_t> tok0;
  std::vector<TableDelta> deltas;
  std::vector<std::pair<int32_t, int32_t>> sync_marks;   // (slot, table entries the device will hold)
  // optional per-kernel timing: 5 events per recorded step
  bool profiling = false;
  std::vector<cudaEvent_t> prof_events;
  std::vector<char> prof_mixed;     // per recorded step: did one launch run tiles and decode rows together
  size_t prof_used = 0;
};

namespace {

int32_t* table_row(ts_ctx* c, int slot) { return c->table.data() + (size_t)slot * c->cfg.max_pages_per_req; }

bool slot_ok(const ts_ctx* c, int32_t slot) {
  return slot >= 0 && slot < c->cfg.max_requests && c->slots[slot].live;
}

int cuda_fail(ts_ctx* c, cudaError_t e) {
  c->last_cuda_error = (int)e;
  return TS_ERR_CUDA;
}

#define TS_CUDA(c, call)                                 \
  do {                                                   \
    cudaError_t e__ = (call);                            \
    if (e__ != cudaSuccess) return cuda_fail((c), e__);  \
  } while (0)

void release_pages(ts_ctx* c, int slot) {
  Slot& s = c->slots[slot];
  int32_t* row = table_row(c, slot);
  for (int i = s.n_pages - 1; i >= 0; --i) {
    c->page_owner[row[i]] = -1;
    c->free_pages.push_back(row[i]);
  }
  s.n_pages = 0;
  s.synced_pages = 0;
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 5-D tensor map over the pool, fastest dimension first: head_dim, slot, KV head, K|V, page.
// Box = 64 elements (128 bytes, the swizzle span) x 16 slots x 1 head x {K, V} x 1 page.
int make_kv_maps(ts_ctx* c) {
  cudaDriverEntryPointQueryResult qres;
  TS_CUDA(c, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_fn, cudaEnableDefault, &qres));
  if (!c->encode_fn || qres != cudaDriverEntryPointSuccess) return cuda_fail(c, cudaErrorNotSupported);
  const cuuint64_t D = c->cfg.head_dim, P = c->cfg.page_size, H = c->cfg.n_kv_heads;
  const cuuint64_t dims[5] = {D, P, H, 2, (cuuint64_t)c->cfg.n_pages};
  const cuuint64_t strides[4] = {D * 2, P * D * 2, H * P * D * 2, 2 * H * P * D * 2};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  // kv_map: K and V of one (page, head) half together, for the decode units; kv_tile_map: one
  // operand only, for the K and V tiles of the prefill path
  for (int both = 1; both >= 0; --both) {
    const cuuint32_t box[5] = {64, (cuuint32_t)P, 1, (cuuint32_t)(both ? 2 : 1), 1};
    const CUresult r = ((EncodeFn)c->encode_fn)(both ? &c->kv_map : &c->kv_tile_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                                5, c->cfg.kv_pool, dims, strides, box, estr,
                                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail(c, cudaErrorInvalidValue);
  }
  return TS_OK;
}

// q viewed as (head_dim, head in group, KV head, token); one box = 64 elements x G heads x 1 x
// 128/G tokens = one 64-column half of a 128-row query tile in packed (token, head) order.
int make_q_map(ts_ctx* c, const void* q, int64_t n_tokens, CUtensorMap* out) {
  const cuuint64_t D = c->cfg.head_dim, G = c->G, H = c->cfg.n_kv_heads;
  const cuuint64_t dims[4] = {D, G, H, (cuuint64_t)n_tokens};
  const cuuint64_t strides[3] = {D * 2, G * D * 2, H * G * D * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)G, 1, (cuuint32_t)(ts::kPackedRowsTc / c->G)};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = ((EncodeFn)c->encode_fn)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims,
                                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cuda_fail(c, cudaErrorInvalidValue);
  return TS_OK;
}

int ensure_cuda(ts_ctx* c, cudaStream_t stream) {
  if (!c->cfg.kv_pool || !c->cfg.workspace) return cuda_fail(c, cudaErrorInvalidDevicePointer);
  TS_CUDA(c, cudaSetDevice(c->cfg.device));
  if (!c->cuda_ready) {
    c->ring_bytes = c->L.delta_bytes;
    for (int i = 0; i < kRing; ++i) {
      TS_CUDA(c, cudaHostAlloc(&c->ring[i].host, c->ring_bytes, cudaHostAllocDefault));
      TS_CUDA(c, cudaEventCreateWithFlags(&c->ring[i].ev, cudaEventDisableTiming));
      TS_CUDA(c, cudaHostAlloc(&c->meta[i].host, c->L.slot_bytes, cudaHostAllocDefault));
      TS_CUDA(c, cudaEventCreateWithFlags(&c->meta[i].copied, cudaEventDisableTiming));
      TS_CUDA(c, cudaEventCreateWithFlags(&c->meta[i].consumed, cudaEventDisableTiming));
    }
    TS_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
    TS_CUDA(c, cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, c->cfg.device));
    int rc = make_kv_maps(c);
    if (rc != TS_OK) return rc;
    c->cuda_ready = true;
  }
  if (!c->status_cleared) {
    TS_CUDA(c, cudaMemsetAsync((char*)c->cfg.workspace + c->L.off_status, 0, kAlign, stream));
    c->status_cleared = true;
  }
  return TS_OK;
}

// Next pinned buffer; waits only if the copy that last used it has not finished.
int ring_acquire(ts_ctx* c, RingBuf** out) {
  RingBuf& r = c->ring[c->ring_next];
  c->ring_next = (c->ring_next + 1) % kRing;
  if (r.in_flight) {
    TS_CUDA(c, cudaEventSynchronize(r.ev));
    r.in_flight = false;
  }
  *out = &r;
  return TS_OK;
}

int ring_send(ts_ctx* c, RingBuf* r, size_t dst_off, size_t bytes, cudaStream_t stream) {
  TS_CUDA(c, cudaMemcpyAsync((char*)c->cfg.workspace + dst_off, r->host, bytes,
                             cudaMemcpyHostToDevice, stream));
  TS_CUDA(c, cudaEventRecord(r->ev, stream));
  r->in_flight = true;
  return TS_OK;
}

// Checks shared by ts_kv_append, ts_mixed_step and ts_plan_step. Fills tok0 (prefix sums).
int validate(ts_ctx* c, const ts_step* st, bool attention, bool need_tensors, int64_t* n_tokens_out,
             int* n_decode_out, int64_t* n_prefill_out) {
  if (!c || !st) return TS_ERR_INVALID;
  if (st->n_rows < 0 || st->n_rows > c->cfg.max_requests) return TS_ERR_INVALID;
  if (st->n_rows > 0 && (!st->slot || !st->q_len || !st->ctx_len)) return TS_ERR_INVALID;
  c->tok0.assign((size_t)st->n_rows + 1, 0);
  ++c->stamp;
  if (c->stamp == 0) {  // wrapped: restart stamps
    for (auto& s : c->slots) s.stamp = 0;
    c->stamp = 1;
  }
  int64_t n = 0, n_prefill = 0;
  int n_decode = 0;
  const int P = c->cfg.page_size;
  for (int r = 0; r < st->n_rows; ++r) {
    const int32_t slot = st->slot[r], ql = st->q_len[r], ctx = st->ctx_len[r];
    if (!slot_ok(c, slot)) return TS_ERR_INVALID;
    Slot& s = c->slots[slot];
    if (s.stamp == c->stamp) return TS_ERR_INVALID;  // slot listed twice
    s.stamp = c->stamp;
    if (ql < 1 || ctx < 0) return TS_ERR_INVALID;
    if (ctx != s.n_tokens) return TS_ERR_INVALID;
    if ((int64_t)ctx + ql > (int64_t)s.n_pages * P) return TS_ERR_TABLE_SHORT;
    n += ql;
    if (n > INT32_MAX / 2) return TS_ERR_INVALID;
    c->tok0[r + 1] = (int32_t)n;
    if (ql == 1) ++n_decode; else n_prefill += ql;
  }
  if (attention) {
    if (c->cfg.chunk_size > 0 && n_prefill + n_decode > c->cfg.chunk_size) return TS_ERR_BUDGET;
    if (n > c->L.max_tokens) return TS_ERR_BUDGET;
  }
  if (n > 0 && need_tensors) {
    if (!st->k_new || !st->v_new) return TS_ERR_INVALID;
    if (attention && (!st->q || !st->out)) return TS_ERR_INVALID;
  }
  *n_tokens_out = n;
  *n_decode_out = n_decode;
  *n_prefill_out = n_prefill;
  return TS_OK;
}

// Builds c->items / c->combines for a validated step.
void plan(ts_ctx* c, const ts_step* st) {
  const int G = c->G;
  int split = c->cfg.decode_split_tokens > 0 ? c->cfg.decode_split_tokens : kDefaultSplit;
  split = ceil_div(split, ts::kKeysPerTile) * ts::kKeysPerTile;
  for (;;) {
    c->items.clear();
    c->combines.clear();
    int partial = 0;
    for (int r = 0; r < st->n_rows; ++r) {
      const int ql = st->q_len[r], ctx = st->ctx_len[r];
      if (ql > 1) {
        // head_dim 128: two query tiles of 128 packed rows per item (128/G whole tokens each);
        // head_dim 64: one tile of 64 packed rows
        const int tt = c->cfg.head_dim == 128 ? 2 * (ts::kPackedRowsTc / G) : ts::kPackedRowsPerTile / G;
        for (int t0 = 0; t0 < ql; t0 += tt) {
          const int cnt = std::min(tt, ql - t0);
          c->items.push_back(WorkItem{r, 1, t0, cnt, 0, ctx + t0 + cnt, -1, 0});
        }
      } else {
        const int n = ctx + 1;
        int ns = ceil_div(n, split);
        if (ns <= 1) {
          c->items.push_back(WorkItem{r, 0, 0, 1, 0, n, -1, 0});
        } else {
          const int per = ceil_div(ceil_div(n, ns), ts::kKeysPerTile) * ts::kKeysPerTile;
          ns = ceil_div(n, per);
          c->combines.push_back(CombineItem{c->tok0[r], partial, ns, 0});
          for (int s = 0; s < ns; ++s) {
            c->items.push_back(WorkItem{r, 0, 0, 1, s * per, std::min(n, (s + 1) * per), partial++, 0});
          }
        }
      }
    }
    if (partial <= c->L.max_partials) break;
    split *= 2;
  }
  // Prefill tiles first, then decode splits; inside each group heaviest first, so that the tail
  // of each launch is made of short items.
  std::stable_sort(c->items.begin(), c->items.end(), [](const WorkItem& a, const WorkItem& b) {
    if (a.kind != b.kind) return a.kind > b.kind;
    return (a.k_end - a.k_begin) > (b.k_end - b.k_begin);
  });
  c->n_prefill_items = 0;
  for (const WorkItem& w : c->items) c->n_prefill_items += w.kind == 1;
}

// Brings the device copy of the rows' block tables up to date (entries added since the last
// step that used the slot). Entries travel by value through the pinned ring, so later host-side
// changes cannot alter what an already enqueued step sees.
int sync_tables(ts_ctx* c, const ts_step* st, cudaStream_t stream, int* n_slot_deltas) {
  *n_slot_deltas = 0;
  c->deltas.clear();
  c->sync_marks.clear();
  for (int r = 0; r < st->n_rows; ++r) {
    Slot& s = c->slots[st->slot[r]];
    const int32_t* row = table_row(c, st->slot[r]);
    for (int i = s.synced_pages; i < s.n_pages; ++i)
      c->deltas.push_back(TableDelta{st->slot[r], i, row[i]});
    // synced_pages only advances once the entries are on their way (commit_table_sync): a step
    // that fails before that leaves the record as it was, and the next step sends them again
    if (s.n_pages > s.synced_pages) c->sync_marks.push_back({st->slot[r], s.n_pages});
  }
  if (c->deltas.size() <= (size_t)kSlotDeltas) {
    // the usual case (a few rows crossed a page boundary): the entries travel with the step's
    // metadata over the copy stream, see upload_meta
    *n_slot_deltas = (int)c->deltas.size();
    return TS_OK;
  }
  size_t at = 0;
  while (at < c->deltas.size()) {
    const size_t n = std::min(c->deltas.size() - at, (size_t)kDeltaCapacity);
    RingBuf* rb;
    int rc = ring_acquire(c, &rb);
    if (rc != TS_OK) return rc;
    std::memcpy(rb->host, c->deltas.data() + at, n * sizeof(TableDelta));
    rc = ring_send(c, rb, c->L.off_delta, n * sizeof(TableDelta), stream);
    if (rc != TS_OK) return rc;
    char* ws = (char*)c->cfg.workspace;
    TS_CUDA(c, ts::launch_table_update((int32_t*)(ws + c->L.off_table), c->cfg.max_pages_per_req,
                                       c->cfg.max_requests, (int32_t*)(ws + c->L.off_status),
                                       (const TableDelta*)(ws + c->L.off_delta), (int)n, stream));
    ++c->cnt.kernel_launches;
    at += n;
  }
  return TS_OK;
}

// The table entries gathered by sync_tables have been enqueued (copy and table_update launch).
void commit_table_sync(ts_ctx* c) {
  for (const auto& m : c->sync_marks) c->slots[m.first].synced_pages = m.second;
  c->sync_marks.clear();
}

// Sends the step's metadata to the next device slot. The copy goes over the context's copy stream:
// it only has to wait for the step that last read this slot (kRing steps ago), so it runs while
// the previous step's kernels are still busy, and the caller's stream just waits for its event.
int upload_meta(ts_ctx* c, const ts_step* st, int n_items, int n_combines, int n_slot_deltas, cudaStream_t stream) {
  const int slot = c->meta_next;
  c->meta_next = (c->meta_next + 1) % kRing;
  c->meta_cur = slot;
  MetaSlot& ms = c->meta[slot];
  if (ms.copy_in_flight) {                 // the pinned buffer is free once its last upload is done
    TS_CUDA(c, cudaEventSynchronize(ms.copied));
    ms.copy_in_flight = false;
  }
  int32_t* m = (int32_t*)ms.host;
  const int R = st->n_rows;
  std::memcpy(m + c->L.m_row_slot, st->slot, sizeof(int32_t) * R);
  std::memcpy(m + c->L.m_row_ctx, st->ctx_len, sizeof(int32_t) * R);
  std::memcpy(m + c->L.m_row_qlen, st->q_len, sizeof(int32_t) * R);
  std::memcpy(m + c->L.m_row_tok0, c->tok0.data(), sizeof(int32_t) * (R + 1));
  size_t used = c->L.m_row_tok0 + R + 1;
  if (n_items > 0) {
    std::memcpy(m + c->L.m_items, c->items.data(), sizeof(WorkItem) * n_items);
    used = c->L.m_items + (size_t)n_items * 8;
  }
  if (n_combines > 0) {
    std::memcpy(m + c->L.m_combines, c->combines.data(), sizeof(CombineItem) * n_combines);
    used = c->L.m_combines + (size_t)n_combines * 4;
  }
  char* dev_slot = (char*)c->cfg.workspace + c->L.off_meta + (size_t)slot * c->L.slot_bytes;
  if (n_slot_deltas > 0)
    std::memcpy((char*)ms.host + c->L.meta_bytes, c->deltas.data(), (size_t)n_slot_deltas * sizeof(TableDelta));
  if (ms.read_in_flight) TS_CUDA(c, cudaStreamWaitEvent(c->copy_stream, ms.consumed, 0));
  TS_CUDA(c, cudaMemcpyAsync(dev_slot, ms.host, used * sizeof(int32_t), cudaMemcpyHostToDevice, c->copy_stream));
  if (n_slot_deltas > 0)
    TS_CUDA(c, cudaMemcpyAsync(dev_slot + c->L.meta_bytes, (char*)ms.host + c->L.meta_bytes,
                               (size_t)n_slot_deltas * sizeof(TableDelta), cudaMemcpyHostToDevice, c->copy_stream));
  TS_CUDA(c, cudaEventRecord(ms.copied, c->copy_stream));
  ms.copy_in_flight = true;
  TS_CUDA(c, cudaStreamWaitEvent(stream, ms.copied, 0));
  if (n_slot_deltas > 0) {
    char* ws = (char*)c->cfg.workspace;
    TS_CUDA(c, ts::launch_table_update((int32_t*)(ws + c->L.off_table), c->cfg.max_pages_per_req,
                                       c->cfg.max_requests, (int32_t*)(ws + c->L.off_status),
                                       (const TableDelta*)(dev_slot + c->L.meta_bytes), n_slot_deltas, stream));
    ++c->cnt.kernel_launches;
  }
  return TS_OK;
}

// After the step's kernels: marks the slot as read once the caller's stream gets here.
int release_meta(ts_ctx* c, cudaStream_t stream) {
  MetaSlot& ms = c->meta[c->meta_cur];
  TS_CUDA(c, cudaEventRecord(ms.consumed, stream));
  ms.read_in_flight = true;
  return TS_OK;
}

void fill_device(ts_ctx* c, const ts_step* st, int64_t n_tokens, ts::StepDevice* d) {
  char* ws = (char*)c->cfg.workspace;
  const int32_t* meta = (const int32_t*)(ws + c->L.off_meta + (size_t)c->meta_cur * c->L.slot_bytes);
  d->pool = (uint16_t*)c->cfg.kv_pool;
  d->table = (int32_t*)(ws + c->L.off_table);
  d->status = (int32_t*)(ws + c->L.off_status);
  d->pf_queue = d->status + 1;
  d->part_acc = (float*)(ws + c->L.off_part_acc);
  d->part_ml = (float*)(ws + c->L.off_part_ml);
  d->row_slot = meta + c->L.m_row_slot;
  d->row_ctx = meta + c->L.m_row_ctx;
  d->row_qlen = meta + c->L.m_row_qlen;
  d->row_tok0 = meta + c->L.m_row_tok0;
  d->items = (const WorkItem*)(meta + c->L.m_items);
  d->combines = (const CombineItem*)(meta + c->L.m_combines);
  d->q = (const uint16_t*)st->q;
  d->k_new = (const uint16_t*)st->k_new;
  d->v_new = (const uint16_t*)st->v_new;
  d->out = (uint16_t*)st->out;
  d->n_rows = st->n_rows;
  d->n_tokens = (int32_t)n_tokens;
  d->n_items = 0;
  d->n_combines = 0;
  d->n_prefill_items = 0;
  d->Hq = c->cfg.n_q_heads;
  d->Hkv = c->cfg.n_kv_heads;
  d->D = c->cfg.head_dim;
  d->n_pages = c->cfg.n_pages;
  d->max_pages_per_req = c->cfg.max_pages_per_req;
  d->max_requests = c->cfg.max_requests;
  d->scale_log2 = c->scale * 1.4426950408889634f;
  d->append_in_decode = 0;
  d->wait_cycles = c->cfg.wait_limit_cycles > 0 ? (long long)c->cfg.wait_limit_cycles : ts::kWaitCycles;
  d->append_ctas = 0;          // both set by the mixed launch
  d->append_arrivals = 0;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// How many CTAs of the mixed kernel take prefill tiles only, the rest streaming the decode rows
// first and joining the prefill queue afterwards. Cost model in SM-microseconds, calibrated on a
// B200: next to streaming decode CTAs a prefill work unit costs ~2.1 us per 128-key block pair
// plus ~2 us; the decode rows move their K/V at a fraction of the full-chip rate that falls off as
// fewer SMs pull on HBM, faster with eight query heads per KV head (twice the arithmetic per page)
// than with four.
//   G <= 4: an SM streams a decode unit at 70 GB/s plus ~2 us per unit, and all of them together
//           at no more than 6.1 TB/s; the step time is flat over a range of splits, of which the
//           middle is taken (its ends are the sensitive ones).
//   G >  4: measured fraction of the full-chip rate by SM count, linear in between:
//           48 0.475, 64 0.62, 74 0.715, 84 0.78, 100 0.85, 116 0.92, 132 0.95, 148 1
// A prefill CTA starts on its first unit once the prefill rows' new tokens are in their pages,
// which next to the decode streams takes ~8 us plus ~11 ns per token.
int choose_prefill_ctas(const ts_ctx* c, int n_ctas, double prefill_block_pairs, double prefill_units,
                        double decode_bytes, double decode_units, double prefill_tokens) {
  static const double kSm8[] = {0, 48, 64, 74, 84, 100, 116, 132, 148};
  static const double kRate8[] = {0, 0.475, 0.62, 0.715, 0.78, 0.85, 0.92, 0.95, 1.0};
  const bool wide = c->G > 4;
  const double w_pf = prefill_block_pairs * 2.1 + prefill_units * 2.0;
  const double t_append = 8.0 + 0.011 * prefill_tokens;
  const double t_dec_full = decode_bytes / 6.1e6;   // us at 6.1 TB/s
  const double unit_bytes = decode_bytes / std::max(1.0, decode_units);
  const double sm_rate = unit_bytes / (unit_bytes / 70e3 + 2.0);   // bytes per us and SM
  auto step_time = [&](int p) {
    double td;
    if (wide) {
      const double d = (double)(n_ctas - p) * 148.0 / c->n_sms;
      int i = 1;
      while (i < 8 && kSm8[i] < d) ++i;
      const double rate =
          d >= 148.0 ? 1.0 : kRate8[i - 1] + (kRate8[i] - kRate8[i - 1]) * (d - kSm8[i - 1]) / (kSm8[i] - kSm8[i - 1]);
      td = t_dec_full / rate;
    } else {
      td = std::max(t_dec_full, decode_bytes / ((double)(n_ctas - p) * sm_rate));
    }
    return std::max(td, (w_pf + (double)p * t_append + (double)(n_ctas - p) * td) / n_ctas);
  };
  int best = 0;
  double best_t = 1e30;
  for (int p = 0; p < n_ctas; p += 2) {
    const double t = step_time(p);
    if (t < best_t - 1e-9) {
      best_t = t;
      best = p;
    }
  }
  if (wide) return best;
  int lo = -1, hi = best;
  for (int p = 0; p < n_ctas; p += 2) {
    if (step_time(p) <= best_t * 1.002) {
      if (lo < 0) lo = p;
      hi = p;
    }
  }
  return ((lo + hi) / 2) & ~1;
}

int run_step(ts_ctx* c, const ts_step* st, void* cuda_stream, bool attention) {
  int64_t n_tokens = 0, n_prefill = 0;
  int n_decode = 0;
  int rc = validate(c, st, attention, true, &n_tokens, &n_decode, &n_prefill);
  if (rc != TS_OK) return rc;
  if (st->n_rows == 0) return TS_OK;
  if (!aligned16(st->k_new) || !aligned16(st->v_new)) return TS_ERR_INVALID;
  if (attention && (!aligned16(st->q) || !aligned16(st->out))) return TS_ERR_INVALID;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (attention) plan(c, st);
  rc = ensure_cuda(c, stream);
  if (rc != TS_OK) return rc;
  int n_slot_deltas = 0;
  rc = sync_tables(c, st, stream, &n_slot_deltas);
  if (rc != TS_OK) return rc;
  const int n_items = attention ? (int)c->items.size() : 0;
  const int n_combines = attention ? (int)c->combines.size() : 0;
  rc = upload_meta(c, st, n_items, n_combines, n_slot_deltas, stream);
  if (rc != TS_OK) return rc;
  commit_table_sync(c);
  ts::StepDevice d;
  fill_device(c, st, n_tokens, &d);
  d.n_items = n_items;
  d.n_combines = n_combines;
  cudaEvent_t* pe = nullptr;
  if (attention && c->profiling) {
    if (c->prof_used + 5 > c->prof_events.size()) {
      for (int i = 0; i < 5; ++i) {
        cudaEvent_t e;
        TS_CUDA(c, cudaEventCreate(&e));
        c->prof_events.push_back(e);
      }
    }
    pe = c->prof_events.data() + c->prof_used;
    c->prof_used += 5;
    c->prof_mixed.push_back(0);
    TS_CUDA(c, cudaEventRecord(pe[0], stream));
  }
  // head_dim 128 steps with prefill tiles: the mixed kernel appends the new K/V itself
  const bool append_in_kernel = attention && c->n_prefill_items > 0 && c->cfg.head_dim == 128;
  // decode rows of decode-only steps and of head_dim 128 steps: the unit that reads a row's last
  // page writes the row's new token into it
  const bool append_in_decode =
      attention && n_items > c->n_prefill_items && (c->n_prefill_items == 0 || append_in_kernel);
  d.append_in_decode = append_in_decode;
  if (!append_in_kernel && !append_in_decode) {
    TS_CUDA(c, ts::launch_kv_append(d, stream));
    ++c->cnt.kernel_launches;
  }
  if (attention) {
    if (pe) TS_CUDA(c, cudaEventRecord(pe[1], stream));
    d.n_prefill_items = c->n_prefill_items;
    bool decode_launched = false;
    if (c->n_prefill_items > 0) {
      if (c->cfg.head_dim == 128) {
        CUtensorMap q_map;
        rc = make_q_map(c, st->q, n_tokens, &q_map);
        if (rc != TS_OK) return rc;
        // One persistent launch: CTAs [0, p) take prefill tiles, the others run the decode
        // splits first and then help with the tiles (decode rows ride along when G <= 8).
        const long long pf_units = (long long)c->n_prefill_items * c->cfg.n_kv_heads;
        const long long dec_units = (long long)(n_items - c->n_prefill_items) * c->cfg.n_kv_heads;
        const bool fuse = dec_units > 0 && c->G <= 8 && c->cfg.mixed_prefill_ctas >= 0;
        int n_ctas = (int)std::min<long long>(c->n_sms, pf_units + (fuse ? dec_units : 0));
        int p = n_ctas;
        if (fuse) {
          if (c->cfg.mixed_prefill_ctas > 0) {
            p = c->cfg.mixed_prefill_ctas;
          } else {
            double pairs = 0.0, bytes = 0.0;
            for (int i = 0; i < c->n_prefill_items; ++i) pairs += ceil_div(c->items[i].k_end, 128);
            for (int i = c->n_prefill_items; i < n_items; ++i)
              bytes += (double)(c->items[i].k_end - c->items[i].k_begin);
            bytes *= 2.0 * c->cfg.n_kv_heads * c->cfg.head_dim * 2.0;
            p = choose_prefill_ctas(c, n_ctas, pairs * c->cfg.n_kv_heads, (double)pf_units, bytes, (double)dec_units,
                                    (double)n_prefill);
          }
          p = (int)std::min<long long>(p, pf_units);
          p = std::min(p, n_ctas - 1);                         // at least one CTA runs the decode splits
          p = std::max(p, n_ctas - (int)std::min<long long>(dec_units, n_ctas));   // no CTA without a decode unit
          decode_launched = true;
        }
        if (pe) c->prof_mixed.back() = decode_launched;
        // every CTA appends a share of the prefill rows' tokens (in a CTA that streams decode rows
        // first its loader warpgroup does, so the page stream starts with the kernel), but only a
        // CTA about to start on prefill work waits for all of them
        d.append_ctas = n_ctas;
        d.append_arrivals = d.append_ctas + ((c->cfg.debug_flags & TS_DEBUG_LOSE_APPEND_ARRIVAL) ? 1 : 0);
        TS_CUDA(c, ts::launch_mixed(d, q_map, c->kv_map, c->kv_tile_map, n_ctas, p, stream));
      } else {
        ts::StepDevice dp = d;
        dp.n_items = c->n_prefill_items;
        TS_CUDA(c, ts::launch_attention(dp, stream));
      }
      ++c->cnt.kernel_launches;
    }
    if (pe) TS_CUDA(c, cudaEventRecord(pe[2], stream));
    if (n_items > c->n_prefill_items && !decode_launched) {
      TS_CUDA(c, ts::launch_decode(d, c->kv_map, c->n_sms, stream));
      ++c->cnt.kernel_launches;
    }
    if (pe) TS_CUDA(c, cudaEventRecord(pe[3], stream));
    if (n_combines > 0 && !decode_launched) {      // the mixed launch merges its own splits
      TS_CUDA(c, ts::launch_combine(d, stream));
      ++c->cnt.kernel_launches;
    }
    if (pe) TS_CUDA(c, cudaEventRecord(pe[4], stream));
    ++c->cnt.steps;
    c->cnt.prefill_tokens += (uint64_t)n_prefill;
    c->cnt.decode_tokens += (uint64_t)n_decode;
  }
  rc = release_meta(c, stream);
  if (rc != TS_OK) return rc;
  if (!(st->flags & TS_STEP_KEEP_LEN)) {
    for (int r = 0; r < st->n_rows; ++r) c->slots[st->slot[r]].n_tokens += st->q_len[r];
  }
  return TS_OK;
}

}  // namespace

namespace ts {
int ctx_view(ts_ctx* c, cudaStream_t stream, CtxView* out) {
  if (!c || !out) return TS_ERR_INVALID;
  const int rc = ensure_cuda(c, stream);
  if (rc != TS_OK) return rc;
  out->cfg = &c->cfg;
  out->n_sms = c->n_sms;
  out->encode_fn = c->encode_fn;
  out->status = (int32_t*)((char*)c->cfg.workspace + c->L.off_status);
  out->wait_cycles = c->cfg.wait_limit_cycles > 0 ? (long long)c->cfg.wait_limit_cycles : kWaitCycles;
  out->max_tokens = c->L.max_tokens;
  return TS_OK;
}
}  // namespace ts

extern "C" {

size_t ts_pool_bytes(const ts_config* cfg) {
  if (!shape_ok(cfg)) return 0;
  return (size_t)cfg->n_pages * 2 * cfg->n_kv_heads * cfg->page_size * cfg->head_dim * 2;
}

size_t ts_workspace_bytes(const ts_config* cfg) {
  if (!shape_ok(cfg)) return 0;
  Layout L;
  compute_layout(cfg, &L);
  return L.total;
}

int ts_create(const ts_config* cfg, ts_ctx** out) {
  if (!out) return TS_ERR_INVALID;
  *out = nullptr;
  if (!cfg) return TS_ERR_INVALID;
  if (!shape_ok(cfg)) return TS_ERR_UNSUPPORTED;
  if (cfg->reserved_pages > cfg->n_pages) return TS_ERR_INVALID;
  if (cfg->debug_flags & ~TS_DEBUG_LOSE_APPEND_ARRIVAL) return TS_ERR_INVALID;
  if ((cfg->debug_flags & TS_DEBUG_LOSE_APPEND_ARRIVAL) &&
      (cfg->wait_limit_cycles <= 0 || cfg->wait_limit_cycles > 50000000))
    return TS_ERR_INVALID;    // a wait that is meant to run out must be short
  Layout L;
  compute_layout(cfg, &L);
  if (cfg->kv_pool && cfg->kv_pool_bytes < ts_pool_bytes(cfg)) return TS_ERR_WORKSPACE;
  if (cfg->workspace && cfg->workspace_bytes < L.total) return TS_ERR_WORKSPACE;
  if (((uintptr_t)cfg->kv_pool | (uintptr_t)cfg->workspace) & (kAlign - 1)) return TS_ERR_INVALID;
  ts_ctx* c = new (std::nothrow) ts_ctx();
  if (!c) return TS_ERR_INVALID;
  c->cfg = *cfg;
  c->L = L;
  c->G = cfg->n_q_heads / cfg->n_kv_heads;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  c->table.assign((size_t)cfg->max_requests * cfg->max_pages_per_req, -1);
  c->slots.assign(cfg->max_requests, Slot());
  c->page_owner.assign(cfg->n_pages, -1);
  c->free_pages.resize(cfg->n_pages);
  for (int i = 0; i < cfg->n_pages; ++i) c->free_pages[i] = cfg->n_pages - 1 - i;  // page 0 on top
  if (cfg->alloc_shuffle_seed) {
    uint64_t s = cfg->alloc_shuffle_seed;
    for (int i = cfg->n_pages - 1; i > 0; --i) {
      const int j = (int)(splitmix64(s) % (uint64_t)(i + 1));
      std::swap(c->free_pages[i], c->free_pages[j]);
    }
  }
  c->free_slots.resize(cfg->max_requests);
  for (int i = 0; i < cfg->max_requests; ++i) c->free_slots[i] = cfg->max_requests - 1 - i;
  std::memset(&c->cnt, 0, sizeof c->cnt);
  *out = c;
  return TS_OK;
}

int ts_destroy(ts_ctx* c) {
  if (!c) return TS_ERR_INVALID;
  if (c->cuda_ready) {
    cudaSetDevice(c->cfg.device);
    for (int i = 0; i < kRing; ++i) {
      if (c->ring[i].in_flight) cudaEventSynchronize(c->ring[i].ev);
      if (c->ring[i].ev) cudaEventDestroy(c->ring[i].ev);
      if (c->ring[i].host) cudaFreeHost(c->ring[i].host);
      if (c->meta[i].copy_in_flight) cudaEventSynchronize(c->meta[i].copied);
      if (c->meta[i].read_in_flight) cudaEventSynchronize(c->meta[i].consumed);
      if (c->meta[i].copied) cudaEventDestroy(c->meta[i].copied);
      if (c->meta[i].consumed) cudaEventDestroy(c->meta[i].consumed);
      if (c->meta[i].host) cudaFreeHost(c->meta[i].host);
    }
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    if (c->up_stream) {
      cudaStreamSynchronize(c->up_stream);
      cudaStreamDestroy(c->up_stream);
    }
    if (c->down_stream) {
      cudaStreamSynchronize(c->down_stream);
      cudaStreamDestroy(c->down_stream);
    }
    for (int i = 0; i < kStageSets; ++i) {
      if (c->up_done[i]) cudaEventDestroy(c->up_done[i]);
      if (c->step_done[i]) cudaEventDestroy(c->step_done[i]);
      if (c->down_done[i]) cudaEventDestroy(c->down_done[i]);
    }
  }
  for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
  delete c;
  return TS_OK;
}

int ts_request_add(ts_ctx* c, int64_t req_id, int32_t prompt_len, int32_t expected_output_len,
                   int32_t* slot_out) {
  if (!c || !slot_out || prompt_len < 0) return TS_ERR_INVALID;
  if (c->free_slots.empty()) return TS_ERR_NO_SLOT;
  const int slot = c->free_slots.back();
  c->free_slots.pop_back();
  Slot& s = c->slots[slot];
  s = Slot();
  s.live = true;
  s.req_id = req_id;
  s.prompt_len = prompt_len;
  s.expected_output_len = expected_output_len;
  *slot_out = slot;
  return TS_OK;
}

int ts_alloc_pages(ts_ctx* c, int32_t slot, int32_t total_tokens, int32_t for_prefill) {
  if (!c || !slot_ok(c, slot) || total_tokens < 0) return TS_ERR_INVALID;
  Slot& s = c->slots[slot];
  const int want = ceil_div(total_tokens, c->cfg.page_size);
  if (want <= s.n_pages) return TS_OK;
  if (want > c->cfg.max_pages_per_req) return TS_ERR_TABLE_SHORT;
  const int need = want - s.n_pages;
  const int64_t usable = (int64_t)c->free_pages.size() - (for_prefill ? 0 : c->cfg.reserved_pages);
  if (need > usable) return TS_ERR_NO_PAGES;
  int32_t* row = table_row(c, slot);
  for (int i = 0; i < need; ++i) {
    const int32_t p = c->free_pages.back();
    c->free_pages.pop_back();
    c->page_owner[p] = slot;
    row[s.n_pages++] = p;
  }
  return TS_OK;
}

int ts_alloc_step(ts_ctx* c, const ts_step* st) {
  if (!c || !st || st->n_rows < 0) return TS_ERR_INVALID;
  if (st->n_rows > 0 && (!st->slot || !st->q_len || !st->ctx_len)) return TS_ERR_INVALID;
  for (int r = 0; r < st->n_rows; ++r) {
    if (st->q_len[r] < 1 || st->ctx_len[r] < 0) return TS_ERR_INVALID;
    const int rc = ts_alloc_pages(c, st->slot[r], st->ctx_len[r] + st->q_len[r], st->q_len[r] > 1);
    if (rc != TS_OK) return rc;
  }
  return TS_OK;
}

int ts_block_table(ts_ctx* c, int32_t slot, const int32_t** pages_out, int32_t* n_pages_out,
                   int32_t* n_tokens_out) {
  if (!c || !slot_ok(c, slot)) return TS_ERR_INVALID;
  if (pages_out) *pages_out = table_row(c, slot);
  if (n_pages_out) *n_pages_out = c->slots[slot].n_pages;
  if (n_tokens_out) *n_tokens_out = c->slots[slot].n_tokens;
  return TS_OK;
}

int ts_block_table_set(ts_ctx* c, int32_t slot, const int32_t* pages, int32_t n_pages) {
  if (!c || !slot_ok(c, slot) || n_pages < 0 || (n_pages > 0 && !pages)) return TS_ERR_INVALID;
  if (n_pages > c->cfg.max_pages_per_req) return TS_ERR_TABLE_SHORT;
  // every requested page must be free or already ours, and listed once
  ++c->stamp;
  std::vector<char> seen;  // small helper bitmap only for this call
  seen.assign(c->cfg.n_pages, 0);
  for (int i = 0; i < n_pages; ++i) {
    const int32_t p = pages[i];
    if (p < 0 || p >= c->cfg.n_pages || seen[p]) return TS_ERR_INVALID;
    if (c->page_owner[p] != -1 && c->page_owner[p] != slot) return TS_ERR_INVALID;
    seen[p] = 1;
  }
  release_pages(c, slot);
  // remove the requested pages from the free stack, keeping the order of the rest
  size_t w = 0;
  for (size_t i = 0; i < c->free_pages.size(); ++i)
    if (!seen[c->free_pages[i]]) c->free_pages[w++] = c->free_pages[i];
  c->free_pages.resize(w);
  Slot& s = c->slots[slot];
  int32_t* row = table_row(c, slot);
  for (int i = 0; i < n_pages; ++i) {
    row[i] = pages[i];
    c->page_owner[pages[i]] = slot;
  }
  s.n_pages = n_pages;
  s.synced_pages = 0;
  if (s.n_tokens > n_pages * c->cfg.page_size) s.n_tokens = n_pages * c->cfg.page_size;
  return TS_OK;
}

int ts_request_free(ts_ctx* c, int32_t slot) {
  if (!c || !slot_ok(c, slot)) return TS_ERR_INVALID;
  Slot& s = c->slots[slot];
  c->cnt.released_tokens += (uint64_t)s.n_tokens;
  c->cnt.released_requests += 1;
  release_pages(c, slot);
  s.live = false;
  s.n_tokens = 0;
  c->free_slots.push_back(slot);
  return TS_OK;
}

int ts_request_set_len(ts_ctx* c, int32_t slot, int32_t n_tokens) {
  if (!c || !slot_ok(c, slot) || n_tokens < 0) return TS_ERR_INVALID;
  if ((int64_t)n_tokens > (int64_t)c->slots[slot].n_pages * c->cfg.page_size) return TS_ERR_TABLE_SHORT;
  c->slots[slot].n_tokens = n_tokens;
  return TS_OK;
}

int ts_kv_append(ts_ctx* c, const ts_step* st, void* cuda_stream) {
  return run_step(c, st, cuda_stream, false);
}

int ts_mixed_step(ts_ctx* c, const ts_step* st, void* cuda_stream) {
  return run_step(c, st, cuda_stream, true);
}

int ts_mixed_step_host(ts_ctx* c, const ts_step* st, void* cuda_stream) {
  if (!c || !st) return TS_ERR_INVALID;
  if (c->cfg.chunk_size <= 0) return TS_ERR_INVALID;
  if (st->n_rows == 0) return TS_OK;
  if (st->n_rows < 0 || !st->q_len) return TS_ERR_INVALID;
  int64_t n = 0;
  for (int r = 0; r < st->n_rows; ++r) {
    if (st->q_len[r] < 1) return TS_ERR_INVALID;
    n += st->q_len[r];
    if (n > c->L.max_tokens) return TS_ERR_BUDGET;
  }
  if (!st->q || !st->k_new || !st->v_new || !st->out) return TS_ERR_INVALID;
  if (!c->cfg.workspace) return cuda_fail(c, cudaErrorInvalidDevicePointer);
  {
    // the step's own checks first: a step that would be refused must not start copying
    int64_t nt = 0, np = 0;
    int nd = 0;
    const int vrc = validate(c, st, true, true, &nt, &nd, &np);
    if (vrc != TS_OK) return vrc;
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  TS_CUDA(c, cudaSetDevice(c->cfg.device));
  if (!c->up_stream) {
    TS_CUDA(c, cudaStreamCreateWithFlags(&c->up_stream, cudaStreamNonBlocking));
    TS_CUDA(c, cudaStreamCreateWithFlags(&c->down_stream, cudaStreamNonBlocking));
    for (int i = 0; i < kStageSets; ++i) {
      TS_CUDA(c, cudaEventCreateWithFlags(&c->up_done[i], cudaEventDisableTiming));
      TS_CUDA(c, cudaEventCreateWithFlags(&c->step_done[i], cudaEventDisableTiming));
      TS_CUDA(c, cudaEventCreateWithFlags(&c->down_done[i], cudaEventDisableTiming));
    }
  }
  // The staging sets take turns. Upload: once the set's previous result has gone down (its
  // step is then done with the inputs too). Step: on the caller's stream, after the upload.
  // Download: after the step. Without TS_STEP_HOST_ASYNC the caller's stream then waits for the
  // downloads and the call for the stream; with it nothing waits, so the following calls'
  // uploads and kernels overlap this step's download, and ts_host_fence orders the stream
  // behind the downloads when the caller wants the results.
  const int b = (int)(c->host_steps % kStageSets);
  char* ws = (char*)c->cfg.workspace + c->L.off_stage + (size_t)b * c->L.stage_set_bytes;
  void* dq = ws;
  void* dout = ws + c->L.stage_q_bytes;
  void* dk = ws + 2 * c->L.stage_q_bytes;
  void* dv = ws + 2 * c->L.stage_q_bytes + c->L.stage_kv_bytes;
  const size_t qb = (size_t)n * c->cfg.n_q_heads * c->cfg.head_dim * 2;
  const size_t kb = (size_t)n * c->cfg.n_kv_heads * c->cfg.head_dim * 2;
  if (c->stage_used[b]) TS_CUDA(c, cudaStreamWaitEvent(c->up_stream, c->down_done[b], 0));
  TS_CUDA(c, cudaMemcpyAsync(dq, st->q, qb, cudaMemcpyHostToDevice, c->up_stream));
  TS_CUDA(c, cudaMemcpyAsync(dk, st->k_new, kb, cudaMemcpyHostToDevice, c->up_stream));
  TS_CUDA(c, cudaMemcpyAsync(dv, st->v_new, kb, cudaMemcpyHostToDevice, c->up_stream));
  TS_CUDA(c, cudaEventRecord(c->up_done[b], c->up_stream));
  TS_CUDA(c, cudaStreamWaitEvent(stream, c->up_done[b], 0));
  ts_step dev = *st;
  dev.q = dq;
  dev.k_new = dk;
  dev.v_new = dv;
  dev.out = dout;
  const int rc = run_step(c, &dev, cuda_stream, true);
  if (rc != TS_OK) {
    cudaStreamSynchronize(c->up_stream);  // the input copies may still be reading the caller's buffers
    return rc;
  }
  TS_CUDA(c, cudaEventRecord(c->step_done[b], stream));
  TS_CUDA(c, cudaStreamWaitEvent(c->down_stream, c->step_done[b], 0));
  TS_CUDA(c, cudaMemcpyAsync(st->out, dout, qb, cudaMemcpyDeviceToHost, c->down_stream));
  TS_CUDA(c, cudaEventRecord(c->down_done[b], c->down_stream));
  c->stage_used[b] = true;
  ++c->host_steps;
  if (!(st->flags & TS_STEP_HOST_ASYNC)) {
    const int rc2 = ts_host_fence(c, cuda_stream);
    if (rc2 != TS_OK) return rc2;
    TS_CUDA(c, cudaStreamSynchronize(stream));
  }
  return TS_OK;
}

int ts_host_fence(ts_ctx* c, void* cuda_stream) {
  if (!c) return TS_ERR_INVALID;
  if (!c->up_stream) return TS_OK;            // no host step has been issued
  TS_CUDA(c, cudaSetDevice(c->cfg.device));
  for (int i = 0; i < kStageSets; ++i)
    if (c->stage_used[i]) TS_CUDA(c, cudaStreamWaitEvent((cudaStream_t)cuda_stream, c->down_done[i], 0));
  return TS_OK;
}

int ts_velocity(ts_ctx* c, ts_velocity_counters* out) {
  if (!c || !out) return TS_ERR_INVALID;
  *out = c->cnt;
  out->pages_free = c->free_pages.size();
  out->pages_in_use = (uint64_t)c->cfg.n_pages - c->free_pages.size();
  return TS_OK;
}

int ts_report_step_time(ts_ctx* c, double seconds) {
  if (!c || !(seconds >= 0.0)) return TS_ERR_INVALID;
  c->cnt.busy_seconds += seconds;
  return TS_OK;
}

int ts_profile_enable(ts_ctx* c, int enable) {
  if (!c) return TS_ERR_INVALID;
  c->profiling = enable != 0;
  return TS_OK;
}

int ts_profile_read(ts_ctx* c, void* cuda_stream, ts_profile* out) {
  if (!c || !out) return TS_ERR_INVALID;
  std::memset(out, 0, sizeof *out);
  if (c->prof_used == 0) return TS_OK;
  TS_CUDA(c, cudaSetDevice(c->cfg.device));
  TS_CUDA(c, cudaStreamSynchronize((cudaStream_t)cuda_stream));
  for (size_t i = 0; i + 5 <= c->prof_used; i += 5) {
    float t[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k = 0; k < 4; ++k)
      TS_CUDA(c, cudaEventElapsedTime(&t[k], c->prof_events[i + k], c->prof_events[i + k + 1]));
    out->append_ms += t[0];
    if (c->prof_mixed[i / 5]) {
      out->mixed_ms += t[1];
      out->mixed_steps += 1;
    } else {
      out->prefill_ms += t[1];
    }
    out->decode_ms += t[2];
    out->combine_ms += t[3];
    out->steps += 1;
  }
  c->prof_used = 0;
  c->prof_mixed.clear();
  return TS_OK;
}

int32_t ts_prefill_budget(const ts_ctx* c, int32_t decode_batch_size) {
  if (!c || decode_batch_size < 0) return 0;
  return std::max(c->cfg.chunk_size - decode_batch_size, 0);
}

int32_t ts_pick_chunk_size(const int32_t* prefill_tokens, const double* iteration_seconds, int32_t n,
                           int32_t decode_batch_size, double tpot_slo_s) {
  if (!prefill_tokens || !iteration_seconds || n <= 0 || decode_batch_size < 0 || !(tpot_slo_s > 0.0))
    return TS_ERR_INVALID;
  for (int i = 0; i < n; ++i) {
    if (prefill_tokens[i] <= 0 || (i > 0 && prefill_tokens[i] <= prefill_tokens[i - 1])) return TS_ERR_INVALID;
    if (!(iteration_seconds[i] >= 0.0)) return TS_ERR_INVALID;
  }
  int32_t best = 0;
  for (int i = 0; i < n; ++i) {                 // the profile stops counting at the first violation
    if (iteration_seconds[i] > tpot_slo_s) break;
    best = prefill_tokens[i] + decode_batch_size;
  }
  return best;
}

double ts_convertible_prefill_velocity(int32_t chunk_size, double decode_batch_size, double tpot_slo_s) {
  if (!(tpot_slo_s > 0.0) || !(decode_batch_size >= 0.0) || (double)chunk_size <= decode_batch_size) return 0.0;
  return ((double)chunk_size - decode_batch_size) / tpot_slo_s;
}

double ts_reserved_memory(double prefill_velocity, double mem_per_token, double ttft_slo_s) {
  if (!(prefill_velocity > 0.0) || !(mem_per_token > 0.0) || !(ttft_slo_s > 0.0)) return 0.0;
  return prefill_velocity * mem_per_token * ttft_slo_s;
}

int32_t ts_reserved_pages(double prefill_velocity, double ttft_slo_s, int32_t page_size) {
  if (!(prefill_velocity > 0.0) || !(ttft_slo_s > 0.0) || page_size <= 0) return 0;
  const double pages = std::ceil(prefill_velocity * ttft_slo_s / (double)page_size - 1e-9);
  return pages > 2147483647.0 ? 2147483647 : (int32_t)pages;
}

int32_t ts_prefiller_instances(double token_rate, double prefill_velocity, double network_velocity) {
  if (!(prefill_velocity > 0.0) || !(network_velocity > 0.0)) return TS_ERR_INVALID;
  if (!(token_rate > 0.0)) return 0;
  const double n = std::ceil(token_rate / std::min(prefill_velocity, network_velocity));
  return n > 2147483647.0 ? 2147483647 : (int32_t)n;
}

double ts_decoder_demand(const double* token_rate, const double* velocity, int32_t n_buckets) {
  if (!token_rate || !velocity || n_buckets <= 0) return -1.0;
  double total = 0.0;
  for (int b = 0; b < n_buckets; ++b) {
    if (!(token_rate[b] >= 0.0) || !(velocity[b] > 0.0)) return -1.0;
    total += token_rate[b] / velocity[b];
  }
  return total;
}

int32_t ts_regular_decoders(double decoder_demand, int32_t convertible_decoders) {
  if (!(decoder_demand > 0.0)) return 0;
  const double need = std::ceil(decoder_demand) - (double)std::max(convertible_decoders, 0);
  return need <= 0.0 ? 0 : need > 2147483647.0 ? 2147483647 : (int32_t)need;
}

int32_t ts_route_prefill(const double* prefiller_inflight_tokens, const double* prefiller_velocity,
                         int32_t n_prefillers, const double* convertible_inflight_tokens,
                         const double* convertible_prefill_velocity, int32_t n_convertible, double slo_s,
                         int32_t* kind_out) {
  if (!kind_out || n_prefillers < 0 || n_convertible < 0) return TS_ERR_INVALID;
  if (n_prefillers > 0 && (!prefiller_inflight_tokens || !prefiller_velocity)) return TS_ERR_INVALID;
  if (n_convertible > 0 && (!convertible_inflight_tokens || !convertible_prefill_velocity)) return TS_ERR_INVALID;
  for (int i = 0; i < n_prefillers; ++i)
    if (!(prefiller_inflight_tokens[i] >= 0.0) || !(prefiller_velocity[i] > 0.0)) return TS_ERR_INVALID;
  for (int i = 0; i < n_convertible; ++i)
    if (!(convertible_inflight_tokens[i] >= 0.0) || !(convertible_prefill_velocity[i] > 0.0)) return TS_ERR_INVALID;
  for (int i = 0; i < n_prefillers; ++i) {          // first round: the prefillers, in order
    if (prefiller_inflight_tokens[i] / prefiller_velocity[i] <= slo_s) {
      *kind_out = TS_ROUTE_PREFILLER;
      return i;
    }
  }
  for (int i = 0; i < n_convertible; ++i) {         // second round: the Convertible Decoders
    if (convertible_inflight_tokens[i] / convertible_prefill_velocity[i] <= slo_s) {
      *kind_out = TS_ROUTE_CONVERTIBLE;
      return i;
    }
  }
  *kind_out = TS_ROUTE_QUEUE;
  return 0;
}

int ts_plan_step(ts_ctx* c, const ts_step* st, int32_t* items, int32_t items_capacity,
                 int32_t* n_items_out) {
  if (!n_items_out) return TS_ERR_INVALID;
  *n_items_out = 0;
  int64_t n_tokens = 0, n_prefill = 0;
  int n_decode = 0;
  // q/out are not needed for planning: validate as an append-only step, then apply the budget.
  int rc = validate(c, st, false, false, &n_tokens, &n_decode, &n_prefill);
  if (rc != TS_OK) return rc;
  if (c->cfg.chunk_size > 0 && n_prefill + n_decode > c->cfg.chunk_size) return TS_ERR_BUDGET;
  if (n_tokens > c->L.max_tokens) return TS_ERR_BUDGET;
  plan(c, st);
  *n_items_out = (int32_t)c->items.size();
  if (items) {
    if (items_capacity < (int32_t)c->items.size()) return TS_ERR_INVALID;
    std::memcpy(items, c->items.data(), c->items.size() * sizeof(WorkItem));
  }
  return TS_OK;
}

int ts_last_device_status(ts_ctx* c, void* cuda_stream, int32_t* status_out) {
  if (!c || !status_out) return TS_ERR_INVALID;
  *status_out = 0;
  if (!c->cfg.workspace) return cuda_fail(c, cudaErrorInvalidDevicePointer);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  TS_CUDA(c, cudaSetDevice(c->cfg.device));
  if (!c->status_cleared) return TS_OK;  // nothing has run yet
  int32_t* dev = (int32_t*)((char*)c->cfg.workspace + c->L.off_status);
  TS_CUDA(c, cudaMemcpyAsync(status_out, dev, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  TS_CUDA(c, cudaStreamSynchronize(stream));
  // a clean status clears only its word; after a failure the kernels' counters next to it may be
  // stale as well, so the whole block goes back to zero
  TS_CUDA(c, cudaMemsetAsync(dev, 0, *status_out ? kAlign : sizeof(int32_t), stream));
  TS_CUDA(c, cudaStreamSynchronize(stream));
  return (*status_out & TS_DEV_TIMEOUT) ? TS_ERR_DEVICE_TIMEOUT : TS_OK;
}

int ts_last_cuda_error(const ts_ctx* c) { return c ? c->last_cuda_error : 0; }

const char* ts_strerror(int code) {
  switch (code) {
    case TS_OK: return "ok";
    case TS_ERR_INVALID: return "invalid argument";
    case TS_ERR_NO_PAGES: return "not enough free pages";
    case TS_ERR_NO_SLOT: return "no free request slot";
    case TS_ERR_TABLE_SHORT: return "block table does not cover the tokens";
    case TS_ERR_BUDGET: return "step exceeds the chunk size";
    case TS_ERR_CUDA: return "CUDA runtime error";
    case TS_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case TS_ERR_UNSUPPORTED: return "unsupported shape";
    case TS_ERR_WORKSPACE: return "pool or workspace too small";
    default: return "unknown error";
  }
}

}  // extern "C"
