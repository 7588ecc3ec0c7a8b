// Internal interface between the host scheduler (ts_host.cpp) and the kernels (ts_kernels.cu).
// Nothing here is part of the public ABI.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tokenscale.h"

#include <utility>

namespace ts {

constexpr int kPageSize = 16;
constexpr int kKeysPerTile = 64;     // keys staged per pipeline stage of the attention kernel
constexpr int kPackedRowsPerTile = 64;  // (token, head) rows of a prefill tile, head_dim 64 path
constexpr int kPackedRowsTc = 128;      // (token, head) rows of a prefill tile, tcgen05 path (head_dim 128)
constexpr long long kWaitCycles = 2000000000LL;  // default limit of a bounded wait: about one second at boost clock
constexpr int kMaxGroup = 16;        // query heads per KV head a decode work item can hold

// One unit of attention work; the KV head comes from the grid.
// Inside a kernel the (token, head-in-group) pairs of an item are "packed rows":
//   packed row pr -> token q_begin + pr / G, query head kv_head*G + pr % G.
struct WorkItem {
  int32_t row;          // index into the step's rows
  int32_t kind;         // 0: decode split, 1: prefill tile
  int32_t q_begin;      // first new token of the row this item covers (decode: 0)
  int32_t q_count;      // tokens in this item (decode: 1; prefill: tile_rows / G at most)
  int32_t k_begin;      // first key position (multiple of kKeysPerTile)
  int32_t k_end;        // one past the last key position any row of the item may see
  int32_t partial_slot; // >= 0: write (m, l, acc) partials there; -1: write out directly
  int32_t reserved;
};
static_assert(sizeof(WorkItem) == 32, "WorkItem is 8 int32");

// One entry per token whose splits must be merged.
struct CombineItem {
  int32_t token;         // flat token index of the step
  int32_t first_partial; // first partial slot
  int32_t n_splits;
  int32_t reserved;
};

struct TableDelta {
  int32_t slot, index, page;
};

// Device pointers of one step, all inside the caller's workspace unless noted.
struct StepDevice {
  // static
  uint16_t* pool;          // caller's KV pool
  int32_t* table;          // [max_requests][max_pages_per_req]
  int32_t* status;         // device status word
  int32_t* pf_queue;       // counters of the mixed kernel, all zero between launches (its last CTA
                           // to leave resets them): [0] next prefill work unit, [1] decode CTAs
                           // that have finished their units, [2] CTAs that have appended their
                           // share of the new tokens, [3] CTAs that have left
  float* part_acc;         // [max_partials][Hq][D]
  float* part_ml;          // [max_partials][Hq][2]  (running max in log2 units, sum)
  // per step (device meta area)
  const int32_t* row_slot;
  const int32_t* row_ctx;
  const int32_t* row_qlen;
  const int32_t* row_tok0; // [n_rows + 1] prefix sums of q_len
  const WorkItem* items;
  const CombineItem* combines;
  // step tensors
  const uint16_t* q;
  const uint16_t* k_new;
  const uint16_t* v_new;
  uint16_t* out;
  // shape
  int32_t n_rows, n_tokens, n_items, n_combines;
  int32_t n_prefill_items;  // items[0, n_prefill_items) are prefill tiles, the rest decode splits
  int32_t append_in_decode; // != 0: the decode units append their rows' new K/V themselves
  int32_t Hq, Hkv, D, n_pages, max_pages_per_req, max_requests;
  float scale_log2;        // softmax scale * log2(e)
  long long wait_cycles;   // limit of every bounded wait of the step's kernels, in clock cycles
  int32_t append_ctas;     // CTAs of the mixed kernel that append the new tokens of the prefill rows: all of them
  int32_t append_arrivals; // what the mixed kernel's CTAs wait for before their first prefill unit:
                           // append_ctas, or one more when ts_config.debug_flags asks for a wait that runs out
};

// Launchers. Each enqueues on `stream` and returns the launch's cudaError_t.
cudaError_t launch_table_update(int32_t* table, int max_pages_per_req, int max_requests, int32_t* status,
                                const TableDelta* deltas, int n_deltas, cudaStream_t stream);
cudaError_t launch_kv_append(const StepDevice& s, cudaStream_t stream);
cudaError_t launch_attention(const StepDevice& s, cudaStream_t stream);
cudaError_t launch_combine(const StepDevice& s, cudaStream_t stream);
// Decode splits items[n_prefill_items, n_items): persistent kernel, one CTA per SM, K/V pages by TMA
// through kv_map (5-D view of the pool: head_dim, slot, KV head, K|V, page; box 64 x 16 x 1 x 2 x 1).
// Prefill tiles items[0, n_prefill_items), head_dim 128: persistent tcgen05/TMEM kernel of n_ctas
// CTAs. The first n_prefill_ctas CTAs work on the prefill queue only; the others first run all
// decode splits (as launch_decode would, needs G <= 8) and then join the prefill queue. The
// kernel also appends the step's new K/V itself (no launch_kv_append before it). With
// n_prefill_ctas == n_ctas the decode splits are left to launch_decode. When it runs the decode
// splits it also merges them (no launch_combine needed).
// q_map views q as (head_dim, G, KV head, token), box 64 x G x 1 x 128/G. kv_tile_map is the pool
// view of kv_map with a box of one operand only (64 x 16 x 1 x 1 x 1): the prefill tiles' K/V copies.
cudaError_t launch_mixed(const StepDevice& s, const CUtensorMap& q_map, const CUtensorMap& kv_map,
                         const CUtensorMap& kv_tile_map, int n_ctas, int n_prefill_ctas, cudaStream_t stream);
cudaError_t launch_decode(const StepDevice& s, const CUtensorMap& kv_map, int n_sms, cudaStream_t stream);

// ---- the decoder layer around the attention step: GEMMs and small kernels (ts_gemm.cu, ts_layer_kernels.cu)
enum { GEMM_EPI_STORE = 0, GEMM_EPI_ROPE = 1, GEMM_EPI_SILU_MUL = 2 };
// C = A . B^T (+ R), A [M][K], B [N][K] bf16 K-major (their tensor maps travel beside this struct).
struct GemmArgs {
  int32_t M, N, K;
  int32_t epi;              // GEMM_EPI_*
  uint16_t* C;              // STORE: [M][ldc]; ROPE: the query heads [M][q_cols]; SILU_MUL: [M][ldc], ldc = N / 2
  const uint16_t* R;        // STORE: residual [M][ldc] added before rounding, or null
  int32_t ldc;
  // ROPE (fused QKV projection, head_dim 128): columns [0, q_cols) are query heads -> C, the next
  // kv_cols key heads -> C2, the last kv_cols value heads -> C3 (not rotated)
  int32_t q_cols, kv_cols;
  uint16_t* C2;
  uint16_t* C3;
  const int32_t* pos;       // [M] position of every token
  const float2* rope_table; // [max_position][64] (cos, sin) of pos * theta^(-2i/128)
  int32_t* status;          // device status word
  long long wait_cycles;    // limit of every bounded wait
};
// What the layer code needs to know of a context (ts_host.cpp fills it in; it also makes sure the
// context's CUDA set-up has run and its status word is cleared).
struct CtxView {
  const ts_config* cfg;
  int n_sms;
  void* encode_fn;          // cuTensorMapEncodeTiled
  int32_t* status;          // device status word of the context
  long long wait_cycles;
  int max_tokens;           // most tokens a step may hold
};
int ctx_view(ts_ctx* c, cudaStream_t stream, CtxView* out);
// Tile height (128 or 256 rows per CTA) that finishes an M x N product in the fewest tile-waves.
int gemm_tile_m(int M, int N, int n_sms);
cudaError_t launch_gemm(const GemmArgs& g, const CUtensorMap& a_map, const CUtensorMap& b_map, int tile_m, int n_sms,
                        cudaStream_t stream);
// out[row] = x[row] / sqrt(mean(x[row]^2) + eps) * gain, bf16 in and out, fp32 inside; width % 8 == 0
cudaError_t launch_rmsnorm(const uint16_t* x, const uint16_t* gain, uint16_t* out, int rows, int width, float eps,
                           cudaStream_t stream);
// table[p][i] = (cos, sin)(p * theta^(-2 i / 128)), p < max_position, i < 64 (computed in fp64)
cudaError_t launch_rope_table(float2* table, int max_position, float theta, cudaStream_t stream);
// dst row 256 b + r = gate row 128 b + r, dst row 256 b + 128 + r = up row 128 b + r (r < 128)
cudaError_t launch_pack_gate_up(const uint16_t* gate, const uint16_t* up, uint16_t* dst, int intermediate, int width,
                                cudaStream_t stream);

// Programmatic dependent launch: every kernel of a step is launched with the attribute that lets
// it become resident while its predecessor in the stream is still draining. Each kernel runs its
// set-up (shared-memory barriers, TMEM allocation, descriptor prefetch), then executes
// griddepcontrol.wait before it touches anything an earlier kernel may have written or may still
// be reading; launch latency and set-up thus overlap the predecessor's tail.
template <typename... Params, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#ifdef __CUDACC__
// Copies the K/V of the step's new tokens into their pages (Sec. 2.1): one warp per token at a time,
// warps `first_warp`, `first_warp + n_warps`, ... of the launch; a lane moves 16-byte chunks, eight
// loads in flight before the first store, and the source loads are issued before the block-table
// look-up they do not depend on. `rows` = a shared-memory copy of the step's row arrays made by
// stage_rows (the token -> row search and the row's slot and length then cost no global round trips).
// Slots and page ids are range checked; a bad one sets a status bit and skips the token.
__device__ __forceinline__ void stage_rows(const StepDevice& s, int32_t* rows, int tid, int n_threads) {
  const int n = s.n_rows + 1;                  // rows[0..n): first-token prefix sums, then ctx, then slot
  for (int i = tid; i < n; i += n_threads) {
    rows[i] = s.row_tok0[i];
    if (i < s.n_rows) {
      rows[n + i] = s.row_ctx[i];
      rows[2 * n + i] = s.row_slot[i];
    }
  }
}
__host__ __device__ inline size_t staged_rows_bytes(int n_rows) { return (size_t)3 * (n_rows + 1) * sizeof(int32_t); }
// One token: its K and V for all KV heads go to position t of the request in table row `slot`.
__device__ __forceinline__ void append_one(const StepDevice& s, int tok, int t, int slot, int lane) {
  const int cpr = s.D / 8;                      // chunks per (token, head) row
  const int per_tok = 2 * s.Hkv * cpr;
  const bool index_ok = (unsigned)slot < (unsigned)s.max_requests && (unsigned)(t >> 4) < (unsigned)s.max_pages_per_req;
  int page = -1;
  for (int base = 0; base < per_tok; base += 256) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int c = base + u * 32 + lane;
      if (c < per_tok) {
        const int kv = c / (s.Hkv * cpr);
        const int rem = c - kv * s.Hkv * cpr;
        const int head = rem / cpr, ch = rem % cpr;
        v[u] = *reinterpret_cast<const uint4*>((kv ? s.v_new : s.k_new) + ((size_t)tok * s.Hkv + head) * s.D + ch * 8);
      }
    }
    if (base == 0) {
      if (!index_ok) {
        if (lane == 0) atomicOr(s.status, TS_DEV_BAD_INDEX);
        break;
      }
      page = s.table[(size_t)slot * s.max_pages_per_req + (t >> 4)];
      if ((unsigned)page >= (unsigned)s.n_pages) {
        if (lane == 0) atomicOr(s.status, TS_DEV_BAD_PAGE);
        break;
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int c = base + u * 32 + lane;
      if (c < per_tok) {
        const int kv = c / (s.Hkv * cpr);
        const int rem = c - kv * s.Hkv * cpr;
        const int head = rem / cpr, ch = rem % cpr;
        uint16_t* dst = s.pool + ((((size_t)page * 2 + kv) * s.Hkv + head) * kPageSize + (t & 15)) * s.D + ch * 8;
        *reinterpret_cast<uint4*>(dst) = v[u];
      }
    }
  }
}
__device__ __forceinline__ void append_tokens(const StepDevice& s, const int32_t* rows, int first_warp, int n_warps,
                                              int lane) {
  const int n = s.n_rows + 1;
  const int32_t* row_start = rows;
  for (int tok = first_warp; tok < s.n_tokens; tok += n_warps) {
    int lo = 0, hi = s.n_rows;                  // row of this token: last r with row_start[r] <= tok
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (row_start[mid] <= tok) lo = mid; else hi = mid;
    }
    if (s.append_in_decode && row_start[lo + 1] - row_start[lo] == 1) continue;
    append_one(s, tok, rows[n + lo] + (tok - row_start[lo]), rows[2 * n + lo], lane);
  }
}
// The same for the tokens of the prefill work items only (they cover every token of every row with
// more than one new token exactly once, `tokens_per_item` at most each): nothing to stage and no
// search, the item names the row and the position. Warps `first_warp`, `first_warp + n_warps`, ...
__device__ __forceinline__ void append_prefill_items(const StepDevice& s, int tokens_per_item, int first_warp, int n_warps,
                                                     int lane) {
  const int total = s.n_prefill_items * tokens_per_item;
  for (int w = first_warp; w < total; w += n_warps) {
    const WorkItem it = s.items[w / tokens_per_item];
    const int j = w % tokens_per_item;
    if (j >= it.q_count) continue;
    append_one(s, s.row_tok0[it.row] + it.q_begin + j, it.k_end - it.q_count + j, s.row_slot[it.row], lane);
  }
}
// Log-sum-exp merge of the splits of one (token, head) for head_dim element d: the exact merge
//   m = max m_i,  l = sum l_i 2^(m_i - m),  O = sum acc_i 2^(m_i - m) / l
// over the partial slots [first_partial, first_partial + n_splits). Eight splits' loads are in
// flight at a time. Reads bypass L1 (the partials may have been written by another SM of the
// same launch).
__device__ __forceinline__ float merge_splits(const StepDevice& s, int first_partial, int n_splits, int h, int d) {
  const float* ml = s.part_ml + ((size_t)first_partial * s.Hq + h) * 2;
  const float* pa = s.part_acc + ((size_t)first_partial * s.Hq + h) * s.D + d;
  const size_t ml_stride = (size_t)s.Hq * 2, pa_stride = (size_t)s.Hq * s.D;
  float m = -__int_as_float(0x7f800000), l = 0.f, acc = 0.f;
  for (int base = 0; base < n_splits; base += 8) {
    float mi[8], li[8], ai[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const bool on = base + j < n_splits;
      mi[j] = on ? __ldcg(ml + (base + j) * ml_stride) : -__int_as_float(0x7f800000);
      li[j] = on ? __ldcg(ml + (base + j) * ml_stride + 1) : 0.f;
      ai[j] = on ? __ldcg(pa + (base + j) * pa_stride) : 0.f;
    }
    float mn = m;
#pragma unroll
    for (int j = 0; j < 8; ++j) mn = fmaxf(mn, mi[j]);
    const float keep = exp2f(m - mn);          // 0 on the first group (m = -inf)
    l *= keep;
    acc *= keep;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float w = exp2f(mi[j] - mn);       // absent split: exp2(-inf) = 0
      l += w * li[j];
      acc += w * ai[j];
    }
    m = mn;
  }
  return acc / l;
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
#endif

}  // namespace ts
