// Internal interface between the host scheduler (ts_host.cpp) and the kernels (ts_kernels.cu).
// Nothing here is part of the public ABI.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace ts {

constexpr int kPageSize = 16;
constexpr int kKeysPerTile = 64;     // keys staged per pipeline stage of the attention kernel
constexpr int kPackedRowsPerTile = 64;  // (token, head) rows of a prefill tile, head_dim 64 path
constexpr int kPackedRowsTc = 128;      // (token, head) rows of a prefill tile, tcgen05 path (head_dim 128)
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
  int32_t* pf_queue;       // next prefill work unit of the step (zeroed by the append kernel)
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
  int32_t Hq, Hkv, D, n_pages, max_pages_per_req, max_requests;
  float scale_log2;        // softmax scale * log2(e)
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
// decode splits (as launch_decode would, needs G <= 8) and then join the prefill queue. With
// n_prefill_ctas == n_ctas the decode splits are left to launch_decode.
// q_map views q as (head_dim, G, KV head, token), box 64 x G x 1 x 128/G.
cudaError_t launch_mixed(const StepDevice& s, const CUtensorMap& q_map, const CUtensorMap& kv_map, int n_ctas,
                         int n_prefill_ctas, cudaStream_t stream);
cudaError_t launch_decode(const StepDevice& s, const CUtensorMap& kv_map, int n_sms, cudaStream_t stream);

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
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
#endif

}  // namespace ts
