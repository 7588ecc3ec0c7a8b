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
  int32_t* pf_queue;       // [0] next prefill work unit of the step, [1] decode CTAs of the mixed
                           // kernel that have finished their units (both zeroed by the append kernel)
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
// n_prefill_ctas == n_ctas the decode splits are left to launch_decode. When it runs the decode
// splits it also merges them (no launch_combine needed).
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
