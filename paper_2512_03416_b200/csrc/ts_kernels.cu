// CUDA kernels (sm_100a) of the mixed paged-attention step:
//   table_update  - applies block-table deltas to the device copy of the tables
//   kv_append     - copies the step's new K/V into their pages (16-byte vector copies)
//   attention     - prefill tiles of head_dim 64 steps, and the kernel behind
//                   ts_decode_attention_static (decode work items): K/V pages staged in shared
//                   memory through a 3-stage cp.async ring, mma.sync bf16 MMAs with fp32 online
//                   softmax (warp-shuffle reductions). head_dim 128 steps run ts_mixed.cu and
//                   ts_decode.cu instead.
//   combine       - log-sum-exp merge of the decode splits
#include <cuda_bf16.h>
#include <math_constants.h>

#include "../../include/tokenscale.h"
#include "ts_internal.h"
#include "ts_ptx.h"

namespace ts {

namespace {

constexpr int kThreads = 128;  // 4 warps per attention CTA
constexpr int kStages = 3;

// ------------------------------------------------------------------------------ small kernels
__global__ void table_update_kernel(int32_t* table, int width, int max_requests, int32_t* status,
                                    const TableDelta* deltas, int n) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const TableDelta d = deltas[i];
  if ((unsigned)d.slot >= (unsigned)max_requests || (unsigned)d.index >= (unsigned)width) {
    atomicOr(status, TS_DEV_BAD_INDEX);        // never expected: the host builds these records
    return;
  }
  table[(size_t)d.slot * width + d.index] = d.page;
}

// KV append as a launch of its own (ts_kv_append, and steps whose attention kernel does not
// append itself): one warp per new token at a time, see append_tokens.
__global__ void kv_append_kernel(StepDevice s) {
  extern __shared__ int32_t rows[];             // staged row arrays, see stage_rows
  pdl_launch_dependents();
  pdl_wait();
  stage_rows(s, rows, threadIdx.x, blockDim.x);
  __syncthreads();
  const int warps = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  append_tokens(s, rows, blockIdx.x * warps + warp, gridDim.x * warps, lane);
}

// Merge of the splits of one token: grid (n_combines, Hq), block D threads.
__global__ void combine_kernel(StepDevice s) {
  pdl_launch_dependents();
  pdl_wait();
  const CombineItem c = s.combines[blockIdx.x];
  const int h = blockIdx.y, d = threadIdx.x;
  const float o = merge_splits(s, c.first_partial, c.n_splits, h, d);
  s.out[((size_t)c.token * s.Hq + h) * s.D + d] = __bfloat16_as_ushort(__float2bfloat16_rn(o));
}

// --------------------------------------------------------------------------- attention kernel
// Shared-memory tile of 64 keys: row r holds D bf16; its 16-byte chunk c sits at chunk
// (c ^ (r & 7)), which makes the 8-row ldmatrix reads conflict-free.
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

template <int D>
__device__ __forceinline__ void load_tile(uint32_t sK, uint32_t sV, const StepDevice& s,
                                          const int32_t* __restrict__ table_row, int kv_head, int kt,
                                          int k_end, int tid) {
  constexpr int CH = D / 8;
  const size_t v_off = (size_t)s.Hkv * kPageSize * D;  // K tile -> V tile of the same page
#pragma unroll
  for (int c = tid; c < kKeysPerTile * CH; c += kThreads) {
    const int row = c / CH, ch = c % CH;
    const int j = kt + row;
    const uint16_t* src = s.pool;
    int bytes = 0;
    if (j < k_end) {
      const int page = table_row[j >> 4];
      if ((unsigned)page < (unsigned)s.n_pages) {
        src = s.pool + ((((size_t)page * 2) * s.Hkv + kv_head) * kPageSize + (j & 15)) * D + ch * 8;
        bytes = 16;
      } else {
        atomicOr(s.status, TS_DEV_BAD_PAGE);
      }
    }
    const uint32_t off = tile_off<D>(row, ch);
    cp_async16(sK + off, src, bytes);
    cp_async16(sV + off, bytes ? src + v_off : src, bytes);
  }
}

// One warp: 16 packed query rows against NT*8 keys of the staged tile, online softmax update.
//   key_row0: first key row inside the stage; key_pos0: its position in the request
//   lim0/lim1: number of visible keys of this lane's two rows (row lane/4 and lane/4 + 8)
template <int D, int NT>
__device__ __forceinline__ void warp_tile(uint32_t sK, uint32_t sV, int key_row0, int key_pos0,
                                          const uint32_t (&qf)[D / 16][4], float (&o)[D / 8][4],
                                          float (&m)[2], float (&l)[2], int lim0, int lim1,
                                          float scale_log2, int lane, bool need_mask) {
  float sc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
    for (int kc = 0; kc < D / 32; ++kc) {
      const int row = key_row0 + nt * 8 + (lane & 7);
      uint32_t r[4];
      ldmatrix_x4(r, sK + tile_off<D>(row, kc * 4 + (lane >> 3)));
      mma_bf16(sc[nt], qf[2 * kc], r[0], r[1]);
      mma_bf16(sc[nt], qf[2 * kc + 1], r[2], r[3]);
    }
  }
  float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float v = sc[nt][e] * scale_log2;
      if (need_mask) {
        const int j = key_pos0 + nt * 8 + 2 * (lane & 3) + (e & 1);
        if (j >= (e < 2 ? lim0 : lim1)) v = -CUDART_INF_F;
      }
      sc[nt][e] = v;
    }
    mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
    mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
  }
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  const float mn0 = fmaxf(m[0], mx0), mn1 = fmaxf(m[1], mx1);
  const float mu0 = mn0 == -CUDART_INF_F ? 0.f : mn0;   // a row that has seen no key yet
  const float mu1 = mn1 == -CUDART_INF_F ? 0.f : mn1;
  const float alpha0 = exp2f(m[0] - mu0), alpha1 = exp2f(m[1] - mu1);
  m[0] = mn0;
  m[1] = mn1;
  float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    sc[nt][0] = exp2f(sc[nt][0] - mu0);
    sc[nt][1] = exp2f(sc[nt][1] - mu0);
    sc[nt][2] = exp2f(sc[nt][2] - mu1);
    sc[nt][3] = exp2f(sc[nt][3] - mu1);
    rs0 += sc[nt][0] + sc[nt][1];
    rs1 += sc[nt][2] + sc[nt][3];
  }
  l[0] = l[0] * alpha0 + rs0;
  l[1] = l[1] * alpha1 + rs1;
#pragma unroll
  for (int dt = 0; dt < D / 8; ++dt) {
    o[dt][0] *= alpha0;
    o[dt][1] *= alpha0;
    o[dt][2] *= alpha1;
    o[dt][3] *= alpha1;
  }
#pragma unroll
  for (int kk = 0; kk < NT / 2; ++kk) {
    uint32_t a[4];
    a[0] = pack_bf16(sc[2 * kk][0], sc[2 * kk][1]);
    a[1] = pack_bf16(sc[2 * kk][2], sc[2 * kk][3]);
    a[2] = pack_bf16(sc[2 * kk + 1][0], sc[2 * kk + 1][1]);
    a[3] = pack_bf16(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
#pragma unroll
    for (int dp = 0; dp < D / 16; ++dp) {
      const int mi = lane >> 3;
      const int row = key_row0 + kk * 16 + (mi & 1) * 8 + (lane & 7);
      uint32_t r[4];
      ldmatrix_x4_trans(r, sV + tile_off<D>(row, 2 * dp + (mi >> 1)));
      mma_bf16(o[2 * dp], a, r[0], r[1]);
      mma_bf16(o[2 * dp + 1], a, r[2], r[3]);
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2) attention_kernel(StepDevice s) {
  extern __shared__ __align__(128) unsigned char smem[];
  pdl_launch_dependents();
  pdl_wait();
  constexpr int kTileBytes = kKeysPerTile * D * 2;
  const uint32_t smem_base = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const WorkItem it = s.items[blockIdx.x];
  const int kv_head = blockIdx.y;
  const int G = s.Hq / s.Hkv;
  const int ctx = s.row_ctx[it.row];
  const int tok0 = s.row_tok0[it.row];
  const int32_t* table_row = s.table + (size_t)s.row_slot[it.row] * s.max_pages_per_req;
  const bool decode = it.kind == 0;

  // The 16 packed rows of this warp: decode -> all warps share rows 0..15; prefill -> 16 each.
  const int row_base = decode ? 0 : warp * 16;
  const int r0 = row_base + (lane >> 2), r1 = r0 + 8;
  const int n_packed = it.q_count * G;                  // packed rows of this item
  const bool real0 = r0 < n_packed, real1 = r1 < n_packed;
  const int pr0 = it.q_begin * G + r0, pr1 = it.q_begin * G + r1;
  const int tokA = pr0 / G, headA = kv_head * G + pr0 % G;
  const int tokB = pr1 / G, headB = kv_head * G + pr1 % G;
  const int lim0 = real0 ? min(ctx + tokA + 1, it.k_end) : it.k_end;
  const int lim1 = real1 ? min(ctx + tokB + 1, it.k_end) : it.k_end;
  int wmin = min(lim0, lim1), wmax = max(real0 ? lim0 : 0, real1 ? lim1 : 0);
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) {
    wmin = min(wmin, __shfl_xor_sync(0xffffffffu, wmin, sft));
    wmax = max(wmax, __shfl_xor_sync(0xffffffffu, wmax, sft));
  }

  // Q fragments straight from global memory (read once per CTA).
  uint32_t qf[D / 16][4];
  {
    const uint16_t* qa = s.q + ((size_t)(tok0 + tokA) * s.Hq + headA) * D + 2 * (lane & 3);
    const uint16_t* qb = s.q + ((size_t)(tok0 + tokB) * s.Hq + headB) * D + 2 * (lane & 3);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      qf[ks][0] = real0 ? *reinterpret_cast<const uint32_t*>(qa + ks * 16) : 0u;
      qf[ks][1] = real1 ? *reinterpret_cast<const uint32_t*>(qb + ks * 16) : 0u;
      qf[ks][2] = real0 ? *reinterpret_cast<const uint32_t*>(qa + ks * 16 + 8) : 0u;
      qf[ks][3] = real1 ? *reinterpret_cast<const uint32_t*>(qb + ks * 16 + 8) : 0u;
    }
  }
  float o[D / 8][4];
#pragma unroll
  for (int dt = 0; dt < D / 8; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;
  float m[2] = {-CUDART_INF_F, -CUDART_INF_F}, l[2] = {0.f, 0.f};

  const int n_tiles = (it.k_end - it.k_begin + kKeysPerTile - 1) / kKeysPerTile;
#pragma unroll
  for (int st = 0; st < kStages - 1; ++st) {
    if (st < n_tiles)
      load_tile<D>(smem_base + st * 2 * kTileBytes, smem_base + st * 2 * kTileBytes + kTileBytes, s,
                   table_row, kv_head, it.k_begin + st * kKeysPerTile, it.k_end, tid);
    cp_async_commit();
  }
  for (int t = 0; t < n_tiles; ++t) {
    cp_async_wait<kStages - 2>();
    __syncthreads();
    const int nxt = t + kStages - 1;
    if (nxt < n_tiles) {
      const int st = nxt % kStages;
      load_tile<D>(smem_base + st * 2 * kTileBytes, smem_base + st * 2 * kTileBytes + kTileBytes, s,
                   table_row, kv_head, it.k_begin + nxt * kKeysPerTile, it.k_end, tid);
    }
    cp_async_commit();
    const int st = t % kStages;
    const uint32_t sK = smem_base + st * 2 * kTileBytes, sV = sK + kTileBytes;
    const int kt = it.k_begin + t * kKeysPerTile;
    if (decode) {
      const int kp = kt + warp * 16;
      if (kp < wmax)
        warp_tile<D, 2>(sK, sV, warp * 16, kp, qf, o, m, l, lim0, lim1, s.scale_log2, lane, kp + 16 > wmin);
    } else {
      if (kt < wmax)
        warp_tile<D, 8>(sK, sV, 0, kt, qf, o, m, l, lim0, lim1, s.scale_log2, lane,
                        kt + kKeysPerTile > wmin);
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  l[0] += __shfl_xor_sync(0xffffffffu, l[0], 1);
  l[0] += __shfl_xor_sync(0xffffffffu, l[0], 2);
  l[1] += __shfl_xor_sync(0xffffffffu, l[1], 1);
  l[1] += __shfl_xor_sync(0xffffffffu, l[1], 2);

  if (!decode) {
    const float inv0 = 1.f / l[0], inv1 = 1.f / l[1];
    uint16_t* oa = s.out + ((size_t)(tok0 + tokA) * s.Hq + headA) * D + 2 * (lane & 3);
    uint16_t* ob = s.out + ((size_t)(tok0 + tokB) * s.Hq + headB) * D + 2 * (lane & 3);
#pragma unroll
    for (int dt = 0; dt < D / 8; ++dt) {
      if (real0) *reinterpret_cast<uint32_t*>(oa + dt * 8) = pack_bf16(o[dt][0] * inv0, o[dt][1] * inv0);
      if (real1) *reinterpret_cast<uint32_t*>(ob + dt * 8) = pack_bf16(o[dt][2] * inv1, o[dt][3] * inv1);
    }
    return;
  }

  // Decode: the four warps hold partial states over disjoint keys of the same rows; merge them.
  float* sm_o = reinterpret_cast<float*>(smem);                    // [4][16][D]
  float* sm_m = sm_o + 4 * 16 * D;                                 // [4][16]
  float* sm_l = sm_m + 4 * 16;                                     // [4][16]
  {
    const int ra = lane >> 2, rb = ra + 8;
    float* wo = sm_o + warp * 16 * D;
#pragma unroll
    for (int dt = 0; dt < D / 8; ++dt) {
      const int d = dt * 8 + 2 * (lane & 3);
      wo[ra * D + d] = o[dt][0];
      wo[ra * D + d + 1] = o[dt][1];
      wo[rb * D + d] = o[dt][2];
      wo[rb * D + d + 1] = o[dt][3];
    }
    if ((lane & 3) == 0) {
      sm_m[warp * 16 + ra] = m[0];
      sm_m[warp * 16 + rb] = m[1];
      sm_l[warp * 16 + ra] = l[0];
      sm_l[warp * 16 + rb] = l[1];
    }
  }
  __syncthreads();
  for (int idx = tid; idx < n_packed * D; idx += kThreads) {
    const int r = idx / D, d = idx % D;
    float mm = sm_m[r];
#pragma unroll
    for (int w = 1; w < 4; ++w) mm = fmaxf(mm, sm_m[w * 16 + r]);
    float ll = 0.f, acc = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float wgt = exp2f(sm_m[w * 16 + r] - mm);   // a warp that saw no key has m = -inf
      ll += wgt * sm_l[w * 16 + r];
      acc += wgt * sm_o[(w * 16 + r) * D + d];
    }
    const int pr = it.q_begin * G + r;
    const int head = kv_head * G + pr % G;
    const int tok = tok0 + pr / G;
    if (it.partial_slot < 0) {
      s.out[((size_t)tok * s.Hq + head) * D + d] = __bfloat16_as_ushort(__float2bfloat16_rn(acc / ll));
    } else {
      const size_t ph = (size_t)it.partial_slot * s.Hq + head;
      s.part_acc[ph * D + d] = acc;
      if (d == 0) {
        s.part_ml[ph * 2] = mm;
        s.part_ml[ph * 2 + 1] = ll;
      }
    }
  }
}

template <int D>
cudaError_t launch_attention_d(const StepDevice& s, cudaStream_t stream) {
  constexpr int smem_pipe = kStages * 2 * kKeysPerTile * D * 2;
  constexpr int smem_merge = (4 * 16 * D + 2 * 4 * 16) * (int)sizeof(float);
  constexpr int smem = smem_pipe > smem_merge ? smem_pipe : smem_merge;
  cudaError_t e = cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(attention_kernel<D>, dim3(s.n_items, s.Hkv), dim3(kThreads), smem, stream, s);
}

}  // namespace

cudaError_t launch_table_update(int32_t* table, int max_pages_per_req, int max_requests, int32_t* status,
                                const TableDelta* deltas, int n_deltas, cudaStream_t stream) {
  if (n_deltas <= 0) return cudaSuccess;
  return launch_pdl(table_update_kernel, dim3((n_deltas + 255) / 256), dim3(256), 0, stream, table, max_pages_per_req,
                    max_requests, status, deltas, n_deltas);
}

cudaError_t launch_kv_append(const StepDevice& s, cudaStream_t stream) {
  if (s.n_tokens <= 0) return cudaSuccess;
  const int threads = 256;                                    // eight warps = eight tokens per block at a time
  const int blocks = (s.n_tokens + 7) / 8;
  const int grid = blocks < 148 * 8 ? blocks : 148 * 8;
  return launch_pdl(kv_append_kernel, dim3(grid), dim3(threads), staged_rows_bytes(s.n_rows), stream, s);
}

cudaError_t launch_attention(const StepDevice& s, cudaStream_t stream) {
  if (s.n_items <= 0) return cudaSuccess;
  return s.D == 128 ? launch_attention_d<128>(s, stream) : launch_attention_d<64>(s, stream);
}

cudaError_t launch_combine(const StepDevice& s, cudaStream_t stream) {
  if (s.n_combines <= 0) return cudaSuccess;
  return launch_pdl(combine_kernel, dim3(s.n_combines, s.Hq), dim3(s.D), 0, stream, s);
}

}  // namespace ts

// ------------------------------------------------------------------------------------------
// ts_decode_attention_static: split-KV decode attention whose scratch (split partials and the
// work list) sits in a fixed device array of this library instead of caller-provided memory.
// It reuses the attention and combine kernels above unchanged; only the planning is different
// (done on the device, a fixed number of splits per row).
// ------------------------------------------------------------------------------------------
namespace ts {
namespace {

constexpr int kStaticMaxRows = 256;
constexpr int kStaticMaxSplits = 16;
constexpr size_t kStaticAccFloats = size_t(1) << 21;               // 8 MiB of split accumulators
constexpr size_t kStaticMlFloats = kStaticAccFloats / 64 * 2;      // (max, sum) per (slot, head), D >= 64
constexpr size_t kStaticItems = size_t(kStaticMaxRows) * kStaticMaxSplits;

struct StaticScratch {
  float part_acc[kStaticAccFloats];
  float part_ml[kStaticMlFloats];
  WorkItem items[kStaticItems];
  CombineItem combines[kStaticMaxRows];
  int32_t row_slot[kStaticMaxRows];
  int32_t row_ctx[kStaticMaxRows];
  int32_t row_tok0[kStaticMaxRows + 1];
  int32_t status;
};

// Lives in every context that loads the library, until the process exits (about 8.4 MiB).
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// One thread per (row, split): writes the row arrays, the work items and the combine list.
__global__ void static_plan_kernel(StaticScratch* sc, const int32_t* kv_len, int n_rows, int n_splits,
                                   int G, int table_width) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx == 0) sc->status = 0;
  if (idx >= n_rows * n_splits) return;
  const int r = idx / n_splits, s = idx % n_splits;
  const int n = kv_len[r];
  const bool ok = n >= 1 && n <= table_width * kPageSize;
  int per = 0, ns = 0;
  if (ok) {
    per = ((n + n_splits - 1) / n_splits + kKeysPerTile - 1) / kKeysPerTile * kKeysPerTile;
    ns = (n + per - 1) / per;
  }
  WorkItem it;
  it.row = r;
  it.kind = 0;
  it.q_begin = 0;
  it.reserved = 0;
  if (s < ns) {
    it.q_count = 1;
    it.k_begin = s * per;
    it.k_end = min(n, (s + 1) * per);
    it.partial_slot = r * n_splits + s;
  } else {          // nothing to do: zero query rows and an empty key range
    it.q_count = 0;
    it.k_begin = 0;
    it.k_end = 0;
    it.partial_slot = -1;
  }
  sc->items[idx] = it;
  if (s == 0) {
    sc->row_slot[r] = r;
    sc->row_ctx[r] = ok ? n - 1 : 0;
    sc->row_tok0[r] = r;
    if (r == n_rows - 1) sc->row_tok0[n_rows] = n_rows;
    CombineItem c;
    c.token = r;
    c.first_partial = r * n_splits;
    c.n_splits = ns;       // 0 for a rejected row: its output becomes NaN
    c.reserved = 0;
    sc->combines[r] = c;
  }
}

constexpr int kMaxDevices = 64;
StaticScratch* g_static_ptr[kMaxDevices] = {};

}  // namespace
}  // namespace ts

extern "C" int ts_decode_attention_static(int32_t device, int32_t n_q_heads, int32_t n_kv_heads,
                                          int32_t head_dim, int32_t n_pages, const void* kv_pool,
                                          const int32_t* block_tables, int32_t table_width,
                                          const int32_t* kv_len, int32_t n_rows, int32_t n_splits,
                                          float softmax_scale, const void* q, void* out,
                                          void* cuda_stream) {
  using namespace ts;
  if (n_rows == 0) return TS_OK;
  if (!kv_pool || !block_tables || !kv_len || !q || !out) return TS_ERR_INVALID;
  if (device < 0 || device >= kMaxDevices || n_rows < 0 || n_pages <= 0 || table_width <= 0)
    return TS_ERR_INVALID;
  if (head_dim != 64 && head_dim != 128) return TS_ERR_UNSUPPORTED;
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads) return TS_ERR_UNSUPPORTED;
  const int G = n_q_heads / n_kv_heads;
  if (G > kMaxGroup) return TS_ERR_UNSUPPORTED;
  if (((uintptr_t)q | (uintptr_t)out | (uintptr_t)kv_pool) & 15u) return TS_ERR_INVALID;
  // the built-in scratch is fixed: refuse what does not fit
  if (n_rows > kStaticMaxRows || n_splits < 1 || n_splits > kStaticMaxSplits) return TS_ERR_WORKSPACE;
  if ((size_t)n_rows * n_splits * n_q_heads * head_dim > kStaticAccFloats) return TS_ERR_WORKSPACE;

  if (cudaSetDevice(device) != cudaSuccess) return TS_ERR_CUDA;
  if (!g_static_ptr[device]) {
    // In host code the array's name is not a device address; ask the runtime for the address
    // of this device's copy, once, with the device current.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return TS_ERR_CUDA;
    g_static_ptr[device] = static_cast<StaticScratch*>(p);
  }
  StaticScratch* sc = g_static_ptr[device];
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  const int n_items = n_rows * n_splits;
  static_plan_kernel<<<(n_items + 127) / 128, 128, 0, stream>>>(sc, kv_len, n_rows, n_splits, G, table_width);
  if (cudaGetLastError() != cudaSuccess) return TS_ERR_CUDA;

  StepDevice d;
  d.pool = (uint16_t*)kv_pool;            // only read by these kernels
  d.table = (int32_t*)block_tables;       // only read
  d.status = &sc->status;
  d.pf_queue = nullptr;
  d.append_in_decode = 0;
  d.part_acc = sc->part_acc;
  d.part_ml = sc->part_ml;
  d.row_slot = sc->row_slot;
  d.row_ctx = sc->row_ctx;
  d.row_qlen = nullptr;                   // not read by attention / combine
  d.row_tok0 = sc->row_tok0;
  d.items = sc->items;
  d.combines = sc->combines;
  d.q = (const uint16_t*)q;
  d.k_new = nullptr;
  d.v_new = nullptr;
  d.out = (uint16_t*)out;
  d.n_rows = n_rows;
  d.n_tokens = n_rows;
  d.n_items = n_items;
  d.n_combines = n_rows;
  d.n_prefill_items = 0;
  d.Hq = n_q_heads;
  d.Hkv = n_kv_heads;
  d.D = head_dim;
  d.n_pages = n_pages;
  d.max_pages_per_req = table_width;
  d.max_requests = n_rows;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
  d.scale_log2 = scale * 1.4426950408889634f;
  if (launch_attention(d, stream) != cudaSuccess) return TS_ERR_CUDA;
  if (launch_combine(d, stream) != cudaSuccess) return TS_ERR_CUDA;
  return TS_OK;
}
