// Host side of the decoder layer around the attention step: RMSNorm, fused QKV projection with
// rotary embedding, ts_mixed_step, output projection, gated MLP. The public ABI is documented in
// include/tokenscale.h.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/tokenscale.h"
#include "ts_internal.h"

namespace {

constexpr size_t kAlign = 256;
constexpr int kPosRing = 4;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D view of a K-major bf16 matrix [rows][k]: box = 64 of K (128 bytes, the swizzle span) x box_rows.
bool make_operand_map(void* encode_fn, const void* ptr, int64_t rows, int64_t k, int box_rows, CUtensorMap* out) {
  const cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)k * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return ((EncodeFn)encode_fn)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct LayerLayout {
  size_t off_table, off_pos, off_h, off_q, off_k, off_v, off_attn, off_y, off_z, total;
};

bool layer_shape_ok(const ts_config* c, const ts_layer_config* l) {
  if (!c || !l) return false;
  if (c->head_dim != 128) return false;                        // the fused rotary epilogue pairs columns i, i + 64
  if (l->hidden <= 0 || l->hidden % 64 || l->intermediate <= 0 || l->intermediate % 128) return false;
  if (l->max_position <= 0) return false;
  return true;
}

void layer_layout(const ts_config* c, const ts_layer_config* l, int max_tokens, LayerLayout* L) {
  const size_t T = (size_t)max_tokens;
  size_t off = 0;
  L->off_table = off; off += align_up((size_t)l->max_position * 64 * sizeof(float2));
  L->off_pos = off; off += align_up(kPosRing * T * sizeof(int32_t));
  L->off_h = off; off += align_up(T * l->hidden * 2);                       // normalised input of a projection (h, then h2)
  L->off_q = off; off += align_up(T * c->n_q_heads * c->head_dim * 2);
  L->off_k = off; off += align_up(T * c->n_kv_heads * c->head_dim * 2);
  L->off_v = off; off += align_up(T * c->n_kv_heads * c->head_dim * 2);
  L->off_attn = off; off += align_up(T * c->n_q_heads * c->head_dim * 2);
  L->off_y = off; off += align_up(T * l->hidden * 2);
  L->off_z = off; off += align_up(T * l->intermediate * 2);
  L->total = off;
}

}  // namespace

struct ts_layer {
  ts_ctx* ctx = nullptr;
  ts_layer_config cfg;
  ts::CtxView view;
  LayerLayout L;
  int max_tokens = 0;
  float eps = 0.f, theta = 0.f;
  CUtensorMap w_qkv, w_o, w_gu, w_down;        // weights: box 64 x 256
  CUtensorMap a_h, a_attn, a_z;                // activations in the workspace: box 64 x 128
  void* pos_host[kPosRing] = {};
  cudaEvent_t pos_ev[kPosRing] = {};
  bool pos_busy[kPosRing] = {};
  int pos_next = 0;
  int last_cuda_error = 0;
};

namespace {
int lfail(ts_layer* l, cudaError_t e) {
  l->last_cuda_error = (int)e;
  return TS_ERR_CUDA;
}
#define TSL_CUDA(l, call)                              \
  do {                                                 \
    cudaError_t e__ = (call);                          \
    if (e__ != cudaSuccess) return lfail((l), e__);    \
  } while (0)
}  // namespace

extern "C" {

size_t ts_layer_workspace_bytes(const ts_config* cfg, const ts_layer_config* layer) {
  if (!layer_shape_ok(cfg, layer) || cfg->chunk_size <= 0) return 0;
  LayerLayout L;
  layer_layout(cfg, layer, cfg->chunk_size, &L);
  return L.total;
}

int ts_pack_gate_up(const void* w_gate, const void* w_up, void* w_gate_up, int32_t intermediate, int32_t hidden,
                    void* cuda_stream) {
  if (!w_gate || !w_up || !w_gate_up || intermediate <= 0 || intermediate % 128 || hidden <= 0 || hidden % 8)
    return TS_ERR_INVALID;
  const cudaError_t e = ts::launch_pack_gate_up((const uint16_t*)w_gate, (const uint16_t*)w_up, (uint16_t*)w_gate_up,
                                                intermediate, hidden, (cudaStream_t)cuda_stream);
  return e == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

int ts_layer_create(ts_ctx* ctx, const ts_layer_config* cfg, void* cuda_stream, ts_layer** out) {
  if (!out) return TS_ERR_INVALID;
  *out = nullptr;
  if (!ctx || !cfg) return TS_ERR_INVALID;
  ts::CtxView view;
  int rc = ts::ctx_view(ctx, (cudaStream_t)cuda_stream, &view);
  if (rc != TS_OK) return rc;
  if (!layer_shape_ok(view.cfg, cfg)) return TS_ERR_UNSUPPORTED;
  if (view.cfg->chunk_size <= 0) return TS_ERR_INVALID;        // the activations are sized by the chunk size
  if (!cfg->w_norm1 || !cfg->w_qkv || !cfg->w_o || !cfg->w_norm2 || !cfg->w_gate_up || !cfg->w_down || !cfg->workspace)
    return TS_ERR_INVALID;
  if (((uintptr_t)cfg->workspace & (kAlign - 1)) || ((uintptr_t)cfg->w_qkv | (uintptr_t)cfg->w_o | (uintptr_t)cfg->w_gate_up |
                                                     (uintptr_t)cfg->w_down | (uintptr_t)cfg->w_norm1 | (uintptr_t)cfg->w_norm2) & 15u)
    return TS_ERR_INVALID;
  ts_layer* l = new (std::nothrow) ts_layer();
  if (!l) return TS_ERR_INVALID;
  l->ctx = ctx;
  l->cfg = *cfg;
  l->view = view;
  l->max_tokens = view.max_tokens;
  layer_layout(view.cfg, cfg, l->max_tokens, &l->L);
  if (cfg->workspace_bytes < l->L.total) {
    delete l;
    return TS_ERR_WORKSPACE;
  }
  l->eps = cfg->rms_eps > 0.f ? cfg->rms_eps : 1e-5f;
  l->theta = cfg->rope_theta > 0.f ? cfg->rope_theta : 500000.f;
  const ts_config* c = view.cfg;
  const int64_t qd = (int64_t)c->n_q_heads * c->head_dim, kvd = (int64_t)c->n_kv_heads * c->head_dim;
  char* ws = (char*)cfg->workspace;
  bool ok = make_operand_map(view.encode_fn, cfg->w_qkv, qd + 2 * kvd, cfg->hidden, 256, &l->w_qkv) &&
            make_operand_map(view.encode_fn, cfg->w_o, cfg->hidden, qd, 256, &l->w_o) &&
            make_operand_map(view.encode_fn, cfg->w_gate_up, 2 * (int64_t)cfg->intermediate, cfg->hidden, 256, &l->w_gu) &&
            make_operand_map(view.encode_fn, cfg->w_down, cfg->hidden, cfg->intermediate, 256, &l->w_down) &&
            make_operand_map(view.encode_fn, ws + l->L.off_h, l->max_tokens, cfg->hidden, 128, &l->a_h) &&
            make_operand_map(view.encode_fn, ws + l->L.off_attn, l->max_tokens, qd, 128, &l->a_attn) &&
            make_operand_map(view.encode_fn, ws + l->L.off_z, l->max_tokens, cfg->intermediate, 128, &l->a_z);
  if (!ok) {
    delete l;
    return TS_ERR_CUDA;
  }
  for (int i = 0; i < kPosRing; ++i) {
    if (cudaHostAlloc(&l->pos_host[i], (size_t)l->max_tokens * sizeof(int32_t), cudaHostAllocDefault) != cudaSuccess ||
        cudaEventCreateWithFlags(&l->pos_ev[i], cudaEventDisableTiming) != cudaSuccess) {
      ts_layer_destroy(l);
      return TS_ERR_CUDA;
    }
  }
  if (ts::launch_rope_table((float2*)(ws + l->L.off_table), cfg->max_position, l->theta, (cudaStream_t)cuda_stream) != cudaSuccess) {
    ts_layer_destroy(l);
    return TS_ERR_CUDA;
  }
  *out = l;
  return TS_OK;
}

int ts_layer_destroy(ts_layer* l) {
  if (!l) return TS_ERR_INVALID;
  for (int i = 0; i < kPosRing; ++i) {
    if (l->pos_busy[i]) cudaEventSynchronize(l->pos_ev[i]);
    if (l->pos_ev[i]) cudaEventDestroy(l->pos_ev[i]);
    if (l->pos_host[i]) cudaFreeHost(l->pos_host[i]);
  }
  delete l;
  return TS_OK;
}

int ts_layer_step(ts_layer* l, const ts_step* st, const void* x_in, void* x_out, void* cuda_stream) {
  if (!l || !st) return TS_ERR_INVALID;
  if (st->n_rows == 0) return TS_OK;
  if (!x_in || !x_out || (((uintptr_t)x_in | (uintptr_t)x_out) & 15u)) return TS_ERR_INVALID;
  // the step's own checks first (host only): a step that would be refused must launch nothing
  int32_t n_items = 0;
  int rc = ts_plan_step(l->ctx, st, nullptr, 0, &n_items);
  if (rc != TS_OK) return rc;
  int64_t n = 0;
  for (int r = 0; r < st->n_rows; ++r) {
    if ((int64_t)st->ctx_len[r] + st->q_len[r] > l->cfg.max_position) return TS_ERR_INVALID;   // beyond the rotary table
    n += st->q_len[r];
  }
  if (n > l->max_tokens) return TS_ERR_BUDGET;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const ts_config* c = l->view.cfg;
  TSL_CUDA(l, cudaSetDevice(c->device));
  char* ws = (char*)l->cfg.workspace;
  // positions of the new tokens: row r's token i sits at ctx_len[r] + i
  const int slot = l->pos_next;
  l->pos_next = (l->pos_next + 1) % kPosRing;
  if (l->pos_busy[slot]) {
    TSL_CUDA(l, cudaEventSynchronize(l->pos_ev[slot]));
    l->pos_busy[slot] = false;
  }
  int32_t* ph = (int32_t*)l->pos_host[slot];
  int64_t at = 0;
  for (int r = 0; r < st->n_rows; ++r)
    for (int i = 0; i < st->q_len[r]; ++i) ph[at++] = st->ctx_len[r] + i;
  int32_t* pos_dev = (int32_t*)(ws + l->L.off_pos) + (size_t)slot * l->max_tokens;
  TSL_CUDA(l, cudaMemcpyAsync(pos_dev, ph, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
  TSL_CUDA(l, cudaEventRecord(l->pos_ev[slot], stream));
  l->pos_busy[slot] = true;

  const int N = (int)n, hidden = l->cfg.hidden, inter = l->cfg.intermediate;
  const int qd = c->n_q_heads * c->head_dim, kvd = c->n_kv_heads * c->head_dim;
  uint16_t* h = (uint16_t*)(ws + l->L.off_h);
  uint16_t* q = (uint16_t*)(ws + l->L.off_q);
  uint16_t* k = (uint16_t*)(ws + l->L.off_k);
  uint16_t* v = (uint16_t*)(ws + l->L.off_v);
  uint16_t* attn = (uint16_t*)(ws + l->L.off_attn);
  uint16_t* y = (uint16_t*)(ws + l->L.off_y);
  uint16_t* z = (uint16_t*)(ws + l->L.off_z);
  ts::GemmArgs g;
  std::memset(&g, 0, sizeof g);
  g.status = l->view.status;
  g.wait_cycles = l->view.wait_cycles;
  g.M = N;

  // h = rmsnorm(x); (q, k, v) = rope(h . W_qkv^T)
  TSL_CUDA(l, ts::launch_rmsnorm((const uint16_t*)x_in, (const uint16_t*)l->cfg.w_norm1, h, N, hidden, l->eps, stream));
  g.N = qd + 2 * kvd; g.K = hidden; g.epi = ts::GEMM_EPI_ROPE;
  g.C = q; g.C2 = k; g.C3 = v; g.q_cols = qd; g.kv_cols = kvd; g.pos = pos_dev;
  g.rope_table = (const float2*)(ws + l->L.off_table);
  TSL_CUDA(l, ts::launch_gemm(g, l->a_h, l->w_qkv, 128, l->view.n_sms, stream));
  // attention over the paged KV cache, with the append of the new K/V
  ts_step inner = *st;
  inner.q = q; inner.k_new = k; inner.v_new = v; inner.out = attn;
  rc = ts_mixed_step(l->ctx, &inner, cuda_stream);
  if (rc != TS_OK) return rc;
  // y = x + attn . W_o^T
  g.N = hidden; g.K = qd; g.epi = ts::GEMM_EPI_STORE; g.C = y; g.R = (const uint16_t*)x_in; g.ldc = hidden;
  TSL_CUDA(l, ts::launch_gemm(g, l->a_attn, l->w_o, ts::gemm_tile_m(N, hidden, l->view.n_sms), l->view.n_sms, stream));
  // h2 = rmsnorm(y); z = silu(h2 . W_gate^T) * (h2 . W_up^T)
  TSL_CUDA(l, ts::launch_rmsnorm(y, (const uint16_t*)l->cfg.w_norm2, h, N, hidden, l->eps, stream));
  g.N = 2 * inter; g.K = hidden; g.epi = ts::GEMM_EPI_SILU_MUL; g.C = z; g.R = nullptr; g.ldc = inter;
  TSL_CUDA(l, ts::launch_gemm(g, l->a_h, l->w_gu, ts::gemm_tile_m(N, 2 * inter, l->view.n_sms), l->view.n_sms, stream));
  // out = y + z . W_down^T
  g.N = hidden; g.K = inter; g.epi = ts::GEMM_EPI_STORE; g.C = (uint16_t*)x_out; g.R = y; g.ldc = hidden;
  TSL_CUDA(l, ts::launch_gemm(g, l->a_z, l->w_down, ts::gemm_tile_m(N, hidden, l->view.n_sms), l->view.n_sms, stream));
  return TS_OK;
}

int ts_gemm_bf16(int32_t device, int32_t M, int32_t N, int32_t K, const void* A, const void* B, const void* R, void* C,
                 int32_t tile_m, int32_t* device_status, void* cuda_stream) {
  if (M < 0 || N <= 0 || K <= 0 || (N % 8) || (K % 8)) return TS_ERR_INVALID;
  if (M == 0) return TS_OK;
  if (!A || !B || !C || !device_status) return TS_ERR_INVALID;
  if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C | (uintptr_t)R) & 15u) return TS_ERR_INVALID;
  if (tile_m != 0 && tile_m != 128 && tile_m != 256) return TS_ERR_INVALID;
  if (cudaSetDevice(device) != cudaSuccess) return TS_ERR_CUDA;
  void* encode_fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &encode_fn, cudaEnableDefault, &qres) != cudaSuccess || !encode_fn)
    return TS_ERR_CUDA;
  int n_sms = 0;
  if (cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return TS_ERR_CUDA;
  CUtensorMap a_map, b_map;
  if (!make_operand_map(encode_fn, A, M, K, 128, &a_map) || !make_operand_map(encode_fn, B, N, K, 256, &b_map)) return TS_ERR_CUDA;
  ts::GemmArgs g;
  std::memset(&g, 0, sizeof g);
  g.M = M; g.N = N; g.K = K; g.epi = ts::GEMM_EPI_STORE;
  g.C = (uint16_t*)C; g.R = (const uint16_t*)R; g.ldc = N;
  g.status = device_status;
  g.wait_cycles = ts::kWaitCycles;
  const int tm = tile_m ? tile_m : ts::gemm_tile_m(M, N, n_sms);
  return ts::launch_gemm(g, a_map, b_map, tm, n_sms, (cudaStream_t)cuda_stream) == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

int ts_layer_last_cuda_error(const ts_layer* l) { return l ? l->last_cuda_error : 0; }

}  // extern "C"
