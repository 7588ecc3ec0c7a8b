/*
 * ts_oracle.c -- CPU oracle of the mixed paged-attention step. TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what one decoder iteration computes
 * (TokenScale, arXiv 2512.03416: Sec. 2.1 for what prefill and decode do with the KV cache,
 * Sec. 3.4 / Sec. 4.4 for a batch made of decode requests plus a causal prefill chunk).
 * It is only ever called by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg; the product never links or imports it and it shares no code with the CUDA path.
 *
 * The paper fixes the problem, not the formula: attention is the textbook definition,
 *     s_j = scale * sum_d q_d K_{j,d}          j = 0 .. n-1,  n = ctx + i + 1
 *     m   = max_j s_j,   p_j = exp(s_j - m),   l = sum_j p_j
 *     O_d = (sum_j p_j V_{j,d}) / l
 * written out once per (token, query head) in fp32 (bf16 inputs widen exactly), two passes,
 * keys visited in position order, no blocking, no online rescaling.
 *
 * Pool layout (restated from the boundary's documentation, indexed by this file's own code):
 *     element (page, kv, head, slot, d) at (((page*2 + kv)*Hkv + head)*P + slot)*D + d,
 *     kv = 0 for K, 1 for V; token t of a request sits in page table[t / P], slot t % P.
 *
 * Parity pins (tests/test_oracle_pins.py): closed forms (one key; equal keys; equal values;
 * zero query; two keys with weights 3/4 and 1/4), a library attention routine on contiguous
 * K/V in fp64, table-permutation invariance, decode == last prefill row, chunked == unchunked,
 * convexity, group symmetry, and planted-needle cases for mask and page/slot indexing.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

int oracle_default_threads(void);

static inline float bf16_to_f32(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

static inline size_t pool_index(int64_t page, int kv, int head, int slot, int Hkv, int P, int D) {
  return ((((size_t)page * 2 + (size_t)kv) * (size_t)Hkv + (size_t)head) * (size_t)P + (size_t)slot) *
         (size_t)D;
}

/*
 * KV append (Sec. 2.1): token i of row r goes to position t = ctx[r] + i of its request, i.e.
 * page tables[r][t / P], slot t % P, for every KV head, K and V. A pure copy of bf16 bit
 * patterns; nothing else in the pool changes.
 * tables is [n_rows][table_stride]; k_new/v_new are [N][Hkv][D] with rows concatenated.
 */
void oracle_kv_append(uint16_t* pool, int Hkv, int D, int P, int n_rows, const int32_t* tables,
                      int table_stride, const int32_t* ctx_len, const int32_t* q_len,
                      const uint16_t* k_new, const uint16_t* v_new) {
  size_t tok = 0;
  for (int r = 0; r < n_rows; ++r) {
    for (int i = 0; i < q_len[r]; ++i, ++tok) {
      int t = ctx_len[r] + i;
      int64_t page = tables[(size_t)r * table_stride + t / P];
      int slot = t % P;
      for (int g = 0; g < Hkv; ++g) {
        const uint16_t* ks = k_new + (tok * Hkv + g) * (size_t)D;
        const uint16_t* vs = v_new + (tok * Hkv + g) * (size_t)D;
        memcpy(pool + pool_index(page, 0, g, slot, Hkv, P, D), ks, sizeof(uint16_t) * D);
        memcpy(pool + pool_index(page, 1, g, slot, Hkv, P, D), vs, sizeof(uint16_t) * D);
      }
    }
  }
}

/*
 * Attention of one (row r, new token i, query head h) against the pool, AFTER the append.
 * out: D floats. Returns sum_j p_j / l (should be 1) for the softmax pin.
 */
static float attend_one(const uint16_t* pool, int Hq, int Hkv, int D, int P, float scale,
                        const int32_t* table, int ctx, int i, int h, const uint16_t* q_tok,
                        float* out, float* s /* scratch, n floats */) {
  const int G = Hq / Hkv;
  const int g = h / G;       /* query head h reads KV head h / G */
  const int n = ctx + i + 1; /* positions 0 .. ctx+i are visible  */
  const uint16_t* qh = q_tok + (size_t)h * D;

  float m = -INFINITY;
  for (int j = 0; j < n; ++j) {
    const uint16_t* kj = pool + pool_index(table[j / P], 0, g, j % P, Hkv, P, D);
    float dot = 0.0f;
    for (int d = 0; d < D; ++d) dot += bf16_to_f32(qh[d]) * bf16_to_f32(kj[d]);
    s[j] = scale * dot;
    if (s[j] > m) m = s[j];
  }
  float l = 0.0f;
  for (int d = 0; d < D; ++d) out[d] = 0.0f;
  for (int j = 0; j < n; ++j) {
    const uint16_t* vj = pool + pool_index(table[j / P], 1, g, j % P, Hkv, P, D);
    float p = expf(s[j] - m);
    s[j] = p;
    l += p;
    for (int d = 0; d < D; ++d) out[d] += p * bf16_to_f32(vj[d]);
  }
  for (int d = 0; d < D; ++d) out[d] /= l;
  float wsum = 0.0f;
  for (int j = 0; j < n; ++j) wsum += s[j] / l;
  return wsum;
}

/*
 * Attention for a step. pool must already contain the step's appended K/V.
 *   q            [N][Hq][D] bf16, rows concatenated in row order
 *   sel          NULL: compute every token; else n_sel flat token indices in [0, N)
 *   out          [n_out][Hq][D] fp32, n_out = N or n_sel, in the order of sel
 *   weight_sum   NULL or [n_out][Hq]: sum of the normalised softmax weights
 *   n_threads    OpenMP threads over (token, head); <= 0 = runtime default
 * Returns 0, or -1 on allocation failure / bad selection.
 */
int oracle_attention(const uint16_t* pool, int Hq, int Hkv, int D, int P, float scale, int n_rows,
                     const int32_t* tables, int table_stride, const int32_t* ctx_len,
                     const int32_t* q_len, const uint16_t* q, int n_sel, const int32_t* sel,
                     float* out, float* weight_sum, int n_threads) {
  size_t N = 0;
  int max_n = 1;
  for (int r = 0; r < n_rows; ++r) {
    N += (size_t)q_len[r];
    if (ctx_len[r] + q_len[r] > max_n) max_n = ctx_len[r] + q_len[r];
  }
  /* flat token index -> (row, i) */
  int32_t* tok_row = (int32_t*)malloc(sizeof(int32_t) * (N ? N : 1));
  int32_t* tok_i = (int32_t*)malloc(sizeof(int32_t) * (N ? N : 1));
  if (!tok_row || !tok_i) {
    free(tok_row);
    free(tok_i);
    return -1;
  }
  {
    size_t tok = 0;
    for (int r = 0; r < n_rows; ++r)
      for (int i = 0; i < q_len[r]; ++i, ++tok) {
        tok_row[tok] = r;
        tok_i[tok] = i;
      }
  }
  const long n_out = sel ? n_sel : (long)N;
  for (long o = 0; o < n_out; ++o) {
    long tok = sel ? sel[o] : o;
    if (tok < 0 || (size_t)tok >= N) {
      free(tok_row);
      free(tok_i);
      return -1;
    }
  }
  int failed = 0;
  const long n_work = n_out * Hq;
  const int nt = n_threads > 0 ? n_threads : oracle_default_threads();
  (void)nt;
#ifdef _OPENMP
#pragma omp parallel num_threads(nt)
#endif
  {
    float* s = (float*)malloc(sizeof(float) * (size_t)max_n);
    if (!s) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
      failed = 1;
    }
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
    for (long w = 0; w < n_work; ++w) {
      if (!s) continue;
      long o = w / Hq;
      int h = (int)(w % Hq);
      long tok = sel ? sel[o] : o;
      int r = tok_row[tok], i = tok_i[tok];
      float ws = attend_one(pool, Hq, Hkv, D, P, scale, tables + (size_t)r * table_stride,
                            ctx_len[r], i, h, q + (size_t)tok * Hq * D,
                            out + ((size_t)o * Hq + h) * D, s);
      if (weight_sum) weight_sum[(size_t)o * Hq + h] = ws;
    }
    free(s);
  }
  free(tok_row);
  free(tok_i);
  return failed ? -1 : 0;
}

/* Threads the OpenMP runtime would use by default (1 when built without OpenMP). */
int oracle_default_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
