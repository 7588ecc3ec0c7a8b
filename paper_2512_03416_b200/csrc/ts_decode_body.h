// Device code of the split-KV flash-decode path (sm_100a), shared by the stand-alone decode kernel
// and by the mixed kernel whose decode CTAs run it before they join the prefill work.
//
// The path is bound by HBM: every cached K/V byte is read once and used for 4*G flops.
//   * each CTA walks a static sequence of the cost-sorted work units (decode work item x KV head),
//     dealt forth and back over the CTAs;
//   * K/V pages (16 tokens) arrive by TMA tensor copies, 128-byte swizzled, straight from the
//     paged pool; the page id is a TMA coordinate, so scattered pages cost nothing extra;
//   * every warp owns a private ring of page stages and issues its own copies: the pages of a
//     unit are dealt round-robin to the warps, a warp's lookahead crosses unit boundaries, and
//     the only CTA-wide synchronisation is the merge at the end of a unit;
//   * the tensor-core product is transposed, S^T = K Q^T and O^T = V^T P^T (mma.sync m16n8k16,
//     keys / head_dim as the M dimension, the G <= 8 query heads of the KV head as N), so no MMA
//     row is padding and the accumulators stay small; P^T is re-laid out with movmatrix;
//   * softmax is online in base 2 with fp32 state per head, reduced with warp shuffles.
#pragma once
#include <cuda_bf16.h>
#include <math_constants.h>

#include "../../include/tokenscale.h"
#include "ts_internal.h"
#include "ts_ptx.h"
#include "ts_tma.h"

namespace ts {
namespace dec {


constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;

// Barrier of the kDecThreads decode threads (id 1; id 0 stays with the whole block).
__device__ __forceinline__ void block_sync() { asm volatile("bar.sync 1, %0;\n" ::"n"(kDecThreads) : "memory"); }
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}
// Shared-memory image of one page stage (written by TMA with the 128-byte swizzle):
//   D = 128: [half 0: K 16x128B | V 16x128B][half 1: K | V]   (two copies of 4 KB)
//   D =  64: [K 16x128B | V 16x128B]                            (one copy of 4 KB)
// Row r, 16-byte chunk c (of the 2*D-byte logical row) of K:
template <int D>
__device__ __forceinline__ uint32_t page_off(int kv, int r, int c) {
  return (uint32_t)((c >> 3) * 4096 + kv * 2048 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// The sequence of pages one warp works on: for unit sequence number k of this CTA
// (unit = k * n_ctas + cta, or + n_ctas - 1 - cta for odd k), the unit's pages j = warp, warp + W, ...
struct UnitInfo {
  int first_page, n_pg;   // pages [first_page, first_page + n_pg) of the row's block table
  int head;               // KV head
  int row;
  int k_begin, k_end;
  int partial_slot;
  const int32_t* table_row;
};

__device__ __forceinline__ bool load_unit(const StepDevice& s, int cta, int n_ctas, int k, UnitInfo& u) {
  const int n_dec = s.n_items - s.n_prefill_items;
  // units are sorted by length: dealing them forth and back (CTA 0 .. n-1, then n-1 .. 0) keeps the
  // CTAs' totals close, where plain round-robin would hand CTA 0 the longest unit of every round
  const long long unit = (long long)k * n_ctas + ((k & 1) ? (long long)(n_ctas - 1 - cta) : (long long)cta);
  if (unit >= (long long)n_dec * s.Hkv) return false;
  const WorkItem it = s.items[s.n_prefill_items + (int)(unit / s.Hkv)];
  u.head = (int)(unit % s.Hkv);
  u.row = it.row;
  u.k_begin = it.k_begin;
  u.k_end = it.k_end;
  u.partial_slot = it.partial_slot;
  u.first_page = it.k_begin >> 4;
  u.n_pg = (it.k_end - it.k_begin + kPageSize - 1) >> 4;
  u.table_row = s.table + (size_t)s.row_slot[it.row] * s.max_pages_per_req;
  return true;
}

template <int D, int STAGES>
__host__ __device__ constexpr size_t decode_smem_bytes(int G) {
  return (size_t)kDecWarps * STAGES * (2 * kPageSize * D * 2) + (size_t)kDecWarps * G * (D + 2) * sizeof(float) +
         (size_t)kDecWarps * STAGES * 8;
}

// Runs this CTA's share of the decode units on the first kDecThreads threads of the block (the
// caller keeps any other threads away). `smem` is the 1024-byte-aligned shared-memory window
// (decode_smem_bytes<D, STAGES>(G) bytes), `base` its shared-space address. The caller has
// executed griddepcontrol.wait; the function leaves no copy in flight when it returns.
template <int D, int NH, int STAGES>
__device__ __forceinline__ void decode_units(const StepDevice& s, const CUtensorMap* kv_map, unsigned char* smem,
                                             uint32_t base, int cta, int n_ctas) {
  constexpr int W = kDecWarps;
  constexpr int STAGE_BYTES = 2 * kPageSize * D * 2;   // K + V of one page and KV head
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int G = s.Hq / s.Hkv;

  const uint32_t ring = base + warp * STAGES * STAGE_BYTES;
  unsigned char* after_rings = smem + W * STAGES * STAGE_BYTES;
  float* merge_o = reinterpret_cast<float*>(after_rings);                 // [W][G][D]
  float* merge_ml = merge_o + W * G * D;                                  // [W][G][2]
  const uint32_t bars = smem_u32(merge_ml + W * G * 2);                   // [W][STAGES] mbarriers
  const uint32_t my_bars = bars + warp * STAGES * 8;

  if (tid == 0) {
    for (int i = 0; i < W * STAGES; ++i) mbar_init(bars + i * 8, 1);
    mbar_init_fence();
  }
  block_sync();

  bool dead = false;           // a wait ran out: stop issuing copies, keep the control flow
  // ---------------------------------------------------------------- producer side (this warp)
  UnitInfo pu;
  int pk = 0;                  // unit sequence number the producer is in
  int pj = warp;               // next local page of this warp in that unit
  bool p_valid = load_unit(s, cta, n_ctas, pk, pu);
  int p_pages = -1;            // lane i holds the page id of local page warp + (p_chunk*32 + i)*W
  int p_chunk = -1;
  auto p_settle = [&]() {      // move to the next unit that has a page for this warp
    while (p_valid && pj >= pu.n_pg) {
      ++pk;
      pj = warp;
      p_chunk = -1;
      p_valid = load_unit(s, cta, n_ctas, pk, pu);
    }
  };
  p_settle();
  auto issue = [&](int stage) {
    const int idx = (pj - warp) / W;
    if ((idx >> 5) != p_chunk) {
      p_chunk = idx >> 5;
      const int j = warp + ((p_chunk << 5) + lane) * W;
      p_pages = j < pu.n_pg ? pu.table_row[pu.first_page + j] : 0;
    }
    int page = __shfl_sync(0xffffffffu, p_pages, idx & 31);
    if (lane == 0 && !dead) {
      if ((unsigned)page >= (unsigned)s.n_pages) {
        atomicOr(s.status, TS_DEV_BAD_PAGE);
        page = s.n_pages;      // out of range on purpose: the copy then delivers zeros
      }
      const uint32_t bar = my_bars + stage * 8;
      const uint32_t dst = ring + stage * STAGE_BYTES;
      fence_proxy_async();
      mbar_expect_tx(bar, STAGE_BYTES);
      tma_load_5d(dst, kv_map, bar, 0, 0, pu.head, 0, page);
      if (D == 128) tma_load_5d(dst + 4096, kv_map, bar, 64, 0, pu.head, 0, page);
    }
    pj += W;
    p_settle();
  };
  int n_consumed = 0;
#pragma unroll 1
  for (int st = 0; st < STAGES; ++st)
    if (p_valid) issue(st);

  // ---------------------------------------------------------------------------- consumer side
  UnitInfo cu;
#pragma unroll 1
  for (int ck = 0; load_unit(s, cta, n_ctas, ck, cu); ++ck) {
    const int tok = s.row_tok0[cu.row];
    const int n = cu.k_end;   // keys at positions >= n are not visible (decode: ctx + 1 or split end)
    const int new_pos = s.row_ctx[cu.row];   // position of the row's new token
    // Q^T fragments: lane (g, t) holds head g (and g + 8), head_dim pairs 2t, 2t+1 (+8)
    uint32_t qf[NH][D / 16][2];
#pragma unroll
    for (int nh = 0; nh < NH; ++nh) {
      const int hh = nh * 8 + g;
      const uint16_t* qp = s.q + ((size_t)tok * s.Hq + cu.head * G + hh) * D + 2 * t;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        qf[nh][ks][0] = hh < G ? *reinterpret_cast<const uint32_t*>(qp + ks * 16) : 0u;
        qf[nh][ks][1] = hh < G ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8) : 0u;
      }
    }
    float o[NH][D / 16][4];
    float m[NH][2], l[NH][2];
#pragma unroll
    for (int nh = 0; nh < NH; ++nh) {
      m[nh][0] = m[nh][1] = -CUDART_INF_F;
      l[nh][0] = l[nh][1] = 0.f;
#pragma unroll
      for (int dt = 0; dt < D / 16; ++dt) o[nh][dt][0] = o[nh][dt][1] = o[nh][dt][2] = o[nh][dt][3] = 0.f;
    }

#pragma unroll 1
    for (int j = warp; j < cu.n_pg; j += W) {
      const int stage = n_consumed % STAGES;
      const uint32_t parity = (n_consumed / STAGES) & 1;
      const uint32_t sp = ring + stage * STAGE_BYTES;
      if (!mbar_wait(my_bars + stage * 8, parity, dead ? 1000 : s.wait_cycles)) {
        if (!dead && lane == 0) atomicOr(s.status, TS_DEV_TIMEOUT);
        dead = true;
      }
      const int pos0 = cu.k_begin + j * kPageSize;   // position of the page's first slot
      if (s.append_in_decode && new_pos >= pos0 && new_pos < pos0 + kPageSize) {
        // KV append (Sec. 2.1) without a launch of its own: this page holds the row's new token,
        // which is not in the pool yet. Lay its K and V over the page image in shared memory and
        // write them to the pool page; a lane moves one 16-byte chunk of K or V.
        constexpr int CH = D / 8;
        const int r = new_pos - pos0;
        const int page = cu.table_row[cu.first_page + j];
        unsigned char* pg = smem + (sp - base);
        for (int i = lane; i < 2 * CH; i += 32) {
          const int kv = i / CH, c = i % CH;
          const uint4 val = *reinterpret_cast<const uint4*>((kv ? s.v_new : s.k_new) + ((size_t)tok * s.Hkv + cu.head) * D + c * 8);
          *reinterpret_cast<uint4*>(pg + page_off<D>(kv, r, c)) = val;
          if ((unsigned)page < (unsigned)s.n_pages)
            *reinterpret_cast<uint4*>(s.pool + ((((size_t)page * 2 + kv) * s.Hkv + cu.head) * kPageSize + r) * D + c * 8) = val;
        }
        __syncwarp();
      }
      const bool ragged = pos0 + kPageSize > n;
      if (ragged) {
        // slots past the last token hold whatever was there before: clear their V rows so
        // that a zero weight times stale bits cannot produce NaN
        const int valid = n - pos0;
        unsigned char* pg = smem + (sp - base);
        for (int i = lane; i < kPageSize * 8 * (D / 64); i += 32) {
          const int half = i / (kPageSize * 8), r = (i / 8) % kPageSize, c = i % 8;
          if (r >= valid)
            *reinterpret_cast<uint4*>(pg + half * 4096 + 2048 + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
      }
      // ---- S^T = K Q^T : 16 keys x 8 heads per n-tile
      // (two accumulators per n-tile, even and odd k-steps: half the dependent MMA chain)
      float sc[NH][4], sc_odd[NH][4];
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        sc[nh][0] = sc[nh][1] = sc[nh][2] = sc[nh][3] = 0.f;
        sc_odd[nh][0] = sc_odd[nh][1] = sc_odd[nh][2] = sc_odd[nh][3] = 0.f;
      }
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t a[4];
        const int mi = lane >> 3;
        ldmatrix_x4(a, sp + page_off<D>(0, (mi & 1) * 8 + (lane & 7), 2 * ks + (mi >> 1)));
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) mma_bf16((ks & 1) ? sc_odd[nh] : sc[nh], a, qf[nh][ks][0], qf[nh][ks][1]);
      }
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        sc[nh][0] += sc_odd[nh][0];
        sc[nh][1] += sc_odd[nh][1];
        sc[nh][2] += sc_odd[nh][2];
        sc[nh][3] += sc_odd[nh][3];
      }
      // ---- online softmax per head (this lane: heads 2t, 2t+1 of each n-tile; keys g, g+8)
      uint32_t pb[NH][2];
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        const bool v0 = !ragged || pos0 + g < n, v1 = !ragged || pos0 + g + 8 < n;
        float s0 = v0 ? sc[nh][0] * s.scale_log2 : -CUDART_INF_F;
        float s1 = v0 ? sc[nh][1] * s.scale_log2 : -CUDART_INF_F;
        float s2 = v1 ? sc[nh][2] * s.scale_log2 : -CUDART_INF_F;
        float s3 = v1 ? sc[nh][3] * s.scale_log2 : -CUDART_INF_F;
        float mx0 = fmaxf(s0, s2), mx1 = fmaxf(s1, s3);
#pragma unroll
        for (int sh = 4; sh < 32; sh <<= 1) {
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
        }
        const float mn0 = fmaxf(m[nh][0], mx0), mn1 = fmaxf(m[nh][1], mx1);
        const float al0 = exp2f(m[nh][0] - mn0), al1 = exp2f(m[nh][1] - mn1);   // first page: exp2(-inf) = 0
        m[nh][0] = mn0;
        m[nh][1] = mn1;
        s0 = exp2f(s0 - mn0);
        s1 = exp2f(s1 - mn1);
        s2 = exp2f(s2 - mn0);
        s3 = exp2f(s3 - mn1);
        l[nh][0] = l[nh][0] * al0 + s0 + s2;
        l[nh][1] = l[nh][1] * al1 + s1 + s3;
#pragma unroll
        for (int dt = 0; dt < D / 16; ++dt) {
          o[nh][dt][0] *= al0;
          o[nh][dt][1] *= al1;
          o[nh][dt][2] *= al0;
          o[nh][dt][3] *= al1;
        }
        // P^T as the B operand: transpose the two 8x8 (key x head) blocks across the warp
        pb[nh][0] = movmatrix_t(pack_bf16(s0, s1));
        pb[nh][1] = movmatrix_t(pack_bf16(s2, s3));
      }
      // ---- O^T += V^T P^T : 16 head_dim rows per m-tile
#pragma unroll
      for (int dt = 0; dt < D / 16; ++dt) {
        uint32_t a[4];
        const int mi = lane >> 3;
        ldmatrix_x4_trans(a, sp + page_off<D>(1, (mi >> 1) * 8 + (lane & 7), 2 * dt + (mi & 1)));
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) mma_bf16(o[nh][dt], a, pb[nh][0], pb[nh][1]);
      }
      __syncwarp();
      ++n_consumed;
      if (p_valid) issue(stage);
    }

    // ---- merge the warps of the CTA (they saw disjoint pages of the same unit)
#pragma unroll
    for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
      for (int sh = 4; sh < 32; sh <<= 1) {
        l[nh][0] += __shfl_xor_sync(0xffffffffu, l[nh][0], sh);
        l[nh][1] += __shfl_xor_sync(0xffffffffu, l[nh][1], sh);
      }
      const int h0 = nh * 8 + 2 * t, h1 = h0 + 1;
      float* wo = merge_o + (size_t)warp * G * D;
#pragma unroll
      for (int dt = 0; dt < D / 16; ++dt) {
        const int d = dt * 16 + g;
        if (h0 < G) {
          wo[h0 * D + d] = o[nh][dt][0];
          wo[h0 * D + d + 8] = o[nh][dt][2];
        }
        if (h1 < G) {
          wo[h1 * D + d] = o[nh][dt][1];
          wo[h1 * D + d + 8] = o[nh][dt][3];
        }
      }
      if (g == 0) {
        if (h0 < G) {
          merge_ml[(warp * G + h0) * 2] = m[nh][0];
          merge_ml[(warp * G + h0) * 2 + 1] = l[nh][0];
        }
        if (h1 < G) {
          merge_ml[(warp * G + h1) * 2] = m[nh][1];
          merge_ml[(warp * G + h1) * 2 + 1] = l[nh][1];
        }
      }
    }
    block_sync();
    for (int idx = tid; idx < G * D; idx += kDecThreads) {
      const int hh = idx / D, d = idx % D;
      float mm = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < W; ++w) mm = fmaxf(mm, merge_ml[(w * G + hh) * 2]);
      float ll = 0.f, acc = 0.f;
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const float wgt = exp2f(merge_ml[(w * G + hh) * 2] - mm);   // a warp without pages: exp2(-inf) = 0
        ll += wgt * merge_ml[(w * G + hh) * 2 + 1];
        acc += wgt * merge_o[((size_t)w * G + hh) * D + d];
      }
      const int head = cu.head * G + hh;
      if (cu.partial_slot < 0) {
        s.out[((size_t)tok * s.Hq + head) * D + d] = __bfloat16_as_ushort(__float2bfloat16_rn(acc / ll));
      } else {
        const size_t ph = (size_t)cu.partial_slot * s.Hq + head;
        s.part_acc[ph * D + d] = acc;
        if (d == 0) {
          s.part_ml[ph * 2] = mm;
          s.part_ml[ph * 2 + 1] = ll;
        }
      }
    }
    block_sync();
  }
  // every page copy has been consumed; give the barriers' shared memory back
  if (tid == 0) {
    for (int i = 0; i < W * STAGES; ++i) asm volatile("mbarrier.inval.shared::cta.b64 [%0];\n" ::"r"(bars + i * 8) : "memory");
  }
}

}  // namespace dec
}  // namespace ts
