// Causal prefill-chunk attention on the 5th-generation tensor cores (sm_100a, head_dim 128).
//
// One CTA = one tile of 128 packed query rows (128/G consecutive tokens x the G query heads of
// one KV head) against all keys the tile may see, 128 keys per block:
//     S = Q K^T   (tcgen05.mma, operands in 128B-swizzled shared memory, fp32 accumulator in TMEM)
//     online softmax by one warpgroup, one query row per thread, straight out of TMEM
//     O += P V    (tcgen05.mma, P read from TMEM as bf16, V from shared memory, O accumulates in TMEM)
// Warp roles: warps 0-3 softmax / epilogue (thread i owns TMEM lane i), warp 4 TMA producer,
// warp 5 MMA issuer and TMEM owner. K and V blocks come page by page (16 keys) through TMA with
// the page id as a coordinate; S is double buffered so that Q K^T of block j+1 overlaps the
// softmax of block j. The O rescale is lazy: the reference maximum of a row only moves when the
// new maximum exceeds it by more than 2^8, so most blocks never touch O.
// Every mbarrier wait is bounded; a wait that runs out raises TS_DEV_TIMEOUT and the CTA drains.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "../../include/tokenscale.h"
#include "ts_internal.h"
#include "ts_tma.h"

namespace ts {
namespace {

constexpr int kPfThreads = 192;
constexpr int kBlockKeys = 128;
constexpr int kD = 128;
constexpr int kTileBytes = 128 * kD * 2;        // one 128 x 128 bf16 operand tile: 32 KB
constexpr int kHalfBytes = kTileBytes / 2;      // 64 head_dim columns of it
constexpr int kKvStages = 3;
constexpr float kRescaleThreshold = 8.0f;       // log2 units

// shared-memory map (offsets from the 1024-aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kTileBytes;
constexpr int kOffV = kOffK + kKvStages * kTileBytes;
constexpr int kOffBar = kOffV + kKvStages * kTileBytes;
enum {
  BAR_Q = 0,
  BAR_K_FULL = 1,                      // [kKvStages]
  BAR_K_EMPTY = BAR_K_FULL + kKvStages,
  BAR_V_FULL = BAR_K_EMPTY + kKvStages,
  BAR_V_EMPTY = BAR_V_FULL + kKvStages,
  BAR_V_FIXED = BAR_V_EMPTY + kKvStages,
  BAR_S_FULL = BAR_V_FIXED + 1,        // [2]
  BAR_P_FULL = BAR_S_FULL + 2,         // [2]
  BAR_O_FULL = BAR_P_FULL + 2,
  BAR_COUNT = BAR_O_FULL + 1
};
constexpr int kOffMisc = kOffBar + BAR_COUNT * 8;   // tmem base address, dead flag
constexpr int kSmemBytes = kOffMisc + 16 + 1024;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// ---- tcgen05 wrappers
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_dst), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar)
               : "memory");
}
// D(tmem) (+)= A(smem) * B(smem)
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D(tmem) (+)= A(tmem) * B(smem)
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d),
      "r"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(float (&v)[32], uint32_t taddr) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,"
      "%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,"
      "%28,%29,%30,%31,%32};\n" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
      "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
      "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle. `lbo`/`sbo` in bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}
// bf16 x bf16 -> fp32, M = 128, N = 128; b_mn_major selects the layout of B.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) |
         ((128u >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kPfThreads, 1)
prefill_kernel(const StepDevice s, const __grid_constant__ CUtensorMap kv_map,
               const __grid_constant__ CUtensorMap q_map) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t bar0 = base + kOffBar;
  auto bar = [&](int i) { return bar0 + (uint32_t)i * 8u; };
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);  // [0] tmem base, [1] dead

  const WorkItem it = s.items[blockIdx.x];
  const int kv_head = blockIdx.y;
  const int G = s.Hq / s.Hkv;
  const int ctx = s.row_ctx[it.row];
  const int q_len = s.row_qlen[it.row];
  const int tok0 = s.row_tok0[it.row];
  const int tile_tok = it.q_begin;                     // first token of the tile (inside the row)
  const int k_end = it.k_end;
  const int nb = (k_end + kBlockKeys - 1) / kBlockKeys;
  const bool fix_last = (k_end % kBlockKeys) != 0;

  if (tid == 0) {
    misc[1] = 0;
    for (int i = 0; i < BAR_COUNT; ++i) {
      const bool softmax_arrives = i >= BAR_P_FULL && i < BAR_P_FULL + 2;
      mbar_init(bar(i), softmax_arrives ? 128 : 1);
    }
    mbar_init_fence();
  }
  if (warp == 5) tmem_alloc(base + kOffMisc, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];
  const uint32_t tS0 = tmem, tO = tmem + 256;          // S buffers at columns 0 and 128, O at 256

  auto give_up = [&]() {
    if (misc[1] == 0) {
      atomicOr(s.status, TS_DEV_TIMEOUT);
      misc[1] = 1;
    }
  };
  auto wait = [&](int i, uint32_t parity) {
    if (!mbar_wait(bar(i), parity, misc[1] ? 2000 : kWaitCycles)) give_up();
  };

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    const int32_t* table_row = s.table + (size_t)s.row_slot[it.row] * s.max_pages_per_req;
    if (lane == 0) {
      tma_prefetch_desc(&kv_map);
      tma_prefetch_desc(&q_map);
      mbar_expect_tx(bar(BAR_Q), kTileBytes);
      tma_load_4d(base + kOffQ, &q_map, bar(BAR_Q), 0, 0, kv_head, tok0 + tile_tok);
      tma_load_4d(base + kOffQ + kHalfBytes, &q_map, bar(BAR_Q), 64, 0, kv_head, tok0 + tile_tok);
    }
    for (int j = 0; j < nb; ++j) {
      const int st = j % kKvStages;
      const uint32_t ph = (j / kKvStages) & 1;
      const int key0 = j * kBlockKeys;
      const int n_pg = min(8, (k_end - key0 + kPageSize - 1) / kPageSize);
      int page = 0;
      if (lane < n_pg) {
        page = table_row[(key0 >> 4) + lane];
        if ((unsigned)page >= (unsigned)s.n_pages) {
          atomicOr(s.status, TS_DEV_BAD_PAGE);
          page = s.n_pages;                            // out of range: the copy delivers zeros
        }
      }
      const int my_page = __shfl_sync(0xffffffffu, page, lane >> 1);
      for (int kv = 0; kv < 2; ++kv) {
        const int full = kv ? BAR_V_FULL : BAR_K_FULL, empty = kv ? BAR_V_EMPTY : BAR_K_EMPTY;
        if (j >= kKvStages) wait(empty + st, ph ^ 1);
        __syncwarp();
        if (!misc[1]) {
          if (lane == 0) mbar_expect_tx(bar(full + st), n_pg * 2 * kPageSize * kD);
          if (lane < 2 * n_pg) {
            const uint32_t dst = base + (kv ? kOffV : kOffK) + st * kTileBytes + (lane & 1) * kHalfBytes +
                                 (lane >> 1) * (kPageSize * 128);
            tma_load_5d(dst, &kv_map, bar(full + st), (lane & 1) * 64, 0, kv_head, kv, my_page);
          }
        }
      }
      if (j == nb - 1 && fix_last) {
        // rows of the V block past the last visible key hold stale bits: clear them, so that
        // a zero weight cannot meet a NaN
        wait(BAR_V_FULL + st, ph);
        const int valid = k_end - key0;
        unsigned char* vb = smem + kOffV + st * kTileBytes;
        for (int i = lane; i < (kBlockKeys - valid) * 16; i += 32) {
          const int r = valid + i / 16, c = i % 16;
          *reinterpret_cast<uint4*>(vb + (c >> 3) * kHalfBytes + r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_V_FIXED));
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(false), idesc_pv = instr_desc(true);
      auto issue_qk = [&](int j) {
        const int st = j % kKvStages;
        wait(BAR_K_FULL + st, (j / kKvStages) & 1);
        tc_fence_after();
        if (!misc[1]) {
          const uint32_t d = tS0 + (j & 1) * 128;
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks) {
            const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
            mma_ss(d, smem_desc(base + kOffQ + off, 0, 1024),
                   smem_desc(base + kOffK + st * kTileBytes + off, 0, 1024), idesc_qk, ks > 0);
          }
          tc_commit(bar(BAR_K_EMPTY + st));
          tc_commit(bar(BAR_S_FULL + (j & 1)));
        }
      };
      wait(BAR_Q, 0);
      issue_qk(0);
      for (int j = 0; j < nb; ++j) {
        if (j + 1 < nb) issue_qk(j + 1);
        const int st = j % kKvStages;
        wait(BAR_P_FULL + (j & 1), (j >> 1) & 1);
        wait(BAR_V_FULL + st, (j / kKvStages) & 1);
        if (j == nb - 1 && fix_last) wait(BAR_V_FIXED, 0);
        tc_fence_after();
        if (!misc[1]) {
          const uint32_t p = tS0 + (j & 1) * 128;      // P(j): bf16 pairs in the first 64 columns of S(j)
#pragma unroll
          for (int kk = 0; kk < kBlockKeys / 16; ++kk) {
            mma_ts(tO, p + kk * 8, smem_desc(base + kOffV + st * kTileBytes + kk * 2048, kHalfBytes, 1024),
                   idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(bar(BAR_V_EMPTY + st));
          tc_commit(bar(BAR_O_FULL));
        }
      }
    }
    __syncwarp();
  } else if (warp < 4) {
    // ---------------------------------------------------- softmax + epilogue (row = tid)
    const int row = tid;
    const int rows_used = (128 / G) * G;
    const int tok = tile_tok + row / G;
    const bool real = row < rows_used && tok < q_len;
    const int lim = real ? ctx + tok + 1 : k_end;       // keys at positions >= lim are masked
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    float m_ref = -CUDART_INF_F, l = 0.f;
    for (int j = 0; j < nb; ++j) {
      const uint32_t tS = tS0 + (j & 1) * 128 + lane_addr;
      wait(BAR_S_FULL + (j & 1), (j >> 1) & 1);
      tc_fence_after();
      float sv[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(sv[c], tS + c * 32);
      tmem_ld_wait();
      const int key0 = j * kBlockKeys;
      const bool need_mask = key0 + kBlockKeys > lim;
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float v = sv[c][i] * s.scale_log2;
          if (need_mask && key0 + c * 32 + i >= lim) v = -CUDART_INF_F;
          sv[c][i] = v;
          mx = fmaxf(mx, v);
        }
      }
      // lazy rescale: move the reference maximum only when it is exceeded by 2^threshold
      const bool move = mx > m_ref + kRescaleThreshold;   // first block: m_ref = -inf, so true
      float alpha = 1.f;
      if (move) {
        alpha = exp2f(m_ref - mx);                        // 0 on the first block
        m_ref = mx;
        l *= alpha;
      }
      if (j > 0 && __any_sync(0xffffffffu, move)) {
        wait(BAR_O_FULL, (j - 1) & 1);                    // P V of block j-1 has landed in O
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float ov[32];
          tmem_ld32(ov, tO + lane_addr + c * 32);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) ov[i] *= alpha;
          tmem_st32(tO + lane_addr + c * 32, ov);
        }
      }
      float rs = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float p0 = exp2f(sv[c][2 * i] - m_ref), p1 = exp2f(sv[c][2 * i + 1] - m_ref);
          rs += p0 + p1;
          pk[i] = pack2(p0, p1);
        }
        tmem_st16(tS + c * 16, pk);                        // P overwrites the part of S already consumed
      }
      l += rs;
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL + (j & 1)));
    }
    // epilogue: O / l -> bf16 -> global
    wait(BAR_O_FULL, (nb - 1) & 1);
    tc_fence_after();
    const float inv = 1.f / l;
    uint16_t* orow = s.out + ((size_t)(tok0 + tok) * s.Hq + kv_head * G + row % G) * kD;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float ov[32];
      tmem_ld32(ov, tO + lane_addr + c * 32);
      tmem_ld_wait();
      if (real) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 w;
          w.x = pack2(ov[8 * i] * inv, ov[8 * i + 1] * inv);
          w.y = pack2(ov[8 * i + 2] * inv, ov[8 * i + 3] * inv);
          w.z = pack2(ov[8 * i + 4] * inv, ov[8 * i + 5] * inv);
          w.w = pack2(ov[8 * i + 6] * inv, ov[8 * i + 7] * inv);
          *reinterpret_cast<uint4*>(orow + c * 32 + i * 8) = w;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 512);
}

}  // namespace

cudaError_t launch_prefill(const StepDevice& s, const CUtensorMap& kv_map, const CUtensorMap& q_map,
                           cudaStream_t stream) {
  if (s.n_prefill_items <= 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  prefill_kernel<<<dim3(s.n_prefill_items, s.Hkv), kPfThreads, kSmemBytes, stream>>>(s, kv_map, q_map);
  return cudaGetLastError();
}

}  // namespace ts
