// bf16 GEMM of the decoder layer around the attention step (sm_100a): C = A . B^T with fp32
// accumulation on the 5th-generation tensor cores.
//
//   A [M][K] bf16 (activations, one token per row), B [N][K] bf16 (weights, [out features][in
//   features]), C [M][N] bf16. Both operands are K-major, exactly as they sit in memory.
//
// One persistent CTA per SM walks the output tiles (tile index t -> column block t / m_tiles, row
// block t % m_tiles, so the CTAs that run at the same time share a few weight blocks through L2).
// A tile is TILE_M x 256: TILE_M = 128 (one tcgen05.mma M = 128, N = 256 per 16 of K) or 256 (two of
// them that share the weight block in shared memory, which cuts the bytes fetched per flop by a
// third). Operands arrive by TMA in 64-wide K blocks (128-byte swizzle) through a ring of stages;
// the accumulators live in TMEM (2 x 256 columns): with TILE_M = 128 they alternate between tiles,
// so the epilogue of a tile overlaps the main loop of the next one; with TILE_M = 256 a tile takes both.
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-5 epilogue
// (thread = accumulator row: TMEM -> registers -> bf16 -> global).
// Epilogues: plain store, store + residual (C = R + A . B^T), rotary embedding of the query and key
// heads of a fused QKV projection, and SiLU-gated product of a fused gate/up projection.
// Every wait is bounded; a wait that runs out raises TS_DEV_TIMEOUT and the CTA drains.
#include <cuda_bf16.h>

#include <algorithm>

#include "../../include/tokenscale.h"
#include "ts_internal.h"
#include "ts_ptx.h"
#include "ts_tc.h"
#include "ts_tma.h"

namespace ts {
namespace {

constexpr int kGemmThreads = 192;
constexpr int kBN = 256, kBK = 64;
constexpr int kABytes = 128 * kBK * 2;          // one 128-row operand block: 16 KB
constexpr int kBBytes = kBN * kBK * 2;          // the 256-row weight block: 32 KB

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// bf16 x bf16 -> fp32, M = 128, N = 256, both operands K-major
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ uint4 pack8(const float* v) {
  uint4 w;
  w.x = pack_bf16(v[0], v[1]);
  w.y = pack_bf16(v[2], v[3]);
  w.z = pack_bf16(v[4], v[5]);
  w.w = pack_bf16(v[6], v[7]);
  return w;
}
__device__ __forceinline__ void unpack8(const uint4& w, float* v) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}

template <int TILE_M, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const GemmArgs g, const __grid_constant__ CUtensorMap a_map, const __grid_constant__ CUtensorMap b_map) {
  constexpr int kMB = TILE_M / 128;                       // accumulators (and M = 128 MMAs per K step) of a tile
  constexpr int kStageBytes = kMB * kABytes + kBBytes;    // 48 KB or 64 KB
  constexpr int kStages = TILE_M == 128 ? 4 : 3;
  constexpr int kOffBar = kStages * kStageBytes;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  // barriers: full[kStages], empty[kStages], acc_full[2], acc_empty[2]
  auto bar = [&](int i) { return base + kOffBar + (uint32_t)i * 8u; };
  const int BAR_FULL = 0, BAR_EMPTY = kStages, BAR_ACC_FULL = 2 * kStages, BAR_ACC_EMPTY = 2 * kStages + 2;
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + kOffBar + (2 * kStages + 4) * 8);   // [0] TMEM base, [1] failure flag
  if (tid == 0) {
    misc[1] = 0;
    for (int i = 0; i < 2 * kStages + 2; ++i) mbar_init(bar(i), 1);
    mbar_init(bar(BAR_ACC_EMPTY), 128);
    mbar_init(bar(BAR_ACC_EMPTY + 1), 128);
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(base + kOffBar + (2 * kStages + 4) * 8, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];
  auto give_up = [&]() {
    if (misc[1] == 0) {
      atomicOr(g.status, TS_DEV_TIMEOUT);
      misc[1] = 1;
    }
  };
  auto wait = [&](int i, uint32_t parity) {
    if (!mbar_wait(bar(i), parity, misc[1] ? 2000 : g.wait_cycles)) give_up();
  };
  const int m_tiles = (g.M + TILE_M - 1) / TILE_M, n_tiles = (g.N + kBN - 1) / kBN;
  const int n_work = m_tiles * n_tiles;
  const int k_blocks = (g.K + kBK - 1) / kBK;
  pdl_wait();                      // the operands may come from the kernel in front of this one

  if (warp == 0) {
    // ---------------------------------------------------------------------- TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&a_map);
      tma_prefetch_desc(&b_map);
      int it = 0;                                          // K blocks issued so far (ring position)
      for (int t = blockIdx.x; t < n_work; t += gridDim.x) {
        const int m0 = (t % m_tiles) * TILE_M, n0 = (t / m_tiles) * kBN;
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const int st = it % kStages;
          if (it >= kStages) wait(BAR_EMPTY + st, ((it / kStages) & 1) ^ 1);
          if (misc[1]) continue;                           // after a failure no new copies are started
          const uint32_t dst = base + st * kStageBytes;
          mbar_expect_tx(bar(BAR_FULL + st), kStageBytes);
#pragma unroll
          for (int mb = 0; mb < kMB; ++mb) tma_load_2d(dst + mb * kABytes, &a_map, bar(BAR_FULL + st), kb * kBK, m0 + mb * 128);
          tma_load_2d(dst + kMB * kABytes, &b_map, bar(BAR_FULL + st), kb * kBK, n0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------ MMA issuer
    const uint32_t issue = elect_one();
    bool dead = false;
    auto iwait = [&](int i, uint32_t parity) {
      if (!mbar_poll(bar(i), parity, dead ? 2000 : g.wait_cycles)) {
        dead = true;
        give_up();
      }
    };
    int it = 0, n_done = 0;                                // K blocks consumed, tiles issued
    for (int t = blockIdx.x; t < n_work; t += gridDim.x, ++n_done) {
      // TILE_M = 128: tile n uses accumulator n % 2; TILE_M = 256: both, so every tile waits for the epilogue
      const int buf = kMB == 1 ? (n_done & 1) : 0;
      const int uses = kMB == 1 ? (n_done >> 1) : n_done;  // earlier tiles that used this accumulator
      if (uses > 0) {
        iwait(BAR_ACC_EMPTY + buf, (uses - 1) & 1);
        if (kMB == 2) iwait(BAR_ACC_EMPTY + 1, (uses - 1) & 1);
      }
      tc_fence_after();
      for (int kb = 0; kb < k_blocks; ++kb, ++it) {
        const int st = it % kStages;
        iwait(BAR_FULL + st, (it / kStages) & 1);
        tc_fence_after();
        if (!dead) {
          const uint64_t b_desc = smem_desc(base + st * kStageBytes + kMB * kABytes, 0, 1024);
#pragma unroll
          for (int mb = 0; mb < kMB; ++mb) {
            const uint64_t a_desc = smem_desc(base + st * kStageBytes + mb * kABytes, 0, 1024);
#pragma unroll
            for (int ks = 0; ks < kBK / 16; ++ks)          // 16 of K = 32 bytes along the swizzled row
              mma_ss(tmem + (kMB == 1 ? buf : mb) * 256, a_desc + (uint64_t)(ks * 2), b_desc + (uint64_t)(ks * 2), kIdesc,
                     (kb > 0 || ks > 0) ? 1u : 0u, issue);
          }
          tc_commit(bar(BAR_EMPTY + st), issue);           // the stage is free once these MMAs have read it
        }
      }
      if (!dead) {
        tc_commit(bar(BAR_ACC_FULL + buf), issue);
        if (kMB == 2) tc_commit(bar(BAR_ACC_FULL + 1), issue);
      }
    }
  } else {
    // --------------------------------------------------------------------------- epilogue
    const int q = warp & 3;                                // the TMEM lanes this warp can reach
    const int row_in_blk = q * 32 + lane;
    int n_done = 0;
    for (int t = blockIdx.x; t < n_work; t += gridDim.x, ++n_done) {
      const int m0 = (t % m_tiles) * TILE_M, n0 = (t / m_tiles) * kBN;
#pragma unroll 1
      for (int mb = 0; mb < kMB; ++mb) {
        const int buf = kMB == 1 ? (n_done & 1) : mb;
        const int uses = kMB == 1 ? (n_done >> 1) : n_done;
        wait(BAR_ACC_FULL + buf, uses & 1);
        tc_fence_after();
        const int row = m0 + mb * 128 + row_in_blk;
        const bool row_ok = row < g.M;
        const uint32_t tacc = tmem + buf * 256 + ((uint32_t)(q * 32) << 16);
        if (EPI == GEMM_EPI_STORE) {
          uint16_t* crow = g.C + (size_t)row * g.ldc + n0;
          const uint16_t* rrow = g.R ? g.R + (size_t)row * g.ldc + n0 : nullptr;
#pragma unroll 1
          for (int c = 0; c < kBN / 32; ++c) {
            float v[32];
            tmem_ld32(v, tacc + c * 32);
            tmem_ld_wait();
            if (c == kBN / 32 - 1) {
              tc_fence_before();
              mbar_arrive(bar(BAR_ACC_EMPTY + buf));       // the accumulator is in registers
            }
            if (row_ok) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int col = n0 + c * 32 + i * 8;
                if (col < g.N) {
                  if (rrow) {
                    float r[8];
                    unpack8(*reinterpret_cast<const uint4*>(rrow + c * 32 + i * 8), r);
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[i * 8 + e] += r[e];
                  }
                  *reinterpret_cast<uint4*>(crow + c * 32 + i * 8) = pack8(v + i * 8);
                }
              }
            }
          }
        } else if (EPI == GEMM_EPI_ROPE) {
          // A tile holds two heads of 128 columns. Query and key heads are rotated: column i < 64 of a
          // head pairs with column i + 64, angle table[pos][i]. Each head goes to its own tensor.
          const float2* cs = g.rope_table + (size_t)(row_ok ? g.pos[row] : 0) * 64;
#pragma unroll 1
          for (int h = 0; h < 2; ++h) {
            const int col0 = n0 + h * 128;
            const bool rotate = col0 < g.q_cols + g.kv_cols;
            uint16_t* dst = col0 < g.q_cols ? g.C + (size_t)row * g.q_cols + col0
                            : rotate        ? g.C2 + (size_t)row * g.kv_cols + (col0 - g.q_cols)
                                            : g.C3 + (size_t)row * g.kv_cols + (col0 - g.q_cols - g.kv_cols);
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
              float lo[32], hi[32];
              tmem_ld32(lo, tacc + h * 128 + c * 32);
              tmem_ld32(hi, tacc + h * 128 + 64 + c * 32);
              tmem_ld_wait();
              if (h == 1 && c == 1) {
                tc_fence_before();
                mbar_arrive(bar(BAR_ACC_EMPTY + buf));
              }
              if (row_ok && col0 < g.N) {
                if (rotate) {
#pragma unroll
                  for (int i = 0; i < 32; ++i) {
                    const float2 t2 = cs[c * 32 + i];     // (cos, sin)
                    const float a = lo[i], b = hi[i];
                    lo[i] = a * t2.x - b * t2.y;
                    hi[i] = b * t2.x + a * t2.y;
                  }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  *reinterpret_cast<uint4*>(dst + c * 32 + i * 8) = pack8(lo + i * 8);
                  *reinterpret_cast<uint4*>(dst + 64 + c * 32 + i * 8) = pack8(hi + i * 8);
                }
              }
            }
          }
        } else {
          // GEMM_EPI_SILU_MUL: the weight rows of a tile are 128 gate rows followed by the 128 up rows of
          // the same intermediate features; out[row][n0 / 2 + i] = silu(gate_i) * up_i, both
          // rounded to bf16 first (they are bf16 tensors of the layer's definition).
          uint16_t* crow = g.C + (size_t)row * g.ldc + n0 / 2;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            float gt[32], up[32];
            tmem_ld32(gt, tacc + c * 32);
            tmem_ld32(up, tacc + 128 + c * 32);
            tmem_ld_wait();
            if (c == 3) {
              tc_fence_before();
              mbar_arrive(bar(BAR_ACC_EMPTY + buf));
            }
            if (row_ok && n0 < g.N) {
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const float a = __bfloat162float(__float2bfloat16_rn(gt[i])), b = __bfloat162float(__float2bfloat16_rn(up[i]));
                gt[i] = a / (1.f + __expf(-a)) * b;
              }
#pragma unroll
              for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(crow + c * 32 + i * 8) = pack8(gt + i * 8);
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

template <int TILE_M, int EPI>
cudaError_t launch_t(const GemmArgs& g, const CUtensorMap& a_map, const CUtensorMap& b_map, int n_sms, cudaStream_t stream) {
  constexpr int kStageBytes = (TILE_M / 128) * kABytes + kBBytes;
  constexpr int kStages = TILE_M == 128 ? 4 : 3;
  const size_t smem = (size_t)kStages * kStageBytes + (2 * kStages + 4) * 8 + 16 + 1024;
  cudaError_t e = cudaFuncSetAttribute(gemm_kernel<TILE_M, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int m_tiles = (g.M + TILE_M - 1) / TILE_M, n_tiles = (g.N + kBN - 1) / kBN;
  const int grid = std::min(n_sms, m_tiles * n_tiles);
  return launch_pdl(gemm_kernel<TILE_M, EPI>, dim3(grid), dim3(kGemmThreads), smem, stream, g, a_map, b_map);
}

}  // namespace

int gemm_tile_m(int M, int N, int n_sms) {
  // Cost of a launch in units of a 128-row tile: waves x tile height, the taller tile being cheaper
  // per flop (it fetches a third fewer operand bytes) but coarser in the wave count.
  auto waves = [&](int tm) { return ((((M + tm - 1) / tm) * ((N + kBN - 1) / kBN)) + n_sms - 1) / n_sms; };
  const double c128 = waves(128) * 1.0, c256 = waves(256) * 2.0 * 0.9;
  return c256 < c128 ? 256 : 128;
}

cudaError_t launch_gemm(const GemmArgs& g, const CUtensorMap& a_map, const CUtensorMap& b_map, int tile_m, int n_sms,
                        cudaStream_t stream) {
  if (g.M <= 0 || g.N <= 0) return cudaSuccess;
  if (g.epi == GEMM_EPI_ROPE) return launch_t<128, GEMM_EPI_ROPE>(g, a_map, b_map, n_sms, stream);
  if (g.epi == GEMM_EPI_SILU_MUL)
    return tile_m == 256 ? launch_t<256, GEMM_EPI_SILU_MUL>(g, a_map, b_map, n_sms, stream)
                         : launch_t<128, GEMM_EPI_SILU_MUL>(g, a_map, b_map, n_sms, stream);
  return tile_m == 256 ? launch_t<256, GEMM_EPI_STORE>(g, a_map, b_map, n_sms, stream)
                       : launch_t<128, GEMM_EPI_STORE>(g, a_map, b_map, n_sms, stream);
}

}  // namespace ts
