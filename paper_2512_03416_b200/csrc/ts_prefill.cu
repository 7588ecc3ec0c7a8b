// Causal prefill-chunk attention on the 5th-generation tensor cores (sm_100a, head_dim 128).
//
// One CTA = one work item = two query tiles A and B of 128 packed rows each (128/G consecutive
// tokens x the G query heads of one KV head per tile) against all keys they may see, 128 keys per
// block. Per tile and block:
//     S = Q K^T   (tcgen05.mma, operands in 128B-swizzled shared memory, fp32 accumulator in TMEM)
//     online softmax by one warpgroup, one query row per thread, straight out of TMEM
//     O += P V    (tcgen05.mma, P read from TMEM as bf16, V from shared memory, O accumulates in TMEM)
// The two tiles share every K/V block (half the shared-memory fill per flop) and run out of phase:
// while one tile's warpgroup is in its softmax, the tensor pipe works for the other tile.
// TMEM (512 columns): S_A, S_B, O_A, O_B, 128 columns each; P overwrites the first 64 columns of
// its S. Warp roles: warps 0-3 softmax/epilogue of tile A, warps 4-7 of tile B (thread = TMEM lane =
// query row; the whole 128-score row of a block sits in the thread's registers), warps 8-9 K loaders, warps 10-11 V loaders (16-byte cp.async through the block table
// into the swizzled operand layout), warp 12 MMA issuer and TMEM owner; the Q tiles come by TMA.
// The O rescale is lazy: a row's reference maximum only moves when the new maximum exceeds it by
// more than 2^8, so most blocks never touch O.
// Every mbarrier wait is bounded; a wait that runs out raises TS_DEV_TIMEOUT and the CTA drains.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "../../include/tokenscale.h"
#include "ts_internal.h"
#include "ts_tma.h"

namespace ts {
namespace {

constexpr int kPfThreads = 512;                 // 8 softmax warps + 4 loader warps + MMA warp (+3 idle)
// Register split (setmaxnreg works on whole warpgroups, hence the three idle warps): the block is
// launched with 128 registers per thread; the two softmax warpgroups grow to hold their score
// row, the loader and MMA warpgroups shrink. 256 * 184 + 128 * 56 + 128 * 88 = 512 * 128.
constexpr int kRegsSoftmax = 184, kRegsLoader = 56, kRegsMma = 88;
static_assert(256 * kRegsSoftmax + 128 * kRegsLoader + 128 * kRegsMma <= 512 * 128,
              "register split exceeds the launch's total");
constexpr int kLoaderThreads = 64;              // per operand (K or V)
constexpr int kWarpLoader0 = 8, kWarpMma = 12;
constexpr int kBlockKeys = 128;
constexpr int kD = 128;
constexpr int kTileBytes = 128 * kD * 2;        // one 128 x 128 bf16 operand tile: 32 KB
constexpr int kHalfBytes = kTileBytes / 2;      // 64 head_dim columns of it
constexpr int kKStages = 3, kVStages = 2;
constexpr float kRescaleThreshold = 8.0f;       // log2 units

// shared-memory map (offsets from the 1024-aligned base)
constexpr int kOffQ = 0;                                    // Q_A, Q_B
constexpr int kOffK = kOffQ + 2 * kTileBytes;
constexpr int kOffV = kOffK + kKStages * kTileBytes;
constexpr int kOffBar = kOffV + kVStages * kTileBytes;
enum {
  BAR_Q = 0,
  BAR_K_FULL = 1,                         // [kKStages]
  BAR_K_EMPTY = BAR_K_FULL + kKStages,    // [kKStages]
  BAR_V_FULL = BAR_K_EMPTY + kKStages,    // [kVStages]
  BAR_V_EMPTY = BAR_V_FULL + kVStages,    // [kVStages]
  BAR_S_FULL = BAR_V_EMPTY + kVStages,    // [2] per tile
  BAR_P_FULL = BAR_S_FULL + 2,            // [2] per tile
  BAR_O_FULL = BAR_P_FULL + 2,            // [2] per tile
  BAR_COUNT = BAR_O_FULL + 2
};
constexpr int kOffMisc = kOffBar + BAR_COUNT * 8;   // tmem base address, dead flag
constexpr int kSmemBytes = kOffMisc + 16 + 1024;
static_assert(kSmemBytes <= 232448, "exceeds the shared memory one CTA can opt into");

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
__device__ __forceinline__ void tmem_ld32(float* v, uint32_t taddr) {
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
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
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  // src_bytes == 0 writes 16 zero bytes and reads nothing
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(N)); }
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Packed pairs of fp32 (sm_100 has two-wide fp32 add/fma): half the issue slots of scalar code.
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;\n" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// One row of a score block: p_i = 2^(v_i * scale + neg_m) for the 128 scores in v, written as bf16
// pairs into TMEM columns [t_p, t_p + 64); returns the row sum of the unrounded p_i.
__device__ __forceinline__ float exp_store(const float (&v)[128], float scale, float neg_m, uint32_t t_p) {
  const uint64_t scale2 = pack_f2(scale, scale), negm2 = pack_f2(neg_m, neg_m);
  uint64_t sum_a = pack_f2(0.f, 0.f), sum_b = sum_a;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int e = c * 32 + 2 * i;
      float x0, x1;
      unpack_f2(fma2(pack_f2(v[e], v[e + 1]), scale2, negm2), x0, x1);
      const float p0 = ex2(x0), p1 = ex2(x1);
      if (i & 1) sum_b = add2(sum_b, pack_f2(p0, p1)); else sum_a = add2(sum_a, pack_f2(p0, p1));
      pk[i] = pack2(p0, p1);
    }
    tmem_st16(t_p + c * 16, pk);
  }
  float a0, a1;
  unpack_f2(add2(sum_a, sum_b), a0, a1);
  return a0 + a1;
}

__global__ void __launch_bounds__(kPfThreads, 1)
prefill_kernel(const StepDevice s, const __grid_constant__ CUtensorMap q_map) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  const uint32_t bar0 = base + kOffBar;
  auto bar = [&](int i) { return bar0 + (uint32_t)i * 8u; };
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);  // [0] tmem base, [1] dead

  const WorkItem it = s.items[blockIdx.y];   // grid = (KV heads, items): every head of a heavy item starts early
  const int kv_head = blockIdx.x;
  const int G = s.Hq / s.Hkv;
  const int ctx = s.row_ctx[it.row];
  const int tok0 = s.row_tok0[it.row];
  // tile A: tokens [q_begin, q_begin + cnt_a), tile B: the cnt_b tokens after them (maybe none)
  const int tile_tokens = 128 / G;
  const int cnt_a = min(it.q_count, tile_tokens), cnt_b = it.q_count - cnt_a;
  const int k_end_a = ctx + it.q_begin + cnt_a, k_end_b = k_end_a + cnt_b;
  const int nb_a = (k_end_a + kBlockKeys - 1) / kBlockKeys;
  const int nb_b = cnt_b > 0 ? (k_end_b + kBlockKeys - 1) / kBlockKeys : 0;
  const int nb = max(nb_a, nb_b);                       // K/V blocks this CTA streams
  const int k_end = max(k_end_a, k_end_b);

  if (tid == 0) {
    misc[1] = 0;
    for (int i = 0; i < BAR_COUNT; ++i) {
      const bool softmax_arrives = i >= BAR_P_FULL && i < BAR_P_FULL + 2;
      const bool loaders_arrive = (i >= BAR_K_FULL && i < BAR_K_FULL + kKStages) ||
                                  (i >= BAR_V_FULL && i < BAR_V_FULL + kVStages);
      mbar_init(bar(i), softmax_arrives ? 128 : loaders_arrive ? kLoaderThreads : 1);
    }
    mbar_init_fence();
  }
  if (warp == kWarpMma) tmem_alloc(base + kOffMisc, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                  // set-up done; from here on the pool, tables and Q are read
  const uint32_t tmem = misc[0];

  auto give_up = [&]() {
    if (misc[1] == 0) {
      atomicOr(s.status, TS_DEV_TIMEOUT);
      misc[1] = 1;
    }
  };
  auto wait = [&](int i, uint32_t parity) {
    if (!mbar_wait(bar(i), parity, misc[1] ? 2000 : kWaitCycles)) give_up();
  };

  if (warp >= kWarpLoader0 && warp < kWarpLoader0 + 4) {
    // ------------------------------------------------------------------ K/V loaders
    reg_dec<kRegsLoader>();
    // 64 threads per operand copy each 128-key tile with 16-byte cp.async straight into the
    // 128-byte-swizzled operand layout. (TMA is not used for K/V: with 16-token pages every
    // tensor copy is only 2 KB, and the copy engine's per-request cost would bound the kernel.)
    // K and V are two independent pipelines. A tile is announced at the start of a later
    // iteration of its own loader, before that iteration waits for a free stage, so the
    // announcement depends only on the copy having landed.
    const int kv = (warp - kWarpLoader0) >> 1;               // 0: K, 1: V
    const int t = tid - 256 - kv * kLoaderThreads;           // 0..63 inside the group
    const int col16 = t & 15, rb = t >> 4;                   // chunk col16 of rows rb + 4 h + 8 i
    const int32_t* table_row = s.table + (size_t)s.row_slot[it.row] * s.max_pages_per_req;
    if (kv == 0 && t == 0) {
      tma_prefetch_desc(&q_map);
      mbar_expect_tx(bar(BAR_Q), (cnt_b > 0 ? 2 : 1) * kTileBytes);
      const int ta = tok0 + it.q_begin;
      tma_load_4d(base + kOffQ, &q_map, bar(BAR_Q), 0, 0, kv_head, ta);
      tma_load_4d(base + kOffQ + kHalfBytes, &q_map, bar(BAR_Q), 64, 0, kv_head, ta);
      if (cnt_b > 0) {
        tma_load_4d(base + kOffQ + kTileBytes, &q_map, bar(BAR_Q), 0, 0, kv_head, ta + tile_tokens);
        tma_load_4d(base + kOffQ + kTileBytes + kHalfBytes, &q_map, bar(BAR_Q), 64, 0, kv_head, ta + tile_tokens);
      }
    }
    const int stages = kv ? kVStages : kKStages;
    const int lag = stages - 1;                              // tiles in flight besides the announced one
    const int full = kv ? BAR_V_FULL : BAR_K_FULL, empty = kv ? BAR_V_EMPTY : BAR_K_EMPTY;
    const uint32_t tile0 = base + (kv ? kOffV : kOffK);
    const size_t head_off = ((size_t)kv * s.Hkv + kv_head) * kPageSize * kD + col16 * 8;
    const size_t page_stride = (size_t)2 * s.Hkv * kPageSize * kD;
    auto fetch_pages = [&](int j, int (&pg)[8]) {
#pragma unroll
      for (int p = 0; p < 8; ++p) {
        const int key = j * kBlockKeys + p * kPageSize;
        int page = -1;
        if (key < k_end) {
          page = table_row[key >> 4];
          if ((unsigned)page >= (unsigned)s.n_pages) {
            atomicOr(s.status, TS_DEV_BAD_PAGE);
            page = -1;
          }
        }
        pg[p] = page;
      }
    };
    auto announce = [&](int tile, int pending_allowed) {
      if (pending_allowed >= 1) cp_async_wait<1>(); else cp_async_wait<0>();
      fence_proxy_async();
      mbar_arrive(bar(full + tile % stages));
    };
    int pg[8];
    fetch_pages(0, pg);
    for (int j = 0; j < nb; ++j) {
      const int st = j % stages;
      const int key0 = j * kBlockKeys;
      if (j >= lag) announce(j - lag, lag - 1);              // K: tile j-2 (j-1 in flight); V: tile j-1
      int pg_next[8];
      if (j + 1 < nb) fetch_pages(j + 1, pg_next);           // table loads fly while this tile is issued
      if (j >= stages) wait(empty + st, ((j / stages) & 1) ^ 1);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r0 = rb + 4 * h;
        const uint32_t dst = tile0 + st * kTileBytes +
                             (uint32_t)((col16 >> 3) * kHalfBytes + r0 * 128 + (((col16 & 7) ^ r0) << 4));
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int row = r0 + 8 * i;
          const int page = pg[i >> 1];
          const bool valid = page >= 0 && key0 + row < k_end;   // rows past the last key are zero-filled
          const uint16_t* src = valid ? s.pool + (size_t)page * page_stride + head_off + (row & 15) * kD : s.pool;
          cp_async16(dst + i * 1024, src, valid ? 16 : 0);
        }
      }
      cp_async_commit();
#pragma unroll
      for (int p = 0; p < 8; ++p) pg[p] = pg_next[p];
    }
    // the last `lag` tiles (fewer when the item is short) have not been announced yet
    for (int tile = max(0, nb - lag); tile < nb; ++tile) announce(tile, nb - 1 - tile);
  } else if (warp == kWarpMma) {
    // ------------------------------------------------------------------- MMA issuer
    reg_dec<kRegsMma>();
    if (lane == 0) {
      // the issuer keeps its own failure flag in a register: nothing on its path reads shared memory
      bool dead = false;
      auto wait = [&](int i, uint32_t parity) {
        if (!mbar_wait(bar(i), parity, dead ? 2000 : kWaitCycles)) {
          dead = true;
          give_up();
        }
      };
      constexpr uint32_t idesc_qk = instr_desc(false), idesc_pv = instr_desc(true);
      // descriptors differ only in their start-address field (16-byte units in the low bits)
      const uint64_t q_desc0 = smem_desc(base + kOffQ, 0, 1024);
      const uint64_t k_desc0 = smem_desc(base + kOffK, 0, 1024);
      const uint64_t v_desc0 = smem_desc(base + kOffV, kHalfBytes, 1024);
      auto issue_qk = [&](int x, int j) {          // S_x = Q_x K(j)^T
        const uint64_t q_desc = q_desc0 + (uint64_t)((x * kTileBytes) >> 4);
        const uint64_t k_desc = k_desc0 + (uint64_t)(((j % kKStages) * kTileBytes) >> 4);
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint64_t off = (uint64_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
          mma_ss(tmem + x * 128, q_desc + off, k_desc + off, idesc_qk, ks > 0);
        }
        tc_commit(bar(BAR_S_FULL + x));
      };
      auto issue_pv = [&](int x, int j) {          // O_x += P_x V(j)
        const uint64_t v_desc = v_desc0 + (uint64_t)(((j % kVStages) * kTileBytes) >> 4);
#pragma unroll
        for (int kk = 0; kk < kBlockKeys / 16; ++kk)
          mma_ts(tmem + 256 + x * 128, tmem + x * 128 + kk * 8, v_desc + (uint64_t)((kk * 2048) >> 4), idesc_pv,
                 (j > 0 || kk > 0) ? 1u : 0u);
        tc_commit(bar(BAR_O_FULL + x));
      };
      // Order: both Q K^T of block 0; then per block, for tile A then tile B:
      // P V of block j followed at once by Q K^T of block j+1 of the same tile, so that the
      // tile's warpgroup gets its next scores while the pipe turns to the other tile.
      wait(BAR_Q, 0);
      wait(BAR_K_FULL + 0, 0);
      tc_fence_after();
      if (!dead) {
        if (nb_a > 0) issue_qk(0, 0);
        if (nb_b > 0) issue_qk(1, 0);
        tc_commit(bar(BAR_K_EMPTY + 0));
      }
      for (int j = 0; j < nb; ++j) {
        const bool next = j + 1 < nb;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int nbx = x ? nb_b : nb_a;
          if (j < nbx) {
            wait(BAR_P_FULL + x, j & 1);
            if (x == 0 || j >= nb_a) wait(BAR_V_FULL + j % kVStages, (j / kVStages) & 1);
            tc_fence_after();
            if (!dead) issue_pv(x, j);
          }
          if (x == 1 && !dead) tc_commit(bar(BAR_V_EMPTY + j % kVStages));   // both tiles are done with V(j)
          if (next) {
            if (x == 0 || j + 1 >= nb_a) wait(BAR_K_FULL + (j + 1) % kKStages, ((j + 1) / kKStages) & 1);
            tc_fence_after();
            if (j + 1 < nbx && !dead) issue_qk(x, j + 1);
            if (x == 1 && !dead) tc_commit(bar(BAR_K_EMPTY + (j + 1) % kKStages));
          }
        }
      }
    }
    __syncwarp();
  } else if (warp < 8) {
    // ------------------------------------------ softmax + epilogue: thread = query row of tile x
    reg_inc<kRegsSoftmax>();
    const int x = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const int nbx = x ? nb_b : nb_a;
    const int cnt = x ? cnt_b : cnt_a;
    const int tok = it.q_begin + x * tile_tokens + row / G;   // token inside the request row
    const bool real = row / G < cnt && row < tile_tokens * G;
    const int k_end_x = x ? k_end_b : k_end_a;
    const int lim = real ? ctx + tok + 1 : k_end_x;           // keys at positions >= lim are masked
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + x * 128 + lane_addr, tO = tmem + 256 + x * 128 + lane_addr;
    const float scale = s.scale_log2;
    float m_ref = -CUDART_INF_F, l = 0.f;
    for (int j = 0; j < nbx; ++j) {
      wait(BAR_S_FULL + x, j & 1);
      tc_fence_after();
      // the whole score row lives in registers: one trip to TMEM per block
      float v[128];
      tmem_ld32(&v[0], tS);
      tmem_ld32(&v[32], tS + 32);
      tmem_ld32(&v[64], tS + 64);
      tmem_ld32(&v[96], tS + 96);
      tmem_ld_wait();
      const int nvalid = lim - j * kBlockKeys;               // keys of this block the row may see
      if (__any_sync(0xffffffffu, nvalid < kBlockKeys)) {    // only the blocks on the diagonal
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (i >= nvalid) v[i] = -CUDART_INF_F;             // 2^(-inf) = 0 exactly
      }
      // row maximum of the raw scores (the scale is positive, so it commutes with max)
      float m0 = max3(v[0], v[1], v[2]), m1 = max3(v[3], v[4], v[5]);
      float m2 = max3(v[6], v[7], v[8]), m3 = max3(v[9], v[10], v[11]);
#pragma unroll
      for (int i = 12; i < 124; i += 8) {
        m0 = max3(m0, v[i], v[i + 1]);
        m1 = max3(m1, v[i + 2], v[i + 3]);
        m2 = max3(m2, v[i + 4], v[i + 5]);
        m3 = max3(m3, v[i + 6], v[i + 7]);
      }
      m0 = max3(m0, v[124], v[125]);
      m1 = max3(m1, v[126], v[127]);
      const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * scale;
      // lazy rescale: move the reference maximum only when it is exceeded by 2^threshold
      const bool move = mx > m_ref + kRescaleThreshold;   // first block: m_ref = -inf, so true
      float alpha = 1.f;
      if (move) {
        alpha = ex2(m_ref - mx);                          // 0 on the first block
        m_ref = mx;
        l *= alpha;
      }
      if (j > 0 && __any_sync(0xffffffffu, move)) {
        wait(BAR_O_FULL + x, (j - 1) & 1);                // P V of block j-1 has landed in O
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float ov[32];
          tmem_ld32(ov, tO + c * 32);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) ov[i] *= alpha;
          tmem_st32(tO + c * 32, ov);
        }
      }
      // p = 2^(s*scale - m_ref) as bf16 over the first 64 columns of S (the scores are in registers)
      l += exp_store(v, scale, -m_ref, tS);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL + x));
    }
    if (nbx > 0) {
      // epilogue: O / l -> bf16 -> global
      wait(BAR_O_FULL + x, (nbx - 1) & 1);
      tc_fence_after();
      const float inv = 1.f / l;
      uint16_t* orow = s.out + ((size_t)(tok0 + tok) * s.Hq + kv_head * G + row % G) * kD;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float ov[32];
        tmem_ld32(ov, tO + c * 32);
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
  } else {
    reg_dec<kRegsMma>();        // warps 13-15 only complete the fourth warpgroup
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) tmem_dealloc(tmem, 512);
}

}  // namespace

cudaError_t launch_prefill(const StepDevice& s, const CUtensorMap& q_map, cudaStream_t stream) {
  if (s.n_prefill_items <= 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  return launch_pdl(prefill_kernel, dim3(s.Hkv, s.n_prefill_items), dim3(kPfThreads), kSmemBytes, stream, s, q_map);
}

}  // namespace ts
