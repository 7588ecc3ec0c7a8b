// The attention kernel of a mixed step (sm_100a, head_dim 128): causal prefill-chunk tiles on the
// 5th-generation tensor cores and, in the same launch, the split-KV decode units.
//
// One persistent CTA per SM. The first n_prefill_ctas CTAs take prefill work units (prefill work
// item x KV head) from a global queue, heaviest first. The remaining CTAs first run their static
// share of the decode units (dec::decode_units: TMA page copies, bound by HBM bandwidth) and then
// join the prefill queue, so that the HBM-bound and the tensor-bound halves of a step overlap
// instead of running back to back, and whichever CTAs finish first pick up what is left.
//
// A prefill work unit = two query tiles A and B of 128 packed rows each (128/G consecutive tokens
// x the G query heads of one KV head per tile) against all keys they may see, 128 keys per block.
// Per tile and block:
//     S = Q K^T   (tcgen05.mma, operands in 128B-swizzled shared memory, fp32 accumulator in TMEM)
//     online softmax by two warpgroups, two threads per query row, half a score row in registers each
//     O += P V    (tcgen05.mma, P read from TMEM as bf16, V from shared memory, O accumulates in TMEM)
// The two tiles share every K/V block (half the shared-memory fill per flop) and run out of phase:
// while one tile's warpgroups are in their softmax, the tensor pipe works for the other tile.
// TMEM (512 columns): S_A, S_B, O_A, O_B, 128 columns each; the P of the keys in a 64-column half
// of S overwrites the first 32 columns of that half.
// Warp roles: warps 0-3 / 8-11 softmax and epilogue of tile A (keys 0-63 / 64-127 of each block,
// head_dim columns 0-63 / 64-127 of O), warps 4-7 / 12-15 the same for tile B (thread = TMEM lane =
// query row; a warp can only reach the 32 lanes its index modulo 4 selects, so a row is split by
// columns). The two threads of a row agree on the row maximum through shared memory and a
// 64-thread mbarrier per block. Two softmax warps per tile and SM sub-partition hide each
// other's instruction latencies: one warp per row quarter left the tensor pipe idle more than
// half of the time although no unit was saturated. Warp 16 K loader, warp 17 V loader (16-byte
// cp.async through the block table into the swizzled operand layout; the K loader's first thread
// also claims the work units), warp 18 MMA issuer and TMEM owner, warp 19 Q loader (TMA).
// All barrier phases follow running block counters, so the roles flow from one work unit into the
// next without a CTA-wide stop: the loaders run ahead into the next unit's K/V, its Q tiles land
// as soon as the last Q K^T of the current unit has been issued, and its first Q K^T overlaps
// the epilogue of the current unit.
// The O rescale is lazy: a row's reference maximum only moves when a block's maximum exceeds it by
// more than 2^8, so most blocks never touch O.
// The kernel appends the step's new K/V to the pages itself, which saves a launch in front of it:
// every CTA copies a share of the prefill rows' tokens (in a CTA that streams decode rows first, the
// loader warpgroup does, next to the stream), and only the CTAs about to start on prefill work wait
// for all of them; the decode units write their rows' own tokens.
// Every wait is bounded; a wait that runs out raises TS_DEV_TIMEOUT and the CTA drains.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "../../include/tokenscale.h"
#include "ts_decode_body.h"
#include "ts_internal.h"
#include "ts_ptx.h"
#include "ts_tc.h"
#include "ts_tma.h"

namespace ts {
namespace {

constexpr int kPfThreads = 640;                 // 16 softmax warps + K loader, V loader, MMA and Q-loader warps
constexpr int kSoftmaxWarps = 16;
// Register split (setmaxnreg works on whole warpgroups): the block is launched with 96 registers
// per thread; the four softmax warpgroups grow to hold their half score row, the fifth warpgroup
// (loaders, MMA issuer) shrinks. In a CTA that runs decode units first, the two warpgroups that run
// them take the registers the other two softmax warpgroups do not need yet.
constexpr int kRegsLaunch = 96, kRegsSoftmax = 104, kRegsAux = 64, kRegsDecode = 168, kRegsParked = 24;
static_assert(4 * 128 * kRegsSoftmax + 128 * kRegsAux <= kPfThreads * kRegsLaunch,
              "register split exceeds the launch's total");
static_assert(2 * 128 * kRegsDecode + 2 * 128 * kRegsParked + 128 * kRegsAux <= kPfThreads * kRegsLaunch,
              "register split of the decode phase exceeds the launch's total");
constexpr int kWarpLoader0 = 16, kWarpMma = 18, kWarpSched = 19;
constexpr int kBlockKeys = 128;
constexpr int kD = 128;
constexpr int kTileBytes = 128 * kD * 2;        // one 128 x 128 bf16 operand tile: 32 KB
constexpr int kHalfBytes = kTileBytes / 2;      // 64 head_dim columns of it
constexpr int kKStages = 2, kVStages = 3;       // measured: a third V stage is worth more than a third K stage (3%)
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
  BAR_O_EMPTY = BAR_O_FULL + 2,           // [2] per tile: the epilogue has read O out of TMEM
  BAR_Q_EMPTY = BAR_O_EMPTY + 2,          // the last Q K^T of a work unit has consumed the Q tiles
  BAR_PAIR = BAR_Q_EMPTY + 1,             // [8] per tile and row quarter: the two warps that share the rows
  BAR_V_LANDED = BAR_PAIR + 8,            // [kVStages] the copies of a V tile are in shared memory
  BAR_COUNT = BAR_V_LANDED + kVStages
};
// misc words: [0] TMEM base address, [1] failure flag, [2] work units published so far;
// then a ring of the published units' records (8 words each)
constexpr int kOffMisc = kOffBar + BAR_COUNT * 8;
constexpr int kOffRing = kOffMisc + 16;
constexpr int kSchedRing = 8;
// row statistics the two threads of a query row exchange: [tile][half][row] floats
constexpr int kOffXchg = kOffRing + kSchedRing * 32;
constexpr int kSmemBytes = kOffXchg + 2 * 2 * 128 * 4;
// The operand tiles need a 1024-byte-aligned base. The kernel has no static shared memory, so its
// dynamic window starts on such a boundary; the kernel checks that and refuses to run otherwise
// (there is no room left for alignment slack).
static_assert(kSmemBytes <= 232448, "exceeds the shared memory one CTA can opt into");

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

// Half a row of a score block: p_i = 2^(x_i), x_i = v_i * scale + neg_m, for the 64 scores in v,
// as bf16 pairs in pk (the scores are not needed afterwards, so their registers come free as
// the loop advances); returns the sum of the unrounded p_i and, in x_max, the largest x_i (it
// rides along in issue slots the exponentials leave free).
__device__ __forceinline__ float exp_pack(const float (&v)[64], float scale, float neg_m, uint32_t (&pk)[32], float& x_max) {
  const uint64_t scale2 = pack_f2(scale, scale), negm2 = pack_f2(neg_m, neg_m);
  uint64_t sum_a = pack_f2(0.f, 0.f), sum_b = sum_a;
  float xm0 = -CUDART_INF_F, xm1 = xm0;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    float x0, x1, p0, p1;
    unpack_f2(fma2(pack_f2(v[2 * i], v[2 * i + 1]), scale2, negm2), x0, x1);
    if (i & 1) xm1 = max3(xm1, x0, x1); else xm0 = max3(xm0, x0, x1);
    p0 = ex2(x0);
    p1 = ex2(x1);
    if (i & 1) sum_b = add2(sum_b, pack_f2(p0, p1)); else sum_a = add2(sum_a, pack_f2(p0, p1));
    pk[i] = pack_bf16(p0, p1);
  }
  x_max = fmaxf(xm0, xm1);
  float a0, a1;
  unpack_f2(add2(sum_a, sum_b), a0, a1);
  return a0 + a1;
}
// Largest of the 64 raw scores of a half row.
__device__ __forceinline__ float max64(const float (&v)[64]) {
  float m0 = max3(v[0], v[1], v[2]), m1 = max3(v[3], v[4], v[5]);
  float m2 = max3(v[6], v[7], v[8]), m3 = max3(v[9], v[10], v[11]);
#pragma unroll
  for (int i = 12; i < 60; i += 8) {
    m0 = max3(m0, v[i], v[i + 1]);
    m1 = max3(m1, v[i + 2], v[i + 3]);
    m2 = max3(m2, v[i + 4], v[i + 5]);
    m3 = max3(m3, v[i + 6], v[i + 7]);
  }
  m0 = max3(m0, v[60], v[61]);
  m1 = max3(m1, v[62], v[63]);
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}
// One prefill work unit as its claimer publishes it in shared memory (8 words), and the shape
// every role derives from it.
struct UnitRec {
  int32_t w;                 // work unit index, -1 = the queue is empty
  int32_t table_slot;        // request slot: row of the block table
  int32_t kv_head, q_begin, q_count;
  int32_t ctx;               // tokens cached before the chunk
  int32_t tok0;              // first token of the request row in the step's tensors
  int32_t pad;
};
static_assert(sizeof(UnitRec) == 32, "UnitRec is 8 words");
struct PfUnit {
  int table_slot, kv_head, q_begin, ctx, tok0;
  int cnt_a, cnt_b;          // tokens of tile A / tile B (tile B may be empty)
  int k_end_a, k_end_b;      // one past the last key any row of the tile may see
  int nb_a, nb_b, nb;        // key blocks per tile, and of the unit
  int k_end;
};
__device__ __forceinline__ PfUnit unit_shape(const UnitRec& r, int tile_tokens) {
  PfUnit u;
  u.table_slot = r.table_slot;
  u.kv_head = r.kv_head;
  u.q_begin = r.q_begin;
  u.ctx = r.ctx;
  u.tok0 = r.tok0;
  u.cnt_a = min(r.q_count, tile_tokens);
  u.cnt_b = r.q_count - u.cnt_a;
  u.k_end_a = u.ctx + r.q_begin + u.cnt_a;
  u.k_end_b = u.k_end_a + u.cnt_b;
  u.nb_a = (u.k_end_a + kBlockKeys - 1) / kBlockKeys;
  u.nb_b = u.cnt_b > 0 ? (u.k_end_b + kBlockKeys - 1) / kBlockKeys : 0;
  u.nb = max(u.nb_a, u.nb_b);
  u.k_end = max(u.k_end_a, u.k_end_b);
  return u;
}

__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 0;\n" ::: "memory"); }

__global__ void __launch_bounds__(kPfThreads, 1)
mixed_kernel(const StepDevice s, const __grid_constant__ CUtensorMap q_map,
             const __grid_constant__ CUtensorMap kv_map, const __grid_constant__ CUtensorMap kv_tile_map,
             const int n_prefill_ctas) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  if (base != smem_u32(smem_raw)) {          // never expected, see kSmemBytes
    if (tid == 0) atomicOr(s.status, TS_DEV_BAD_INDEX);
    return;
  }
  const uint32_t bar0 = base + kOffBar;
  auto bar = [&](int i) { return bar0 + (uint32_t)i * 8u; };
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  const int G = s.Hq / s.Hkv;
  const int tile_tokens = 128 / G;
  const int n_units = s.n_prefill_items * s.Hkv;
  const bool decode_first = (int)blockIdx.x >= n_prefill_ctas;

  auto give_up = [&]() {
    if (misc[1] == 0) {
      atomicOr(s.status, TS_DEV_TIMEOUT);
      misc[1] = 1;
    }
  };
  auto wait = [&](int i, uint32_t parity) {
    if (!mbar_wait(bar(i), parity, misc[1] ? 2000 : s.wait_cycles)) give_up();
  };
  // k-th work unit of this CTA (w = -1 after the last one), published by the K loaders' first thread
  volatile int4* ring = reinterpret_cast<volatile int4*>(smem + kOffRing);
  auto get_work = [&](int k, PfUnit& u) -> bool {
    if ((int)misc[2] <= k) {
      const long long t0 = clock64();
      while ((int)misc[2] <= k) {
        if (clock64() - t0 > (misc[1] ? 2000 : s.wait_cycles)) {
          give_up();
          return false;
        }
      }
    }
    UnitRec r;
    const int e = (k & (kSchedRing - 1)) * 2;
    const int4 lo = make_int4(ring[e].x, ring[e].y, ring[e].z, ring[e].w);
    const int4 hi = make_int4(ring[e + 1].x, ring[e + 1].y, ring[e + 1].z, ring[e + 1].w);
    r.w = lo.x; r.table_slot = lo.y; r.kv_head = lo.z; r.q_begin = lo.w;
    r.q_count = hi.x; r.ctx = hi.y; r.tok0 = hi.z;
    if (r.w < 0) return false;
    u = unit_shape(r, tile_tokens);
    return true;
  };
  // The set-up every warp class runs between the decode phase and the prefill phase.
  auto prefill_setup = [&]() {
    if (tid == 0) {
      misc[1] = 0;
      misc[2] = 0;
      {   // the prefill rows' new K/V must be in their pages before the first tile is read
        const volatile int32_t* arrived = s.pf_queue + 2;
        const long long t0 = clock64();
        while (*arrived < s.append_arrivals) {
          if (clock64() - t0 > s.wait_cycles) {
            atomicOr(s.status, TS_DEV_TIMEOUT);
            break;
          }
        }
        __threadfence();
      }
      for (int i = 0; i < BAR_COUNT; ++i) {
        const bool softmax_arrives = (i >= BAR_P_FULL && i < BAR_P_FULL + 2) || (i >= BAR_O_EMPTY && i < BAR_O_EMPTY + 2);
        const bool pair = i >= BAR_PAIR && i < BAR_PAIR + 8;
        mbar_init(bar(i), softmax_arrives ? 256 : pair ? 64 : 1);
      }
      mbar_init_fence();
    }
    if (warp == kWarpMma) tmem_alloc(base + kOffMisc, 512);
    // When G does not divide 128 a query tile holds tile_tokens * G < 128 packed rows and the Q
    // copies never write the rest: clear those rows once, so that the MMA reads zeros there and
    // not whatever the shared memory held before.
    const int used_rows = tile_tokens * G;
    if (used_rows < 128) {
      const int n16 = (128 - used_rows) * 8;                 // 16-byte chunks per 64-column half tile
      for (int i = tid; i < 4 * n16; i += kPfThreads) {
        const int half = i / n16, c = i % n16;
        *reinterpret_cast<uint4*>(smem + kOffQ + half * kHalfBytes + used_rows * 128 + c * 16) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async();
    }
    tc_fence_before();
    cta_sync();
    tc_fence_after();
  };
  // ---------------------------------------------------------------- KV append (Sec. 2.1)
  // Every CTA copies a share of the new tokens of the prefill rows into their pages, straight from
  // the prefill work items (which cover those tokens exactly once), and counts itself; a CTA waits
  // for that count only before its first prefill unit (prefill_setup). In a CTA that takes prefill
  // units from the start all twenty warps copy. In a CTA that streams decode rows first only the
  // fifth warpgroup copies (aux_setup) while warps 0-7 are already on their decode units: nothing
  // those read depends on this append (the new token of a decode row is written by the decode unit
  // that reads the row's last page), so the page stream starts with the kernel.
  constexpr int kWarpsAll = kPfThreads / 32, kWarpsAux = 4;
  const int append_warps = n_prefill_ctas * kWarpsAll + ((int)gridDim.x - n_prefill_ctas) * kWarpsAux;
  // The fifth warpgroup (loaders, MMA issuer, Q loader): gives registers to the softmax warpgroups
  // and, in a decode-first CTA, appends and then waits while warps 0-7 run the CTA's decode units.
  auto aux_setup = [&]() {
    reg_dec<kRegsAux>();
    if (decode_first) {
      append_prefill_items(s, 2 * tile_tokens,
                           n_prefill_ctas * kWarpsAll + ((int)blockIdx.x - n_prefill_ctas) * kWarpsAux + (warp - kSoftmaxWarps),
                           append_warps, lane);
      __threadfence();         // this thread's page writes are visible before the CTA counts itself
      asm volatile("bar.sync 2, 128;\n" ::: "memory");
      if (tid == kSoftmaxWarps * 32) atomicAdd(s.pf_queue + 2, 1);
      cta_sync();
    }
    prefill_setup();
  };

  pdl_wait();                  // the previous step's kernels are done with the pool and the counters
  if (!decode_first) {
    append_prefill_items(s, 2 * tile_tokens, (int)blockIdx.x * kWarpsAll + warp, append_warps, lane);
    __threadfence();
    cta_sync();
    if (tid == 0) atomicAdd(s.pf_queue + 2, 1);
  }

  if (warp < kSoftmaxWarps) {
    // ------------------ softmax + epilogue: thread = half of a query row of tile x (64 of the 128
    // keys of every block, 64 of the 128 head_dim columns of O)
    if (decode_first) {
      if (warp < 8) {
        reg_inc<kRegsDecode>();       // waits until the parked warpgroups have given their registers up
        dec::decode_units<128, 1, 3>(s, &kv_map, smem, base, (int)blockIdx.x - n_prefill_ctas,
                                     (int)gridDim.x - n_prefill_ctas);
        if (tid == 0) {          // this CTA's split partials are written: count it as done
          __threadfence();
          atomicAdd(s.pf_queue + 1, 1);
        }
        fence_proxy_async();     // the prefill phase reuses this shared memory through other proxies
        reg_dec<kRegsSoftmax>();
        cta_sync();
      } else {
        reg_dec<kRegsParked>();
        cta_sync();
        reg_inc<kRegsSoftmax>();
      }
    } else {
      reg_inc<kRegsSoftmax>();
    }
    prefill_setup();
    const uint32_t tmem = misc[0];
    const int x = (warp >> 2) & 1;          // tile
    const int hf = warp >> 3;               // which half of the keys / of the head_dim columns
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + x * 128 + hf * 64 + lane_addr;         // my 64 score columns; P goes to the first 32
    const uint32_t tO = tmem + 256 + x * 128 + hf * 64 + lane_addr;   // my 64 columns of O
    // The two warps that share a quarter of a tile's rows meet on an mbarrier (a bounded wait, like
    // every other one here) around each exchange through shared memory.
    const int pair_bar = BAR_PAIR + x * 4 + (warp & 3);
    int n_pair = 0;
    auto pair_arrive = [&]() { mbar_arrive(bar(pair_bar)); };
    auto pair_wait = [&]() {
      wait(pair_bar, n_pair & 1);
      ++n_pair;
    };
    auto pair_sync = [&]() {
      pair_arrive();
      pair_wait();
    };
    float* xchg = reinterpret_cast<float*>(smem + kOffXchg) + x * 256;   // [half][row] of my tile
    float* xchg_mine = xchg + hf * 128 + row;
    const float* xchg_other = xchg + (hf ^ 1) * 128 + row;
    const float scale = s.scale_log2;
    int sx = 0;                 // blocks of this tile in earlier work units: barrier phases follow it
    for (int k = 0;; ++k) {
      PfUnit u;
      if (!get_work(k, u)) break;
      const int nbx = x ? u.nb_b : u.nb_a;
      const int cnt = x ? u.cnt_b : u.cnt_a;
      const int tok = u.q_begin + x * tile_tokens + row / G;   // token inside the request row
      const bool real = row / G < cnt && row < tile_tokens * G;
      const int lim = real ? u.ctx + tok + 1 : (x ? u.k_end_b : u.k_end_a);   // keys at positions >= lim are masked
      const int tok0 = u.tok0;
      float m_ref = -CUDART_INF_F, l = 0.f;
      for (int j = 0; j < nbx; ++j) {
        wait(BAR_S_FULL + x, (sx + j) & 1);
        tc_fence_after();
        // my half of the score row comes into registers: one trip to TMEM per block
        float v[64];
        const int nvalid = lim - j * kBlockKeys - hf * 64;     // keys of my half the row may see
        auto load_scores = [&]() {
          tmem_ld32(&v[0], tS);
          tmem_ld32(&v[32], tS + 32);
          tmem_ld_wait();
          if (__any_sync(0xffffffffu, nvalid < 64)) {          // only the blocks on the diagonal
#pragma unroll
            for (int i = 0; i < 64; ++i)
              if (i >= nvalid) v[i] = -CUDART_INF_F;           // 2^(-inf) = 0 exactly
          }
        };
        load_scores();
        // p = 2^(s*scale - m_ref) as bf16, to go over the first 32 columns of my half of S. Any
        // common reference is exact; p <= 2^threshold keeps the bf16 P and the fp32 sums
        // comfortable, so the reference only moves (and O is only rescaled) when the block maximum
        // exceeds it by more than the threshold. The two threads of a row post the maxima of their
        // halves (the scale is positive, so it commutes with max) and read the same two numbers,
        // so they take the same decision. After the first block of a unit the exponentials are
        // taken at once against the reference the row already has, and the maximum rides along
        // with them: that is nearly always the final answer. P stays in registers until the
        // decision is known, so the scores are still in TMEM for a warp with a row that does
        // move: it fetches them again and takes the exponentials once more. A row of the last,
        // diagonal block may be masked completely; it keeps its reference (block 0 always holds
        // key 0, which every row sees).
        uint32_t pk[32];
        float ls, x_max;
        if (j == 0) {
          *xchg_mine = max64(v) * scale;                       // first block of a unit: the maximum itself
          pair_sync();
          m_ref = fmaxf(*xchg_mine, *xchg_other);
          ls = exp_pack(v, scale, -m_ref, pk, x_max);
        } else {
          ls = exp_pack(v, scale, -m_ref, pk, x_max);
          *xchg_mine = x_max + m_ref;                          // largest s*scale of my half
          pair_sync();
          const float m_blk = fmaxf(*xchg_mine, *xchg_other);
          const bool move = m_blk > m_ref + kRescaleThreshold;
          if (__any_sync(0xffffffffu, move)) {
            float alpha = 1.f;
            if (move) {
              alpha = ex2(m_ref - m_blk);
              m_ref = m_blk;
              l *= alpha;
            }
            wait(BAR_O_FULL + x, (sx + j - 1) & 1);           // P V of block j-1 has landed in O
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              float ov[16];
              tmem_ld16(ov, tO + c * 16);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) ov[i] *= alpha;
              tmem_st16(tO + c * 16, *reinterpret_cast<const uint32_t(*)[16]>(ov));
            }
            load_scores();
            ls = exp_pack(v, scale, -m_ref, pk, x_max);
          }
        }
        tmem_st16(tS, *reinterpret_cast<const uint32_t(*)[16]>(&pk[0]));
        tmem_st16(tS + 16, *reinterpret_cast<const uint32_t(*)[16]>(&pk[16]));
        l += ls;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(bar(BAR_P_FULL + x));
      }
      if (nbx > 0) {
        // epilogue: O / l -> bf16 -> global; l is the sum over both halves of the keys. (The last
        // P V has been issued, so the partner has arrived for the last block and is done with
        // that block's exchange slots.)
        wait(BAR_O_FULL + x, (sx + nbx - 1) & 1);
        tc_fence_after();
        *xchg_mine = l;
        pair_sync();
        const float inv = 1.f / (l + *xchg_other);
        pair_sync();                      // both have read: the slots may be written again
        uint16_t* orow = s.out + ((size_t)(tok0 + tok) * s.Hq + u.kv_head * G + row % G) * kD + hf * 64;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          float ov[32];
          tmem_ld32(ov, tO + c * 32);
          tmem_ld_wait();
          if (c == 1) {
            tc_fence_before();
            mbar_arrive(bar(BAR_O_EMPTY + x));   // O is in registers: the next unit may overwrite it
          }
          if (real) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 wv;
              wv.x = pack_bf16(ov[8 * i] * inv, ov[8 * i + 1] * inv);
              wv.y = pack_bf16(ov[8 * i + 2] * inv, ov[8 * i + 3] * inv);
              wv.z = pack_bf16(ov[8 * i + 4] * inv, ov[8 * i + 5] * inv);
              wv.w = pack_bf16(ov[8 * i + 6] * inv, ov[8 * i + 7] * inv);
              *reinterpret_cast<uint4*>(orow + c * 32 + i * 8) = wv;
            }
          }
        }
      }
      sx += nbx;
    }
    // -------------------------------------------------------------- merge of the decode splits
    // By now the decode CTAs are normally long done; once all of them have counted themselves,
    // the first eight warps of every CTA merge the split rows between them.
    const int n_decode_ctas = (int)gridDim.x - n_prefill_ctas;
    if (warp < 8 && s.n_combines > 0 && n_decode_ctas > 0) {
      if (tid == 0) {
        const volatile int32_t* done = s.pf_queue + 1;
        const long long t0 = clock64();
        while (*done < n_decode_ctas) {
          if (clock64() - t0 > (misc[1] ? 2000 : s.wait_cycles)) {
            give_up();
            break;
          }
        }
        __threadfence();
      }
      dec::block_sync();
      // one warp per (split row, query head), dealt round-robin over all warps of the launch;
      // a lane merges four head_dim elements
      const int n_pairs = s.n_combines * s.Hq;
      for (int pi = (int)blockIdx.x * 8 + warp; pi < n_pairs; pi += (int)gridDim.x * 8) {
        const CombineItem c = s.combines[pi / s.Hq];
        const int h = pi % s.Hq;
        const float* ml = s.part_ml + ((size_t)c.first_partial * s.Hq + h) * 2;
        const float* pa = s.part_acc + ((size_t)c.first_partial * s.Hq + h) * kD + lane * 4;
        const size_t ml_stride = (size_t)s.Hq * 2, pa_stride = (size_t)s.Hq * kD;
        float m = -CUDART_INF_F, l = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int b0 = 0; b0 < c.n_splits; b0 += 8) {
          float mi[8], li[8];
          float4 ai[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const bool on = b0 + j < c.n_splits;
            mi[j] = on ? __ldcg(ml + (b0 + j) * ml_stride) : -CUDART_INF_F;
            li[j] = on ? __ldcg(ml + (b0 + j) * ml_stride + 1) : 0.f;
            ai[j] = on ? __ldcg(reinterpret_cast<const float4*>(pa + (b0 + j) * pa_stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
          float mn = m;
#pragma unroll
          for (int j = 0; j < 8; ++j) mn = fmaxf(mn, mi[j]);
          const float keep = exp2f(m - mn);          // 0 on the first group (m = -inf)
          l *= keep;
          acc.x *= keep; acc.y *= keep; acc.z *= keep; acc.w *= keep;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float wgt = exp2f(mi[j] - mn);     // absent split: exp2(-inf) = 0
            l += wgt * li[j];
            acc.x += wgt * ai[j].x; acc.y += wgt * ai[j].y; acc.z += wgt * ai[j].z; acc.w += wgt * ai[j].w;
          }
          m = mn;
        }
        const float inv = 1.f / l;
        uint2 o;
        o.x = pack_bf16(acc.x * inv, acc.y * inv);
        o.y = pack_bf16(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(s.out + ((size_t)c.token * s.Hq + h) * kD + lane * 4) = o;
      }
    }
  } else {
    // warps 16-19 are one warpgroup: they change their register count with one instruction
    aux_setup();
    if (warp < kWarpLoader0 + 2) {
      // ------------------------------------------------------------------ K/V loaders
      // One warp per operand. A 128-key tile is sixteen tensor copies of 2 KB (one page of one KV
      // head, 64 head_dim columns each; the page id is a coordinate of the copy, so scattered pages
      // cost nothing extra), issued by sixteen lanes at once and landing in the 128-byte-swizzled
      // operand layout the MMA reads. K tiles complete their "full" barrier by transaction bytes.
      // V tiles complete a "landed" barrier first: the warp then clears, in shared memory, the V
      // rows of a ragged last page (slots past the last key may hold anything, and 0 * NaN would
      // poison O; the same rows of K only produce scores that are masked) and announces the tile.
      // The loaders run up to a ring of stages ahead of the tensor pipe.
      const int kv = warp - kWarpLoader0;                      // 0: K, 1: V
      const int stages = kv ? kVStages : kKStages;
      const int lag = stages - 1;                              // V tiles in flight besides the announced one
      const int full = kv ? BAR_V_FULL : BAR_K_FULL, empty = kv ? BAR_V_EMPTY : BAR_K_EMPTY;
      const uint32_t tile0 = base + (kv ? kOffV : kOffK);
      if (lane == 0) tma_prefetch_desc(&kv_tile_map);
      // The K loader's first thread takes work units off the global queue, one at a time and only
      // when the K loader is ready for it (it runs a few key blocks ahead of the tensor pipe, which
      // hides the round trip), and publishes each to the other roles through a small ring.
      int fetched = 0;
      auto fetch_one = [&]() {
        const int w = atomicAdd(s.pf_queue, 1);
        UnitRec r = {};
        r.w = -1;
        if (w < n_units) {
          const WorkItem it = s.items[w / s.Hkv];
          r.w = w;
          r.table_slot = s.row_slot[it.row];
          r.kv_head = w % s.Hkv;
          r.q_begin = it.q_begin;
          r.q_count = it.q_count;
          r.ctx = it.k_end - it.q_begin - it.q_count;
          r.tok0 = s.row_tok0[it.row];
          if ((unsigned)r.table_slot >= (unsigned)s.max_requests) {
            atomicOr(s.status, TS_DEV_BAD_INDEX);
            r.w = -1;
          }
        }
        const int e = (fetched & (kSchedRing - 1)) * 2;
        ring[e].x = r.w; ring[e].y = r.table_slot; ring[e].z = r.kv_head; ring[e].w = r.q_begin;
        ring[e + 1].x = r.q_count; ring[e + 1].y = r.ctx; ring[e + 1].z = r.tok0; ring[e + 1].w = 0;
        __threadfence_block();
        misc[2] = (uint32_t)++fetched;
      };
      int g0 = 0;                                              // key blocks of earlier work units
      for (int k = 0;; ++k) {
        if (kv == 0 && lane == 0) fetch_one();
        __syncwarp();
        PfUnit u;
        if (!get_work(k, u)) break;
        const int32_t* table_row = s.table + (size_t)u.table_slot * s.max_pages_per_req;
        // lane i < 16 copies page i / 2 of the tile, head_dim columns [64 (i % 2), +64)
        auto fetch_page = [&](int j) {
          const int key = j * kBlockKeys + (lane >> 1) * kPageSize;
          int page = s.n_pages;                                // out of range on purpose: the copy delivers zeros
          if (lane < 16 && key < u.k_end) {
            page = table_row[key >> 4];
            if ((unsigned)page >= (unsigned)s.n_pages) {
              atomicOr(s.status, TS_DEV_BAD_PAGE);
              page = s.n_pages;
            }
          }
          return page;
        };
        auto announce = [&](int tile) {                        // V only; tile = block index within the unit
          const int gt = g0 + tile, st = gt % stages;
          wait(BAR_V_LANDED + st, (gt / stages) & 1);
          const int first_bad = u.k_end - tile * kBlockKeys;   // rows from here on hold no key of the unit
          if (first_bad < kBlockKeys && (first_bad & 15)) {
            const int n_rows = 16 - (first_bad & 15);          // up to the end of that page; later pages were not copied
            unsigned char* vt = smem + kOffV + st * kTileBytes;
            for (int i = lane; i < n_rows * 16; i += 32) {
              const int r = first_bad + (i >> 4), c = i & 15;  // a row is 8 chunks of 16 bytes in each 64-column half
              *reinterpret_cast<uint4*>(vt + (c >> 3) * kHalfBytes + r * 128 + ((c & 7) << 4)) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async();
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(full + st));
        };
        int page = fetch_page(0);
        for (int j = 0; j < u.nb; ++j) {
          const int g = g0 + j;
          const int st = g % stages;
          if (kv && j >= lag) announce(j - lag);
          const int page_next = j + 1 < u.nb ? fetch_page(j + 1) : 0;   // the table load flies while this tile is issued
          if (g >= stages) wait(empty + st, ((g / stages) & 1) ^ 1);
          const uint32_t landed = bar(kv ? BAR_V_LANDED + st : full + st);
          if (misc[1] == 0) {                                  // after a failure no new copies are started
            if (lane == 0) mbar_expect_tx(landed, kTileBytes);
            __syncwarp();
            if (lane < 16)
              tma_load_5d(tile0 + st * kTileBytes + (lane & 1) * kHalfBytes + (lane >> 1) * 2048, &kv_tile_map, landed,
                          (lane & 1) * 64, 0, u.kv_head, kv, page);
          }
          page = page_next;
        }
        // the last `lag` V tiles (fewer when the unit is short) have not been announced yet
        if (kv)
          for (int tile = max(0, u.nb - lag); tile < u.nb; ++tile) announce(tile);
        g0 += u.nb;
      }
    } else {
      // ------------------------------------------------------------------- MMA issuer
      if (warp == kWarpMma) {
        const uint32_t tmem = misc[0];
        const uint32_t issue = elect_one();
        // the warp keeps its own failure flag in a register: nothing on its path reads shared memory
        bool dead = false;
        // The issuer polls its barriers instead of parking on them: it is the only warp that does,
        // and every cycle between a tile's P and its next scores is on the critical path.
        auto iwait = [&](int i, uint32_t parity) {
          if (!mbar_poll(bar(i), parity, dead ? 2000 : s.wait_cycles)) {
            dead = true;
            give_up();
          }
        };
        constexpr uint32_t idesc_qk = instr_desc(false), idesc_pv = instr_desc(true);
        // descriptors differ only in their start-address field (16-byte units in the low bits)
        const uint64_t q_desc0 = smem_desc(base + kOffQ, 0, 1024);
        const uint64_t k_desc0 = smem_desc(base + kOffK, 0, 1024);
        const uint64_t v_desc0 = smem_desc(base + kOffV, kHalfBytes, 1024);
        auto issue_qk = [&](int x, int g) {          // S_x = Q_x K(g)^T
          const uint64_t q_desc = q_desc0 + (uint64_t)((x * kTileBytes) >> 4);
          const uint64_t k_desc = k_desc0 + (uint64_t)(((g % kKStages) * kTileBytes) >> 4);
#pragma unroll
          for (int ks = 0; ks < kD / 16; ++ks) {
            const uint64_t off = (uint64_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
            mma_ss(tmem + x * 128, q_desc + off, k_desc + off, idesc_qk, ks > 0, issue);
          }
          tc_commit(bar(BAR_S_FULL + x), issue);
        };
        auto issue_pv = [&](int x, int g, bool first) {   // O_x (+)= P_x V(g)
          const uint64_t v_desc = v_desc0 + (uint64_t)(((g % kVStages) * kTileBytes) >> 4);
#pragma unroll
          for (int kk = 0; kk < kBlockKeys / 16; ++kk)   // P of keys 0-63 sits in columns 0-31 of S, of keys 64-127 in 64-95
            mma_ts(tmem + 256 + x * 128, tmem + x * 128 + (kk >> 2) * 64 + (kk & 3) * 8,
                   v_desc + (uint64_t)((kk * 2048) >> 4), idesc_pv, (!first || kk > 0) ? 1u : 0u, issue);
          tc_commit(bar(BAR_O_FULL + x), issue);
        };
        int g0 = 0;                 // key blocks of earlier work units (K/V ring position)
        int sxb[2] = {0, 0};        // blocks per tile in earlier work units (S/P/O phases)
        int used[2] = {0, 0};       // earlier work units in which the tile had rows (O_EMPTY phases)
        for (int k = 0;; ++k) {
          PfUnit u;
          if (!get_work(k, u)) break;
          // Order: both Q K^T of block 0; then per block, for tile A then tile B:
          // P V of block j followed at once by Q K^T of block j+1 of the same tile, so that the
          // tile's warpgroup gets its next scores while the pipe turns to the other tile.
          iwait(BAR_Q, k & 1);
          iwait(BAR_K_FULL + g0 % kKStages, (g0 / kKStages) & 1);
          tc_fence_after();
          if (!dead) {
            if (u.nb_a > 0) issue_qk(0, g0);
            if (u.nb_b > 0) issue_qk(1, g0);
            tc_commit(bar(BAR_K_EMPTY + g0 % kKStages), issue);
            if (u.nb == 1) tc_commit(bar(BAR_Q_EMPTY), issue);
          }
          for (int j = 0; j < u.nb; ++j) {
            const int g = g0 + j;
            const bool next = j + 1 < u.nb;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              const int nbx = x ? u.nb_b : u.nb_a;
              if (j < nbx) {
                iwait(BAR_P_FULL + x, (sxb[x] + j) & 1);
                if (x == 0 || j >= u.nb_a) iwait(BAR_V_FULL + g % kVStages, (g / kVStages) & 1);
                if (j == 0 && used[x] > 0) iwait(BAR_O_EMPTY + x, (used[x] - 1) & 1);   // the previous unit's O has been read
                tc_fence_after();
                if (!dead) issue_pv(x, g, j == 0);
              }
              if (x == 1 && !dead) tc_commit(bar(BAR_V_EMPTY + g % kVStages), issue);   // both tiles are done with V(g)
              if (next) {
                if (x == 0 || j + 1 >= u.nb_a) iwait(BAR_K_FULL + (g + 1) % kKStages, ((g + 1) / kKStages) & 1);
                tc_fence_after();
                if (j + 1 < nbx && !dead) issue_qk(x, g + 1);
                if (x == 1 && !dead) {
                  tc_commit(bar(BAR_K_EMPTY + (g + 1) % kKStages), issue);
                  if (j + 2 == u.nb) tc_commit(bar(BAR_Q_EMPTY), issue);   // that was the unit's last Q K^T
                }
              }
            }
          }
          g0 += u.nb;
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const int nbx = x ? u.nb_b : u.nb_a;
            sxb[x] += nbx;
            used[x] += nbx > 0;
          }
        }
      }
      if (warp == kWarpSched && lane == 0) {
        // ------------------------------------------------------------------ Q loader
        // Brings in each work unit's Q tiles by TMA once the previous unit's last Q K^T is done.
        tma_prefetch_desc(&q_map);
        for (int k = 0;; ++k) {
          PfUnit u;
          if (!get_work(k, u)) break;
          const int ta = u.tok0 + u.q_begin;
          if (k > 0) wait(BAR_Q_EMPTY, (k - 1) & 1);
          // a box delivers 64 columns of tile_tokens * G packed rows (all 128 only when G divides 128)
          mbar_expect_tx(bar(BAR_Q), (u.cnt_b > 0 ? 2 : 1) * 2 * (tile_tokens * G * 128));
          tma_load_4d(base + kOffQ, &q_map, bar(BAR_Q), 0, 0, u.kv_head, ta);
          tma_load_4d(base + kOffQ + kHalfBytes, &q_map, bar(BAR_Q), 64, 0, u.kv_head, ta);
          if (u.cnt_b > 0) {
            tma_load_4d(base + kOffQ + kTileBytes, &q_map, bar(BAR_Q), 0, 0, u.kv_head, ta + tile_tokens);
            tma_load_4d(base + kOffQ + kTileBytes + kHalfBytes, &q_map, bar(BAR_Q), 64, 0, u.kv_head, ta + tile_tokens);
          }
        }
      }
      __syncwarp();
    }
  }
  tc_fence_before();
  cta_sync();
  if (warp == kWarpMma) tmem_dealloc(misc[0], 512);
  if (tid == 0) {
    // the last CTA to leave puts the launch's counters back to zero for the next launch
    __threadfence();
    if (atomicAdd(s.pf_queue + 3, 1) == (int)gridDim.x - 1) {
      s.pf_queue[0] = 0;
      s.pf_queue[1] = 0;
      s.pf_queue[2] = 0;
      s.pf_queue[3] = 0;
    }
  }
}

}  // namespace

cudaError_t launch_mixed(const StepDevice& s, const CUtensorMap& q_map, const CUtensorMap& kv_map,
                         const CUtensorMap& kv_tile_map, int n_ctas, int n_prefill_ctas, cudaStream_t stream) {
  if (s.n_prefill_items <= 0 || n_ctas <= 0) return cudaSuccess;
  const int G = s.Hq / s.Hkv;
  size_t smem = kSmemBytes;
  if (n_prefill_ctas < n_ctas) {
    const size_t dec_smem = 1024 + dec::decode_smem_bytes<128, 3>(G);
    if (dec_smem > smem) smem = dec_smem;
  }
  cudaError_t e = cudaFuncSetAttribute(mixed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(mixed_kernel, dim3(n_ctas), dim3(kPfThreads), smem, stream, s, q_map, kv_map, kv_tile_map, n_prefill_ctas);
}

}  // namespace ts
