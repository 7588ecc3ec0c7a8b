// Stand-alone split-KV flash-decode kernel for the 1-token rows (sm_100a): one persistent CTA
// per SM running dec::decode_units (ts_decode_body.h) over all decode units of the step.
// On a decode-only step (StepDevice::append_in_decode) the units also append the rows' new K/V.
#include "ts_decode_body.h"

namespace ts {
namespace {

using dec::kDecThreads;

template <int D, int NH, int STAGES>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_kernel(const StepDevice s, const __grid_constant__ CUtensorMap kv_map) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  pdl_launch_dependents();
  if (threadIdx.x == 0) tma_prefetch_desc(&kv_map);
  pdl_wait();                  // from here on the pool, tables and Q are read
  dec::decode_units<D, NH, STAGES>(s, &kv_map, smem, base, blockIdx.x, gridDim.x);
}

template <int D, int NH, int STAGES>
cudaError_t launch_decode_t(const StepDevice& s, const CUtensorMap& map, int n_sms, cudaStream_t stream) {
  const int G = s.Hq / s.Hkv;
  const size_t smem = 1024 + dec::decode_smem_bytes<D, STAGES>(G);
  cudaError_t e = cudaFuncSetAttribute(decode_kernel<D, NH, STAGES>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long units = (long long)(s.n_items - s.n_prefill_items) * s.Hkv;
  const int grid = (int)(units < n_sms ? units : n_sms);
  return launch_pdl(decode_kernel<D, NH, STAGES>, dim3(grid), dim3(kDecThreads), smem, stream, s, map);
}

}  // namespace

cudaError_t launch_decode(const StepDevice& s, const CUtensorMap& kv_map, int n_sms, cudaStream_t stream) {
  if (s.n_items - s.n_prefill_items <= 0) return cudaSuccess;
  const int G = s.Hq / s.Hkv;
  if (s.D == 128) {
    return G <= 8 ? launch_decode_t<128, 1, 3>(s, kv_map, n_sms, stream)
                  : launch_decode_t<128, 2, 2>(s, kv_map, n_sms, stream);
  }
  return G <= 8 ? launch_decode_t<64, 1, 4>(s, kv_map, n_sms, stream)
                : launch_decode_t<64, 2, 4>(s, kv_map, n_sms, stream);
}

}  // namespace ts
