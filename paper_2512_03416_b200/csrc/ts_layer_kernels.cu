// Small kernels of the decoder layer around the attention step (sm_100a): RMSNorm, the rotary
// table, and the packing of the gate and up projection weights into the row order the fused
// gate/up GEMM reads.
#include <cuda_bf16.h>

#include "../../include/tokenscale.h"
#include "ts_internal.h"
#include "ts_ptx.h"

namespace ts {
namespace {

constexpr int kNormThreads = 256;

// One CTA per row: every thread keeps its 16-byte chunks of the row in registers between the
// sum of squares and the scaling (up to four chunks: widths up to 8192; wider rows read twice).
__global__ void __launch_bounds__(kNormThreads) rmsnorm_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ gain,
                                                               uint16_t* __restrict__ out, int width, float eps) {
  __shared__ float partial[kNormThreads / 32];
  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, n_chunks = width / 8;
  const uint16_t* row = x + (size_t)blockIdx.x * width;
  uint4 keep[4];
  float ss = 0.f;
  for (int c = tid, i = 0; c < n_chunks; c += kNormThreads, ++i) {
    const uint4 w = *reinterpret_cast<const uint4*>(row + c * 8);
    if (i < 4) keep[i] = w;
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = __uint_as_float(u[e] << 16), b = __uint_as_float(u[e] & 0xFFFF0000u);
      ss += a * a + b * b;
    }
  }
#pragma unroll
  for (int sh = 16; sh > 0; sh >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, sh);
  if ((tid & 31) == 0) partial[tid >> 5] = ss;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int w = 0; w < kNormThreads / 32; ++w) total += partial[w];
  const float inv = rsqrtf(total / (float)width + eps);
  uint16_t* orow = out + (size_t)blockIdx.x * width;
  for (int c = tid, i = 0; c < n_chunks; c += kNormThreads, ++i) {
    const uint4 w = i < 4 ? keep[i] : *reinterpret_cast<const uint4*>(row + c * 8);
    const uint4 gw = *reinterpret_cast<const uint4*>(gain + c * 8);
    const uint32_t u[4] = {w.x, w.y, w.z, w.w}, gu[4] = {gw.x, gw.y, gw.z, gw.w};
    uint4 o;
    uint32_t* ou = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = __uint_as_float(u[e] << 16) * inv * __uint_as_float(gu[e] << 16);
      const float b = __uint_as_float(u[e] & 0xFFFF0000u) * inv * __uint_as_float(gu[e] & 0xFFFF0000u);
      ou[e] = pack_bf16(a, b);
    }
    *reinterpret_cast<uint4*>(orow + c * 8) = o;
  }
}

__global__ void rope_table_kernel(float2* table, int max_position, double log2_theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_position * 64) return;
  const int p = idx / 64, i = idx % 64;
  const double inv_freq = exp2(-2.0 * (double)i / 128.0 * log2_theta);
  double s, c;
  sincos((double)p * inv_freq, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

__global__ void pack_gate_up_kernel(const uint16_t* __restrict__ gate, const uint16_t* __restrict__ up, uint16_t* __restrict__ dst,
                                    int width) {
  const int r = blockIdx.x;                     // destination row
  const int b = r / 256, w = r % 256;
  const uint16_t* src = (w < 128 ? gate : up) + (size_t)(b * 128 + (w & 127)) * width;
  for (int c = threadIdx.x; c < width / 8; c += blockDim.x)
    *reinterpret_cast<uint4*>(dst + (size_t)r * width + c * 8) = *reinterpret_cast<const uint4*>(src + c * 8);
}

}  // namespace

cudaError_t launch_rmsnorm(const uint16_t* x, const uint16_t* gain, uint16_t* out, int rows, int width, float eps,
                           cudaStream_t stream) {
  if (rows <= 0) return cudaSuccess;
  return launch_pdl(rmsnorm_kernel, dim3(rows), dim3(kNormThreads), 0, stream, x, gain, out, width, eps);
}

cudaError_t launch_rope_table(float2* table, int max_position, float theta, cudaStream_t stream) {
  const int n = max_position * 64;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, stream>>>(table, max_position, log2((double)theta));
  return cudaGetLastError();
}

cudaError_t launch_pack_gate_up(const uint16_t* gate, const uint16_t* up, uint16_t* dst, int intermediate, int width,
                                cudaStream_t stream) {
  pack_gate_up_kernel<<<2 * intermediate, 128, 0, stream>>>(gate, up, dst, width);
  return cudaGetLastError();
}

}  // namespace ts
