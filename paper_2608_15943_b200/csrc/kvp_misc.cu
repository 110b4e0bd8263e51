// Small memory-bound helpers: fp32 -> bf16 rounding of the donor-group gradient sums before they
// enter the projection GEMMs.
#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

__global__ void cast_f32_bf16_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, size_t n4) {
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const float4 v = src[i];
    dst[i] = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
  }
}

}  // namespace

// n must be a multiple of 4 (it is a multiple of the head dimension).
int cast_f32_to_bf16(const float* src, void* dst, size_t n, cudaStream_t stream) {
  if ((n & 3) != 0) return KVP_ERR_UNSUPPORTED;
  const size_t n4 = n / 4;
  const int threads = 256;
  const int blocks = int(min(size_t(sm_count()) * 8, (n4 + threads - 1) / threads));
  cast_f32_bf16_kernel<<<blocks, threads, 0, stream>>>(reinterpret_cast<const float4*>(src),
                                                       reinterpret_cast<uint2*>(dst), n4);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

}  // namespace kvp
