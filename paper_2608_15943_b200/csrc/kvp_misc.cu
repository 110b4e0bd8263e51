// Small memory-bound helpers: fp32 -> bf16 rounding (the donor-group gradient sums before they enter the
// projection GEMMs; fp32 inputs of the KVP_F32 interface) and bf16 -> fp32 widening (its outputs).
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

__global__ void cast_bf16_f32_kernel(const uint2* __restrict__ src, float4* __restrict__ dst, size_t n4) {
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const uint2 v = src[i];
    dst[i] = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                         __uint_as_float(v.y & 0xffff0000u));
  }
}

}  // namespace

int cast_bf16_to_f32(const void* src, float* dst, size_t n, cudaStream_t stream) {
  if ((n & 3) != 0) return KVP_ERR_UNSUPPORTED;
  const size_t n4 = n / 4;
  const int threads = 256;
  const int blocks = int(min(size_t(sm_count()) * 8, (n4 + threads - 1) / threads));
  cast_bf16_f32_kernel<<<blocks, threads, 0, stream>>>(reinterpret_cast<const uint2*>(src), reinterpret_cast<float4*>(dst), n4);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

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
