// Element-wise operators of a decoder stage (RMSNorm, rotary position embedding, SwiGLU, residual add), so
// that a whole pipeline stage's forward pass can be timed with this library's kernels (the paper's stage
// tables list a forward time per stage).  All four are bound by HBM bandwidth: 16-byte accesses, fp32
// arithmetic, bf16 storage, one pass over the data, grids sized to the SM count.
#include <math.h>

#include <algorithm>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  return make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
}

// y = x / sqrt(mean(x^2) + eps) * w.  One CTA of 256 threads per row, the row kept in registers between the
// reduction and the scaling (D <= 256 * 8 * kMaxChunks elements).
constexpr int kNormThreads = 256;
constexpr int kMaxChunks = 4;  // D <= 8192
__global__ void __launch_bounds__(kNormThreads) rmsnorm_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w,
                                                               uint4* __restrict__ y, int T, int D8, float inv_d, float eps) {
  __shared__ float part[kNormThreads / 32];
  auto load_row = [&](int row, uint4 (&v)[kMaxChunks]) {
    const uint4* xr = x + size_t(row) * D8;
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c) {
      const int i = c * kNormThreads + threadIdx.x;
      if (i < D8) v[c] = xr[i];
    }
  };
  uint4 v[kMaxChunks], vn[kMaxChunks];
  if (int(blockIdx.x) < T) load_row(blockIdx.x, v);
  for (int row = blockIdx.x; row < T; row += gridDim.x) {
    // the next row of this CTA is requested before the current one is reduced: its latency hides under the two
    // block barriers and the stores of this row
    const int next = row + gridDim.x;
    if (next < T) load_row(next, vn);
    float ss = 0.f;
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c) {
      const int i = c * kNormThreads + threadIdx.x;
      if (i < D8) {
        float f[8];
        unpack8(v[c], f);
#pragma unroll
        for (int k = 0; k < 8; ++k) ss = fmaf(f[k], f[k], ss);
      }
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int k = 0; k < kNormThreads / 32; ++k) tot += part[k];
    __syncthreads();  // part[] is reused by the next row
    const float r = rsqrtf(tot * inv_d + eps);
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c) {
      const int i = c * kNormThreads + threadIdx.x;
      if (i < D8) {
        float f[8], g[8];
        unpack8(v[c], f);
        unpack8(w[i], g);
#pragma unroll
        for (int k = 0; k < 8; ++k) f[k] = f[k] * r * g[k];
        y[size_t(row) * D8 + i] = pack8(f);
      }
    }
#pragma unroll
    for (int c = 0; c < kMaxChunks; ++c) v[c] = vn[c];
  }
}

// In-place rotary embedding of x [B, S, H, dh]: pair i of every head turns by (pos0 + s) * theta^(-2i/dh).
// One thread per (token, 8 consecutive elements of the head dimension): it forms the four rotations once and
// applies them to that slice of EVERY head of the token, so the sines and cosines cost 1/H of a per-element
// evaluation and the kernel is left with its loads and stores.  The frequencies arrive as float pairs hi + lo
// rounded from the host's double values; the angle pos * f is formed as an exact product p = pos * hi plus its
// rounding error and the lo term, sine and cosine of the float p are taken after an exact range reduction, and the
// small remainder is applied as a second-order correction.
constexpr int kMaxRopePairs = 128;
struct RopeFreq {
  float2 f[kMaxRopePairs];
};
__global__ void rope_kernel(uint4* __restrict__ x, uint32_t n_work, uint32_t S, uint32_t H, uint32_t dh8, int pos0,
                            const __grid_constant__ RopeFreq fr) {
  // lanes of a warp need different table entries: shared memory serves them in one pass, the constant bank
  // that holds kernel parameters would replay once per distinct address
  __shared__ float2 freq[kMaxRopePairs];
  for (int k = threadIdx.x; k < kMaxRopePairs; k += blockDim.x) freq[k] = fr.f[k];
  __syncthreads();
  const uint32_t stride = gridDim.x * blockDim.x;
  const uint32_t per_tok = H * dh8;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_work; i += stride) {  // 32-bit index arithmetic only
    const uint32_t c = i % dh8;                       // which group of 4 pairs inside the head
    const uint32_t tok = i / dh8;                     // b * S + s
    const float pos = float(pos0 + int(tok % S));     // exact
    float sn2[4], cs2[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 fq = freq[c * 4 + k];
      const float p = pos * fq.x;
      const float d = fmaf(pos, fq.y, fmaf(pos, fq.x, -p));   // angle - p
      // p (< 2^18) reduced to [-pi, pi] with 2*pi split into three floats whose first has 8 significant
      // bits, so that k * 6.28125 is exact and the subtraction loses nothing (error about 1e-7)
      const float kk = rintf(p * 0.15915494309189535f);
      float rr = fmaf(-kk, 6.28125f, p);
      rr = fmaf(-kk, 0.00193023681640625f, rr);
      rr = fmaf(-kk, 5.070363386039389e-06f, rr);
      const float sn = __sinf(rr), cs = __cosf(rr);
      const float h = 0.5f * d * d;
      sn2[k] = sn + d * cs - h * sn;
      cs2[k] = cs - d * sn - h * cs;
    }
    uint4* const base = x + size_t(tok) * per_tok + c;
    constexpr uint32_t UNROLL = 4;   // loads in flight per thread
    for (uint32_t h0 = 0; h0 < H; h0 += UNROLL) {
      uint4 v[UNROLL];
#pragma unroll
      for (uint32_t u = 0; u < UNROLL; ++u)
        if (h0 + u < H) v[u] = base[size_t(h0 + u) * dh8];
#pragma unroll
      for (uint32_t u = 0; u < UNROLL; ++u) {
        if (h0 + u < H) {
          float f[8];
          unpack8(v[u], f);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float a = f[2 * k], b = f[2 * k + 1];
            f[2 * k] = a * cs2[k] - b * sn2[k];
            f[2 * k + 1] = a * sn2[k] + b * cs2[k];
          }
          base[size_t(h0 + u) * dh8] = pack8(f);
        }
      }
    }
  }
}

// out = silu(gate) * up
__global__ void swiglu_kernel(const uint4* __restrict__ gate, const uint4* __restrict__ up, uint4* __restrict__ out, size_t n8) {
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n8; i += stride) {
    float g[8], u[8];
    unpack8(gate[i], g);
    unpack8(up[i], u);
#pragma unroll
    for (int k = 0; k < 8; ++k) g[k] = g[k] * __frcp_rn(1.f + __expf(-g[k])) * u[k];
    out[i] = pack8(g);
  }
}

__global__ void add_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b, uint4* __restrict__ out, size_t n8) {
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n8; i += stride) {
    float f[8], g[8];
    unpack8(a[i], f);
    unpack8(b[i], g);
#pragma unroll
    for (int k = 0; k < 8; ++k) f[k] += g[k];
    out[i] = pack8(f);
  }
}

bool is_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
int streaming_blocks(size_t n8, int threads) { return int(min(size_t(sm_count()) * 8, (n8 + threads - 1) / threads)); }

}  // namespace
}  // namespace kvp

using namespace kvp;

extern "C" int kvp_rmsnorm(int32_t T, int32_t D, const void* x, const void* w, float eps, void* y, kvp_stream_t stream) {
  if (T < 0 || D < 1 || x == nullptr || w == nullptr || y == nullptr || !(eps >= 0.f)) return KVP_ERR_INVALID_ARG;
  if (D % 8 != 0 || D > 8 * kNormThreads * kMaxChunks || !is_aligned16(x) || !is_aligned16(w) || !is_aligned16(y)) return KVP_ERR_UNSUPPORTED;
  if (T == 0) return KVP_OK;
  const int blocks = min(T, sm_count() * 8);
  rmsnorm_kernel<<<blocks, kNormThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4*>(x), reinterpret_cast<const uint4*>(w), reinterpret_cast<uint4*>(y), T, D / 8, 1.f / float(D), eps);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

extern "C" int kvp_rope(int32_t B, int32_t S, int32_t H, int32_t dh, float theta, int32_t pos0, void* x, kvp_stream_t stream) {
  if (B < 0 || S < 0 || H < 1 || dh < 2 || x == nullptr || !(theta > 1.f) || pos0 < 0) return KVP_ERR_INVALID_ARG;
  if (dh % 8 != 0 || dh / 2 > kMaxRopePairs || !is_aligned16(x) || int64_t(pos0) + S > (int64_t(1) << 18)) return KVP_ERR_UNSUPPORTED;
  const size_t n8 = size_t(B) * S * H * (dh / 8);
  if (n8 == 0) return KVP_OK;
  RopeFreq fr;
  for (int i = 0; i < kMaxRopePairs; ++i) {
    const double f = i < dh / 2 ? pow(double(theta), -2.0 * i / dh) : 0.0;
    fr.f[i].x = float(f);
    fr.f[i].y = float(f - double(fr.f[i].x));
  }
  // 16-byte groups are indexed with 32 bits: larger tensors go in slices of whole sequences
  const size_t per_seq = size_t(S) * H * (dh / 8);
  if (per_seq >= (size_t(1) << 31)) return KVP_ERR_UNSUPPORTED;
  const int seqs_per_launch = int(std::max<size_t>(1, ((size_t(1) << 31) - 1) / per_seq));
  for (int b0 = 0; b0 < B; b0 += seqs_per_launch) {
    const uint32_t n_work = uint32_t(size_t(std::min(seqs_per_launch, B - b0)) * S * (dh / 8));   // (token, 8-element slice)
    rope_kernel<<<streaming_blocks(n_work, 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<uint4*>(x) + size_t(b0) * per_seq, n_work, uint32_t(S), uint32_t(H), uint32_t(dh / 8), pos0, fr);
    note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

extern "C" int kvp_swiglu(int64_t n, const void* gate, const void* up, void* out, kvp_stream_t stream) {
  if (n < 0 || gate == nullptr || up == nullptr || out == nullptr) return KVP_ERR_INVALID_ARG;
  if (n % 8 != 0 || !is_aligned16(gate) || !is_aligned16(up) || !is_aligned16(out)) return KVP_ERR_UNSUPPORTED;
  if (n == 0) return KVP_OK;
  swiglu_kernel<<<streaming_blocks(size_t(n / 8), 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4*>(gate), reinterpret_cast<const uint4*>(up), reinterpret_cast<uint4*>(out), size_t(n / 8));
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

extern "C" int kvp_add(int64_t n, const void* a, const void* b, void* out, kvp_stream_t stream) {
  if (n < 0 || a == nullptr || b == nullptr || out == nullptr) return KVP_ERR_INVALID_ARG;
  if (n % 8 != 0 || !is_aligned16(a) || !is_aligned16(b) || !is_aligned16(out)) return KVP_ERR_UNSUPPORTED;
  if (n == 0) return KVP_OK;
  add_kernel<<<streaming_blocks(size_t(n / 8), 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4*>(a), reinterpret_cast<const uint4*>(b), reinterpret_cast<uint4*>(out), size_t(n / 8));
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}
