// Host utilities of the library: status strings, TMA descriptor construction, device status.
#include <atomic>
#include <mutex>

#include "kvp_host.h"

namespace kvp {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}
}  // namespace

int make_tensor_map(CUtensorMap* out, const void* base, int elem_bytes, int rank, const uint64_t* dims,
                    const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return KVP_ERR_CUDA;
  cuuint64_t gdim[5];
  cuuint64_t gstride[4];
  cuuint32_t bdim[5];
  cuuint32_t estride[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bdim[i] = box[i];
    estride[i] = 1;
    if (i + 1 < rank) gstride[i] = strides_bytes[i];
  }
  const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  const CUresult r = fn(out, dt, cuuint32_t(rank), const_cast<void*>(base), gdim, gstride, bdim, estride,
                        CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? KVP_OK : KVP_ERR_CUDA;
}

namespace {
std::atomic<unsigned long long> g_launches{0};
struct TimingSlot {
  cudaEvent_t* starts = nullptr;
  cudaEvent_t* stops = nullptr;
  int capacity = 0;
  int used = 0;
};
TimingSlot g_timing[KVP_KERNEL_COUNT];
}  // namespace

void note_launch(int n) { g_launches.fetch_add(static_cast<unsigned long long>(n), std::memory_order_relaxed); }

void timing_before(int kernel, cudaStream_t stream) {
  TimingSlot& t = g_timing[kernel];
  if (t.used < t.capacity) cudaEventRecord(t.starts[t.used], stream);
}
void timing_after(int kernel, cudaStream_t stream) {
  TimingSlot& t = g_timing[kernel];
  if (t.used < t.capacity) {
    cudaEventRecord(t.stops[t.used], stream);
    ++t.used;
  }
}

int sm_count() {
  // per device: a process may drive more than one GPU
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

}  // namespace kvp

extern "C" const char* kvp_status_string(int status) {
  switch (status) {
    case KVP_OK: return "ok";
    case KVP_ERR_INVALID_ARG: return "invalid argument";
    case KVP_ERR_BAD_DONOR: return "bad donor map";
    case KVP_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
    case KVP_ERR_WORKSPACE: return "workspace missing or too small";
    case KVP_ERR_CUDA: return "CUDA error";
    case KVP_ERR_TIMEOUT: return "a kernel gave up on a bounded wait";
    case KVP_ERR_STATIC_SCRATCH: return "request needs more than the library's built-in scratch array";
    default: return "unknown status";
  }
}

extern "C" int kvp_device_status(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return KVP_ERR_CUDA;
  int bad = 0;
  int v;
  v = kvp::gemm_read_status();
  if (v < 0) return KVP_ERR_CUDA;
  bad |= v;
  v = kvp::attn_fwd_read_status();
  if (v < 0) return KVP_ERR_CUDA;
  bad |= v;
  v = kvp::attn_bwd_read_status();
  if (v < 0) return KVP_ERR_CUDA;
  bad |= v;
  v = kvp::decode_read_status();
  if (v < 0) return KVP_ERR_CUDA;
  bad |= v;
  return bad ? KVP_ERR_TIMEOUT : KVP_OK;
}

extern "C" unsigned long long kvp_launch_count(void) { return kvp::g_launches.load(std::memory_order_relaxed); }

extern "C" int kvp_set_timing_events(int kernel, void** starts, void** stops, int n) {
  if (kernel < 0 || kernel >= kvp::KVP_KERNEL_COUNT || n < 0 || (n > 0 && (starts == nullptr || stops == nullptr)))
    return KVP_ERR_INVALID_ARG;
  kvp::TimingSlot& t = kvp::g_timing[kernel];
  t.starts = reinterpret_cast<cudaEvent_t*>(starts);
  t.stops = reinterpret_cast<cudaEvent_t*>(stops);
  t.capacity = n;
  t.used = 0;
  return KVP_OK;
}

extern "C" int kvp_timing_events_used(int kernel) {
  if (kernel < 0 || kernel >= kvp::KVP_KERNEL_COUNT) return -1;
  return kvp::g_timing[kernel].used;
}

extern "C" void kvp_set_gemm_pair_mode(int mode) { kvp::gemm_set_pair_mode(mode < 0 ? 0 : mode > 2 ? 2 : mode); }

extern "C" int kvp_gemm(int M, int N, int K, const void* a, int64_t lda, int a_mn, const void* b, int64_t ldb,
                        int b_mn, void* c, int64_t ldc, int out_f32, kvp_stream_t stream) {
  kvp::GemmSeg seg{a, b, lda, ldb, K};
  return kvp::gemm_bf16(M, N, &seg, 1, a_mn ? 1 : 0, b_mn ? 1 : 0, c, ldc, out_f32 ? 1 : 0,
                        reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int kvp_selftest_bounded_wait(void* scratch, size_t scratch_bytes, kvp_stream_t stream) {
  // A [128, 512] and B [256, 512] bf16, C [128, 256] fp32; the values do not matter
  const size_t a_bytes = 128 * 512 * 2, b_bytes = 256 * 512 * 2, c_bytes = 128 * 256 * 4;
  if (scratch == nullptr || scratch_bytes < a_bytes + b_bytes + c_bytes || !kvp::aligned16(scratch)) return KVP_ERR_WORKSPACE;
  uint8_t* base = reinterpret_cast<uint8_t*>(scratch);
  kvp::GemmSeg seg{base, base + a_bytes, 512, 512, 512};
  // eight k-blocks through a four-stage ring: the arrival that frees the first stage is withheld, so the
  // producer's wait for that stage runs out after 5 ms
  return kvp::gemm_bf16(128, 256, &seg, 1, 0, 0, base + a_bytes + b_bytes, 256, 1, reinterpret_cast<cudaStream_t>(stream), 1,
                        5000000ull);
}

extern "C" int kvp_selftest_bounded_wait_pair(void* scratch, size_t scratch_bytes, kvp_stream_t stream) {
  // A [256, 512] and B [256, 512] bf16, C [256, 256] fp32: one tile of the CTA-pair kernel
  const size_t a_bytes = 256 * 512 * 2, b_bytes = 256 * 512 * 2, c_bytes = 256 * 256 * 4;
  if (scratch == nullptr || scratch_bytes < a_bytes + b_bytes + c_bytes || !kvp::aligned16(scratch)) return KVP_ERR_WORKSPACE;
  uint8_t* base = reinterpret_cast<uint8_t*>(scratch);
  kvp::GemmSeg seg{base, base + a_bytes, 512, 512, 512};
  // eight k-blocks through a six-stage ring: the arrivals that free the first stage in both CTAs are withheld, so
  // both producers' waits for that stage run out after 5 ms
  if (kvp::gemm_pair_mode() == 0) return KVP_ERR_UNSUPPORTED;
  return kvp::gemm_bf16(256, 256, &seg, 1, 0, 0, base + a_bytes + b_bytes, 256, 1, reinterpret_cast<cudaStream_t>(stream), 1,
                        5000000ull, true);
}
