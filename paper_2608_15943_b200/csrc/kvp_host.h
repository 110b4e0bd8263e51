// Host-side helpers shared by the translation units of the library (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/kvp.h"

namespace kvp {

// Builds a tiled TMA descriptor over a row-major bf16/fp32 tensor of up to 4 dimensions.
// dims[0] is the innermost (contiguous) extent in elements; strides_bytes[i] is the byte stride
// of dims[i+1].  box[] is the tile copied per request.  swizzle128 selects the 128-byte swizzle
// (the inner box extent must then span exactly 128 bytes).  Returns KVP_OK or KVP_ERR_CUDA.
int make_tensor_map(CUtensorMap* out, const void* base, int elem_bytes, int rank, const uint64_t* dims,
                    const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// One GEMM "segment": C += op(A) * op(B) over this segment's K extent.
struct GemmSeg {
  const void* a;   // bf16
  const void* b;   // bf16
  int64_t lda;     // elements: row stride of the stored matrix
  int64_t ldb;
  int K;
};

// C[M,N] = sum over segments of A_s * B_s, bf16 inputs, fp32 accumulation in TMEM.
//   a_mn == 0: A_s stored [M, K] row-major (K-major);  a_mn == 1: stored [K, M] row-major.
//   b_mn == 0: B_s stored [N, K] row-major (K-major);  b_mn == 1: stored [K, N] row-major.
//   out_f32: C is fp32 (else bf16); ldc in elements.
// withhold_at / wait_limit_ns serve the self-test of the bounded waits (kvp_selftest_bounded_wait) only.
// prefer_pair: run on CTA pairs (256 x 256 tiles) when M > 128 and the pair mode allows it.
int gemm_bf16(int M, int N, const GemmSeg* segs, int nseg, int a_mn, int b_mn, void* c, int64_t ldc, int out_f32,
              cudaStream_t stream, int withhold_at = 0, unsigned long long wait_limit_ns = 0, bool prefer_pair = true);

// One problem of a grouped launch: C[M,N] = sum over segments, with its own operand modes and output type.
struct GemmProblem {
  int M, N;
  GemmSeg segs[3];
  int nseg;
  int a_mn, b_mn;
  void* c;
  int64_t ldc;
  int out_f32;
};

// All problems in as few launches as the kernel's parameter block allows (32 problems and 48 segments per launch);
// the tiles are walked in the order of the list, so the problems with the longest tiles should come first.
// prefer_pair: CTA-pair tiles for this group (taken when every problem has more than 128 rows and the pair mode
// allows it).  The forward projections ask for pairs; the gradient GEMMs of a training step do not: under the
// board's power limit the attention backward sharing the step with them slowed by more than the pairs gained.
int gemm_grouped(const GemmProblem* probs, int n, cudaStream_t stream, bool prefer_pair);

void gemm_set_pair_mode(int mode);   // 0: single-CTA tiles only, 1: pairs where the caller prefers them, 2: pairs everywhere
int gemm_pair_mode();
int gemm_read_status();
int attn_fwd_read_status();
int attn_bwd_read_status();
int decode_read_status();

int sm_count();

// Bookkeeping for benchmarks: every kernel launch of the library is counted, and a caller may
// ask for CUDA events to be recorded around the launches of one named kernel.
enum {
  KVP_KERNEL_GEMM = 0,
  KVP_KERNEL_ATTN_FWD = 1,
  KVP_KERNEL_ATTN_BWD = 2,      // single-pass backward kernel (dQ partials, dK, dV)
  KVP_KERNEL_DECODE = 3,
  KVP_KERNEL_ATTN_BWD_AUX = 4,  // backward helper passes: Delta, accumulator clear, dQ conversion
  KVP_KERNEL_COUNT = 5
};
void note_launch(int n = 1);
void timing_before(int kernel, cudaStream_t stream);
void timing_after(int kernel, cudaStream_t stream);

}  // namespace kvp
