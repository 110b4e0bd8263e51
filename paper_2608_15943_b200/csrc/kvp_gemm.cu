// bf16 GEMM on tcgen05 tensor cores with TMEM accumulators, operands staged by TMA.
// Used for the Q / K / V / output projections (Eq. 1 of the paper) and their chain rule.
//
// One persistent CTA per SM walks 128 x 256 output tiles.  Warp 0 issues TMA loads into a
// 4-stage shared-memory ring, warp 1 issues tcgen05.mma into one of two 256-column TMEM
// accumulators, warps 2-5 drain the other accumulator (tcgen05.ld -> registers -> global), so
// the epilogue of tile i overlaps the main loop of tile i+1.  Either operand may be K-major or
// MN-major in memory; that only changes the TMA box and the shared-memory descriptor.
// The K extent may be split over up to three operand pairs ("segments") that accumulate into the
// same tile, which is how dX = dQ Wq + dK Wk + dV Wv is produced with one output pass.
#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;            // 16 KB
constexpr int B_BYTES = BN * BK * 2;            // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;  // 48 KB
constexpr int GEMM_THREADS = 192;
constexpr int MAX_SEG = 3;
constexpr int GROUP_M = 16;  // m-tiles per rasterisation group (keeps an A slab resident in L2)
constexpr size_t GEMM_SMEM = 1024 + size_t(STAGES) * STAGE_BYTES + 256;

__device__ int g_gemm_status;

struct GemmParams {
  CUtensorMap map_a[MAX_SEG];
  CUtensorMap map_b[MAX_SEG];
  int kblocks[MAX_SEG];  // k-blocks (of BK) per segment
  int nseg;
  int M, N;
  int a_mn, b_mn;
  int out_f32;
  long long ldc;
  void* c;
  uint32_t idesc;
  // Self-test of the bounded waits (0 in every ordinary launch): the k-block count, plus one, at which the MMA
  // warp of CTA 0 withholds the arrival that frees a ring stage, and the wait limit that launch runs with.
  int withhold_at;
  unsigned long long wait_limit_ns;
};

__global__ void __launch_bounds__(GEMM_THREADS, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + size_t(STAGES) * STAGE_BYTES);
  uint64_t* full = bars;                  // [STAGES]
  uint64_t* empty = bars + STAGES;        // [STAGES]
  uint64_t* acc_full = bars + 2 * STAGES; // [2]
  uint64_t* acc_empty = acc_full + 2;     // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_gemm_status;

  const int m_tiles = (p.M + BM - 1) / BM;
  const int n_tiles = (p.N + BN - 1) / BN;
  const int total_tiles = m_tiles * n_tiles;
  int total_kb = 0;
  for (int s = 0; s < p.nseg; ++s) total_kb += p.kblocks[s];

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 4);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  auto tile_coords = [&](int t, int& tm, int& tn) {
    const int per_group = GROUP_M * n_tiles;
    const int g = t / per_group;
    const int within = t - g * per_group;
    const int gm = min(GROUP_M, m_tiles - g * GROUP_M);
    tm = g * GROUP_M + within % gm;
    tn = within / gm;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      if (lane == 0)
        for (int s = 0; s < p.nseg; ++s) {
          tma_prefetch_desc(&p.map_a[s]);
          tma_prefetch_desc(&p.map_b[s]);
        }
      __syncwarp();
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int tm, tn;
        tile_coords(t, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        for (int seg = 0; seg < p.nseg && ok; ++seg) {
          for (int kb = 0; kb < p.kblocks[seg]; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1;
            if (!mbar_wait(&empty[s], ph ^ 1, err, p.wait_limit_ns)) { ok = false; break; }
            uint8_t* sa = smem + size_t(s) * STAGE_BYTES;
            uint8_t* sb = sa + A_BYTES;
            mbar_expect_tx_e(&full[s], STAGE_BYTES, leader);
            const int k0 = kb * BK;
            if (p.a_mn == 0) {
              tma_load_2d_e(sa, &p.map_a[seg], &full[s], k0, m0, leader);
            } else {
#pragma unroll
              for (int j = 0; j < BM / 64; ++j) tma_load_2d_e(sa + j * 8192, &p.map_a[seg], &full[s], m0 + 64 * j, k0, leader);
            }
            if (p.b_mn == 0) {
              tma_load_2d_e(sb, &p.map_b[seg], &full[s], k0, n0, leader);
            } else {
#pragma unroll
              for (int j = 0; j < BN / 64; ++j) tma_load_2d_e(sb + j * 8192, &p.map_b[seg], &full[s], n0 + 64 * j, k0, leader);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      uint32_t it = 0;
      uint32_t tile_i = 0;
      bool ok = true;
      const uint32_t a_step = p.a_mn ? 2048u : 32u;   // bytes per 16-deep K step
      const uint32_t b_step = p.b_mn ? 2048u : 32u;
      const uint32_t a_lbo = p.a_mn ? 8192u : 0u;
      const uint32_t b_lbo = p.b_mn ? 8192u : 0u;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_i) {
        const int acc = tile_i & 1;
        const uint32_t acc_ph = (tile_i >> 1) & 1;
        if (!mbar_wait(&acc_empty[acc], acc_ph ^ 1, err, p.wait_limit_ns)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < total_kb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&full[s], ph, err, p.wait_limit_ns)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(smem + size_t(s) * STAGE_BYTES);
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = smem_desc_sw128(sa + k * a_step, a_lbo, 1024);
            const uint64_t db = smem_desc_sw128(sb + k * b_step, b_lbo, 1024);
            umma_ss(d_tmem, da, db, p.idesc, (kb | k) != 0, leader);
          }
          // frees the smem stage once these MMAs have read it
          if (!(p.withhold_at != 0 && blockIdx.x == 0 && it + 1 == uint32_t(p.withhold_at))) umma_commit(&empty[s], leader);
        }
        if (ok) umma_commit(&acc_full[acc], leader);
      }
    }
  } else {
    // ------------------------------ epilogue (warps 2..5) ------------------------------
    const int quarter = warp & 3;  // TMEM lane quarter this warp may access
    uint32_t tile_i = 0;
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++tile_i) {
      int tm, tn;
      tile_coords(t, tm, tn);
      const int acc = tile_i & 1;
      const uint32_t acc_ph = (tile_i >> 1) & 1;
      bool ok = mbar_wait(&acc_full[acc], acc_ph, err, p.wait_limit_ns);
      if (!__all_sync(0xffffffffu, ok)) break;
      tc_fence_after_sync();
      const int row = tm * BM + quarter * 32 + lane;
      const int n0 = tn * BN;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + acc * BN;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        if (n0 + c0 >= p.N) break;  // uniform across the warp
        uint32_t r[32];
        tmem_ld_x32(taddr + c0, r);
        tmem_ld_wait();
        if (row < p.M) {
          if (p.out_f32) {
            float* dst = reinterpret_cast<float*>(p.c) + size_t(row) * p.ldc + n0 + c0;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
              if (n0 + c0 + v * 4 < p.N) {
                uint4 val = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                *reinterpret_cast<uint4*>(dst + v * 4) = val;
              }
            }
          } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.c) + size_t(row) * p.ldc + n0 + c0;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (n0 + c0 + v * 8 < p.N) {
                uint4 val;
                val.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
                val.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                val.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                val.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                *reinterpret_cast<uint4*>(dst + v * 8) = val;
              }
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
    }
  }

  // ------------------------------ teardown ------------------------------
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

int gemm_read_status() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_gemm_status, sizeof(int)) != cudaSuccess) return -1;
  if (v != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_gemm_status, &zero, sizeof(int));
  }
  return v;
}

int gemm_bf16(int M, int N, const GemmSeg* segs, int nseg, int a_mn, int b_mn, void* c, int64_t ldc, int out_f32,
              cudaStream_t stream, int withhold_at, unsigned long long wait_limit_ns) {
  if (M <= 0 || N <= 0 || nseg < 1 || nseg > MAX_SEG || c == nullptr) return KVP_ERR_INVALID_ARG;
  if ((N % 8) != 0 || (ldc % 8) != 0 || !aligned16(c)) return KVP_ERR_UNSUPPORTED;
  GemmParams p;
  p.nseg = nseg;
  p.M = M;
  p.N = N;
  p.a_mn = a_mn;
  p.b_mn = b_mn;
  p.out_f32 = out_f32;
  p.ldc = ldc;
  p.c = c;
  p.idesc = umma_idesc_bf16(BM, BN, a_mn, b_mn);
  p.withhold_at = withhold_at;
  p.wait_limit_ns = wait_limit_ns != 0 ? wait_limit_ns : kWaitLimitNs;
  for (int s = 0; s < nseg; ++s) {
    const GemmSeg& g = segs[s];
    if (g.a == nullptr || g.b == nullptr || g.K <= 0) return KVP_ERR_INVALID_ARG;
    if ((g.K % 8) != 0 || (g.lda % 8) != 0 || (g.ldb % 8) != 0 || !aligned16(g.a) || !aligned16(g.b))
      return KVP_ERR_UNSUPPORTED;
    p.kblocks[s] = (g.K + BK - 1) / BK;
    int rc;
    if (a_mn == 0) {
      uint64_t dims[2] = {uint64_t(g.K), uint64_t(M)};
      uint64_t strides[1] = {uint64_t(g.lda) * 2};
      uint32_t box[2] = {BK, BM};
      rc = make_tensor_map(&p.map_a[s], g.a, 2, 2, dims, strides, box, true);
    } else {
      uint64_t dims[2] = {uint64_t(M), uint64_t(g.K)};
      uint64_t strides[1] = {uint64_t(g.lda) * 2};
      uint32_t box[2] = {64, BK};
      rc = make_tensor_map(&p.map_a[s], g.a, 2, 2, dims, strides, box, true);
    }
    if (rc != KVP_OK) return rc;
    if (b_mn == 0) {
      uint64_t dims[2] = {uint64_t(g.K), uint64_t(N)};
      uint64_t strides[1] = {uint64_t(g.ldb) * 2};
      uint32_t box[2] = {BK, BN};
      rc = make_tensor_map(&p.map_b[s], g.b, 2, 2, dims, strides, box, true);
    } else {
      uint64_t dims[2] = {uint64_t(N), uint64_t(g.K)};
      uint64_t strides[1] = {uint64_t(g.ldb) * 2};
      uint32_t box[2] = {64, BK};
      rc = make_tensor_map(&p.map_b[s], g.b, 2, 2, dims, strides, box, true);
    }
    if (rc != KVP_OK) return rc;
  }
  for (int s = nseg; s < MAX_SEG; ++s) {
    p.kblocks[s] = 0;
    p.map_a[s] = p.map_a[0];
    p.map_b[s] = p.map_b[0];
  }
  static const cudaError_t attr =
      cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(GEMM_SMEM));
  if (attr != cudaSuccess) return KVP_ERR_CUDA;
  const int m_tiles = (M + BM - 1) / BM, n_tiles = (N + BN - 1) / BN;
  const int grid = min(m_tiles * n_tiles, sm_count());
  timing_before(KVP_KERNEL_GEMM, stream);
  gemm_kernel<<<grid, GEMM_THREADS, GEMM_SMEM, stream>>>(p);
  timing_after(KVP_KERNEL_GEMM, stream);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

}  // namespace kvp
