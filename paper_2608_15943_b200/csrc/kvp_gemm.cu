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
// One launch walks the tiles of a whole list of problems (different shapes, operands, operand modes and output
// types): the Q, K and V projections of every layer are one launch, so are all weight and input gradients of a
// backward pass, and the SMs idle only behind the last tile of the list instead of behind each GEMM's last wave.
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
constexpr int MAX_PROB = 32;   // problems per launch
constexpr int MAX_MAPS = 96;   // tensor maps per launch (two per segment)

__device__ int g_gemm_status;

struct Problem {
  int M, N;
  int m_tiles, n_tiles;
  int tile_end;            // one past this problem's last tile in the launch's tile order
  int nseg;
  int kblocks[MAX_SEG];    // k-blocks (of BK) per segment
  int total_kb;
  short map_a[MAX_SEG];    // indices into GemmParams::maps
  short map_b[MAX_SEG];
  int a_mn, b_mn;
  int out_f32;
  uint32_t idesc;
  long long ldc;
  void* c;
};

struct GemmParams {
  CUtensorMap maps[MAX_MAPS];
  Problem prob[MAX_PROB];
  int nprob;
  int total_tiles;
  // Self-test of the bounded waits (0 in every ordinary launch): the k-block count, plus one, at which the MMA
  // warp of CTA 0 withholds the arrival that frees a ring stage, and the wait limit that launch runs with.
  int withhold_at;
  unsigned long long wait_limit_ns;
};

// Position of tile t inside its problem: groups of GROUP_M m-tiles are walked n-tile by n-tile, which keeps an
// A slab resident in L2 while the B tiles stream past it.
__device__ __forceinline__ void tile_coords(int within_problem, int m_tiles, int n_tiles, int& tm, int& tn) {
  const int per_group = GROUP_M * n_tiles;
  const int g = within_problem / per_group;
  const int within = within_problem - g * per_group;
  const int gm = min(GROUP_M, m_tiles - g * GROUP_M);
  tm = g * GROUP_M + within % gm;
  tn = within / gm;
}

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
  const int total_tiles = p.total_tiles;

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

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      uint32_t it = 0;
      bool ok = true;
      int pi = 0;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        while (t >= p.prob[pi].tile_end) ++pi;
        const Problem& pr = p.prob[pi];
        int tm, tn;
        tile_coords(t - (pi ? p.prob[pi - 1].tile_end : 0), pr.m_tiles, pr.n_tiles, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        const int a_mn = pr.a_mn, b_mn = pr.b_mn;
        for (int seg = 0; seg < pr.nseg && ok; ++seg) {
          const CUtensorMap* map_a = &p.maps[pr.map_a[seg]];
          const CUtensorMap* map_b = &p.maps[pr.map_b[seg]];
          const int nkb = pr.kblocks[seg];
          for (int kb = 0; kb < nkb; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1;
            if (!mbar_wait(&empty[s], ph ^ 1, err, p.wait_limit_ns)) { ok = false; break; }
            uint8_t* sa = smem + size_t(s) * STAGE_BYTES;
            uint8_t* sb = sa + A_BYTES;
            mbar_expect_tx_e(&full[s], STAGE_BYTES, leader);
            const int k0 = kb * BK;
            if (a_mn == 0) {
              tma_load_2d_e(sa, map_a, &full[s], k0, m0, leader);
            } else {
#pragma unroll
              for (int j = 0; j < BM / 64; ++j) tma_load_2d_e(sa + j * 8192, map_a, &full[s], m0 + 64 * j, k0, leader);
            }
            if (b_mn == 0) {
              tma_load_2d_e(sb, map_b, &full[s], k0, n0, leader);
            } else {
#pragma unroll
              for (int j = 0; j < BN / 64; ++j) tma_load_2d_e(sb + j * 8192, map_b, &full[s], n0 + 64 * j, k0, leader);
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
      int pi = 0;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_i) {
        while (t >= p.prob[pi].tile_end) ++pi;
        const Problem& pr = p.prob[pi];
        const uint32_t a_step = pr.a_mn ? 2048u : 32u;   // bytes per 16-deep K step
        const uint32_t b_step = pr.b_mn ? 2048u : 32u;
        const uint32_t a_lbo = pr.a_mn ? 8192u : 0u;
        const uint32_t b_lbo = pr.b_mn ? 8192u : 0u;
        const uint32_t idesc = pr.idesc;
        const int total_kb = pr.total_kb;
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
            umma_ss(d_tmem, da, db, idesc, (kb | k) != 0, leader);
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
    int pi = 0;
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++tile_i) {
      while (t >= p.prob[pi].tile_end) ++pi;
      const Problem& pr = p.prob[pi];
      int tm, tn;
      tile_coords(t - (pi ? p.prob[pi - 1].tile_end : 0), pr.m_tiles, pr.n_tiles, tm, tn);
      const int M = pr.M, N = pr.N, out_f32 = pr.out_f32;
      const long long ldc = pr.ldc;
      void* const c = pr.c;
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
        if (n0 + c0 >= N) break;  // uniform across the warp
        uint32_t r[32];
        tmem_ld_x32(taddr + c0, r);
        tmem_ld_wait();
        if (row < M) {
          if (out_f32) {
            float* dst = reinterpret_cast<float*>(c) + size_t(row) * ldc + n0 + c0;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
              if (n0 + c0 + v * 4 < N) {
                uint4 val = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                *reinterpret_cast<uint4*>(dst + v * 4) = val;
              }
            }
          } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(c) + size_t(row) * ldc + n0 + c0;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (n0 + c0 + v * 8 < N) {
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


// ------------------------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs: 256 x 256 output tiles, one per pair of SMs (a cluster of two CTAs).  Each CTA of the
// pair loads 128 rows of A and 128 of the tile's 256 rows of B per k-block (32 KB per stage instead of 48 KB, so
// the ring is six stages deep) and drains its own 128 accumulator rows; the even CTA issues the M = 256 MMAs for
// both.  An MMA then reads 8 KB of operands per SM where the single-CTA tile reads 12 KB, which takes the shared-
// memory port off the critical path.  Barriers: full[s] lives in the even CTA and counts the bytes of both CTAs'
// loads; empty[s] and acc_full[a] exist in both CTAs and receive one MMA-completion arrival each; acc_empty[a]
// lives in the even CTA and collects the eight epilogue warps of the pair.
// ------------------------------------------------------------------------------------------------------------
constexpr int PBM = 256;                          // tile rows per pair
constexpr int PHALF = 128;                        // rows of A, and rows of B, per CTA
constexpr int PSTAGES = 6;
constexpr int PA_BYTES = PHALF * BK * 2;          // 16 KB
constexpr int PB_BYTES = PHALF * BK * 2;          // 16 KB
constexpr int PSTAGE_BYTES = PA_BYTES + PB_BYTES; // 32 KB per CTA
constexpr size_t PAIR_SMEM = 1024 + size_t(PSTAGES) * PSTAGE_BYTES + 256;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
    gemm_pair_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + size_t(PSTAGES) * PSTAGE_BYTES);
  uint64_t* full = bars;                    // [PSTAGES]  (used in the even CTA)
  uint64_t* empty = bars + PSTAGES;         // [PSTAGES]
  uint64_t* acc_full = bars + 2 * PSTAGES;  // [2]
  uint64_t* acc_empty = acc_full + 2;       // [2]        (used in the even CTA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_gemm_status;
  const int total_tiles = p.total_tiles;
  const uint32_t rank = cluster_ctarank();  // 0: issues the MMAs; 1: partner
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 8);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the partner's barriers exist before anything of this CTA can signal them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    {
      const uint32_t leader = elect_one();
      uint32_t it = 0;
      bool ok = true;
      int pi = 0;
      for (int t = pair; t < total_tiles && ok; t += n_pairs) {
        while (t >= p.prob[pi].tile_end) ++pi;
        const Problem& pr = p.prob[pi];
        int tm, tn;
        tile_coords(t - (pi ? p.prob[pi - 1].tile_end : 0), pr.m_tiles, pr.n_tiles, tm, tn);
        const int m0 = tm * PBM + int(rank) * PHALF, n0 = tn * BN + int(rank) * PHALF;
        const int a_mn = pr.a_mn, b_mn = pr.b_mn;
        for (int seg = 0; seg < pr.nseg && ok; ++seg) {
          const CUtensorMap* map_a = &p.maps[pr.map_a[seg]];
          const CUtensorMap* map_b = &p.maps[pr.map_b[seg]];
          const int nkb = pr.kblocks[seg];
          for (int kb = 0; kb < nkb; ++kb, ++it) {
            const int s = it % PSTAGES;
            const uint32_t ph = (it / PSTAGES) & 1;
            if (!mbar_wait(&empty[s], ph ^ 1, err, p.wait_limit_ns)) { ok = false; break; }
            uint8_t* sa = smem + size_t(s) * PSTAGE_BYTES;
            uint8_t* sb = sa + PA_BYTES;
            if (rank == 0) mbar_expect_tx_e(&full[s], 2 * PSTAGE_BYTES, leader);   // both CTAs' bytes
            const uint32_t bar = cluster_addr_of(&full[s], 0);
            const int k0 = kb * BK;
            if (a_mn == 0) {
              tma_load_2d_pair_e(sa, map_a, bar, k0, m0, leader);
            } else {
#pragma unroll
              for (int j = 0; j < PHALF / 64; ++j) tma_load_2d_pair_e(sa + j * 8192, map_a, bar, m0 + 64 * j, k0, leader);
            }
            if (b_mn == 0) {
              tma_load_2d_pair_e(sb, map_b, bar, k0, n0, leader);
            } else {
#pragma unroll
              for (int j = 0; j < PHALF / 64; ++j) tma_load_2d_pair_e(sb + j * 8192, map_b, bar, n0 + 64 * j, k0, leader);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (even CTA only) ------------------------------
    if (rank == 0) {
      const uint32_t leader = elect_one();
      uint32_t it = 0;
      uint32_t tile_i = 0;
      bool ok = true;
      int pi = 0;
      for (int t = pair; t < total_tiles && ok; t += n_pairs, ++tile_i) {
        while (t >= p.prob[pi].tile_end) ++pi;
        const Problem& pr = p.prob[pi];
        const uint32_t a_step = pr.a_mn ? 2048u : 32u;   // bytes per 16-deep K step
        const uint32_t b_step = pr.b_mn ? 2048u : 32u;
        const uint32_t a_lbo = pr.a_mn ? 8192u : 0u;
        const uint32_t b_lbo = pr.b_mn ? 8192u : 0u;
        const uint32_t idesc = pr.idesc;
        const int total_kb = pr.total_kb;
        const int acc = tile_i & 1;
        const uint32_t acc_ph = (tile_i >> 1) & 1;
        if (!mbar_wait(&acc_empty[acc], acc_ph ^ 1, err, p.wait_limit_ns)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < total_kb; ++kb, ++it) {
          const int s = it % PSTAGES;
          const uint32_t ph = (it / PSTAGES) & 1;
          if (!mbar_wait(&full[s], ph, err, p.wait_limit_ns)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(smem + size_t(s) * PSTAGE_BYTES);
          const uint32_t sb = sa + PA_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = smem_desc_sw128(sa + k * a_step, a_lbo, 1024);
            const uint64_t db = smem_desc_sw128(sb + k * b_step, b_lbo, 1024);
            umma_ss_pair(d_tmem, da, db, idesc, (kb | k) != 0, leader);
          }
          // frees the stage in both CTAs once these MMAs have read it
          if (!(p.withhold_at != 0 && pair == 0 && it + 1 == uint32_t(p.withhold_at))) {
            umma_commit_pair(cluster_addr_of(&empty[s], 0), leader);
            umma_commit_pair(cluster_addr_of(&empty[s], 1), leader);
          }
        }
        if (ok) {
          umma_commit_pair(cluster_addr_of(&acc_full[acc], 0), leader);
          umma_commit_pair(cluster_addr_of(&acc_full[acc], 1), leader);
        }
      }
    }
  } else {
    // ------------------------------ epilogue (warps 2..5 of both CTAs) ------------------------------
    const int quarter = warp & 3;  // TMEM lane quarter this warp may access
    uint32_t tile_i = 0;
    int pi = 0;
    for (int t = pair; t < total_tiles; t += n_pairs, ++tile_i) {
      while (t >= p.prob[pi].tile_end) ++pi;
      const Problem& pr = p.prob[pi];
      int tm, tn;
      tile_coords(t - (pi ? p.prob[pi - 1].tile_end : 0), pr.m_tiles, pr.n_tiles, tm, tn);
      const int M = pr.M, N = pr.N, out_f32 = pr.out_f32;
      const long long ldc = pr.ldc;
      void* const c = pr.c;
      const int acc = tile_i & 1;
      const uint32_t acc_ph = (tile_i >> 1) & 1;
      bool ok = mbar_wait(&acc_full[acc], acc_ph, err, p.wait_limit_ns);
      if (!__all_sync(0xffffffffu, ok)) break;
      tc_fence_after_sync();
      const int row = tm * PBM + int(rank) * PHALF + quarter * 32 + lane;
      const int n0 = tn * BN;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + acc * BN;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        if (n0 + c0 >= N) break;  // uniform across the warp
        uint32_t r[32];
        tmem_ld_x32(taddr + c0, r);
        tmem_ld_wait();
        if (row < M) {
          if (out_f32) {
            float* dst = reinterpret_cast<float*>(c) + size_t(row) * ldc + n0 + c0;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
              if (n0 + c0 + v * 4 < N) {
                uint4 val = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                *reinterpret_cast<uint4*>(dst + v * 4) = val;
              }
            }
          } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(c) + size_t(row) * ldc + n0 + c0;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (n0 + c0 + v * 8 < N) {
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
      if (lane == 0) mbar_arrive_cluster(cluster_addr_of(&acc_empty[acc], 0));
    }
  }

  // ------------------------------ teardown ------------------------------
  // Neither CTA may leave, or free its TMEM, while the partner can still signal its barriers or while MMAs of the
  // pair can still write its accumulator: both wait for each other first.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 512);
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

namespace {

int check_problem(const GemmProblem& g) {
  if (g.M <= 0 || g.N <= 0 || g.nseg < 1 || g.nseg > MAX_SEG || g.c == nullptr) return KVP_ERR_INVALID_ARG;
  if ((g.N % 8) != 0 || (g.ldc % 8) != 0 || !aligned16(g.c)) return KVP_ERR_UNSUPPORTED;
  for (int s = 0; s < g.nseg; ++s) {
    const GemmSeg& e = g.segs[s];
    if (e.a == nullptr || e.b == nullptr || e.K <= 0) return KVP_ERR_INVALID_ARG;
    if ((e.K % 8) != 0 || (e.lda % 8) != 0 || (e.ldb % 8) != 0 || !aligned16(e.a) || !aligned16(e.b))
      return KVP_ERR_UNSUPPORTED;
  }
  return KVP_OK;
}

// Tensor maps of one operand pair; the box depends on the operand mode and on the rows of B one CTA loads.
int encode_segment(const GemmProblem& g, const GemmSeg& e, CUtensorMap* map_a, CUtensorMap* map_b, uint32_t b_rows) {
  int rc;
  if (g.a_mn == 0) {
    uint64_t dims[2] = {uint64_t(e.K), uint64_t(g.M)};
    uint64_t strides[1] = {uint64_t(e.lda) * 2};
    uint32_t box[2] = {BK, BM};
    rc = make_tensor_map(map_a, e.a, 2, 2, dims, strides, box, true);
  } else {
    uint64_t dims[2] = {uint64_t(g.M), uint64_t(e.K)};
    uint64_t strides[1] = {uint64_t(e.lda) * 2};
    uint32_t box[2] = {64, BK};
    rc = make_tensor_map(map_a, e.a, 2, 2, dims, strides, box, true);
  }
  if (rc != KVP_OK) return rc;
  if (g.b_mn == 0) {
    uint64_t dims[2] = {uint64_t(e.K), uint64_t(g.N)};
    uint64_t strides[1] = {uint64_t(e.ldb) * 2};
    uint32_t box[2] = {BK, b_rows};
    rc = make_tensor_map(map_b, e.b, 2, 2, dims, strides, box, true);
  } else {
    uint64_t dims[2] = {uint64_t(g.N), uint64_t(e.K)};
    uint64_t strides[1] = {uint64_t(e.ldb) * 2};
    uint32_t box[2] = {64, BK};
    rc = make_tensor_map(map_b, e.b, 2, 2, dims, strides, box, true);
  }
  return rc;
}

int launch_group(const GemmProblem* probs, int n, cudaStream_t stream, int withhold_at, unsigned long long wait_limit_ns,
                 bool pair) {
  const int bm = pair ? PBM : BM;
  static thread_local GemmParams p;   // 15 KB: kept off the stack
  p.nprob = n;
  p.withhold_at = withhold_at;
  p.wait_limit_ns = wait_limit_ns != 0 ? wait_limit_ns : kWaitLimitNs;
  int n_maps = 0, tiles = 0;
  for (int i = 0; i < n; ++i) {
    const GemmProblem& g = probs[i];
    Problem& q = p.prob[i];
    q.M = g.M;
    q.N = g.N;
    q.m_tiles = (g.M + bm - 1) / bm;
    q.n_tiles = (g.N + BN - 1) / BN;
    tiles += q.m_tiles * q.n_tiles;
    q.tile_end = tiles;
    q.nseg = g.nseg;
    q.total_kb = 0;
    for (int s = 0; s < MAX_SEG; ++s) {
      q.kblocks[s] = 0;
      q.map_a[s] = q.map_b[s] = 0;
    }
    for (int s = 0; s < g.nseg; ++s) {
      q.kblocks[s] = (g.segs[s].K + BK - 1) / BK;
      q.total_kb += q.kblocks[s];
      q.map_a[s] = short(n_maps);
      q.map_b[s] = short(n_maps + 1);
      const int rc = encode_segment(g, g.segs[s], &p.maps[n_maps], &p.maps[n_maps + 1], pair ? PHALF : BN);
      if (rc != KVP_OK) return rc;
      n_maps += 2;
    }
    q.a_mn = g.a_mn;
    q.b_mn = g.b_mn;
    q.out_f32 = g.out_f32;
    q.idesc = umma_idesc_bf16(bm, BN, g.a_mn, g.b_mn);
    q.ldc = g.ldc;
    q.c = g.c;
  }
  for (int i = n; i < MAX_PROB; ++i) p.prob[i] = p.prob[n - 1];
  p.total_tiles = tiles;
  static const cudaError_t attr =
      cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(GEMM_SMEM));
  static const cudaError_t attr_pair =
      cudaFuncSetAttribute(gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(PAIR_SMEM));
  if (attr != cudaSuccess || attr_pair != cudaSuccess) return KVP_ERR_CUDA;
  timing_before(KVP_KERNEL_GEMM, stream);
  if (pair)
    gemm_pair_kernel<<<2 * min(tiles, sm_count() / 2), GEMM_THREADS, PAIR_SMEM, stream>>>(p);
  else
    gemm_kernel<<<min(tiles, sm_count()), GEMM_THREADS, GEMM_SMEM, stream>>>(p);
  timing_after(KVP_KERNEL_GEMM, stream);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

// 0: single-CTA tiles only; 1: CTA pairs where the caller prefers them (forward GEMMs); 2: CTA pairs everywhere.
// Pairs are never used for a group with a problem of at most 128 rows (half of every pair tile would be padding).
int g_pair_mode = 1;

bool use_pair(const GemmProblem* probs, int n, bool prefer_pair) {
  if (g_pair_mode == 0 || (g_pair_mode == 1 && !prefer_pair)) return false;
  for (int i = 0; i < n; ++i)
    if (probs[i].M <= BM) return false;
  return true;
}

}  // namespace

void gemm_set_pair_mode(int mode) { g_pair_mode = mode; }
int gemm_pair_mode() { return g_pair_mode; }

int gemm_grouped(const GemmProblem* probs, int n, cudaStream_t stream, bool prefer_pair) {
  if (n < 0 || (n > 0 && probs == nullptr)) return KVP_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    const int rc = check_problem(probs[i]);
    if (rc != KVP_OK) return rc;
  }
  // as many problems per launch as the parameter block holds
  int begin = 0;
  while (begin < n) {
    int end = begin, maps = 0;
    while (end < n && end - begin < MAX_PROB && maps + 2 * probs[end].nseg <= MAX_MAPS) maps += 2 * probs[end++].nseg;
    const int rc = launch_group(probs + begin, end - begin, stream, 0, 0, use_pair(probs + begin, end - begin, prefer_pair));
    if (rc != KVP_OK) return rc;
    begin = end;
  }
  return KVP_OK;
}

int gemm_bf16(int M, int N, const GemmSeg* segs, int nseg, int a_mn, int b_mn, void* c, int64_t ldc, int out_f32,
              cudaStream_t stream, int withhold_at, unsigned long long wait_limit_ns, bool prefer_pair) {
  if (nseg < 1 || nseg > MAX_SEG || segs == nullptr) return KVP_ERR_INVALID_ARG;
  GemmProblem g{};
  g.M = M;
  g.N = N;
  g.nseg = nseg;
  for (int s = 0; s < nseg; ++s) g.segs[s] = segs[s];
  g.a_mn = a_mn;
  g.b_mn = b_mn;
  g.c = c;
  g.ldc = ldc;
  g.out_f32 = out_f32;
  const int rc = check_problem(g);
  if (rc != KVP_OK) return rc;
  return launch_group(&g, 1, stream, withhold_at, wait_limit_ns, use_pair(&g, 1, prefer_pair));
}

}  // namespace kvp
