// Flash-attention backward over a donor map (chain rule of Eq. 2-3 of the paper), two kernels:
//
//  dkdv_kernel  KV-stationary.  One CTA owns a 128-row K/V tile of one (batch, KV head) of a DONOR
//               layer, keeps K and V in shared memory and the dK / dV accumulators in TMEM (fp32)
//               while it walks every query stream that reads the tile: the donor itself and all its
//               consumer layers, the Hq/Hkv query heads of the KV head's group, and every 64-row query
//               tile the causal mask lets see the keys.  dK and dV of the donor are therefore summed on
//               chip across layers and heads and written to HBM once.  Per step, transposed so that TMEM
//               lane == key row:  S^T = K Q^T, dP^T = V dO^T (tcgen05, operands in shared memory), each
//               followed by one rank-3 MMA that subtracts the query's LSE/scale resp. Delta (a bf16
//               three-term split against a tile of ones), so the accumulators already hold the
//               exponent and dP - Delta; P^T = exp2(c acc), dS^T = P^T acc' are written back as bf16
//               over the same TMEM columns and fed to dV += P^T dO, dK += dS^T Q as the A operand FROM
//               TMEM -- P and dS never touch shared memory.  Two TMEM buffer sets alternate between
//               steps; both compute warpgroups work on every step, each on half of its query columns.
//
//  dq_kernel    Q-stationary (like the forward).  One CTA owns a 128-row query tile of one (layer,
//               batch, query head) and walks the donor's K/V tiles: S = Q K^T, dP = dO V^T,
//               dS = P (dP - Delta) written as bf16 over dP's TMEM columns, dQ += dS K with dS as the A
//               operand from TMEM and K as an MN-major B operand.  dQ accumulates in TMEM and is
//               written once, as bf16, already scaled: no atomics, no fp32 dQ round trip through HBM.
//
// Delta = rowsum(dO * O) comes from a small pre-pass.  Recomputing S and dP in both kernels costs
// two extra GEMMs per tile pair; it removes 64 KB of fp32 reduction traffic per tile pair, which is
// what bounded the single-kernel form.
#include <math.h>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int BT = 128;    // key rows per tile (both kernels), query rows per tile in dq_kernel
constexpr int BQ2 = 64;    // query rows per step in dkdv_kernel
constexpr int MAX_GROUP = 8;  // layers of one donor group per dkdv launch
constexpr uint32_t HALF_BYTES = 128 * 128;  // [128 rows x 128 B] block
constexpr uint32_t QHALF_BYTES = 64 * 128;  // [ 64 rows x 128 B] block

__device__ int g_bwd_status;

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// =============================================================================================
// dK / dV
// =============================================================================================
constexpr int DKDV_THREADS = 320;  // warp 0 TMA, warp 1 MMA, warps 2-5 and 6-9 two compute warpgroups
constexpr int DKDV_STAGES = 4;     // ring of (Q, dO) 64-row tiles

template <int DH>
struct DkdvSmem {
  static constexpr int KV_TILE = BT * DH * 2;
  static constexpr int Q_TILE = BQ2 * DH * 2;
  static constexpr int STAGE = 2 * Q_TILE;  // Q then dO
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = OFF_K + KV_TILE;
  static constexpr int OFF_RING = OFF_V + KV_TILE;
  static constexpr int OFF_ONES = OFF_RING + DKDV_STAGES * STAGE;  // [128 x 16] bf16, unswizzled K-major
  static constexpr int OFF_STAT = OFF_ONES + 4096;                 // [4 steps][lse, delta][64 x 16] bf16
  static constexpr int OFF_BAR = OFF_STAT + 8 * 2048;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;
};

struct DkdvParams {
  CUtensorMap map_k, map_v;       // donor K, V: [B,S,Hkv,dh], box rows 128
  CUtensorMap map_q[MAX_GROUP];   // per layer of the group, box rows 64
  CUtensorMap map_do[MAX_GROUP];
  const float* lse[MAX_GROUP];    // [B,Hq,S]
  const float* delta[MAX_GROUP];  // [B,Hq,S]
  float* dk_sum;                  // fp32 [B,S,Hkv,dh]
  float* dv_sum;
  int n_layers;
  int B, S, Hq, Hkv;
  int causal;
  int chunk;                      // (batch, KV head) pairs per dispatch chunk
  float scale;
  float scale_log2;
};

// Unswizzled K-major operand tile of 16 bf16 per row: two halves of 8 columns, each half stored as
// rows of 16 bytes (8 rows = one 128-byte core matrix).  SBO = 128, LBO = rows * 16.
__host__ __device__ constexpr uint32_t desc_hi_plain(uint32_t sbo_bytes) { return ((sbo_bytes >> 4) & 0x3FFF) | (1u << 14); }
__device__ __forceinline__ uint32_t desc_lo_plain(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFF) >> 4) | (((lbo_bytes >> 4) & 0x3FFF) << 16);
}
// v = h + m + l with h, m, l bf16: 24 significant bits, so a bf16 MMA can add v exactly enough
__device__ __forceinline__ uint4 split3_bf16(float v) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(h);
  const __nv_bfloat16 m = __float2bfloat16_rn(r1);
  const __nv_bfloat16 l = __float2bfloat16_rn(r1 - __bfloat162float(m));
  uint4 out;
  out.x = uint32_t(__bfloat16_as_ushort(h)) | (uint32_t(__bfloat16_as_ushort(m)) << 16);
  out.y = uint32_t(__bfloat16_as_ushort(l));
  out.z = 0u;
  out.w = 0u;
  return out;
}

// Per 64-query step, transposed so that TMEM lane == key row: S^T = K Q^T and dP^T = V dO^T.  The
// per-query statistics are applied BY THE TENSOR CORE: one extra K-step multiplies a [128 x 16] tile
// of ones (first three columns) with a [64 x 16] tile holding -LSE/scale (resp. -Delta) of each query
// split into three bf16 terms, so the accumulators already hold S - LSE/scale and dP - Delta and the
// threads need no per-column operand: P^T = exp2(c * acc), dS^T = P^T * acc'.
template <int DH>
__global__ void __launch_bounds__(DKDV_THREADS, 1) dkdv_kernel(const __grid_constant__ DkdvParams p) {
  using L = DkdvSmem<DH>;
  constexpr int HALVES = DH / 64;
  constexpr int KSTEPS_DH = DH / 16;
  constexpr int KSTEPS_Q = BQ2 / 16;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* kv_full = bars + 0;
  uint64_t* q_full = bars + 1;                    // [STAGES]
  uint64_t* q_empty = q_full + DKDV_STAGES;       // [STAGES]
  uint64_t* st_full = q_empty + DKDV_STAGES;      // [2]  S^T and dP^T of buffer set b are in TMEM
  uint64_t* pds_ready = st_full + 2;              // [2]  P^T, dS^T written and the set's next statistics staged
  uint64_t* stat0 = pds_ready + 2;                // statistics of the first two steps staged (256 arrivals)
  uint64_t* acc_done = stat0 + 1;                 // all MMAs have completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_done + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_bwd_status;

  // Blocks are dispatched in index order.  The (batch, KV head) pairs are taken in chunks of p.chunk pairs;
  // inside a chunk the key tile is the slow index, so that under the causal mask the chunk's heaviest tiles
  // (tile 0 sees every query tile) start first, while all CTAs that stream the same Q / dO tiles run within
  // a wave or two of each other and find them in L2.
  const int n_jt = (p.S + BT - 1) / BT;
  const int n_pairs = p.Hkv * p.B;
  const int chunk_i = blockIdx.x / (p.chunk * n_jt);
  const int in_chunk = blockIdx.x - chunk_i * p.chunk * n_jt;
  const int chunk_n = min(p.chunk, n_pairs - chunk_i * p.chunk);  // the last chunk may be short
  const int jt = in_chunk / chunk_n;
  const int pair = chunk_i * p.chunk + (in_chunk - jt * chunk_n);
  const int hk = pair % p.Hkv;
  const int b = pair / p.Hkv;
  const int G = p.Hq / p.Hkv;
  const int kv0 = jt * BT;
  const int n_qt = (p.S + BQ2 - 1) / BQ2;
  const int qt_first = p.causal ? (kv0 / BQ2) : 0;
  const int per_stream = n_qt - qt_first;
  const int n_iter = p.n_layers * G * per_stream;

  if (threadIdx.x == 0) {
    mbar_init(kv_full, 1);
    for (int s = 0; s < DKDV_STAGES; ++s) {
      mbar_init(&q_full[s], 1);
      mbar_init(&q_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&st_full[i], 1);
      mbar_init(&pds_ready[i], 256);
    }
    mbar_init(stat0, 256);
    mbar_init(acc_done, 1);
    mbar_fence_init();
  }
  // constant operand tiles: ones in the first three columns; statistics tiles start as zeros
  for (int i = threadIdx.x; i < (4096 + 8 * 2048) / 16; i += blockDim.x) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (i < 128) v = make_uint4(0x3F803F80u, 0x00003F80u, 0u, 0u);  // row i, columns 0-7 = 1,1,1,0,0,0,0,0
    *reinterpret_cast<uint4*>(smem + L::OFF_ONES + i * 16) = v;
  }
  fence_proxy_async_smem();
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // buffer set i: S^T at [i*128, i*128+64), dP^T at [i*128+64, i*128+128); accumulators above
  const uint32_t tm_dk = tmem_base + 256;
  const uint32_t tm_dv = tmem_base + 384;

  auto decode_iter = [&](int it, int& li, int& hq, int& q0) {
    const int stream = it / per_stream;
    const int qi = it - stream * per_stream;
    li = stream / G;
    hq = hk * G + (stream - li * G);
    q0 = (qt_first + qi) * BQ2;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      if (leader) tma_prefetch_desc(&p.map_k);
      if (leader) tma_prefetch_desc(&p.map_v);
      mbar_expect_tx_e(kv_full, 2 * L::KV_TILE, leader);
#pragma unroll
      for (int h = 0; h < HALVES; ++h) {
        tma_load_4d_e(smem + L::OFF_K + h * HALF_BYTES, &p.map_k, kv_full, h * 64, hk, kv0, b, leader);
        tma_load_4d_e(smem + L::OFF_V + h * HALF_BYTES, &p.map_v, kv_full, h * 64, hk, kv0, b, leader);
      }
      for (int it = 0; it < n_iter; ++it) {
        int li, hq, q0;
        decode_iter(it, li, hq, q0);
        const int s = it % DKDV_STAGES;
        const uint32_t ph = (it / DKDV_STAGES) & 1;
        if (!mbar_wait(&q_empty[s], ph ^ 1, err)) break;
        mbar_expect_tx_e(&q_full[s], L::STAGE, leader);
        uint8_t* dst = smem + L::OFF_RING + s * L::STAGE;
#pragma unroll
        for (int h = 0; h < HALVES; ++h) {
          tma_load_4d_e(dst + h * QHALF_BYTES, &p.map_q[li], &q_full[s], h * 64, hq, q0, b, leader);
          tma_load_4d_e(dst + L::Q_TILE + h * QHALF_BYTES, &p.map_do[li], &q_full[s], h * 64, hq, q0, b, leader);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      constexpr uint32_t idesc_st = umma_idesc_bf16(BT, BQ2, 0, 0);   // [128 keys x 64 queries]
      constexpr uint32_t idesc_acc = umma_idesc_bf16(BT, DH, 0, 1);   // A from TMEM, B MN-major
      constexpr uint32_t hi = desc_hi_sw128(1024);
      constexpr uint32_t hi_plain = desc_hi_plain(128);
      // low descriptor words of the resident tiles; per MMA only a constant is added
      const uint32_t k_lo = desc_lo_sw128(smem_u32(smem + L::OFF_K), 0);
      const uint32_t v_lo = desc_lo_sw128(smem_u32(smem + L::OFF_V), 0);
      const uint32_t ones_lo = desc_lo_plain(smem_u32(smem + L::OFF_ONES), 2048);
      const uint32_t stat_base = smem_u32(smem + L::OFF_STAT);
      const uint32_t ring = smem_u32(smem + L::OFF_RING);
      bool ok = mbar_wait(kv_full, 0, err);
      if (ok) ok = mbar_wait(stat0, 0, err);
      auto issue_scores = [&](int it) -> bool {
        const int s = it % DKDV_STAGES;
        if (!mbar_wait(&q_full[s], (it / DKDV_STAGES) & 1, err)) return false;
        tc_fence_after_sync();
        const uint32_t q_lo = desc_lo_sw128(ring + s * L::STAGE, 0);
        const uint32_t do_lo = desc_lo_sw128(ring + s * L::STAGE + L::Q_TILE, 0);
        const uint32_t tm = tmem_base + (it & 1) * 128;
        const uint32_t stat_lo = desc_lo_plain(stat_base + (it & 3) * 4096, 1024);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t offa = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          const uint32_t offb = (ks / 4) * QHALF_BYTES + (ks % 4) * 32;
          umma_ss_w(tm, desc_lo_add(k_lo, offa), desc_lo_add(q_lo, offb), hi, idesc_st, ks != 0, leader);
        }
        umma_ss_w(tm, ones_lo, stat_lo, hi_plain, idesc_st, 1, leader);                          // S^T -= LSE / scale
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t offa = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          const uint32_t offb = (ks / 4) * QHALF_BYTES + (ks % 4) * 32;
          umma_ss_w(tm + 64, desc_lo_add(v_lo, offa), desc_lo_add(do_lo, offb), hi, idesc_st, ks != 0, leader);
        }
        umma_ss_w(tm + 64, ones_lo, desc_lo_add(stat_lo, 2048), hi_plain, idesc_st, 1, leader);  // dP^T -= Delta
        umma_commit(&st_full[it & 1], leader);
        return true;
      };
      if (ok && n_iter > 0) ok = issue_scores(0);
      for (int it = 0; it < n_iter && ok; ++it) {
        // scores of the next step go to the other buffer set; its previous readers (the accumulate
        // MMAs of step it-1) precede this in the in-order tensor pipe, and its statistics tile was
        // staged before pds_ready(it-1)
        if (it + 1 < n_iter && !issue_scores(it + 1)) { ok = false; break; }
        if (!mbar_wait(&pds_ready[it & 1], (it >> 1) & 1, err)) { ok = false; break; }
        tc_fence_after_sync();
        const int s = it % DKDV_STAGES;
        const uint32_t qmn_lo = desc_lo_sw128(ring + s * L::STAGE, QHALF_BYTES);                 // Q  as MN-major B
        const uint32_t domn_lo = desc_lo_sw128(ring + s * L::STAGE + L::Q_TILE, QHALF_BYTES);    // dO as MN-major B
        const uint32_t tm = tmem_base + (it & 1) * 128;
#pragma unroll
        for (int ks = 0; ks < KSTEPS_Q; ++ks)  // dV += P^T dO
          umma_ts_w(tm_dv, tm + ks * 8 + (ks / 2) * 32, desc_lo_add(domn_lo, ks * 2048), hi, idesc_acc, (it | ks) != 0, leader);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_Q; ++ks)  // dK += dS^T Q
          umma_ts_w(tm_dk, tm + 64 + ks * 8 + (ks / 2) * 32, desc_lo_add(qmn_lo, ks * 2048), hi, idesc_acc, (it | ks) != 0, leader);
        umma_commit(&q_empty[s], leader);
      }
      if (ok) umma_commit(acc_done, leader);
    }
  } else {
    // ------------------------------ compute warpgroups ------------------------------
    const int wg = (warp - 2) >> 2;     // query columns [wg*32, wg*32+32) of every step
    const int quarter = warp & 3;       // TMEM lane quarter of this warp
    const int r = quarter * 32 + lane;  // key row inside the tile == TMEM lane
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    const int kv_row = kv0 + r;
    const float inv_scale = 1.f / p.scale;
    // Statistics: in each warpgroup, lane quarter 0 stages -LSE/scale and quarter 1 stages -Delta of
    // the warpgroup's 32 query columns.  Values are fetched two steps before they are staged, so the
    // global-memory latency never shows.
    const int stat_kind = quarter ^ 2;  // 0 lse, 1 delta, others idle: the warps whose scheduler hosts no TMA / MMA warp
    uint8_t* stat_row = smem + L::OFF_STAT + (stat_kind & 1) * 2048 + (wg * 32 + lane) * 16;
    // Loads are unconditional (from a clamped, always valid address) and their raw values travel in
    // registers together with a validity flag; sign, 1/scale and the padding value are applied when a
    // value is staged two steps later, so that no instruction depends on a load in the step that issues it.
    const float stat_mul = stat_kind == 0 ? -inv_scale : -1.f;
    const float stat_pad = stat_kind == 0 ? -30000.f : 0.f;  // a query beyond the sequence: exp2 underflows to zero
    // Two cursors walk the steps in order (incremental decode of step -> layer, head, query tile): one
    // for the step whose statistics are loaded next, one kStatAhead steps further that only pulls the
    // line into L2 -- the loads are a few steps ahead of their use, which hides an L2 hit but not DRAM.
    constexpr int kStatAhead = 12;
    struct Cursor {
      int it = 0, qi = 0, g = 0, li = 0;
    };
    auto advance = [&](Cursor& c) {
      ++c.it;
      if (++c.qi == per_stream) {
        c.qi = 0;
        if (++c.g == G) {
          c.g = 0;
          ++c.li;
        }
      }
    };
    const float* f_ptr = p.lse[0];
    auto locate = [&](const Cursor& c, bool& valid) {  // address of this lane's statistic of step c (clamped, always valid)
      valid = false;
      if (stat_kind < 2 && c.it < n_iter) {
        const int qc = (qt_first + c.qi) * BQ2 + wg * 32 + lane;
        valid = qc < p.S;
        const float* src = stat_kind == 0 ? p.lse[c.li] : p.delta[c.li];
        f_ptr = src + (size_t(b) * p.Hq + hk * G + c.g) * p.S + (valid ? qc : p.S - 1);
      }
      return f_ptr;
    };
    Cursor cf, cp;
    for (int i = 0; i < kStatAhead; ++i) advance(cp);
    auto fetch = [&](bool& valid) -> float {
      bool ahead_valid;
      const float* ahead = locate(cp, ahead_valid);
      if (lane == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(ahead));
      advance(cp);
      const float* ptr = locate(cf, valid);
      advance(cf);
      return __ldg(ptr);
    };
    auto stage = [&](int tile, float raw, bool valid) {
      if (stat_kind < 2) *reinterpret_cast<uint4*>(stat_row + tile * 4096) = split3_bf16(valid ? raw * stat_mul : stat_pad);
    };
    bool v0, v1;
    float s0, s1;
#pragma unroll 1
    for (int i = 0; i < 3; ++i) {  // the tiles of steps 0..2; step n+3's tile is staged at the end of step n
      s0 = fetch(v0);
      stage(i, s0, v0);
    }
    fence_proxy_async_smem();
    mbar_arrive(stat0);
    s0 = fetch(v0);
    s1 = fetch(v1);
    const uint64_t c2 = pack_f2(p.scale_log2, p.scale_log2);
    // P^T and dS^T (bf16 pairs) overwrite the first half of the warpgroup's OWN score columns: 32-bit
    // columns [wg*48, wg*48+16) of S^T resp. dP^T, which the other warpgroup never reads
    const uint32_t col_ld = wg * 32, col_st = wg * 48;
    int qi = 0;  // query tile index of the current step inside its stream
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int set = it & 1;
      const uint32_t tm = tmem_base + set * 128;
      ok = mbar_wait(&st_full[set], (it >> 1) & 1, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      uint32_t st[32], dp[32];
      tmem_ld_x32(tm + lane_sel + col_ld, st);
      tmem_ld_x32(tm + 64 + lane_sel + col_ld, dp);
      // issued here, so that the load has returned before the fences below (which wait for it)
      bool v_new;
      const float s_new = fetch(v_new);
      const bool diag = p.causal && qi < BT / BQ2;                  // the first two query tiles straddle the diagonal
      const int first_visible = diag ? r - qi * BQ2 - wg * 32 : 0;  // own columns below this are masked for this key row
      uint32_t pk[16], dk[16];
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const uint64_t x = fmul2(pack_f2(__uint_as_float(st[2 * i]), __uint_as_float(st[2 * i + 1])), c2);
        float e0 = fast_exp2(f2_lo(x)), e1 = fast_exp2(f2_hi(x));
        if (diag) {
          e0 = 2 * i < first_visible ? 0.f : e0;
          e1 = 2 * i + 1 < first_visible ? 0.f : e1;
        }
        pk[i] = pack_bf16(e0, e1);
        const uint64_t d = fmul2(pack_f2(e0, e1), pack_f2(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])));
        dk[i] = pack_bf16(f2_lo(d), f2_hi(d));
      }
      // keys beyond the sequence contribute nothing (their K/V rows are zero-filled; dK/dV rows are not stored)
      tmem_st_x16(tm + lane_sel + col_st, pk);
      tmem_st_x16(tm + 64 + lane_sel + col_st, dk);
      tmem_st_wait();
      fence_proxy_async_smem();  // the statistics staged one step ago are read by the tensor core's proxy
      tc_fence_before_sync();
      mbar_arrive(&pds_ready[set]);
      // Off the critical path: the tile of step it+3 (last read by the scores of step it-1, which have
      // completed).  The next step's arrive publishes it, before the scores of step it+3 are issued.
      stage((it + 3) & 3, s0, v0);
      s0 = s1;
      v0 = v1;
      s1 = s_new;
      v1 = v_new;
      if (++qi == per_stream) qi = 0;
    }
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      bool w = mbar_wait(acc_done, 0, err);
      ok = __all_sync(0xffffffffu, w);
    }
    if (ok) {
      tc_fence_after_sync();
      // warpgroup 0 writes dK (scaled), warpgroup 1 writes dV; every lane loads, valid rows store
      const bool valid = kv_row < p.S;
      const size_t row_off = ((size_t(b) * p.S + (valid ? kv_row : 0)) * p.Hkv + hk) * DH;
      float* dst = (wg == 0 ? p.dk_sum : p.dv_sum) + row_off;
      const uint32_t src = (wg == 0 ? tm_dk : tm_dv) + lane_sel;
      const float mul = wg == 0 ? p.scale : 1.f;
#pragma unroll 1
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t a[32];
        tmem_ld_x32(src + c * 32, a);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int v4 = 0; v4 < 8; ++v4)
            *reinterpret_cast<float4*>(dst + c * 32 + v4 * 4) =
                make_float4(__uint_as_float(a[4 * v4]) * mul, __uint_as_float(a[4 * v4 + 1]) * mul,
                            __uint_as_float(a[4 * v4 + 2]) * mul, __uint_as_float(a[4 * v4 + 3]) * mul);
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// =============================================================================================
// dQ
// =============================================================================================
constexpr int DQ_THREADS = 320;  // warp 0 TMA, warp 1 MMA, warps 2-5 query tile A, warps 6-9 query tile B
constexpr int DQ_KSTAGES = 2;

template <int DH>
struct DqSmem {
  static constexpr int TILE = BT * DH * 2;
  static constexpr int OFF_Q = 0;                          // [2] query tiles A, B
  static constexpr int OFF_DO = OFF_Q + 2 * TILE;          // [2]
  static constexpr int OFF_K = OFF_DO + 2 * TILE;          // [DQ_KSTAGES]
  static constexpr int OFF_V = OFF_K + DQ_KSTAGES * TILE;  // one stage: V_j is only read by the two dP products
  static constexpr int OFF_BAR = OFF_V + TILE;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;
};

struct DqParams {
  CUtensorMap map_q, map_do, map_k, map_v;  // box rows 128
  const float* lse;                         // [B,Hq,S]
  const float* delta;                       // [B,Hq,S]
  __nv_bfloat16* dq;                        // [B,S,Hq,dh]
  int B, S, Hq, Hkv;
  int causal;
  float scale;
  float scale_log2;
};

// Two adjacent query tiles (A, B) share every K/V tile the CTA fetches.  Each query tile owns one
// 128-column TMEM buffer that is reused through a key tile's life -- S (fp32) -> read by the tile's
// warpgroup -> dP (fp32, same columns) -> read -> dS (bf16 pairs, first 64 columns) -> A operand of
// dQ += dS K -- plus a DH-column dQ accumulator.  While one tile's exponentials run, the tensor pipe
// works on the other tile.
template <int DH>
__global__ void __launch_bounds__(DQ_THREADS, 1) dq_kernel(const __grid_constant__ DqParams p) {
  using L = DqSmem<DH>;
  constexpr int HALVES = DH / 64;
  constexpr int KSTEPS_DH = DH / 16;
  constexpr int KSTEPS_KV = BT / 16;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* qdo_full = bars + 0;
  uint64_t* k_full = bars + 1;                 // [KSTAGES]
  uint64_t* k_empty = k_full + DQ_KSTAGES;     // [KSTAGES]
  uint64_t* v_full = k_empty + DQ_KSTAGES;
  uint64_t* v_empty = v_full + 1;
  uint64_t* s_full = v_empty + 1;              // [2] per query tile
  uint64_t* s_read = s_full + 2;               // [2] S of the tile is in registers (128 arrivals)
  uint64_t* dp_full = s_read + 2;              // [2]
  uint64_t* ds_ready = dp_full + 2;            // [2] dS of the tile written (128 arrivals)
  uint64_t* dq_done = ds_ready + 2;            // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dq_done + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_bwd_status;

  const int hq = blockIdx.x % p.Hq;
  const int b = blockIdx.x / p.Hq;
  const int n_qtiles = (p.S + BT - 1) / BT;
  const int n_pairs = (n_qtiles + 1) / 2;
  const int pair = n_pairs - 1 - blockIdx.y;  // heaviest pairs first
  const int hk = hq / (p.Hq / p.Hkv);
  const int q0 = pair * 2 * BT;
  int n_kv[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    const int qs = q0 + x * BT;
    const int kv_end = p.causal ? min(p.S, qs + BT) : p.S;
    n_kv[x] = qs < p.S ? (kv_end + BT - 1) / BT : 0;
  }
  const int n_max = max(n_kv[0], n_kv[1]);

  if (threadIdx.x == 0) {
    mbar_init(qdo_full, 1);
    for (int i = 0; i < DQ_KSTAGES; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], 1);
    }
    mbar_init(v_full, 1);
    mbar_init(v_empty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&s_read[i], 128);
      mbar_init(&dp_full[i], 1);
      mbar_init(&ds_ready[i], 128);
      mbar_init(&dq_done[i], 1);
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
  // query tile x: working buffer at [x*128, x*128+128), dQ accumulator at [256 + x*128, ...)

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      if (leader) tma_prefetch_desc(&p.map_q);
      if (leader) tma_prefetch_desc(&p.map_do);
      if (leader) tma_prefetch_desc(&p.map_k);
      if (leader) tma_prefetch_desc(&p.map_v);
      mbar_expect_tx_e(qdo_full, 4 * L::TILE, leader);  // rows beyond the sequence are zero-filled
#pragma unroll
      for (int x = 0; x < 2; ++x)
#pragma unroll
        for (int h = 0; h < HALVES; ++h) {
          tma_load_4d_e(smem + L::OFF_Q + x * L::TILE + h * HALF_BYTES, &p.map_q, qdo_full, h * 64, hq, q0 + x * BT, b, leader);
          tma_load_4d_e(smem + L::OFF_DO + x * L::TILE + h * HALF_BYTES, &p.map_do, qdo_full, h * 64, hq, q0 + x * BT, b, leader);
        }
      auto load_k = [&](int j) -> bool {
        const int s = j % DQ_KSTAGES;
        if (!mbar_wait(&k_empty[s], ((j / DQ_KSTAGES) & 1) ^ 1, err)) return false;
        mbar_expect_tx_e(&k_full[s], L::TILE, leader);
#pragma unroll
        for (int h = 0; h < HALVES; ++h)
          tma_load_4d_e(smem + L::OFF_K + s * L::TILE + h * HALF_BYTES, &p.map_k, &k_full[s], h * 64, hk, j * BT, b, leader);
        return true;
      };
      auto load_v = [&](int j) -> bool {
        if (!mbar_wait(v_empty, (j & 1) ^ 1, err)) return false;
        mbar_expect_tx_e(v_full, L::TILE, leader);
#pragma unroll
        for (int h = 0; h < HALVES; ++h)
          tma_load_4d_e(smem + L::OFF_V + h * HALF_BYTES, &p.map_v, v_full, h * 64, hk, j * BT, b, leader);
        return true;
      };
      bool ok = n_max > 0 ? load_k(0) : true;
      for (int j = 0; j < n_max && ok; ++j) {
        ok = load_v(j);
        if (ok && j + 1 < n_max) ok = load_k(j + 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      constexpr uint32_t idesc_s = umma_idesc_bf16(BT, BT, 0, 0);
      constexpr uint32_t idesc_dq = umma_idesc_bf16(BT, DH, 0, 1);  // A = dS from TMEM, B = K MN-major
      constexpr uint32_t hi = desc_hi_sw128(1024);
      const uint32_t k_base = smem_u32(smem + L::OFF_K);
      const uint32_t v_lo = desc_lo_sw128(smem_u32(smem + L::OFF_V), 0);
      bool ok = mbar_wait(qdo_full, 0, err);
      auto issue_s = [&](int x, int j) {  // S_x(j) = Q_x K_j^T
        const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::OFF_Q + x * L::TILE), 0);
        const uint32_t k_lo = desc_lo_sw128(k_base + (j % DQ_KSTAGES) * L::TILE, 0);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          umma_ss_w(tmem_base + x * BT, desc_lo_add(q_lo, off), desc_lo_add(k_lo, off), hi, idesc_s, ks != 0, leader);
        }
        umma_commit(&s_full[x], leader);
      };
      if (ok && n_max > 0) {
        ok = mbar_wait(&k_full[0], 0, err);
        if (ok) {
          tc_fence_after_sync();
          if (n_kv[0] > 0) issue_s(0, 0);
          if (n_kv[1] > 0) issue_s(1, 0);
        }
      }
      for (int j = 0; j < n_max && ok; ++j) {
        const uint32_t ph = j & 1;
        if (!mbar_wait(v_full, ph, err)) { ok = false; break; }
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (j < n_kv[x]) {
            // dP_x(j) overwrites S_x(j) once the warpgroup holds S_x(j) in registers
            if (!mbar_wait(&s_read[x], ph, err)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t do_lo = desc_lo_sw128(smem_u32(smem + L::OFF_DO + x * L::TILE), 0);
#pragma unroll
            for (int ks = 0; ks < KSTEPS_DH; ++ks) {
              const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
              umma_ss_w(tmem_base + x * BT, desc_lo_add(do_lo, off), desc_lo_add(v_lo, off), hi, idesc_s, ks != 0, leader);
            }
            umma_commit(&dp_full[x], leader);
          }
        }
        if (!ok) break;
        umma_commit(v_empty, leader);
        const bool next = j + 1 < n_max;
        if (next && !mbar_wait(&k_full[(j + 1) % DQ_KSTAGES], ((j + 1) / DQ_KSTAGES) & 1, err)) { ok = false; break; }
        const uint32_t kmn_lo = desc_lo_sw128(k_base + (j % DQ_KSTAGES) * L::TILE, HALF_BYTES);  // K_j as MN-major B
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (j < n_kv[x]) {
            if (!mbar_wait(&ds_ready[x], ph, err)) { ok = false; break; }
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < KSTEPS_KV; ++ks)  // dQ_x += dS_x(j) K_j
              umma_ts_w(tmem_base + 256 + x * 128, tmem_base + x * BT + ks * 8, desc_lo_add(kmn_lo, ks * 2048), hi,
                        idesc_dq, (j | ks) != 0, leader);
            if (j + 1 == n_kv[x]) umma_commit(&dq_done[x], leader);
            // the tile's buffer takes the next scores right behind dQ_x(j) in the in-order tensor pipe
            if (j + 1 < n_kv[x]) issue_s(x, j + 1);
          }
        }
        if (!ok) break;
        umma_commit(&k_empty[j % DQ_KSTAGES], leader);
      }
    }
  } else {
    // ------------------------------ compute warpgroups ------------------------------
    const int x = (warp - 2) >> 2;      // query tile of this warpgroup
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;  // query row inside the tile == TMEM lane
    const int q_row = q0 + x * BT + r;
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    const uint32_t tb = tmem_base + x * BT + lane_sel;
    const int my_n = n_kv[x];
    const size_t stat_idx = (size_t(b) * p.Hq + hq) * p.S + (q_row < p.S ? q_row : 0);
    const float lse2 = q_row < p.S ? p.lse[stat_idx] * 1.4426950408889634f : INFINITY;
    const float dl = q_row < p.S ? p.delta[stat_idx] : 0.f;
    const uint64_t c2 = pack_f2(p.scale_log2, p.scale_log2);
    const uint64_t nl2 = pack_f2(-lse2, -lse2);
    const uint64_t ndl2 = pack_f2(-dl, -dl);
    bool ok = true;
    for (int j = 0; j < my_n; ++j) {
      const uint32_t ph = j & 1;
      ok = mbar_wait(&s_full[x], ph, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      const int kvb = j * BT;
      int lim = p.S - kvb;
      if (p.causal) lim = min(lim, q_row - kvb + 1);
      uint32_t pb[BT / 2];  // P as bf16 pairs, kept across the dP product
      {
        uint32_t t0[32], t1[32], t2[32], t3[32];
        tmem_ld_x32(tb, t0);
        tmem_ld_x32(tb + 32, t1);
        tmem_ld_x32(tb + 64, t2);
        tmem_ld_x32(tb + 96, t3);
        tmem_ld_wait();
        tc_fence_before_sync();
        mbar_arrive(&s_read[x]);  // the scores are in registers: dP may overwrite them
        auto expo = [&](const uint32_t* t, uint32_t* out) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint64_t v = ffma2(pack_f2(__uint_as_float(t[2 * i]), __uint_as_float(t[2 * i + 1])), c2, nl2);
            out[i] = pack_bf16(fast_exp2(f2_lo(v)), fast_exp2(f2_hi(v)));
          }
        };
        expo(t0, pb);
        expo(t1, pb + 16);
        expo(t2, pb + 32);
        expo(t3, pb + 48);
      }
      if (__any_sync(0xffffffffu, lim < BT)) {  // diagonal or ragged tile: zero the masked columns
#pragma unroll
        for (int i = 0; i < BT / 2; ++i) {
          uint32_t v = pb[i];
          if (2 * i >= lim) v &= 0xffff0000u;
          if (2 * i + 1 >= lim) v &= 0x0000ffffu;
          pb[i] = v;
        }
      }
      ok = mbar_wait(&dp_full[x], ph, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
#pragma unroll
      for (int c = 0; c < BT / 32; ++c) {
        uint32_t tmp[32];
        tmem_ld_x32(tb + c * 32, tmp);
        tmem_ld_wait();
        uint32_t ds[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint32_t pv = pb[c * 16 + i];
          const uint64_t pf = pack_f2(__uint_as_float(pv << 16), __uint_as_float(pv & 0xffff0000u));
          const uint64_t d = fmul2(pf, fadd2(pack_f2(__uint_as_float(tmp[2 * i]), __uint_as_float(tmp[2 * i + 1])), ndl2));
          ds[i] = pack_bf16(f2_lo(d), f2_hi(d));
        }
        // dS (bf16 pairs) over dP's own columns: chunk c lands in columns [16c, 16c+16), already read
        tmem_st_x16(tb + c * 16, ds);
      }
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&ds_ready[x]);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (ok && my_n > 0) {
      bool w = mbar_wait(&dq_done[x], 0, err);
      ok = __all_sync(0xffffffffu, w);
    }
    if (ok && my_n > 0) {
      tc_fence_after_sync();
      const bool valid = q_row < p.S;
      __nv_bfloat16* dst = p.dq + ((size_t(b) * p.S + (valid ? q_row : 0)) * p.Hq + hq) * DH;
      const uint32_t src = tmem_base + 256 + x * 128 + lane_sel;
#pragma unroll 1
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t a[32];
        tmem_ld_x32(src + c * 32, a);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(a[8 * v4 + 0]) * p.scale, __uint_as_float(a[8 * v4 + 1]) * p.scale);
            v.y = pack_bf16(__uint_as_float(a[8 * v4 + 2]) * p.scale, __uint_as_float(a[8 * v4 + 3]) * p.scale);
            v.z = pack_bf16(__uint_as_float(a[8 * v4 + 4]) * p.scale, __uint_as_float(a[8 * v4 + 5]) * p.scale);
            v.w = pack_bf16(__uint_as_float(a[8 * v4 + 6]) * p.scale, __uint_as_float(a[8 * v4 + 7]) * p.scale);
            *reinterpret_cast<uint4*>(dst + c * 32 + v4 * 8) = v;
          }
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// Delta[b,hq,s] = sum_c dO[b,s,hq,c] * O[b,s,hq,c].  A row of DH bf16 is DH/8 16-byte pieces: each warp takes
// 256/DH rows at a time (one piece per lane, every lane busy), two such groups per iteration so that four
// loads per lane are in flight, and reduces inside the DH/8-lane segments.
template <int DH>
__global__ void delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                             float* __restrict__ delta, int B, int S, int Hq) {
  constexpr int LANES = DH / 8;          // lanes per row
  constexpr int ROWS = 32 / LANES;       // rows per warp and load
  const size_t rows = size_t(B) * S * Hq;
  const int lane = threadIdx.x & 31;
  const int sub = lane / LANES, piece = lane % LANES;
  const size_t warp_global = (size_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const size_t n_warps = (size_t(gridDim.x) * blockDim.x) >> 5;
  auto dot8 = [](const uint4& a, const uint4& g) {
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 fa = __bfloat1622float2(pa[i]), fg = __bfloat1622float2(pg[i]);
      acc += fa.x * fg.x + fa.y * fg.y;
    }
    return acc;
  };
  for (size_t base = warp_global * (2 * ROWS); base < rows; base += n_warps * (2 * ROWS)) {
    const size_t r0 = base + sub, r1 = base + ROWS + sub;
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    const uint4 a0 = r0 < rows ? *reinterpret_cast<const uint4*>(o + r0 * DH + piece * 8) : z;
    const uint4 g0 = r0 < rows ? *reinterpret_cast<const uint4*>(d_o + r0 * DH + piece * 8) : z;
    const uint4 a1 = r1 < rows ? *reinterpret_cast<const uint4*>(o + r1 * DH + piece * 8) : z;
    const uint4 g1 = r1 < rows ? *reinterpret_cast<const uint4*>(d_o + r1 * DH + piece * 8) : z;
    float acc0 = dot8(a0, g0), acc1 = dot8(a1, g1);
#pragma unroll
    for (int sft = LANES / 2; sft > 0; sft >>= 1) {
      acc0 += __shfl_xor_sync(0xffffffffu, acc0, sft);
      acc1 += __shfl_xor_sync(0xffffffffu, acc1, sft);
    }
    if (piece == 0) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const size_t row = u == 0 ? r0 : r1;
        if (row < rows) {
          const int hq = int(row % Hq);
          const size_t tok = row / Hq;
          const int sx = int(tok % S);
          const int bx = int(tok / S);
          delta[(size_t(bx) * Hq + hq) * S + sx] = u == 0 ? acc0 : acc1;
        }
      }
    }
  }
}

int make_map_bshd(CUtensorMap* m, const void* base, int B, int S, int H, int dh, int rows) {
  uint64_t dims[4] = {uint64_t(dh), uint64_t(H), uint64_t(S), uint64_t(B)};
  uint64_t strides[3] = {uint64_t(dh) * 2, uint64_t(H) * dh * 2, uint64_t(S) * H * dh * 2};
  uint32_t box[4] = {64, 1, uint32_t(rows), 1};
  return make_tensor_map(m, base, 2, 4, dims, strides, box, true);
}

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace

int attn_bwd_read_status() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_bwd_status, sizeof(int)) != cudaSuccess) return -1;
  if (v != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_bwd_status, &zero, sizeof(int));
  }
  return v;
}

// Workspace: Delta [B,Hq,S] fp32 for every layer.
size_t attn_bwd_workspace(const kvp_shape* s, const int32_t* donor) {
  (void)donor;
  return size_t(s->L) * align256(size_t(s->B) * s->Hq * s->S * 4);
}

int attn_bwd_all(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                 const void* const* k, const void* const* v, const void* const* o, const void* const* d_o,
                 const float* const* lse, void* const* dq, float* const* dk_sum, float* const* dv_sum, void* ws,
                 size_t ws_bytes, cudaStream_t stream) {
  (void)ws_bytes;
  const int dh = s->dh;
  const float sc = scale == 0.f ? 1.f / sqrtf(float(dh)) : scale;
  const size_t delta_bytes = align256(size_t(s->B) * s->Hq * s->S * 4);
  uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);
  cudaError_t e1, e2;
  if (dh == 128) {
    e1 = cudaFuncSetAttribute(dkdv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DkdvSmem<128>::TOTAL);
    e2 = cudaFuncSetAttribute(dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<128>::TOTAL);
  } else {
    e1 = cudaFuncSetAttribute(dkdv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DkdvSmem<64>::TOTAL);
    e2 = cudaFuncSetAttribute(dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<64>::TOTAL);
  }
  if (e1 != cudaSuccess || e2 != cudaSuccess) return KVP_ERR_CUDA;

  // Delta for every layer
  for (int l = 0; l < s->L; ++l) {
    float* dl = reinterpret_cast<float*>(wsb + size_t(l) * delta_bytes);
    const size_t rows = size_t(s->B) * s->S * s->Hq;
    const int blocks = int(min(size_t(sm_count()) * 16, (rows + 7) / 8));
    if (dh == 128)
      delta_kernel<128><<<blocks, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(o[l]),
                                                    reinterpret_cast<const __nv_bfloat16*>(d_o[l]), dl, s->B, s->S,
                                                    s->Hq);
    else
      delta_kernel<64><<<blocks, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(o[l]),
                                                   reinterpret_cast<const __nv_bfloat16*>(d_o[l]), dl, s->B, s->S,
                                                   s->Hq);
    note_launch();
  }
  if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;

  // dQ, one launch per layer
  for (int l = 0; l < s->L; ++l) {
    const int d = donor[l];
    DqParams p;
    int rc = make_map_bshd(&p.map_q, q[l], s->B, s->S, s->Hq, dh, BT);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_do, d_o[l], s->B, s->S, s->Hq, dh, BT);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_k, k[d], s->B, s->S, s->Hkv, dh, BT);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_v, v[d], s->B, s->S, s->Hkv, dh, BT);
    if (rc != KVP_OK) return rc;
    p.lse = lse[l];
    p.delta = reinterpret_cast<const float*>(wsb + size_t(l) * delta_bytes);
    p.dq = reinterpret_cast<__nv_bfloat16*>(dq[l]);
    p.B = s->B;
    p.S = s->S;
    p.Hq = s->Hq;
    p.Hkv = s->Hkv;
    p.causal = causal;
    p.scale = sc;
    p.scale_log2 = sc * 1.4426950408889634f;
    dim3 grid(s->B * s->Hq, ((s->S + BT - 1) / BT + 1) / 2);
    timing_before(KVP_KERNEL_ATTN_BWD_DQ, stream);
    if (dh == 128)
      dq_kernel<128><<<grid, DQ_THREADS, DqSmem<128>::TOTAL, stream>>>(p);
    else
      dq_kernel<64><<<grid, DQ_THREADS, DqSmem<64>::TOTAL, stream>>>(p);
    timing_after(KVP_KERNEL_ATTN_BWD_DQ, stream);
    note_launch();
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
  }

  // dK / dV, one launch per donor group.  A launch writes (does not add to) the accumulators, so a
  // donor shared by more than MAX_GROUP layers is not supported.
  for (int d = 0; d < s->L; ++d) {
    if (donor[d] != d) continue;
    int members[MAX_GROUP];
    int n = 0;
    for (int l = d; l < s->L; ++l)
      if (donor[l] == d) {
        if (n == MAX_GROUP) return KVP_ERR_UNSUPPORTED;
        members[n++] = l;
      }
    DkdvParams p;
    int rc = make_map_bshd(&p.map_k, k[d], s->B, s->S, s->Hkv, dh, BT);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_v, v[d], s->B, s->S, s->Hkv, dh, BT);
    if (rc != KVP_OK) return rc;
    for (int i = 0; i < MAX_GROUP; ++i) {
      const int l = members[i < n ? i : 0];
      rc = make_map_bshd(&p.map_q[i], q[l], s->B, s->S, s->Hq, dh, BQ2);
      if (rc == KVP_OK) rc = make_map_bshd(&p.map_do[i], d_o[l], s->B, s->S, s->Hq, dh, BQ2);
      if (rc != KVP_OK) return rc;
      p.lse[i] = lse[l];
      p.delta[i] = reinterpret_cast<const float*>(wsb + size_t(l) * delta_bytes);
    }
    p.dk_sum = dk_sum[d];
    p.dv_sum = dv_sum[d];
    p.n_layers = n;
    p.B = s->B;
    p.S = s->S;
    p.Hq = s->Hq;
    p.Hkv = s->Hkv;
    p.causal = causal;
    p.scale = sc;
    p.scale_log2 = sc * 1.4426950408889634f;
    // chunk: the smallest divisor of the pair count that still fills the SMs 1.5 times with CTAs
    const int n_jt = (s->S + BT - 1) / BT, n_pairs = s->Hkv * s->B;
    p.chunk = n_pairs;
    for (int d = 1; d <= n_pairs; ++d)
      if (n_pairs % d == 0 && 2 * d * n_jt >= 3 * sm_count()) {
        p.chunk = d;
        break;
      }
    dim3 grid(n_pairs * n_jt);
    timing_before(KVP_KERNEL_ATTN_BWD, stream);
    if (dh == 128)
      dkdv_kernel<128><<<grid, DKDV_THREADS, DkdvSmem<128>::TOTAL, stream>>>(p);
    else
      dkdv_kernel<64><<<grid, DKDV_THREADS, DkdvSmem<64>::TOTAL, stream>>>(p);
    timing_after(KVP_KERNEL_ATTN_BWD, stream);
    note_launch();
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
  }
  return KVP_OK;
}

}  // namespace kvp
