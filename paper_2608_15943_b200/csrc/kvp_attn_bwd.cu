// Flash-attention backward over a donor map (chain rule of Eq. 2-3 of the paper) in ONE pass.
//
//  bwd_kernel   KV-stationary.  One CTA owns a 128-row K/V tile of one (batch, KV head) of a DONOR
//               layer, keeps K and V in shared memory and the dK / dV accumulators in TMEM (fp32)
//               while it walks every query stream that reads the tile: the donor itself and all its
//               consumer layers, the Hq/Hkv query heads of the KV head's group, and every 64-row query
//               tile the causal mask lets see the keys.  dK and dV of the donor are therefore summed on
//               chip across layers and heads and written to HBM once.  Per step, transposed so that TMEM
//               lane == key row:  S^T = K Q^T, dP^T = V dO^T (tcgen05, operands in shared memory), each
//               followed by one rank-3 MMA that subtracts the query's LSE/scale resp. Delta (a bf16
//               three-term split against a tile of ones), so the accumulators already hold the
//               exponent and dP - Delta; P^T = exp2(c acc), dS^T = P^T acc' are written back as bf16
//               over the score columns and fed to dV += P^T dO, dK += dS^T Q as the A operand FROM
//               TMEM.  dS^T also goes to shared memory, where it is the B operand of the fifth product
//               dQ^T = K^T dS^T (K read as an MN-major A operand): the step's [dh x 64] partial of dQ
//               lands in TMEM, a third warpgroup moves it to shared memory and adds it to an fp32
//               accumulator in global memory with bulk reductions (cp.reduce.async.bulk .add.f32, 2 KB
//               each), so S and dP are computed once for all three gradients.
//
//  dq_convert_kernel  scales the fp32 dQ accumulators and writes dQ as bf16 [B,S,Hq,dh].
//
// Delta = rowsum(dO * O) comes from a small pre-pass.  The dQ accumulators live in the caller's
// workspace in a blocked layout ([b][hq][64-query tile][32-column quarter][64][32] fp32) so that every
// reduction is one contiguous 2 KB run; they are cleared before each donor group's launch.  The order in
// which the key tiles' partials reach an accumulator is not fixed, so dQ (unlike dK, dV) is reproducible
// only up to fp32 rounding order.
#include <math.h>

#include <algorithm>
#include <vector>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int BT = 128;    // key rows per tile
constexpr int BQ2 = 64;    // query rows per step
constexpr int MAX_GROUP = 8;  // layers of one donor group per launch
constexpr uint32_t HALF_BYTES = 128 * 128;  // [128 rows x 128 B] block
constexpr uint32_t QHALF_BYTES = 64 * 128;  // [ 64 rows x 128 B] block

__device__ int g_bwd_status;

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// warp 0 TMA, warp 1 MMA, warps 2-5 and 6-9 two compute warpgroups, warps 10-13 dQ drain
constexpr int BWD_THREADS = 448;
constexpr int BWD_STAGES = 3;        // ring of (Q, dO) 64-row tiles
constexpr int DQ_STAGE_BYTES = BQ2 * 32 * 4;  // one drain warp's share of a step: [64 queries x 32 columns] fp32
// A CTA's window of query tiles is sized so that it runs about this many steps (window x streams): long enough
// to amortise its prologue and its dK / dV reduction, short enough that a wave's footprint stays in L2.
constexpr int kStepsPerCta = 256;
constexpr int kMinWindow = 16;

template <int DH>
struct BwdSmem {
  static constexpr int KV_TILE = BT * DH * 2;
  static constexpr int Q_TILE = BQ2 * DH * 2;
  static constexpr int STAGE = 2 * Q_TILE;  // Q then dO
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = OFF_K + KV_TILE;
  static constexpr int OFF_RING = OFF_V + KV_TILE;
  static constexpr int OFF_DS = OFF_RING + BWD_STAGES * STAGE;     // dS^T [128 keys x 64 queries] bf16, 128-B swizzle
  static constexpr int OFF_DQ = OFF_DS + BT * BQ2 * 2;             // [4 drain warps][64 x 32] fp32
  static constexpr int OFF_ONES = OFF_DQ + 4 * DQ_STAGE_BYTES;     // [128 x 8] bf16: columns 0-7 of the tile of ones
  static constexpr int OFF_STAT = OFF_ONES + 2048;                 // [4 steps][lse, delta][64 x 8] bf16: columns 0-7
  static constexpr int OFF_ZERO = OFF_STAT + 8 * 1024;             // [128 x 8] zeros: columns 8-15 of all of the above
  static constexpr int OFF_RAW = OFF_ZERO + 2048;                  // [8 steps][lse, delta][64] fp32 as loaded
  static constexpr int OFF_BAR = OFF_RAW + 4096;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;
};

// One launch serves several donor groups (up to MAX_GROUP member layers in all): slot i of the per-layer arrays is
// the i-th member layer, group g owns slots [first_slot[g], first_slot[g + 1]) and blocks [cta_begin[g],
// cta_begin[g + 1]).  Groups are sorted by size, largest first, so that only the last, shortest CTAs of the whole
// backward pass run on a partly idle device.
struct BwdParams {
  CUtensorMap map_k[MAX_GROUP], map_v[MAX_GROUP];   // per group: donor K, V [B,S,Hkv,dh], box rows 128
  CUtensorMap map_q[MAX_GROUP], map_do[MAX_GROUP];  // per member layer, box rows 64
  const float* lse[MAX_GROUP];    // [B,Hq,S]
  const float* delta[MAX_GROUP];  // [B,Hq,S]
  float* dq_acc[MAX_GROUP];       // blocked fp32 accumulators, see dq_acc_floats()
  float* dk_sum[MAX_GROUP];       // per group: fp32 [B,S,Hkv,dh]
  float* dv_sum[MAX_GROUP];
  int first_slot[MAX_GROUP + 1];
  int cta_begin[MAX_GROUP + 1];
  int window[MAX_GROUP];          // query tiles per CTA
  int ctas_per_pair[MAX_GROUP];   // CTAs of one (batch, KV head): sum over windows of the key tiles that see the window
  int n_groups;
  int B, S, Hq, Hkv;
  int causal;
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

// Floats of one layer's dQ accumulator: [B][Hq][ceil(S/64)][DH/32][64][32].
__host__ __device__ inline size_t dq_acc_floats(int B, int S, int Hq, int dh) {
  return size_t(B) * Hq * ((S + BQ2 - 1) / BQ2) * BQ2 * dh;
}

// TMEM columns: S^T of step parity i at [i*64, i*64+64) (P^T and dS^T overwrite it as bf16), dP^T at
// [128, 192), the step's dQ^T at [192, 256), dK at [256, 256+DH), dV above it.
//
// The per-query statistics are applied BY THE TENSOR CORE: one extra K-step multiplies a [128 x 16] tile
// of ones (first three columns) with a [64 x 16] tile holding -LSE/scale (resp. -Delta) of each query
// split into three bf16 terms, so the accumulators already hold S - LSE/scale and dP - Delta and the
// threads need no per-column operand: P^T = exp2(c * acc), dS^T = P^T * acc'.
template <int DH>
__global__ void __launch_bounds__(BWD_THREADS, 1) bwd_kernel(const __grid_constant__ BwdParams p) {
  using L = BwdSmem<DH>;
  constexpr int HALVES = DH / 64;
  constexpr int KSTEPS_DH = DH / 16;
  constexpr int KSTEPS_Q = BQ2 / 16;
  constexpr int KSTEPS_KV = BT / 16;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* kv_full = bars + 0;
  uint64_t* q_full = bars + 1;                    // [STAGES]
  uint64_t* q_empty = q_full + BWD_STAGES;        // [STAGES]
  uint64_t* st_full = q_empty + BWD_STAGES;       // S^T and dP^T of the step are in TMEM
  uint64_t* dp_free = st_full + 1;                // dP^T of the step is in registers (256 arrivals)
  uint64_t* pds_ready = dp_free + 1;              // [2] P^T, dS^T written (TMEM and shared memory), next statistics staged
  uint64_t* dq_full = pds_ready + 2;              // dQ^T of the step is in TMEM; its dS^T tile may be overwritten
  uint64_t* dq_free = dq_full + 1;                // dQ^T of the step is in registers, statistics of step +3 staged (128 arrivals)
  uint64_t* stat0 = dq_free + 1;                  // statistics of the first steps staged (128 arrivals)
  uint64_t* acc_done = stat0 + 1;                 // all MMAs have completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_done + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_bwd_status;

  // Work decomposition.  A CTA is one donor group, one (batch, KV head), one 128-row key tile and one WINDOW of
  // consecutive 64-row query tiles, for every query stream of the donor group.  All CTAs therefore take
  // (nearly) the same number of steps per stream and walk the streams at the same pace, so the CTAs that
  // run at the same time read the same few Q / dO tiles and add to the same few dQ accumulator tiles:
  // what a wave touches over its lifetime stays in L2.  Blocks are dispatched in index order: (batch, KV
  // head) slowest, then the window, then the key tiles that see it.  The windows of one key tile add their
  // dK / dV partials to the (cleared) output with reductions.
  const int n_jt = (p.S + BT - 1) / BT;
  const int n_qt = (p.S + BQ2 - 1) / BQ2;
  int grp = 0;
  while (grp + 1 < p.n_groups && int(blockIdx.x) >= p.cta_begin[grp + 1]) ++grp;
  const int slot0 = p.first_slot[grp];
  const int n_layers = p.first_slot[grp + 1] - slot0;
  const int window = p.window[grp];
  const int in_group = blockIdx.x - p.cta_begin[grp];
  const int pair = in_group / p.ctas_per_pair[grp];
  int jt = in_group - pair * p.ctas_per_pair[grp];
  int win = 0;
  for (;; ++win) {
    const int vis = p.causal ? min(n_jt, ((win + 1) * window * BQ2 + BT - 1) / BT) : n_jt;
    if (jt < vis) break;
    jt -= vis;
  }
  const int hk = pair % p.Hkv;
  const int b = pair / p.Hkv;
  const int G = p.Hq / p.Hkv;
  const int kv0 = jt * BT;
  const int qt_first = max(p.causal ? (kv0 / BQ2) : 0, win * window);
  const int per_stream = min(n_qt, (win + 1) * window) - qt_first;
  const int n_iter = n_layers * G * per_stream;

  if (threadIdx.x == 0) {
    mbar_init(kv_full, 1);
    for (int s = 0; s < BWD_STAGES; ++s) {
      mbar_init(&q_full[s], 1);
      mbar_init(&q_empty[s], 1);
    }
    mbar_init(st_full, 1);
    mbar_init(dp_free, 256);
    for (int i = 0; i < 2; ++i) mbar_init(&pds_ready[i], 256);
    mbar_init(dq_full, 1);
    mbar_init(dq_free, 128);
    mbar_init(stat0, 128);
    mbar_init(acc_done, 1);
    mbar_fence_init();
  }
  // constant operand tiles: ones in the first three columns; statistics tiles and the shared zero half start as zeros
  for (int i = threadIdx.x; i < (L::OFF_RAW - L::OFF_ONES) / 16; i += blockDim.x) {
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
  const uint32_t tm_dp = tmem_base + 128;
  const uint32_t tm_dq = tmem_base + 192;
  const uint32_t tm_dk = tmem_base + 256;
  const uint32_t tm_dv = tmem_base + 256 + DH;

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
      if (leader) tma_prefetch_desc(&p.map_k[grp]);
      if (leader) tma_prefetch_desc(&p.map_v[grp]);
      mbar_expect_tx_e(kv_full, 2 * L::KV_TILE, leader);
#pragma unroll
      for (int h = 0; h < HALVES; ++h) {
        tma_load_4d_e(smem + L::OFF_K + h * HALF_BYTES, &p.map_k[grp], kv_full, h * 64, hk, kv0, b, leader);
        tma_load_4d_e(smem + L::OFF_V + h * HALF_BYTES, &p.map_v[grp], kv_full, h * 64, hk, kv0, b, leader);
      }
      for (int it = 0; it < n_iter; ++it) {
        int li, hq, q0;
        decode_iter(it, li, hq, q0);
        const int s = it % BWD_STAGES;
        const uint32_t ph = (it / BWD_STAGES) & 1;
        if (!mbar_wait(&q_empty[s], ph ^ 1, err)) break;
        mbar_expect_tx_e(&q_full[s], L::STAGE, leader);
        uint8_t* dst = smem + L::OFF_RING + s * L::STAGE;
#pragma unroll
        for (int h = 0; h < HALVES; ++h) {
          tma_load_4d_e(dst + h * QHALF_BYTES, &p.map_q[slot0 + li], &q_full[s], h * 64, hq, q0, b, leader);
          tma_load_4d_e(dst + L::Q_TILE + h * QHALF_BYTES, &p.map_do[slot0 + li], &q_full[s], h * 64, hq, q0, b, leader);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      constexpr uint32_t idesc_st = umma_idesc_bf16(BT, BQ2, 0, 0);   // [128 keys x 64 queries]
      constexpr uint32_t idesc_acc = umma_idesc_bf16(BT, DH, 0, 1);   // A from TMEM, B MN-major
      // dQ^T [dh x 64 queries] = K^T dS^T, both operands MN-major.  The instruction always spans 128 rows; with
      // DH == 64 the upper 64 are fed from the V tile that follows K in shared memory and are never read.
      constexpr uint32_t idesc_dq = umma_idesc_bf16(128, BQ2, 1, 1);
      constexpr uint32_t hi = desc_hi_sw128(1024);
      constexpr uint32_t hi_plain = desc_hi_plain(128);
      // low descriptor words of the resident tiles; per MMA only a constant is added
      const uint32_t k_lo = desc_lo_sw128(smem_u32(smem + L::OFF_K), 0);
      const uint32_t v_lo = desc_lo_sw128(smem_u32(smem + L::OFF_V), 0);
      const uint32_t kmn_lo = desc_lo_sw128(smem_u32(smem + L::OFF_K), HALF_BYTES);   // K as MN-major A
      const uint32_t ds_lo = desc_lo_sw128(smem_u32(smem + L::OFF_DS), 0);            // dS^T as MN-major B
      // 16-column K-major tiles whose columns 8-15 are all zero share one block of zeros: the leading-dimension
      // offset of each descriptor is the distance from the tile's first half to that block
      const uint32_t zero_addr = smem_u32(smem + L::OFF_ZERO);
      const uint32_t ones_lo = desc_lo_plain(smem_u32(smem + L::OFF_ONES), zero_addr - smem_u32(smem + L::OFF_ONES));
      const uint32_t stat_base = smem_u32(smem + L::OFF_STAT);
      const uint32_t ring = smem_u32(smem + L::OFF_RING);
      bool ok = mbar_wait(kv_full, 0, err);
      if (ok) ok = mbar_wait(stat0, 0, err);
      auto issue_scores = [&](int it) -> bool {
        const int s = it % BWD_STAGES;
        if (!mbar_wait(&q_full[s], (it / BWD_STAGES) & 1, err)) return false;
        tc_fence_after_sync();
        const uint32_t q_lo = desc_lo_sw128(ring + s * L::STAGE, 0);
        const uint32_t do_lo = desc_lo_sw128(ring + s * L::STAGE + L::Q_TILE, 0);
        const uint32_t tm = tmem_base + (it & 1) * 64;
        const uint32_t lse_addr = stat_base + (it & 3) * 2048;
        const uint32_t stat_lo = desc_lo_plain(lse_addr, zero_addr - lse_addr);
        const uint32_t delta_lo = desc_lo_plain(lse_addr + 1024, zero_addr - lse_addr - 1024);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t offa = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          const uint32_t offb = (ks / 4) * QHALF_BYTES + (ks % 4) * 32;
          umma_ss_w(tm, desc_lo_add(k_lo, offa), desc_lo_add(q_lo, offb), hi, idesc_st, ks != 0, leader);
        }
        umma_ss_w(tm, ones_lo, stat_lo, hi_plain, idesc_st, 1, leader);                          // S^T -= LSE / scale
        // the single dP^T buffer takes the next step once the compute warps hold the previous one in registers
        if (it > 0 && !mbar_wait(dp_free, (it - 1) & 1, err)) return false;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t offa = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          const uint32_t offb = (ks / 4) * QHALF_BYTES + (ks % 4) * 32;
          umma_ss_w(tm_dp, desc_lo_add(v_lo, offa), desc_lo_add(do_lo, offb), hi, idesc_st, ks != 0, leader);
        }
        umma_ss_w(tm_dp, ones_lo, delta_lo, hi_plain, idesc_st, 1, leader);                      // dP^T -= Delta
        umma_commit(st_full, leader);
        return true;
      };
      if (ok && n_iter > 0) ok = issue_scores(0);
      for (int it = 0; it < n_iter && ok; ++it) {
        // S^T of the next step goes to the other score buffer; its previous readers (the accumulate MMAs
        // of step it-1) precede this in the in-order tensor pipe, and its statistics tile was staged
        // before pds_ready(it-1)
        if (it + 1 < n_iter && !issue_scores(it + 1)) { ok = false; break; }
        if (!mbar_wait(&pds_ready[it & 1], (it >> 1) & 1, err)) { ok = false; break; }
        tc_fence_after_sync();
        const int s = it % BWD_STAGES;
        const uint32_t qmn_lo = desc_lo_sw128(ring + s * L::STAGE, QHALF_BYTES);                 // Q  as MN-major B
        const uint32_t domn_lo = desc_lo_sw128(ring + s * L::STAGE + L::Q_TILE, QHALF_BYTES);    // dO as MN-major B
        const uint32_t tm = tmem_base + (it & 1) * 64;
        // P^T of queries [32w, 32w+32) sits in 32-bit columns [32w, 32w+16) of the score buffer, dS^T in [32w+16, 32w+32)
#pragma unroll
        for (int ks = 0; ks < KSTEPS_Q; ++ks)  // dV += P^T dO
          umma_ts_w(tm_dv, tm + (ks / 2) * 32 + (ks % 2) * 8, desc_lo_add(domn_lo, ks * 2048), hi, idesc_acc, (it | ks) != 0, leader);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_Q; ++ks)  // dK += dS^T Q
          umma_ts_w(tm_dk, tm + (ks / 2) * 32 + 16 + (ks % 2) * 8, desc_lo_add(qmn_lo, ks * 2048), hi, idesc_acc, (it | ks) != 0, leader);
        umma_commit(&q_empty[s], leader);  // the ring stage is free as soon as dV and dK have read it
        if (it > 0 && !mbar_wait(dq_free, (it - 1) & 1, err)) { ok = false; break; }
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < KSTEPS_KV; ++ks)  // dQ^T = K^T dS^T
          umma_ss_w(tm_dq, desc_lo_add(kmn_lo, ks * 2048), desc_lo_add(ds_lo, ks * 2048), hi, idesc_dq, ks != 0, leader);
        umma_commit(dq_full, leader);
      }
      if (ok) umma_commit(acc_done, leader);
    }
  } else if (warp < 10) {
    // ------------------------------ compute warpgroups ------------------------------
    const int wg = (warp - 2) >> 2;     // query columns [wg*32, wg*32+32) of every step
    const int quarter = warp & 3;       // TMEM lane quarter of this warp
    const int r = quarter * 32 + lane;  // key row inside the tile == TMEM lane
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    const int kv_row = kv0 + r;
    const uint64_t c2 = pack_f2(p.scale_log2, p.scale_log2);
    // P^T and dS^T (bf16 pairs) overwrite the warpgroup's OWN score columns, which the other warpgroup never
    // reads: P^T in 32-bit columns [wg*32, wg*32+16), dS^T in [wg*32+16, wg*32+32)
    const uint32_t col = wg * 32;
    uint8_t* ds_smem = smem + L::OFF_DS;
    int qi = 0;  // query tile index of the current step inside its stream
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int set = it & 1;
      const uint32_t tm = tmem_base + set * 64;
      ok = mbar_wait(st_full, it & 1, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      uint32_t st[32], dp[32];
      tmem_ld_x32(tm + lane_sel + col, st);
      tmem_ld_x32(tm_dp + lane_sel + col, dp);
      const int q_col0 = (qt_first + qi) * BQ2 + wg * 32;           // query of this warpgroup's first column
      const bool diag = p.causal && q_col0 - wg * 32 < kv0 + BT;    // the query tile straddles the diagonal
      const int first_visible = diag ? kv_row - q_col0 : 0;         // own columns below this are masked for this key row
      uint32_t pk[16], dk[16];
      tmem_ld_wait();
      tc_fence_before_sync();
      mbar_arrive(dp_free);
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
      tmem_st_x16(tm + lane_sel + col, pk);
      tmem_st_x16(tm + lane_sel + col + 16, dk);
      // dS^T also goes to shared memory as the B operand of dQ^T = K^T dS^T; the previous step's product
      // must have finished reading the tile
      if (it > 0) {
        ok = mbar_wait(dq_full, (it - 1) & 1, err);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<uint4*>(ds_smem + sw128_offset(r, wg * 4 + j)) =
            make_uint4(dk[4 * j], dk[4 * j + 1], dk[4 * j + 2], dk[4 * j + 3]);
      tmem_st_wait();
      fence_proxy_async_smem();  // dS^T is read by the tensor core's proxy
      tc_fence_before_sync();
      mbar_arrive(&pds_ready[set]);
      if (++qi == per_stream) qi = 0;
    }
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      bool w = mbar_wait(acc_done, 0, err);
      ok = __all_sync(0xffffffffu, w);
    }
    if (ok) {
      tc_fence_after_sync();
      // warpgroup 0 adds dK (scaled), warpgroup 1 adds dV; every lane loads, valid rows reduce
      const bool valid = kv_row < p.S;
      const size_t row_off = ((size_t(b) * p.S + (valid ? kv_row : 0)) * p.Hkv + hk) * DH;
      float* dst = (wg == 0 ? p.dk_sum[grp] : p.dv_sum[grp]) + row_off;
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
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + c * 32 + v4 * 4),
                         "f"(__uint_as_float(a[4 * v4]) * mul), "f"(__uint_as_float(a[4 * v4 + 1]) * mul),
                         "f"(__uint_as_float(a[4 * v4 + 2]) * mul), "f"(__uint_as_float(a[4 * v4 + 3]) * mul)
                         : "memory");
        }
      }
    }
  } else {
    // ------------------------------ dQ drain warpgroup ------------------------------
    // TMEM lane == column of dQ (dh index): this warp owns dh columns [32*quarter, 32*quarter + 32) of the
    // step's 64 queries, lays them out as [64 queries x 32 columns] fp32 in shared memory and adds them to the
    // accumulator with one 8 KB bulk reduction, which has a whole step to read the buffer before it is rewritten.
    const int quarter = warp & 3;
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    const bool active = quarter * 32 < DH;  // with DH == 64 the upper lanes hold nothing
    float* stg = reinterpret_cast<float*>(smem + L::OFF_DQ + (warp - 10) * DQ_STAGE_BYTES);
    const uint32_t stg_s = smem_u32(stg);
    // Statistics.  This warpgroup also prepares the per-query operand tiles the tensor core adds to the scores:
    // thread t < 64 handles -LSE/scale of query column t, thread 64 + t handles -Delta of column t, as the
    // three-term bf16 split.  The raw fp32 values come in through cp.async into a small ring in shared memory,
    // requested eight steps before the step that uses them and staged as an operand tile three steps before: no
    // register ever waits on global memory, and the compute warpgroups never touch the statistics.
    const int stat_tid = threadIdx.x - 10 * 32;
    const int stat_kind = stat_tid >> 6;   // 0 lse, 1 delta
    const int stat_col = stat_tid & 63;
    uint8_t* stat_row = smem + L::OFF_STAT + stat_kind * 1024 + stat_col * 16;
    float* raw = reinterpret_cast<float*>(smem + L::OFF_RAW) + stat_tid;   // ring slot s at raw[s * 128]
    const float stat_mul = stat_kind == 0 ? -1.f / p.scale : -1.f;
    const float stat_pad = stat_kind == 0 ? -30000.f : 0.f;  // a query beyond the sequence: exp2 underflows to zero
    // Two cursors walk the steps in order (incremental decode of step -> layer, head, query tile): one for the
    // step whose statistics are requested next, one kStatAhead steps further that only pulls the line into L2.
    // `row` is the statistic row of the cursor's (layer, head): it is looked up (an indexed read of the kernel
    // parameters) only when the stream changes, never on the per-step path.
    constexpr int kStatAhead = 12;
    struct Cursor {
      int it = 0, qi = 0, g = 0, li = 0;
      const float* row = nullptr;
    };
    auto row_of = [&](int li, int g) {
      const int slot = slot0 + (li < n_layers ? li : 0);
      const float* src = stat_kind == 0 ? p.lse[slot] : p.delta[slot];
      return src + (size_t(b) * p.Hq + hk * G + g) * p.S;
    };
    auto advance = [&](Cursor& c) {
      ++c.it;
      if (++c.qi == per_stream) {
        c.qi = 0;
        if (++c.g == G) {
          c.g = 0;
          ++c.li;
        }
        c.row = row_of(c.li, c.g);
      }
    };
    auto locate = [&](const Cursor& c, bool& valid) {  // address of this thread's statistic of step c (clamped, always valid)
      const int qc = (qt_first + c.qi) * BQ2 + stat_col;
      valid = c.it < n_iter && qc < p.S;
      return c.row + (valid ? qc : p.S - 1);
    };
    Cursor cf, cp;
    cf.row = cp.row = row_of(0, 0);
    for (int i = 0; i < kStatAhead; ++i) advance(cp);
    auto request = [&]() -> bool {  // cp.async of the next step's value into its ring slot; returns its validity
      bool ahead_valid, valid;
      const float* ahead = locate(cp, ahead_valid);
      if ((stat_col & 31) == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(ahead));
      advance(cp);
      const float* ptr = locate(cf, valid);
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(raw + (cf.it & 7) * 128)), "l"(ptr) : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
      advance(cf);
      return valid;
    };
    auto stage = [&](int step, bool valid) {  // the value of `step` has landed: split it into the step's operand tile
      *reinterpret_cast<uint4*>(stat_row + (step & 3) * 2048) = split3_bf16(valid ? raw[(step & 7) * 128] * stat_mul : stat_pad);
    };
    // validity flags of the requests in flight, oldest (step it+3) in bit 0
    uint32_t vbits = 0;
    {
      const bool a0 = request(), a1 = request(), a2 = request();
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      stage(0, a0);
      stage(1, a1);
      stage(2, a2);
      // steps 3..7; from here on a ring slot is requested again only after its previous value has been staged
#pragma unroll
      for (int i = 0; i < 5; ++i) vbits |= uint32_t(request()) << i;
    }
    fence_proxy_async_smem();
    mbar_arrive(stat0);
    int li = 0, g = 0, qi = 0;
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      ok = mbar_wait(dq_full, it & 1, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      uint32_t a[32], c[32];
      tmem_ld_x32(tm_dq + lane_sel, a);
      tmem_ld_x32(tm_dq + lane_sel + 32, c);
      tmem_ld_wait();
      // The operand tile of step it+3 (last read by the scores of step it-1, which completed before this step's
      // dQ^T did) and the request for step it+8.  The arrival below publishes the tile: the issuing warp waits for
      // it before the next step's dQ^T, a whole step before the scores of step it+3 are issued.
      vbits |= uint32_t(request()) << 5;
      asm volatile("cp.async.wait_group 5;" ::: "memory");
      stage(it + 3, vbits & 1u);
      vbits >>= 1;
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(dq_free);
      if (active) {
        const size_t tile = ((size_t(b) * p.Hq + hk * G + g) * n_qt + (qt_first + qi)) * (DH / 32) + quarter;
        float* dst = p.dq_acc[slot0 + li] + tile * (BQ2 * 32);
        // the previous step's reduction has read the buffer
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int q = 0; q < BQ2; ++q) stg[q * 32 + lane] = __uint_as_float(q < 32 ? a[q & 31] : c[q & 31]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(dst), "r"(stg_s),
                       "n"(DQ_STAGE_BYTES)
                       : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      if (++qi == per_stream) {
        qi = 0;
        if (++g == G) {
          g = 0;
          ++li;
        }
      }
    }
    // the reductions must have completed before the block's shared memory goes away and the grid ends
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// dq[b,s,hq,:] = bf16(scale * accumulator), from the blocked fp32 layout [b][hq][tile][quarter][64][32].
// One thread per 8 consecutive columns of one query row: two 16-byte loads, one 16-byte store.
template <int DH>
__global__ void dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, int B, int S, int Hq,
                                  float scale) {
  constexpr int TPR = DH / 8;  // threads per query row
  const int n_qt = (S + BQ2 - 1) / BQ2;
  const size_t rows = size_t(B) * Hq * n_qt * BQ2;
  const size_t stride = size_t(gridDim.x) * blockDim.x / TPR;
  const int j = threadIdx.x % TPR;
  const int quarter = j / 4, d0 = (j % 4) * 8;
  for (size_t row = (size_t(blockIdx.x) * blockDim.x + threadIdx.x) / TPR; row < rows; row += stride) {
    const int q = int(row % BQ2);
    const size_t tile = row / BQ2;  // (b * Hq + hq) * n_qt + qt
    const int qt = int(tile % n_qt);
    const size_t bh = tile / n_qt;
    const int s = qt * BQ2 + q;
    if (s >= S) continue;
    const float* src = acc + ((tile * (DH / 32) + quarter) * BQ2 + q) * 32 + d0;
    const float4 lo = *reinterpret_cast<const float4*>(src);
    const float4 hi = *reinterpret_cast<const float4*>(src + 4);
    uint4 v;
    v.x = pack_bf16(lo.x * scale, lo.y * scale);
    v.y = pack_bf16(lo.z * scale, lo.w * scale);
    v.z = pack_bf16(hi.x * scale, hi.y * scale);
    v.w = pack_bf16(hi.z * scale, hi.w * scale);
    const int hq = int(bh % Hq);
    const int bb = int(bh / Hq);
    *reinterpret_cast<uint4*>(dq + ((size_t(bb) * S + s) * Hq + hq) * DH + quarter * 32 + d0) = v;
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

// Member layers of the launches' accumulators that are live at once: a launch takes whole donor groups until it
// holds MAX_GROUP member layers.
int max_layers_per_launch(const kvp_shape* s) { return s->L < MAX_GROUP ? s->L : MAX_GROUP; }

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

// Workspace: Delta [B,Hq,S] fp32 for every layer, then the fp32 dQ accumulators of the member layers of one launch
// (launches run one after the other and reuse them).
size_t attn_bwd_workspace(const kvp_shape* s, const int32_t* donor) {
  (void)donor;
  return size_t(s->L) * align256(size_t(s->B) * s->Hq * s->S * 4) +
         size_t(max_layers_per_launch(s)) * align256(dq_acc_floats(s->B, s->S, s->Hq, s->dh) * 4);
}

int attn_bwd_all(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                 const void* const* k, const void* const* v, const void* const* o, const void* const* d_o,
                 const float* const* lse, void* const* dq, float* const* dk_sum, float* const* dv_sum, void* ws,
                 size_t ws_bytes, cudaStream_t stream) {
  (void)ws_bytes;
  const int dh = s->dh;
  const float sc = scale == 0.f ? 1.f / sqrtf(float(dh)) : scale;
  const size_t delta_bytes = align256(size_t(s->B) * s->Hq * s->S * 4);
  const size_t acc_bytes = align256(dq_acc_floats(s->B, s->S, s->Hq, dh) * 4);
  uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);
  uint8_t* acc_base = wsb + size_t(s->L) * delta_bytes;
  static const cudaError_t attr = [] {
    cudaError_t e = cudaFuncSetAttribute(bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<128>::TOTAL);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<64>::TOTAL);
  }();
  if (attr != cudaSuccess) return KVP_ERR_CUDA;

  // Delta for every layer
  timing_before(KVP_KERNEL_ATTN_BWD_AUX, stream);
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
  timing_after(KVP_KERNEL_ATTN_BWD_AUX, stream);
  if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;

  // Donor groups, largest first; a launch takes groups until it holds MAX_GROUP member layers.  A launch writes
  // dK / dV of its donors through reductions into cleared buffers, so a donor shared by more than MAX_GROUP
  // layers is not supported.
  struct Group {
    int owner, n;
    int members[MAX_GROUP];
  };
  std::vector<Group> groups;
  for (int d = 0; d < s->L; ++d) {
    if (donor[d] != d) continue;
    Group g;
    g.owner = d;
    g.n = 0;
    for (int l = d; l < s->L; ++l)
      if (donor[l] == d) {
        if (g.n == MAX_GROUP) return KVP_ERR_UNSUPPORTED;
        g.members[g.n++] = l;
      }
    groups.push_back(g);
  }
  std::stable_sort(groups.begin(), groups.end(), [](const Group& a, const Group& b) { return a.n > b.n; });
  const int n_jt = (s->S + BT - 1) / BT, n_qt = (s->S + BQ2 - 1) / BQ2, n_pairs = s->Hkv * s->B;
  const int G = s->Hq / s->Hkv;
  const size_t kv_bytes = size_t(s->B) * s->S * s->Hkv * dh * 4;
  size_t gi = 0;
  while (gi < groups.size()) {
    BwdParams p;
    int slots = 0, ng = 0;
    int slot_layer[MAX_GROUP];
    p.cta_begin[0] = 0;
    p.first_slot[0] = 0;
    while (gi < groups.size() && slots + groups[gi].n <= MAX_GROUP) {
      const Group& g = groups[gi];
      int rc = make_map_bshd(&p.map_k[ng], k[g.owner], s->B, s->S, s->Hkv, dh, BT);
      if (rc == KVP_OK) rc = make_map_bshd(&p.map_v[ng], v[g.owner], s->B, s->S, s->Hkv, dh, BT);
      if (rc != KVP_OK) return rc;
      for (int i = 0; i < g.n; ++i) {
        const int l = g.members[i];
        rc = make_map_bshd(&p.map_q[slots], q[l], s->B, s->S, s->Hq, dh, BQ2);
        if (rc == KVP_OK) rc = make_map_bshd(&p.map_do[slots], d_o[l], s->B, s->S, s->Hq, dh, BQ2);
        if (rc != KVP_OK) return rc;
        p.lse[slots] = lse[l];
        p.delta[slots] = reinterpret_cast<const float*>(wsb + size_t(l) * delta_bytes);
        p.dq_acc[slots] = reinterpret_cast<float*>(acc_base + size_t(slots) * acc_bytes);
        slot_layer[slots] = l;
        ++slots;
      }
      p.dk_sum[ng] = dk_sum[g.owner];
      p.dv_sum[ng] = dv_sum[g.owner];
      p.window[ng] = std::min(n_qt, std::max(kMinWindow, (kStepsPerCta + g.n * G - 1) / (g.n * G)));
      p.ctas_per_pair[ng] = 0;
      for (int w = 0; w * p.window[ng] < n_qt; ++w)
        p.ctas_per_pair[ng] += causal ? std::min(n_jt, ((w + 1) * p.window[ng] * BQ2 + BT - 1) / BT) : n_jt;
      p.first_slot[ng + 1] = slots;
      p.cta_begin[ng + 1] = p.cta_begin[ng] + n_pairs * p.ctas_per_pair[ng];
      ++ng;
      ++gi;
    }
    for (int i = slots; i < MAX_GROUP; ++i) {   // unused entries repeat slot 0, so that no descriptor is left unset
      p.map_q[i] = p.map_q[0];
      p.map_do[i] = p.map_do[0];
      p.lse[i] = p.lse[0];
      p.delta[i] = p.delta[0];
      p.dq_acc[i] = p.dq_acc[0];
    }
    for (int i = ng; i < MAX_GROUP; ++i) {
      p.map_k[i] = p.map_k[0];
      p.map_v[i] = p.map_v[0];
      p.dk_sum[i] = p.dk_sum[0];
      p.dv_sum[i] = p.dv_sum[0];
      p.window[i] = p.window[0];
      p.ctas_per_pair[i] = p.ctas_per_pair[0];
      p.first_slot[i + 1] = slots;
      p.cta_begin[i + 1] = p.cta_begin[ng];
    }
    p.n_groups = ng;
    p.B = s->B;
    p.S = s->S;
    p.Hq = s->Hq;
    p.Hkv = s->Hkv;
    p.causal = causal;
    p.scale = sc;
    p.scale_log2 = sc * 1.4426950408889634f;
    timing_before(KVP_KERNEL_ATTN_BWD_AUX, stream);
    if (cudaMemsetAsync(acc_base, 0, size_t(slots) * acc_bytes, stream) != cudaSuccess) return KVP_ERR_CUDA;
    for (int i = 0; i < ng; ++i)
      if (cudaMemsetAsync(p.dk_sum[i], 0, kv_bytes, stream) != cudaSuccess ||
          cudaMemsetAsync(p.dv_sum[i], 0, kv_bytes, stream) != cudaSuccess)
        return KVP_ERR_CUDA;
    timing_after(KVP_KERNEL_ATTN_BWD_AUX, stream);
    dim3 grid(p.cta_begin[ng]);
    timing_before(KVP_KERNEL_ATTN_BWD, stream);
    if (dh == 128)
      bwd_kernel<128><<<grid, BWD_THREADS, BwdSmem<128>::TOTAL, stream>>>(p);
    else
      bwd_kernel<64><<<grid, BWD_THREADS, BwdSmem<64>::TOTAL, stream>>>(p);
    timing_after(KVP_KERNEL_ATTN_BWD, stream);
    note_launch();
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
    timing_before(KVP_KERNEL_ATTN_BWD_AUX, stream);
    for (int i = 0; i < slots; ++i) {
      const size_t threads = dq_acc_floats(s->B, s->S, s->Hq, dh) / 8;
      const int blocks = int(min(size_t(sm_count()) * 16, (threads + 255) / 256));
      if (dh == 128)
        dq_convert_kernel<128><<<blocks, 256, 0, stream>>>(p.dq_acc[i], reinterpret_cast<__nv_bfloat16*>(dq[slot_layer[i]]),
                                                           s->B, s->S, s->Hq, sc);
      else
        dq_convert_kernel<64><<<blocks, 256, 0, stream>>>(p.dq_acc[i], reinterpret_cast<__nv_bfloat16*>(dq[slot_layer[i]]),
                                                          s->B, s->S, s->Hq, sc);
      note_launch();
    }
    timing_after(KVP_KERNEL_ATTN_BWD_AUX, stream);
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
  }
  return KVP_OK;
}

}  // namespace kvp
