// Causal GQA flash-attention forward over a donor map (Eq. 2-3 of the paper): layer l attends
// with its own queries to the keys/values of layer donor[l].
//
// A work item is TWO adjacent 128-row query tiles (A, B) of one (batch, query head); the CTA walks the
// donor's K/V tiles once for both, so every K/V tile fetched by TMA feeds twice the tensor work.  CTAs are
// persistent (one per SM) and take a balanced list of items each.
//   warp 0      TMA producer: Q_A, Q_B once, then K_j / V_j rings
//   warps 1, 2  tcgen05.mma issuers, one per query tile (on two different warp schedulers: issuing an MMA costs
//               its scheduler some tens of cycles, which the softmax warps of that scheduler would otherwise
//               have).  Every 128-key tile is worked on as two 64-key sub-blocks c = 2j, 2j+1:
//               S_X(c) = Q_X K_c^T goes into one of TWO 64-column score buffers of tile X (c & 1), and
//               O_X += P_X(c) V_c takes P_X(c) as the A operand FROM TMEM (bf16 pairs written back over the
//               first 32 columns of that score buffer) and V_c as an MN-major B operand.  S_X(c+2) is issued
//               right behind P_X(c) V_c, so the scores of sub-block c+1 are already complete when the softmax
//               of sub-block c ends: the softmax warps never wait for the tensor pipe to turn around.
//   warp 3      idle
//   warps 4-7   softmax of tile A, warps 8-11 softmax of tile B: one thread per query row (TMEM lane
//               == row, so the row maximum and sum need no cross-thread traffic), packed fp32x2
//               arithmetic, O rescaled in TMEM only when the running maximum moved by more than 2^8 (and
//               then only after the P V product still in flight has completed)
// While one tile's exponentials run, the tensor pipe works on the other tile and on the next scores of this one.
#include <math.h>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int BC = 64;            // keys per sub-block (one score buffer)
constexpr int FWD_THREADS = 384;
constexpr int FWD_KSTAGES = 3;
constexpr int FWD_VSTAGES = 2;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr uint32_t HALF_BYTES = 128 * 128;  // one [128 rows x 128 B] block

__device__ int g_fwd_status;

template <int DH>
struct FwdSmem {
  static constexpr int Q_BYTES = BQ * DH * 2;   // one query tile
  static constexpr int KV_BYTES = BKV * DH * 2;
  static constexpr int OFF_Q = 0;               // [2]
  static constexpr int OFF_K = OFF_Q + 2 * Q_BYTES;
  static constexpr int OFF_V = OFF_K + FWD_KSTAGES * KV_BYTES;
  static constexpr int OFF_BAR = OFF_V + FWD_VSTAGES * KV_BYTES;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;  // + alignment slack
};

constexpr int FWD_MAX_LAYERS = 8;   // layers per launch

struct FwdParams {
  // per layer: 4-D [B, S, H, dh] tensors, box {64, 1, 128, 1}; K and V are those of the layer's donor
  CUtensorMap map_q[FWD_MAX_LAYERS], map_k[FWD_MAX_LAYERS], map_v[FWD_MAX_LAYERS];
  __nv_bfloat16* o[FWD_MAX_LAYERS];  // [B, S, Hq, dh]
  float* lse[FWD_MAX_LAYERS];        // [B, Hq, S]
  int n_layers;
  int B, S, Hq, Hkv;
  int causal;
  float scale_log2;                 // scale * log2(e)
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Work items of a launch: (layer, batch, query head, pair of query tiles), the deepest causal pairs first.  The list is
// dealt out in rounds of gridDim.x items, forwards in even rounds and backwards in odd ones, so that the CTA that
// got the longest item of one round gets the shortest of the next: every CTA ends up with nearly the same work.
__device__ __forceinline__ int fwd_item_index(int round) {
  const int g = int(gridDim.x), i = int(blockIdx.x);
  return round * g + ((round & 1) ? g - 1 - i : i);
}
struct FwdItem {
  int layer, b, hq, hk, q0;
  int n_kv[2];  // key tiles each query tile walks (tile B may not exist at a ragged end)
  int n_max;
};
__device__ __forceinline__ FwdItem fwd_item(const FwdParams& p, int t, int n_pairs) {
  FwdItem w;
  const int bh = p.B * p.Hq, lbh = p.n_layers * bh;
  const int pair = n_pairs - 1 - t / lbh;
  const int r = t % lbh;
  w.layer = r / bh;
  w.hq = r % p.Hq;
  w.b = (r % bh) / p.Hq;
  w.hk = w.hq / (p.Hq / p.Hkv);
  w.q0 = pair * 2 * BQ;  // first row of tile A; tile B starts at q0 + 128
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    const int qs = w.q0 + x * BQ;
    const int kv_end = p.causal ? min(p.S, qs + BQ) : p.S;
    w.n_kv[x] = qs < p.S ? (kv_end + BKV - 1) / BKV : 0;
  }
  w.n_max = max(w.n_kv[0], w.n_kv[1]);
  return w;
}

template <int DH>
__global__ void __launch_bounds__(FWD_THREADS, 1) attn_fwd_kernel(const __grid_constant__ FwdParams p) {
  using L = FwdSmem<DH>;
  constexpr int KSTEPS_QK = DH / 16;   // K dimension of S = Q K^T is dh
  constexpr int HALVES = DH / 64;      // 64-column (128-byte) blocks per row of Q / K / V

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* q_empty = bars + 1;                 // 2 arrivals: both issuing warps are done with the query tiles
  uint64_t* k_full = bars + 2;                  // [KSTAGES]
  uint64_t* k_empty = k_full + FWD_KSTAGES;     // [KSTAGES]
  uint64_t* v_full = k_empty + FWD_KSTAGES;     // [VSTAGES]
  uint64_t* v_empty = v_full + FWD_VSTAGES;     // [VSTAGES]
  uint64_t* s_full = v_empty + FWD_VSTAGES;     // [2][2] per query tile and score buffer
  uint64_t* p_ready = s_full + 4;               // [2][2] per query tile and score buffer (128 arrivals)
  uint64_t* pv_done = p_ready + 4;              // [2] per query tile: one completion per sub-block's P V product
  uint64_t* o_done = pv_done + 2;               // [2] per query tile: the item's last P V product has completed
  uint64_t* o_free = o_done + 2;                // [2] per query tile: the softmax warps have read O out (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_free + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_fwd_status;

  const int n_qtiles = (p.S + BQ - 1) / BQ;
  const int n_pairs = (n_qtiles + 1) / 2;
  const int n_items = n_pairs * p.n_layers * p.B * p.Hq;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_empty, 2);
    for (int i = 0; i < FWD_KSTAGES; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], 2);   // one MMA-completion arrival per issuing warp
    }
    for (int i = 0; i < FWD_VSTAGES; ++i) {
      mbar_init(&v_full[i], 1);
      mbar_init(&v_empty[i], 2);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&p_ready[i], 128);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&pv_done[i], 1);
      mbar_init(&o_done[i], 1);
      mbar_init(&o_free[i], 128);
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
  // tile X: score buffer u at [X*128 + u*64, +64) with P over its first 32 columns; output accumulator at
  // [256 + X*128, +128)
  //
  // The CTA is persistent: every role walks the same list of items and keeps running counts (items, key tiles,
  // sub-blocks per query tile), from which ring stages, score buffers and barrier parities follow.  The K / V rings
  // simply keep streaming across item boundaries; the next item's query tiles are loaded as soon as the last score
  // MMAs of the current one have completed, and its first scores are computed while the softmax warps still
  // normalise and store the current output.

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      uint32_t it = 0, kg = 0, vg = 0;  // items, K tiles and V tiles requested so far
      bool ok = true;
      for (int round = 0; round * int(gridDim.x) < n_items && ok; ++round) {
        const int t = fwd_item_index(round);
        if (t >= n_items) continue;   // only the last round can be short
        const FwdItem w = fwd_item(p, t, n_pairs);
        if (!mbar_wait(q_empty, (it & 1) ^ 1, err)) { ok = false; break; }
        mbar_expect_tx_e(q_full, 2 * L::Q_BYTES, leader);  // rows beyond the sequence are zero-filled
#pragma unroll
        for (int x = 0; x < 2; ++x)
#pragma unroll
          for (int h = 0; h < HALVES; ++h)
            tma_load_4d_e(smem + L::OFF_Q + x * L::Q_BYTES + h * HALF_BYTES, &p.map_q[w.layer], q_full, h * 64, w.hq, w.q0 + x * BQ, w.b, leader);
        auto load_k = [&](int j) -> bool {
          const int s = kg % FWD_KSTAGES;
          if (!mbar_wait(&k_empty[s], ((kg / FWD_KSTAGES) & 1) ^ 1, err)) return false;
          mbar_expect_tx_e(&k_full[s], L::KV_BYTES, leader);
#pragma unroll
          for (int h = 0; h < HALVES; ++h)
            tma_load_4d_e(smem + L::OFF_K + s * L::KV_BYTES + h * HALF_BYTES, &p.map_k[w.layer], &k_full[s], h * 64, w.hk, j * BKV, w.b, leader);
          ++kg;
          return true;
        };
        auto load_v = [&](int j) -> bool {
          const int s = vg % FWD_VSTAGES;
          if (!mbar_wait(&v_empty[s], ((vg / FWD_VSTAGES) & 1) ^ 1, err)) return false;
          mbar_expect_tx_e(&v_full[s], L::KV_BYTES, leader);
#pragma unroll
          for (int h = 0; h < HALVES; ++h)
            tma_load_4d_e(smem + L::OFF_V + s * L::KV_BYTES + h * HALF_BYTES, &p.map_v[w.layer], &v_full[s], h * 64, w.hk, j * BKV, w.b, leader);
          ++vg;
          return true;
        };
        ok = load_k(0);
        for (int j = 0; j < w.n_max && ok; ++j) {
          if (j + 1 < w.n_max) ok = load_k(j + 1);  // scores run one tile ahead of the P V products
          if (ok) ok = load_v(j);
        }
        ++it;
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------ MMA issuer of query tile x ------------------------------
    {
      const uint32_t leader = elect_one();  // the whole warp runs the loop; one lane issues
      constexpr uint32_t idesc_qk = umma_idesc_bf16(BQ, BC, 0, 0);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(BQ, DH, 0, 1);
      constexpr uint32_t hi = desc_hi_sw128(1024);
      constexpr int KSTEPS_SUB = BC / 16;  // K steps of one sub-block's P V product
      const uint32_t k_base = smem_u32(smem + L::OFF_K), v_base = smem_u32(smem + L::OFF_V);
      const int x = warp - 1;
      const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::OFF_Q + x * L::Q_BYTES), 0);
      const uint32_t tm_sx = tmem_base + x * BKV, tm_ox = tmem_base + 256 + x * 128;
      uint32_t it = 0;    // items so far
      uint32_t jg = 0;    // key tiles of earlier items (ring position of this item's tile 0)
      uint32_t g0 = 0;    // sub-blocks of earlier items of this query tile (always even)
      bool ok = true;
      for (int round = 0; round * int(gridDim.x) < n_items && ok; ++round) {
        const int t = fwd_item_index(round);
        if (t >= n_items) continue;
        const FwdItem w = fwd_item(p, t, n_pairs);
        const int n_cx = 2 * w.n_kv[x];
        const int n_cmax = 2 * w.n_max;
        auto k_stage = [&](int j) { return (jg + j) % FWD_KSTAGES; };
        auto k_parity = [&](int j) { return ((jg + j) / FWD_KSTAGES) & 1; };
        auto v_stage = [&](int j) { return (jg + j) % FWD_VSTAGES; };
        auto v_parity = [&](int j) { return ((jg + j) / FWD_VSTAGES) & 1; };
        auto issue_s = [&](int c) {  // S_x(c) = Q_x K_c^T; the key tile holding sub-block c is known to be resident
          const int j = c >> 1, u = c & 1;
          // keys 64u .. 64u+63 of the tile are rows 64u .. of each 128-byte-wide block: 64 rows x 128 B further on
          const uint32_t k_lo = desc_lo_sw128(k_base + k_stage(j) * L::KV_BYTES + u * (BC * 128), 0);
#pragma unroll
          for (int ks = 0; ks < KSTEPS_QK; ++ks) {
            const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
            umma_ss_w(tm_sx + u * BC, desc_lo_add(q_lo, off), desc_lo_add(k_lo, off), hi, idesc_qk, ks != 0, leader);
          }
          umma_commit(&s_full[2 * x + u], leader);
        };
        auto issue_pv = [&](int c) {  // O_x += P_x(c) V_c
          const int j = c >> 1, u = c & 1;
          const uint32_t v_lo = desc_lo_sw128(v_base + v_stage(j) * L::KV_BYTES, HALF_BYTES);
#pragma unroll
          for (int ks = 0; ks < KSTEPS_SUB; ++ks)
            umma_ts_w(tm_ox, tm_sx + u * BC + ks * 8, desc_lo_add(v_lo, (u * KSTEPS_SUB + ks) * 2048), hi, idesc_pv,
                      (c | ks) != 0, leader);
        };
        if (!mbar_wait(q_full, it & 1, err)) { ok = false; break; }
        if (!mbar_wait(&k_full[k_stage(0)], k_parity(0), err)) { ok = false; break; }
        tc_fence_after_sync();
        // (the score buffers are free: the previous item's last P V products were issued by this thread)
#pragma unroll
        for (int c = 0; c < 2; ++c)
          if (c < n_cx) issue_s(c);
        umma_commit(&k_empty[k_stage(0)], leader);
        if (n_cx <= 2) umma_commit(q_empty, leader);  // no further score MMAs of this item from this warp
        // O_x is overwritten by the first P V product: the softmax warps must have read the previous item's out
        if (it > 0 && !mbar_wait(&o_free[x], (it - 1) & 1, err)) { ok = false; break; }
        // Every round releases its K / V stages from this warp too when this tile has run out of sub-blocks (the
        // other tile may be one key tile longer): an arrival with nothing outstanding completes at once.
        for (int c = 0; c < n_cmax && ok; ++c) {
          const int j = c >> 1, u = c & 1;
          const int cn = c + 2, jn = cn >> 1;   // the scores issued in this round: sub-block c + 2
          // (it still waits for every stage to fill first, so it can never arrive twice in one phase of a stage)
          if (u == 0 && !mbar_wait(&v_full[v_stage(j)], v_parity(j), err)) { ok = false; break; }
          if (cn < n_cmax && (cn & 1) == 0) {
            if (!mbar_wait(&k_full[k_stage(jn)], k_parity(jn), err)) { ok = false; break; }
          }
          if (c < n_cx) {
            if (!mbar_wait(&p_ready[2 * x + u], ((g0 + c) >> 1) & 1, err)) { ok = false; break; }
            tc_fence_after_sync();
            issue_pv(c);
            umma_commit(&pv_done[x], leader);
            if (c + 1 == n_cx) umma_commit(&o_done[x], leader);
            // score buffer u is free again once P_x(c) V_c has been issued (in-order pipe, same issuing thread)
            if (cn < n_cx) {
              issue_s(cn);
              if (cn + 1 == n_cx) umma_commit(q_empty, leader);  // that was this item's last score MMA of this tile
            }
          }
          if (u == 1) umma_commit(&v_empty[v_stage(j)], leader);
          if (cn < n_cmax && (cn & 1) == 1) umma_commit(&k_empty[k_stage(jn)], leader);
        }
        jg += w.n_max;
        g0 += n_cx;
        ++it;
      }
    }
  } else if (warp >= 4) {
    // ------------------------------ softmax + epilogue ------------------------------
    const int x = (warp - 4) >> 2;      // query tile of this warpgroup
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;  // row inside the query tile == TMEM lane
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    const uint32_t tm_s = tmem_base + x * BKV + lane_sel;
    const uint32_t tm_o = tmem_base + 256 + x * 128 + lane_sel;
    const uint64_t c2 = pack_f2(p.scale_log2, p.scale_log2);
    uint32_t g0 = 0;       // sub-blocks of earlier items of this query tile (always even)
    uint32_t n_done = 0;   // earlier items in which this query tile existed
    bool ok = true;
    for (int round = 0; round * int(gridDim.x) < n_items && ok; ++round) {
      const int t = fwd_item_index(round);
      if (t >= n_items) continue;
      const FwdItem w = fwd_item(p, t, n_pairs);
      const int q_row = w.q0 + x * BQ + r;
      const int my_n = w.n_kv[x];
      const int my_c = 2 * my_n;
      float m_used = -INFINITY;  // running maximum (log2 domain) the exponentials are taken against
      uint64_t l2 = 0ull, l2b = 0ull;  // four partial row sums (two packed pairs, for independent add chains)
      for (int c = 0; c < my_c; ++c) {
        const int u = c & 1;
        ok = mbar_wait(&s_full[2 * x + u], ((g0 + c) >> 1) & 1, err);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t tm_su = tm_s + u * BC;
        uint32_t sv[BC];  // raw scores of this row
        tmem_ld_x32(tm_su, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld_x32(tm_su + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_ld_wait();
        // columns of this sub-block visible to this row
        const int kv0 = c * BC;
        int lim = p.S - kv0;
        if (p.causal) lim = min(lim, q_row - kv0 + 1);
        // (no vote for the sub-blocks that every row of the tile sees in full: the common case)
        const bool all_visible = kv0 + BC <= p.S && (!p.causal || kv0 + BC - 1 <= w.q0 + x * BQ);
        if (!all_visible && __any_sync(0xffffffffu, lim < BC)) {
#pragma unroll
          for (int i = 0; i < BC; ++i)
            if (i >= lim) sv[i] = 0xff800000u;  // -inf
        }
        // four independent partial maxima: one long dependent chain would cost its full latency per sub-block
        float mp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) mp[k] = fmaxf(__uint_as_float(sv[2 * k]), __uint_as_float(sv[2 * k + 1]));
#pragma unroll
        for (int i = 8; i < BC; i += 8)
#pragma unroll
          for (int k = 0; k < 4; ++k) mp[k] = fmax3(mp[k], __uint_as_float(sv[i + 2 * k]), __uint_as_float(sv[i + 2 * k + 1]));
        const float m_raw = fmaxf(fmaxf(mp[0], mp[1]), fmaxf(mp[2], mp[3]));
        const float m_tile = m_raw * p.scale_log2;  // the scale is positive, so the maximum commutes with it
        float alpha = 1.f;
        bool rescale = false;
        if (c == 0) {
          m_used = m_tile;
        } else if (m_tile > m_used + kRescaleThreshold) {
          alpha = fast_exp2(m_used - m_tile);
          m_used = m_tile;
          l2 = fmul2(l2, pack_f2(alpha, alpha));
          l2b = fmul2(l2b, pack_f2(alpha, alpha));
          rescale = true;
        }
        const uint64_t nm2 = pack_f2(-m_used, -m_used);
#pragma unroll
        for (int g = 0; g < BC / 32; ++g) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint64_t e2 = ffma2(pack_f2(__uint_as_float(sv[g * 32 + 2 * i]), __uint_as_float(sv[g * 32 + 2 * i + 1])), c2, nm2);
            const uint64_t e = pack_f2(fast_exp2(f2_lo(e2)), fast_exp2(f2_hi(e2)));
            if (i & 1) l2b = fadd2(l2b, e); else l2 = fadd2(l2, e);
            pk[i] = pack_bf16(f2_lo(e), f2_hi(e));
          }
          tmem_st_x16(tm_su + g * 16, pk);  // P as bf16 pairs over the first 32 columns of this score buffer
        }
        // O_x may still be receiving P_x(c-1) V_(c-1): a rescale waits for that product first.  P_x(c) V_c is not
        // issued before this warpgroup's arrival below.
        if (c > 0 && __any_sync(0xffffffffu, rescale)) {
          bool wt = mbar_wait(&pv_done[x], (g0 + c - 1) & 1, err);
          if (!__all_sync(0xffffffffu, wt)) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int g = 0; g < DH / 32; ++g) {
            uint32_t tmp[32];
            tmem_ld_x32(tm_o + g * 32, tmp);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) tmp[i] = __float_as_uint(__uint_as_float(tmp[i]) * alpha);
            tmem_st_x32(tm_o + g * 32, tmp);
          }
        }
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(&p_ready[2 * x + u]);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (ok && my_n > 0) {
        bool wt = mbar_wait(&o_done[x], n_done & 1, err);
        ok = __all_sync(0xffffffffu, wt);
      }
      if (ok && my_n > 0) {
        tc_fence_after_sync();
        const float l_sum = (f2_lo(l2) + f2_hi(l2)) + (f2_lo(l2b) + f2_hi(l2b));
        const float inv_l = 1.f / l_sum;
        const bool valid = q_row < p.S;
        __nv_bfloat16* dst = p.o[w.layer] + ((size_t(w.b) * p.S + (valid ? q_row : 0)) * p.Hq + w.hq) * DH;
#pragma unroll
        for (int g = 0; g < DH / 32; ++g) {
          uint32_t tmp[32];
          tmem_ld_x32(tm_o + g * 32, tmp);
          tmem_ld_wait();
          if (g == DH / 32 - 1) {  // O_x has been read out: the next item's first P V product may overwrite it
            tc_fence_before_sync();
            mbar_arrive(&o_free[x]);
          }
          if (valid) {
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
              uint4 v;
              v.x = pack_bf16(__uint_as_float(tmp[8 * v4 + 0]) * inv_l, __uint_as_float(tmp[8 * v4 + 1]) * inv_l);
              v.y = pack_bf16(__uint_as_float(tmp[8 * v4 + 2]) * inv_l, __uint_as_float(tmp[8 * v4 + 3]) * inv_l);
              v.z = pack_bf16(__uint_as_float(tmp[8 * v4 + 4]) * inv_l, __uint_as_float(tmp[8 * v4 + 5]) * inv_l);
              v.w = pack_bf16(__uint_as_float(tmp[8 * v4 + 6]) * inv_l, __uint_as_float(tmp[8 * v4 + 7]) * inv_l);
              *reinterpret_cast<uint4*>(dst + g * 32 + v4 * 8) = v;
            }
          }
        }
        if (valid) p.lse[w.layer][(size_t(w.b) * p.Hq + w.hq) * p.S + q_row] = (m_used + log2f(l_sum)) * 0.6931471805599453f;
      } else if (ok) {
        mbar_arrive(&o_free[x]);  // this query tile does not exist in this item: nothing to read out
      }
      g0 += my_c;
      n_done += my_n > 0 ? 1 : 0;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

int make_map_bshd(CUtensorMap* m, const void* base, int B, int S, int H, int dh, int box_rows) {
  uint64_t dims[4] = {uint64_t(dh), uint64_t(H), uint64_t(S), uint64_t(B)};
  uint64_t strides[3] = {uint64_t(dh) * 2, uint64_t(H) * dh * 2, uint64_t(S) * H * dh * 2};
  uint32_t box[4] = {64, 1, uint32_t(box_rows), 1};
  return make_tensor_map(m, base, 2, 4, dims, strides, box, true);
}

}  // namespace

int attn_fwd_read_status() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_fwd_status, sizeof(int)) != cudaSuccess) return -1;
  if (v != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_fwd_status, &zero, sizeof(int));
  }
  return v;
}

// n layers (at most FWD_MAX_LAYERS) in one launch: q[i] [B,S,Hq,dh], k[i] / v[i] [B,S,Hkv,dh] of layer i's donor.
int attn_fwd_layers(const kvp_shape* s, int causal, float scale, const void* const* q, const void* const* k,
                    const void* const* v, void* const* o, float* const* lse, int n, cudaStream_t stream) {
  if (n < 1 || n > FWD_MAX_LAYERS) return KVP_ERR_INVALID_ARG;
  static thread_local FwdParams p;   // 3 KB of tensor maps: kept off the stack
  for (int i = 0; i < FWD_MAX_LAYERS; ++i) {
    const int l = i < n ? i : 0;
    int rc = make_map_bshd(&p.map_q[i], q[l], s->B, s->S, s->Hq, s->dh, BQ);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_k[i], k[l], s->B, s->S, s->Hkv, s->dh, BKV);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_v[i], v[l], s->B, s->S, s->Hkv, s->dh, BKV);
    if (rc != KVP_OK) return rc;
    p.o[i] = reinterpret_cast<__nv_bfloat16*>(o[l]);
    p.lse[i] = lse[l];
  }
  p.n_layers = n;
  p.B = s->B;
  p.S = s->S;
  p.Hq = s->Hq;
  p.Hkv = s->Hkv;
  p.causal = causal;
  const float sc = scale == 0.f ? 1.f / sqrtf(float(s->dh)) : scale;
  p.scale_log2 = sc * 1.4426950408889634f;
  const int n_qtiles = (s->S + BQ - 1) / BQ;
  const long long n_items = (long long)n * s->B * s->Hq * ((n_qtiles + 1) / 2);
  if (n_items > 0x7fffffffLL) return KVP_ERR_UNSUPPORTED;
  // persistent: one CTA per SM walks a list of (layer, b, hq, tile pair) items
  const int grid = int(n_items < (long long)sm_count() ? n_items : (long long)sm_count());
  static const cudaError_t attr128 =
      cudaFuncSetAttribute(attn_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<128>::TOTAL);
  static const cudaError_t attr64 =
      cudaFuncSetAttribute(attn_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<64>::TOTAL);
  if (attr128 != cudaSuccess || attr64 != cudaSuccess) return KVP_ERR_CUDA;
  timing_before(KVP_KERNEL_ATTN_FWD, stream);
  if (s->dh == 128) {
    attn_fwd_kernel<128><<<grid, FWD_THREADS, FwdSmem<128>::TOTAL, stream>>>(p);
  } else if (s->dh == 64) {
    attn_fwd_kernel<64><<<grid, FWD_THREADS, FwdSmem<64>::TOTAL, stream>>>(p);
  } else {
    return KVP_ERR_UNSUPPORTED;
  }
  timing_after(KVP_KERNEL_ATTN_FWD, stream);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

int attn_fwd_max_layers() { return FWD_MAX_LAYERS; }

}  // namespace kvp
