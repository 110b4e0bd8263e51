// Causal GQA flash-attention forward over a donor map (Eq. 2-3 of the paper): layer l attends
// with its own queries to the keys/values of layer donor[l].
//
// One CTA owns a 128-row query tile of one (batch, query head) and walks the donor's K/V tiles.
//   warp 0      TMA producer: Q once, then K_j / V_j into three-stage rings
//   warp 1      tcgen05.mma issuer: S_j = Q K_j^T into one of two TMEM score buffers, and
//               O += P_j V_j with P_j as the A operand FROM TMEM and V_j as an MN-major operand
//   warps 2-5   online softmax, one thread per query row (TMEM lane == row, so the row maximum
//               and sum need no cross-thread traffic); write P_j (bf16 pairs) back over the first
//               64 columns of its score buffer; rescale O in TMEM only when the running maximum
//               moved by more than 2^8
// QK_{j+1} is issued before the softmax of tile j finishes, so the tensor pipe works on the next
// scores while the exponentials of the current tile are computed.
#include <math.h>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int FWD_THREADS = 192;
constexpr int FWD_STAGES = 3;  // K and V rings: deep enough to hide the TMA latency of a tile
constexpr float kRescaleThreshold = 8.0f;  // log2 units

__device__ int g_fwd_status;

template <int DH>
struct FwdSmem {
  static constexpr int Q_BYTES = BQ * DH * 2;
  static constexpr int KV_BYTES = BKV * DH * 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + FWD_STAGES * KV_BYTES;
  static constexpr int OFF_BAR = OFF_V + FWD_STAGES * KV_BYTES;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;  // + alignment slack
};

struct FwdParams {
  CUtensorMap map_q, map_k, map_v;  // 4-D [B, S, H, dh] tensors, box {64, 1, 128, 1}
  __nv_bfloat16* o;                 // [B, S, Hq, dh]
  float* lse;                       // [B, Hq, S]
  int B, S, Hq, Hkv;
  int causal;
  float scale_log2;                 // scale * log2(e)
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int DH>
__global__ void __launch_bounds__(FWD_THREADS, 1) attn_fwd_kernel(const __grid_constant__ FwdParams p) {
  using L = FwdSmem<DH>;
  constexpr int KSTEPS_QK = DH / 16;   // K dimension of S = Q K^T is dh
  constexpr int KSTEPS_PV = BKV / 16;  // K dimension of O = P V is the kv tile
  constexpr int HALVES = DH / 64;      // 64-column (128-byte) blocks per row of Q / K / V
  constexpr uint32_t HALF_BYTES = 128 * 128;  // one [128 rows x 128 B] block

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;     // [FWD_STAGES]
  uint64_t* k_empty = bars + 4;    // [FWD_STAGES]
  uint64_t* v_full = bars + 7;     // [FWD_STAGES]
  uint64_t* v_empty = bars + 10;   // [FWD_STAGES]
  uint64_t* s_full = bars + 13;    // [2]
  uint64_t* s_free = bars + 15;    // [2]
  uint64_t* p_ready = bars + 17;   // [2]
  uint64_t* pv_done = bars + 19;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_fwd_status;

  const int hq = blockIdx.x % p.Hq;
  const int b = blockIdx.x / p.Hq;
  const int n_qtiles = (p.S + BQ - 1) / BQ;
  const int qt = n_qtiles - 1 - blockIdx.y;  // heaviest (deepest causal) tiles are dispatched first
  const int hk = hq / (p.Hq / p.Hkv);
  const int q0 = qt * BQ;
  const int kv_end = p.causal ? min(p.S, q0 + BQ) : p.S;
  const int n_kv = (kv_end + BKV - 1) / BKV;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < FWD_STAGES; ++i) {
      mbar_init(&k_full[i], 1);
      mbar_init(&k_empty[i], 1);
      mbar_init(&v_full[i], 1);
      mbar_init(&v_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&s_free[i], 128);
      mbar_init(&p_ready[i], 128);
    }
    mbar_init(pv_done, 1);
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
  const uint32_t tmem_s = tmem_base;        // two score buffers of 128 columns
  const uint32_t tmem_o = tmem_base + 256;  // DH columns

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&p.map_q);
      tma_prefetch_desc(&p.map_k);
      tma_prefetch_desc(&p.map_v);
      mbar_expect_tx(q_full, L::Q_BYTES);
#pragma unroll
      for (int h = 0; h < HALVES; ++h) tma_load_4d(smem + L::OFF_Q + h * HALF_BYTES, &p.map_q, q_full, h * 64, hq, q0, b);
      bool ok = true;
      for (int j = 0; j < n_kv && ok; ++j) {
        const int s = j % FWD_STAGES;
        const uint32_t ph = (j / FWD_STAGES) & 1;
        if (!mbar_wait(&k_empty[s], ph ^ 1, err)) { ok = false; break; }
        mbar_expect_tx(&k_full[s], L::KV_BYTES);
#pragma unroll
        for (int h = 0; h < HALVES; ++h)
          tma_load_4d(smem + L::OFF_K + s * L::KV_BYTES + h * HALF_BYTES, &p.map_k, &k_full[s], h * 64, hk, j * BKV, b);
        if (!mbar_wait(&v_empty[s], ph ^ 1, err)) { ok = false; break; }
        mbar_expect_tx(&v_full[s], L::KV_BYTES);
#pragma unroll
        for (int h = 0; h < HALVES; ++h)
          tma_load_4d(smem + L::OFF_V + s * L::KV_BYTES + h * HALF_BYTES, &p.map_v, &v_full[s], h * 64, hk, j * BKV, b);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_qk = umma_idesc_bf16(BQ, BKV, 0, 0);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(BQ, DH, 0, 1);
      constexpr uint32_t hi = desc_hi_sw128(1024);
      const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::OFF_Q), 0);
      bool ok = mbar_wait(q_full, 0, err);
      auto issue_qk = [&](int j) -> bool {
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        const int st = j % FWD_STAGES;
        if (j >= 2 && !mbar_wait(&s_free[s], ph ^ 1, err)) return false;
        if (!mbar_wait(&k_full[st], (j / FWD_STAGES) & 1, err)) return false;
        tc_fence_after_sync();
        const uint32_t k_lo = desc_lo_sw128(smem_u32(smem + L::OFF_K + st * L::KV_BYTES), 0);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_QK; ++ks) {
          const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          umma_ss_w(tmem_s + s * BKV, desc_lo_add(q_lo, off), desc_lo_add(k_lo, off), hi, idesc_qk, ks != 0);
        }
        umma_commit(&k_empty[st]);
        umma_commit(&s_full[s]);
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int j = 0; j < n_kv && ok; ++j) {
        if (j + 1 < n_kv && !issue_qk(j + 1)) { ok = false; break; }
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        const int st = j % FWD_STAGES;
        if (!mbar_wait(&p_ready[s], ph, err)) { ok = false; break; }
        if (!mbar_wait(&v_full[st], (j / FWD_STAGES) & 1, err)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t sv = smem_u32(smem + L::OFF_V + st * L::KV_BYTES);
#pragma unroll
        for (int ks = 0; ks < KSTEPS_PV; ++ks) {
          umma_ts_w(tmem_o, tmem_s + s * BKV + ks * 8, desc_lo_add(desc_lo_sw128(sv, HALF_BYTES), ks * 2048), hi,
                    idesc_pv, (j | ks) != 0);
        }
        umma_commit(&v_empty[st]);
        umma_commit(pv_done);
      }
    }
  } else {
    // ------------------------------ softmax + epilogue ------------------------------
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;  // row inside the query tile == TMEM lane
    const int q_row = q0 + r;
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    float m_used = -INFINITY;  // running maximum (log2 domain) the exponentials are taken against
    float l_sum = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      const int s = j & 1;
      const uint32_t ph = (j >> 1) & 1;
      ok = mbar_wait(&s_full[s], ph, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      float x[BKV];
#pragma unroll
      for (int c = 0; c < BKV / 32; ++c) {
        uint32_t tmp[32];
        tmem_ld_x32(tmem_s + lane_sel + s * BKV + c * 32, tmp);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) x[c * 32 + i] = __uint_as_float(tmp[i]) * p.scale_log2;
      }
      tc_fence_before_sync();
      mbar_arrive(&s_free[s]);

      // columns of this tile visible to this row
      const int kv0 = j * BKV;
      int lim = p.S - kv0;
      if (p.causal) lim = min(lim, q_row - kv0 + 1);
      if (lim < BKV) {
#pragma unroll
        for (int i = 0; i < BKV; ++i)
          if (i >= lim) x[i] = -INFINITY;
      }
      float m_tile = x[0];
#pragma unroll
      for (int i = 1; i < BKV; ++i) m_tile = fmaxf(m_tile, x[i]);
      float alpha = 1.f;
      bool rescale = false;
      if (j == 0) {
        m_used = m_tile;
      } else if (m_tile > m_used + kRescaleThreshold) {
        alpha = fast_exp2(m_used - m_tile);
        m_used = m_tile;
        l_sum *= alpha;
        rescale = true;
      }
#pragma unroll
      for (int c = 0; c < BKV / 64; ++c) {
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float e0 = fast_exp2(x[c * 64 + 2 * i] - m_used);
          const float e1 = fast_exp2(x[c * 64 + 2 * i + 1] - m_used);
          l_sum += e0 + e1;
          pk[i] = pack_bf16(e0, e1);
        }
        tmem_st_x32(tmem_s + lane_sel + s * BKV + c * 32, pk);
      }
      tmem_st_wait();
      if (j > 0) {
        // O may only be touched once P_{j-1} V_{j-1} has landed; this also protects the P buffer
        // that tile j+1 will overwrite.
        ok = mbar_wait(pv_done, (j - 1) & 1, err);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        tc_fence_after_sync();
        if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
          for (int c = 0; c < DH / 32; ++c) {
            uint32_t tmp[32];
            tmem_ld_x32(tmem_o + lane_sel + c * 32, tmp);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) tmp[i] = __float_as_uint(__uint_as_float(tmp[i]) * alpha);
            tmem_st_x32(tmem_o + lane_sel + c * 32, tmp);
          }
          tmem_st_wait();
        }
        tc_fence_before_sync();
      }
      mbar_arrive(&p_ready[s]);
    }
    if (ok) {
      ok = mbar_wait(pv_done, (n_kv - 1) & 1, err);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after_sync();
      const float inv_l = 1.f / l_sum;
      const bool valid = q_row < p.S;
      __nv_bfloat16* dst = p.o + ((size_t(b) * p.S + q_row) * p.Hq + hq) * DH;
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t tmp[32];
        tmem_ld_x32(tmem_o + lane_sel + c * 32, tmp);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(tmp[8 * v4 + 0]) * inv_l, __uint_as_float(tmp[8 * v4 + 1]) * inv_l);
            v.y = pack_bf16(__uint_as_float(tmp[8 * v4 + 2]) * inv_l, __uint_as_float(tmp[8 * v4 + 3]) * inv_l);
            v.z = pack_bf16(__uint_as_float(tmp[8 * v4 + 4]) * inv_l, __uint_as_float(tmp[8 * v4 + 5]) * inv_l);
            v.w = pack_bf16(__uint_as_float(tmp[8 * v4 + 6]) * inv_l, __uint_as_float(tmp[8 * v4 + 7]) * inv_l);
            *reinterpret_cast<uint4*>(dst + c * 32 + v4 * 8) = v;
          }
        }
      }
      if (valid) p.lse[(size_t(b) * p.Hq + hq) * p.S + q_row] = (m_used + log2f(l_sum)) * 0.6931471805599453f;
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

// One layer: q [B,S,Hq,dh], k/v [B,S,Hkv,dh] of the layer's donor.
int attn_fwd_layer(const kvp_shape* s, int causal, float scale, const void* q, const void* k, const void* v, void* o,
                   float* lse, cudaStream_t stream) {
  FwdParams p;
  int rc = make_map_bshd(&p.map_q, q, s->B, s->S, s->Hq, s->dh, BQ);
  if (rc == KVP_OK) rc = make_map_bshd(&p.map_k, k, s->B, s->S, s->Hkv, s->dh, BKV);
  if (rc == KVP_OK) rc = make_map_bshd(&p.map_v, v, s->B, s->S, s->Hkv, s->dh, BKV);
  if (rc != KVP_OK) return rc;
  p.o = reinterpret_cast<__nv_bfloat16*>(o);
  p.lse = lse;
  p.B = s->B;
  p.S = s->S;
  p.Hq = s->Hq;
  p.Hkv = s->Hkv;
  p.causal = causal;
  const float sc = scale == 0.f ? 1.f / sqrtf(float(s->dh)) : scale;
  p.scale_log2 = sc * 1.4426950408889634f;
  dim3 grid(s->B * s->Hq, (s->S + BQ - 1) / BQ);
  cudaError_t e;
  timing_before(KVP_KERNEL_ATTN_FWD, stream);
  if (s->dh == 128) {
    e = cudaFuncSetAttribute(attn_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<128>::TOTAL);
    if (e != cudaSuccess) return KVP_ERR_CUDA;
    attn_fwd_kernel<128><<<grid, FWD_THREADS, FwdSmem<128>::TOTAL, stream>>>(p);
  } else if (s->dh == 64) {
    e = cudaFuncSetAttribute(attn_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<64>::TOTAL);
    if (e != cudaSuccess) return KVP_ERR_CUDA;
    attn_fwd_kernel<64><<<grid, FWD_THREADS, FwdSmem<64>::TOTAL, stream>>>(p);
  } else {
    return KVP_ERR_UNSUPPORTED;
  }
  timing_after(KVP_KERNEL_ATTN_FWD, stream);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? KVP_OK : KVP_ERR_CUDA;
}

}  // namespace kvp
