// Flash-attention backward over a donor map (chain rule of Eq. 2-3 of the paper).
//
// The unit of work is one 128-row K/V tile of one (batch, KV head) of a DONOR layer.  The CTA keeps
// that K/V tile in shared memory and its dK / dV accumulators in TMEM (fp32) while it walks every
// query stream that reads the tile: the donor itself and all its consumer layers, the Hq/Hkv query
// heads of the KV head's group, and every query tile the causal mask lets see the keys.  dK and dV
// of the donor are therefore summed on chip across layers and heads and written to HBM once.
//
// Per (layer, head, query tile), with everything transposed so that TMEM lane == key row:
//   S^T  = K Q^T,  dP^T = V dO^T                       (tcgen05, both operands K-major)
//   P^T  = exp2(S^T c - LSE),  dS^T = P^T (dP^T - Delta)   (one thread per key row)
//   dV  += P^T dO,   dK += dS^T Q                       (A from shared memory, B MN-major)
//   dQ   = dS K                                         (A = dS^T read MN-major, B = K MN-major)
// dQ tiles are added into an fp32 accumulator in the workspace with vector reductions and
// rounded to bf16 (times the softmax scale) by a small post-pass; Delta = rowsum(dO * O) comes
// from a pre-pass.
#include <math.h>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int BT = 128;            // tile rows for both queries and keys
constexpr int BWD_THREADS = 192;   // warp 0 TMA, warp 1 MMA, warps 2-5 compute
constexpr int MAX_GROUP = 8;       // layers of one donor group per launch
constexpr uint32_t HALF_BYTES = 128 * 128;

__device__ int g_bwd_status;

template <int DH>
struct BwdSmem {
  static constexpr int TILE = BT * DH * 2;       // K, V, Q, dO tiles
  static constexpr int PT = BT * BT * 2;         // P^T, dS^T tiles
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = OFF_K + TILE;
  static constexpr int OFF_Q = OFF_V + TILE;
  static constexpr int OFF_DO = OFF_Q + TILE;
  static constexpr int OFF_PT = OFF_DO + TILE;
  static constexpr int OFF_DST = OFF_PT + PT;
  static constexpr int OFF_LSE = OFF_DST + PT;   // 128 floats
  static constexpr int OFF_DELTA = OFF_LSE + 512;
  static constexpr int OFF_BAR = OFF_DELTA + 512;
  static constexpr int TOTAL = OFF_BAR + 128 + 1024;
};

struct BwdParams {
  CUtensorMap map_k, map_v;             // donor K, V: [B,S,Hkv,dh]
  CUtensorMap map_q[MAX_GROUP];         // per layer of the group: Q  [B,S,Hq,dh]
  CUtensorMap map_do[MAX_GROUP];        // per layer of the group: dO [B,S,Hq,dh]
  const float* lse[MAX_GROUP];          // [B,Hq,S]
  const float* delta[MAX_GROUP];        // [B,Hq,S]
  float* dq_acc[MAX_GROUP];             // fp32 [B,S,Hq,dh], zero-initialised
  float* dk_sum;                        // fp32 [B,S,Hkv,dh]
  float* dv_sum;
  int n_layers;
  int B, S, Hq, Hkv;
  int causal;
  float scale;
  float scale_log2;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}
__device__ __forceinline__ void compute_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int DH>
__global__ void __launch_bounds__(BWD_THREADS, 1) attn_bwd_kernel(const __grid_constant__ BwdParams p) {
  using L = BwdSmem<DH>;
  constexpr int HALVES = DH / 64;
  constexpr int KSTEPS_DH = DH / 16;
  constexpr int KSTEPS_T = BT / 16;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* kv_full = bars + 0;
  uint64_t* qdo_full = bars + 1;   // Q and dO of this iteration landed
  uint64_t* qdo_empty = bars + 2;  // MMAs that read Q, dO, P^T, dS^T have completed
  uint64_t* st_full = bars + 3;    // S^T and dP^T are in TMEM
  uint64_t* pds_ready = bars + 4;  // P^T, dS^T written to shared memory (128 arrivals)
  uint64_t* dq_full = bars + 5;    // dV, dK, dQ MMAs of this iteration have completed
  uint64_t* dq_free = bars + 6;    // dQ drained from TMEM (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  float* s_lse = reinterpret_cast<float*>(smem + L::OFF_LSE);
  float* s_delta = reinterpret_cast<float*>(smem + L::OFF_DELTA);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  int* err = &g_bwd_status;

  const int jt = blockIdx.x;  // key tile; tile 0 sees every query tile under the causal mask -> heaviest first
  const int hk = blockIdx.y;
  const int b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  const int kv0 = jt * BT;
  const int n_qt = (p.S + BT - 1) / BT;
  const int qt_first = p.causal ? jt : 0;
  const int per_stream = n_qt - qt_first;
  const int n_iter = p.n_layers * G * per_stream;

  if (threadIdx.x == 0) {
    mbar_init(kv_full, 1);
    mbar_init(qdo_full, 1);
    mbar_init(qdo_empty, 1);
    mbar_init(st_full, 1);
    mbar_init(pds_ready, 128);
    mbar_init(dq_full, 1);
    mbar_init(dq_free, 128);
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
  const uint32_t tm_st = tmem_base;         // S^T, 128 columns
  const uint32_t tm_dp = tmem_base + 128;   // dP^T, then dQ (aliased)
  const uint32_t tm_dk = tmem_base + 256;   // DH columns
  const uint32_t tm_dv = tmem_base + 384;   // DH columns

  auto decode_iter = [&](int it, int& li, int& hq, int& q0) {
    const int stream = it / per_stream;
    const int qi = it - stream * per_stream;
    li = stream / G;
    hq = hk * G + (stream - li * G);
    q0 = (qt_first + qi) * BT;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&p.map_k);
      tma_prefetch_desc(&p.map_v);
      mbar_expect_tx(kv_full, 2 * L::TILE);
#pragma unroll
      for (int h = 0; h < HALVES; ++h) {
        tma_load_4d(smem + L::OFF_K + h * HALF_BYTES, &p.map_k, kv_full, h * 64, hk, kv0, b);
        tma_load_4d(smem + L::OFF_V + h * HALF_BYTES, &p.map_v, kv_full, h * 64, hk, kv0, b);
      }
      for (int it = 0; it < n_iter; ++it) {
        int li, hq, q0;
        decode_iter(it, li, hq, q0);
        if (!mbar_wait(qdo_empty, (it & 1) ^ 1, err)) break;
        mbar_expect_tx(qdo_full, 2 * L::TILE);
#pragma unroll
        for (int h = 0; h < HALVES; ++h) {
          tma_load_4d(smem + L::OFF_Q + h * HALF_BYTES, &p.map_q[li], qdo_full, h * 64, hq, q0, b);
          tma_load_4d(smem + L::OFF_DO + h * HALF_BYTES, &p.map_do[li], qdo_full, h * 64, hq, q0, b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc_st = umma_idesc_bf16(BT, BT, 0, 0);
      constexpr uint32_t idesc_acc = umma_idesc_bf16(BT, DH, 0, 1);
      constexpr uint32_t idesc_dq = umma_idesc_bf16(BT, DH, 1, 1);
      const uint32_t sk = smem_u32(smem + L::OFF_K), sv = smem_u32(smem + L::OFF_V);
      const uint32_t sq = smem_u32(smem + L::OFF_Q), sdo = smem_u32(smem + L::OFF_DO);
      const uint32_t spt = smem_u32(smem + L::OFF_PT), sdst = smem_u32(smem + L::OFF_DST);
      bool ok = mbar_wait(kv_full, 0, err);
      for (int it = 0; it < n_iter && ok; ++it) {
        const uint32_t ph = it & 1;
        if (!mbar_wait(qdo_full, ph, err)) break;
        // S^T may be overwritten once the compute warps have read the previous one (pds_ready of
        // it-1, waited below); dP^T / dQ columns once dQ of it-1 has been drained.
        if (it > 0 && !mbar_wait(dq_free, ph ^ 1, err)) break;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          umma_ss(tm_st, smem_desc_sw128(sk + off, 0, 1024), smem_desc_sw128(sq + off, 0, 1024), idesc_st, ks != 0);
        }
#pragma unroll
        for (int ks = 0; ks < KSTEPS_DH; ++ks) {
          const uint32_t off = (ks / 4) * HALF_BYTES + (ks % 4) * 32;
          umma_ss(tm_dp, smem_desc_sw128(sv + off, 0, 1024), smem_desc_sw128(sdo + off, 0, 1024), idesc_st, ks != 0);
        }
        umma_commit(st_full);
        if (!mbar_wait(pds_ready, ph, err)) break;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < KSTEPS_T; ++ks) {  // dV += P^T dO
          const uint64_t da = smem_desc_sw128(spt + (ks / 4) * HALF_BYTES + (ks % 4) * 32, 0, 1024);
          const uint64_t db = smem_desc_sw128(sdo + ks * 2048, HALF_BYTES, 1024);
          umma_ss(tm_dv, da, db, idesc_acc, (it | ks) != 0);
        }
#pragma unroll
        for (int ks = 0; ks < KSTEPS_T; ++ks) {  // dK += dS^T Q
          const uint64_t da = smem_desc_sw128(sdst + (ks / 4) * HALF_BYTES + (ks % 4) * 32, 0, 1024);
          const uint64_t db = smem_desc_sw128(sq + ks * 2048, HALF_BYTES, 1024);
          umma_ss(tm_dk, da, db, idesc_acc, (it | ks) != 0);
        }
#pragma unroll
        for (int ks = 0; ks < KSTEPS_T; ++ks) {  // dQ = dS K   (A = dS^T tile read MN-major)
          const uint64_t da = smem_desc_sw128(sdst + ks * 2048, HALF_BYTES, 1024);
          const uint64_t db = smem_desc_sw128(sk + ks * 2048, HALF_BYTES, 1024);
          umma_ss(tm_dp, da, db, idesc_dq, ks != 0);
        }
        umma_commit(qdo_empty);
        umma_commit(dq_full);
      }
    }
  } else {
    // ------------------------------ compute warps ------------------------------
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;  // key row for S^T / dP^T, query row for dQ
    const int tid = r;
    const uint32_t lane_sel = uint32_t(quarter * 32) << 16;
    const int kv_row = kv0 + r;
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      int li, hq, q0;
      decode_iter(it, li, hq, q0);
      const uint32_t ph = it & 1;
      // stage LSE and Delta of the 128 query columns (visible to every thread after the barrier)
      {
        const int qc = q0 + tid;
        const size_t idx = (size_t(b) * p.Hq + hq) * p.S + qc;
        const float l2 = qc < p.S ? p.lse[li][idx] * 1.4426950408889634f : INFINITY;
        const float dl = qc < p.S ? p.delta[li][idx] : 0.f;
        compute_bar_sync();  // previous iteration's readers are done with the staging arrays
        s_lse[tid] = l2;
        s_delta[tid] = dl;
        compute_bar_sync();
      }
      ok = mbar_wait(st_full, ph, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      const bool diag = p.causal && (q0 < kv0 + BT);  // some (key, query) pairs of this tile are masked
#pragma unroll 1
      for (int c = 0; c < BT / 32; ++c) {
        uint32_t st[32], dp[32];
        tmem_ld_x32(tm_st + lane_sel + c * 32, st);
        tmem_ld_x32(tm_dp + lane_sel + c * 32, dp);
        tmem_ld_wait();
        uint32_t pt[16], ds[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float pv[2], dv[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int col = c * 32 + i + u;
            float pr = fast_exp2(__uint_as_float(st[i + u]) * p.scale_log2 - s_lse[col]);
            if (diag && (q0 + col < kv_row)) pr = 0.f;
            if (kv_row >= p.S) pr = 0.f;
            pv[u] = pr;
            dv[u] = pr * (__uint_as_float(dp[i + u]) - s_delta[col]);
          }
          pt[i / 2] = pack_bf16(pv[0], pv[1]);
          ds[i / 2] = pack_bf16(dv[0], dv[1]);
        }
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          const int chunk = c * 4 + v4;  // 16-byte chunk (8 query columns) of this key row
          const uint32_t off = (chunk / 8) * HALF_BYTES + sw128_offset(r, chunk % 8);
          *reinterpret_cast<uint4*>(smem + L::OFF_PT + off) =
              make_uint4(pt[4 * v4], pt[4 * v4 + 1], pt[4 * v4 + 2], pt[4 * v4 + 3]);
          *reinterpret_cast<uint4*>(smem + L::OFF_DST + off) =
              make_uint4(ds[4 * v4], ds[4 * v4 + 1], ds[4 * v4 + 2], ds[4 * v4 + 3]);
        }
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(pds_ready);

      ok = mbar_wait(dq_full, ph, err);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      tc_fence_after_sync();
      {
        const int q_row = q0 + r;
        float* dst = p.dq_acc[li] + ((size_t(b) * p.S + q_row) * p.Hq + hq) * DH;
#pragma unroll 1
        for (int c = 0; c < DH / 32; ++c) {
          uint32_t acc[32];
          tmem_ld_x32(tm_dp + lane_sel + c * 32, acc);
          tmem_ld_wait();
          if (q_row < p.S) {
#pragma unroll
            for (int v4 = 0; v4 < 8; ++v4)
              red_add_v4(dst + c * 32 + v4 * 4, __uint_as_float(acc[4 * v4]), __uint_as_float(acc[4 * v4 + 1]),
                         __uint_as_float(acc[4 * v4 + 2]), __uint_as_float(acc[4 * v4 + 3]));
          }
        }
      }
      tc_fence_before_sync();
      mbar_arrive(dq_free);
    }
    if (ok && n_iter > 0) {
      // dq_full of the last iteration also covers the last dV / dK MMAs
      tc_fence_after_sync();
      // tcgen05.ld is warp-collective: every lane loads, only rows inside the sequence store
      const bool valid = kv_row < p.S;
      const size_t row_off = ((size_t(b) * p.S + (valid ? kv_row : 0)) * p.Hkv + hk) * DH;
      float* dk = p.dk_sum + row_off;
      float* dv = p.dv_sum + row_off;
#pragma unroll 1
      for (int c = 0; c < DH / 32; ++c) {
        uint32_t a[32];
        tmem_ld_x32(tm_dk + lane_sel + c * 32, a);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int v4 = 0; v4 < 8; ++v4)
            *reinterpret_cast<float4*>(dk + c * 32 + v4 * 4) =
                make_float4(__uint_as_float(a[4 * v4]) * p.scale, __uint_as_float(a[4 * v4 + 1]) * p.scale,
                            __uint_as_float(a[4 * v4 + 2]) * p.scale, __uint_as_float(a[4 * v4 + 3]) * p.scale);
        }
        tmem_ld_x32(tm_dv + lane_sel + c * 32, a);
        tmem_ld_wait();
        if (valid) {
#pragma unroll
          for (int v4 = 0; v4 < 8; ++v4)
            *reinterpret_cast<float4*>(dv + c * 32 + v4 * 4) =
                make_float4(__uint_as_float(a[4 * v4]), __uint_as_float(a[4 * v4 + 1]), __uint_as_float(a[4 * v4 + 2]),
                            __uint_as_float(a[4 * v4 + 3]));
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

// Delta[b,hq,s] = sum_c dO[b,s,hq,c] * O[b,s,hq,c]; one warp per (token, head) row.
template <int DH>
__global__ void delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                             float* __restrict__ delta, int B, int S, int Hq) {
  const size_t rows = size_t(B) * S * Hq;
  const int lane = threadIdx.x & 31;
  const size_t warp_global = (size_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const size_t n_warps = (size_t(gridDim.x) * blockDim.x) >> 5;
  for (size_t row = warp_global; row < rows; row += n_warps) {
    float acc = 0.f;
    if (lane * 8 < DH) {  // DH/8 lanes each take 16 bytes
      const uint4 a = *reinterpret_cast<const uint4*>(o + row * DH + lane * 8);
      const uint4 g = *reinterpret_cast<const uint4*>(d_o + row * DH + lane * 8);
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 fa = __bfloat1622float2(pa[i]), fg = __bfloat1622float2(pg[i]);
        acc += fa.x * fg.x + fa.y * fg.y;
      }
    }
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
    if (lane == 0) {
      const int hq = int(row % Hq);
      const size_t tok = row / Hq;
      const int s = int(tok % S);
      const int b = int(tok / S);
      delta[(size_t(b) * Hq + hq) * S + s] = acc;
    }
  }
}

__global__ void dq_finish_kernel(const float4* __restrict__ acc, uint2* __restrict__ dq, size_t n4, float scale) {
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const float4 v = acc[i];
    dq[i] = make_uint2(pack_bf16(v.x * scale, v.y * scale), pack_bf16(v.z * scale, v.w * scale));
  }
}

int make_map_bshd(CUtensorMap* m, const void* base, int B, int S, int H, int dh) {
  uint64_t dims[4] = {uint64_t(dh), uint64_t(H), uint64_t(S), uint64_t(B)};
  uint64_t strides[3] = {uint64_t(dh) * 2, uint64_t(H) * dh * 2, uint64_t(S) * H * dh * 2};
  uint32_t box[4] = {64, 1, BT, 1};
  return make_tensor_map(m, base, 2, 4, dims, strides, box, true);
}

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

int max_group_size(int L, const int32_t* donor) {
  int best = 0;
  for (int d = 0; d < L; ++d) {
    if (donor[d] != d) continue;
    int n = 0;
    for (int l = d; l < L; ++l) n += donor[l] == d;
    best = n > best ? n : best;
  }
  return best;
}

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

// Workspace: Delta for the layers of one launch and the fp32 dQ accumulators of one launch.
size_t attn_bwd_workspace(const kvp_shape* s, const int32_t* donor) {
  int g = max_group_size(s->L, donor);
  if (g > MAX_GROUP) g = MAX_GROUP;
  const size_t delta = align256(size_t(s->B) * s->Hq * s->S * 4);
  const size_t dq = align256(size_t(s->B) * s->S * s->Hq * s->dh * 4);
  return size_t(g) * (delta + dq);
}

int attn_bwd_all(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                 const void* const* k, const void* const* v, const void* const* o, const void* const* d_o,
                 const float* const* lse, void* const* dq, float* const* dk_sum, float* const* dv_sum, void* ws,
                 size_t ws_bytes, cudaStream_t stream) {
  (void)ws_bytes;
  const int dh = s->dh;
  const float sc = scale == 0.f ? 1.f / sqrtf(float(dh)) : scale;
  const size_t delta_bytes = align256(size_t(s->B) * s->Hq * s->S * 4);
  const size_t dq_bytes = align256(size_t(s->B) * s->S * s->Hq * dh * 4);
  const size_t n_q = size_t(s->B) * s->S * s->Hq * dh;
  uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);
  int gmax = max_group_size(s->L, donor);
  if (gmax > MAX_GROUP) gmax = MAX_GROUP;
  uint8_t* ws_delta = wsb;
  uint8_t* ws_dq = wsb + size_t(gmax) * delta_bytes;
  cudaError_t e;
  if (dh == 128)
    e = cudaFuncSetAttribute(attn_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<128>::TOTAL);
  else
    e = cudaFuncSetAttribute(attn_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<64>::TOTAL);
  if (e != cudaSuccess) return KVP_ERR_CUDA;

  for (int d = 0; d < s->L; ++d) {
    if (donor[d] != d) continue;
    int members[64];
    int n = 0;
    for (int l = d; l < s->L; ++l)
      if (donor[l] == d) {
        if (n == MAX_GROUP) return KVP_ERR_UNSUPPORTED;  // more than MAX_GROUP layers share one donor
        members[n++] = l;
      }
    BwdParams p;
    int rc = make_map_bshd(&p.map_k, k[d], s->B, s->S, s->Hkv, dh);
    if (rc == KVP_OK) rc = make_map_bshd(&p.map_v, v[d], s->B, s->S, s->Hkv, dh);
    if (rc != KVP_OK) return rc;
    if (cudaMemsetAsync(ws_dq, 0, size_t(n) * dq_bytes, stream) != cudaSuccess) return KVP_ERR_CUDA;
    for (int i = 0; i < MAX_GROUP; ++i) {
      const int l = members[i < n ? i : 0];
      rc = make_map_bshd(&p.map_q[i], q[l], s->B, s->S, s->Hq, dh);
      if (rc == KVP_OK) rc = make_map_bshd(&p.map_do[i], d_o[l], s->B, s->S, s->Hq, dh);
      if (rc != KVP_OK) return rc;
      const int slot = i < n ? i : 0;
      p.lse[i] = lse[l];
      p.delta[i] = reinterpret_cast<const float*>(ws_delta + size_t(slot) * delta_bytes);
      p.dq_acc[i] = reinterpret_cast<float*>(ws_dq + size_t(slot) * dq_bytes);
    }
    for (int i = 0; i < n; ++i) {
      const int l = members[i];
      float* dl = reinterpret_cast<float*>(ws_delta + size_t(i) * delta_bytes);
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
    dim3 grid((s->S + BT - 1) / BT, s->Hkv, s->B);
    timing_before(KVP_KERNEL_ATTN_BWD, stream);
    if (dh == 128)
      attn_bwd_kernel<128><<<grid, BWD_THREADS, BwdSmem<128>::TOTAL, stream>>>(p);
    else
      attn_bwd_kernel<64><<<grid, BWD_THREADS, BwdSmem<64>::TOTAL, stream>>>(p);
    timing_after(KVP_KERNEL_ATTN_BWD, stream);
    note_launch(1 + 2 * n);  // main kernel, n delta pre-passes, n dQ finish passes
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
    for (int i = 0; i < n; ++i) {
      const int l = members[i];
      const size_t n4 = n_q / 4;
      const int blocks = int(min(size_t(sm_count()) * 8, (n4 + 255) / 256));
      dq_finish_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const float4*>(ws_dq + size_t(i) * dq_bytes),
                                                   reinterpret_cast<uint2*>(dq[l]), n4, sc);
    }
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
  }
  return KVP_OK;
}

}  // namespace kvp
