// Split-KV decode attention over the shared paged cache, and the cache append.
//
// A work unit is (donor group, sequence, KV head, split).  The CTA streams its share of the DONOR's
// K/V pages from HBM exactly once and applies them to every query row that reads them: the Hq/Hkv
// query heads of the KV head's group for the donor layer AND for each consumer layer of the group
// (Eq. 3 of the paper: consumers reuse the donor's K/V), up to 16 rows, as the M dimension of
// mma.sync m16n8k16 (bf16 in, fp32 accumulate).  The kernel is bound by HBM bandwidth, so the
// design is about bytes in flight: every warp owns a three-stage ring of 16-token granules (8 KB:
// 4 KB of K, 4 KB of V) filled by 16-byte cp.async copies that are fully coalesced (a page block
// of one KV head is contiguous), two CTAs per SM, and no transposes in HBM -- V fragments come from
// ldmatrix.trans on the swizzled ring.  Partial (max, sum, output) triples per split are merged by
// a second small kernel.
#include <math.h>

#include <mutex>

#include "kvp_host.h"
#include "kvp_sm100.cuh"

namespace kvp {
namespace {

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;
constexpr int GRAN = 16;           // tokens per ring stage
constexpr int DEC_STAGES = 3;
constexpr int MAX_DEC_GROUPS = 64;
constexpr int MAX_MEMBERS = 4;     // layers of a donor group served by one pass (rows = members * G <= 16)

__device__ int g_dec_status;

struct DecGroup {
  const __nv_bfloat16* k_cache;
  const __nv_bfloat16* v_cache;
  const void* q[MAX_MEMBERS];            // [B,Hq,dh], bf16 or (io_f32) fp32
  void* o[MAX_MEMBERS];                  // [B,Hq,dh], bf16 or (io_f32) fp32
  float* lse[MAX_MEMBERS];               // [B,Hq]
  int n_members;
  int pad;
};

struct DecParams {
  DecGroup grp[MAX_DEC_GROUPS];
  const int32_t* block_table;  // [B, max_pages]
  const int32_t* lengths;      // [B]
  float* part_o;               // [n_groups][B][Hkv][NS][16][DH]
  float* part_ml;              // [n_groups][B][Hkv][NS][16][2]
  int B, Hq, Hkv, page_size, max_pages, n_pages, num_splits;
  int io_f32;                  // queries are read and outputs written as fp32 (rounded to bf16 on load / widened on store)
  float scale_log2;
};

// 16-byte asynchronous copy; with src_bytes == 0 nothing is read and the destination is filled with zeros
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Ring stage layout: GRAN rows of DH bf16 (DH*2 bytes per row) for K, then the same for V.  The
// 16-byte chunk index is XOR-ed with (row & 7) so that ldmatrix reads are bank-conflict free.
template <int DH>
__device__ __forceinline__ uint32_t ring_off(int row, int chunk) {
  return uint32_t(row) * (DH * 2) + (uint32_t(chunk ^ (row & 7)) << 4);
}

template <int DH>
__global__ void __launch_bounds__(DEC_THREADS, 2) decode_kernel(const __grid_constant__ DecParams p) {
  constexpr int ROW_BYTES = DH * 2;
  constexpr int CHUNKS = ROW_BYTES / 16;           // 16-byte chunks per row
  constexpr int TILE_BYTES = GRAN * ROW_BYTES;     // K (or V) part of a stage
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  constexpr int CP_PER_LANE = TILE_BYTES / 16 / 32;
  constexpr int KSTEPS = DH / 16;
  constexpr int NBLK = DH / 8;

  extern __shared__ __align__(128) uint8_t dsmem[];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;

  const int split = blockIdx.x;
  const int b = blockIdx.y / p.Hkv;
  const int hk = blockIdx.y % p.Hkv;
  const int gi = blockIdx.z;
  const DecGroup& grp = p.grp[gi];
  const int G = p.Hq / p.Hkv;
  const int R = grp.n_members * G;  // valid query rows (<= 16)

  int len = p.lengths[b];
  const int cap = p.max_pages * p.page_size;
  if (len < 1 || len > cap) {
    if (threadIdx.x == 0) atomicOr(&g_dec_status, 2);  // clamped length
    len = len < 1 ? 1 : cap;
  }
  // this split's token range, in whole granules
  const int n_gran = (len + GRAN - 1) / GRAN;
  const int gran_per_split = (n_gran + p.num_splits - 1) / p.num_splits;
  const int gran_begin = split * gran_per_split;
  const int gran_end = min(n_gran, gran_begin + gran_per_split);

  // ---- query fragments (A operand, rows = members x heads of the group, zero beyond R) ----
  uint32_t qa[KSTEPS][4];
  {
    const int r0 = g, r1 = g + 8;
    const size_t off0 = r0 < R ? (size_t(b) * p.Hq + hk * G + r0 % G) * DH : 0;
    const size_t off1 = r1 < R ? (size_t(b) * p.Hq + hk * G + r1 % G) * DH : 0;
    auto pair_at = [&](const void* base, size_t off, int c) -> uint32_t {   // elements c, c+1 of a query row as bf16
      if (p.io_f32) {
        const float2 f = *reinterpret_cast<const float2*>(reinterpret_cast<const float*>(base) + off + c);
        return pack_bf16(f.x, f.y);
      }
      return *reinterpret_cast<const uint32_t*>(reinterpret_cast<const __nv_bfloat16*>(base) + off + c);
    };
    const void* q0 = r0 < R ? grp.q[r0 / G] : nullptr;
    const void* q1 = r1 < R ? grp.q[r1 / G] : nullptr;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      const int c = ks * 16 + t * 2;
      qa[ks][0] = q0 ? pair_at(q0, off0, c) : 0u;
      qa[ks][1] = q1 ? pair_at(q1, off1, c) : 0u;
      qa[ks][2] = q0 ? pair_at(q0, off0, c + 8) : 0u;
      qa[ks][3] = q1 ? pair_at(q1, off1, c + 8) : 0u;
    }
  }

  float oacc[NBLK][4];
#pragma unroll
  for (int n = 0; n < NBLK; ++n) oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};  // rows g, g+8 (log2 domain)
  float l_run[2] = {0.f, 0.f};              // per-lane partial sums

  uint8_t* ring = dsmem + size_t(warp) * DEC_STAGES * STAGE_BYTES;
  const uint32_t ring_u32 = smem_u32(ring);
  const int32_t* bt = p.block_table + size_t(b) * p.max_pages;

  auto issue = [&](int gran, int stage) {
    const int tok = gran * GRAN;
    int page = bt[tok / p.page_size];
    page = min(max(page, 0), p.n_pages - 1);
    const size_t elem = ((size_t(page) * p.Hkv + hk) * p.page_size + tok % p.page_size) * DH;
    const uint8_t* ksrc = reinterpret_cast<const uint8_t*>(grp.k_cache + elem);
    const uint8_t* vsrc = reinterpret_cast<const uint8_t*>(grp.v_cache + elem);
    const uint32_t dst = ring_u32 + stage * STAGE_BYTES;
#pragma unroll
    for (int i = 0; i < CP_PER_LANE; ++i) {
      const int idx = i * 32 + lane;          // 16-byte chunk index inside the contiguous granule
      const int row = idx / CHUNKS, chunk = idx % CHUNKS;
      const uint32_t off = ring_off<DH>(row, chunk);
      // Slots at or past the sequence length were never appended and may hold anything (a NaN there would
      // survive the zero probability in P V): they are filled with zeros instead of being read.
      const uint32_t nbytes = tok + row < len ? 16u : 0u;
      cp_async16(dst + off, ksrc + size_t(idx) * 16, nbytes);
      cp_async16(dst + TILE_BYTES + off, vsrc + size_t(idx) * 16, nbytes);
    }
  };

  // granules of the split are dealt round-robin to the warps
  const int first = gran_begin + warp;
  int n_mine = first < gran_end ? (gran_end - first + DEC_WARPS - 1) / DEC_WARPS : 0;
#pragma unroll
  for (int s = 0; s < DEC_STAGES - 1; ++s) {
    if (s < n_mine) issue(first + s * DEC_WARPS, s);
    cp_async_commit();
  }
  for (int i = 0; i < n_mine; ++i) {
    cp_async_wait<DEC_STAGES - 2>();
    __syncwarp();
    // prefetch granule i + STAGES-1 into the stage freed by iteration i-1
    {
      const int nx = i + DEC_STAGES - 1;
      if (nx < n_mine) issue(first + nx * DEC_WARPS, nx % DEC_STAGES);
      cp_async_commit();
    }
    const int gran = first + i * DEC_WARPS;
    const uint32_t sK = ring_u32 + (i % DEC_STAGES) * STAGE_BYTES;
    const uint32_t sV = sK + TILE_BYTES;

    // ---- S[16 rows, 16 tokens] = Q K^T ----
    float sacc[2][4];
#pragma unroll
    for (int nb = 0; nb < 2; ++nb) sacc[nb][0] = sacc[nb][1] = sacc[nb][2] = sacc[nb][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      // four 8x8 matrices: (tokens 0-7, dh ks*16..+7), (tokens 0-7, +8..15), (tokens 8-15, ...), (tokens 8-15, +8)
      const int mat = lane >> 3, rr = lane & 7;
      const int row = (mat >> 1) * 8 + rr;
      const int chunk = ks * 2 + (mat & 1);
      uint32_t b00, b01, b10, b11;
      ldsm_x4(sK + ring_off<DH>(row, chunk), b00, b01, b10, b11);
      mma_bf16(sacc[0], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b00, b01);
      mma_bf16(sacc[1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b10, b11);
    }
    // ---- online softmax over the 16 tokens ----
    const int tok0 = gran * GRAN;
    float mt[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nb = 0; nb < 2; ++nb) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int tk = tok0 + nb * 8 + t * 2 + (u & 1);
        float x = sacc[nb][u] * p.scale_log2;
        if (tk >= len) x = -INFINITY;
        sacc[nb][u] = x;
        mt[u >> 1] = fmaxf(mt[u >> 1], x);
      }
    }
    float alpha[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mt[h] = fmaxf(mt[h], __shfl_xor_sync(0xffffffffu, mt[h], 1));
      mt[h] = fmaxf(mt[h], __shfl_xor_sync(0xffffffffu, mt[h], 2));
      const float m_new = fmaxf(m_run[h], mt[h]);
      alpha[h] = m_run[h] == -INFINITY ? 0.f : fast_exp2(m_run[h] - m_new);
      m_run[h] = m_new;
      l_run[h] *= alpha[h];
    }
    uint32_t pa[4];
    {
      float pr[2][4];
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          pr[nb][u] = fast_exp2(sacc[nb][u] - m_run[u >> 1]);
          l_run[u >> 1] += pr[nb][u];
        }
      pa[0] = pack_bf16(pr[0][0], pr[0][1]);
      pa[1] = pack_bf16(pr[0][2], pr[0][3]);
      pa[2] = pack_bf16(pr[1][0], pr[1][1]);
      pa[3] = pack_bf16(pr[1][2], pr[1][3]);
    }
    if (!__all_sync(0xffffffffu, alpha[0] == 1.f && alpha[1] == 1.f)) {
#pragma unroll
      for (int n = 0; n < NBLK; ++n) {
        oacc[n][0] *= alpha[0];
        oacc[n][1] *= alpha[0];
        oacc[n][2] *= alpha[1];
        oacc[n][3] *= alpha[1];
      }
    }
    // ---- O[16 rows, DH] += P[16 rows, 16 tokens] V[16 tokens, DH] ----
#pragma unroll
    for (int n2 = 0; n2 < NBLK / 2; ++n2) {
      // four 8x8 matrices (transposed on load): (tokens 0-7, dh n2*16..+7), (tokens 8-15, same dh),
      // (tokens 0-7, dh +8..15), (tokens 8-15, dh +8..15)
      const int mat = lane >> 3, rr = lane & 7;
      const int row = (mat & 1) * 8 + rr;
      const int chunk = n2 * 2 + (mat >> 1);
      uint32_t v00, v01, v10, v11;
      ldsm_x4_t(sV + ring_off<DH>(row, chunk), v00, v01, v10, v11);
      mma_bf16(oacc[2 * n2], pa[0], pa[1], pa[2], pa[3], v00, v01);
      mma_bf16(oacc[2 * n2 + 1], pa[0], pa[1], pa[2], pa[3], v10, v11);
    }
    __syncwarp();  // every lane is done with this stage before it is refilled
  }
  cp_async_wait<0>();

  // ---- merge the four warps of the CTA, then write this split's partial ----
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
  }
  __syncthreads();  // all rings are idle: reuse the memory
  float* s_o = reinterpret_cast<float*>(dsmem);                   // [DEC_WARPS][16][DH]
  float* s_ml = s_o + DEC_WARPS * 16 * DH;                        // [DEC_WARPS][16][2]
#pragma unroll
  for (int n = 0; n < NBLK; ++n) {
    float* base = s_o + (size_t(warp) * 16) * DH + n * 8 + t * 2;
    base[size_t(g) * DH] = oacc[n][0];
    base[size_t(g) * DH + 1] = oacc[n][1];
    base[size_t(g + 8) * DH] = oacc[n][2];
    base[size_t(g + 8) * DH + 1] = oacc[n][3];
  }
  if (t == 0) {
    s_ml[(warp * 16 + g) * 2] = m_run[0];
    s_ml[(warp * 16 + g) * 2 + 1] = l_run[0];
    s_ml[(warp * 16 + g + 8) * 2] = m_run[1];
    s_ml[(warp * 16 + g + 8) * 2 + 1] = l_run[1];
  }
  __syncthreads();
  const size_t unit = ((size_t(gi) * p.B + b) * p.Hkv + hk) * p.num_splits + split;
  float* po = p.part_o + unit * 16 * DH;
  float* pml = p.part_ml + unit * 16 * 2;
  for (int idx = threadIdx.x; idx < R * DH; idx += DEC_THREADS) {
    const int row = idx / DH, col = idx % DH;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) mm = fmaxf(mm, s_ml[(w * 16 + row) * 2]);
    float acc = 0.f, ll = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
      const float mw = s_ml[(w * 16 + row) * 2];
      const float f = mw == -INFINITY ? 0.f : fast_exp2(mw - mm);
      acc += f * s_o[(size_t(w) * 16 + row) * DH + col];
      ll += f * s_ml[(w * 16 + row) * 2 + 1];
    }
    po[size_t(row) * DH + col] = acc;
    if (col == 0) {
      pml[row * 2] = mm;
      pml[row * 2 + 1] = ll;
    }
  }
}

// One CTA per (group, sequence, KV head): merge the splits and write bf16 outputs and LSE.
template <int DH>
__global__ void decode_combine_kernel(const __grid_constant__ DecParams p) {
  const int b = blockIdx.y / p.Hkv;
  const int hk = blockIdx.y % p.Hkv;
  const int gi = blockIdx.z;
  const DecGroup& grp = p.grp[gi];
  const int G = p.Hq / p.Hkv;
  const int R = grp.n_members * G;
  const size_t unit0 = ((size_t(gi) * p.B + b) * p.Hkv + hk) * p.num_splits;
  for (int idx = threadIdx.x; idx < R * DH; idx += blockDim.x) {
    const int row = idx / DH, col = idx % DH;
    float mm = -INFINITY;
    for (int s = 0; s < p.num_splits; ++s) mm = fmaxf(mm, p.part_ml[((unit0 + s) * 16 + row) * 2]);
    float acc = 0.f, ll = 0.f;
    for (int s = 0; s < p.num_splits; ++s) {
      const float ms = p.part_ml[((unit0 + s) * 16 + row) * 2];
      const float f = ms == -INFINITY ? 0.f : fast_exp2(ms - mm);
      acc += f * p.part_o[((unit0 + s) * 16 + row) * DH + col];
      ll += f * p.part_ml[((unit0 + s) * 16 + row) * 2 + 1];
    }
    const int mem = row / G, hq = hk * G + row % G;
    const __nv_bfloat16 val = __float2bfloat16_rn(acc / ll);   // rounded to bf16 either way: one set of results
    const size_t at = (size_t(b) * p.Hq + hq) * DH + col;
    if (p.io_f32) reinterpret_cast<float*>(grp.o[mem])[at] = __bfloat162float(val);
    else reinterpret_cast<__nv_bfloat16*>(grp.o[mem])[at] = val;
    if (col == 0) grp.lse[mem][size_t(b) * p.Hq + hq] = (mm + log2f(ll)) * 0.6931471805599453f;
  }
}

// Owners write the new token's K and V rows into their pages.
struct AppendParams {
  const void* k_new[MAX_DEC_GROUPS];   // [B,Hkv,dh] bf16, or fp32 when new_f32 (rounded to bf16 as it is stored)
  const void* v_new[MAX_DEC_GROUPS];
  __nv_bfloat16* k_cache[MAX_DEC_GROUPS];
  __nv_bfloat16* v_cache[MAX_DEC_GROUPS];
  const int32_t* block_table;
  const int32_t* lengths;
  int B, Hkv, dh, page_size, max_pages, n_pages;
  int new_f32;
};

__global__ void append_kernel(const __grid_constant__ AppendParams p) {
  const int layer = blockIdx.y;
  const int b = blockIdx.x;
  int len = p.lengths[b];
  const int cap = p.max_pages * p.page_size;
  if (len < 1 || len > cap) return;  // nothing sensible to write; decode flags the bad length
  const int pos = len - 1;
  int page = p.block_table[size_t(b) * p.max_pages + pos / p.page_size];
  if (page < 0 || page >= p.n_pages) return;
  const int row_chunks = p.dh / 8;  // 16-byte chunks per head row
  for (int idx = threadIdx.x; idx < p.Hkv * row_chunks; idx += blockDim.x) {
    const int hk = idx / row_chunks, c = idx % row_chunks;
    const size_t src = (size_t(b) * p.Hkv + hk) * p.dh + c * 8;
    const size_t dst = ((size_t(page) * p.Hkv + hk) * p.page_size + pos % p.page_size) * p.dh + c * 8;
    auto eight = [&](const void* base) -> uint4 {   // eight consecutive elements as bf16
      if (p.new_f32) {
        const float4 a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + src);
        const float4 c4 = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + src + 4);
        return make_uint4(pack_bf16(a.x, a.y), pack_bf16(a.z, a.w), pack_bf16(c4.x, c4.y), pack_bf16(c4.z, c4.w));
      }
      return *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + src);
    };
    *reinterpret_cast<uint4*>(p.k_cache[layer] + dst) = eight(p.k_new[layer]);
    *reinterpret_cast<uint4*>(p.v_cache[layer] + dst) = eight(p.v_new[layer]);
  }
}

int check_desc(const kvp_decode_desc* d) {
  if (d == nullptr) return KVP_ERR_INVALID_ARG;
  if (d->L < 1 || d->B < 1 || d->Hq < 1 || d->Hkv < 1 || d->max_pages < 1 || d->n_pages < 1 || d->num_splits < 0)
    return KVP_ERR_INVALID_ARG;
  if (d->dtype != KVP_BF16 && d->dtype != KVP_F32) return KVP_ERR_UNSUPPORTED;
  if ((d->dh != 64 && d->dh != 128) || d->Hq % d->Hkv != 0 || d->Hq / d->Hkv > 16 || d->page_size < GRAN ||
      d->page_size % GRAN != 0)
    return KVP_ERR_UNSUPPORTED;
  return KVP_OK;
}

int pick_splits(const kvp_decode_desc* d) {
  if (d->num_splits > 0) return d->num_splits;
  const long long cap = (long long)d->max_pages * d->page_size;
  long long ns = (cap + 2047) / 2048;
  if (ns < 1) ns = 1;
  if (ns > 32) ns = 32;
  return int(ns);
}

// Sub-groups of at most min(MAX_MEMBERS, 16 / G) layers that share a donor inside [begin, end).
struct SubGroup {
  int owner;
  int members[MAX_MEMBERS];
  int n;
};

int build_groups(const kvp_decode_desc* d, const int32_t* donor, int begin, int end, SubGroup* out, int max_out) {
  const int G = d->Hq / d->Hkv;
  int per = 16 / G;
  if (per > MAX_MEMBERS) per = MAX_MEMBERS;
  int n_out = 0;
  for (int own = 0; own < d->L; ++own) {
    if (donor[own] != own) continue;
    SubGroup cur;
    cur.owner = own;
    cur.n = 0;
    for (int l = begin > own ? begin : own; l < end; ++l) {
      if (donor[l] != own) continue;
      cur.members[cur.n++] = l;
      if (cur.n == per) {
        if (n_out == max_out) return -1;
        out[n_out++] = cur;
        cur.n = 0;
      }
    }
    if (cur.n > 0) {
      if (n_out == max_out) return -1;
      out[n_out++] = cur;
    }
  }
  return n_out;
}

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

// Bytes of per-split partials that decoding layers [begin, end) needs: one launch holds at most MAX_DEC_GROUPS
// sub-groups and launches reuse the space.  0 when the request cannot be served at all.
size_t decode_scratch_bytes(const kvp_decode_desc* d, const int32_t* donor, int begin, int end) {
  static thread_local SubGroup tmp[4096];
  const int n_sub = build_groups(d, donor, begin, end, tmp, 4096);
  if (n_sub <= 0) return 0;
  const int per_launch = n_sub < MAX_DEC_GROUPS ? n_sub : MAX_DEC_GROUPS;
  const size_t units = size_t(per_launch) * d->B * d->Hkv * pick_splits(d);
  return align256(units * 16 * d->dh * 4) + align256(units * 16 * 2 * 4);
}

}  // namespace

int decode_read_status() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_dec_status, sizeof(int)) != cudaSuccess) return -1;
  if (v != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_dec_status, &zero, sizeof(int));
  }
  return v & 1;  // bit 1 (clamped length) is informational
}

}  // namespace kvp

using namespace kvp;

extern "C" size_t kvp_decode_workspace_bytes(const kvp_decode_desc* d, const int32_t* donor) {
  if (check_desc(d) != KVP_OK || donor == nullptr) return 0;
  return decode_scratch_bytes(d, donor, 0, d->L);
}

extern "C" int kvp_cache_append(const kvp_decode_desc* d, const int32_t* donor, const void* const* k_new,
                                const void* const* v_new, void* const* k_cache, void* const* v_cache,
                                const int32_t* block_table, const int32_t* lengths, kvp_stream_t stream_) {
  int rc = check_desc(d);
  if (rc != KVP_OK) return rc;
  if (donor == nullptr || k_new == nullptr || v_new == nullptr || k_cache == nullptr || v_cache == nullptr ||
      block_table == nullptr || lengths == nullptr)
    return KVP_ERR_INVALID_ARG;
  for (int l = 0; l < d->L; ++l)
    if (donor[l] < 0 || donor[l] > l || donor[donor[l]] != donor[l]) return KVP_ERR_BAD_DONOR;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  AppendParams p;
  p.block_table = block_table;
  p.lengths = lengths;
  p.B = d->B;
  p.Hkv = d->Hkv;
  p.dh = d->dh;
  p.page_size = d->page_size;
  p.max_pages = d->max_pages;
  p.n_pages = d->n_pages;
  p.new_f32 = d->dtype == KVP_F32;
  int n = 0;
  for (int l = 0; l <= d->L; ++l) {
    const bool owner = l < d->L && donor[l] == l;  // consumers store nothing (Eq. 3)
    if (owner) {
      if (k_new[l] == nullptr || v_new[l] == nullptr || k_cache[l] == nullptr || v_cache[l] == nullptr)
        return KVP_ERR_INVALID_ARG;
      p.k_new[n] = k_new[l];
      p.v_new[n] = v_new[l];
      p.k_cache[n] = reinterpret_cast<__nv_bfloat16*>(k_cache[l]);
      p.v_cache[n] = reinterpret_cast<__nv_bfloat16*>(v_cache[l]);
      ++n;
    }
    if (n == MAX_DEC_GROUPS || (l == d->L && n > 0)) {
      append_kernel<<<dim3(d->B, n), 128, 0, stream>>>(p);
      note_launch();
      if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
      n = 0;
    }
  }
  return KVP_OK;
}

extern "C" int kvp_decode(const kvp_decode_desc* d, const int32_t* donor, float scale, const void* const* q,
                          const void* const* k_cache, const void* const* v_cache, const int32_t* block_table,
                          const int32_t* lengths, void* const* o, float* const* lse, int layer_begin, int layer_end,
                          void* ws, size_t ws_bytes, kvp_stream_t stream_) {
  int rc = check_desc(d);
  if (rc != KVP_OK) return rc;
  if (donor == nullptr || q == nullptr || k_cache == nullptr || v_cache == nullptr || block_table == nullptr ||
      lengths == nullptr || o == nullptr || lse == nullptr || scale < 0.f)
    return KVP_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end > d->L || layer_begin >= layer_end) return KVP_ERR_INVALID_ARG;
  for (int l = 0; l < d->L; ++l)
    if (donor[l] < 0 || donor[l] > l || donor[donor[l]] != donor[l]) return KVP_ERR_BAD_DONOR;
  static thread_local SubGroup subs[4096];
  const int n_sub = build_groups(d, donor, layer_begin, layer_end, subs, 4096);
  if (n_sub < 0) return KVP_ERR_UNSUPPORTED;
  const int ns = pick_splits(d);
  const int per_launch = n_sub < MAX_DEC_GROUPS ? n_sub : MAX_DEC_GROUPS;
  const size_t units = size_t(per_launch) * d->B * d->Hkv * ns;
  const size_t po_bytes = align256(units * 16 * d->dh * 4), pml_bytes = align256(units * 16 * 2 * 4);
  if (ws == nullptr || ws_bytes < po_bytes + pml_bytes || !aligned16(ws)) return KVP_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);

  DecParams p;
  p.block_table = block_table;
  p.lengths = lengths;
  p.part_o = reinterpret_cast<float*>(ws);
  p.part_ml = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(ws) + po_bytes);
  p.B = d->B;
  p.Hq = d->Hq;
  p.Hkv = d->Hkv;
  p.page_size = d->page_size;
  p.max_pages = d->max_pages;
  p.n_pages = d->n_pages;
  p.num_splits = ns;
  p.io_f32 = d->dtype == KVP_F32;
  const float sc = scale == 0.f ? 1.f / sqrtf(float(d->dh)) : scale;
  p.scale_log2 = sc * 1.4426950408889634f;

  const int smem = DEC_WARPS * DEC_STAGES * 2 * GRAN * d->dh * 2;
  cudaError_t e;
  if (d->dh == 128)
    e = cudaFuncSetAttribute(decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  else
    e = cudaFuncSetAttribute(decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return KVP_ERR_CUDA;

  for (int s0 = 0; s0 < n_sub; s0 += MAX_DEC_GROUPS) {
    const int n = n_sub - s0 < MAX_DEC_GROUPS ? n_sub - s0 : MAX_DEC_GROUPS;
    for (int i = 0; i < n; ++i) {
      const SubGroup& sg = subs[s0 + i];
      DecGroup& g = p.grp[i];
      if (k_cache[sg.owner] == nullptr || v_cache[sg.owner] == nullptr) return KVP_ERR_INVALID_ARG;
      g.k_cache = reinterpret_cast<const __nv_bfloat16*>(k_cache[sg.owner]);
      g.v_cache = reinterpret_cast<const __nv_bfloat16*>(v_cache[sg.owner]);
      g.n_members = sg.n;
      g.pad = 0;
      for (int m = 0; m < MAX_MEMBERS; ++m) {
        const int l = sg.members[m < sg.n ? m : 0];
        if (q[l] == nullptr || o[l] == nullptr || lse[l] == nullptr) return KVP_ERR_INVALID_ARG;
        g.q[m] = q[l];
        g.o[m] = o[l];
        g.lse[m] = lse[l];
      }
    }
    dim3 grid(ns, d->B * d->Hkv, n);
    dim3 cgrid(1, d->B * d->Hkv, n);
    timing_before(KVP_KERNEL_DECODE, stream);
    if (d->dh == 128)
      decode_kernel<128><<<grid, DEC_THREADS, smem, stream>>>(p);
    else
      decode_kernel<64><<<grid, DEC_THREADS, smem, stream>>>(p);
    timing_after(KVP_KERNEL_DECODE, stream);
    if (d->dh == 128)
      decode_combine_kernel<128><<<cgrid, 128, 0, stream>>>(p);
    else
      decode_combine_kernel<64><<<cgrid, 128, 0, stream>>>(p);
    note_launch(2);
    if (cudaGetLastError() != cudaSuccess) return KVP_ERR_CUDA;
  }
  return KVP_OK;
}

// ---------------------------------------------------------------------------------------------
// Decode without any caller-provided or allocated scratch.
//
// Some callers cannot allocate device memory at the point where they decode: a serving loop that
// has handed the whole device to its own cache pool and has nothing left to carve a workspace
// from, a plug-in running inside a host application that forbids cudaMalloc on its hot path, or a
// worker that must not touch the allocator because another thread holds it.  For them the per-split
// partial results live in a fixed array that is part of the library image.
// ---------------------------------------------------------------------------------------------
namespace kvp {
namespace {

static __device__ __align__(256) unsigned char g_decode_scratch[KVP_DECODE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};  // device address of g_decode_scratch, per device ordinal

// The array's name is only a host-side handle here; kernels need its device address, which differs
// per device and is looked up once with that device current.
int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KVP_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || p == nullptr) return KVP_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return KVP_OK;
}

}  // namespace
}  // namespace kvp

extern "C" int kvp_decode_static(const kvp_decode_desc* d, const int32_t* donor, float scale, const void* const* q,
                                 const void* const* k_cache, const void* const* v_cache, const int32_t* block_table,
                                 const int32_t* lengths, void* const* o, float* const* lse, int layer_begin,
                                 int layer_end, kvp_stream_t stream) {
  int rc = check_desc(d);
  if (rc != KVP_OK) return rc;
  if (donor == nullptr) return KVP_ERR_INVALID_ARG;
  for (int l = 0; l < d->L; ++l)
    if (donor[l] < 0 || donor[l] > l || donor[donor[l]] != donor[l]) return KVP_ERR_BAD_DONOR;
  if (layer_begin < 0 || layer_end > d->L || layer_begin >= layer_end) return KVP_ERR_INVALID_ARG;
  // only the donor groups that the layer range touches need room, so a narrower range can fit where all layers do not
  const size_t need = decode_scratch_bytes(d, donor, layer_begin, layer_end);
  if (need == 0) return KVP_ERR_UNSUPPORTED;
  if (need > size_t(KVP_DECODE_STATIC_SCRATCH_BYTES)) return KVP_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  rc = static_scratch_address(&scratch);
  if (rc != KVP_OK) return rc;
  return kvp_decode(d, donor, scale, q, k_cache, v_cache, block_table, lengths, o, lse, layer_begin, layer_end,
                    scratch, size_t(KVP_DECODE_STATIC_SCRATCH_BYTES), stream);
}
