// C-ABI entry points of the training / prefill path: argument validation and the sequence of
// kernel launches per layer.  No allocation, no synchronisation.
#include <algorithm>
#include <vector>

#include "kvp_host.h"

namespace kvp {
int attn_fwd_layers(const kvp_shape* s, int causal, float scale, const void* const* q, const void* const* k,
                    const void* const* v, void* const* o, float* const* lse, int n, cudaStream_t stream);
int attn_fwd_max_layers();
size_t attn_bwd_workspace(const kvp_shape* s, const int32_t* donor);
int attn_bwd_all(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                 const void* const* k, const void* const* v, const void* const* o, const void* const* d_o,
                 const float* const* lse, void* const* dq, float* const* dk_sum, float* const* dv_sum, void* ws,
                 size_t ws_bytes, cudaStream_t stream);
int cast_f32_to_bf16(const float* src, void* dst, size_t n, cudaStream_t stream);
int cast_bf16_to_f32(const void* src, float* dst, size_t n, cudaStream_t stream);

namespace {

int check_donor(int L, const int32_t* donor) {
  if (donor == nullptr) return KVP_ERR_INVALID_ARG;
  for (int l = 0; l < L; ++l) {
    const int d = donor[l];
    if (d < 0 || d > l || donor[d] != d) return KVP_ERR_BAD_DONOR;
  }
  return KVP_OK;
}

int check_shape(const kvp_shape* s) {
  if (s == nullptr) return KVP_ERR_INVALID_ARG;
  if (s->L < 1 || s->B < 1 || s->S < 1 || s->D < 1 || s->Hq < 1 || s->Hkv < 1) return KVP_ERR_INVALID_ARG;
  if (s->dtype != KVP_BF16 && s->dtype != KVP_F32) return KVP_ERR_UNSUPPORTED;
  if ((s->dh != 64 && s->dh != 128) || s->Hq % s->Hkv != 0 || s->D % 64 != 0) return KVP_ERR_UNSUPPORTED;
  return KVP_OK;
}

bool ptrs_ok(const void* const* arr, int L, const int32_t* donor, bool owners_only) {
  if (arr == nullptr) return false;
  for (int l = 0; l < L; ++l) {
    if (owners_only && donor[l] != l) continue;
    if (arr[l] == nullptr || !aligned16(arr[l])) return false;
  }
  return true;
}

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

// ---------------------------------------------------------------------------------------------
// KVP_F32 interface: bf16 shadow copies of the caller's fp32 tensors, carved from the workspace behind the
// operation's own scratch.  Inputs are rounded on the way in, outputs widened on the way out; in between the
// bf16 entry point runs unchanged.
// ---------------------------------------------------------------------------------------------
struct TensorSet {   // one per-layer tensor array of an entry point
  size_t elems;      // elements per layer
  bool owners_only;
};

size_t shadow_bytes(const kvp_shape* s, const int32_t* donor, const TensorSet* sets, int n_sets) {
  size_t total = 0;
  for (int i = 0; i < n_sets; ++i)
    for (int l = 0; l < s->L; ++l)
      if (!sets[i].owners_only || donor[l] == l) total += align256(sets[i].elems * 2);
  return total;
}

class Shadows {
 public:
  Shadows(const kvp_shape* s, const int32_t* donor, void* ws, size_t offset, cudaStream_t stream)
      : s_(s), donor_(donor), cur_(reinterpret_cast<uint8_t*>(ws) + offset), stream_(stream) {}
  // bf16 copies of an fp32 input array
  const void* const* in(const void* const* src, const TensorSet& t) {
    std::vector<void*>& arr = reserve(t);
    for (int l = 0; l < s_->L; ++l)
      if (arr[l] != nullptr && rc_ == KVP_OK) rc_ = cast_f32_to_bf16(reinterpret_cast<const float*>(src[l]), arr[l], t.elems, stream_);
    return reinterpret_cast<const void* const*>(arr.data());
  }
  // bf16 buffers standing in for an fp32 output array; finish() widens them into the caller's tensors
  void* const* out(void* const* dst, const TensorSet& t) {
    std::vector<void*>& arr = reserve(t);
    for (int l = 0; l < s_->L; ++l)
      if (arr[l] != nullptr) pending_.push_back(Pending{arr[l], reinterpret_cast<float*>(dst[l]), t.elems});
    return arr.data();
  }
  int status() const { return rc_; }
  int finish() {
    for (const Pending& p : pending_)
      if (rc_ == KVP_OK) rc_ = cast_bf16_to_f32(p.src, p.dst, p.elems, stream_);
    return rc_;
  }

 private:
  struct Pending {
    const void* src;
    float* dst;
    size_t elems;
  };
  std::vector<void*>& reserve(const TensorSet& t) {
    arrays_.emplace_back(size_t(s_->L), nullptr);
    std::vector<void*>& arr = arrays_.back();
    for (int l = 0; l < s_->L; ++l)
      if (!t.owners_only || donor_[l] == l) {
        arr[l] = cur_;
        cur_ += align256(t.elems * 2);
      }
    return arr;
  }
  const kvp_shape* s_;
  const int32_t* donor_;
  uint8_t* cur_;
  cudaStream_t stream_;
  int rc_ = KVP_OK;
  std::vector<std::vector<void*>> arrays_;
  std::vector<Pending> pending_;
};

struct Sizes {
  TensorSet x, wq, wkv, q, kv;
};
Sizes sizes_of(const kvp_shape* s) {
  const size_t T = size_t(s->B) * s->S, D = s->D, nq = size_t(s->Hq) * s->dh, nkv = size_t(s->Hkv) * s->dh;
  return Sizes{{T * D, false}, {nq * D, false}, {nkv * D, true}, {T * nq, false}, {T * nkv, true}};
}

// Layers per grouped launch of the projection backward: 8 layers are at most 32 problems and 48 operand pairs.
constexpr int kProjBwdChunk = 8;

GemmProblem problem(int M, int N, GemmSeg seg, int a_mn, int b_mn, void* c, int64_t ldc, int out_f32) {
  GemmProblem g{};
  g.M = M;
  g.N = N;
  g.segs[0] = seg;
  g.nseg = 1;
  g.a_mn = a_mn;
  g.b_mn = b_mn;
  g.c = c;
  g.ldc = ldc;
  g.out_f32 = out_f32;
  return g;
}

// scratch the bf16 form of an operation needs (before any shadows)
size_t op_scratch_bytes(int op, const kvp_shape* s, const int32_t* donor) {
  switch (op) {
    case KVP_OP_PROJ_BWD: {
      // bf16 copies of dk_sum and dv_sum of the owners of one chunk of layers
      int owners = 0;
      for (int l = 0; l < s->L; ++l) owners += donor[l] == l;
      return size_t(2 * std::min(owners, kProjBwdChunk)) * align256(size_t(s->B) * s->S * s->Hkv * s->dh * 2);
    }
    case KVP_OP_ATTN_BWD:
      return attn_bwd_workspace(s, donor);
    default:
      return 0;
  }
}

size_t op_shadow_bytes(int op, const kvp_shape* s, const int32_t* donor) {
  if (s->dtype != KVP_F32) return 0;
  const Sizes z = sizes_of(s);
  switch (op) {
    case KVP_OP_PROJ_FWD: {
      const TensorSet sets[] = {z.x, z.wq, z.wkv, z.wkv, z.q, z.kv, z.kv};
      return shadow_bytes(s, donor, sets, 7);
    }
    case KVP_OP_PROJ_BWD: {
      const TensorSet sets[] = {z.x, z.wq, z.wkv, z.wkv, z.q, z.x};   // x, wq, wk, wv, dq in; dx out
      return shadow_bytes(s, donor, sets, 6);
    }
    case KVP_OP_ATTN_FWD: {
      const TensorSet sets[] = {z.q, z.kv, z.kv, z.q};                // q, k, v in; o out
      return shadow_bytes(s, donor, sets, 4);
    }
    case KVP_OP_ATTN_BWD: {
      const TensorSet sets[] = {z.q, z.kv, z.kv, z.q, z.q, z.q};      // q, k, v, o, dO in; dq out
      return shadow_bytes(s, donor, sets, 6);
    }
    default:
      return 0;
  }
}

}  // namespace
}  // namespace kvp

using namespace kvp;

extern "C" size_t kvp_workspace_bytes(int op, const kvp_shape* s, const int32_t* donor) {
  if (check_shape(s) != KVP_OK || check_donor(s->L, donor) != KVP_OK) return 0;
  return align256(op_scratch_bytes(op, s, donor)) + op_shadow_bytes(op, s, donor);
}

extern "C" int kvp_proj_fwd(const kvp_shape* s, const int32_t* donor, const void* const* x, const void* const* wq,
                            const void* const* wk, const void* const* wv, void* const* q, void* const* k,
                            void* const* v, void* ws, size_t ws_bytes, kvp_stream_t stream_) {
  int rc = check_shape(s);
  if (rc == KVP_OK) rc = check_donor(s->L, donor);
  if (rc != KVP_OK) return rc;
  if (!ptrs_ok(x, s->L, donor, false) || !ptrs_ok(wq, s->L, donor, false) || !ptrs_ok(wk, s->L, donor, true) ||
      !ptrs_ok(wv, s->L, donor, true) || !ptrs_ok(q, s->L, donor, false) || !ptrs_ok(k, s->L, donor, true) ||
      !ptrs_ok(v, s->L, donor, true))
    return KVP_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (s->dtype == KVP_F32) {
    if (ws == nullptr || ws_bytes < kvp_workspace_bytes(KVP_OP_PROJ_FWD, s, donor) || !aligned16(ws)) return KVP_ERR_WORKSPACE;
    const Sizes z = sizes_of(s);
    Shadows sh(s, donor, ws, align256(op_scratch_bytes(KVP_OP_PROJ_FWD, s, donor)), stream);
    const void* const* x16 = sh.in(x, z.x);
    const void* const* wq16 = sh.in(wq, z.wq);
    const void* const* wk16 = sh.in(wk, z.wkv);
    const void* const* wv16 = sh.in(wv, z.wkv);
    void* const* q16 = sh.out(q, z.q);
    void* const* k16 = sh.out(k, z.kv);
    void* const* v16 = sh.out(v, z.kv);
    if (sh.status() != KVP_OK) return sh.status();
    kvp_shape s16 = *s;
    s16.dtype = KVP_BF16;
    rc = kvp_proj_fwd(&s16, donor, x16, wq16, wk16, wv16, q16, k16, v16, ws, ws_bytes, stream_);
    return rc != KVP_OK ? rc : sh.finish();
  }
  const int T = s->B * s->S, D = s->D, Nq = s->Hq * s->dh, Nkv = s->Hkv * s->dh;
  // Every projection of every layer in one grouped launch; consumers have no K/V projections (Eq. 3).
  std::vector<GemmProblem> probs;
  probs.reserve(size_t(3) * s->L);
  for (int l = 0; l < s->L; ++l) probs.push_back(problem(T, Nq, {x[l], wq[l], D, D, D}, 0, 0, q[l], Nq, 0));
  for (int l = 0; l < s->L; ++l) {
    if (donor[l] != l) continue;
    probs.push_back(problem(T, Nkv, {x[l], wk[l], D, D, D}, 0, 0, k[l], Nkv, 0));
    probs.push_back(problem(T, Nkv, {x[l], wv[l], D, D, D}, 0, 0, v[l], Nkv, 0));
  }
  return gemm_grouped(probs.data(), int(probs.size()), stream, true);
}

extern "C" int kvp_proj_bwd(const kvp_shape* s, const int32_t* donor, const void* const* x, const void* const* wq,
                            const void* const* wk, const void* const* wv, const void* const* dq,
                            const float* const* dk_sum, const float* const* dv_sum, float* const* dwq,
                            float* const* dwk, float* const* dwv, void* const* dx, void* ws, size_t ws_bytes,
                            kvp_stream_t stream_) {
  return kvp_proj_bwd_range(s, donor, x, wq, wk, wv, dq, dk_sum, dv_sum, dwq, dwk, dwv, dx, 0, s != nullptr ? s->L : 0, ws,
                            ws_bytes, stream_);
}

extern "C" int kvp_proj_bwd_range(const kvp_shape* s, const int32_t* donor, const void* const* x,
                                  const void* const* wq, const void* const* wk, const void* const* wv,
                                  const void* const* dq, const float* const* dk_sum, const float* const* dv_sum,
                                  float* const* dwq, float* const* dwk, float* const* dwv, void* const* dx,
                                  int layer_begin, int layer_end, void* ws, size_t ws_bytes, kvp_stream_t stream_) {
  int rc = check_shape(s);
  if (rc == KVP_OK) rc = check_donor(s->L, donor);
  if (rc != KVP_OK) return rc;
  if (layer_begin < 0 || layer_end > s->L || layer_begin > layer_end) return KVP_ERR_INVALID_ARG;
  if (!ptrs_ok(x, s->L, donor, false) || !ptrs_ok(wq, s->L, donor, false) || !ptrs_ok(wk, s->L, donor, true) ||
      !ptrs_ok(wv, s->L, donor, true) || !ptrs_ok(dq, s->L, donor, false) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dk_sum), s->L, donor, true) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dv_sum), s->L, donor, true) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dwq), s->L, donor, false) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dwk), s->L, donor, true) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dwv), s->L, donor, true) || !ptrs_ok(dx, s->L, donor, false))
    return KVP_ERR_INVALID_ARG;
  const size_t need = kvp_workspace_bytes(KVP_OP_PROJ_BWD, s, donor);
  if (ws == nullptr || ws_bytes < need || !aligned16(ws)) return KVP_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (s->dtype == KVP_F32) {
    const Sizes z = sizes_of(s);
    Shadows sh(s, donor, ws, align256(op_scratch_bytes(KVP_OP_PROJ_BWD, s, donor)), stream);
    const void* const* x16 = sh.in(x, z.x);
    const void* const* wq16 = sh.in(wq, z.wq);
    const void* const* wk16 = sh.in(wk, z.wkv);
    const void* const* wv16 = sh.in(wv, z.wkv);
    const void* const* dq16 = sh.in(dq, z.q);
    void* const* dx16 = sh.out(dx, z.x);
    if (sh.status() != KVP_OK) return sh.status();
    kvp_shape s16 = *s;
    s16.dtype = KVP_BF16;
    if (layer_begin != 0 || layer_end != s->L) return KVP_ERR_UNSUPPORTED;   // the fp32 interface converts whole arrays
    rc = kvp_proj_bwd(&s16, donor, x16, wq16, wk16, wv16, dq16, dk_sum, dv_sum, dwq, dwk, dwv, dx16, ws, ws_bytes, stream_);
    return rc != KVP_OK ? rc : sh.finish();
  }
  const int T = s->B * s->S, D = s->D, Nq = s->Hq * s->dh, Nkv = s->Hkv * s->dh;
  const size_t n_kv = size_t(T) * Nkv;
  const size_t slot = align256(n_kv * 2);
  uint8_t* bf = reinterpret_cast<uint8_t*>(ws);
  // Chunks of up to kProjBwdChunk layers: the fp32 donor-group sums of the chunk's owners are rounded to bf16 into
  // the workspace, then ONE grouped launch produces every gradient of the chunk.  The weight gradients come first
  // in the list (their tiles run over all T tokens, the longest), then dX = dQ Wq + dK Wk + dV Wv of the owners
  // (three K segments into one accumulator), then the consumers' dX = dQ Wq.
  std::vector<GemmProblem> probs;
  for (int c0 = layer_begin; c0 < layer_end; c0 += kProjBwdChunk) {
    const int c1 = std::min(layer_end, c0 + kProjBwdChunk);
    probs.clear();
    std::vector<uint8_t*> dk_bf(size_t(c1 - c0), nullptr), dv_bf(size_t(c1 - c0), nullptr);
    int owners = 0;
    for (int l = c0; l < c1; ++l) {
      if (donor[l] != l) continue;
      dk_bf[l - c0] = bf + size_t(2 * owners) * slot;
      dv_bf[l - c0] = bf + size_t(2 * owners + 1) * slot;
      ++owners;
      rc = cast_f32_to_bf16(dk_sum[l], dk_bf[l - c0], n_kv, stream);
      if (rc == KVP_OK) rc = cast_f32_to_bf16(dv_sum[l], dv_bf[l - c0], n_kv, stream);
      if (rc != KVP_OK) return rc;
    }
    // dWq = dQ^T X : A = dQ stored [T, Nq] (MN-major for M = Nq), B = X stored [T, D] (MN-major for N = D)
    for (int l = c0; l < c1; ++l) probs.push_back(problem(Nq, D, {dq[l], x[l], Nq, D, T}, 1, 1, dwq[l], D, 1));
    for (int l = c0; l < c1; ++l) {
      if (donor[l] != l) continue;
      probs.push_back(problem(Nkv, D, {dk_bf[l - c0], x[l], Nkv, D, T}, 1, 1, dwk[l], D, 1));
      probs.push_back(problem(Nkv, D, {dv_bf[l - c0], x[l], Nkv, D, T}, 1, 1, dwv[l], D, 1));
    }
    for (int l = c0; l < c1; ++l) {
      if (donor[l] != l) continue;
      GemmProblem g = problem(T, D, {dq[l], wq[l], Nq, D, Nq}, 0, 1, dx[l], D, 0);
      g.segs[1] = {dk_bf[l - c0], wk[l], Nkv, D, Nkv};
      g.segs[2] = {dv_bf[l - c0], wv[l], Nkv, D, Nkv};
      g.nseg = 3;
      probs.push_back(g);
    }
    for (int l = c0; l < c1; ++l)
      if (donor[l] != l) probs.push_back(problem(T, D, {dq[l], wq[l], Nq, D, Nq}, 0, 1, dx[l], D, 0));
    rc = gemm_grouped(probs.data(), int(probs.size()), stream, false);
    if (rc != KVP_OK) return rc;
  }
  return KVP_OK;
}

extern "C" int kvp_out_proj_fwd(const kvp_shape* s, const void* const* o, const void* const* wo, void* const* y,
                                kvp_stream_t stream_) {
  int rc = check_shape(s);
  if (rc != KVP_OK) return rc;
  if (s->dtype != KVP_BF16) return KVP_ERR_UNSUPPORTED;
  if (o == nullptr || wo == nullptr || y == nullptr) return KVP_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  const int T = s->B * s->S, D = s->D, Nq = s->Hq * s->dh;
  std::vector<GemmProblem> probs;
  for (int l = 0; l < s->L; ++l) {
    if (o[l] == nullptr || wo[l] == nullptr || y[l] == nullptr) return KVP_ERR_INVALID_ARG;
    probs.push_back(problem(T, D, {o[l], wo[l], Nq, Nq, Nq}, 0, 0, y[l], D, 0));
  }
  return gemm_grouped(probs.data(), int(probs.size()), stream, true);
}

extern "C" int kvp_out_proj_bwd(const kvp_shape* s, const void* const* o, const void* const* wo,
                                const void* const* dy, void* const* d_o, float* const* dwo, kvp_stream_t stream_) {
  int rc = check_shape(s);
  if (rc != KVP_OK) return rc;
  if (s->dtype != KVP_BF16) return KVP_ERR_UNSUPPORTED;
  if (o == nullptr || wo == nullptr || dy == nullptr || d_o == nullptr || dwo == nullptr) return KVP_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  const int T = s->B * s->S, D = s->D, Nq = s->Hq * s->dh;
  std::vector<GemmProblem> probs;
  for (int l = 0; l < s->L; ++l)
    if (o[l] == nullptr || wo[l] == nullptr || dy[l] == nullptr || d_o[l] == nullptr || dwo[l] == nullptr)
      return KVP_ERR_INVALID_ARG;
  // dWo = dY^T O : [D, Nq], both operands stored token-major (the longest tiles: first in the list)
  for (int l = 0; l < s->L; ++l) probs.push_back(problem(D, Nq, {dy[l], o[l], D, Nq, T}, 1, 1, dwo[l], Nq, 1));
  // dO = dY Wo : A = dY [T, D] K-major, B = Wo stored [D, Nq] = [K, N] (MN-major)
  for (int l = 0; l < s->L; ++l) probs.push_back(problem(T, Nq, {dy[l], wo[l], D, Nq, D}, 0, 1, d_o[l], Nq, 0));
  return gemm_grouped(probs.data(), int(probs.size()), stream, false);
}

extern "C" int kvp_attn_fwd(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                            const void* const* k, const void* const* v, void* const* o, float* const* lse, void* ws,
                            size_t ws_bytes, kvp_stream_t stream_) {
  int rc = check_shape(s);
  if (rc == KVP_OK) rc = check_donor(s->L, donor);
  if (rc != KVP_OK) return rc;
  if (!ptrs_ok(q, s->L, donor, false) || !ptrs_ok(k, s->L, donor, true) || !ptrs_ok(v, s->L, donor, true) ||
      !ptrs_ok(o, s->L, donor, false) || !ptrs_ok(reinterpret_cast<const void* const*>(lse), s->L, donor, false))
    return KVP_ERR_INVALID_ARG;
  if (scale < 0.f) return KVP_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (s->dtype == KVP_F32) {
    if (ws == nullptr || ws_bytes < kvp_workspace_bytes(KVP_OP_ATTN_FWD, s, donor) || !aligned16(ws)) return KVP_ERR_WORKSPACE;
    const Sizes z = sizes_of(s);
    Shadows sh(s, donor, ws, align256(op_scratch_bytes(KVP_OP_ATTN_FWD, s, donor)), stream);
    const void* const* q16 = sh.in(q, z.q);
    const void* const* k16 = sh.in(k, z.kv);
    const void* const* v16 = sh.in(v, z.kv);
    void* const* o16 = sh.out(o, z.q);
    if (sh.status() != KVP_OK) return sh.status();
    kvp_shape s16 = *s;
    s16.dtype = KVP_BF16;
    rc = kvp_attn_fwd(&s16, donor, causal, scale, q16, k16, v16, o16, lse, ws, ws_bytes, stream_);
    return rc != KVP_OK ? rc : sh.finish();
  }
  // up to eight layers per launch, each with the K / V of its donor
  std::vector<const void*> kd(size_t(s->L)), vd(size_t(s->L));
  for (int l = 0; l < s->L; ++l) {
    kd[l] = k[donor[l]];
    vd[l] = v[donor[l]];
  }
  const int chunk = attn_fwd_max_layers();
  for (int l0 = 0; l0 < s->L; l0 += chunk) {
    const int n = std::min(chunk, s->L - l0);
    rc = attn_fwd_layers(s, causal, scale, q + l0, kd.data() + l0, vd.data() + l0, o + l0, lse + l0, n, stream);
    if (rc != KVP_OK) return rc;
  }
  return KVP_OK;
}

extern "C" int kvp_attn_bwd(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                            const void* const* k, const void* const* v, const void* const* o,
                            const void* const* d_o, const float* const* lse, void* const* dq, float* const* dk_sum,
                            float* const* dv_sum, void* ws, size_t ws_bytes, kvp_stream_t stream_) {
  int rc = check_shape(s);
  if (rc == KVP_OK) rc = check_donor(s->L, donor);
  if (rc != KVP_OK) return rc;
  if (!ptrs_ok(q, s->L, donor, false) || !ptrs_ok(k, s->L, donor, true) || !ptrs_ok(v, s->L, donor, true) ||
      !ptrs_ok(o, s->L, donor, false) || !ptrs_ok(d_o, s->L, donor, false) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(lse), s->L, donor, false) || !ptrs_ok(dq, s->L, donor, false) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dk_sum), s->L, donor, true) ||
      !ptrs_ok(reinterpret_cast<const void* const*>(dv_sum), s->L, donor, true))
    return KVP_ERR_INVALID_ARG;
  if (scale < 0.f) return KVP_ERR_INVALID_ARG;
  const size_t need = kvp_workspace_bytes(KVP_OP_ATTN_BWD, s, donor);
  if (need > 0 && (ws == nullptr || ws_bytes < need || !aligned16(ws))) return KVP_ERR_WORKSPACE;
  if (s->dtype == KVP_F32) {
    const Sizes z = sizes_of(s);
    Shadows sh(s, donor, ws, align256(op_scratch_bytes(KVP_OP_ATTN_BWD, s, donor)), reinterpret_cast<cudaStream_t>(stream_));
    const void* const* q16 = sh.in(q, z.q);
    const void* const* k16 = sh.in(k, z.kv);
    const void* const* v16 = sh.in(v, z.kv);
    const void* const* o16 = sh.in(o, z.q);
    const void* const* do16 = sh.in(d_o, z.q);
    void* const* dq16 = sh.out(dq, z.q);
    if (sh.status() != KVP_OK) return sh.status();
    kvp_shape s16 = *s;
    s16.dtype = KVP_BF16;
    rc = kvp_attn_bwd(&s16, donor, causal, scale, q16, k16, v16, o16, do16, lse, dq16, dk_sum, dv_sum, ws, ws_bytes, stream_);
    return rc != KVP_OK ? rc : sh.finish();
  }
  return attn_bwd_all(s, donor, causal, scale, q, k, v, o, d_o, lse, dq, dk_sum, dv_sum, ws, ws_bytes,
                      reinterpret_cast<cudaStream_t>(stream_));
}
