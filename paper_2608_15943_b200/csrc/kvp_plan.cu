// Offline planner: FIR (Eq. 4-5), stage totals under a conversion mask (Eq. 6-7), Algorithm 1
// (architecture-balanced, tail-first, bottleneck-retargeting conversion), the safe-layer
// guardrail, the two comparison placements, the donor map and the analytic FLOPs helper.
// Pure host code in exact integer arithmetic (128-bit products), off the hot path.
#include <algorithm>
#include <vector>

#include "kvp_host.h"

namespace {

typedef unsigned __int128 u128;

struct Fir {
  uint64_t num;  // max_i F_i * P
  uint64_t den;  // sum_i F_i
};

bool stage_sums_fit(const std::vector<uint64_t>& stage) {
  u128 sum = 0, mx = 0;
  for (uint64_t f : stage) {
    sum += f;
    if (f > mx) mx = f;
  }
  const u128 lim = ~uint64_t(0);
  return sum <= lim && mx * stage.size() <= lim;
}

Fir fir_of(const std::vector<uint64_t>& stage) {
  uint64_t mx = 0, sum = 0;
  for (uint64_t f : stage) {
    sum += f;
    if (f > mx) mx = f;
  }
  return Fir{mx * uint64_t(stage.size()), sum};
}

// a/b > c/d for positive denominators
bool frac_gt(u128 a, u128 b, u128 c, u128 d) { return a * d > c * b; }

bool admissible(int l, int stage_first, const kvp_plan_in* in) {
  if (l == 0) return false;
  if ((in->flags & KVP_PLAN_STAGE_LOCAL_DONOR) && l == stage_first) return false;
  if (in->alpha_num != 0) {
    // 1-indexed layer l+1 must satisfy l+1 >= ceil(alpha * L)
    const uint64_t need = (uint64_t(in->alpha_num) * uint64_t(in->L) + in->alpha_den - 1) / in->alpha_den;
    if (uint64_t(l) + 1 < need) return false;
  }
  return true;
}

int deepest_convertible(const kvp_plan_in* in, const uint8_t* z, int stage) {
  const int first = in->stage_begin[stage], last = in->stage_begin[stage + 1];
  for (int l = last - 1; l >= first; --l)
    if (!z[l] && admissible(l, first, in)) return l;
  return -1;
}

// deepest unconverted layer of a stage for the comparison placements (only layer 0 is excluded)
int deepest_plain(const kvp_plan_in* in, const uint8_t* z, int stage) {
  for (int l = in->stage_begin[stage + 1] - 1; l >= in->stage_begin[stage]; --l)
    if (!z[l] && l > 0) return l;
  return -1;
}

void place_uniform(const kvp_plan_in* in, uint8_t* z, int m) {
  const int P = in->P;
  int i = P - 1, t = 0, idle = 0;
  while (t < m && idle < P) {
    const int l = deepest_plain(in, z, i);
    if (l >= 0) {
      z[l] = 1;
      ++t;
      idle = 0;
    } else {
      ++idle;
    }
    i = i > 0 ? i - 1 : P - 1;
  }
}

void place_bipolar(const kvp_plan_in* in, uint8_t* z, int m) {
  const int P = in->P;
  int anchors[2] = {P - 1, P / 2 - 1 > 0 ? P / 2 - 1 : 0};
  int t = 0, turn = 0, idle = 0;
  while (t < m && idle < 2 * P) {
    const int a = turn % 2;
    const int i = anchors[a];
    const int l = i >= 0 ? deepest_plain(in, z, i) : -1;
    if (l >= 0) {
      z[l] = 1;
      ++t;
      idle = 0;
      ++turn;
    } else {
      anchors[a] -= 1;
      ++idle;
      if (anchors[a] < 0) ++turn;
    }
  }
}

}  // namespace

extern "C" int kvp_layer_flops(const kvp_model_desc* m, uint64_t* f_full, uint64_t* f_share, uint64_t* f_lm_head) {
  if (m == nullptr || f_full == nullptr || f_share == nullptr || f_lm_head == nullptr) return KVP_ERR_INVALID_ARG;
  if (m->h <= 0 || m->f < 0 || m->a <= 0 || m->g <= 0 || m->dh <= 0 || m->s <= 0 || m->vocab < 0 || m->a % m->g != 0)
    return KVP_ERR_INVALID_ARG;
  const uint64_t h = m->h, f = m->f, qd = uint64_t(m->a) * m->dh, kvd = uint64_t(m->g) * m->dh, s = m->s;
  const uint64_t scores = (m->causal_half ? 2u : 4u) * s * qd;
  *f_full = 2 * h * qd + 4 * h * kvd + 2 * qd * h + scores + 6 * h * f;
  *f_share = *f_full - 4 * h * kvd;
  *f_lm_head = 2 * h * uint64_t(m->vocab);
  return KVP_OK;
}

extern "C" int kvp_plan(const kvp_plan_in* in, kvp_plan_out* out) {
  if (in == nullptr || out == nullptr) return KVP_ERR_INVALID_ARG;
  const int L = in->L, P = in->P;
  if (L < 1 || P < 1 || P > L || in->stage_begin == nullptr || in->f_full == nullptr || in->f_share == nullptr ||
      in->stage_extra == nullptr || out->z == nullptr || out->donor == nullptr || out->stage_flops == nullptr ||
      out->stage_ratio == nullptr || in->eps_den == 0 || in->max_conv < 0 ||
      (in->alpha_num != 0 && (in->alpha_den == 0 || in->alpha_num >= in->alpha_den)))
    return KVP_ERR_INVALID_ARG;
  if (in->stage_begin[0] != 0 || in->stage_begin[P] != L) return KVP_ERR_UNSUPPORTED;
  for (int i = 0; i < P; ++i)
    if (in->stage_begin[i + 1] <= in->stage_begin[i]) return KVP_ERR_UNSUPPORTED;  // contiguous, non-empty stages
  for (int l = 0; l < L; ++l)
    if (in->f_share[l] >= in->f_full[l]) return KVP_ERR_INVALID_ARG;

  uint8_t* z = out->z;
  for (int l = 0; l < L; ++l) z[l] = 0;
  std::vector<uint64_t> stage(P);
  {
    std::vector<u128> wide(P);
    for (int i = 0; i < P; ++i) {
      wide[i] = in->stage_extra[i];
      for (int l = in->stage_begin[i]; l < in->stage_begin[i + 1]; ++l) wide[i] += in->f_full[l];
      if (wide[i] > u128(~uint64_t(0))) return KVP_ERR_UNSUPPORTED;
      stage[i] = uint64_t(wide[i]);
    }
  }
  if (!stage_sums_fit(stage)) return KVP_ERR_UNSUPPORTED;

  const int m = in->max_conv ? in->max_conv : L;
  const u128 en = in->eps_num, ed = in->eps_den;
  int t = 0;
  int reason = KVP_STOP_TOLERANCE;

  if (in->placement == KVP_PLACE_UNIFORM || in->placement == KVP_PLACE_BIPOLAR) {
    if (in->placement == KVP_PLACE_UNIFORM) place_uniform(in, z, m); else place_bipolar(in, z, m);
    for (int i = 0; i < P; ++i)
      for (int l = in->stage_begin[i]; l < in->stage_begin[i + 1]; ++l)
        if (z[l]) {
          stage[i] -= in->f_full[l] - in->f_share[l];
          ++t;
        }
    reason = KVP_STOP_BUDGET;
  } else if (in->placement == KVP_PLACE_ARCH_BALANCED) {
    for (;;) {
      const Fir f = fir_of(stage);
      if (!(u128(f.num) * ed > (ed + en) * u128(f.den))) {  // FIR <= 1 + eps
        reason = KVP_STOP_TOLERANCE;
        break;
      }
      if (!(t < m)) {
        reason = KVP_STOP_BUDGET;
        break;
      }
      int i_star = P - 1;  // the tail stage
      if (u128(stage[i_star]) * uint64_t(P) * ed <= (ed + en) * u128(f.den)) {
        uint64_t mx = 0;
        for (int j = 0; j < P; ++j)
          if (stage[j] >= mx) {  // ties -> highest stage index
            mx = stage[j];
            i_star = j;
          }
      }
      const int l_star = deepest_convertible(in, z, i_star);
      if (l_star < 0) {
        reason = KVP_STOP_EXHAUSTED;
        break;
      }
      const uint64_t delta = in->f_full[l_star] - in->f_share[l_star];
      if (in->flags & KVP_PLAN_STOP_ON_NO_IMPROVE) {
        std::vector<uint64_t> trial(stage);
        trial[i_star] -= delta;
        const Fir g = fir_of(trial);
        if (!frac_gt(f.num, f.den, g.num, g.den)) {  // FIR would not strictly drop
          reason = KVP_STOP_NO_IMPROVE;
          break;
        }
      }
      z[l_star] = 1;
      stage[i_star] -= delta;
      ++t;
    }
  } else {
    return KVP_ERR_INVALID_ARG;
  }

  int last_owner = -1;
  for (int l = 0; l < L; ++l) {
    if (!z[l]) last_owner = l;
    out->donor[l] = last_owner;
  }
  const Fir f = fir_of(stage);
  for (int i = 0; i < P; ++i) {
    out->stage_flops[i] = stage[i];
    out->stage_ratio[i] = double(stage[i]) * double(P) / double(f.den);
  }
  out->fir_num = f.num;
  out->fir_den = f.den;
  out->fir = double(f.num) / double(f.den);
  out->n_conv = t;
  out->stop_reason = reason;
  return KVP_OK;
}

// 1F1B timing model.  Event-driven: every stage keeps a cursor into its operation sequence and a clock; a
// sweep over the stages executes every operation whose remote input has been produced, until nothing is
// left.  Finish times of forwards and backwards live in two P x M tables (-1 = not produced yet).
extern "C" int kvp_sim_1f1b(int32_t P, int32_t M, const int64_t* t_fwd, const int64_t* t_bwd, kvp_sim_out* out) {
  if (P < 1 || M < 1 || t_fwd == nullptr || t_bwd == nullptr || out == nullptr) return KVP_ERR_INVALID_ARG;
  if (int64_t(P) * int64_t(M) > (int64_t(1) << 24)) return KVP_ERR_INVALID_ARG;
  for (int i = 0; i < P; ++i)
    if (t_fwd[i] < 0 || t_bwd[i] < 0) return KVP_ERR_INVALID_ARG;
  std::vector<int64_t> fin_f(size_t(P) * M, -1), fin_b(size_t(P) * M, -1), clock(P, 0);
  std::vector<int32_t> next_f(P, 0), next_b(P, 0);  // micro-batch of the stage's next forward / backward
  int64_t remaining = int64_t(2) * P * M;
  while (remaining > 0) {
    bool progressed = false;
    for (int i = 0; i < P; ++i) {
      for (;;) {
        if (next_f[i] >= M && next_b[i] >= M) break;
        const int warm = std::min(P - 1 - i, M);
        // position in the sequence: warm-up forwards, then (F, B) pairs, then the draining backwards
        bool forward;
        if (next_f[i] < warm) forward = true;
        else if (next_f[i] < M) forward = (next_f[i] - warm == next_b[i]);  // pair k = F(warm+k) then B(k)
        else forward = false;
        if (forward) {
          const int m = next_f[i];
          int64_t ready = 0;
          if (i > 0) {
            ready = fin_f[size_t(i - 1) * M + m];
            if (ready < 0) break;
          }
          clock[i] = std::max(clock[i], ready) + t_fwd[i];
          fin_f[size_t(i) * M + m] = clock[i];
          ++next_f[i];
        } else {
          const int m = next_b[i];
          const int64_t ready = i + 1 < P ? fin_b[size_t(i + 1) * M + m] : fin_f[size_t(i) * M + m];
          if (ready < 0) break;
          clock[i] = std::max(clock[i], ready) + t_bwd[i];
          fin_b[size_t(i) * M + m] = clock[i];
          ++next_b[i];
        }
        --remaining;
        progressed = true;
      }
    }
    if (!progressed) return KVP_ERR_UNSUPPORTED;  // cannot happen for this schedule; never spin
  }
  int64_t makespan = 0;
  for (int i = 0; i < P; ++i) makespan = std::max(makespan, clock[i]);
  out->makespan = makespan;
  if (out->idle != nullptr)
    for (int i = 0; i < P; ++i) out->idle[i] = makespan - int64_t(M) * (t_fwd[i] + t_bwd[i]);
  return KVP_OK;
}
