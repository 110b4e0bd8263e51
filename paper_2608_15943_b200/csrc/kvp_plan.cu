// Offline planner: FIR (Eq. 4-5), stage totals under a conversion mask (Eq. 6-7), Algorithm 1
// (architecture-balanced, tail-first, bottleneck-retargeting conversion), the safe-layer
// guardrail, the two comparison placements, the donor map and the analytic FLOPs helper.
// Pure host code in exact integer arithmetic (128-bit products), off the hot path.
#include <algorithm>
#include <vector>

#include "kvp_host.h"

namespace {

typedef unsigned __int128 u128;

// The planner's working state: per-stage totals (Eq. 6) kept incrementally with their sum, and for every stage
// the index below which its layers are still unconverted (conversions inside a stage always go deepest-first,
// so the converted layers of a stage form a suffix of it).
struct PlanState {
  const kvp_plan_in* in;
  int L, P;
  std::vector<uint64_t> total;   // F_stage_i(z)
  u128 sum;                      // sum_i F_stage_i(z)
  std::vector<int> frontier;     // stage i: layers [frontier[i], stage_begin[i+1]) are converted
  int lowest_admissible;         // smallest layer index the guardrail and "never layer 0" admit

  uint64_t saving(int l) const { return in->f_full[l] - in->f_share[l]; }
  uint64_t heaviest() const { return *std::max_element(total.begin(), total.end()); }

  // deepest layer of stage i that Algorithm 1 may still convert, or -1
  int candidate(int i) const {
    const int l = frontier[i] - 1;
    int floor_l = std::max(in->stage_begin[i], lowest_admissible);
    if ((in->flags & KVP_PLAN_STAGE_LOCAL_DONOR) && floor_l == in->stage_begin[i]) ++floor_l;
    return l >= floor_l ? l : -1;
  }
  void convert(int i, uint8_t* z) {
    const int l = --frontier[i];
    z[l] = 1;
    total[i] -= saving(l);
    sum -= saving(l);
  }
};

// value / (sum / P) > 1 + en/ed, in integers
bool above_tolerance(u128 value, int P, u128 sum, u128 en, u128 ed) { return value * u128(P) * ed > (ed + en) * sum; }

// Uniform placement: rounds over the stages from the last one leftwards, one conversion per stage and round,
// until m are placed.  In closed form: stage i, which can give up cap_i layers, takes min(cap_i, R) in the R
// complete rounds that fit and one more if it is among the first stages (from the right) of the partial round.
void place_uniform(PlanState& st, uint8_t* z, int m) {
  const int P = st.P;
  std::vector<int> cap(P), take(P, 0);
  int64_t all = 0;
  for (int i = 0; i < P; ++i) {
    cap[i] = st.in->stage_begin[i + 1] - std::max(st.in->stage_begin[i], 1);   // layer 0 is never converted
    all += cap[i];
  }
  const int64_t want = std::min<int64_t>(m, all);
  const int deepest_stage = *std::max_element(cap.begin(), cap.end());
  int rounds = 0;
  while (rounds < deepest_stage) {   // the largest R whose complete rounds place no more than `want`
    int64_t placed = 0;
    for (int i = 0; i < P; ++i) placed += std::min(cap[i], rounds + 1);
    if (placed > want) break;
    ++rounds;
  }
  int64_t left = want;
  for (int i = 0; i < P; ++i) {
    take[i] = std::min(cap[i], rounds);
    left -= take[i];
  }
  for (int i = P - 1; i >= 0 && left > 0; --i)
    if (cap[i] > rounds) {
      ++take[i];
      --left;
    }
  for (int i = 0; i < P; ++i)
    for (int k = 0; k < take[i]; ++k) st.convert(i, z);
}

// Symmetric-Bipolar placement: two cursors, one starting at the deepest layer of the last stage and one at the
// deepest layer of the middle stage (index P/2 - 1), take turns; a cursor converts the deepest unconverted
// layer at or below its position and, stages being contiguous, simply walks down the layer indices; a cursor
// that has run past layer 1 loses its turns.
void place_bipolar(PlanState& st, uint8_t* z, int m) {
  const int P = st.P;
  const int mid = std::max(P / 2 - 1, 0);
  int cursor[2] = {st.L - 1, st.in->stage_begin[mid + 1] - 1};
  std::vector<int> stage_of(st.L);
  for (int i = 0; i < P; ++i)
    for (int l = st.in->stage_begin[i]; l < st.in->stage_begin[i + 1]; ++l) stage_of[l] = i;
  int placed = 0;
  for (int turn = 0; placed < m && (cursor[0] >= 1 || cursor[1] >= 1); ++turn) {
    int& c = cursor[turn & 1];
    while (c >= 1 && z[c]) --c;
    if (c < 1) continue;
    // within a stage conversions are deepest-first for both cursors, so c is that stage's frontier layer
    st.convert(stage_of[c], z);
    ++placed;
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
  PlanState st;
  st.in = in;
  st.L = L;
  st.P = P;
  st.total.resize(P);
  st.frontier.resize(P);
  st.sum = 0;
  for (int i = 0; i < P; ++i) {
    u128 wide = in->stage_extra[i];
    for (int l = in->stage_begin[i]; l < in->stage_begin[i + 1]; ++l) wide += in->f_full[l];
    if (wide > u128(~uint64_t(0))) return KVP_ERR_UNSUPPORTED;
    st.total[i] = uint64_t(wide);
    st.sum += wide;
    st.frontier[i] = in->stage_begin[i + 1];
  }
  // the exact fraction max * P / sum is returned in 64-bit words
  if (st.sum > u128(~uint64_t(0)) || u128(st.heaviest()) * u128(P) > u128(~uint64_t(0))) return KVP_ERR_UNSUPPORTED;
  st.lowest_admissible = 1;
  if (in->alpha_num != 0) {
    // 1-indexed layer l+1 >= ceil(alpha L)  <=>  l >= ceil(alpha L) - 1
    const uint64_t need = (uint64_t(in->alpha_num) * uint64_t(L) + in->alpha_den - 1) / in->alpha_den;
    st.lowest_admissible = std::max<int>(1, int(need) - 1);
  }

  const int budget = in->max_conv ? in->max_conv : L;
  const u128 en = in->eps_num, ed = in->eps_den;
  int reason = KVP_STOP_BUDGET;
  int n_conv = 0;

  if (in->placement == KVP_PLACE_UNIFORM) {
    place_uniform(st, z, budget);
  } else if (in->placement == KVP_PLACE_BIPOLAR) {
    place_bipolar(st, z, budget);
  } else if (in->placement == KVP_PLACE_ARCH_BALANCED) {
    for (;;) {
      const uint64_t top = st.heaviest();
      if (!above_tolerance(top, P, st.sum, en, ed)) {
        reason = KVP_STOP_TOLERANCE;
        break;
      }
      if (n_conv >= budget) {
        reason = KVP_STOP_BUDGET;
        break;
      }
      // the tail stage while it is still too heavy, otherwise the heaviest stage, the deepest among equals
      int target = P - 1;
      if (!above_tolerance(st.total[target], P, st.sum, en, ed))
        for (int j = P - 1; j >= 0; --j)
          if (st.total[j] > st.total[target]) target = j;
      const int l = st.candidate(target);
      if (l < 0) {
        reason = KVP_STOP_EXHAUSTED;
        break;
      }
      if (in->flags & KVP_PLAN_STOP_ON_NO_IMPROVE) {
        // FIR after the conversion: the new maximum is the lighter target or the heaviest of the others
        uint64_t top_after = st.total[target] - st.saving(l);
        for (int j = 0; j < P; ++j)
          if (j != target && st.total[j] > top_after) top_after = st.total[j];
        const u128 sum_after = st.sum - st.saving(l);
        if (!(u128(top_after) * st.sum < u128(top) * sum_after)) {   // top_after/sum_after < top/sum ?
          reason = KVP_STOP_NO_IMPROVE;
          break;
        }
      }
      st.convert(target, z);
      ++n_conv;
    }
  } else {
    return KVP_ERR_INVALID_ARG;
  }
  if (in->placement != KVP_PLACE_ARCH_BALANCED)
    for (int l = 0; l < L; ++l) n_conv += z[l];

  int last_owner = -1;
  for (int l = 0; l < L; ++l) {
    if (!z[l]) last_owner = l;
    out->donor[l] = last_owner;
  }
  const uint64_t top = st.heaviest();
  for (int i = 0; i < P; ++i) {
    out->stage_flops[i] = st.total[i];
    out->stage_ratio[i] = double(st.total[i]) * double(P) / double(uint64_t(st.sum));
  }
  out->fir_num = top * uint64_t(P);
  out->fir_den = uint64_t(st.sum);
  out->fir = double(out->fir_num) / double(out->fir_den);
  out->n_conv = n_conv;
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
