// Runtime planner: scoring of the legal bitwidth reductions and their greedy selection (Sec. 3.2, Alg. 1,
// Eqs. 4-8).  Host code only -- scalar work over a few thousand page-table rows per call -- and free of CUDA
// calls, so it also runs on a machine without a GPU.  Its runtime inputs are what the observation taps
// produce on the device (routing mass, routed-input features); its output is the list of steps the caller
// carries out with pw_demote_block, pw_set_page_table and pw_offload_page.
#include <math.h>

#include <algorithm>
#include <new>
#include <vector>

#include "pw_common.cuh"

namespace {

constexpr int kLevels = 5;
const int kLevelBits[kLevels] = {16, 8, 4, 3, 2};

int level_of(int bits) {
  for (int i = 0; i < kLevels; ++i)
    if (kLevelBits[i] == bits) return i;
  return -1;
}

struct Cand {           // the next legal step of one block
  double ratio, damage;
  uint64_t delta;
  int to_level;
  bool ok;
};

}  // namespace

extern "C" uint64_t pw_kv_pressure_bytes(int64_t free_block_threshold, int64_t free_blocks, uint64_t kv_block_bytes) {
  const int64_t need = free_block_threshold + 1 - free_blocks;      // Eq. 7
  return need > 0 ? (uint64_t)need * kv_block_bytes : 0;
}

namespace {

pw_status check_tables(const pw_plan_tables* t) {
  if (!t) return PW_ERR_INVALID_ARG;
  const int L = t->n_layers, E = t->n_experts, S = t->n_experts + t->n_shared;
  if (L < 1 || E < 1 || t->n_shared < 0 || t->n_buckets < 1 || t->n_stages < 1) return PW_ERR_INVALID_ARG;
  if (!t->committed || !t->supported || !t->sensitivity || !t->page_bytes || !t->mass || !t->bucket_share ||
      !t->bucket_mu || !t->stage_floor)
    return PW_ERR_INVALID_ARG;
  if ((t->head_w || t->head_a || t->head_c) && !(t->head_w && t->head_a && t->head_c && t->phi))
    return PW_ERR_INVALID_ARG;
  const size_t n_rows = (size_t)L * S * 3;
  for (size_t i = 0; i < n_rows; ++i)
    if (level_of(t->committed[i]) < 0) return PW_ERR_BITS;
  for (int s = 0; s < t->n_stages * t->n_buckets; ++s)
    if (level_of(t->stage_floor[s]) < 0) return PW_ERR_BITS;

  return PW_OK;
}

// routing buckets of every (layer, expert)
std::vector<int> routing_buckets(const pw_plan_tables* t) {
  const int L = t->n_layers, E = t->n_experts;
  // routing buckets: experts of a layer ranked by mass, hottest first (ties: lower index); bucket j holds the
  // ranks below share[j] * E
  std::vector<int> bucket((size_t)L * E);
  {
    std::vector<int> order(E);
    for (int l = 0; l < L; ++l) {
      const float* m = t->mass + (size_t)l * E;
      for (int e = 0; e < E; ++e) order[e] = e;
      std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return m[a] > m[b]; });
      for (int rank = 0; rank < E; ++rank) {
        int j = 0;
        while (j < t->n_buckets - 1 && (double)rank >= (double)t->bucket_share[j] * E) ++j;
        bucket[(size_t)l * E + order[rank]] = j;
      }
    }
  }

  return bucket;
}

// ScoreActions + GreedySelect of Alg. 1 for one bitwidth-floor stage: the ordered steps that release `target` bytes
// (or all the stage's floors allow) and the bytes they release.
void plan_stage(const pw_plan_tables* t, const std::vector<int>& bucket, int stage, uint64_t target,
                std::vector<pw_plan_item>& plan, uint64_t& released) {
  const int E = t->n_experts, S = t->n_experts + t->n_shared;
  const size_t n_rows = (size_t)t->n_layers * S * 3;
  std::vector<uint8_t> cur(n_rows);
  std::vector<Cand> cand(n_rows);
  const uint8_t* floor_of = t->stage_floor + (size_t)stage * t->n_buckets;
  for (size_t i = 0; i < n_rows; ++i) cur[i] = t->committed[i];
  plan.clear();
  released = 0;
  // the next legal step of block i from its current bitwidth: the next lower supported bitwidth, unless it
  // lies below the floor of the expert's bucket (Eqs. 4-6 and 8 give its damage)
  auto next_step = [&](size_t i) {
    Cand c{};
    c.ok = false;
    const int u = (int)(i % 3), e = (int)((i / 3) % S), l = (int)(i / 3 / S);
    if (e >= E) return c;                                     // shared experts are never touched
    const int li = level_of(cur[i]);
    for (int lj = li + 1; lj < kLevels; ++lj) {
      if (!t->supported[i * kLevels + lj]) continue;
      const int bk = bucket[(size_t)l * E + e];
      if (kLevelBits[lj] < floor_of[bk]) return c;
      const double g = std::max((double)t->sensitivity[i * kLevels + lj] - (double)t->sensitivity[i * kLevels + li], 0.0);
      double eta = 1.0;
      if (t->head_w) {
        const float* phi = t->phi + i * 3;
        if (phi[0] != 0.f || phi[1] != 0.f || phi[2] != 0.f) {
          const size_t h = ((size_t)u * kLevels + li) * kLevels + lj;
          double rho = (double)t->head_a[h];
          for (int d = 0; d < 3; ++d) rho += (double)t->head_w[h * 3 + d] * (double)phi[d];
          rho = std::min(std::max(rho, (double)t->rho_min), (double)t->rho_max);
          eta = exp((double)t->alpha * (double)t->head_c[h] * rho);
        }
      }
      c.damage = std::max((double)t->epsilon, (double)t->bucket_mu[bk] * g * eta);
      const uint64_t m_from = t->page_bytes[i * kLevels + li], m_to = t->page_bytes[i * kLevels + lj];
      if (m_to >= m_from) return c;                             // a size table that does not shrink: nothing to release
      c.delta = m_from - m_to;
      c.ratio = c.damage / (double)c.delta;
      c.to_level = lj;
      c.ok = c.delta > 0;
      return c;
    }
    return c;
  };
  for (size_t i = 0; i < n_rows; ++i) cand[i] = next_step(i);
  while (released < target) {
    size_t best = n_rows;
    for (size_t i = 0; i < n_rows; ++i)
      if (cand[i].ok && (best == n_rows || cand[i].ratio < cand[best].ratio)) best = i;
    if (best == n_rows) break;
    pw_plan_item it{};
    it.layer = (int32_t)(best / 3 / S);
    it.expert = (int32_t)((best / 3) % S);
    it.kind = (int32_t)(best % 3);
    it.from_bits = cur[best];
    it.to_bits = (uint8_t)kLevelBits[cand[best].to_level];
    it.released_bytes = cand[best].delta;
    it.damage = cand[best].damage;
    plan.push_back(it);
    released += cand[best].delta;
    cur[best] = it.to_bits;
    cand[best] = next_step(best);
  }
}

}  // namespace

extern "C" pw_status pw_plan_step(const pw_plan_tables* t, uint64_t target, pw_plan_item* steps, size_t max_steps,
                                  size_t* n_steps_out, uint64_t* released_out, int32_t* stage_out) {
  if (!n_steps_out || (!steps && max_steps)) return PW_ERR_INVALID_ARG;
  const pw_status vs = check_tables(t);
  if (vs != PW_OK) return vs;
  try {
    const std::vector<int> bucket = routing_buckets(t);
    std::vector<pw_plan_item> plan;
    uint64_t released = 0;
    int stage = 0;
    for (stage = 0; stage < t->n_stages; ++stage) {
      plan_stage(t, bucket, stage, target, plan, released);
      if (released >= target) break;
    }
    if (stage == t->n_stages) stage = t->n_stages - 1;
    *n_steps_out = plan.size();
    if (released_out) *released_out = released;
    if (stage_out) *stage_out = stage;
    if (plan.size() > max_steps) return PW_ERR_NOMEM;
    for (size_t i = 0; i < plan.size(); ++i) steps[i] = plan[i];
    return PW_OK;
  } catch (const std::bad_alloc&) {
    return PW_ERR_NOMEM;                             // nothing crosses the C boundary
  }
}

// ---- the plan queue of Alg. 1 ---------------------------------------------------------------------------
struct pw_plan_queue {
  struct Entry {
    std::vector<pw_plan_item> plan;                  // the stage's candidate plan of the latest refresh
    uint64_t target = 0, released = 0, refreshed_at = 0;
    bool valid = false;
  };
  std::vector<Entry> stage;
  uint64_t steps = 0;                                // planner steps taken so far
};

extern "C" pw_status pw_plan_queue_create(pw_plan_queue** out, int32_t n_stages) {
  if (!out || n_stages < 1) return PW_ERR_INVALID_ARG;
  *out = nullptr;
  try {
    pw_plan_queue* q = new pw_plan_queue();
    q->stage.resize((size_t)n_stages);
    *out = q;
    return PW_OK;
  } catch (const std::bad_alloc&) {
    return PW_ERR_NOMEM;
  }
}

extern "C" pw_status pw_plan_queue_destroy(pw_plan_queue* q) {
  if (!q) return PW_ERR_INVALID_ARG;
  delete q;
  return PW_OK;
}

extern "C" pw_status pw_plan_queue_step(pw_plan_queue* q, const pw_plan_tables* t, int64_t free_block_threshold,
                                        int64_t free_blocks, uint64_t kv_block_bytes, uint64_t lookahead_bytes,
                                        pw_plan_item* steps, size_t max_steps, size_t* n_steps_out, uint64_t* released_out,
                                        int32_t* stage_out, int32_t* triggered_out) {
  if (!q || !n_steps_out || (!steps && max_steps)) return PW_ERR_INVALID_ARG;
  const pw_status vs = check_tables(t);
  if (vs != PW_OK) return vs;
  if ((size_t)t->n_stages != q->stage.size()) return PW_ERR_INVALID_ARG;
  try {
    // D_t of Eq. 7; without pressure the queue is refreshed for the bytes the caller expects to need next
    const uint64_t D = pw_kv_pressure_bytes(free_block_threshold, free_blocks, kv_block_bytes);
    const bool triggered = D > 0;
    const uint64_t target = triggered ? D : lookahead_bytes;
    const std::vector<int> bucket = routing_buckets(t);
    ++q->steps;
    for (int s = 0; s < t->n_stages; ++s) {              // ScoreActions, GreedySelect, RefreshPlanQueue per stage
      pw_plan_queue::Entry& e = q->stage[(size_t)s];
      plan_stage(t, bucket, s, target, e.plan, e.released);
      e.target = target;
      e.refreshed_at = q->steps;
      e.valid = true;
    }
    *n_steps_out = 0;
    if (released_out) *released_out = 0;
    if (stage_out) *stage_out = -1;
    if (triggered_out) *triggered_out = triggered ? 1 : 0;
    if (!triggered) return PW_OK;
    // SelectBestPlan: the first stage (the highest floors) whose plan meets the target, else the last stage's
    int best = t->n_stages - 1;
    for (int s = 0; s < t->n_stages; ++s)
      if (q->stage[(size_t)s].released >= D) {
        best = s;
        break;
      }
    const pw_plan_queue::Entry& e = q->stage[(size_t)best];
    *n_steps_out = e.plan.size();
    if (released_out) *released_out = e.released;
    if (stage_out) *stage_out = best;
    if (e.plan.size() > max_steps) return PW_ERR_NOMEM;
    for (size_t i = 0; i < e.plan.size(); ++i) steps[i] = e.plan[i];
    return PW_OK;
  } catch (const std::bad_alloc&) {
    return PW_ERR_NOMEM;
  }
}

extern "C" pw_status pw_plan_queue_peek(const pw_plan_queue* q, int32_t stage, uint64_t* target_out, uint64_t* released_out,
                                        size_t* n_steps_out, uint64_t* refreshed_at_out) {
  if (!q || stage < 0 || (size_t)stage >= q->stage.size()) return PW_ERR_INVALID_ARG;
  const pw_plan_queue::Entry& e = q->stage[(size_t)stage];
  if (!e.valid) return PW_ERR_STATE;
  if (target_out) *target_out = e.target;
  if (released_out) *released_out = e.released;
  if (n_steps_out) *n_steps_out = e.plan.size();
  if (refreshed_at_out) *refreshed_at_out = e.refreshed_at;
  return PW_OK;
}
