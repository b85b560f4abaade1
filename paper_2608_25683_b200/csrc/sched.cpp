// Workload model (Eq. 1), load-balanced group placement (Sec. 4.2) and token-wise micro-batching
// (Sec. 4.3).  See include/psrl_sched.h.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <new>
#include <numeric>
#include <vector>

#include "../../include/psrl_sched.h"

namespace {

struct Sample {
  std::vector<int32_t> fresh;  // segments of the path not computed by an earlier sample, root side first
  int64_t h, l;
  int32_t group;
};

double cost(const psrl_cost_model_t& m, int64_t l, int64_t h) {
  const double suf = double(l - h);
  return m.a1 * suf * double(l) + m.a2 * suf + m.a3;
}

// samples in canonical (DFS) order with their cached prefix
psrl_status_t walk(int32_t n, const int32_t* parent, const int32_t* seg_len, const uint8_t* flags,
                   std::vector<Sample>& samples, int32_t& n_groups) {
  if (n < 1 || !parent || !seg_len) return PSRL_ERR_INVALID_ARG;
  std::vector<int32_t> first_child(n, -1), last_child(n, -1), next_sib(n, -1), roots;
  for (int32_t s = 0; s < n; ++s) {
    const int32_t p = parent[s];
    if (seg_len[s] < 1) return PSRL_ERR_BAD_TREE;
    if (p == -1) {
      roots.push_back(s);
    } else if (p >= 0 && p < s) {
      if (first_child[p] < 0) first_child[p] = s; else next_sib[last_child[p]] = s;
      last_child[p] = s;
    } else {
      return PSRL_ERR_BAD_TREE;
    }
  }
  for (int32_t s = 0; s < n; ++s)
    if (flags && first_child[s] < 0 && !(flags[s] & PSRL_SEG_SAMPLE_END)) return PSRL_ERR_BAD_TREE;
  n_groups = static_cast<int32_t>(roots.size());
  std::vector<uint8_t> done(n, 0);
  std::vector<int32_t> stack, path;
  for (int32_t g = 0; g < n_groups; ++g) {
    stack.assign(1, roots[g]);
    while (!stack.empty()) {
      const int32_t e = stack.back();
      stack.pop_back();
      // children in ascending index order: push in reverse
      path.clear();
      for (int32_t c = first_child[e]; c >= 0; c = next_sib[c]) path.push_back(c);
      for (auto it = path.rbegin(); it != path.rend(); ++it) stack.push_back(*it);
      const bool ends = flags ? (flags[e] & PSRL_SEG_SAMPLE_END) != 0 : first_child[e] < 0;
      if (!ends) continue;
      path.clear();
      for (int32_t s = e; s != -1; s = parent[s]) path.push_back(s);
      std::reverse(path.begin(), path.end());
      Sample sm;
      sm.h = 0; sm.l = 0; sm.group = g;
      for (int32_t s : path) {
        sm.l += seg_len[s];
        if (done[s]) sm.h += seg_len[s]; else sm.fresh.push_back(s);
        done[s] = 1;
      }
      samples.push_back(std::move(sm));
    }
  }
  return PSRL_OK;
}

// largest x in [0, most] with cost of the piece [c0, c0 + x) <= room
int64_t fit(const psrl_cost_model_t& m, int64_t c0, double room, int64_t most) {
  if (room <= m.a3) return 0;
  int64_t x;
  if (m.a1 > 0) {
    const double bq = m.a1 * double(c0) + m.a2;
    x = static_cast<int64_t>(std::floor((-bq + std::sqrt(bq * bq + 4 * m.a1 * (room - m.a3))) / (2 * m.a1)));
  } else if (m.a2 > 0) {
    x = static_cast<int64_t>(std::floor((room - m.a3) / m.a2));
  } else {
    x = most;
  }
  x = std::max<int64_t>(0, std::min(x, most));
  while (x > 0 && cost(m, c0 + x, c0) > room) --x;  // guard the rounding of the root
  while (x + 1 <= most && cost(m, c0 + x + 1, c0) <= room) ++x;
  return x;
}

bool valid_model(const psrl_cost_model_t* m) {
  return m && std::isfinite(m->a1) && std::isfinite(m->a2) && std::isfinite(m->a3) && m->a1 >= 0 && m->a2 >= 0 &&
         m->a3 >= 0;
}

}  // namespace

extern "C" {

double psrl_cost_sequence(const psrl_cost_model_t* model, int64_t l, int64_t h) {
  return model ? cost(*model, l, h) : 0.0;
}

psrl_status_t psrl_group_workloads(int32_t n, const int32_t* parent, const int32_t* seg_len, const uint8_t* flags,
                                   const psrl_cost_model_t* model, int32_t n_groups, double* workload) {
  if (!valid_model(model) || !workload) return PSRL_ERR_INVALID_ARG;
  try {
    std::vector<Sample> samples;
    int32_t groups = 0;
    const psrl_status_t st = walk(n, parent, seg_len, flags, samples, groups);
    if (st != PSRL_OK) return st;
    if (groups != n_groups) return PSRL_ERR_INVALID_ARG;
    std::fill(workload, workload + n_groups, 0.0);
    for (const Sample& s : samples) workload[s.group] += cost(*model, s.l, s.h);
  } catch (const std::bad_alloc&) {
    return PSRL_ERR_HOST_OOM;
  }
  return PSRL_OK;
}

psrl_status_t psrl_place_groups(int32_t n_groups, const double* workload, int32_t n_workers, int32_t* worker_of_group,
                                double* worker_load) {
  if (n_groups < 0 || n_workers < 1 || (n_groups > 0 && (!workload || !worker_of_group))) return PSRL_ERR_INVALID_ARG;
  for (int32_t g = 0; g < n_groups; ++g)
    if (!std::isfinite(workload[g]) || workload[g] < 0) return PSRL_ERR_INVALID_ARG;
  try {
    std::vector<int32_t> order(n_groups);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return workload[a] > workload[b]; });
    std::vector<double> load(n_workers, 0.0);
    for (int32_t g : order) {
      int32_t k = 0;
      for (int32_t j = 1; j < n_workers; ++j)
        if (load[j] < load[k]) k = j;
      worker_of_group[g] = k;
      load[k] += workload[g];
    }
    if (worker_load) std::copy(load.begin(), load.end(), worker_load);
  } catch (const std::bad_alloc&) {
    return PSRL_ERR_HOST_OOM;
  }
  return PSRL_OK;
}

psrl_status_t psrl_microbatch_tokens(int32_t n, const int32_t* parent, const int32_t* seg_len, const uint8_t* flags,
                                     const psrl_cost_model_t* model, int32_t n_mb, int32_t capacity, int32_t* n_pieces,
                                     int32_t* piece_parent, int32_t* piece_len, int32_t* piece_mb, int32_t* piece_seg,
                                     int32_t* piece_begin, double* budget_out) {
  if (!valid_model(model) || n_mb < 1 || capacity < 0 || !n_pieces || !piece_parent || !piece_len || !piece_mb ||
      !piece_seg || !piece_begin)
    return PSRL_ERR_INVALID_ARG;
  *n_pieces = 0;
  try {
    std::vector<Sample> samples;
    int32_t groups = 0;
    const psrl_status_t st = walk(n, parent, seg_len, flags, samples, groups);
    if (st != PSRL_OK) return st;
    double total = 0;
    for (const Sample& s : samples) total += cost(*model, s.l, s.h);
    const double budget = total / n_mb;
    if (budget_out) *budget_out = budget;
    std::vector<int32_t> last_piece(n, -1);  // last piece emitted for each input segment
    int32_t count = 0, mb = 0;
    double used = 0;
    bool full = false;
    auto emit = [&](const Sample& sm, int64_t a, int64_t b) {
      int64_t pos = sm.h;
      for (int32_t s : sm.fresh) {
        const int64_t lo = std::max(a, pos), hi = std::min(b, pos + seg_len[s]);
        if (lo < hi) {
          if (count >= capacity) { full = true; return; }
          piece_parent[count] = last_piece[s] >= 0 ? last_piece[s] : (parent[s] == -1 ? -1 : last_piece[parent[s]]);
          piece_len[count] = static_cast<int32_t>(hi - lo);
          piece_mb[count] = mb;
          piece_seg[count] = s;
          piece_begin[count] = static_cast<int32_t>(lo - pos);
          last_piece[s] = count++;
        }
        pos += seg_len[s];
      }
    };
    for (const Sample& sm : samples) {
      int64_t a = sm.h;
      while (a < sm.l && !full) {
        const double rest = cost(*model, sm.l, a);
        if (mb == n_mb - 1 || used + rest <= budget) {
          emit(sm, a, sm.l);
          used += rest;
          break;
        }
        int64_t x = fit(*model, a, budget - used, sm.l - a - 1);
        if (x == 0 && used == 0.0) x = 1;
        if (x > 0) {
          emit(sm, a, a + x);
          a += x;
        }
        ++mb;
        used = 0;
      }
      if (full) return PSRL_ERR_WORKSPACE;
    }
    *n_pieces = count;
  } catch (const std::bad_alloc&) {
    return PSRL_ERR_HOST_OOM;
  }
  return PSRL_OK;
}

}  // extern "C"
