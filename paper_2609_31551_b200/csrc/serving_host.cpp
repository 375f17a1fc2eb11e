// Host-side control logic around the encoder: Poisson-gap micro-batcher, deficit-counter router with envelope
// planning, SM lookup table.  Pure host code behind the C ABI of include/eas_serving.h.
#include "../../include/eas_serving.h"

#include <cmath>
#include <limits>
#include <new>
#include <vector>
#include <algorithm>

// ------------------------------------------------------------------------------------ micro-batcher (Eq. 5)
extern "C" double eas_poisson_gap_kappa(int32_t B, double p) {
  if (!(p > 0.0 && p < 1.0)) return std::numeric_limits<double>::quiet_NaN();
  if (B <= 1) return 0.0;
  return -std::log(1.0 - std::pow(p, 1.0 / static_cast<double>(B - 1)));
}

struct eas_batcher {
  int32_t bound;
  double gap, max_age;
  int32_t size;       // requests waiting
  double first, last; // arrival times of the first and the latest waiting request
};

extern "C" eas_batcher* eas_batcher_create(int32_t B, double lambda, double p, double max_age) {
  if (B < 1 || !(lambda > 0.0) || !(p > 0.0 && p < 1.0) || !(max_age > 0.0)) return nullptr;
  eas_batcher* b = new (std::nothrow) eas_batcher();
  if (b == nullptr) return nullptr;
  b->bound = B;
  b->gap = eas_poisson_gap_kappa(B, p) / lambda;
  b->max_age = max_age;
  b->size = 0;
  b->first = b->last = 0.0;
  return b;
}
extern "C" void eas_batcher_destroy(eas_batcher* b) { delete b; }
extern "C" double eas_batcher_gap(const eas_batcher* b) { return b ? b->gap : std::numeric_limits<double>::quiet_NaN(); }

extern "C" double eas_batcher_deadline(const eas_batcher* b) {
  if (b == nullptr || b->size == 0) return std::numeric_limits<double>::infinity();
  return std::fmin(b->last + b->gap, b->first + b->max_age);
}

extern "C" int32_t eas_batcher_on_timer(eas_batcher* b, double now, int32_t* size, double* time) {
  if (b == nullptr || size == nullptr || time == nullptr) return -1;
  if (b->size == 0) return 0;
  const double deadline = eas_batcher_deadline(b);
  if (!(now > deadline)) return 0;   // idle > g or age > A, both strict
  *size = b->size;
  *time = deadline;
  b->size = 0;
  return 1;
}

extern "C" int32_t eas_batcher_on_arrival(eas_batcher* b, double t, int32_t* sizes, double* times) {
  if (b == nullptr || sizes == nullptr || times == nullptr) return -1;
  int32_t n = 0;
  int32_t s;
  double when;
  if (eas_batcher_on_timer(b, t, &s, &when) == 1) { sizes[n] = s; times[n] = when; ++n; }
  if (b->size == 0) b->first = t;
  b->last = t;
  ++b->size;
  if (b->size >= b->bound) {
    sizes[n] = b->size; times[n] = t; ++n;
    b->size = 0;
  }
  return n;
}

// ------------------------------------------------------------------------------------ router and envelopes
extern "C" int32_t eas_router_init(eas_router* r, int64_t num, int64_t den) {
  if (r == nullptr || den <= 0 || num < 0 || num > den) return -1;
  r->num = num; r->den = den; r->acc = 0;
  return 0;
}

extern "C" int32_t eas_router_init_from_double(eas_router* r, double s, int64_t max_den) {
  if (r == nullptr || !(s >= 0.0 && s <= 1.0) || max_den < 1) return -1;
  // closest fraction by walking the continued-fraction convergents of s
  int64_t p0 = 0, q0 = 1, p1 = 1, q1 = 0;
  double x = s;
  int64_t best_p = 0, best_q = 1;
  for (int it = 0; it < 64; ++it) {
    const double fl = std::floor(x);
    const int64_t a = static_cast<int64_t>(fl);
    const int64_t p2 = a * p1 + p0, q2 = a * q1 + q0;
    if (q2 > max_den || q2 <= 0) break;
    best_p = p2; best_q = q2;
    p0 = p1; q0 = q1; p1 = p2; q1 = q2;
    const double frac = x - fl;
    if (frac < 1e-12 || std::fabs(static_cast<double>(p2) / static_cast<double>(q2) - s) < 1e-15) break;
    x = 1.0 / frac;
  }
  return eas_router_init(r, best_p, best_q);
}

extern "C" int32_t eas_router_next(eas_router* r) {
  r->acc += r->num;
  if (r->acc >= r->den) { r->acc -= r->den; return 1; }
  return 0;
}

extern "C" int32_t eas_envelope_plan(const int32_t* dest, const int32_t* rows, int32_t n, int32_t n_dest,
                                     int64_t* row_offset, int64_t* dest_rows) {
  if (dest == nullptr || rows == nullptr || row_offset == nullptr || dest_rows == nullptr || n < 0 || n_dest <= 0) return -1;
  for (int32_t k = 0; k < n_dest; ++k) dest_rows[k] = 0;
  for (int32_t i = 0; i < n; ++i) {
    if (dest[i] < 0 || dest[i] >= n_dest || rows[i] < 0) return -1;
    row_offset[i] = dest_rows[dest[i]];
    dest_rows[dest[i]] += rows[i];
  }
  return 0;
}

extern "C" int32_t eas_envelope_order(const int32_t* dest, const int32_t* rows, int32_t n, int32_t n_dest, int32_t* order,
                                      int64_t* env_first_row) {
  if (dest == nullptr || rows == nullptr || order == nullptr || env_first_row == nullptr || n < 0 || n_dest <= 0) return -1;
  // counting sort by destination (stable: arrival order is kept inside an envelope)
  std::vector<int64_t> count(static_cast<size_t>(n_dest) + 1, 0), total(static_cast<size_t>(n_dest), 0);
  for (int32_t i = 0; i < n; ++i) {
    if (dest[i] < 0 || dest[i] >= n_dest || rows[i] < 0) return -1;
    ++count[static_cast<size_t>(dest[i]) + 1];
    total[static_cast<size_t>(dest[i])] += rows[i];
  }
  int64_t first = 0;
  for (int32_t k = 0; k < n_dest; ++k) {
    count[static_cast<size_t>(k) + 1] += count[static_cast<size_t>(k)];
    env_first_row[k] = first;
    first += total[static_cast<size_t>(k)];
  }
  for (int32_t i = 0; i < n; ++i) order[count[static_cast<size_t>(dest[i])]++] = i;
  return 0;
}

// ------------------------------------------------------------------------------------ SM lookup table
extern "C" int32_t eas_sm_table_build(const int32_t* sm_counts, int32_t n_levels, const int32_t* batches, int32_t n_batches,
                                      const double* latency, const double* exclusive, double tolerance, eas_sm_table* out) {
  if (sm_counts == nullptr || batches == nullptr || latency == nullptr || exclusive == nullptr || out == nullptr) return -1;
  if (n_levels < 1 || n_levels > EAS_SM_TABLE_MAX_LEVELS || n_batches < 1 || !(tolerance >= 0.0)) return -1;
  for (int32_t l = 1; l < n_levels; ++l) if (sm_counts[l] <= sm_counts[l - 1]) return -1;
  for (int32_t b = 1; b < n_batches; ++b) if (batches[b] <= batches[b - 1]) return -1;
  out->n_levels = n_levels;
  for (int32_t l = 0; l < n_levels; ++l) {
    out->sm_count[l] = sm_counts[l];
    int32_t best = 0;
    for (int32_t b = 0; b < n_batches; ++b) {
      if (latency[l * n_batches + b] <= (1.0 + tolerance) * exclusive[b]) best = batches[b];
      else break;
    }
    out->max_batch[l] = best;
  }
  return 0;
}

extern "C" int32_t eas_sm_table_lookup(const eas_sm_table* t, int32_t batch) {
  if (t == nullptr || t->n_levels < 1 || t->n_levels > EAS_SM_TABLE_MAX_LEVELS) return -1;
  for (int32_t l = 0; l < t->n_levels; ++l)
    if (t->max_batch[l] >= batch) return t->sm_count[l];
  return t->sm_count[t->n_levels - 1];
}

// ------------------------------------------------------------------------------------ HAS Stage 1 (Eq. 3, Eq. 4)
extern "C" int32_t eas_has_stage1(eas_has_candidate* c, int32_t n, double rate, double c_e, double c_p, double c_d,
                                  double alpha, double prune_factor, int32_t top_k) {
  if (c == nullptr || n < 1 || !(rate > 0) || !(c_e > 0) || !(c_p > 0) || !(c_d > 0) || !(alpha >= 0 && alpha <= 1) ||
      !(prune_factor >= 1) || top_k < 1)
    return -1;
  const double inf = std::numeric_limits<double>::infinity();
  double best = inf;
  for (int32_t i = 0; i < n; ++i) {
    eas_has_candidate& a = c[i];
    if (a.n_encode < 1 || a.n_prefill < 0 || a.n_decode < 1 || a.n_local < 0) return -1;
    const double prefill_workers = a.n_prefill + a.n_local * alpha;
    a.rho_e = (rate / a.n_encode) / c_e;
    a.rho_p = prefill_workers > 0 ? rate / (c_p * prefill_workers) : inf;
    a.rho_d = (rate / a.n_decode) / c_d;
    a.score = std::max(a.rho_e, std::max(a.rho_p, a.rho_d));
    a.b_max = static_cast<int32_t>(std::ceil(rate / a.n_encode));
    a.s_star = prefill_workers > 0 ? a.n_prefill / prefill_workers : 0.0;
    a.kept = a.score < 1.0 ? 1 : 0;                     // an overloaded stage rules the allocation out
    if (a.kept) best = std::min(best, a.score);
  }
  std::vector<int32_t> order;
  for (int32_t i = 0; i < n; ++i) {
    if (c[i].kept && c[i].score > prune_factor * best) c[i].kept = 0;
    if (c[i].kept) order.push_back(i);
  }
  std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return c[x].score < c[y].score; });
  for (size_t k = static_cast<size_t>(top_k); k < order.size(); ++k) c[order[k]].kept = 0;
  return static_cast<int32_t>(std::min<size_t>(order.size(), static_cast<size_t>(top_k)));
}
