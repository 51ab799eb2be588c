// Host-side selection plan (Section 3.3 Eq. 2/3, Section 4.1, Eq. 6, Eq. 7, Appendix B).
// Built once per model; nothing here runs per request.
#include <algorithm>
#include <cmath>
#include <limits>
#include <numeric>

#include "dasc_internal.h"

namespace {

// Eq. 2 with the gate logit fixed at `a`; numerically safe softplus.
double static_log_decay(double A_log, double dt_bias, double a) {
  const double x = a + dt_bias;
  const double sp = x > 0.0 ? x + std::log1p(std::exp(-x)) : std::log1p(std::exp(x));
  return -std::exp(A_log) * sp;
}

// Smallest power of two >= h (h > 0); exact powers map to themselves.
double pow2_ceil(double h) {
  if (!(h > 0.0)) return 0.0;
  if (std::isinf(h)) return h;
  const double p = std::exp2(std::floor(std::log2(h)));
  // log2/floor can be off by one ulp at exact powers; fix up with comparisons.
  double r = p;
  while (r < h) r *= 2.0;
  while (r * 0.5 >= h) r *= 0.5;
  return r;
}

// Published splitmix64 finaliser: the counter-based generator of the random selector.
uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

int64_t group_keep_count(double ratio, int64_t n) {
  const double x = ratio * static_cast<double>(n) - 1e-9;
  int64_t r = static_cast<int64_t>(std::ceil(x));
  return std::min<int64_t>(n, std::max<int64_t>(0, r));
}

}  // namespace

dasc_status_t dasc_build_plan_host(const dasc_plan_desc_t *d, dasc_plan_s *p) {
  if (!d || !p) return DASC_ERR_INVALID_ARG;
  if (d->kind != DASC_KDA && d->kind != DASC_GDN) return DASC_ERR_INVALID_ARG;
  if (d->n_layers <= 0 || d->n_v_heads <= 0 || d->n_k_heads <= 0 || d->d_k <= 0 || d->d_v <= 0)
    return DASC_ERR_SHAPE;
  if (d->n_v_heads % d->n_k_heads != 0) return DASC_ERR_SHAPE;
  if (d->d_v % 4 != 0) return DASC_ERR_SHAPE;
  if (!d->A_log || !d->dt_bias) return DASC_ERR_INVALID_ARG;
  if (!(d->eps > 0.0) || !(d->eps < 1.0)) return DASC_ERR_INVALID_ARG;
  if (d->sel != DASC_SEL_THRESHOLD && d->sel != DASC_SEL_TOP_RATIO && d->sel != DASC_SEL_EXPLICIT)
    return DASC_ERR_INVALID_ARG;
  if (d->sel == DASC_SEL_EXPLICIT && !d->explicit_mask) return DASC_ERR_INVALID_ARG;
  if (d->sel == DASC_SEL_TOP_RATIO) {
    if (!(d->keep_ratio >= 0.0 && d->keep_ratio <= 1.0)) return DASC_ERR_INVALID_ARG;
    if (d->scope != DASC_SCOPE_HEAD && d->scope != DASC_SCOPE_LAYER && d->scope != DASC_SCOPE_MODEL)
      return DASC_ERR_INVALID_ARG;
  }
  if (d->sel == DASC_SEL_THRESHOLD && std::isnan(d->w_max)) return DASC_ERR_INVALID_ARG;
  if (d->conv_bytes_per_ckpt < 0) return DASC_ERR_INVALID_ARG;

  const int64_t L = d->n_layers;
  const int64_t uph = d->kind == DASC_KDA ? d->d_k : 1;  // units per head
  const int64_t n_l = static_cast<int64_t>(d->n_v_heads) * uph;
  const int64_t n_all = n_l * L;
  const int64_t unit_floats = d->kind == DASC_KDA ? d->d_v : static_cast<int64_t>(d->d_k) * d->d_v;
  const int64_t rows_per_unit = d->kind == DASC_KDA ? 1 : d->d_k;
  const int64_t rows_per_layer = static_cast<int64_t>(d->n_v_heads) * d->d_k;
  if (rows_per_layer * L >= std::numeric_limits<int32_t>::max()) return DASC_ERR_SHAPE;

  // --- scores -------------------------------------------------------------
  p->horizon.resize(n_all);
  const double ln_eps = std::log(d->eps);
  for (int64_t u = 0; u < n_all; ++u) {
    const double g = static_log_decay(d->A_log[u], d->dt_bias[u], d->a);
    p->horizon[u] = ln_eps / g;
  }

  // --- selection ----------------------------------------------------------
  p->mask.assign(n_all, 0);
  if (d->sel == DASC_SEL_THRESHOLD) {
    for (int64_t u = 0; u < n_all; ++u) p->mask[u] = p->horizon[u] > d->w_max ? 1 : 0;
  } else if (d->sel == DASC_SEL_EXPLICIT) {
    for (int64_t u = 0; u < n_all; ++u) p->mask[u] = d->explicit_mask[u] ? 1 : 0;
  } else {
    const int64_t group = d->scope == DASC_SCOPE_HEAD ? uph : d->scope == DASC_SCOPE_LAYER ? n_l : n_all;
    const int64_t keep = group_keep_count(d->keep_ratio, group);
    std::vector<int64_t> order(group);
    for (int64_t base = 0; base < n_all; base += group) {
      std::iota(order.begin(), order.end(), int64_t{0});
      const double *h = p->horizon.data() + base;
      // longest horizon first; equal horizons keep the lower index first
      std::stable_sort(order.begin(), order.end(), [h](int64_t x, int64_t y) { return h[x] > h[y]; });
      for (int64_t i = 0; i < keep; ++i) p->mask[base + order[i]] = 1;
    }
  }

  if (d->randomize) {
    std::vector<std::pair<uint64_t, int64_t>> keyed(n_l);
    for (int64_t l = 0; l < L; ++l) {
      uint8_t *m = p->mask.data() + l * n_l;
      const int64_t r = std::count(m, m + n_l, uint8_t{1});
      for (int64_t u = 0; u < n_l; ++u)
        keyed[u] = {mix64(d->seed + (static_cast<uint64_t>(l) << 32) + static_cast<uint64_t>(u)), u};
      std::sort(keyed.begin(), keyed.end());  // by key, then by unit index
      std::fill(m, m + n_l, uint8_t{0});
      for (int64_t i = 0; i < r; ++i) m[keyed[i].second] = 1;
    }
  }

  // --- ragged layout (Appendix B) and ratios (Eq. 6) -----------------------
  p->layer_count.assign(L, 0);
  p->layer_offset.assign(L + 1, 0);
  int64_t r_max = 0;
  for (int64_t l = 0; l < L; ++l) {
    const uint8_t *m = p->mask.data() + l * n_l;
    const int64_t r = std::count(m, m + n_l, uint8_t{1});
    p->layer_count[l] = r;
    p->layer_offset[l + 1] = p->layer_offset[l] + r;
    r_max = std::max(r_max, r);
  }
  const int64_t sum_r = p->layer_offset[L];

  // --- replay windows (Eq. 7) ---------------------------------------------
  double cap = d->w_max;
  if (d->sel != DASC_SEL_THRESHOLD && !(d->w_max > 0.0)) {
    double hmax = 0.0;
    for (int64_t u = 0; u < n_all; ++u)
      if (!p->mask[u]) hmax = std::max(hmax, p->horizon[u]);
    cap = pow2_ceil(hmax);
    if (hmax > 0.0) cap = std::max(cap, 4.0);
  }
  p->window.resize(n_all);
  double w_replay = 0.0;
  const double w_clip = 9.0e18;  // keep the int64 conversion defined for absurd caps
  for (int64_t u = 0; u < n_all; ++u) {
    double w = std::max(pow2_ceil(p->horizon[u]), 4.0);
    w = std::min(w, cap);
    p->window[u] = static_cast<int64_t>(std::min(w, w_clip));
    if (!p->mask[u]) w_replay = std::max(w_replay, w);
  }

  dasc_plan_info_t &o = p->info;
  o.kind = d->kind;
  o.n_layers = d->n_layers;
  o.n_v_heads = d->n_v_heads;
  o.n_k_heads = d->n_k_heads;
  o.d_k = d->d_k;
  o.d_v = d->d_v;
  o.units_per_layer = n_l;
  o.unit_floats = unit_floats;
  o.units_total = n_all;
  o.units_retained = sum_r;
  o.r_max = r_max;
  o.slot_floats = sum_r * unit_floats;
  o.dense_floats_per_layer = rows_per_layer * d->d_v;
  const double inf = std::numeric_limits<double>::infinity();
  o.c_temp_rag = sum_r ? static_cast<double>(n_all) / static_cast<double>(sum_r) : inf;
  o.c_temp_pad = r_max ? static_cast<double>(n_all) / (static_cast<double>(L) * static_cast<double>(r_max)) : inf;
  const double b_dense = static_cast<double>(n_all) * unit_floats * 4.0;
  const double b_rag = static_cast<double>(sum_r) * unit_floats * 4.0;
  const double b_conv = static_cast<double>(d->conv_bytes_per_ckpt);
  o.c_ckpt_rag = (b_rag + b_conv) > 0.0 ? (b_dense + b_conv) / (b_rag + b_conv) : inf;
  o.w_max_used = cap;
  o.w_replay = static_cast<int64_t>(std::min(w_replay, w_clip));
  o.device = -1;
  dasc_plan_row_tables(p);
  return DASC_OK;
}

// Row tables of the copy kernels from info + mask (also used when a saved plan is loaded): a row is d_v floats, a GDN
// unit is d_k consecutive rows; row_src lists the retained rows in packed order, row_pos is its inverse (-1 = omitted).
void dasc_plan_row_tables(dasc_plan_s *p) {
  const dasc_plan_info_t &o = p->info;
  const int64_t L = o.n_layers, n_l = o.units_per_layer;
  const int64_t rows_per_unit = o.unit_floats / o.d_v;
  const int64_t rows_per_layer = n_l * rows_per_unit;
  p->rows_per_layer = rows_per_layer;
  p->packed_rows = o.units_retained * rows_per_unit;
  p->row_src.clear();
  p->row_src.reserve(p->packed_rows);
  p->row_pos.assign(L * rows_per_layer, -1);
  for (int64_t l = 0; l < L; ++l) {
    for (int64_t u = 0; u < n_l; ++u) {
      if (!p->mask[l * n_l + u]) continue;
      for (int64_t j = 0; j < rows_per_unit; ++j) {
        const int64_t row = u * rows_per_unit + j;
        p->row_pos[l * rows_per_layer + row] = static_cast<int32_t>(p->row_src.size());
        p->row_src.push_back({static_cast<int32_t>(l), static_cast<int32_t>(row)});
      }
    }
  }
}
