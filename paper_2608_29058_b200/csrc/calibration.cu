// Offline calibration statistics (Section 3.5) and the cost table of Section 3.1, as host functions of the library:
// the one-sided residual quantile delta_q, the monotone predictor e of Eq. 4 (non-negative weights by least squares,
// then a non-decreasing step function of the weighted score), and the apportioning of measured kernel times over the
// items of a layer.  Plain C++ on a few hundred records; nothing here touches the GPU.
#include <algorithm>
#include <cmath>
#include <vector>

#include "common.cuh"

namespace {

constexpr int kMaxFeatures = 16;

// min ||X w - y||^2 subject to w >= 0: projected gradient with step 1 / trace(X^T X) (an upper bound of the largest
// eigenvalue), run until the iterate stops moving.
void nonneg_least_squares(int n, int nf, const double* X, const double* y, double* w) {
  std::vector<double> G((size_t)nf * nf, 0.0), b(nf, 0.0);
  for (int i = 0; i < n; ++i)
    for (int a = 0; a < nf; ++a) {
      b[a] += X[(size_t)i * nf + a] * y[i];
      for (int c = 0; c < nf; ++c) G[(size_t)a * nf + c] += X[(size_t)i * nf + a] * X[(size_t)i * nf + c];
    }
  double tr = 0.0;
  for (int a = 0; a < nf; ++a) tr += G[(size_t)a * nf + a];
  for (int a = 0; a < nf; ++a) w[a] = 0.0;
  if (!(tr > 0.0)) return;
  const double step = 1.0 / tr;
  std::vector<double> g(nf);
  for (int it = 0; it < 2000000; ++it) {
    double moved = 0.0;
    for (int a = 0; a < nf; ++a) {
      double acc = -b[a];
      for (int c = 0; c < nf; ++c) acc += G[(size_t)a * nf + c] * w[c];
      g[a] = acc;
    }
    for (int a = 0; a < nf; ++a) {
      const double nw = std::max(0.0, w[a] - step * g[a]);
      moved = std::max(moved, std::fabs(nw - w[a]));
      w[a] = nw;
    }
    if (moved < 1e-15) break;
  }
}

struct Block { double z, sum, cnt; };

}  // namespace

extern "C" int rs_calibration_fit(int n_records, int n_features, const double* features, const double* target,
                                  const double* residual, double q, int max_breakpoints, double* delta_q, double* w,
                                  double* bp_z, double* bp_e, int* n_bp) {
  if (n_records <= 0 || n_features <= 0 || n_features > kMaxFeatures || !features || !target || !residual || !delta_q ||
      !w || !bp_z || !bp_e || !n_bp || max_breakpoints < 1 || !(q > 0.0) || q > 1.0)
    return RS_ERR_INVALID_ARG;
  const int n = n_records, nf = n_features;
  // delta_q: the ceil(q n)-th smallest residual, floored at 0 (only over-estimates of the mass are corrected)
  {
    std::vector<double> r(residual, residual + n);
    std::sort(r.begin(), r.end());
    int k = (int)std::ceil(q * n);
    k = std::min(std::max(k, 1), n);
    *delta_q = std::max(0.0, r[k - 1]);
  }
  nonneg_least_squares(n, nf, features, target, w);
  bool any = false;
  for (int a = 0; a < nf; ++a) any |= w[a] > 0.0;
  if (!any) w[0] = 1.0;                                   // fall back to the first feature alone (1 - m_hat)
  // non-decreasing least-squares step function of the target on z = features . w: records in order of z (ties form one
  // point), neighbouring blocks merged while the left mean exceeds the right mean
  std::vector<std::pair<double, double>> zy(n);
  for (int i = 0; i < n; ++i) {
    double z = 0.0;
    for (int a = 0; a < nf; ++a) z += features[(size_t)i * nf + a] * w[a];
    zy[i] = {z, target[i]};
  }
  std::stable_sort(zy.begin(), zy.end(), [](const std::pair<double, double>& a, const std::pair<double, double>& b) { return a.first < b.first; });
  std::vector<Block> st;
  for (int i = 0; i < n;) {
    Block blk{zy[i].first, 0.0, 0.0};
    int j = i;
    while (j < n && zy[j].first == zy[i].first) { blk.sum += zy[j].second; blk.cnt += 1.0; ++j; }
    st.push_back(blk);
    while (st.size() > 1) {
      Block& a = st[st.size() - 2];
      Block& b = st[st.size() - 1];
      if (a.sum * b.cnt > b.sum * a.cnt) { a.sum += b.sum; a.cnt += b.cnt; st.pop_back(); }
      else break;
    }
    i = j;
  }
  // at most max_breakpoints steps (the device table's size): the breakpoint with the smallest jump goes first
  std::vector<double> bz, be;
  for (const Block& b : st) { bz.push_back(b.z); be.push_back(b.sum / b.cnt); }
  while ((int)bz.size() > max_breakpoints) {
    size_t k = 0;
    for (size_t i = 1; i + 1 < bz.size(); ++i)
      if (be[i + 1] - be[i] < be[k + 1] - be[k]) k = i;
    bz.erase(bz.begin() + (long)k + 1);
    be.erase(be.begin() + (long)k + 1);
  }
  *n_bp = (int)bz.size();
  for (size_t i = 0; i < bz.size(); ++i) { bp_z[i] = bz[i]; bp_e[i] = be[i]; }
  return RS_OK;
}

extern "C" int rs_cost_table_from_times(int n_items, int n_cand, const double* cand_ms, const uint64_t* pairs,
                                        int64_t* table) {
  if (n_items <= 0 || n_cand <= 0 || !cand_ms || !pairs || !table) return RS_ERR_INVALID_ARG;
  for (int c = 0; c < n_cand; ++c) {
    long double tot = 0.0L;
    for (int it = 0; it < n_items; ++it) tot += (long double)pairs[(size_t)it * n_cand + c];
    for (int it = 0; it < n_items; ++it) {
      const double share = tot > 0.0L ? (double)((long double)pairs[(size_t)it * n_cand + c] / tot) : 1.0 / n_items;
      const double ns = std::nearbyint(cand_ms[c] * 1e6 * share);
      table[(size_t)it * n_cand + c] = ns < 1.0 ? 1 : (int64_t)ns;
    }
  }
  return RS_OK;
}
