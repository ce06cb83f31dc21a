// Host-side planning of the Newton-Schulz polynomial schedule.
//
// Each step applies an odd quintic p(x) = a x + b x^3 + c x^5 to the singular values of the
// iterate X (so U V^T, the polar factor, is untouched).  Two kinds of step:
//
//   lifting   the SAME quintic p_f every step: the minimax quintic for |1 - p| on [l_f, 1], rescaled so
//             that its range on [l_f, 1] is [floor, 1/(1+margin)].  Singular values below l_f grow by the
//             factor a_f per step, and a singular value that has reached [l_f, 1] can never fall below
//             `floor` again.  (The minimax quintic for the interval the spectrum is actually known to lie
//             in, [l, 1] with l tiny, grows small singular values a little faster, but it maps some LARGE
//             singular values back down to about l, where rounding noise destroys their directions.)
//   endgame   the minimax quintics for [floor, 1], then for the interval that one maps to, and so on
//             until the equioscillation error is below `final_err`; the last ones tend to (15, -10, 3)/8.
//
// The number of lifting steps is fixed by the assumed lower bound l0 on sigma_min(X_0): p_f is applied until it has
// carried l0 above l_f (about log(l_f / l0) / log(a_f) times); the endgame starts from the value reached.
//
// The kernels evaluate a step in shifted residual form.  With G = X^T X = tau I + E,
//   p:  X <- X (a + b G + c G^2) = gamma X + X (beta1 E + beta2 E^2),
//   gamma = a + b tau + c tau^2,  beta1 = b + 2 c tau,  beta2 = c,
// for any shift tau (tau = mean sigma^2 keeps E small at both ends of the iteration).
#pragma once
#include <algorithm>
#include <cmath>
#include <vector>

namespace conqur {

struct NsStep {
  double a, b, c;   // already rescaled: p maps [l, 1] into [l_next, 1/(1+margin)]
  double l, err;    // interval lower end the quintic was fitted for; its equioscillation error
  int lift;         // 1: a lifting step (repeated polynomial)
  int seg_x;        // tensor-core mode: 2 = the iterate enters the last product as hi + lo, 1 = hi only
};

namespace detail {
inline bool solve4(double m[4][5]) {
  for (int col = 0; col < 4; ++col) {          // Gaussian elimination with partial pivoting
    int piv = col;
    for (int r = col + 1; r < 4; ++r)
      if (std::fabs(m[r][col]) > std::fabs(m[piv][col])) piv = r;
    if (m[piv][col] == 0.0) return false;
    if (piv != col)
      for (int k = 0; k < 5; ++k) std::swap(m[piv][k], m[col][k]);
    for (int r = 0; r < 4; ++r) {
      if (r == col) continue;
      const double f = m[r][col] / m[col][col];
      for (int k = col; k < 5; ++k) m[r][k] -= f * m[col][k];
    }
  }
  return true;
}
// coefficients with p(x_r) + s_r E = 1 at the four reference points, s = +,-,+,-
inline bool fit4(const double x[4], double& a, double& b, double& c, double& e) {
  double m[4][5];
  for (int r = 0; r < 4; ++r) {
    const double t = x[r], t3 = t * t * t;
    m[r][0] = t; m[r][1] = t3; m[r][2] = t3 * t * t; m[r][3] = (r & 1) ? -1.0 : 1.0; m[r][4] = 1.0;
  }
  if (!solve4(m)) return false;
  a = m[0][4] / m[0][0]; b = m[1][4] / m[1][1]; c = m[2][4] / m[2][2]; e = m[3][4] / m[3][3];
  return std::isfinite(a) && std::isfinite(b) && std::isfinite(c) && std::isfinite(e);
}
}  // namespace detail

// Minimax odd quintic for |1 - p| on [l, 1]: p = 1-E at l, 1+E at x1, 1-E at x2, 1+E at 1.
// Remez exchange on a grid (robust for every l in [1e-12, 1)), then polished on the exact stationary points.
inline bool remez_quintic(double l, double& a, double& b, double& c, double& err) {
  if (l >= 1.0 - 1e-7) {
    a = 15.0 / 8.0; b = -10.0 / 8.0; c = 3.0 / 8.0; err = 0.0;
    return true;
  }
  const int NG = 4096;
  std::vector<double> g(2 * NG);
  const double ll = std::log(l);
  for (int i = 0; i < NG; ++i) {
    g[i] = std::exp(ll * (1.0 - (double)i / (NG - 1)));          // log-spaced l .. 1
    g[NG + i] = l + (1.0 - l) * (double)i / (NG - 1);             // linearly spaced
  }
  std::sort(g.begin(), g.end());
  const int n = (int)g.size();
  double x[4] = {l, (l < 0.09) ? std::sqrt(l) : l + 0.35 * (1.0 - l), (l < 0.6) ? 0.8 : l + 0.75 * (1.0 - l), 1.0};
  bool ok = false;
  for (int it = 0; it < 100; ++it) {
    if (!detail::fit4(x, a, b, c, err)) return false;
    ok = true;
    int i1 = 1, i2 = -1;
    double best = 1e300;
    for (int i = 1; i < n - 2; ++i) {                             // where p is largest
      const double t = g[i], t2 = t * t, w = 1.0 - t * (a + t2 * (b + t2 * c));
      if (w < best) { best = w; i1 = i; }
    }
    best = -1e300;
    for (int i = i1 + 1; i < n - 1; ++i) {                        // where p is smallest to the right of it
      const double t = g[i], t2 = t * t, w = 1.0 - t * (a + t2 * (b + t2 * c));
      if (w > best) { best = w; i2 = i; }
    }
    if (i2 < 0) break;
    const double moved = std::fabs(g[i1] - x[1]) + std::fabs(g[i2] - x[2]);
    x[1] = g[i1]; x[2] = g[i2];
    if (moved < 1e-14) break;
  }
  if (!ok) return false;
  for (int it = 0; it < 60; ++it) {                               // polish: interior extrema of p solve a + 3 b t + 5 c t^2 = 0
    double a2, b2, c2, e2;
    if (!detail::fit4(x, a2, b2, c2, e2)) break;
    a = a2; b = b2; c = c2; err = e2;
    const double disc = 9.0 * b * b - 20.0 * a * c;
    if (!(disc > 0.0) || c == 0.0) break;
    const double sq = std::sqrt(disc);
    double t1 = (-3.0 * b - sq) / (10.0 * c), t2 = (-3.0 * b + sq) / (10.0 * c);
    if (t1 > t2) std::swap(t1, t2);
    if (!(t1 > 0.0)) break;
    const double n1 = std::sqrt(t1), n2 = std::sqrt(t2);
    if (!(l < n1 && n1 < n2 && n2 < 1.0)) break;
    const double moved = std::fabs(n1 - x[1]) + std::fabs(n2 - x[2]);
    x[1] = n1; x[2] = n2;
    if (moved < 1e-15) break;
  }
  err = std::fabs(err);
  return std::isfinite(a) && std::isfinite(b) && std::isfinite(c) && std::isfinite(err);
}

struct NsPlanParams {
  double l0 = 1e-9;          // assumed lower bound on sigma_min(X_0) (X_0 = M / (||M||_F (1+margin)))
  double l_lift = 0.05;      // l_f: interval lower end of the repeated lifting quintic
  double margin = 2e-2;      // shrink of every quintic fitted for l < 0.5: keeps rounding from pushing a singular value above 1
  double final_err = 1e-6;
  int max_len = 100;
  int d = 0;                 // for seg_x; 0: always 2
  double gap_budget = 5e-4;  // worst-case bound on the Procrustes gap given up by dropping the iterate's lo part
};

// One endgame/lifting quintic for the interval [l, 1], rescaled; returns the lower end of its range.
inline double ns_make_step(double l, double margin, NsStep* s) {
  s->l = l;
  if (!remez_quintic(l, s->a, s->b, s->c, s->err)) {
    s->a = 15.0 / 8.0; s->b = -10.0 / 8.0; s->c = 3.0 / 8.0; s->err = 0.0;
  }
  const double mg = (l < 0.5) ? margin : 0.0;
  const double sc = 1.0 / ((1.0 + s->err) * (1.0 + mg));
  s->a *= sc; s->b *= sc; s->c *= sc;
  s->lift = 0; s->seg_x = 2;
  return (1.0 - s->err) / (1.0 + s->err) / (1.0 + mg);
}

// The schedule for a spectrum assumed to lie in [l0, 1].  *first_endgame receives the index of the first
// endgame step (the number of lifting steps).
inline std::vector<NsStep> plan_schedule(const NsPlanParams& p, int* first_endgame = nullptr) {
  std::vector<NsStep> out;
  double l = std::min(std::max(p.l0, 1e-12), 1.0);
  int n_lift = 0;
  if (l < p.l_lift) {
    NsStep f;
    ns_make_step(p.l_lift, p.margin, &f);
    f.lift = 1;
    // follow the assumed lower bound through the lifting steps (p_f is increasing below its first maximum)
    while (l < p.l_lift && n_lift < p.max_len - 1) {
      const double l2 = l * l;
      l = l * (f.a + l2 * (f.b + l2 * f.c));
      out.push_back(f);
      ++n_lift;
    }
  }
  if (first_endgame) *first_endgame = n_lift;
  while ((int)out.size() < p.max_len) {
    NsStep s;
    const double next = ns_make_step(l, p.margin, &s);
    out.push_back(s);
    if (s.err <= p.final_err) break;
    l = next;
  }
  // Precision of the iterate in the last product.  bf16 rounding of X adds noise of spectral size about
  // 2^-8 * rms(sigma) <= 2^-8; after a cumulative growth G of the small singular values, the directions it can
  // scramble had sigma_0 <= 2^-8 / G relative to the largest, at most d of them: Procrustes gap <= d 2^-8 / G.
  double G = 1.0;
  for (NsStep& s : out) {
    s.seg_x = (p.d <= 0 || (double)p.d * (1.0 / 256.0) / G > p.gap_budget) ? 2 : 1;
    G *= s.a;
  }
  return out;
}

// The schedule the device runs: entry 0 is the lifting quintic p_f, entries 1.. are the endgame for a spectrum in
// [floor, 1], floor being the lower end of p_f's range on [l_f, 1].  How many times p_f is applied is decided per
// update on the device; *n_lift receives the count that carries the assumed bound l0 above the floor.
inline std::vector<NsStep> plan_device_schedule(const NsPlanParams& p, int* n_lift) {
  NsStep f;
  const double floor = ns_make_step(p.l_lift, p.margin, &f);
  f.lift = 1;
  std::vector<NsStep> out;
  out.push_back(f);
  NsPlanParams q = p;
  q.l0 = floor;
  q.max_len = p.max_len - 1;
  for (const NsStep& s : plan_schedule(q)) out.push_back(s);
  double l = std::min(std::max(p.l0, 1e-12), 1.0);
  int n = 0;
  while (l < floor && n < 60) {
    const double l2 = l * l;
    l = l * (f.a + l2 * (f.b + l2 * f.c));
    ++n;
  }
  if (n_lift) *n_lift = n;
  return out;
}

// The most conservative schedule (smallest l0) that still has at most `steps` entries.
inline std::vector<NsStep> plan_schedule_for_steps(int steps, NsPlanParams p, int* first_endgame = nullptr) {
  double lo = std::log(1e-12), hi = std::log(0.9);
  p.max_len = steps + 1;
  for (int it = 0; it < 60; ++it) {
    const double mid = 0.5 * (lo + hi);
    p.l0 = std::exp(mid);
    if ((int)plan_schedule(p).size() <= steps) hi = mid; else lo = mid;
  }
  p.l0 = std::exp(hi);
  return plan_schedule(p, first_endgame);
}

}  // namespace conqur
