// Host-side planning of the Newton-Schulz polynomial schedule.
//
// Each step applies an odd quintic p(x) = a x + b x^3 + c x^5 to the singular values of the
// iterate.  For a spectrum known to lie in [l, 1] the step uses the quintic that minimises
// max |1 - p(x)| on [l, 1] (equioscillation at l, x1, x2, 1, found by a Remez exchange); after
// rescaling by 1/(1+E) the spectrum lies in [(1-E)/(1+E), 1] and the next step is planned for
// that interval.  For l -> 1 the quintic tends to the classical (15, -10, 3)/8.
//
// The kernels evaluate the step in residual form, with E = X^T X - I:
//   X <- gamma X + X (beta1 E + beta2 E^2),  gamma = a+b+c, beta1 = b+2c, beta2 = c,
// which keeps the matrix that is split into bf16 terms small near convergence.
#pragma once
#include <cmath>
#include <vector>

namespace conqur {

struct NsStep {
  double a, b, c;   // already rescaled so that p([l,1]) lies in [l_next, 1/(1+margin)]
  double l, err;    // interval lower end the step was planned for; equioscillation error
};

// Minimax odd quintic on [l, 1].  Returns false if the exchange failed (never seen for l in [1e-12, 1)).
inline bool remez_quintic(double l, double& a, double& b, double& c, double& err) {
  if (l >= 1.0 - 1e-7) {
    a = 15.0 / 8.0; b = -10.0 / 8.0; c = 3.0 / 8.0; err = 0.0;
    return true;
  }
  double x1 = (l < 0.09) ? std::sqrt(l) : l + (1.0 - l) / 3.0;
  double x2 = (l < 0.6) ? 0.8 : l + 2.0 * (1.0 - l) / 3.0;
  for (int it = 0; it < 300; ++it) {
    // solve [x x^3 x^5 s] [a b c E]^T = 1 at the four reference points, s = +1,-1,+1,-1
    const double px[4] = {l, x1, x2, 1.0};
    double m[4][5];
    for (int r = 0; r < 4; ++r) {
      const double x = px[r], x3 = x * x * x;
      m[r][0] = x; m[r][1] = x3; m[r][2] = x3 * x * x; m[r][3] = (r & 1) ? -1.0 : 1.0; m[r][4] = 1.0;
    }
    for (int col = 0; col < 4; ++col) {          // Gaussian elimination with partial pivoting
      int piv = col;
      for (int r = col + 1; r < 4; ++r)
        if (std::fabs(m[r][col]) > std::fabs(m[piv][col])) piv = r;
      if (m[piv][col] == 0.0) return false;
      if (piv != col)
        for (int k = 0; k < 5; ++k) { const double t = m[piv][k]; m[piv][k] = m[col][k]; m[col][k] = t; }
      for (int r = 0; r < 4; ++r) {
        if (r == col) continue;
        const double f = m[r][col] / m[col][col];
        for (int k = col; k < 5; ++k) m[r][k] -= f * m[col][k];
      }
    }
    a = m[0][4] / m[0][0]; b = m[1][4] / m[1][1]; c = m[2][4] / m[2][2]; err = m[3][4] / m[3][3];
    // interior extrema of p: a + 3 b t + 5 c t^2 = 0, t = x^2
    const double disc = 9.0 * b * b - 20.0 * a * c;
    if (!(disc > 0.0) || c == 0.0) return false;
    const double sq = std::sqrt(disc);
    double t1 = (-3.0 * b - sq) / (10.0 * c), t2 = (-3.0 * b + sq) / (10.0 * c);
    if (t1 > t2) { const double t = t1; t1 = t2; t2 = t; }
    if (!(t1 > 0.0)) return false;
    const double n1 = std::sqrt(t1), n2 = std::sqrt(t2);
    const double moved = std::fabs(n1 - x1) + std::fabs(n2 - x2);
    x1 = n1; x2 = n2;
    if (moved < 1e-15) break;
  }
  return std::isfinite(a) && std::isfinite(b) && std::isfinite(c) && std::isfinite(err);
}

// Steps that take a spectrum in [l0, 1] to within `final_err` of 1.  `margin` shrinks the output of the
// steps planned for l < 0.5 so that rounding cannot push a singular value above 1.
inline std::vector<NsStep> plan_schedule(double l0, double margin, double final_err, int max_len) {
  std::vector<NsStep> out;
  double l = l0;
  while ((int)out.size() < max_len) {
    NsStep s;
    s.l = l;
    if (!remez_quintic(l, s.a, s.b, s.c, s.err)) {
      s.a = 15.0 / 8.0; s.b = -10.0 / 8.0; s.c = 3.0 / 8.0; s.err = 0.0;
    }
    const double mg = (l < 0.5) ? margin : 0.0;
    const double sc = 1.0 / ((1.0 + s.err) * (1.0 + mg));
    s.a *= sc; s.b *= sc; s.c *= sc;
    out.push_back(s);
    if (s.err <= final_err) break;
    l = (1.0 - s.err) / (1.0 + s.err) / (1.0 + mg);
  }
  return out;
}

// Smallest-l0 (most conservative) schedule that still has at most `steps` entries.
inline std::vector<NsStep> plan_schedule_for_steps(int steps, double margin, double final_err) {
  double lo = std::log(1e-12), hi = std::log(0.5);
  for (int it = 0; it < 60; ++it) {
    const double mid = 0.5 * (lo + hi);
    if ((int)plan_schedule(std::exp(mid), margin, final_err, steps + 1).size() <= steps) hi = mid; else lo = mid;
  }
  return plan_schedule(std::exp(hi), margin, final_err, steps + 1);
}

}  // namespace conqur
