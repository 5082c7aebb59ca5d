// Load-aware dynamic transfer (Section 4.4): Algorithm 2 (Dynamic Transfer Scheduling) and Algorithm 3 (Load-aware
// Re-scheduling) as host utilities.  Pure host code, double precision, no context.
//
// A round executes tensors 0..n-1 in order.  b[i] is the default backend of tensor i (static placement); a GPU-resident
// tensor stays on the GPU, a host tensor either runs on the host or is promoted: its weights cross PCIe while the tensors
// before it execute, and only the part of the transfer that the window does not hide is paid.
//
//   seg(j, i)  = sum over k strictly between j and i of  t_k on backend b_k  +  c_k [b_{k-1} != b_k]      (default path)
//   T(rb)      = sum_i t_i on rb_i  +  sum_{i>=1} c_i [rb_{i-1} != rb_i]  +  sum over promoted i of max(w_i - seg(j_i, i), 0)
//
// With cost_k = t_k^{b_k} + c_k [b_{k-1} != b_k] (no switch for k = 0) and prefix sums P, seg(j, i) = P[i] - P[j + 1] for a
// start tensor j and P[i] for the round start, so the table of interval values is never stored: O(n) space, O(n^2) time.
//
// Readings of the listing (stated once here, used by both entry points):
//  * the round start is a legal transfer start point (state value 0), so the first host tensor of a round can be promoted;
//  * the switch cost at a promoted tensor follows the objective: c_i is paid when its default predecessor is on the host;
//  * the start point j_i of each promoted tensor's transfer is part of the plan (the listing minimises over it): it is the
//    round start or a host tensor that runs on the host, and nothing between j_i and i is promoted.
// Ties keep the earlier candidate: same-backend predecessor before the other, smaller j first, host before GPU at the end.
#include <cmath>
#include <limits>
#include <vector>

#include "ats_internal.h"

namespace {

constexpr double kInf = std::numeric_limits<double>::infinity();
constexpr int32_t kNoTransfer = -2, kRoundStart = -1;

struct Inputs {
  const uint8_t* b;
  const double *t_gpu, *t_host, *c, *w;
  uint32_t n;
};

bool finite_nonneg(const double* v, uint32_t n) {
  for (uint32_t i = 0; i < n; ++i)
    if (!(v[i] >= 0.0) || std::isinf(v[i])) return false;
  return true;
}

int32_t check_inputs(const Inputs& in) {
  if (in.n == 0) return ATS_OK;
  if (!in.b || !in.t_gpu || !in.t_host || !in.c || !in.w) return ATS_ERR_INVALID;
  for (uint32_t i = 0; i < in.n; ++i)
    if (in.b[i] != ATS_HOST && in.b[i] != ATS_GPU) return ATS_ERR_INVALID;
  if (!finite_nonneg(in.t_gpu, in.n) || !finite_nonneg(in.t_host, in.n) || !finite_nonneg(in.c, in.n) || !finite_nonneg(in.w, in.n))
    return ATS_ERR_INVALID;
  return ATS_OK;
}

// P[k] = cost of default-path tensors 0..k-1
std::vector<double> default_prefix(const Inputs& in) {
  std::vector<double> P(in.n + 1, 0.0);
  for (uint32_t k = 0; k < in.n; ++k) {
    double cost = in.b[k] == ATS_GPU ? in.t_gpu[k] : in.t_host[k];
    if (k > 0 && in.b[k - 1] != in.b[k]) cost += in.c[k];
    P[k + 1] = P[k] + cost;
  }
  return P;
}

// seg between start point j (kRoundStart or a tensor index) and tensor i
inline double window(const std::vector<double>& P, int32_t j, uint32_t i) { return j == kRoundStart ? P[i] : P[i] - P[(size_t)j + 1]; }

void solve(const Inputs& in, uint8_t* rb, int32_t* start, double* latency) {
  const uint32_t n = in.n;
  const std::vector<double> P = default_prefix(in);
  // value of the best partial schedule that ends with tensor i on the host / on the GPU, and where it came from
  std::vector<double> vh(n, kInf), vg(n, kInf);
  std::vector<int32_t> from_h(n, kRoundStart), from_g(n, kRoundStart);  // predecessor tensor (kRoundStart = none)
  std::vector<uint8_t> from_h_state(n, ATS_HOST), from_g_state(n, ATS_HOST);
  for (uint32_t i = 0; i < n; ++i) {
    // extending the previous tensor: same backend first, then the other one plus the switch
    auto extend = [&](uint8_t to, double* val, int32_t* from, uint8_t* from_state) {
      if (i == 0) {
        *val = 0.0;
        *from = kRoundStart;
        *from_state = to;
        return;
      }
      const double same = to == ATS_GPU ? vg[i - 1] : vh[i - 1];
      const double other = (to == ATS_GPU ? vh[i - 1] : vg[i - 1]) + in.c[i];
      *from = (int32_t)i - 1;
      if (same <= other) {
        *val = same;
        *from_state = to;
      } else {
        *val = other;
        *from_state = to == ATS_GPU ? ATS_HOST : ATS_GPU;
      }
    };
    if (in.b[i] == ATS_GPU) {
      double v;
      extend(ATS_GPU, &v, &from_g[i], &from_g_state[i]);
      vg[i] = v + in.t_gpu[i];
      continue;
    }
    double v;
    extend(ATS_HOST, &v, &from_h[i], &from_h_state[i]);
    vh[i] = v + in.t_host[i];
    // promotion: the transfer starts at the round start or right after a host tensor j that ran on the host; what lies
    // between runs on its default backend, and the slower of the transfer and that window is what passes before i
    double best = std::max(in.w[i], window(P, kRoundStart, i));
    int32_t best_j = kRoundStart;
    for (uint32_t j = 0; j < i; ++j) {
      if (in.b[j] != ATS_HOST) continue;
      const double cand = vh[j] + std::max(in.w[i], window(P, (int32_t)j, i));
      if (cand < best) {
        best = cand;
        best_j = (int32_t)j;
      }
    }
    const double into = (i > 0 && in.b[i - 1] == ATS_HOST) ? in.c[i] : 0.0;
    vg[i] = best + into + in.t_gpu[i];
    from_g[i] = best_j;
    from_g_state[i] = ATS_HOST;
  }
  for (uint32_t i = 0; i < n; ++i) {
    rb[i] = in.b[i];
    if (start) start[i] = kNoTransfer;
  }
  if (n == 0) {
    if (latency) *latency = 0.0;
    return;
  }
  uint8_t s = vh[n - 1] <= vg[n - 1] ? ATS_HOST : ATS_GPU;
  if (latency) *latency = s == ATS_HOST ? vh[n - 1] : vg[n - 1];
  int32_t i = (int32_t)n - 1;
  while (i >= 0) {
    rb[i] = s;
    const int32_t pj = s == ATS_GPU ? from_g[i] : from_h[i];
    const uint8_t ps = s == ATS_GPU ? from_g_state[i] : from_h_state[i];
    if (in.b[i] == ATS_HOST && s == ATS_GPU && start) start[i] = pj;  // tensors between pj and i keep rb = b
    i = pj;
    s = ps;
  }
}

double latency_of(const Inputs& in, const uint8_t* rb, const int32_t* start, bool* ok) {
  const std::vector<double> P = default_prefix(in);
  double total = 0.0;
  *ok = true;
  for (uint32_t i = 0; i < in.n; ++i) {
    total += rb[i] == ATS_GPU ? in.t_gpu[i] : in.t_host[i];
    if (i > 0 && rb[i - 1] != rb[i]) total += in.c[i];
    if (in.b[i] == ATS_GPU && rb[i] != ATS_GPU) *ok = false;  // resident tensors stay on the GPU
    if (in.b[i] == ATS_HOST && rb[i] == ATS_GPU) {
      const int32_t j = start[i];
      if (j != kRoundStart && (j < 0 || (uint32_t)j >= i)) {
        *ok = false;
        continue;
      }
      total += std::max(in.w[i] - window(P, j, i), 0.0);
    }
  }
  return total;
}

}  // namespace

extern "C" {

int32_t ats_host_dynamic_transfer(const uint8_t* b, const double* t_gpu, const double* t_host, const double* c, const double* w,
                                  uint32_t n, uint8_t* out_rb, int32_t* out_start, double* out_latency) {
  const Inputs in{b, t_gpu, t_host, c, w, n};
  const int32_t st = check_inputs(in);
  if (st != ATS_OK) return st;
  if (n && !out_rb) return ATS_ERR_INVALID;
  solve(in, out_rb, out_start, out_latency);
  return ATS_OK;
}

int32_t ats_host_transfer_latency(const uint8_t* rb, const int32_t* start, const uint8_t* b, const double* t_gpu, const double* t_host,
                                  const double* c, const double* w, uint32_t n, double* out_latency) {
  const Inputs in{b, t_gpu, t_host, c, w, n};
  const int32_t st = check_inputs(in);
  if (st != ATS_OK) return st;
  if (!out_latency || (n && (!rb || !start))) return ATS_ERR_INVALID;
  for (uint32_t i = 0; i < n; ++i)
    if (rb[i] != ATS_HOST && rb[i] != ATS_GPU) return ATS_ERR_INVALID;
  bool ok = true;
  const double t = latency_of(in, rb, start, &ok);
  if (!ok) return ATS_ERR_INVALID;
  *out_latency = t;
  return ATS_OK;
}

double ats_host_deviation(const double* m_prev, const double* m_cur, uint32_t n) {
  double d = 0.0;
  if (!m_prev || !m_cur) return d;
  for (uint32_t i = 0; i < n; ++i) {
    if (m_prev[i] == m_cur[i]) continue;
    d = std::max(d, m_prev[i] != 0.0 ? std::fabs(m_cur[i] - m_prev[i]) / std::fabs(m_prev[i]) : kInf);
  }
  return d;
}

int32_t ats_host_reschedule(const uint8_t* b, uint32_t n, double* m_ref, const double* m_cur, double eps, double tau, double t_now,
                            double* t_last, uint8_t* rb, int32_t* start, int32_t* out_replanned) {
  if (!t_last || !out_replanned || (n && (!b || !m_ref || !m_cur || !rb))) return ATS_ERR_INVALID;
  *out_replanned = 0;
  const double d = ats_host_deviation(m_ref, m_cur, 4 * n);
  if (d < eps || t_now - *t_last < tau) return ATS_OK;  // keep the previous assignment
  const int32_t st = ats_host_dynamic_transfer(b, m_cur, m_cur + n, m_cur + 2 * (size_t)n, m_cur + 3 * (size_t)n, n, rb, start, nullptr);
  if (st != ATS_OK) return st;
  for (size_t i = 0; i < 4 * (size_t)n; ++i) m_ref[i] = m_cur[i];
  *t_last = t_now;
  *out_replanned = 1;
  return ATS_OK;
}

}  // extern "C"
