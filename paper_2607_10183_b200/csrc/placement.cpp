// Static tensor placement (Algorithm 1; objective and constraint of Section 4.3.2).
//
//   maximise  sum_i r_i [b_i = GPU]  -  sum_{i>=2} c_i [b_i != b_{i-1}]   s.t.  sum_i s_i [b_i = GPU] <= M
//
// solved by a knapsack dynamic program over (tensor, memory units, backend of the tensor) with the
// placement recovered by backtracking; O(nM) time and space with sizes and budget quantised to a
// granule (the paper uses MB granularity).  Pure host integer code.
#include <limits>

#include "ats_internal.h"

namespace ats {

namespace {
constexpr int64_t kNeg = std::numeric_limits<int64_t>::min() / 4;  // "infeasible"
}

// State V[i][m][B]: best objective of tensors 0..i using at most m units, tensor i on backend B.
// Ties keep the predecessor that is on the same backend; a final tie keeps HOST.
void solve_knapsack_dp(const std::vector<int64_t>& s, const std::vector<int64_t>& r, const std::vector<int64_t>& c,
                       int64_t M, std::vector<uint8_t>* b, int64_t* objective) {
  const size_t n = s.size();
  b->assign(n, ATS_HOST);
  if (objective) *objective = 0;
  if (n == 0) return;
  if (M < 0) M = 0;
  const size_t W = (size_t)M + 1;
  std::vector<int64_t> vh(n * W, 0), vg(n * W, kNeg);
  std::vector<uint8_t> ph(n * W, ATS_HOST), pg(n * W, ATS_HOST);  // backend of tensor i-1 on the best path
  for (size_t i = 0; i < n; ++i) {
    const int64_t si = s[i], ri = r[i], ci = c[i];
    for (size_t m = 0; m < W; ++m) {
      if (i == 0) {
        if ((int64_t)m >= si) vg[m] = ri;
        continue;
      }
      {  // tensor i on the host
        const int64_t same = vh[(i - 1) * W + m];
        const int64_t g = vg[(i - 1) * W + m];
        const int64_t other = g > kNeg / 2 ? g - ci : kNeg;
        if (same >= other) {
          vh[i * W + m] = same;
          ph[i * W + m] = ATS_HOST;
        } else {
          vh[i * W + m] = other;
          ph[i * W + m] = ATS_GPU;
        }
      }
      if ((int64_t)m >= si) {  // tensor i on the GPU
        const size_t mm = m - (size_t)si;
        const int64_t same = vg[(i - 1) * W + mm];
        const int64_t other = vh[(i - 1) * W + mm] - ci;
        if (same > kNeg / 2 && same >= other) {
          vg[i * W + m] = ri + same;
          pg[i * W + m] = ATS_GPU;
        } else {
          vg[i * W + m] = ri + other;
          pg[i * W + m] = ATS_HOST;
        }
      }
    }
  }
  const int64_t fh = vh[(n - 1) * W + M], fg = vg[(n - 1) * W + M];
  uint8_t cur = fh >= fg ? ATS_HOST : ATS_GPU;
  if (objective) *objective = fh >= fg ? fh : fg;
  size_t m = (size_t)M;
  for (size_t i = n; i-- > 0;) {
    (*b)[i] = cur;
    uint8_t prev;
    if (cur == ATS_GPU) {
      prev = pg[i * W + m];
      m -= (size_t)s[i];
    } else {
      prev = ph[i * W + m];
    }
    cur = prev;
  }
}

// Algorithm 1 with its expert / non-expert partition for MoE models: if the non-expert tensors fit the budget they
// all become resident and the DP distributes what is left over the expert tensors; otherwise every expert tensor
// stays on the host and the DP runs over the non-expert tensors with the full budget.
void static_placement(const std::vector<int64_t>& s, const std::vector<int64_t>& r, const std::vector<int64_t>& c,
                      const std::vector<uint8_t>& is_expert, int64_t M, std::vector<uint8_t>* b) {
  const size_t n = s.size();
  bool any_expert = false;
  for (size_t i = 0; i < n; ++i) any_expert |= is_expert[i] != 0;
  if (!any_expert) {
    solve_knapsack_dp(s, r, c, M, b, nullptr);
    return;
  }
  std::vector<size_t> sub;
  int64_t s_non = 0;
  for (size_t i = 0; i < n; ++i)
    if (!is_expert[i]) s_non += s[i];
  b->assign(n, ATS_HOST);
  int64_t rest;
  if (M >= s_non) {
    for (size_t i = 0; i < n; ++i)
      if (!is_expert[i]) (*b)[i] = ATS_GPU;
    for (size_t i = 0; i < n; ++i)
      if (is_expert[i]) sub.push_back(i);
    rest = M - s_non;
  } else {
    for (size_t i = 0; i < n; ++i)
      if (!is_expert[i]) sub.push_back(i);
    rest = M;
  }
  std::vector<int64_t> ss, rr, cc;
  for (size_t i : sub) {
    ss.push_back(s[i]);
    rr.push_back(r[i]);
    cc.push_back(c[i]);
  }
  std::vector<uint8_t> sol;
  solve_knapsack_dp(ss, rr, cc, rest, &sol, nullptr);
  for (size_t j = 0; j < sub.size(); ++j) (*b)[sub[j]] = sol[j];
}

// Interchange layout -> internal slice layout (see ats_internal.h).  Per 4 input bytes (8 codes):
// nibble k of the input goes to word position (k even ? k/2 : 4 + k/2), XOR 8 turns two's complement into offset binary.
void repack_q4(const uint8_t* codes_in, const uint16_t* scales_in, uint8_t* slice_out, uint64_t n_rows, uint64_t K) {
  const uint64_t words = n_rows * K / 8;
  const uint32_t* in = reinterpret_cast<const uint32_t*>(codes_in);
  uint32_t* out = reinterpret_cast<uint32_t*>(slice_out);
  const bool aligned = (reinterpret_cast<uintptr_t>(codes_in) & 3) == 0;
  for (uint64_t w = 0; w < words; ++w) {
    uint32_t v;
    if (aligned) {
      v = in[w];
    } else {
      const uint8_t* p = codes_in + 4 * w;
      v = (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
    }
    v ^= 0x88888888u;
    // even nibbles (k = 0,2,4,6) sit at bit 0,8,16,24 of v; odd ones at bit 4,12,20,28
    const uint32_t ev = v & 0x0F0F0F0Fu, od = (v >> 4) & 0x0F0F0F0Fu;
    const uint32_t evp = (ev & 0xF) | ((ev >> 4) & 0xF0) | ((ev >> 8) & 0xF00) | ((ev >> 12) & 0xF000);
    const uint32_t odp = (od & 0xF) | ((od >> 4) & 0xF0) | ((od >> 8) & 0xF00) | ((od >> 12) & 0xF000);
    out[w] = evp | (odp << 16);
  }
  uint16_t* so = reinterpret_cast<uint16_t*>(slice_out + n_rows * K / 2);
  const uint64_t ns = n_rows * (K / kBlock);
  for (uint64_t i = 0; i < ns; ++i) so[i] = scales_in[i];
}

// The microscaling 4-bit format into the same slice layout.  The element encodings are kept (no offset), in the same
// nibble order; a scale byte b (2^(b - 127), accepted range 104..140) becomes the fp16 with that value: a normal number
// for exponents >= -14, a subnormal (one mantissa bit) below.
void repack_mxfp4(const uint8_t* codes_in, const uint8_t* scale_bytes_in, uint8_t* slice_out, uint64_t n_rows, uint64_t K) {
  const uint64_t words = n_rows * K / 8;
  uint32_t* out = reinterpret_cast<uint32_t*>(slice_out);
  for (uint64_t w = 0; w < words; ++w) {
    const uint8_t* p = codes_in + 4 * w;
    const uint32_t v = (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
    const uint32_t ev = v & 0x0F0F0F0Fu, od = (v >> 4) & 0x0F0F0F0Fu;
    const uint32_t evp = (ev & 0xF) | ((ev >> 4) & 0xF0) | ((ev >> 8) & 0xF00) | ((ev >> 12) & 0xF000);
    const uint32_t odp = (od & 0xF) | ((od >> 4) & 0xF0) | ((od >> 8) & 0xF00) | ((od >> 12) & 0xF000);
    out[w] = evp | (odp << 16);
  }
  uint16_t* so = reinterpret_cast<uint16_t*>(slice_out + n_rows * K / 2);
  const uint64_t ns = n_rows * (K / kBlock);
  for (uint64_t i = 0; i < ns; ++i) {
    const int e = (int)scale_bytes_in[i] - 127;
    so[i] = e >= -14 ? (uint16_t)((e + 15) << 10) : (uint16_t)(1u << (e + 24));
  }
}

}  // namespace ats

extern "C" {

int32_t ats_host_solve_placement(const int64_t* s, const int64_t* r, const int64_t* c, const uint8_t* is_expert, uint32_t n,
                                 int64_t M, uint8_t* out_b, int64_t* out_objective) {
  if (n && (!s || !r || !c || !out_b)) return ATS_ERR_INVALID;
  for (uint32_t i = 0; i < n; ++i)
    if (s[i] < 0 || c[i] < 0) return ATS_ERR_INVALID;
  std::vector<int64_t> sv(s, s + n), rv(r, r + n), cv(c, c + n);
  std::vector<uint8_t> ev(n, 0), b;
  if (is_expert)
    for (uint32_t i = 0; i < n; ++i) ev[i] = is_expert[i] ? 1 : 0;
  ats::static_placement(sv, rv, cv, ev, M, &b);
  int64_t obj = 0;
  for (uint32_t i = 0; i < n; ++i) {
    out_b[i] = b[i];
    if (b[i] == ATS_GPU) obj += r[i];
    if (i > 0 && b[i] != b[i - 1]) obj -= c[i];
  }
  if (out_objective) *out_objective = obj;
  return ATS_OK;
}

int32_t ats_host_group_pairs(const int32_t* ids, uint32_t P, uint32_t E, int32_t* order, int32_t* pos, int32_t* off,
                             int32_t* max_rows) {
  if (!ids || !order || !pos || !off || !max_rows || E == 0) return ATS_ERR_INVALID;
  std::vector<int32_t> cnt((size_t)E + 1, 0);
  for (uint32_t p = 0; p < P; ++p) {
    if (ids[p] < 0 || (uint32_t)ids[p] >= E) return ATS_ERR_INVALID;
    cnt[(size_t)ids[p] + 1]++;
  }
  int32_t mx = 0;
  for (uint32_t e = 0; e < E; ++e) {
    mx = std::max(mx, cnt[e + 1]);
    cnt[e + 1] += cnt[e];
  }
  for (uint32_t e = 0; e <= E; ++e) off[e] = cnt[e];
  for (uint32_t p = 0; p < P; ++p) {  // stable: pairs of an expert keep their (token, slot) order
    const int32_t r = cnt[ids[p]]++;
    order[r] = (int32_t)p;
    pos[p] = r;
  }
  *max_rows = mx;
  return ATS_OK;
}

int32_t ats_host_repack_q4(const void* codes, const void* scales, void* out_slice, uint32_t n_out, uint32_t k_in) {
  if (!codes || !scales || !out_slice) return ATS_ERR_INVALID;
  if (k_in % ats::kBlock || n_out == 0 || k_in == 0) return ATS_ERR_SHAPE;
  ats::repack_q4((const uint8_t*)codes, (const uint16_t*)scales, (uint8_t*)out_slice, n_out, k_in);
  return ATS_OK;
}

int32_t ats_host_unpack_q4(const void* slice, void* out_codes, void* out_scales, uint32_t n_out, uint32_t k_in) {
  if (!slice || !out_codes || !out_scales) return ATS_ERR_INVALID;
  if (k_in % ats::kBlock || n_out == 0 || k_in == 0) return ATS_ERR_SHAPE;
  const uint64_t words = (uint64_t)n_out * k_in / 8;
  const uint32_t* in = (const uint32_t*)slice;
  uint8_t* out = (uint8_t*)out_codes;
  for (uint64_t w = 0; w < words; ++w) {
    const uint32_t v = in[w];
    uint32_t o = 0;
    for (int k = 0; k < 8; ++k) {
      const int p = (k & 1) ? 4 + k / 2 : k / 2;  // word position of code k
      o |= (((v >> (4 * p)) & 0xFu) ^ 8u) << (4 * k);
    }
    out[4 * w] = (uint8_t)o;
    out[4 * w + 1] = (uint8_t)(o >> 8);
    out[4 * w + 2] = (uint8_t)(o >> 16);
    out[4 * w + 3] = (uint8_t)(o >> 24);
  }
  const uint16_t* si = (const uint16_t*)((const uint8_t*)slice + (uint64_t)n_out * k_in / 2);
  uint16_t* so = (uint16_t*)out_scales;
  for (uint64_t i = 0; i < (uint64_t)n_out * (k_in / ats::kBlock); ++i) so[i] = si[i];
  return ATS_OK;
}

}  // extern "C"
