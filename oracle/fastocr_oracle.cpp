// CPU oracle for the FastOCR decode-step attention hot path.
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, plain statement of what the
// path computes; it shares no code, header, table or helper with the CUDA
// library and must never be reached from the product path. Only tests, the
// smoke check and the bench's cpu_baseline / reference arm may load it.
//
// Every function works on ONE sequence whose cache is laid out contiguously as
// K[S][Hkv][d], V[S][Hkv][d] in bf16 (passed as raw 16-bit patterns and widened
// exactly to fp32). Query head h reads KV head h / (H / Hkv).
//
// Arithmetic: Acc = float reproduces an fp32 implementation (products, sums,
// expf in fp32, tokens visited in ascending position order); Acc = double is
// the same algorithm with double accumulation, used to bound the fp32 path's
// own rounding. Results are returned as fp32 in both cases.
//
// Parity pins (tests/test_oracle_*.py): library softmax/matmul/topk routines,
// closed forms (one-token cache, constant keys, probabilities summing to one),
// brute-force rank counting for top-k, and the identities tau=1 == dense,
// sparse == masked dense == dense on a compacted cache. The paper prints no
// worked numeric example of scores, selections or outputs, so no printed value
// pins those numbers ("parity unpinned" against printed values); the integer
// rules (kept count, focal-layer count, gap) and the cost formula ARE pinned to
// numbers the paper prints.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {

inline float widen(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

inline float  exp_of(float x)  { return std::exp(x); }
inline double exp_of(double x) { return std::exp(x); }

// Attention probabilities of one query head over a list of cache positions
// (Appendix B: softmax(q K^T / sqrt(d_k)); the scale is passed in).
// pos == nullptr means positions 0..n-1.
template <class Acc>
void head_probs(const uint16_t* q_h, const uint16_t* K, int kv_head, int Hkv, int d, float sm_scale,
                const int32_t* pos, int n, std::vector<Acc>& p) {
  p.assign(n, Acc(0));
  Acc m = -std::numeric_limits<Acc>::infinity();
  for (int i = 0; i < n; ++i) {
    const int64_t j = pos ? pos[i] : i;
    const uint16_t* k = K + (j * Hkv + kv_head) * static_cast<int64_t>(d);
    Acc dot = 0;
    for (int c = 0; c < d; ++c) dot += static_cast<Acc>(widen(q_h[c])) * static_cast<Acc>(widen(k[c]));
    p[i] = static_cast<Acc>(sm_scale) * dot;
    m = std::max(m, p[i]);
  }
  Acc sum = 0;
  for (int i = 0; i < n; ++i) { p[i] = exp_of(p[i] - m); sum += p[i]; }
  for (int i = 0; i < n; ++i) p[i] = p[i] / sum;
}

// o_h = sum_j p_j V_j over the same position list (Eq. 2, either case).
template <class Acc>
void attend(const uint16_t* q, const uint16_t* K, const uint16_t* V, int H, int Hkv, int d, float sm_scale,
            const int32_t* pos, int n, float* out) {
  const int G = H / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int h = 0; h < H; ++h) {
    std::vector<Acc> p;
    head_probs<Acc>(q + static_cast<int64_t>(h) * d, K, h / G, Hkv, d, sm_scale, pos, n, p);
    std::vector<Acc> o(d, Acc(0));
    for (int i = 0; i < n; ++i) {
      const int64_t j = pos ? pos[i] : i;
      const uint16_t* v = V + (j * Hkv + h / G) * static_cast<int64_t>(d);
      for (int c = 0; c < d; ++c) o[c] += p[i] * static_cast<Acc>(widen(v[c]));
    }
    for (int c = 0; c < d; ++c) out[static_cast<int64_t>(h) * d + c] = static_cast<float>(o[c]);
  }
}

// Kept set K = T u F as an ascending position list (Section 3.1.2): every text
// position plus vis_start + idx[i] for the selected image tokens.
std::vector<int32_t> kept_positions(int S, int vis_start, int N, const int32_t* idx, int k) {
  std::vector<int32_t> pos;
  pos.reserve(static_cast<size_t>(S - N + k));
  for (int j = 0; j < vis_start; ++j) pos.push_back(j);
  std::vector<int32_t> sel(idx, idx + k);
  std::sort(sel.begin(), sel.end());
  for (int i = 0; i < k; ++i) pos.push_back(vis_start + sel[i]);
  for (int j = vis_start + N; j < S; ++j) pos.push_back(j);
  return pos;
}

bool bad_shape(int S, int H, int Hkv, int d) { return S <= 0 || H <= 0 || Hkv <= 0 || d <= 0 || H % Hkv != 0; }

}  // namespace

extern "C" {

// Dense decode attention over the whole cache (Eq. 2, focal-layer case; Appendix B).
// out: [H][d] fp32.
int fastocr_oracle_dense(const uint16_t* q, const uint16_t* K, const uint16_t* V, int S, int H, int Hkv, int d,
                         float sm_scale, int acc64, float* out) {
  if (bad_shape(S, H, Hkv, d)) return 1;
  if (acc64) attend<double>(q, K, V, H, Hkv, d, sm_scale, nullptr, S, out);
  else       attend<float>(q, K, V, H, Hkv, d, sm_scale, nullptr, S, out);
  return 0;
}

// All attention probabilities p[h][j] over the full cache, fp32 [H][S] (test helper).
int fastocr_oracle_probs(const uint16_t* q, const uint16_t* K, int S, int H, int Hkv, int d, float sm_scale,
                         int acc64, float* probs) {
  if (bad_shape(S, H, Hkv, d)) return 1;
  const int G = H / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int h = 0; h < H; ++h) {
    if (acc64) {
      std::vector<double> p;
      head_probs<double>(q + static_cast<int64_t>(h) * d, K, h / G, Hkv, d, sm_scale, nullptr, S, p);
      for (int j = 0; j < S; ++j) probs[static_cast<int64_t>(h) * S + j] = static_cast<float>(p[j]);
    } else {
      std::vector<float> p;
      head_probs<float>(q + static_cast<int64_t>(h) * d, K, h / G, Hkv, d, sm_scale, nullptr, S, p);
      for (int j = 0; j < S; ++j) probs[static_cast<int64_t>(h) * S + j] = p[j];
    }
  }
  return 0;
}

// Head-averaged image attention (Section 3.1.1's a-bar, Eq. 2's TopK argument):
// for image token i, the mean over all H query heads of the post-softmax weight,
// the softmax being taken over the FULL cache (text included).
// scores: [N] fp32; image_mass (optional): sum_i scores[i] = Eq. 1's ratio r
// (numerator and denominator of Eq. 1 add up to the whole distribution, i.e. 1).
int fastocr_oracle_scores(const uint16_t* q, const uint16_t* K, int S, int H, int Hkv, int d, float sm_scale,
                          int vis_start, int N, int acc64, float* scores, float* image_mass) {
  if (bad_shape(S, H, Hkv, d) || vis_start < 0 || N < 0 || vis_start + N > S) return 1;
  std::vector<float> probs(static_cast<size_t>(H) * S);
  fastocr_oracle_probs(q, K, S, H, Hkv, d, sm_scale, acc64, probs.data());
  double mass = 0;
  for (int i = 0; i < N; ++i) {
    if (acc64) {
      double s = 0;
      for (int h = 0; h < H; ++h) s += probs[static_cast<int64_t>(h) * S + vis_start + i];
      scores[i] = static_cast<float>(s / H);
    } else {
      float s = 0;
      for (int h = 0; h < H; ++h) s += probs[static_cast<int64_t>(h) * S + vis_start + i];
      scores[i] = s / static_cast<float>(H);
    }
    mass += scores[i];
  }
  if (image_mass) *image_mass = static_cast<float>(mass);
  return 0;
}

// TopK: the k image tokens with the largest scores, as a stable full sort would
// order them (larger score first; equal scores: lower index first; -0 == +0; NaN
// below every number), returned in ascending index order.
int fastocr_oracle_topk(const float* scores, int N, int k, int32_t* idx_out) {
  if (N < 0 || k < 0 || k > N) return 1;
  std::vector<int32_t> order(N);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
    const float x = scores[a], y = scores[b];
    const bool xn = std::isnan(x), yn = std::isnan(y);
    if (xn || yn) return !xn && yn;
    return x > y;
  });
  std::vector<int32_t> sel(order.begin(), order.begin() + k);
  std::sort(sel.begin(), sel.end());
  std::copy(sel.begin(), sel.end(), idx_out);
  return 0;
}

// Pruned attention (Eq. 2, non-focal case): softmax and weighted sum restricted
// to the kept set: all text positions plus the k selected image tokens.
int fastocr_oracle_sparse(const uint16_t* q, const uint16_t* K, const uint16_t* V, int S, int H, int Hkv, int d,
                          float sm_scale, int vis_start, int N, const int32_t* idx, int k, int acc64,
                          float* out) {
  if (bad_shape(S, H, Hkv, d) || vis_start < 0 || N < 0 || vis_start + N > S || k < 0 || k > N) return 1;
  for (int i = 0; i < k; ++i) if (idx[i] < 0 || idx[i] >= N) return 2;
  std::vector<int32_t> pos = kept_positions(S, vis_start, N, idx, k);
  if (pos.empty()) return 3;
  if (acc64) attend<double>(q, K, V, H, Hkv, d, sm_scale, pos.data(), static_cast<int>(pos.size()), out);
  else       attend<float>(q, K, V, H, Hkv, d, sm_scale, pos.data(), static_cast<int>(pos.size()), out);
  return 0;
}

// Dense attention with an additive mask (0 or -inf per position); used only to
// state "pruned attention == dense attention with unselected image tokens
// masked out" as a separate computation.
int fastocr_oracle_masked_dense(const uint16_t* q, const uint16_t* K, const uint16_t* V, int S, int H, int Hkv,
                                int d, float sm_scale, const uint8_t* keep, float* out) {
  if (bad_shape(S, H, Hkv, d)) return 1;
  const int G = H / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int h = 0; h < H; ++h) {
    std::vector<double> s(S);
    double m = -std::numeric_limits<double>::infinity();
    for (int j = 0; j < S; ++j) {
      const uint16_t* k = K + (static_cast<int64_t>(j) * Hkv + h / G) * d;
      double dot = 0;
      for (int c = 0; c < d; ++c) dot += static_cast<double>(widen(q[static_cast<int64_t>(h) * d + c])) * widen(k[c]);
      s[j] = keep[j] ? sm_scale * dot : -std::numeric_limits<double>::infinity();
      m = std::max(m, s[j]);
    }
    double sum = 0;
    for (int j = 0; j < S; ++j) { s[j] = std::exp(s[j] - m); sum += s[j]; }
    std::vector<double> o(d, 0.0);
    for (int j = 0; j < S; ++j) {
      const uint16_t* v = V + (static_cast<int64_t>(j) * Hkv + h / G) * d;
      for (int c = 0; c < d; ++c) o[c] += s[j] / sum * widen(v[c]);
    }
    for (int c = 0; c < d; ++c) out[static_cast<int64_t>(h) * d + c] = static_cast<float>(o[c]);
  }
  return 0;
}

// |F| = ceil(tau * N) (Section 3.1.2), clamped to [0, N]; a 1e-9 guard keeps
// products such as 0.05 * 4096 = 204.8000000001 from rounding the wrong way.
int fastocr_oracle_kept_count(int N, double tau) {
  if (N <= 0 || !(tau > 0)) return 0;
  double k = std::ceil(tau * static_cast<double>(N) - 1e-9);
  if (k < 0) k = 0;
  if (k > N) k = N;
  return static_cast<int>(k);
}

// Focal Layer Selection (Section 3.1.1, Algorithm 1's profiling block): rank the
// layers by mean image-attention ratio, descending (equal ratios: lower layer
// first), then accept greedily while |C| < floor(rho * L) and every accepted
// layer is more than `gap` layers away. Returns |C|; C_out ascending.
int fastocr_oracle_focal_layers(const double* mean_ratio, int L, double rho, int gap, int32_t* C_out) {
  const int budget = static_cast<int>(std::floor(rho * L + 1e-9));
  std::vector<int> order(L);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return mean_ratio[a] > mean_ratio[b]; });
  std::vector<int32_t> C;
  for (int li : order) {
    if (static_cast<int>(C.size()) >= budget) break;
    bool ok = true;
    for (int lj : C) if (std::abs(li - lj) <= gap) ok = false;
    if (ok) C.push_back(li);
  }
  std::sort(C.begin(), C.end());
  std::copy(C.begin(), C.end(), C_out);
  return static_cast<int>(C.size());
}

// Appendix B: self-attention FLOPs of one decode step, b * l * (8 h^2 + 4 h s).
double fastocr_oracle_attn_flops(double b, double l, double h, double s) { return b * l * (8.0 * h * h + 4.0 * h * s); }

// The same count for a pruned step (how Tables 1 and 2 arrive at the method's "FLOPs (G)"):
// the projection term 8 h^2 is paid by every layer; `full_layers` of the l layers attend the whole
// sequence s, the others attend s_kept tokens. The tables' values are reproduced with
// s_kept = tau * s (the representative sequence counted as image tokens throughout).
double fastocr_oracle_attn_flops_pruned(double b, double l, double h, double s, double full_layers, double s_kept) {
  const double full = full_layers * (8.0 * h * h + 4.0 * h * s);
  const double pruned = (l - full_layers) * (8.0 * h * h + 4.0 * h * s_kept);
  return b * (full + pruned);
}

}  // extern "C"
