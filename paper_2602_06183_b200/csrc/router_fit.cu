// Offline clustering of the hidden features into balanced experts (Section 3.1: "in an offline phase
// ... W1's columns are clustered into non overlapping subsets"; Figure 4a: cluster centres, L2 distance).
// Host code: it runs once, during the dense warm-up steps, not inside the training step.
//
// Balanced k-means: Lloyd iterations whose assignment step gives every expert exactly F / E features.
// Centres start as the means of E contiguous blocks of features; the assignment walks all
// (feature, expert) pairs in order of increasing squared distance (then feature, then expert) and
// gives a feature to the first expert that still has room. All arithmetic is float64.
#include "sf_common.cuh"

#include <algorithm>
#include <cstring>
#include <thread>
#include <vector>

namespace sf {
namespace {

inline double bf16_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return static_cast<double>(f);
}

inline uint16_t double_to_bf16(double x) {
  float f = static_cast<float>(x);
  uint32_t u;
  std::memcpy(&u, &f, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);               // round to nearest, ties to even
  return static_cast<uint16_t>(u >> 16);
}

}  // namespace
}  // namespace sf

using namespace sf;

extern "C" int sf_router_fit_host(const void* host_W1, int64_t F, int64_t D, int E, int iters, void* host_expert,
                                  void* host_perm, void* host_means) {
  if (!host_W1 || !host_expert || !host_perm || !host_means) return SF_ERR_NULL;
  if (F <= 0 || D <= 0 || E < 1 || E > 16 || F % E || iters < 0) return SF_ERR_SHAPE;
  const uint16_t* Wb = static_cast<const uint16_t*>(host_W1);
  int32_t* expert = static_cast<int32_t*>(host_expert);
  int32_t* perm = static_cast<int32_t*>(host_perm);
  uint16_t* means = static_cast<uint16_t*>(host_means);
  const int64_t cap = F / E;
  std::vector<double> W((size_t)F * D), C((size_t)E * D, 0.0), wn((size_t)F), d2((size_t)F * E);
  for (int64_t i = 0; i < F * D; ++i) W[i] = bf16_to_double(Wb[i]);
  for (int64_t f = 0; f < F; ++f) {
    double s = 0;
    for (int64_t k = 0; k < D; ++k) s += W[f * D + k] * W[f * D + k];
    wn[f] = s;
  }
  std::vector<int32_t> assign((size_t)F), next((size_t)F);
  for (int64_t f = 0; f < F; ++f) assign[f] = (int32_t)(f / cap);
  auto centres_from = [&](const std::vector<int32_t>& a) {
    std::fill(C.begin(), C.end(), 0.0);
    for (int64_t f = 0; f < F; ++f)
      for (int64_t k = 0; k < D; ++k) C[(size_t)a[f] * D + k] += W[f * D + k];
    for (auto& c : C) c /= (double)cap;
  };
  centres_from(assign);
  const unsigned nthreads = std::max(1u, std::min(16u, std::thread::hardware_concurrency()));
  std::vector<int64_t> order((size_t)F * E);
  for (int it = 0; it < iters; ++it) {
    std::vector<double> cn((size_t)E, 0.0);
    for (int e = 0; e < E; ++e)
      for (int64_t k = 0; k < D; ++k) cn[e] += C[(size_t)e * D + k] * C[(size_t)e * D + k];
    auto work = [&](int64_t f0, int64_t f1) {
      for (int64_t f = f0; f < f1; ++f)
        for (int e = 0; e < E; ++e) {
          double dot = 0;
          for (int64_t k = 0; k < D; ++k) dot += W[f * D + k] * C[(size_t)e * D + k];
          d2[f * E + e] = wn[f] - 2.0 * dot + cn[e];
        }
    };
    std::vector<std::thread> pool;
    const int64_t chunk = (F + nthreads - 1) / nthreads;
    for (unsigned t = 0; t < nthreads; ++t) {
      const int64_t f0 = t * chunk, f1 = std::min<int64_t>(F, f0 + chunk);
      if (f0 < f1) pool.emplace_back(work, f0, f1);
    }
    for (auto& th : pool) th.join();
    for (int64_t i = 0; i < F * E; ++i) order[i] = i;
    std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) {
      if (d2[a] != d2[b]) return d2[a] < d2[b];
      return a < b;                                   // index = f * E + e: feature first, then expert
    });
    std::fill(next.begin(), next.end(), -1);
    std::vector<int64_t> room((size_t)E, cap);
    int64_t left = F;
    for (int64_t idx : order) {
      const int64_t f = idx / E;
      const int e = (int)(idx % E);
      if (next[f] < 0 && room[e] > 0) {
        next[f] = e;
        --room[e];
        if (--left == 0) break;
      }
    }
    if (next == assign) break;
    assign = next;
    centres_from(assign);
  }
  for (int64_t f = 0; f < F; ++f) expert[f] = assign[f];
  // expert-major order, stable inside an expert: feature perm[i] of the old numbering becomes feature i
  int64_t at = 0;
  for (int e = 0; e < E; ++e)
    for (int64_t f = 0; f < F; ++f)
      if (assign[f] == e) perm[at++] = (int32_t)f;
  for (int64_t i = 0; i < (int64_t)E * D; ++i) means[i] = double_to_bf16(C[i]);
  return SF_OK;
}
