// Pipeline partitioner (host code): which consecutive layers run on which device so that the
// slowest pipeline stage is as fast as possible (paper Section 3.3: Eq. 1 T_comm = P_j / b(u,v),
// Eq. 2 T_period = max(T_comp, T_comm), Eq. 3 the optimal-substructure recurrence).
//
// The recurrence is evaluated here in "arrival" form.  A state records how many devices of each
// kind are already occupied (a mixed-radix number: with every device its own kind this is a
// plain subset bitmask) and two tables are kept per number of finished layers j:
//   G(j, S, v)  best slowest-period of any mapping of layers [0, j) onto the devices of S whose
//               last stage runs on v (v in S); only needed for one j at a time
//   F(j, S, u)  = min over v in S of max( G(j, S, v), P_j / b(v, u) ): the best period with which
//               the activations of layer j can arrive at a still free device u
// and G(j, S, v) = min over i < j with layers (i, j] fitting v of
//                  max( T_comp(i..j, v), i == 0 ? [S = {v}] : F(i, S - v, v) ).
// The answer is min G(L, S, v).  Stage times and memory come from per-device prefix sums, so one
// (j, S, v) costs O(L) and one F entry O(D): O(states * L * D * (L + D)) in total.  The mapping is
// recovered by re-deriving, from the last stage backwards, which (i, v) attains each value; only
// F is kept, which halves the memory of a table-per-choice scheme.
#include "../../include/vit.h"

#include <cmath>
#include <cstdint>
#include <limits>
#include <new>
#include <vector>

namespace {

constexpr double INF = std::numeric_limits<double>::infinity();

struct Solver {
  int L, N;                         // layers, kinds of device
  std::vector<int> cap;             // devices per kind
  std::vector<size_t> mul;          // mixed-radix weights, mul[N] = number of states
  std::vector<double> pt, pm;       // prefix sums: pt[v * (L+1) + j] time of layers [0,j) on v; pm[j] memory
  const vit_partition_problem* p;
  std::vector<double> F;            // [(j * nstate + S) * N + u], j in [1, L)
  size_t nstate;

  int used(size_t S, int c) const { return (int)(S / mul[c] % (size_t)(cap[c] + 1)); }
  size_t fidx(int j, size_t S, int u) const { return ((size_t)j * nstate + S) * N + u; }
  double comp(int i, int j, int v) const { return pt[(size_t)v * (L + 1) + j] - pt[(size_t)v * (L + 1) + i]; }
  bool fits(int i, int j, int v) const { return pm[j] - pm[i] <= p->device_mem[v]; }
  // Eq. 1 for the output of layer j (1-based) sent from v to u
  double comm(int v, int u, int j) const { return p->out_bytes[j - 1] / p->bandwidth[(size_t)v * N + u]; }

  // best period of layers [0, j) on the devices of S with the last stage on v (v occupied in S);
  // *best_i receives the first layer index of that last stage
  double G(int j, size_t S, int v, int* best_i) const {
    const size_t Sv = S - mul[v];
    double best = INF;
    int arg = -1;
    for (int i = j - 1; i >= 0; --i) {
      if (!fits(i, j, v)) break;                       // memory only grows as the stage grows
      const double before = i == 0 ? (Sv == 0 ? 0.0 : INF) : F[fidx(i, Sv, v)];
      if (before == INF) continue;
      const double c = comp(i, j, v);
      const double period = c > before ? c : before;   // Eq. 2
      if (period < best) { best = period; arg = i; }
    }
    if (best_i) *best_i = arg;
    return best;
  }

  int solve(double* t_opt, int32_t* n_stages, int32_t* stage_layers, int32_t* stage_device) {
    nstate = mul[N];
    F.assign((size_t)L * nstate * N, INF);
    std::vector<double> g(N);
    double answer = INF;
    size_t ans_S = 0;
    int ans_v = -1;
    for (int j = 1; j <= L; ++j) {
      for (size_t S = 1; S < nstate; ++S) {
        bool any = false;
        for (int v = 0; v < N; ++v) {
          g[v] = used(S, v) > 0 ? G(j, S, v, nullptr) : INF;
          any = any || g[v] != INF;
        }
        if (!any) continue;
        if (j == L) {                                  // the last stage sends nothing
          for (int v = 0; v < N; ++v)
            if (g[v] < answer) { answer = g[v]; ans_S = S; ans_v = v; }
          continue;
        }
        for (int u = 0; u < N; ++u) {
          if (used(S, u) >= cap[u]) continue;          // no free device of this kind left
          double best = INF;
          for (int v = 0; v < N; ++v) {
            if (g[v] == INF) continue;
            const double c = comm(v, u, j);
            const double period = g[v] > c ? g[v] : c;
            if (period < best) best = period;
          }
          F[fidx(j, S, u)] = best;
        }
      }
    }
    if (answer == INF) return VIT_ERR_INFEASIBLE;
    // back-trace: find the stage that attains each value, last stage first
    std::vector<int32_t> lay, dev;
    int j = L, v = ans_v;
    size_t S = ans_S;
    for (;;) {
      int i = -1;
      G(j, S, v, &i);
      lay.push_back(j - i);
      dev.push_back(v);
      if (i == 0) break;
      S -= mul[v];
      const double target = F[fidx(i, S, v)];
      int from = -1;
      for (int w = 0; w < N && from < 0; ++w) {
        if (used(S, w) == 0) continue;
        const double gw = G(i, S, w, nullptr);
        if (gw == INF) continue;
        const double c = comm(w, v, i);
        if ((gw > c ? gw : c) == target) from = w;
      }
      if (from < 0) return VIT_ERR_INFEASIBLE;         // cannot happen: F was built from these values
      j = i;
      v = from;
    }
    *t_opt = answer;
    *n_stages = (int32_t)lay.size();
    for (size_t k = 0; k < lay.size(); ++k) {
      stage_layers[k] = lay[lay.size() - 1 - k];
      stage_device[k] = dev[dev.size() - 1 - k];
    }
    return VIT_OK;
  }
};

inline bool finite_nonneg(double x) { return x >= 0.0 && x < INF; }

// `count` == nullptr: every device is its own kind.
int partition_common(const vit_partition_problem* p, const int32_t* count, int max_kinds, double* t_opt,
                     int32_t* n_stages, int32_t* stage_layers, int32_t* stage_device) {
  if (!p || !t_opt || !n_stages || !stage_layers || !stage_device) return VIT_ERR_INVALID_ARG;
  if (p->layers < 1 || p->devices < 1 || p->devices > max_kinds) return VIT_ERR_INVALID_ARG;
  if (!p->layer_time || !p->out_bytes || !p->layer_mem || !p->device_mem || !p->bandwidth) return VIT_ERR_INVALID_ARG;
  const int L = p->layers, N = p->devices;
  for (int j = 0; j < L; ++j)
    if (!finite_nonneg(p->out_bytes[j]) || !finite_nonneg(p->layer_mem[j])) return VIT_ERR_INVALID_ARG;
  for (int v = 0; v < N; ++v) {
    if (!(p->device_mem[v] >= 0.0)) return VIT_ERR_INVALID_ARG;            // +inf allowed, NaN is not
    for (int j = 0; j < L; ++j)
      if (!finite_nonneg(p->layer_time[(size_t)v * L + j])) return VIT_ERR_INVALID_ARG;
    for (int u = 0; u < N; ++u)
      if (!(p->bandwidth[(size_t)v * N + u] > 0.0)) return VIT_ERR_INVALID_ARG;   // zero, negative, NaN
  }
  try {
    Solver s;
    s.L = L; s.N = N; s.p = p;
    s.cap.resize(N);
    s.mul.assign(N + 1, 1);
    for (int c = 0; c < N; ++c) {
      s.cap[c] = count ? count[c] : 1;
      if (s.cap[c] < 0) return VIT_ERR_INVALID_ARG;
      s.mul[c + 1] = s.mul[c] * (size_t)(s.cap[c] + 1);
      if (s.mul[c + 1] > ((size_t)1 << 24)) return VIT_ERR_INVALID_ARG;
    }
    s.pt.assign((size_t)N * (L + 1), 0.0);
    s.pm.assign(L + 1, 0.0);
    for (int j = 0; j < L; ++j) s.pm[j + 1] = s.pm[j] + p->layer_mem[j];
    for (int v = 0; v < N; ++v)
      for (int j = 0; j < L; ++j)
        s.pt[(size_t)v * (L + 1) + j + 1] = s.pt[(size_t)v * (L + 1) + j] + p->layer_time[(size_t)v * L + j];
    return s.solve(t_opt, n_stages, stage_layers, stage_device);
  } catch (const std::bad_alloc&) {
    return VIT_ERR_TOO_LARGE;
  }
}

}  // namespace

extern "C" int vit_partition(const vit_partition_problem* p, double* t_opt, int32_t* n_stages,
                             int32_t* stage_layers, int32_t* stage_device) {
  return partition_common(p, nullptr, 16, t_opt, n_stages, stage_layers, stage_device);
}

// Devices grouped into categories of identical devices: `devices` is the number of categories,
// category_count[c] how many devices it has; layer_time, device_mem, bandwidth are per category
// (bandwidth[c][c] is the bandwidth between two devices of the same category).  The state holds
// how many devices of each category are used.  stage_device receives category indices.
extern "C" int vit_partition_categories(const vit_partition_problem* p, const int32_t* category_count,
                                        double* t_opt, int32_t* n_stages, int32_t* stage_layers,
                                        int32_t* stage_device) {
  if (!category_count) return VIT_ERR_INVALID_ARG;
  return partition_common(p, category_count, 8, t_opt, n_stages, stage_layers, stage_device);
}
