// Pipeline partitioner (host code): which consecutive layers run on which device so that the
// slowest pipeline stage is as fast as possible.  Dynamic programme over (layers processed, set
// of devices used, device of the next stage) with the transition
//   h(j, S + {u}, v) = min over i < j, u not in S of max( h(i, S, u), T_comm(u, v, P_j), T_comp(i..j, u) )
// (paper Section 3.3, Eq. 1-3, Algorithm 1), and the variant that groups identical devices into
// categories so that the state holds a count per category instead of a subset.
#include "../../include/vit.h"

#include <cmath>
#include <cstdint>
#include <limits>
#include <vector>

namespace {

constexpr double INF = std::numeric_limits<double>::infinity();

bool problem_ok(const vit_partition_problem* p, int max_devices) {
  if (!p || p->layers < 1 || p->devices < 1 || p->devices > max_devices) return false;
  if (!p->layer_time || !p->out_bytes || !p->layer_mem || !p->device_mem || !p->bandwidth) return false;
  return true;
}

// Eq. 1: T_comm(u, v, P_j) = P_j / b(u, v)
inline double t_comm(const vit_partition_problem* p, int u, int v, int j /*layers done, 1-based last layer*/) {
  return p->out_bytes[j - 1] / p->bandwidth[(size_t)u * p->devices + v];
}

struct Pre { int32_t i; int32_t u; };

}  // namespace

extern "C" int vit_partition(const vit_partition_problem* p, double* t_opt, int32_t* n_stages,
                             int32_t* stage_layers, int32_t* stage_device) {
  if (!problem_ok(p, 16) || !t_opt || !n_stages || !stage_layers || !stage_device) return VIT_ERR_INVALID_ARG;
  const int L = p->layers, D = p->devices;
  const size_t nsub = (size_t)1 << D;
  // h[(i * nsub + S) * D + u]: best slowest-stage time with the first i layers done on the devices
  // of S, u being the device of the next stage
  std::vector<double> h((size_t)(L + 1) * nsub * D, INF);
  std::vector<Pre> pre(h.size(), Pre{-1, -1});
  auto at = [&](int i, size_t S, int u) { return ((size_t)i * nsub + S) * D + u; };
  for (int u = 0; u < D; ++u) h[at(0, 0, u)] = 0.0;   // the first stage may go to any device
  double answer = INF;
  int ans_i = -1, ans_u = -1;
  size_t ans_S = 0;
  for (int i = 0; i < L; ++i) {
    for (size_t S = 0; S < nsub; ++S) {
      for (int u = 0; u < D; ++u) {
        if (S >> u & 1) continue;
        const double hi = h[at(i, S, u)];
        if (hi == INF) continue;
        double mem = 0.0, comp = 0.0;
        for (int j = i + 1; j <= L; ++j) {
          mem += p->layer_mem[j - 1];
          if (mem > p->device_mem[u]) break;              // layers i+1..j no longer fit on u
          comp += p->layer_time[(size_t)u * L + (j - 1)];
          const double stage = hi > comp ? hi : comp;
          if (j == L) {                                   // last stage: nothing to send on
            if (stage < answer) { answer = stage; ans_i = i; ans_u = u; ans_S = S; }
          } else {
            const size_t S2 = S | ((size_t)1 << u);
            for (int v = 0; v < D; ++v) {
              if (S2 >> v & 1) continue;
              const double c = t_comm(p, u, v, j);
              const double C = stage > c ? stage : c;     // Eq. 2 and Eq. 3
              const size_t k = at(j, S2, v);
              if (C < h[k]) { h[k] = C; pre[k] = Pre{i, u}; }
            }
          }
        }
      }
    }
  }
  if (answer == INF) return VIT_ERR_INFEASIBLE;
  // walk the precursors back from the last stage
  std::vector<int32_t> lay, dev;
  int j = L, i = ans_i, u = ans_u;
  size_t S = ans_S;
  for (;;) {
    lay.push_back(j - i);
    dev.push_back(u);
    if (i == 0) break;
    const Pre q = pre[at(i, S, u)];
    j = i;
    i = q.i;
    u = q.u;
    S &= ~((size_t)1 << u);
  }
  *t_opt = answer;
  *n_stages = (int32_t)lay.size();
  for (size_t k = 0; k < lay.size(); ++k) {
    stage_layers[k] = lay[lay.size() - 1 - k];
    stage_device[k] = dev[dev.size() - 1 - k];
  }
  return VIT_OK;
}

// Devices grouped into categories of identical devices: `devices` is the number of categories,
// category_count[c] how many devices it has; layer_time, device_mem, bandwidth are per category
// (bandwidth[c][c] is the bandwidth between two devices of the same category).  The state holds
// how many devices of each category are used.  stage_device receives category indices.
extern "C" int vit_partition_categories(const vit_partition_problem* p, const int32_t* category_count,
                                        double* t_opt, int32_t* n_stages, int32_t* stage_layers,
                                        int32_t* stage_device) {
  if (!problem_ok(p, 8) || !category_count || !t_opt || !n_stages || !stage_layers || !stage_device)
    return VIT_ERR_INVALID_ARG;
  const int L = p->layers, N = p->devices;
  std::vector<size_t> mul(N + 1, 1);
  for (int c = 0; c < N; ++c) {
    if (category_count[c] < 0) return VIT_ERR_INVALID_ARG;
    mul[c + 1] = mul[c] * (size_t)(category_count[c] + 1);
    if (mul[c + 1] > ((size_t)1 << 24)) return VIT_ERR_INVALID_ARG;
  }
  const size_t nstate = mul[N];
  auto used = [&](size_t s, int c) { return (int)(s / mul[c] % (size_t)(category_count[c] + 1)); };
  std::vector<double> h((size_t)(L + 1) * nstate * N, INF);
  std::vector<Pre> pre(h.size(), Pre{-1, -1});
  auto at = [&](int i, size_t s, int a) { return ((size_t)i * nstate + s) * N + a; };
  for (int a = 0; a < N; ++a)
    if (category_count[a] > 0) h[at(0, 0, a)] = 0.0;
  double answer = INF;
  int ans_i = -1, ans_a = -1;
  size_t ans_s = 0;
  for (int i = 0; i < L; ++i) {
    for (size_t s = 0; s < nstate; ++s) {
      for (int a = 0; a < N; ++a) {
        if (used(s, a) >= category_count[a]) continue;    // no unused device of this category
        const double hi = h[at(i, s, a)];
        if (hi == INF) continue;
        const size_t s2 = s + mul[a];
        double mem = 0.0, comp = 0.0;
        for (int j = i + 1; j <= L; ++j) {
          mem += p->layer_mem[j - 1];
          if (mem > p->device_mem[a]) break;
          comp += p->layer_time[(size_t)a * L + (j - 1)];
          const double stage = hi > comp ? hi : comp;
          if (j == L) {
            if (stage < answer) { answer = stage; ans_i = i; ans_a = a; ans_s = s; }
          } else {
            for (int b = 0; b < N; ++b) {
              if (used(s2, b) >= category_count[b]) continue;
              const double c = t_comm(p, a, b, j);
              const double C = stage > c ? stage : c;
              const size_t k = at(j, s2, b);
              if (C < h[k]) { h[k] = C; pre[k] = Pre{i, a}; }
            }
          }
        }
      }
    }
  }
  if (answer == INF) return VIT_ERR_INFEASIBLE;
  std::vector<int32_t> lay, dev;
  int j = L, i = ans_i, a = ans_a;
  size_t s = ans_s;
  for (;;) {
    lay.push_back(j - i);
    dev.push_back(a);
    if (i == 0) break;
    const Pre q = pre[at(i, s, a)];
    j = i;
    i = q.i;
    a = q.u;
    s -= mul[a];
  }
  *t_opt = answer;
  *n_stages = (int32_t)lay.size();
  for (size_t k = 0; k < lay.size(); ++k) {
    stage_layers[k] = lay[lay.size() - 1 - k];
    stage_device[k] = dev[dev.size() - 1 - k];
  }
  return VIT_OK;
}
