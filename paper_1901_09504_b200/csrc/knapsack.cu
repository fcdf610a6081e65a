// ocs_knapsack_allocate: Section 3.4's alternative to ceil(r*C) splits per layer -- the split counts of all
// layers chosen at once.  reward_l(s) = (curve_l[0] - curve_l[s]) / curve_l[0] (the fraction by which s splits
// shrink the layer's dynamic range; curve from ocs_range_curve), cost_l(s) = s * unit_cost[l] weight elements.
// Maximise the summed reward subject to the summed cost staying within the budget: a multiple-choice knapsack,
// solved exactly by dynamic programming over the budget in units of gcd(unit_cost).
//
// One CTA: the layers are dependent steps (layer l's table needs layer l-1's), the budget axis is the parallel
// one -- thread t owns budgets t, t + 1024, ...  Tables live in the caller's workspace (they stay in L2).
#include "common.cuh"

namespace ocs {
namespace {

constexpr int kKnapThreads = 1024;
constexpr long long kKnapMaxUnits = 1ll << 22;

struct KnapLayer {
  long long curve_off;
  long long cost_units;
  int s_max;
  int pad;
};

__global__ void __launch_bounds__(kKnapThreads, 1)
knapsack_kernel(const float* __restrict__ curves, const KnapLayer* __restrict__ layers, int n_layers, long long Bu,
                double* dp0, double* dp1, int32_t* __restrict__ choice, int32_t* __restrict__ S_out,
                double* __restrict__ total_reward) {
  double* prev = dp0;
  double* cur = dp1;
  for (long long b = threadIdx.x; b <= Bu; b += kKnapThreads) prev[b] = 0.0;
  __syncthreads();
  for (int l = 0; l < n_layers; ++l) {
    const KnapLayer L = layers[l];
    const float* cv = curves + L.curve_off;
    const double c0 = (double)cv[0];
    int32_t* ch = choice + (size_t)l * (size_t)(Bu + 1);
    for (long long b = threadIdx.x; b <= Bu; b += kKnapThreads) {
      double best = prev[b];   // s = 0: nothing spent on this layer
      int sbest = 0;
      for (int s = 1; s <= L.s_max; ++s) {   // ascending; a later s must be strictly better
        const long long spent = (long long)s * L.cost_units;
        if (spent > b) break;
        const double reward = c0 > 0.0 ? __ddiv_rn(__dsub_rn(c0, (double)cv[s]), c0) : 0.0;
        const double v = __dadd_rn(prev[b - spent], reward);
        if (v > best) { best = v; sbest = s; }
      }
      cur[b] = best;
      ch[b] = sbest;
    }
    __syncthreads();
    double* t = prev; prev = cur; cur = t;
  }
  if (threadIdx.x == 0) {
    if (total_reward) *total_reward = prev[Bu];
    long long b = Bu;
    for (int l = n_layers - 1; l >= 0; --l) {
      const int sc = choice[(size_t)l * (size_t)(Bu + 1) + (size_t)b];
      S_out[l] = sc;
      b -= (long long)sc * layers[l].cost_units;
    }
  }
}

long long gcd_ll(long long a, long long b) {
  while (b) { const long long t = a % b; a = b; b = t; }
  return a;
}

struct KnapWs {
  KnapLayer* layers;
  double* dp0;
  double* dp1;
  int32_t* choice;
  size_t total;
};

// budget units and table layout; false when an argument is out of range
bool knap_layout(int n_layers, const int64_t* unit_cost, int64_t budget, void* ws, long long* Bu_out, long long* g_out,
                 KnapWs* out) {
  if (n_layers <= 0 || !unit_cost || budget < 0) return false;
  long long g = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (unit_cost[l] <= 0) return false;
    g = gcd_ll(g, unit_cost[l]);
  }
  const long long Bu = budget / g;   // a remainder cannot be spent
  *Bu_out = Bu; *g_out = g;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    unsigned char* p = ws ? reinterpret_cast<unsigned char*>(ws) + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  out->layers = reinterpret_cast<KnapLayer*>(take(sizeof(KnapLayer) * (size_t)n_layers));
  out->dp0 = reinterpret_cast<double*>(take(8 * (size_t)(Bu + 1)));
  out->dp1 = reinterpret_cast<double*>(take(8 * (size_t)(Bu + 1)));
  out->choice = reinterpret_cast<int32_t*>(take(4 * (size_t)n_layers * (size_t)(Bu + 1)));
  out->total = off;
  return true;
}

}  // namespace
}  // namespace ocs

using namespace ocs;

extern "C" size_t ocs_knapsack_workspace_bytes(int n_layers, const int64_t* unit_cost, int64_t budget) {
  long long Bu, g;
  KnapWs w;
  if (!knap_layout(n_layers, unit_cost, budget, nullptr, &Bu, &g, &w) || Bu > kKnapMaxUnits) return 0;
  return w.total;
}

extern "C" ocs_status ocs_knapsack_allocate(int n_layers, const float* curves, const int64_t* curve_off,
                                            const int32_t* s_max, const int64_t* unit_cost, int64_t budget,
                                            int32_t* S_out, double* total_reward, void* ws, size_t ws_bytes,
                                            void* stream_) {
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  if (!curves || !curve_off || !s_max || !unit_cost || !S_out) return OCS_ERR_INVALID_ARG;
  long long Bu, g;
  KnapWs w;
  if (!knap_layout(n_layers, unit_cost, budget, ws, &Bu, &g, &w)) return OCS_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (s_max[l] < 0 || curve_off[l] < 0) return OCS_ERR_INVALID_ARG;
  if (Bu > kKnapMaxUnits || n_layers > 4096) return OCS_ERR_UNSUPPORTED;
  if (!ws || !aligned(ws, 256) || ws_bytes < w.total) return OCS_ERR_WORKSPACE;
  ocs_status st = check_device();
  if (st != OCS_OK) return st;
  // the layer table travels as a kernel-sized copy: small, and the host arrays need not outlive the call
  KnapLayer host_layers[64];
  for (int l0 = 0; l0 < n_layers; l0 += 64) {
    const int cnt = n_layers - l0 < 64 ? n_layers - l0 : 64;
    for (int i = 0; i < cnt; ++i) {
      host_layers[i].curve_off = curve_off[l0 + i];
      host_layers[i].cost_units = unit_cost[l0 + i] / g;
      host_layers[i].s_max = s_max[l0 + i];
      host_layers[i].pad = 0;
    }
    if (cudaMemcpyAsync(w.layers + l0, host_layers, sizeof(KnapLayer) * (size_t)cnt, cudaMemcpyHostToDevice, stream) !=
        cudaSuccess)
      return OCS_ERR_CUDA;
    // host_layers is pageable stack memory: the copy has been staged when the call returns
  }
  LaunchScope ls("knapsack_kernel", stream);
  knapsack_kernel<<<1, kKnapThreads, 0, stream>>>(curves, w.layers, n_layers, Bu, w.dp0, w.dp1, w.choice, S_out,
                                                  total_reward);
  return launch_status();
}
