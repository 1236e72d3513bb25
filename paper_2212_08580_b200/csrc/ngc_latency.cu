// Latency engine (Section IV): Monte Carlo of the stopping rule under the response-time model of
// Section II-D, one trial per thread.  Task times come from the SplitMix64 stream exactly as
// ngc_sample_times draws them, with the trial's own seed, so that any trial can be reproduced on the host.
#include <cmath>

#include "ngc_device.h"
#include "ngc_pdl.cuh"

namespace ngc {
namespace {

__host__ __device__ inline uint64_t splitmix64_at(uint64_t seed, uint64_t k) {
  uint64_t z = seed + k * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

struct McParams {
  int n, L, tasks;
  int levels[NGC_MAX_LEVELS];
  uint64_t seed;
  long long trials;
  double shift, rate, p_fail, gamma, eps;
  double *latency;
  int *level;
};

__global__ void __launch_bounds__(128) latency_mc_kernel(const McParams p) {
  pdl_sync();
  const long long trial = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (trial >= p.trials) return;
  const uint64_t seed = splitmix64_at(p.seed ^ 0xD1B54A32D192ED03ull, (uint64_t)trial + 1);
  // One level at a time (the task times are regenerated from the counter-based stream instead of being kept):
  // done[i] = completion instant of the first s_l + 1 tasks of worker i, summed left to right.
  double done[NGC_MAX_N];
  double best = INFINITY;
  int best_l = -1;
  for (int l = 0; l < p.L; ++l) {
    const int need = p.levels[l] + 1;
    for (int i = 0; i < p.n; ++i) {
      const uint64_t base = (uint64_t)i * (p.tasks + 1);
      const double uf = (double)(splitmix64_at(seed, 1ull + base) >> 11) / 9007199254740992.0;
      double acc = 0.0;
      if (uf < p.p_fail) acc = INFINITY;
      else
        for (int m = 0; m < need; ++m) {
          const uint64_t bits = splitmix64_at(seed, 2ull + base + m) >> 11;
          const double u = ((double)bits + 0.5) / 9007199254740992.0;
          acc = acc + (p.shift - log(u) / p.rate);
        }
      done[i] = acc;
    }
    const int kth = p.n - p.levels[l];  // the instant at which `kth` workers have finished
    double D = INFINITY;
    for (int a = 0; a < p.n; ++a) {
      const double x = done[a];
      int less = 0, leq = 0;
      for (int b = 0; b < p.n; ++b) {
        less += done[b] < x;
        leq += done[b] <= x;
      }
      if (less < kth && kth <= leq) { D = x; break; }
    }
    if (D < best) { best = D; best_l = l; }
  }
  if (p.latency) p.latency[trial] = best_l < 0 ? INFINITY : p.gamma + p.eps + best;
  if (p.level) p.level[trial] = best_l;
}

}  // namespace

cudaError_t launch_latency_mc(const ngc_plan_s &plan, uint64_t seed, long long trials, double shift, double rate,
                              double p_fail, double *latency_dev, int *level_dev, cudaStream_t stream) {
  McParams p;
  p.n = plan.n; p.L = plan.L; p.tasks = plan.levels.back() + 1;
  for (int l = 0; l < plan.L; ++l) p.levels[l] = plan.levels[l];
  p.seed = seed; p.trials = trials; p.shift = shift; p.rate = rate; p.p_fail = p_fail;
  p.gamma = plan.gamma; p.eps = plan.eps;
  p.latency = latency_dev; p.level = level_dev;
  launch_k(latency_mc_kernel, (unsigned)((trials + 127) / 128), 128, 0, stream, p);
  return cudaGetLastError();
}

}  // namespace ngc
