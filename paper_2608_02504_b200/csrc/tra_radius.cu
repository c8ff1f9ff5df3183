// Entropy -> budget -> radius (Eq. 8, Eq. 14; Appendix "Entropy-to-budget-to-radius lookup").
#include <math.h>

#include "tra_common.cuh"

// One thread per (batch*head, token).  The budget (uniform-support map of Eq. 8, or the lognormal
// map of the appendix) is evaluated in fp64 so that the ceiling is
// taken on the same number a host fp64 evaluation sees; the radius is the first entry of the
// token's count-table row that reaches the budget (the row is non-decreasing in the candidate
// index, so a binary search finds the minimum of Eq. 14).
__global__ void tra_budget_radius_kernel(const float* __restrict__ entropy,
                                         const uint32_t* __restrict__ coord_packed,
                                         const uint32_t* __restrict__ counts,
                                         const float* __restrict__ radii, int32_t* __restrict__ budget,
                                         float* __restrict__ radius, uint16_t* __restrict__ ridx,
                                         int N, int S, int H, int W, int n_radii, double tau,
                                         int budget_map, double z_tau, double log_n, long long total) {
  long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= total) return;
  int p = (int)(g % S);
  if (p >= N) {                      // text token: sees every key (Section 3.2, last paragraph)
    if (budget) budget[g] = S;
    if (radius) radius[g] = INFINITY;
    ridx[g] = (uint16_t)(n_radii - 1);
    return;
  }
  double v;
  if (budget_map == TRA_BUDGET_LOGNORMAL) {
    // sigma = sqrt(2 (log N - H)),  B = Phibar(sigma - Phi^-1(tau)),  K = ceil(N B)
    double gap = log_n - (double)entropy[g];
    if (gap < 0.0) gap = 0.0;
    v = ceil((double)N * 0.5 * erfc((sqrt(2.0 * gap) - z_tau) * 0.70710678118654752440));
  } else {
    v = ceil(tau * exp((double)entropy[g]));
  }
  if (!(v >= 1.0)) v = 1.0;          // also catches NaN
  if (v > (double)N) v = (double)N;
  uint32_t need = (uint32_t)v;
  uint32_t c = coord_packed[p];
  size_t row = ((size_t)(tra_coord_t(c) * H + tra_coord_y(c)) * W + tra_coord_x(c)) * n_radii;
  const uint32_t* cnt = counts + row;
  int lo = 0, hi = n_radii - 1;      // cnt[n_radii-1] == N >= need
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(cnt + mid) >= need) hi = mid; else lo = mid + 1;
  }
  if (budget) budget[g] = (int32_t)need;
  if (radius) radius[g] = radii[lo];
  ridx[g] = (uint16_t)lo;
}

extern "C" int tra_budget_radius(const tra_plan_t* plan, const float* entropy, int32_t* budget,
                                 float* radius, uint16_t* ridx, int B, int heads, void* stream_) {
  if (!plan || !entropy || !ridx || B < 1 || heads < 1) return TRA_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  long long total = (long long)B * heads * plan->S;
  long long grid = (total + 255) / 256;
  if (grid > 0x7fffffffll) return TRA_ERR_UNSUPPORTED;
  tra_budget_radius_kernel<<<(unsigned)grid, 256, 0, stream>>>(
      entropy, plan->d_coord_packed, plan->d_counts, plan->d_radii_f32, budget, radius, ridx,
      plan->N, plan->S, plan->cfg.H, plan->cfg.W, plan->n_radii, plan->cfg.tau, plan->cfg.budget_map, plan->z_tau,
      log((double)plan->N), total);
  TRA_CUDA_CHECK(cudaGetLastError());
  return TRA_OK;
}
