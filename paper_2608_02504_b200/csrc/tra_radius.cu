// Entropy -> budget -> radius (Eq. 8, Eq. 14; Appendix "Entropy-to-budget-to-radius lookup").
#include <math.h>

#include "tra_common.cuh"

namespace {

struct RadiusArgs {
  const float* entropy;
  const uint32_t* coord_packed;
  const uint32_t* counts;
  const float* radii;
  int32_t* budget;
  float* radius;
  uint16_t* ridx;
  int N, S, H, W, n_radii, budget_map;
  double tau, z_tau, log_n;
  long long total;
  int* status;
};

// The budget (uniform-support map of Eq. 8, or the lognormal map of the appendix) is evaluated in
// fp64 so that the ceiling is taken on the same number a host fp64 evaluation sees.
__device__ __forceinline__ uint32_t tra_budget_of(const RadiusArgs& a, float entropy) {
  double v;
  if (a.budget_map == TRA_BUDGET_LOGNORMAL) {
    // sigma = sqrt(2 (log N - H)),  B = Phibar(sigma - Phi^-1(tau)),  K = ceil(N B)
    double gap = a.log_n - (double)entropy;
    if (gap < 0.0) gap = 0.0;
    v = ceil((double)a.N * 0.5 * erfc((sqrt(2.0 * gap) - a.z_tau) * 0.70710678118654752440));
  } else {
    v = ceil(a.tau * exp((double)entropy));
  }
  if (!(v >= 1.0)) v = 1.0;          // also catches NaN
  if (v > (double)a.N) v = (double)a.N;
  return (uint32_t)v;
}

// The count-table row of the token at tile-major position p (the row is non-decreasing in the
// candidate index, so a binary search finds the minimum of Eq. 14).
__device__ __forceinline__ const uint32_t* tra_count_row(const RadiusArgs& a, uint32_t c) {
  return a.counts + ((size_t)(tra_coord_t(c) * a.H + tra_coord_y(c)) * a.W + tra_coord_x(c)) * a.n_radii;
}

// Candidate sets of up to 128 radii (the built-in sets have about 110): the search takes two steps
// of independent loads instead of seven dependent ones.  The first reads the token's row of the
// coarse table (every eighth entry of its count-table row, 64 bytes, four 16-byte loads) and counts
// the entries below the budget, which names the group of eight that holds the answer; the second
// reads that group (one aligned 32-byte sector of a copy of the count table with rows padded to 128
// entries; the rows of the table itself are not sector-aligned) and counts again.  Rows are
// non-decreasing, so "entries below the budget" is the index of the first entry that reaches it
// (Eq. 14).
__global__ void __launch_bounds__(256) tra_budget_radius_2round_kernel(RadiusArgs a, const uint32_t* __restrict__ coarse) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= a.total) return;
  const int p = (int)(g % a.S);
  if (p >= a.N) {                      // text token: sees every key (Section 3.2, last paragraph)
    if (a.budget) a.budget[g] = a.S;
    if (a.radius) a.radius[g] = INFINITY;
    a.ridx[g] = (uint16_t)(a.n_radii - 1);
    return;
  }
  const uint32_t c = __ldg(a.coord_packed + p);
  size_t cell = (size_t)(tra_coord_t(c) * a.H + tra_coord_y(c)) * a.W + tra_coord_x(c);
  if (!TRA_IDX(cell, a.N, a.status)) cell = 0;
  const uint4* cr = reinterpret_cast<const uint4*>(coarse + cell * 16);
  const uint4 q0 = __ldg(cr), q1 = __ldg(cr + 1), q2 = __ldg(cr + 2), q3 = __ldg(cr + 3);
  const uint32_t need = tra_budget_of(a, __ldg(a.entropy + g));
  const int grp = (q0.x < need) + (q0.y < need) + (q0.z < need) + (q0.w < need) + (q1.x < need) + (q1.y < need) +
                  (q1.z < need) + (q1.w < need) + (q2.x < need) + (q2.y < need) + (q2.z < need) + (q2.w < need) +
                  (q3.x < need) + (q3.y < need) + (q3.z < need) + (q3.w < need);
  // the group of eight: one aligned 32-byte sector of the padded copy of the count table that follows the
  // coarse table (rows of 128 entries, the entries past n_radii hold the largest value)
  const int base = min(grp, 15) * 8;   // grp <= (n_radii - 1) / 8: the last entry of a row is N >= need
  const uint4* fr = reinterpret_cast<const uint4*>(coarse + (size_t)a.N * 16 + cell * 128 + base);
  const uint4 e0 = __ldg(fr), e1 = __ldg(fr + 1);
  int lo = base + (e0.x < need) + (e0.y < need) + (e0.z < need) + (e0.w < need) + (e1.x < need) + (e1.y < need) +
           (e1.z < need) + (e1.w < need);
  if (!TRA_IDX(lo, a.n_radii, a.status)) lo = a.n_radii - 1;
  if (a.budget) a.budget[g] = (int32_t)need;
  if (a.radius) a.radius[g] = __ldg(a.radii + lo);
  a.ridx[g] = (uint16_t)lo;
}

// coarse[cell][i] = counts[cell][min(8 i + 7, n_radii - 1)] for the groups that exist, else the largest value;
// behind the coarse table, padded[cell][j] = counts[cell][j] for j < n_radii, else the largest value (j < 128).
__global__ void tra_coarse_table_kernel(const uint32_t* __restrict__ counts, uint32_t* __restrict__ coarse,
                                        long long cells, int n_radii, int* __restrict__ status) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= cells * 128) return;
  const long long cell = g >> 7;
  const int j = (int)(g & 127);
  const long long src_j = cell * n_radii + j;
  coarse[cells * 16 + g] = j < n_radii && TRA_IDX(src_j, cells * n_radii, status) ? counts[src_j] : 0xffffffffu;
  if (j < 16) {
    const long long src = cell * n_radii + min(8 * j + 7, n_radii - 1);
    coarse[cell * 16 + j] = 8 * j < n_radii && TRA_IDX(src, cells * n_radii, status) ? counts[src] : 0xffffffffu;
  }
}

// Binary search in the count-table row: candidate sets of more than 128 radii.
__global__ void __launch_bounds__(256) tra_budget_radius_kernel(RadiusArgs a) {
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= a.total) return;
  const int p = (int)(g % a.S);
  if (p >= a.N) {                      // text token
    if (a.budget) a.budget[g] = a.S;
    if (a.radius) a.radius[g] = INFINITY;
    a.ridx[g] = (uint16_t)(a.n_radii - 1);
    return;
  }
  const uint32_t need = tra_budget_of(a, a.entropy[g]);
  const uint32_t* cnt = tra_count_row(a, a.coord_packed[p]);
  if (!TRA_IDX(cnt - a.counts, (long long)a.N * a.n_radii - a.n_radii + 1, a.status)) cnt = a.counts;
  int lo = 0, hi = a.n_radii - 1;      // cnt[n_radii-1] == N >= need
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(cnt + mid) >= need) hi = mid; else lo = mid + 1;
  }
  if (a.budget) a.budget[g] = (int32_t)need;
  if (a.radius) a.radius[g] = a.radii[lo];
  a.ridx[g] = (uint16_t)lo;
}

}  // namespace

// Plan time: the coarse table of the two-round search and the padded copy of the count table behind it, 16 + 128
// words per cell (called by tra_plan_create for sets of <= 128 radii).
int tra_build_coarse_table(const uint32_t* counts, uint32_t* coarse, long long cells, int n_radii, int* status,
                           cudaStream_t stream) {
  const long long total = cells * 128;
  tra_coarse_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(counts, coarse, cells, n_radii,
                                                                               status);
  return cudaGetLastError() == cudaSuccess ? TRA_OK : TRA_ERR_CUDA;
}

extern "C" int tra_budget_radius(const tra_plan_t* plan, const float* entropy, int32_t* budget,
                                 float* radius, uint16_t* ridx, int B, int heads, void* stream_) {
  if (!plan || !entropy || !ridx || B < 1 || heads < 1) return TRA_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const long long total = (long long)B * heads * plan->S;
  const RadiusArgs a = {entropy, plan->d_coord_packed, plan->d_counts, plan->d_radii_f32, budget, radius, ridx,
                        plan->N, plan->S, plan->cfg.H, plan->cfg.W, plan->n_radii, plan->cfg.budget_map,
                        plan->cfg.tau, plan->z_tau, log((double)plan->N), total, plan->d_status};
  const long long grid = (total + 255) / 256;
  if (grid > 0x7fffffffll) return TRA_ERR_UNSUPPORTED;
  if (plan->d_counts_coarse)
    tra_budget_radius_2round_kernel<<<(unsigned)grid, 256, 0, stream>>>(a, plan->d_counts_coarse);
  else
    tra_budget_radius_kernel<<<(unsigned)grid, 256, 0, stream>>>(a);
  TRA_CUDA_CHECK(cudaGetLastError());
  return TRA_OK;
}
