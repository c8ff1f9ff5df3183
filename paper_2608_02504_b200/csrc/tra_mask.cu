// Block-mask construction from per-query radii (Algorithm 1) and its CSR active-block list.
#include "tra_common.cuh"

#define TRA_MASK_THREADS 128
#define TRA_MASK_WARPS (TRA_MASK_THREADS / 32)

// ---------------------------------------------------------------------------------------
// Vote kernel.  One CTA per (batch*head, query block u).
//
// The vote keeps (u, v) iff some key column is reached (c_j > 0) and more than 60% of the
// reached columns are "high" (3*c_j > b).  Let need = floor(b/3) + 1 be the smallest high
// count and r* the need-th largest candidate index among the valid queries of u; thresholds
// grow with the candidate index and shrink with the frame distance.  With the boxes of the
// two blocks (groups of tokens, each with a frame range and a spatial box):
//   - if for every box pair even r* at the smallest frame distance cannot bridge the smallest
//     box distance, at most need-1 queries reach anything in v: no high column, vote = 0;
//   - if for every box pair r* at the largest frame distance covers the largest box distance,
//     at least `need` queries reach every key of v: every column is high, vote = 1;
//   - otherwise the b x b token tests are done: one warp per key block, each lane owning up
//     to four key columns and looping over the queries held in shared memory.
// The outcome equals the unpruned vote bit for bit.
// ---------------------------------------------------------------------------------------
template <bool kThetaInSmem>
__global__ void __launch_bounds__(TRA_MASK_THREADS)
tra_block_vote_kernel(const uint16_t* __restrict__ ridx, const uint32_t* __restrict__ coord_packed,
                      const int32_t* __restrict__ theta, const tra_block_boxes_t* __restrict__ boxes,
                      uint8_t* __restrict__ block_mask, int32_t* __restrict__ row_ptr, int N, int NB,
                      int b, int T, int n_radii, int keep_diagonal) {
  extern __shared__ int32_t s_dyn[];
  __shared__ int4 s_q[128];            // x, y, t, ridx*T of each valid query of the block
  __shared__ int s_rank_ridx[128];
  __shared__ tra_block_boxes_t s_ubox;
  __shared__ int s_rstar, s_ntest, s_count;

  int32_t* s_theta_star = s_dyn;                       // [T]
  uint16_t* s_test = (uint16_t*)(s_dyn + T);           // [NB] key blocks needing the token tests
  int32_t* s_theta = s_dyn + T + ((NB + 1) / 2);       // [n_radii*T] when kThetaInSmem
  const int32_t* th = kThetaInSmem ? s_theta : theta;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.x;
  const long long bh = blockIdx.y;
  const uint16_t* ridx_h = ridx + bh * N;
  uint8_t* mask_row = block_mask + (bh * NB + u) * (long long)NB;

  const int q0 = u * b;
  const int nq = min(b, N - q0);                       // valid queries of this block
  const int need = b / 3 + 1;

  if (kThetaInSmem)
    for (int i = tid; i < n_radii * T; i += TRA_MASK_THREADS) s_theta[i] = theta[i];
  if (tid < nq) {
    uint32_t c = coord_packed[q0 + tid];
    int r = ridx_h[q0 + tid];
    s_q[tid] = make_int4(tra_coord_x(c), tra_coord_y(c), tra_coord_t(c), r * T);
    s_rank_ridx[tid] = r;
  }
  if (tid == 0) {
    s_ubox = boxes[u];
    s_ntest = 0;
    s_count = 0;
    s_rstar = -1;
  }
  __syncthreads();

  // r*: the need-th largest candidate index (ties broken by lane order)
  if (tid < nq) {
    int mine = s_rank_ridx[tid], rank = 0;
    for (int j = 0; j < nq; ++j) {
      int o = s_rank_ridx[j];
      rank += (o > mine) || (o == mine && j < tid);
    }
    if (rank == need - 1) s_rstar = mine;
  }
  __syncthreads();
  const int rstar = s_rstar;                            // -1: fewer than `need` valid queries
  if (rstar >= 0)
    for (int i = tid; i < T; i += TRA_MASK_THREADS) s_theta_star[i] = th[rstar * T + i];
  __syncthreads();

  // classify every key block
  int kept = 0;
  for (int v = tid; v < NB; v += TRA_MASK_THREADS) {
    int decided = 0;   // 0 = vote 0, 1 = vote 1, 2 = needs the token tests
    if (rstar >= 0) {
      tra_block_boxes_t vb = boxes[v];
      bool all_reject = true, all_accept = true;
      for (int iu = 0; iu < s_ubox.n_box; ++iu) {
        const tra_box_t a = s_ubox.box[iu];
        for (int iv = 0; iv < vb.n_box; ++iv) {
          const tra_box_t c = vb.box[iv];
          int dt_min = max(0, max(a.t0 - c.t1, c.t0 - a.t1));
          int dt_max = max(a.t1 - c.t0, c.t1 - a.t0);
          int gy = max(0, max(a.y0 - c.y1, c.y0 - a.y1));
          int gx = max(0, max(a.x0 - c.x1, c.x0 - a.x1));
          int fy = max(a.y1 - c.y0, c.y1 - a.y0);
          int fx = max(a.x1 - c.x0, c.x1 - a.x0);
          if (s_theta_star[dt_min] >= gy * gy + gx * gx) all_reject = false;
          if (s_theta_star[dt_max] < fy * fy + fx * fx) all_accept = false;
        }
      }
      decided = all_reject ? 0 : (all_accept ? 1 : 2);
    }
    if (keep_diagonal && v == u) decided = 1;
    if (decided == 2) {
      s_test[atomicAdd(&s_ntest, 1)] = (uint16_t)v;
    } else {
      mask_row[v] = (uint8_t)decided;
      kept += decided;
    }
  }
  if (kept) atomicAdd(&s_count, kept);
  __syncthreads();

  // token tests for the undecided key blocks: warp per key block
  const int ntest = s_ntest;
  for (int it = warp; it < ntest; it += TRA_MASK_WARPS) {
    const int v = s_test[it];
    int kx[4], ky[4], kt[4], cnt[4];
    bool kvalid[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      int j = lane + 32 * m;
      int k = v * b + j;
      kvalid[m] = (j < b) && (k < N);
      uint32_t c = kvalid[m] ? coord_packed[k] : 0u;
      kx[m] = tra_coord_x(c);
      ky[m] = tra_coord_y(c);
      kt[m] = tra_coord_t(c);
      cnt[m] = 0;
    }
    for (int i = 0; i < nq; ++i) {
      const int4 q = s_q[i];
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        int dt = abs(q.z - kt[m]);
        int dx = q.x - kx[m], dy = q.y - ky[m];
        cnt[m] += (dx * dx + dy * dy <= th[q.w + dt]) ? 1 : 0;
      }
    }
    int nonempty = 0, high = 0;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      nonempty += __popc(__ballot_sync(0xffffffffu, kvalid[m] && cnt[m] > 0));
      high += __popc(__ballot_sync(0xffffffffu, kvalid[m] && 3 * cnt[m] > b));
    }
    if (lane == 0) {
      int keep = (nonempty > 0) && (10 * high > 6 * nonempty);
      mask_row[v] = (uint8_t)keep;
      if (keep) atomicAdd(&s_count, 1);
    }
  }
  __syncthreads();
  if (tid == 0) row_ptr[bh * NB + u + 1] = s_count;   // per-row count; scanned in place afterwards
}

// ---------------------------------------------------------------------------------------
// In-place exclusive scan of the per-row counts held in row_ptr[1..rows] (one CTA).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
tra_row_ptr_scan_kernel(int32_t* __restrict__ row_ptr, long long rows, long long capacity,
                        int64_t* __restrict__ nnz_out, int* __restrict__ status) {
  __shared__ long long s_part[1024];
  const int tid = threadIdx.x;
  const long long chunk = (rows + 1023) / 1024;
  const long long lo = min(rows, tid * chunk), hi = min(rows, lo + chunk);
  long long sum = 0;
  for (long long i = lo; i < hi; ++i) sum += row_ptr[i + 1];
  s_part[tid] = sum;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {
    long long add = tid >= off ? s_part[tid - off] : 0;
    __syncthreads();
    s_part[tid] += add;
    __syncthreads();
  }
  long long run = s_part[tid] - sum;                   // exclusive prefix of this chunk
  const long long total = s_part[1023];
  for (long long i = lo; i < hi; ++i) {
    run += row_ptr[i + 1];
    row_ptr[i + 1] = (int32_t)run;
  }
  if (tid == 0) {
    row_ptr[0] = 0;
    if (nnz_out) *nnz_out = total;
    if (total > capacity || total > 0x7fffffffll) tra_set_status(status, TRA_ERR_CAPACITY);
  }
}

// ---------------------------------------------------------------------------------------
// col_idx fill: one warp per row, ascending key blocks (ballot + prefix popcount).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
tra_col_idx_fill_kernel(const uint8_t* __restrict__ block_mask, const int32_t* __restrict__ row_ptr,
                        int32_t* __restrict__ col_idx, long long rows, int NB, long long capacity) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const uint8_t* m = block_mask + row * NB;
  long long base = row_ptr[row];
  for (int v0 = 0; v0 < NB; v0 += 32) {
    int v = v0 + lane;
    bool keep = v < NB && m[v] != 0;
    unsigned bal = __ballot_sync(0xffffffffu, keep);
    if (keep) {
      long long pos = base + __popc(bal & ((1u << lane) - 1u));
      if (pos < capacity) col_idx[pos] = v;
    }
    base += __popc(bal);
  }
}

extern "C" int tra_build_block_mask(const tra_plan_t* plan, const uint16_t* ridx, uint8_t* block_mask,
                                    int32_t* row_ptr, int32_t* col_idx, int64_t col_idx_capacity,
                                    int64_t* nnz_out, int B, int heads, void* stream_) {
  if (!plan || !ridx || !block_mask || !row_ptr || !col_idx || B < 1 || heads < 1 ||
      col_idx_capacity < 0)
    return TRA_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const int NB = plan->NB, T = plan->cfg.T, nr = plan->n_radii;
  const long long BH = (long long)B * heads;
  if (NB > 65535 || BH > 65535) return TRA_ERR_UNSUPPORTED;
  const long long rows = BH * NB;

  size_t base_words = (size_t)T + (NB + 1) / 2;
  size_t smem_with_theta = (base_words + (size_t)nr * T) * sizeof(int32_t);
  dim3 grid((unsigned)NB, (unsigned)BH);
  if (smem_with_theta <= 160 * 1024) {
    if (smem_with_theta > 48 * 1024)
      TRA_CUDA_CHECK(cudaFuncSetAttribute(tra_block_vote_kernel<true>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)smem_with_theta));
    tra_block_vote_kernel<true><<<grid, TRA_MASK_THREADS, smem_with_theta, stream>>>(
        ridx, plan->d_coord_packed, plan->d_theta, plan->d_boxes, block_mask, row_ptr, plan->N, NB,
        plan->cfg.block, T, nr, (plan->cfg.flags & TRA_KEEP_DIAGONAL) ? 1 : 0);
  } else {
    size_t smem = base_words * sizeof(int32_t);
    if (smem > 48 * 1024)
      TRA_CUDA_CHECK(cudaFuncSetAttribute(tra_block_vote_kernel<false>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    tra_block_vote_kernel<false><<<grid, TRA_MASK_THREADS, smem, stream>>>(
        ridx, plan->d_coord_packed, plan->d_theta, plan->d_boxes, block_mask, row_ptr, plan->N, NB,
        plan->cfg.block, T, nr, (plan->cfg.flags & TRA_KEEP_DIAGONAL) ? 1 : 0);
  }
  TRA_CUDA_CHECK(cudaGetLastError());
  tra_row_ptr_scan_kernel<<<1, 1024, 0, stream>>>(row_ptr, rows, (long long)col_idx_capacity, nnz_out,
                                                  plan->d_status);
  TRA_CUDA_CHECK(cudaGetLastError());
  tra_col_idx_fill_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, stream>>>(
      block_mask, row_ptr, col_idx, rows, NB, (long long)col_idx_capacity);
  TRA_CUDA_CHECK(cudaGetLastError());
  return TRA_OK;
}
