// Plan construction, plan-time tables and the tile-major layout kernels.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "tra_common.cuh"

// ---------------------------------------------------------------------------------------
// Count table C_grid (Eq. 13), the per-coordinate lookup table of Section 3.2.
// One thread per (y, x, candidate k).  The in-frame count
//   A(theta) = #{(y', x') : (y'-y)^2 + (x'-x)^2 <= theta}
// is a sweep over rows: each row contributes the clipped length of an x-interval.
// C(f) = sum_t A(theta[k][|t - f|]) is carried from frame to frame:
//   C(f+1) = C(f) + A(theta[f+1]) - A(theta[T-1-f]).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int tra_isqrt(int n) {
  int s = (int)sqrtf((float)n);
  while (s * s > n) --s;
  while ((s + 1) * (s + 1) <= n) ++s;
  return s;
}

__device__ __forceinline__ uint32_t tra_frame_count(int y, int x, int H, int W, int theta) {
  int R = tra_isqrt(theta);
  int ylo = max(0, y - R), yhi = min(H - 1, y + R);
  uint32_t c = 0;
  for (int yy = ylo; yy <= yhi; ++yy) {
    int dy = yy - y;
    int w = tra_isqrt(theta - dy * dy);
    c += (uint32_t)(min(x + w, W - 1) - max(x - w, 0) + 1);
  }
  return c;
}

__global__ void tra_count_table_kernel(int T, int H, int W, int n_radii,
                                       const int32_t* __restrict__ theta,
                                       uint32_t* __restrict__ counts, int* __restrict__ status) {
  int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= H * W * n_radii) return;
  int k = g % n_radii;
  int yx = g / n_radii;
  int y = yx / W, x = yx % W;
  const int32_t* th = theta + (size_t)k * T;
  uint32_t c = 0;
  for (int delta = 0; delta < T; ++delta) c += tra_frame_count(y, x, H, W, th[delta]);
  size_t frame_stride = (size_t)H * W * n_radii;
  size_t base = (size_t)yx * n_radii + k;
  [[maybe_unused]] const size_t n_counts = frame_stride * T;
  if (TRA_IDX(base, n_counts, status)) counts[base] = c;  // f = 0
  for (int f = 0; f + 1 < T; ++f) {
    c += tra_frame_count(y, x, H, W, th[f + 1]);
    c -= tra_frame_count(y, x, H, W, th[T - 1 - f]);
    if (TRA_IDX(base + (size_t)(f + 1) * frame_stride, n_counts, status))
      counts[base + (size_t)(f + 1) * frame_stride] = c;
  }
}

// ---------------------------------------------------------------------------------------
// Tile-major gather / scatter of token rows (Section 3.3).  16 bytes per thread.
// ---------------------------------------------------------------------------------------
template <bool kGather>
__global__ void tra_permute_rows_kernel(const int32_t* __restrict__ raster_of_pos,
                                        const uint4* __restrict__ src, uint4* __restrict__ dst,
                                        int N, int S, int chunks_per_row, long long total_chunks,
                                        int* __restrict__ status) {
  long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= total_chunks) return;
  int chunk = (int)(g % chunks_per_row);
  long long row = g / chunks_per_row;  // bh * S + p
  int p = (int)(row % S);
  long long bh = row / S;
  long long other = bh * S + (p < N ? raster_of_pos[p] : p);   // text tokens stay in place
  if (!TRA_IDX(other * chunks_per_row + chunk, total_chunks, status)) return;
  if (kGather)
    dst[row * chunks_per_row + chunk] = src[other * chunks_per_row + chunk];
  else
    dst[other * chunks_per_row + chunk] = src[row * chunks_per_row + chunk];
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
// Phi^-1(p) for p in (0, 1]: bisection on erfc (monotone), to the last bit that matters here.
static double tra_inverse_normal_cdf(double p) {
  if (p >= 1.0) return INFINITY;
  double lo = -40.0, hi = 40.0;
  for (int it = 0; it < 200; ++it) {
    double mid = 0.5 * (lo + hi);
    double cdf = 0.5 * erfc(-mid / sqrt(2.0));
    if (cdf < p) lo = mid; else hi = mid;
  }
  return 0.5 * (lo + hi);
}

static void tra_plan_free(tra_plan* p) {
  if (!p) return;
  free(p->h_radii);
  free(p->h_theta);
  free(p->h_coord);
  cudaFree(p->d_coord_packed);
  cudaFree(p->d_slice);
  cudaFree(p->d_raster_of_pos);
  cudaFree(p->d_slice_raster);
  cudaFree(p->d_theta);
  cudaFree(p->d_radii_f32);
  cudaFree(p->d_counts);
  cudaFree(p->d_counts_coarse);
  cudaFree(p->d_boxes);
  cudaFree(p->d_field_pos);
  cudaFree(p->d_status);
  if (p->pair_stream) cudaStreamDestroy(p->pair_stream);
  if (p->pair_fork) cudaEventDestroy(p->pair_fork);
  if (p->pair_join) cudaEventDestroy(p->pair_join);
  if (p->copy_in) cudaStreamDestroy(p->copy_in);
  if (p->copy_out) cudaStreamDestroy(p->copy_out);
  for (int i = 0; i < p->n_events; ++i) cudaEventDestroy(p->events[i]);
  free(p->events);
  delete p;
}

extern "C" int tra_plan_create(tra_plan_t** out, const tra_config_t* cfg, void* stream_) {
  if (!out || !cfg) return TRA_ERR_INVALID_ARG;
  *out = nullptr;
  cudaStream_t stream = (cudaStream_t)stream_;
  const int T = cfg->T, H = cfg->H, W = cfg->W;
  if (T < 1 || H < 1 || W < 1 || cfg->tile_h < 1 || cfg->tile_w < 1) return TRA_ERR_INVALID_ARG;
  if (!(cfg->tau > 0.0 && cfg->tau <= 1.0) || !(cfg->gamma >= 0.0)) return TRA_ERR_INVALID_ARG;
  if (T > 1023 || H > 1023 || W > 1023) return TRA_ERR_UNSUPPORTED;
  if (cfg->block < 16 || cfg->block > 128) return TRA_ERR_UNSUPPORTED;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return TRA_ERR_UNSUPPORTED;
  if ((long long)T * H * W > (1ll << 30)) return TRA_ERR_UNSUPPORTED;
  if (cfg->budget_map != TRA_BUDGET_UNIFORM && cfg->budget_map != TRA_BUDGET_LOGNORMAL)
    return TRA_ERR_INVALID_ARG;
  if (cfg->n_text < 0 || cfg->n_text > (1 << 24)) return TRA_ERR_INVALID_ARG;
  if (cfg->flags & ~(TRA_KEEP_DIAGONAL | TRA_ORDER_RASTER | TRA_ORDER_RASTER_QO)) return TRA_ERR_INVALID_ARG;

  tra_plan* p = new tra_plan();
  memset(p, 0, sizeof(*p));
  p->cfg = *cfg;
  p->cfg.radii = nullptr;
  p->N = T * H * W;
  p->S = p->N + cfg->n_text;
  p->NB = (p->S + cfg->block - 1) / cfg->block;
  // video blocks: made of video tokens only when text follows (the block that holds both kinds is
  // kept dense like a text block, so that every text key stays visible: Section 3.2, last paragraph)
  p->NBv = cfg->n_text > 0 ? p->N / cfg->block : (p->N + cfg->block - 1) / cfg->block;
  p->z_tau = tra_inverse_normal_cdf(cfg->tau);
  if (cudaGetDevice(&p->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device) != cudaSuccess) {
    delete p;
    return TRA_ERR_CUDA;
  }

  // candidate radii (set R of Eq. 14)
  const double diag2 = (double)(H - 1) * (H - 1) + (double)(W - 1) * (W - 1);
  std::vector<double> radii;
  if (cfg->radii) {
    if (cfg->n_radii < 1 || cfg->n_radii > 65535) {
      delete p;
      return TRA_ERR_INVALID_ARG;
    }
    for (int i = 0; i < cfg->n_radii; ++i) {
      if (!(cfg->radii[i] >= 0.0) || (i > 0 && !(cfg->radii[i] > cfg->radii[i - 1]))) {
        delete p;
        return TRA_ERR_INVALID_ARG;
      }
      radii.push_back(cfg->radii[i]);
    }
  } else {
    const int D = (int)ceil(sqrt(diag2));
    for (int r = 0; r <= D; ++r) radii.push_back((double)r);
    if (cfg->radius_policy == TRA_RADII_LITERAL) {
      radii.push_back(INFINITY);
    } else if (cfg->radius_policy == TRA_RADII_EXTENDED) {
      for (int m = 1; m < T; ++m) {
        double r = (double)D * exp(cfg->gamma * (double)m);
        if (r > radii.back()) radii.push_back(r);
      }
      // the last one is the full-support radius: when the diagonal is an integer, rounding can leave
      // r^2 exp(-2 gamma (T-1)) just below its square; the radius then moves up by single steps until it covers
      while (!(radii.back() * radii.back() * exp(-2.0 * cfg->gamma * (double)(T - 1)) >= diag2))
        radii.back() = nextafter(radii.back(), INFINITY);
    } else {
      delete p;
      return TRA_ERR_INVALID_ARG;
    }
  }
  if (radii.size() > 65535) {
    delete p;
    return TRA_ERR_UNSUPPORTED;
  }
  p->n_radii = (int)radii.size();
  const int nr = p->n_radii;

  // thresholds theta[k][delta] = min(floor(r_k^2 exp(-2 gamma delta)), diag^2)   (Eq. 10, Eq. 15)
  p->h_radii = (double*)malloc(sizeof(double) * nr);
  p->h_theta = (int32_t*)malloc(sizeof(int32_t) * nr * T);
  p->h_coord = (int32_t*)malloc(sizeof(int32_t) * 3 * (size_t)p->N);
  std::vector<float> radii_f32(nr);
  for (int k = 0; k < nr; ++k) {
    p->h_radii[k] = radii[k];
    radii_f32[k] = (float)radii[k];
    for (int delta = 0; delta < T; ++delta) {
      double v = diag2;
      if (!isinf(radii[k])) {
        double decayed = radii[k] * radii[k] * exp(-2.0 * cfg->gamma * (double)delta);
        if (decayed < diag2) v = decayed;
      }
      p->h_theta[k * T + delta] = (int32_t)floor(v);
    }
  }
  // the last candidate must be the full-support radius at every frame distance
  for (int delta = 0; delta < T; ++delta)
    if (p->h_theta[(nr - 1) * T + delta] != (int32_t)diag2) {
      tra_plan_free(p);
      return TRA_ERR_INVALID_ARG;
    }

  // tile-major order and per-block boxes (Section 3.3)
  std::vector<uint32_t> packed(p->N + 128, 0u);   // padded by one block for vector loads past the end
  std::vector<int32_t> raster(p->N);
  std::vector<int32_t> tile_of_pos(p->N);
  {
    int pos = 0, tile_id = 0;
    for (int t = 0; t < T; ++t)
      for (int y0 = 0; y0 < H; y0 += cfg->tile_h)
        for (int x0 = 0; x0 < W; x0 += cfg->tile_w) {
          for (int y = y0; y < H && y < y0 + cfg->tile_h; ++y)
            for (int x = x0; x < W && x < x0 + cfg->tile_w; ++x) {
              p->h_coord[3 * pos] = t;
              p->h_coord[3 * pos + 1] = y;
              p->h_coord[3 * pos + 2] = x;
              packed[pos] = tra_pack_coord(t, y, x);
              raster[pos] = (t * H + y) * W + x;
              tile_of_pos[pos] = tile_id;
              ++pos;
            }
          ++tile_id;
        }
  }
  std::vector<tra_block_boxes_t> boxes(p->NB);
  for (int u = 0; u < p->NB; ++u) {   // text-only blocks keep n_box = 0
    tra_block_boxes_t bb;
    memset(&bb, 0, sizeof(bb));
    int nb = 0, last_tile = -1;
    for (int pos = u * cfg->block; pos < p->N && pos < (u + 1) * cfg->block; ++pos) {
      int t = p->h_coord[3 * pos], y = p->h_coord[3 * pos + 1], x = p->h_coord[3 * pos + 2];
      if (tile_of_pos[pos] != last_tile && nb < TRA_MAX_SEG) {
        tra_box_t b = {(int16_t)t, (int16_t)t, (int16_t)y, (int16_t)y, (int16_t)x, (int16_t)x, 0, 0};
        bb.box[nb++] = b;
      } else {
        tra_box_t& b = bb.box[nb - 1];
        if (t < b.t0) b.t0 = (int16_t)t;
        if (t > b.t1) b.t1 = (int16_t)t;
        if (y < b.y0) b.y0 = (int16_t)y;
        if (y > b.y1) b.y1 = (int16_t)y;
        if (x < b.x0) b.x0 = (int16_t)x;
        if (x > b.x1) b.x1 = (int16_t)x;
      }
      last_tile = tile_of_pos[pos];
    }
    bb.n_box = nb;
    boxes[u] = bb;
  }

  // 16-position slices that are a run of one frame row (the token mask inside blocks tests such a
  // slice as an x-interval)
  const size_t n_slice = (((size_t)p->NB * cfg->block / 16) + 7) & ~(size_t)7;
  std::vector<uint32_t> slices(n_slice, 0u);
  for (size_t si = 0; si < n_slice; ++si) {
    const long long p0 = (long long)si * 16;
    if (p0 + 15 >= p->N) continue;
    const int t = p->h_coord[3 * p0], y = p->h_coord[3 * p0 + 1], x = p->h_coord[3 * p0 + 2];
    bool run = true;
    for (int j = 1; j < 16 && run; ++j)
      run = p->h_coord[3 * (p0 + j)] == t && p->h_coord[3 * (p0 + j) + 1] == y &&
            p->h_coord[3 * (p0 + j) + 2] == x + j;
    if (run) slices[si] = tra_pack_coord(t, y, x) | (1u << 30);
  }

  // block vote: where the count of a frame cell goes in the frame's tile-major order
  std::vector<uint16_t> field_pos;
  const bool field_pos_fits = (long long)H * W <= 65535;
  if (field_pos_fits) {
    std::vector<int32_t> pos_of((size_t)H * W);
    for (int i = 0; i < H * W; ++i) pos_of[(size_t)p->h_coord[3 * i + 1] * W + p->h_coord[3 * i + 2]] = i;
    bool quads = W % 4 == 0 && cfg->block % 4 == 0;      // a group of four positions never straddles two blocks
    for (int c = 0; c < H * W && quads; c += 4)
      quads = pos_of[c] % 4 == 0 && pos_of[c + 1] == pos_of[c] + 1 && pos_of[c + 2] == pos_of[c] + 2 &&
              pos_of[c + 3] == pos_of[c] + 3;
    // 2: moreover the sixteen cells (y, 16 m .. 16 m + 15) are sixteen consecutive positions that start at a
    // multiple of sixteen and lie inside one block in every frame
    bool seg16 = quads && W % 16 == 0 && cfg->block % 16 == 0;
    for (int c = 0; c < H * W && seg16; c += 16)
      for (int i = 0; i < 16 && seg16; ++i) seg16 = pos_of[c] % 16 == 0 && pos_of[c + i] == pos_of[c] + i;
    p->field_quads = seg16 ? 2 : (quads ? 1 : 0);
    const int per = seg16 ? 16 : (quads ? 4 : 1);        // cells per entry: entry i = position of cell i * per, / per
    const size_t n = (size_t)H * W / per;
    field_pos.assign((n + 7) & ~(size_t)7, 0);
    for (size_t i = 0; i < n; ++i) field_pos[i] = (uint16_t)(pos_of[per * i] / per);
  }

  // Raster-order attention (TRA_ORDER_RASTER, TRA_ORDER_RASTER_QO): the raster row at which every run of 16 consecutive tile-major
  // positions starts.  Needs every such run to be 16 consecutive raster rows (W and the tile width multiples of
  // 16) and blocks that start on run boundaries; entries past the sequence hold S, a row outside the tensor (the
  // load of such a run is filled with zeros).
  std::vector<int32_t> slice_raster;
  if (cfg->flags & (TRA_ORDER_RASTER | TRA_ORDER_RASTER_QO)) {
    bool runs = cfg->block % 16 == 0 && p->N % 16 == 0;
    for (int s0 = 0; s0 < p->N && runs; s0 += 16)
      for (int i = 1; i < 16 && runs; ++i) runs = raster[s0 + i] == raster[s0] + i;
    if (!runs) {
      tra_plan_free(p);
      return TRA_ERR_UNSUPPORTED;
    }
    slice_raster.assign((size_t)p->S / 16 + 32, p->S);
    for (int s0 = 0; s0 < p->S; s0 += 16) slice_raster[s0 / 16] = s0 < p->N ? raster[s0] : s0;   // text stays in place
  }

  // device tables
  const size_t count_elems = (size_t)p->N * nr;
  bool ok = cudaMalloc(&p->d_coord_packed, sizeof(uint32_t) * (p->N + 128)) == cudaSuccess &&
            cudaMalloc(&p->d_slice, sizeof(uint32_t) * n_slice) == cudaSuccess &&
            cudaMalloc(&p->d_raster_of_pos, sizeof(int32_t) * p->N) == cudaSuccess &&
            cudaMalloc(&p->d_theta, sizeof(int32_t) * nr * T) == cudaSuccess &&
            cudaMalloc(&p->d_radii_f32, sizeof(float) * nr) == cudaSuccess &&
            cudaMalloc(&p->d_counts, sizeof(uint32_t) * count_elems) == cudaSuccess &&
            (nr > 128 || cudaMalloc(&p->d_counts_coarse, sizeof(uint32_t) * (16 + 128) * (size_t)p->N) == cudaSuccess) &&
            cudaMalloc(&p->d_boxes, sizeof(tra_block_boxes_t) * p->NB) == cudaSuccess &&
            (!field_pos_fits || cudaMalloc(&p->d_field_pos, sizeof(uint16_t) * field_pos.size()) == cudaSuccess) &&
            cudaMalloc(&p->d_status, sizeof(int)) == cudaSuccess &&
            (slice_raster.empty() ||
             cudaMalloc(&p->d_slice_raster, sizeof(int32_t) * slice_raster.size()) == cudaSuccess) &&
            cudaStreamCreateWithFlags(&p->pair_stream, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&p->pair_fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p->pair_join, cudaEventDisableTiming) == cudaSuccess;
  ok = ok &&
       cudaMemcpyAsync(p->d_coord_packed, packed.data(), sizeof(uint32_t) * (p->N + 128),
                       cudaMemcpyHostToDevice, stream) == cudaSuccess &&
       cudaMemcpyAsync(p->d_slice, slices.data(), sizeof(uint32_t) * n_slice, cudaMemcpyHostToDevice,
                       stream) == cudaSuccess &&
       cudaMemcpyAsync(p->d_raster_of_pos, raster.data(), sizeof(int32_t) * p->N,
                       cudaMemcpyHostToDevice, stream) == cudaSuccess &&
       (slice_raster.empty() ||
        cudaMemcpyAsync(p->d_slice_raster, slice_raster.data(), sizeof(int32_t) * slice_raster.size(),
                        cudaMemcpyHostToDevice, stream) == cudaSuccess) &&
       cudaMemcpyAsync(p->d_theta, p->h_theta, sizeof(int32_t) * nr * T, cudaMemcpyHostToDevice,
                       stream) == cudaSuccess &&
       cudaMemcpyAsync(p->d_radii_f32, radii_f32.data(), sizeof(float) * nr,
                       cudaMemcpyHostToDevice, stream) == cudaSuccess &&
       cudaMemcpyAsync(p->d_boxes, boxes.data(), sizeof(tra_block_boxes_t) * p->NB,
                       cudaMemcpyHostToDevice, stream) == cudaSuccess &&
       (!field_pos_fits || cudaMemcpyAsync(p->d_field_pos, field_pos.data(), sizeof(uint16_t) * field_pos.size(),
                                           cudaMemcpyHostToDevice, stream) == cudaSuccess) &&
       cudaMemsetAsync(p->d_status, 0, sizeof(int), stream) == cudaSuccess;
  if (ok) {
    int total = H * W * nr;
    tra_count_table_kernel<<<(total + 127) / 128, 128, 0, stream>>>(T, H, W, nr, p->d_theta,
                                                                    p->d_counts, p->d_status);
    ok = cudaGetLastError() == cudaSuccess;
    if (ok && p->d_counts_coarse)
      ok = tra_build_coarse_table(p->d_counts, p->d_counts_coarse, (long long)p->N, nr, p->d_status, stream) == TRA_OK;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  }
  if (!ok) {
    tra_plan_free(p);
    return TRA_ERR_CUDA;
  }
  *out = p;
  return TRA_OK;
}

extern "C" int tra_plan_destroy(tra_plan_t* plan) {
  if (!plan) return TRA_ERR_INVALID_ARG;
  tra_plan_free(plan);
  return TRA_OK;
}

extern "C" int tra_plan_num_tokens(const tra_plan_t* plan) { return plan ? plan->S : TRA_ERR_INVALID_ARG; }
extern "C" int tra_plan_num_video_tokens(const tra_plan_t* plan) { return plan ? plan->N : TRA_ERR_INVALID_ARG; }
extern "C" int tra_plan_num_blocks(const tra_plan_t* plan) { return plan ? plan->NB : TRA_ERR_INVALID_ARG; }
extern "C" int tra_plan_num_radii(const tra_plan_t* plan) { return plan ? plan->n_radii : TRA_ERR_INVALID_ARG; }
extern "C" int tra_plan_num_tile_pairs(const tra_plan_t* plan) {
  if (!plan) return TRA_ERR_INVALID_ARG;
  if (plan->cfg.block <= 32) return 0;                 // no attention launch for such blocks
  const int G = tra_blocks_per_tile(plan->cfg.block);
  return ((plan->NB + G - 1) / G + 1) / 2;
}

extern "C" int tra_plan_tables(const tra_plan_t* plan, double* radii, int32_t* theta, int32_t* coord) {
  if (!plan) return TRA_ERR_INVALID_ARG;
  if (radii) memcpy(radii, plan->h_radii, sizeof(double) * plan->n_radii);
  if (theta) memcpy(theta, plan->h_theta, sizeof(int32_t) * plan->n_radii * plan->cfg.T);
  if (coord) memcpy(coord, plan->h_coord, sizeof(int32_t) * 3 * (size_t)plan->N);
  return TRA_OK;
}

extern "C" int tra_plan_count_table(const tra_plan_t* plan, uint32_t* counts) {
  if (!plan || !counts) return TRA_ERR_INVALID_ARG;
  TRA_CUDA_CHECK(cudaMemcpy(counts, plan->d_counts, sizeof(uint32_t) * (size_t)plan->N * plan->n_radii,
                            cudaMemcpyDeviceToHost));
  return TRA_OK;
}

extern "C" int tra_plan_status(tra_plan_t* plan, void* stream_) {
  if (!plan) return TRA_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  int code = 0;
  TRA_CUDA_CHECK(cudaMemcpyAsync(&code, plan->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream));
  TRA_CUDA_CHECK(cudaMemsetAsync(plan->d_status, 0, sizeof(int), stream));
  TRA_CUDA_CHECK(cudaStreamSynchronize(stream));
  return code;
}

extern "C" const char* tra_status_string(int status) {
  switch (status) {
    case TRA_OK: return "ok";
    case TRA_ERR_INVALID_ARG: return "invalid argument";
    case TRA_ERR_UNSUPPORTED: return "unsupported head_dim, block or grid size";
    case TRA_ERR_CAPACITY: return "col_idx capacity too small";
    case TRA_ERR_CUDA: return "CUDA call failed";
    case TRA_ERR_TIMEOUT: return "bounded device-side wait expired";
    case TRA_ERR_BOUNDS: return "debug build: index out of range or inconsistent work lists";
    default: return "unknown status";
  }
}

static int tra_permute(const tra_plan_t* plan, const void* src, void* dst, int n_bh, int row_bytes,
                       void* stream_, bool gather) {
  if (!plan || !src || !dst || n_bh < 1 || row_bytes < 16 || (row_bytes & 15)) return TRA_ERR_INVALID_ARG;
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return TRA_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  int chunks = row_bytes / 16;
  long long total = (long long)n_bh * plan->S * chunks;
  long long grid = (total + 255) / 256;
  if (grid > 0x7fffffffll) return TRA_ERR_UNSUPPORTED;
  if (gather)
    tra_permute_rows_kernel<true><<<(unsigned)grid, 256, 0, stream>>>(
        plan->d_raster_of_pos, (const uint4*)src, (uint4*)dst, plan->N, plan->S, chunks, total, plan->d_status);
  else
    tra_permute_rows_kernel<false><<<(unsigned)grid, 256, 0, stream>>>(
        plan->d_raster_of_pos, (const uint4*)src, (uint4*)dst, plan->N, plan->S, chunks, total, plan->d_status);
  TRA_CUDA_CHECK(cudaGetLastError());
  return TRA_OK;
}

extern "C" int tra_tile_major_gather(const tra_plan_t* plan, const void* src_raster, void* dst_tile_major,
                                     int n_bh, int row_bytes, void* stream) {
  return tra_permute(plan, src_raster, dst_tile_major, n_bh, row_bytes, stream, true);
}

extern "C" int tra_tile_major_scatter(const tra_plan_t* plan, const void* src_tile_major, void* dst_raster,
                                      int n_bh, int row_bytes, void* stream) {
  return tra_permute(plan, src_tile_major, dst_raster, n_bh, row_bytes, stream, false);
}
