/*
 * fp64 CPU oracle for the Token Radius Attention hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition of what the
 * CUDA library computes, written from the paper's equations.  It shares no code,
 * header, table or constant with the CUDA path, and nothing in the product path
 * may call it: only the tests, the smoke check and the benchmark's CPU-baseline
 * leg load it.
 *
 * Conventions
 *   - a token's coordinate is (t, y, x): frame, row, column of the T x H x W grid
 *     (the paper's (f, y, x) with x the horizontal axis);
 *   - "position" p = index of a token in tile-major order (Section 3.3, "Flash
 *     Radius Mask Kernel"); blocks are b consecutive positions (Algorithm 1:
 *     q = u*b + i, guarded by q < N);
 *   - entropies are in nats (Appendix "Fused Attention Entropy Kernel");
 *   - Q/K/V arrive as bf16 bit patterns (uint16) and are widened exactly.
 *
 * Readings taken where the paper is silent are stated at each function.
 * Parity status: every function here is pinned by tests/test_oracle_*.py except
 * the absolute choice of tau, gamma and the candidate-radius set, which the paper
 * does not fix ("parity unpinned" for those three choices only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_widen(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

int tra_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------- *
 * Tile-major token order (Section 3.3; Appendix "Kernel execution").
 * Every H x W frame is cut into tile_h x tile_w tiles (edge tiles clipped);
 * tokens are listed frame by frame, tile row by tile row, tile by tile, and
 * row-major inside a tile.  coord[p] = (t, y, x) of position p.
 * ------------------------------------------------------------------------- */
int tra_oracle_tile_major(int T, int H, int W, int tile_h, int tile_w, int32_t* coord) {
  int p = 0;
  for (int t = 0; t < T; ++t)
    for (int y0 = 0; y0 < H; y0 += tile_h)
      for (int x0 = 0; x0 < W; x0 += tile_w)
        for (int y = y0; y < y0 + tile_h && y < H; ++y)
          for (int x = x0; x < x0 + tile_w && x < W; ++x) {
            coord[3 * p + 0] = t;
            coord[3 * p + 1] = y;
            coord[3 * p + 2] = x;
            ++p;
          }
  return p;
}

/* ------------------------------------------------------------------------- *
 * Candidate radii: the set R of Eq. 14, which the paper describes only as the
 * radii available on the latent grid plus one that reaches full support, without
 * listing them; reading taken:
 *   policy 0 ("extended"): 0,1,...,D with D = ceil(frame diagonal), then
 *       D*exp(gamma*m) for m = 1..T-1; the last one covers the diagonal even
 *       at the largest frame distance, so it is the full-support radius.
 *   policy 1 ("literal"):  0,1,...,D and +infinity as the full-support radius.
 * Returns the number of radii written (strictly ascending), or -1 if cap is
 * too small.
 * ------------------------------------------------------------------------- */
int tra_oracle_default_radii(int T, int H, int W, double gamma, int policy, double* out, int cap) {
  double diag2 = (double)(H - 1) * (H - 1) + (double)(W - 1) * (W - 1);
  int D = (int)ceil(sqrt(diag2));
  int n = 0;
  for (int r = 0; r <= D; ++r) {
    if (n >= cap) return -1;
    out[n++] = (double)r;
  }
  if (policy == 1) {
    if (n >= cap) return -1;
    out[n++] = INFINITY;
    return n;
  }
  for (int m = 1; m <= T - 1; ++m) {
    double r = (double)D * exp(gamma * (double)m);
    if (r > out[n - 1]) {
      if (n >= cap) return -1;
      out[n++] = r;
    }
  }
  /* The last candidate is the full-support radius: it must cover the diagonal at the largest frame
   * distance.  In exact arithmetic D*exp(gamma*(T-1)) does; when the diagonal is an integer (D^2 =
   * diag2) the rounded product r*r*exp(-2*gamma*(T-1)) can fall just below diag2, and the radius is
   * then moved up by single floating-point steps until it covers. */
  while (!(out[n - 1] * out[n - 1] * exp(-2.0 * gamma * (double)(T - 1)) >= diag2)) out[n - 1] = nextafter(out[n - 1], INFINITY);
  return n;
}

/* ------------------------------------------------------------------------- *
 * Squared-distance thresholds.  Eq. 15 keeps key j for query i when
 * d_s(i,j) <= r_i * phi(|f_j - f_i|), phi(delta) = exp(-gamma*delta) (Eq. 10).
 * Squared distances on the grid are integers, so the test is the same as
 * d_s^2 <= floor(r^2 * exp(-2*gamma*delta)); the floor is clamped to the
 * squared frame diagonal (beyond it every key of the frame is inside).
 * theta[k*T + delta] for candidate k.
 * ------------------------------------------------------------------------- */
void tra_oracle_theta(const double* radii, int n_radii, int T, int H, int W, double gamma,
                      int32_t* theta) {
  double diag2 = (double)(H - 1) * (H - 1) + (double)(W - 1) * (W - 1);
  for (int k = 0; k < n_radii; ++k)
    for (int delta = 0; delta < T; ++delta) {
      double v;
      if (isinf(radii[k])) {
        v = diag2;
      } else {
        v = radii[k] * radii[k] * exp(-2.0 * gamma * (double)delta);
        if (!(v < diag2)) v = diag2;
      }
      theta[k * T + delta] = (int32_t)floor(v);
    }
}

/* ------------------------------------------------------------------------- *
 * Boundary-aware support count, Eq. 13, by direct enumeration of every key of
 * the grid.  theta_row = thresholds of one candidate radius (T entries).
 * ------------------------------------------------------------------------- */
int64_t tra_oracle_grid_count_brute(int T, int H, int W, const int32_t* theta_row, int f, int y,
                                    int x) {
  int64_t c = 0;
  for (int t = 0; t < T; ++t) {
    int delta = t > f ? t - f : f - t;
    for (int yy = 0; yy < H; ++yy)
      for (int xx = 0; xx < W; ++xx) {
        int d2 = (yy - y) * (yy - y) + (xx - x) * (xx - x);
        if (d2 <= theta_row[delta]) ++c;
      }
  }
  return c;
}

/* ------------------------------------------------------------------------- *
 * The same count for every (t, y, x, candidate): counts[((t*H+y)*W+x)*n_radii+k].
 * Instead of re-enumerating the frame for every threshold, the squared
 * distances from (y, x) are histogrammed once and summed cumulatively, so
 * cum[v] = #{(y',x') : d^2 <= v}; Eq. 13 is then the sum over frames of
 * cum[theta].  Checked against tra_oracle_grid_count_brute in the tests.
 * ------------------------------------------------------------------------- */
void tra_oracle_grid_count_table(int T, int H, int W, const int32_t* theta, int n_radii,
                                 uint32_t* counts) {
  int diag2 = (H - 1) * (H - 1) + (W - 1) * (W - 1);
#pragma omp parallel
  {
    uint32_t* cum = (uint32_t*)malloc((size_t)(diag2 + 1) * sizeof(uint32_t));
#pragma omp for schedule(dynamic, 8)
    for (int yx = 0; yx < H * W; ++yx) {
      int y = yx / W, x = yx % W;
      memset(cum, 0, (size_t)(diag2 + 1) * sizeof(uint32_t));
      for (int yy = 0; yy < H; ++yy)
        for (int xx = 0; xx < W; ++xx) cum[(yy - y) * (yy - y) + (xx - x) * (xx - x)] += 1;
      for (int v = 1; v <= diag2; ++v) cum[v] += cum[v - 1];
      for (int f = 0; f < T; ++f)
        for (int k = 0; k < n_radii; ++k) {
          uint32_t c = 0;
          for (int t = 0; t < T; ++t) {
            int delta = t > f ? t - f : f - t;
            c += cum[theta[k * T + delta]];
          }
          counts[((size_t)(f * H + y) * W + x) * n_radii + k] = c;
        }
    }
    free(cum);
  }
}

/* ------------------------------------------------------------------------- *
 * Entropy-to-budget map, Eq. 8: K = ceil(tau * exp(H)), clamped to [1, N].
 * H is the fp32 entropy handed to the stage, widened to fp64.
 * fragile[i] = 1 when tau*exp(H) lies within a few ulps of an integer, so that
 * a differently rounded exp() could move the ceiling; parity tests skip and
 * count those elements.
 * ------------------------------------------------------------------------- */
void tra_oracle_budget(const float* entropy, int64_t n, double tau, int N, int32_t* budget,
                       uint8_t* fragile) {
  for (int64_t i = 0; i < n; ++i) {
    double v = tau * exp((double)entropy[i]);
    double k = ceil(v);
    if (fragile) {
      double scale = v > 1.0 ? v : 1.0;
      fragile[i] = (fabs(v - rint(v)) <= 1e-13 * scale) && (v < (double)N + 1.0);
    }
    if (k < 1.0) k = 1.0;
    if (k > (double)N) k = (double)N;
    budget[i] = (int32_t)k;
  }
}

/* ------------------------------------------------------------------------- *
 * Lognormal entropy-to-budget map (Appendix "Distributional Analysis", entropy-
 * identified Lognormal mapping): sigma = sqrt(2 (log N - H)),
 * B = Phibar(sigma - Phi^{-1}(tau)), K = ceil(N * B) clamped to [1, N].
 * z_tau = Phi^{-1}(tau) is passed in (a constant of the configuration);
 * Phibar(z) = erfc(z / sqrt 2) / 2.  H above log N (rounding) is treated as log N.
 * fragile[i] = 1 when N*B lies within 1e-11 (relative) of an integer.
 * ------------------------------------------------------------------------- */
void tra_oracle_budget_lognormal(const float* entropy, int64_t n, double z_tau, int N,
                                 int32_t* budget, uint8_t* fragile) {
  const double logN = log((double)N);
  for (int64_t i = 0; i < n; ++i) {
    double gap = logN - (double)entropy[i];
    if (gap < 0.0) gap = 0.0;
    double sigma = sqrt(2.0 * gap);
    double B = 0.5 * erfc((sigma - z_tau) / sqrt(2.0));
    double v = (double)N * B;
    double k = ceil(v);
    if (fragile) {
      double scale = v > 1.0 ? v : 1.0;
      fragile[i] = (fabs(v - rint(v)) <= 1e-11 * scale) && (v < (double)N + 1.0);
    }
    if (!(k >= 1.0)) k = 1.0;
    if (k > (double)N) k = (double)N;
    budget[i] = (int32_t)k;
  }
}

/* ------------------------------------------------------------------------- *
 * Radius selection, Eq. 14: the smallest candidate whose grid count reaches
 * the budget.  coord = tile-major coordinates; counts = table above.  The last
 * candidate has count N, so the scan always stops.
 * ------------------------------------------------------------------------- */
void tra_oracle_select_radius(const int32_t* budget, int heads, int N, const int32_t* coord, int H,
                              int W, const uint32_t* counts, int n_radii, uint16_t* ridx) {
  for (int h = 0; h < heads; ++h)
    for (int p = 0; p < N; ++p) {
      int t = coord[3 * p], y = coord[3 * p + 1], x = coord[3 * p + 2];
      const uint32_t* row = counts + ((size_t)(t * H + y) * W + x) * n_radii;
      int k = 0;
      while (k < n_radii - 1 && (int64_t)row[k] < (int64_t)budget[(size_t)h * N + p]) ++k;
      ridx[(size_t)h * N + p] = (uint16_t)k;
    }
}

/* Token-radius mask entry, Eq. 15, in the integer form described above. */
static int token_visible(const int32_t* coord, int qi, int kj, const int32_t* theta, int T,
                         int ridx_q) {
  int dt = coord[3 * qi] - coord[3 * kj];
  if (dt < 0) dt = -dt;
  int dy = coord[3 * qi + 1] - coord[3 * kj + 1];
  int dx = coord[3 * qi + 2] - coord[3 * kj + 2];
  return dy * dy + dx * dx <= theta[ridx_q * T + dt];
}

/* One row of the logical token mask M (Eq. 15) for query position qi. */
void tra_oracle_token_mask_row(const int32_t* coord, int N, int T, const int32_t* theta, int qi,
                               int ridx_q, uint8_t* row) {
  for (int j = 0; j < N; ++j) row[j] = (uint8_t)token_visible(coord, qi, j, theta, T, ridx_q);
}

/* ------------------------------------------------------------------------- *
 * Block vote of Algorithm 1 for one head and a list of query blocks, with no
 * bounding-box shortcut: for every key block v, c_j counts the valid queries
 * of block u whose disk reaches key column j; C = {j : c_j > 0},
 * C_hi = {j : c_j > b/3}; the block is kept when |C| > 0 and
 * 10|C_hi| > 6|C|.  Rows and columns past N do not exist (q < N, k < N).
 * c_j > b/3 is taken between real numbers, i.e. 3*c_j > b.  keep_diagonal != 0
 * forces M[u][u] = 1 (a reading for block rows that would otherwise be empty).
 * ridx_head: [N] candidate index per query position of this head.
 * out: [n_u][NB] bytes.
 * ------------------------------------------------------------------------- */
void tra_oracle_block_vote(const int32_t* coord, int N, int T, int b, const int32_t* theta,
                           const uint16_t* ridx_head, const int32_t* u_list, int n_u,
                           int keep_diagonal, int n_text, uint8_t* out) {
  /* Joint text-video attention (Section 3.2, last paragraph; Algorithm 1): the sequence holds the
   * N video tokens followed by n_text text tokens, S = N + n_text, NB = ceil(S / b) blocks.  With
   * text present the video blocks are the first B_v = floor(N / b) blocks, the ones made of video
   * tokens only; a pair with u >= B_v or v >= B_v is kept (Algorithm 1 leaves non-video blocks
   * dense).  The block that holds the last video tokens and the first text tokens counts as
   * non-video: Section 3.2 keeps every text key visible to every query and lets a text query see
   * every key, which a vote over that block's video tokens could break.  Without text the ragged
   * last block is a video block like any other (q < N, k < N). */
  int NB = (N + n_text + b - 1) / b;
  int NBv = n_text > 0 ? N / b : (N + b - 1) / b;
#pragma omp parallel for schedule(dynamic, 1)
  for (int iu = 0; iu < n_u; ++iu) {
    int u = u_list[iu];
    for (int v = 0; v < NB; ++v) {
      if (u >= NBv || v >= NBv) {
        out[(size_t)iu * NB + v] = 1;
        continue;
      }
      int n_nonempty = 0, n_high = 0;
      for (int j = 0; j < b; ++j) {
        int k = v * b + j;
        if (k >= N) continue;
        int c = 0;
        for (int i = 0; i < b; ++i) {
          int q = u * b + i;
          if (q >= N) continue;
          c += token_visible(coord, q, k, theta, T, ridx_head[q]);
        }
        if (c > 0) ++n_nonempty;
        if (3 * c > b) ++n_high;
      }
      int keep = (n_nonempty > 0) && (10 * n_high > 6 * n_nonempty);
      if (keep_diagonal && u == v) keep = 1;
      out[(size_t)iu * NB + v] = (uint8_t)keep;
    }
  }
}

/* ------------------------------------------------------------------------- *
 * Attention rows, Eq. 1 restricted to a visible key set, with the entropy of
 * Eq. 2 in its two closed forms.
 *   s_j = scale * <q, k_j>;  m = max s;  Z = sum exp(s - m);  p = exp(s-m)/Z;
 *   o = sum p_j v_j;
 *   H_def = -sum p ln p   (0 ln 0 := 0);
 *   H_lse = m + ln Z - sum p s      (the rewrite used by the fused kernel).
 * rows[r] = query position; visible = NULL (all keys) or [n_rows][N] bytes.
 * An empty visible set gives o = 0, H = 0, lse = -inf.
 * Outputs may be NULL.
 * ------------------------------------------------------------------------- */
void tra_oracle_attention_rows(const uint16_t* Q, const uint16_t* K, const uint16_t* V, int N,
                               int d, double scale, const int32_t* rows, int n_rows,
                               const uint8_t* visible, double* O, double* H_def, double* H_lse,
                               double* lse) {
#pragma omp parallel
  {
    double* s = (double*)malloc((size_t)N * sizeof(double));
    double* q = (double*)malloc((size_t)d * sizeof(double));
    double* acc = (double*)malloc((size_t)d * sizeof(double));
#pragma omp for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
      int qi = rows[r];
      const uint8_t* vis = visible ? visible + (size_t)r * N : NULL;
      for (int c = 0; c < d; ++c) q[c] = bf16_widen(Q[(size_t)qi * d + c]);
      double m = -INFINITY;
      int n_vis = 0;
      for (int j = 0; j < N; ++j) {
        if (vis && !vis[j]) continue;
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += q[c] * bf16_widen(K[(size_t)j * d + c]);
        s[j] = dot * scale;
        if (s[j] > m) m = s[j];
        ++n_vis;
      }
      for (int c = 0; c < d; ++c) acc[c] = 0.0;
      double Z = 0.0, ps = 0.0, plogp = 0.0;
      if (n_vis > 0) {
        for (int j = 0; j < N; ++j) {
          if (vis && !vis[j]) continue;
          Z += exp(s[j] - m);
        }
        for (int j = 0; j < N; ++j) {
          if (vis && !vis[j]) continue;
          double p = exp(s[j] - m) / Z;
          ps += p * s[j];
          if (p > 0.0) plogp += p * log(p);
          for (int c = 0; c < d; ++c) acc[c] += p * bf16_widen(V[(size_t)j * d + c]);
        }
      }
      if (O)
        for (int c = 0; c < d; ++c) O[(size_t)r * d + c] = acc[c];
      if (H_def) H_def[r] = n_vis > 0 ? -plogp : 0.0;
      if (H_lse) H_lse[r] = n_vis > 0 ? m + log(Z) - ps : 0.0;
      if (lse) lse[r] = n_vis > 0 ? m + log(Z) : -INFINITY;
    }
    free(s);
    free(q);
    free(acc);
  }
}

/* ------------------------------------------------------------------------- *
 * The online form of Algorithm 2 in fp64, written as a merge of partial
 * softmax states.  A state summarises a set of keys for one query by
 *   ref  a reference score (the largest score of the set),
 *   mass = sum exp(s - ref),   smass = sum exp(s - ref) s,
 *   acc  = sum exp(s - ref) v   (a vector of d values).
 * Two states of disjoint key sets merge by moving both to the larger reference
 * (every sum is multiplied by exp(old ref - new ref)) and adding.  The keys are
 * cut into tiles of `tile` columns, each tile's state is formed on its own and
 * merged into the running one, as the algorithm's block loop does; at the end
 * O = acc / mass and H = log mass + ref - smass / mass.  All keys visible (the
 * dense warm-up pass).  The result does not depend on `tile` beyond rounding.
 * ------------------------------------------------------------------------- */
typedef struct {
  double ref, mass, smass;
  double* acc;
} softmax_state;

static void state_clear(softmax_state* st, int d) {
  st->ref = -INFINITY;
  st->mass = 0.0;
  st->smass = 0.0;
  for (int c = 0; c < d; ++c) st->acc[c] = 0.0;
}

/* into <- into merged with part */
static void state_merge(softmax_state* into, const softmax_state* part, int d) {
  double ref = into->ref > part->ref ? into->ref : part->ref;
  if (ref == -INFINITY) return;                        /* both empty */
  double f_into = exp(into->ref - ref), f_part = exp(part->ref - ref);   /* exp(-inf) = 0 for an empty side */
  into->mass = f_into * into->mass + f_part * part->mass;
  into->smass = f_into * into->smass + f_part * part->smass;
  for (int c = 0; c < d; ++c) into->acc[c] = f_into * into->acc[c] + f_part * part->acc[c];
  into->ref = ref;
}

void tra_oracle_attention_rows_alg2(const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                                    int N, int d, double scale, int tile, const int32_t* rows,
                                    int n_rows, double* O, double* H) {
#pragma omp parallel
  {
    double* q = (double*)malloc((size_t)d * sizeof(double));
    double* s = (double*)malloc((size_t)tile * sizeof(double));
    softmax_state run, part;
    run.acc = (double*)malloc((size_t)d * sizeof(double));
    part.acc = (double*)malloc((size_t)d * sizeof(double));
#pragma omp for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
      int qi = rows[r];
      for (int c = 0; c < d; ++c) q[c] = bf16_widen(Q[(size_t)qi * d + c]);
      state_clear(&run, d);
      for (int j0 = 0; j0 < N; j0 += tile) {
        int w = N - j0 < tile ? N - j0 : tile;
        /* the state of this tile alone */
        state_clear(&part, d);
        for (int j = 0; j < w; ++j) {
          double dot = 0.0;
          for (int c = 0; c < d; ++c) dot += q[c] * bf16_widen(K[(size_t)(j0 + j) * d + c]);
          s[j] = scale * dot;
          if (s[j] > part.ref) part.ref = s[j];
        }
        for (int j = 0; j < w; ++j) {
          double e = exp(s[j] - part.ref);
          part.mass += e;
          part.smass += e * s[j];
          for (int c = 0; c < d; ++c) part.acc[c] += e * bf16_widen(V[(size_t)(j0 + j) * d + c]);
        }
        state_merge(&run, &part, d);
      }
      if (O)
        for (int c = 0; c < d; ++c) O[(size_t)r * d + c] = run.acc[c] / run.mass;
      if (H) H[r] = log(run.mass) + run.ref - run.smass / run.mass;
    }
    free(q);
    free(s);
    free(run.acc);
    free(part.acc);
  }
}

/* ------------------------------------------------------------------------- *
 * Visible key sets of the sparse pass for a list of query positions of one head.
 *   mode 0: what the block-sparse execution computes (Section 3.2 after Eq. 16;
 *           "Limitations": retained blocks are evaluated in full): every valid
 *           key of every retained block of the query's block row;
 *   mode 1: mode 0 intersected with the token mask of Eq. 15;
 *   mode 2: Eq. 16 itself: the token mask alone, blocks ignored.
 * block_rows: [n_rows][NB] bytes, row r = block-mask row of the query block
 * that contains rows[r] (unused in mode 2).
 * ------------------------------------------------------------------------- */
void tra_oracle_visible_rows(const int32_t* coord, int N, int T, int b, const int32_t* theta,
                             const uint16_t* ridx_head, const int32_t* rows, int n_rows,
                             const uint8_t* block_rows, int mode, int n_text, uint8_t* visible) {
  /* With text tokens (positions N .. N + n_text - 1) the token mask applies to the video-key
   * submatrix only: a text key, and any key seen from a text query, counts as inside the disk. */
  int S = N + n_text;
  int NB = (S + b - 1) / b;
  for (int r = 0; r < n_rows; ++r) {
    int qi = rows[r];
    for (int j = 0; j < S; ++j) {
      int in_block = mode == 2 ? 1 : block_rows[(size_t)r * NB + j / b];
      int in_disk = (mode == 0 || qi >= N || j >= N)
                        ? 1
                        : token_visible(coord, qi, j, theta, T, ridx_head[qi]);
      visible[(size_t)r * S + j] = (uint8_t)(in_block && in_disk);
    }
  }
}
