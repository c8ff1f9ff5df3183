// Block-mask construction from per-query radii (Algorithm 1) and its CSR active-block list.
#include <algorithm>
#include <mutex>

#include "tra_common.cuh"

#define TRA_MASK_THREADS 128
#define TRA_MASK_WARPS (TRA_MASK_THREADS / 32)

// ---------------------------------------------------------------------------------------
// Vote kernel.  One CTA per (batch*head, query block u); one thread per query of the block.
//
// The vote keeps (u, v) iff some key column is reached (c_j > 0) and more than 60% of the
// reached columns are "high" (3*c_j > b), where c_j counts the queries of u whose disk
// (Eq. 15) holds key j.  Two exact devices keep the work far below the b*b tests per pair of
// the algorithm as printed:
//
// 1. Box pre-classification.  Let need = floor(b/3) + 1 be the smallest high count and r* the
//    need-th largest candidate index among the valid queries of u; thresholds grow with the
//    candidate index and shrink with the frame distance.  With the boxes of the two blocks
//    (groups of tokens, each with a frame range and a spatial box):
//      - if for every box pair even r* at the smallest frame distance cannot bridge the
//        smallest box distance, at most need-1 queries reach anything in v: no high column,
//        vote = 0;
//      - if for every box pair r* at the largest frame distance covers the largest box
//        distance, at least `need` queries reach every key of v: every column is high, vote = 1.
// 2. Count field.  For a key frame f that still holds an undecided key block, the count
//    c(y', x') = #{queries i : (x'-x_i)^2 + (y'-y_i)^2 <= theta[ridx_i][|f - t_i|]} is built for
//    the whole frame at once: a query's disk meets row y' in the x-interval of half-width
//    floor(sqrt(theta - (y'-y_i)^2)), which adds +1 / -1 to a difference array in shared
//    memory (rows y_i - dy and y_i + dy share the half-width; a disk that covers the whole frame
//    is only counted once).  The running sum along a row then gives the counts.  When four
//    cells of a row are four consecutive tile-major positions of one key block (the usual
//    case), the same pass compares the four counts, one per byte of a word, with the two
//    thresholds at once (adding 127 - t to a byte sets its top bit iff the byte exceeds t) and adds
//    the reached and high columns to the counter word of the key block they belong to: two threads
//    per row, one summing from the left end, one from the right.  Otherwise one thread per row
//    stores the counts as bytes in the frame's tile-major order and every undecided key block
//    reads the counts of its own keys back, four per word.  When the query block lies in one
//    frame t0 the frames t0 - k and t0 + k see the same thresholds, so one field serves both.
// The outcome equals the unpruned vote bit for bit.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int tra_isqrt_small(int n) {
  // floor(sqrt(n)) for 0 <= n < 2^22: sqrt(n + 0.5) stays at least 0.25/sqrt(n) away from every
  // integer, far more than the error of the approximate square root
  float r;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"((float)n + 0.5f));
  return (int)r;
}

__device__ __forceinline__ tra_box_t tra_load_box(const tra_box_t* p) {
  union { int4 v; tra_box_t b; } u;
  u.v = __ldg(reinterpret_cast<const int4*>(p));
  return u.b;
}

// kMode = plan->field_quads.  0: the plan's position table has one entry per cell; 1: one entry per four cells of
// a row (see tra_plan::d_field_pos); 2: moreover sixteen cells of a row are sixteen consecutive positions of one block.
// ten resident CTAs per SM: 48 registers per thread without spills (12 CTAs, 40 registers, measured no faster)
#define TRA_VOTE_MIN_CTAS 10
template <int kMode>
__global__ void __launch_bounds__(TRA_MASK_THREADS, TRA_VOTE_MIN_CTAS)
tra_block_vote_kernel(const uint16_t* __restrict__ ridx, const uint32_t* __restrict__ coord_packed,
                      const int32_t* __restrict__ theta, const tra_block_boxes_t* __restrict__ boxes,
                      const uint16_t* __restrict__ field_pos, uint8_t* __restrict__ block_mask,
                      int32_t* __restrict__ row_ptr, int N, int S, int NB, int NBv, int b, int T, int H, int W,
                      int n_radii, int keep_diagonal, int* __restrict__ status) {
  constexpr bool kQuads = kMode != 0;
  extern __shared__ int32_t s_dyn[];
  __shared__ tra_block_boxes_t s_ubox;
  __shared__ int s_rstar, s_count, s_whole[2];

  const int Wp = tra_field_row_words(W);
  const int Tp = (T + 3) & ~3;                                     // keeps s_diff 16-byte aligned
  const int n_diff = H * Wp;                                       // words of the count field
  int32_t* s_theta_star = s_dyn;                                   // [T]
  int32_t* s_frame_ylo = s_dyn + Tp;                               // [T] rows of the frame that hold keys of an
  int32_t* s_frame_yhi = s_dyn + 2 * Tp;                           // [T] undecided key block (yhi < 0: none)
  int32_t* s_diff = s_dyn + 3 * Tp;                                // [H][Wp] (at least 320 words with kQuads)
  const int diff_words = kQuads ? max(n_diff, 320) : n_diff;
  uint32_t* s_cols = (uint32_t*)(s_diff + diff_words);             // [NB] reached columns | high columns << 16 |
                                                                   // state << 30 (0 / 1 decided, 2 undecided)
  const int HW = H * W;
  // entries of the plan's position table: per cell, per four cells, per sixteen cells
  const int n_pos = kMode == 2 ? HW / 16 : (kQuads ? HW / 4 : HW);
  const int cnt_bytes = kQuads ? 0 : max(HW, 1280);
  uint32_t* s_cnt = s_cols + (NB + 3) / 4 * 4;                     // [cnt_bytes] bytes (16-byte aligned), without
                                                                   // kQuads only: counts in tile-major order
  uint16_t* s_pos = (uint16_t*)(s_cnt + (cnt_bytes + 15) / 16 * 4);       // [n_pos] the plan's position table
  // The sort of the queries by candidate index borrows 1280 bytes: of the byte array (it is over before the first
  // counts are written) or, with kQuads, of the count field (which is zeroed after the sort).
  uint32_t* s_scratch = kQuads ? (uint32_t*)s_diff : s_cnt;
  int* s_rank_key = (int*)s_scratch;                               // [128]
  uint32_t* s_sorted = s_scratch + 128;     // [128] queries in descending candidate index: coord, and ...
  uint16_t* s_sorted_r = (uint16_t*)(s_scratch + 256);             // [128] ... their candidate index

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.x;
  const long long bh = blockIdx.y;
  const uint16_t* ridx_h = ridx + bh * S;
  uint8_t* mask_row = block_mask + (bh * NB + u) * (long long)NB;

  // Rows of text blocks (u >= NBv) keep every block: Algorithm 1 leaves non-video blocks dense.
  if (u >= NBv) {
    for (int v = tid; v < NB; v += TRA_MASK_THREADS) mask_row[v] = 1;
    if (tid == 0) row_ptr[bh * NB + u + 1] = NB;
    return;
  }
  const int q0 = u * b;
  const int nq = min(b, N - q0);                       // valid queries of this block
  const int need = b / 3 + 1;

  // this thread's query
  int qx = 0, qy = 0, qt = 0, qr = 0;
  if (tid < nq && TRA_IDX(q0 + tid, N, status)) {
    uint32_t c = coord_packed[q0 + tid];
    qx = tra_coord_x(c);
    qy = tra_coord_y(c);
    qt = tra_coord_t(c);
    qr = min((int)ridx_h[q0 + tid], n_radii - 1);      // a candidate index past the table reads its last row
  }
  // sort key: candidate index, then lane order (unique per query); -1 for the threads without a query
  s_rank_key[tid] = tid < nq ? (qr << 7) | (TRA_MASK_THREADS - 1 - tid) : -1;
  for (int i = tid; i < (n_pos + 7) / 8; i += TRA_MASK_THREADS)
    reinterpret_cast<uint4*>(s_pos)[i] = __ldg(reinterpret_cast<const uint4*>(field_pos) + i);
#ifdef TRA_DEBUG
  if (tid < nq && (qx >= W || qy >= H || qt >= T)) tra_set_status(status, TRA_ERR_BOUNDS);   // indexes the count field
#endif
  if (tid == 0) {
    s_ubox = boxes[u];
    s_count = 0;
    s_rstar = -1;
    s_whole[0] = s_whole[1] = 0;
  }
  for (int i = tid; i < T; i += TRA_MASK_THREADS) {
    s_frame_ylo[i] = H;
    s_frame_yhi[i] = -1;
  }
  __syncthreads();

  // r*: the need-th largest candidate index (ties broken by lane order).  The ranks also re-deal
  // the queries to the threads in descending candidate order, so that the threads of a warp draw
  // disks of similar size (the row loops below run as long as the largest disk of the warp).
  if (tid < nq) {
    const int key = (qr << 7) | (TRA_MASK_THREADS - 1 - tid);
    int rank = 0;
#pragma unroll 4
    for (int j = 0; j < TRA_MASK_THREADS / 4; ++j) {
      const int4 o = reinterpret_cast<const int4*>(s_rank_key)[j];
      rank += (o.x > key) + (o.y > key) + (o.z > key) + (o.w > key);
    }
    if (rank == need - 1) s_rstar = qr;
    if (TRA_IDX(rank, nq, status)) {
      s_sorted[rank] = tra_pack_coord(qt, qy, qx);
      s_sorted_r[rank] = (uint16_t)qr;
    }
  }
  __syncthreads();
  if (tid < nq) {
    const uint32_t c = s_sorted[tid];
    qx = tra_coord_x(c);
    qy = tra_coord_y(c);
    qt = tra_coord_t(c);
    qr = s_sorted_r[tid];
  }
  const int rstar = s_rstar;                            // -1: fewer than `need` valid queries
  if (rstar >= 0)
    for (int i = tid; i < T; i += TRA_MASK_THREADS) s_theta_star[i] = theta[rstar * T + i];
  __syncthreads();

  // ---- 1. classify every key block with the boxes -----------------------------------------
  // (the count field starts all zero; every pass over its rows leaves them zeroed again)
  for (int i = tid; i < n_diff / 4; i += TRA_MASK_THREADS)
    reinterpret_cast<uint4*>(s_diff)[i] = make_uint4(0u, 0u, 0u, 0u);
  int kept = 0;
  for (int v = tid; v < NB; v += TRA_MASK_THREADS) {
    int decided = 0;   // 0 = vote 0, 1 = vote 1, 2 = undecided
    // the boxes of v sit in registers: five independent 16-byte loads, and loops over them that are unrolled in
    // full (a private copy indexed by a loop variable would live in local memory)
    tra_box_t vbox[TRA_MAX_SEG];
    int vb_n = 0;
    if (v >= NBv) {
      decided = 1;     // text key block
    } else if (rstar >= 0) {
#pragma unroll
      for (int iv = 0; iv < TRA_MAX_SEG; ++iv) vbox[iv] = tra_load_box(boxes[v].box + iv);
      vb_n = min(__ldg(&boxes[v].n_box), TRA_MAX_SEG);
      bool all_reject = true, all_accept = true;
      for (int iu = 0; iu < s_ubox.n_box; ++iu) {
        const tra_box_t a = s_ubox.box[iu];
#pragma unroll
        for (int iv = 0; iv < TRA_MAX_SEG; ++iv) {
          if (iv >= vb_n) break;
          const tra_box_t c = vbox[iv];
          int dt_min = max(0, max(a.t0 - c.t1, c.t0 - a.t1));
          int dt_max = max(a.t1 - c.t0, c.t1 - a.t0);
          int gy = max(0, max(a.y0 - c.y1, c.y0 - a.y1));
          int gx = max(0, max(a.x0 - c.x1, c.x0 - a.x1));
          int fy = max(a.y1 - c.y0, c.y1 - a.y0);
          int fx = max(a.x1 - c.x0, c.x1 - a.x0);
          if (!TRA_IDX(dt_max, T, status)) continue;       // dt_min <= dt_max
          if (s_theta_star[dt_min] >= gy * gy + gx * gx) all_reject = false;
          if (s_theta_star[dt_max] < fy * fy + fx * fx) all_accept = false;
        }
        if (!all_reject && !all_accept) break;     // undecided whatever the other boxes say
      }
      decided = all_reject ? 0 : (all_accept ? 1 : 2);
    }
    if (keep_diagonal && v == u) decided = 1;
    s_cols[v] = (uint32_t)decided << 30;
    if (decided == 2) {
      // frames this key block has tokens in, and the rows of each that hold them
#pragma unroll
      for (int iv = 0; iv < TRA_MAX_SEG; ++iv) {
        if (iv >= vb_n) break;
        const tra_box_t c = vbox[iv];
        for (int f = c.t0; f <= c.t1; ++f) {
          if (!TRA_IDX(f, T, status)) break;
          atomicMin(&s_frame_ylo[f], (int)c.y0);
          atomicMax(&s_frame_yhi[f], (int)c.y1);
        }
      }
    } else {
      mask_row[v] = (uint8_t)decided;
      kept += decided;
    }
  }
  if (kept) atomicAdd(&s_count, kept);
  __syncthreads();

  // ---- 2. count field of every frame that holds an undecided key block ---------------------
  // builds the field for the frame distance dist(thread) -> |f - t_i| of every query and returns the
  // number of queries whose disk covers the whole frame (they are left out of the field).
  // Only the rows win_lo .. win_hi of the frame are read afterwards: the field is built for them alone.
  int n_field = 0;
  // Row intervals of every query's disk at the frame distance dist_of_query(), added to the difference array
  // (rows win_lo .. win_hi only).  Ends with a barrier; returns the word that holds the number of queries whose
  // disk covers the whole frame (they are left out of the field).
  auto add_disk_rows = [&](auto dist_of_query, int win_lo, int win_hi) -> int* {
    // The field is all zero here (set at the start, and again by every prefix pass), and no warp still
    // reads it.
    const int th = tid < nq ? __ldg(theta + qr * T + dist_of_query()) : 0;
    int* whole = &s_whole[n_field & 1];     // alternates: the last field's readers may still be at work
    int* whole_next = &s_whole[++n_field & 1];
    if (tid < nq) {
      const int far_x = max(qx, W - 1 - qx), far_y = max(qy, H - 1 - qy);
      if (th >= far_x * far_x + far_y * far_y) {
        atomicAdd(whole, 1);                          // the disk covers the whole frame
      } else {
        // rows qy - dy and qy + dy meet the disk in the same x-interval: one half-width serves both
        // (a half-width that reaches both frame edges clamps to the whole row by itself)
        const int R = tra_isqrt_small(th);
        const int d_first = max(0, max(win_lo - qy, qy - win_hi));
        const int d_last = min(R, max(qy - win_lo, win_hi - qy));
        const unsigned span = (unsigned)(win_hi - win_lo);
#pragma unroll 2
        for (int dy = d_first; dy <= d_last; ++dy) {
          const int w = tra_isqrt_small(th - dy * dy);
          const int lo = max(0, qx - w), hi = min(W - 1, qx + w) + 1;      // lo < hi <= W < Wp
          const int ya = qy - dy, yb = qy + dy;
          if ((unsigned)(ya - win_lo) <= span && TRA_IDX(ya * Wp + hi, H * Wp, status)) {
            atomicAdd(&s_diff[ya * Wp + lo], 1);
            atomicAdd(&s_diff[ya * Wp + hi], -1);
          }
          if (dy > 0 && (unsigned)(yb - win_lo) <= span && TRA_IDX(yb * Wp + hi, H * Wp, status)) {
            atomicAdd(&s_diff[yb * Wp + lo], 1);
            atomicAdd(&s_diff[yb * Wp + hi], -1);
          }
        }
      }
    }
    __syncthreads();
    if (tid == 0) *whole_next = 0;          // its last readers passed the barrier above
    return whole;
  };
  // A count c (without the `whole` queries) is reached iff c > -whole and high iff c > floor(b/3) - whole; with
  // t >= -1 the byte c + (127 - t) <= 255 has its top bit set iff c > t (c <= b - whole, and t = -1 only when
  // whole >= 1): four keys per 32-bit word are compared at once.
  //
  // Position table with one entry per four cells (kQuads): running sums and counting in one pass.  The row's
  // differences sum to zero (every interval closes inside the row, column W included), so the count of a cell is
  // the sum of the differences at and left of it, and also minus the sum of those right of it: the left half of
  // a row is summed from the left by one thread (warps 0 and 1) and the right half from the right by another
  // (warps 2 and 3).  Four cells of a row are four consecutive tile-major positions inside one key block (the
  // block size is a multiple of four); their reached and high columns are added to the block's counter word
  // whenever the block changes along the row.  fa / fb: the frames this field stands for (-1: not needed); the
  // rows are zeroed again for the next field.  Ends with a barrier.
  auto sum_and_count_rows = [&](int win_lo, int win_hi, int fa, int fb, int whole) {
    const uint32_t add_reached = 0x01010101u * (uint32_t)(127 - max(-whole, -1));
    const uint32_t add_high = 0x01010101u * (uint32_t)(127 - max(b / 3 - whole, -1));
    const uint32_t magic = 0xffffffffu / (uint32_t)b + 1u;          // umulhi(p, magic) = p / b for p < 2^32 / b
    const int nQ = W / 4, nL = (nQ + 1) / 2;                        // quads of a row; the left half's share
    const bool right = tid >= TRA_MASK_THREADS / 2;
    const uint32_t base_a = (uint32_t)((fa >= 0 ? fa : fb) * HW), base_b = (uint32_t)((fb >= 0 ? fb : fa) * HW);
    for (int yy = win_lo + (tid & (TRA_MASK_THREADS / 2 - 1)); yy <= win_hi; yy += TRA_MASK_THREADS / 2) {
      uint4* row = reinterpret_cast<uint4*>(s_diff + yy * Wp);
      const uint16_t* pos = s_pos + yy * (kMode == 2 ? W / 16 : nQ);
      uint32_t acc_r = 0, acc_h = 0, cur_a = 0xffffffffu, cur_b = 0xffffffffu;
      auto flush = [&]() {
        const uint32_t acc = acc_r + (acc_h << 16);
        if (acc == 0) return;
        if (fa >= 0 && TRA_IDX(cur_a, NB, status)) atomicAdd(&s_cols[cur_a], acc);
        if (fb >= 0 && TRA_IDX(cur_b, NB, status)) atomicAdd(&s_cols[cur_b], acc);
      };
      // x: the counts of the quad's four cells, one per byte.  Its key block is looked up when it can differ from
      // the previous quad's: for every quad, or (kMode 2) for the first quad met of every group of four.
      auto count_quad = [&](int j, bool may_change, uint32_t x) {
        if (may_change) {
          const uint32_t p4 = kMode == 2 ? 16u * pos[j >> 2] : 4u * pos[j];
          const uint32_t va = __umulhi(base_a + p4, magic), vb = __umulhi(base_b + p4, magic);
          if (va != cur_a || vb != cur_b) {
            flush();
            acc_r = acc_h = 0;
            cur_a = va;
            cur_b = vb;
          }
        }
        acc_r += __popc((x + add_reached) & 0x80808080u);
        acc_h += __popc((x + add_high) & 0x80808080u);
      };
      // The packed counts come from multiplications: with differences d0..d3 and the count `run` left of the quad,
      // run * 0x01010101 + d0 * 0x01010101 + d1 * 0x01010100 + d2 * 0x01010000 + d3 * 0x01000000 holds
      // run + d0 + .. + dk in byte k (every such sum is a count in 0..128, so no byte borrows from its neighbour
      // in the end, whatever the order of the additions modulo 2^32).  From the right: c3 = run, c2 = c3 - d3, ...
      if (!right) {
        uint32_t run = 0;
#pragma unroll 1
        for (int j = 0; j < nL; ++j) {
          const uint4 v = row[j];
          row[j] = make_uint4(0u, 0u, 0u, 0u);
          const uint32_t x = run * 0x01010101u + v.x * 0x01010101u + v.y * 0x01010100u + v.z * 0x01010000u +
                             v.w * 0x01000000u;
          run = x >> 24;
          count_quad(j, kMode != 2 || (j & 3) == 0, x);
        }
      } else {
        uint32_t run = 0u - row[nQ].x;                              // column W: minus the differences right of W - 1
        row[nQ] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
        for (int j = nQ - 1; j >= nL; --j) {
          const uint4 v = row[j];
          row[j] = make_uint4(0u, 0u, 0u, 0u);
          const uint32_t x = run * 0x01010101u - v.w * 0x00010101u - v.z * 0x00000101u - v.y;
          run = (x & 0xffu) - v.x;
          count_quad(j, kMode != 2 || (j & 3) == 3 || j == nQ - 1, x);
        }
      }
      flush();
    }
    __syncthreads();
  };
  // Position table with one entry per cell: running sum along x, one thread per row; the counts (at most
  // b <= 128) go out as bytes in tile-major order, and the row (column W included) is zeroed for the next field.
  // Ends with a barrier.
  auto sum_rows_to_bytes = [&](int win_lo, int win_hi) {
    for (int yy = win_lo + tid; yy <= win_hi; yy += TRA_MASK_THREADS) {
      uint32_t run = 0;
      int32_t* row = s_diff + yy * Wp;
      const uint16_t* pos = s_pos + yy * W;
      for (int x = 0; x < W; ++x) {
        run += (uint32_t)row[x];
        row[x] = 0;
        if (TRA_IDX(pos[x], HW, status)) reinterpret_cast<uint8_t*>(s_cnt)[pos[x]] = (uint8_t)run;
      }
      row[W] = 0;
    }
    __syncthreads();
  };
  // ... after which the undecided key blocks with tokens in frame f read their keys' counts: one warp per block,
  // four keys per lane and word.
  auto count_frame = [&](int f, int whole) {
    const uint32_t add_reached = 0x01010101u * (uint32_t)(127 - max(-whole, -1));
    const uint32_t add_high = 0x01010101u * (uint32_t)(127 - max(b / 3 - whole, -1));
    const int p_begin = f * HW, p_end = min(N, (f + 1) * HW);
    const int v_first = p_begin / b, v_last = (p_end - 1) / b;     // video blocks only: p_end <= N
    for (int v = v_first + warp; v <= v_last; v += TRA_MASK_WARPS) {
      if ((s_cols[v] >> 30) != 2u) continue;
      const int i0 = max(v * b, p_begin) - p_begin, i1 = min((v + 1) * b, p_end) - p_begin;   // bytes [i0, i1)
      int acc = 0;                                        // reached | high << 16 of this lane's keys
      if (((i0 | i1) & 3) == 0 && i1 - i0 == 128) {       // 32 whole words, one per lane (uniform across the warp)
        const uint32_t x = s_cnt[(i0 >> 2) + lane];
        acc = __popc((x + add_reached) & 0x80808080u) + (__popc((x + add_high) & 0x80808080u) << 16);
      } else {
        for (int wd = (i0 >> 2) + lane; 4 * wd < i1; wd += 32) {
          const uint32_t x = s_cnt[wd];
          uint32_t m = 0x80808080u;                       // bytes of the word that belong to [i0, i1)
          if (i0 > 4 * wd) m &= 0xffffffffu << (8 * (i0 - 4 * wd));
          if (i1 < 4 * wd + 4) m &= 0xffffffffu >> (8 * (4 * wd + 4 - i1));
          acc += __popc((x + add_reached) & m) + (__popc((x + add_high) & m) << 16);
        }
      }
      acc = __reduce_add_sync(0xffffffffu, acc);
      if (lane == 0) s_cols[v] += (uint32_t)acc;   // one warp owns v inside a frame; frames are processed in turn
    }
  };
  // the field of one frame distance, counted for the frames fa and fb (-1: not needed)
  auto field = [&](auto dist_of_query, int win_lo, int win_hi, int fa, int fb) {
    const int whole = *add_disk_rows(dist_of_query, win_lo, win_hi);
    if constexpr (kQuads) {
      sum_and_count_rows(win_lo, win_hi, fa, fb, whole);
    } else {
      sum_rows_to_bytes(win_lo, win_hi);
      if (fa >= 0) count_frame(fa, whole);
      if (fb >= 0) count_frame(fb, whole);
    }
  };
  // A query block that lies in one frame t0 sees frames t0 - k and t0 + k at the same distance:
  // their fields are the same, so one field serves both.
  bool one_frame = s_ubox.n_box > 0;
  for (int iu = 0; iu < s_ubox.n_box; ++iu)
    one_frame = one_frame && s_ubox.box[iu].t0 == s_ubox.box[0].t0 && s_ubox.box[iu].t1 == s_ubox.box[0].t0;
  if (one_frame) {
    const int t0 = s_ubox.box[0].t0;
    for (int k = 0; k < T; ++k) {
      const int fa = t0 - k, fb = t0 + k;
      const bool need_a = fa >= 0 && s_frame_yhi[fa] >= 0;
      const bool need_b = k > 0 && fb < T && s_frame_yhi[fb] >= 0;
      if (!need_a && !need_b) continue;                 // uniform across the CTA
      int win_lo = min(need_a ? s_frame_ylo[fa] : H, need_b ? s_frame_ylo[fb] : H);
      int win_hi = max(need_a ? s_frame_yhi[fa] : -1, need_b ? s_frame_yhi[fb] : -1);
      if (!TRA_IDX(win_lo, H, status) || !TRA_IDX(win_hi, H, status)) win_lo = 0, win_hi = H - 1;
      field([&]() { return k; }, win_lo, win_hi, need_a ? fa : -1, need_b ? fb : -1);
    }
  } else {
    for (int f = 0; f < T; ++f) {
      if (s_frame_yhi[f] < 0) continue;                 // uniform across the CTA
      field([&]() { return abs(qt - f); }, s_frame_ylo[f], s_frame_yhi[f], f, -1);
    }
  }

  // ---- 3. votes of the undecided key blocks -------------------------------------------------
  __syncthreads();
  kept = 0;
  for (int v = tid; v < NB; v += TRA_MASK_THREADS) {
    const uint32_t cv = s_cols[v];
    if ((cv >> 30) != 2u) continue;
    const int ne = (int)(cv & 0xffffu), hi = (int)((cv >> 16) & 0x3fffu);
    const int keep = (ne > 0) && (10 * hi > 6 * ne);
    mask_row[v] = (uint8_t)keep;
    kept += keep;
  }
  if (kept) atomicAdd(&s_count, kept);
  __syncthreads();
  if (tid == 0) row_ptr[bh * NB + u + 1] = s_count;   // per-row count; scanned in place afterwards
}

// ---------------------------------------------------------------------------------------
// In-place exclusive scan of the per-row counts held in row_ptr[1..rows] (one CTA).  When the
// total exceeds the capacity of col_idx every offset is clamped to the capacity, so that a
// later attention launch that reads col_idx[row_ptr[r] .. row_ptr[r+1]) stays inside the buffer
// (rows past the capacity come out short or empty; the error is in the plan status).
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
  const long long cap = min(capacity, 0x7fffffffll);
  for (long long i = lo; i < hi; ++i) {
    run += row_ptr[i + 1];
    row_ptr[i + 1] = (int32_t)min(run, cap);
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
                        int32_t* __restrict__ col_idx, long long rows, int NB, long long capacity,
                        int* __restrict__ status) {
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
      if (pos < capacity && TRA_IDX(pos, capacity, status)) col_idx[pos] = v;
    }
    base += __popc(bal);
  }
}

// ---------------------------------------------------------------------------------------
// Tile pairing for the block-sparse attention launch.  That launch gives every CTA two 128-row
// query tiles which walk the union of their key-block lists; a key block only one of the two
// retains leaves the other tile idle.  This kernel pairs tiles with similar lists, per (batch,
// head); tile t covers the query blocks [t G, (t + 1) G), G = 128 / block.
//   1. row bitmaps of a window of tiles are built in shared memory (ballots over the byte mask),
//      and for every tile u the number of key blocks that u and each of its candidates do not
//      share is stored.  The candidates are the next TRA_PAIR_WINDOW tiles and, when a frame holds
//      more tiles than that, the three tiles about one frame ahead (the same place in the next
//      frame: with a slow temporal decay those share far more key blocks than spatial neighbours);
//   2. one warp matches the tiles greedily in ascending order: the first unmatched tile takes the
//      unmatched candidate with the fewest unshared key blocks, or, when none is left, the next
//      unmatched tile after the window.
// Up to four CTAs per (batch, head), as many as fit the device in one wave, take a part of the tiles
// each and match inside it.  Every tile is
// matched (one is left alone when their number is odd): pairs[i] = (u, v) for i < ceil(NT / 2),
// v = -1 for a lone tile.
// Any perfect matching gives the same attention output; the choice only moves time.
// ---------------------------------------------------------------------------------------
#ifndef TRA_PAIR_WINDOW
#define TRA_PAIR_WINDOW 8
#endif
#define TRA_PAIR_CANDS (TRA_PAIR_WINDOW + 3)
#define TRA_PAIR_CHUNK 32
#define TRA_PAIR_THREADS 512
#define TRA_PAIR_LOADS 24          // byte loads of one row a lane keeps in flight

__global__ void __launch_bounds__(TRA_PAIR_THREADS)
tra_pair_tiles_kernel(const uint8_t* __restrict__ block_mask, int32_t* __restrict__ pairs, int NB, int NT, int G,
                      int frame_tiles, int* __restrict__ status) {
  extern __shared__ uint32_t s_pair[];
  const int words = (NB + 31) >> 5;
  // candidate c of tile u is u + 1 + c for c < TRA_PAIR_WINDOW, then u + frame_tiles - 1, + 0, + 1
  const bool far_cands = frame_tiles - 1 > TRA_PAIR_WINDOW;
  const int reach = far_cands ? frame_tiles + 1 : TRA_PAIR_WINDOW;           // largest candidate offset
  auto cand_offset = [&](int c) { return c < TRA_PAIR_WINDOW ? 1 + c : frame_tiles - 1 + (c - TRA_PAIR_WINDOW); };
  const int win_rows = TRA_PAIR_CHUNK + reach;
  uint32_t* s_win = s_pair;                                                  // [win_rows][words]
  uint16_t* s_band = (uint16_t*)(s_win + win_rows * words);                  // [NT][TRA_PAIR_CANDS]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long bh = blockIdx.x;
  const uint8_t* mask_h = block_mask + bh * NB * (long long)NB;
  int32_t* out = pairs + bh * ((NT + 1) / 2) * 2;

  // This CTA's part of the tiles (gridDim.y parts of an even number of tiles, so only the last part
  // can leave a tile alone); candidates stay inside the part.
  const int n_seg = (int)gridDim.y;
  const int seg_len = ((NT + n_seg - 1) / n_seg + 1) & ~1;
  const int seg_begin = (int)blockIdx.y * seg_len, seg_end = min(NT, seg_begin + seg_len);
  if (seg_begin >= seg_end) return;

  // The window is a ring: the bitmap of tile t sits in row t % win_rows.  A chunk needs the tiles
  // chunk0 .. chunk0 + TRA_PAIR_CHUNK - 1 + reach; all but the last TRA_PAIR_CHUNK are there already.
  for (int chunk0 = seg_begin; chunk0 < seg_end; chunk0 += TRA_PAIR_CHUNK) {
    const int t_begin = chunk0 > seg_begin ? chunk0 + reach : seg_begin, t_end = min(seg_end, chunk0 + win_rows);
    __syncthreads();                         // the previous chunk's readers are done with the rows replaced now
    // one warp per tile; the loads of TRA_PAIR_LOADS words of a mask row are in flight together
    for (int t = t_begin + warp; t < t_end; t += TRA_PAIR_THREADS / 32) {
      uint32_t* dst = s_win + (t % win_rows) * words;
      for (int wd0 = 0; wd0 < words; wd0 += TRA_PAIR_LOADS) {
        uint32_t on[TRA_PAIR_LOADS];
#pragma unroll
        for (int q = 0; q < TRA_PAIR_LOADS; ++q) on[q] = 0u;
        for (int g = 0; g < G; ++g) {
          const int u = t * G + g;
          if (u >= NB) break;
          const uint8_t* row = mask_h + (long long)u * NB;
          uint32_t got[TRA_PAIR_LOADS];
#pragma unroll
          for (int q = 0; q < TRA_PAIR_LOADS; ++q)             // independent loads (past the row: its last byte)
            got[q] = __ldg(row + min((wd0 + q) * 32 + lane, NB - 1));
#pragma unroll
          for (int q = 0; q < TRA_PAIR_LOADS; ++q) on[q] |= got[q];
        }
#pragma unroll
        for (int q = 0; q < TRA_PAIR_LOADS; ++q) {
          const uint32_t bits = __ballot_sync(0xffffffffu, on[q] != 0u && (wd0 + q) * 32 + lane < NB);
          if (lane == 0 && wd0 + q < words) dst[wd0 + q] = bits;
        }
      }
    }
    __syncthreads();
    for (int task = tid; task < TRA_PAIR_CHUNK * TRA_PAIR_CANDS; task += TRA_PAIR_THREADS) {
      const int ul = task / TRA_PAIR_CANDS, c = task - ul * TRA_PAIR_CANDS;
      const int u = chunk0 + ul, v = u + cand_offset(c);
      if (u >= seg_end) continue;
      uint32_t d = 0xffffu;
      if (v < seg_end && (c < TRA_PAIR_WINDOW || far_cands)) {
        d = 0;
        const uint32_t* a = s_win + (u % win_rows) * words;
        const uint32_t* b = s_win + (v % win_rows) * words;
        for (int wd = 0; wd < words; ++wd) d += __popc(a[wd] ^ b[wd]);
        d = min(d, 0xfffeu);
      }
      s_band[(u - seg_begin) * TRA_PAIR_CANDS + c] = (uint16_t)d;
    }
  }
  __syncthreads();
  // Greedy matching by one warp.  The "matched" flags of all tiles live in registers: lane l holds the
  // 64 tiles [64 l, 64 l + 64) (NT <= 2048), so a step costs a few shuffles and no shared-memory round trip.
  if (warp != 0) return;
  unsigned long long used = 0ull;
  auto first_free_from = [&](int from) -> int {          // the first unmatched tile in [from, seg_end), or seg_end
    unsigned long long free_bits = ~used;
    const int lo = 64 * lane;
    if (lo + 63 < from) free_bits = 0ull;
    else if (lo < from) free_bits &= ~0ull << (from - lo);
    if (lo >= seg_end) free_bits = 0ull;
    else if (seg_end - lo < 64) free_bits &= (1ull << (seg_end - lo)) - 1ull;
    const uint32_t cand = free_bits ? (uint32_t)(lo + __ffsll((long long)free_bits) - 1) : (uint32_t)seg_end;
    return (int)__reduce_min_sync(0xffffffffu, cand);
  };
  auto mark = [&](int t) {
    if (t >= 0 && lane == (t >> 6)) used |= 1ull << (t & 63);
  };
  int n_out = seg_begin / 2;
  for (int u = first_free_from(seg_begin); u < seg_end; u = first_free_from(u + 1)) {
    const int vo = u + cand_offset(min(lane, TRA_PAIR_CANDS - 1));
    const int vc = min(vo, seg_end - 1);
    const unsigned long long w = __shfl_sync(0xffffffffu, used, vc >> 6);
    uint32_t key = 0xffffffffu;              // (unshared blocks, candidate number) of this lane's candidate
    if (lane < TRA_PAIR_CANDS && vo < seg_end && !((w >> (vc & 63)) & 1ull)) {
      const uint32_t d = s_band[(u - seg_begin) * TRA_PAIR_CANDS + lane];
      if (d != 0xffffu) key = (d << 8) | (uint32_t)lane;
    }
    key = __reduce_min_sync(0xffffffffu, key);
    int v;
    if (key != 0xffffffffu) {
      v = u + cand_offset((int)(key & 0xffu));
    } else {                                 // no candidate left: the next unmatched tile after the window, if any
      mark(u);
      v = first_free_from(u + 1 + TRA_PAIR_WINDOW);
      if (v >= seg_end) v = -1;
    }
    mark(u);
    mark(v);
    if (lane == 0 && TRA_IDX(n_out, (NT + 1) / 2, status) && (v == -1 || TRA_IDX(v, NT, status))) {
      out[2 * n_out] = u;
      out[2 * n_out + 1] = v;
    }
    ++n_out;
  }
}


extern "C" int tra_build_block_mask(const tra_plan_t* plan, const uint16_t* ridx, uint8_t* block_mask,
                                    int32_t* row_ptr, int32_t* col_idx, int64_t col_idx_capacity,
                                    int64_t* nnz_out, int32_t* tile_pairs, int B, int heads, void* stream_) {
  if (!plan || !ridx || !block_mask || !row_ptr || !col_idx || B < 1 || heads < 1 ||
      col_idx_capacity < 0)
    return TRA_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const int NB = plan->NB, T = plan->cfg.T;
  const long long BH = (long long)B * heads;
  if (NB > 65535 || BH > 65535) return TRA_ERR_UNSUPPORTED;
  if (tile_pairs && plan->cfg.block <= 32) return TRA_ERR_UNSUPPORTED;   // no attention launch, no query tiles
  const long long rows = BH * NB;

  const int H = plan->cfg.H, W = plan->cfg.W;
  // thresholds and frame windows, count field, counter words, byte array (without quads), position table:
  // the layout at the top of the kernel
  const int mode = plan->field_quads;
  const size_t n_diff = (size_t)H * tra_field_row_words(W);
  const size_t n_pos = (size_t)H * W / (mode == 2 ? 16 : (mode ? 4 : 1));
  size_t smem = ((size_t)3 * ((T + 3) & ~3) + (mode ? std::max<size_t>(n_diff, 320) : n_diff)) * sizeof(int32_t) +
                ((size_t)NB + 3) / 4 * 16 + (mode ? 0 : (std::max<size_t>((size_t)H * W, 1280) + 15) / 16 * 16) +
                ((n_pos + 7) & ~(size_t)7) * sizeof(uint16_t);
  if (smem > 200 * 1024 || !plan->d_field_pos) return TRA_ERR_UNSUPPORTED;   // frame too large for the count field
  // tile pairing (checked before anything is launched)
  int G = 1, NT = 0, frame_tiles = 0;
  size_t pair_smem = 0;
  if (tile_pairs) {
    // query tiles of the attention launch: G blocks each
    const int b = plan->cfg.block;
    G = tra_blocks_per_tile(b);
    NT = (NB + G - 1) / G;
    // tiles per frame, rounded: the tile one frame ahead of u is u + frame_tiles or a neighbour of it
    const long long tile_tokens = (long long)b * G;
    frame_tiles = (int)(((long long)plan->cfg.H * plan->cfg.W + tile_tokens / 2) / tile_tokens);
    const int reach = frame_tiles - 1 > TRA_PAIR_WINDOW ? frame_tiles + 1 : TRA_PAIR_WINDOW;
    pair_smem = ((size_t)(TRA_PAIR_CHUNK + reach) * ((NB + 31) / 32)) * 4 + (size_t)NT * TRA_PAIR_CANDS * 2;
    if (pair_smem > 200 * 1024 || NT > 2048) return TRA_ERR_UNSUPPORTED;
    if (pair_smem > 48 * 1024)
      TRA_CUDA_CHECK(cudaFuncSetAttribute(tra_pair_tiles_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)pair_smem));
  }
  dim3 grid((unsigned)NB, (unsigned)BH);
  auto vote = plan->field_quads == 2 ? tra_block_vote_kernel<2>
                                     : (plan->field_quads ? tra_block_vote_kernel<1> : tra_block_vote_kernel<0>);
  if (smem > 48 * 1024)
    TRA_CUDA_CHECK(cudaFuncSetAttribute(vote, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  vote<<<grid, TRA_MASK_THREADS, smem, stream>>>(
      ridx, plan->d_coord_packed, plan->d_theta, plan->d_boxes, plan->d_field_pos, block_mask, row_ptr, plan->N,
      plan->S, NB, plan->NBv, plan->cfg.block, T, H, W, plan->n_radii, (plan->cfg.flags & TRA_KEEP_DIAGONAL) ? 1 : 0,
      plan->d_status);
  TRA_CUDA_CHECK(cudaGetLastError());
  // The tile pairs need the Boolean mask only, the list kernels too: the pairing runs beside them on the plan's
  // own stream, forked from and joined to the caller's stream by events (legal inside a stream capture as well).
  if (tile_pairs) {
    const unsigned n_seg = (unsigned)std::max(1ll, std::min(4ll, (long long)plan->sm_count / BH));   // one CTA per SM
    TRA_CUDA_CHECK(cudaEventRecord(plan->pair_fork, stream));
    TRA_CUDA_CHECK(cudaStreamWaitEvent(plan->pair_stream, plan->pair_fork, 0));
    tra_pair_tiles_kernel<<<dim3((unsigned)BH, n_seg), TRA_PAIR_THREADS, pair_smem, plan->pair_stream>>>(
        block_mask, tile_pairs, NB, NT, G, frame_tiles, plan->d_status);
    TRA_CUDA_CHECK(cudaGetLastError());
    TRA_CUDA_CHECK(cudaEventRecord(plan->pair_join, plan->pair_stream));
  }
  tra_row_ptr_scan_kernel<<<1, 1024, 0, stream>>>(row_ptr, rows, (long long)col_idx_capacity, nnz_out,
                                                  plan->d_status);
  TRA_CUDA_CHECK(cudaGetLastError());
  tra_col_idx_fill_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, stream>>>(
      block_mask, row_ptr, col_idx, rows, NB, (long long)col_idx_capacity, plan->d_status);
  TRA_CUDA_CHECK(cudaGetLastError());
  if (tile_pairs) TRA_CUDA_CHECK(cudaStreamWaitEvent(stream, plan->pair_join, 0));
  return TRA_OK;
}


// ---------------------------------------------------------------------------------------
// Active-block list without any allocation.  A caller that only feeds tra_sparse_attn needs
// row_ptr / col_idx (and the tile pairs); the Boolean mask between the vote and the list is then
// scratch.  Here that scratch is a fixed array in the library's device image, so the call works
// for code that may not allocate: a plugin running inside another framework's memory pool, a
// serving loop whose device memory is fully committed at start-up, a real-time thread that must
// not enter the allocator's lock.
//
// In host code `tra_static_block_mask` is only a handle of the symbol, not a device address; the
// address a kernel can use comes from cudaGetSymbolAddress, asked once per device with that device
// current, and is kept in g_static_mask_addr.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) uint8_t tra_static_block_mask[TRA_STATIC_BLOCK_MASK_BYTES];

#define TRA_STATIC_MAX_DEVICES 64
static uint8_t* g_static_mask_addr[TRA_STATIC_MAX_DEVICES];   // NULL until the device's first call
static std::mutex g_static_mask_lock;

extern "C" int tra_build_block_list_static(const tra_plan_t* plan, const uint16_t* ridx, int32_t* row_ptr,
                                           int32_t* col_idx, int64_t col_idx_capacity, int64_t* nnz_out,
                                           int32_t* tile_pairs, int B, int heads, void* stream) {
  if (!plan || !ridx || !row_ptr || !col_idx || B < 1 || heads < 1 || col_idx_capacity < 0)
    return TRA_ERR_INVALID_ARG;
  int dev = -1;
  TRA_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev != plan->device || dev < 0 || dev >= TRA_STATIC_MAX_DEVICES) return TRA_ERR_INVALID_ARG;
  // the Boolean mask of this call must fit the fixed array
  const long long need = (long long)B * heads * plan->NB * (long long)plan->NB;
  if (need > (long long)TRA_STATIC_BLOCK_MASK_BYTES) return TRA_ERR_CAPACITY;
  uint8_t* mask = nullptr;
  {
    std::lock_guard<std::mutex> guard(g_static_mask_lock);
    if (!g_static_mask_addr[dev]) {
      void* addr = nullptr;
      if (cudaGetSymbolAddress(&addr, tra_static_block_mask) != cudaSuccess || !addr) {
        cudaGetLastError();
        return TRA_ERR_CUDA;
      }
      g_static_mask_addr[dev] = (uint8_t*)addr;
    }
    mask = g_static_mask_addr[dev];
  }
  // The vote writes every entry of the mask rows it owns, so nothing has to be cleared first.
  return tra_build_block_mask(plan, ridx, mask, row_ptr, col_idx, col_idx_capacity, nnz_out, tile_pairs, B, heads,
                              stream);
}
