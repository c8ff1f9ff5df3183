// Shared declarations of the TRA B200 library (internal; the public ABI is include/tra.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "tra.h"

#define TRA_MAX_SEG 4       // bounding boxes kept per block
#define TRA_MAX_T 1024

// A box around a group of tokens of one block: frame range and spatial extent.
struct tra_box_t {
  int16_t t0, t1, y0, y1, x0, x1, pad0, pad1;
};
static_assert(sizeof(tra_box_t) == 16, "box is one 16-byte load");

struct __align__(16) tra_block_boxes_t {
  tra_box_t box[TRA_MAX_SEG];
  int32_t n_box;
  int32_t pad[3];
};
static_assert(sizeof(tra_block_boxes_t) == 80, "block boxes");

struct tra_plan {
  tra_config_t cfg;
  int N, NB, n_radii;   // N = T*H*W video tokens; NB = blocks of the whole sequence
  int S, NBv;           // S = N + n_text tokens in the sequence; NBv = video blocks (see tra_plan_create)
  int device;
  int sm_count;         // multiprocessors of the device
  double z_tau;       // Phi^-1(tau), for the lognormal budget map
  // host copies
  double* h_radii;
  int32_t* h_theta;   // [n_radii][T]
  int32_t* h_coord;   // [N][3]
  // device tables
  uint32_t* d_coord_packed;       // [N]  x | y << 10 | t << 20   per tile-major position
  uint32_t* d_slice;              // [NB * block / 16, padded to 8]  one word per 16 consecutive positions:
                                  // x0 | y << 10 | t << 20 | 1 << 30 when they are 16 video tokens of
                                  // one frame and one row with x = x0 .. x0 + 15, else 0
  int32_t* d_raster_of_pos;       // [N]
  int32_t* d_slice_raster;        // TRA_ORDER_RASTER: [S / 16 + 32] raster row of every 16 consecutive positions
  int32_t* d_theta;               // [n_radii][T]
  float* d_radii_f32;             // [n_radii]
  uint32_t* d_counts;             // [T*H*W][n_radii]  (raster-indexed)
  uint32_t* d_counts_coarse;      // n_radii <= 128: [T*H*W][16] every eighth entry of a row, then [T*H*W][128] the
                                  // rows padded to 128 entries (sector-aligned groups of eight); else NULL
  tra_block_boxes_t* d_boxes;     // [NB]
  uint16_t* d_field_pos;          // block vote: where frame cell (y, x) sits in the frame's tile-major order (the
                                  // order repeats frame by frame).  field_quads = 0: [H][W] the position of every
                                  // cell; 1: [H][W/4] position / 4 of the cells (y, 4j .. 4j+3), which are four
                                  // consecutive positions starting at a multiple of four, inside one block; 2:
                                  // [H][W/16] position / 16 of the cells (y, 16m .. 16m+15), sixteen consecutive
                                  // positions starting at a multiple of sixteen, inside one block
  int field_quads;
  int* d_status;                  // device status word
  // tra_build_block_mask: the tile-pair kernel runs on a stream of its own beside the list kernels (fork and join
  // events on the caller's stream); created with the plan
  cudaStream_t pair_stream;
  cudaEvent_t pair_fork, pair_join;
  // copy streams and events of tra_hot_path_host, created on its first calls with this plan and kept
  cudaStream_t copy_in, copy_out;
  cudaEvent_t* events;
  int n_events;
};

__host__ __device__ inline uint32_t tra_pack_coord(int t, int y, int x) {
  return (uint32_t)x | ((uint32_t)y << 10) | ((uint32_t)t << 20);
}
__host__ __device__ inline int tra_coord_x(uint32_t c) { return (int)(c & 1023u); }
__host__ __device__ inline int tra_coord_y(uint32_t c) { return (int)((c >> 10) & 1023u); }
__host__ __device__ inline int tra_coord_t(uint32_t c) { return (int)(c >> 20); }

// Words per row of the block vote's count field: at least W + 1 (its difference array writes column
// W), a whole number of 16-byte vectors, and an odd number of them so that threads that walk
// neighbouring rows with 16-byte accesses fall into different shared-memory banks.
__host__ __device__ inline int tra_field_row_words(int W) { return 4 * (((W + 4) / 4) | 1); }

#define TRA_CUDA_CHECK(expr)                      \
  do {                                            \
    cudaError_t _e = (expr);                      \
    if (_e != cudaSuccess) return TRA_ERR_CUDA;   \
  } while (0)

// Query blocks per 128-row query tile of the attention launches, for blocks of more than 32 tokens: a tile holds two
// blocks of up to 64 tokens or one larger block (its first G * b rows are used).
inline int tra_blocks_per_tile(int block) { return block <= 64 ? 2 : 1; }

// Plan time: the coarse table of the two-round radius search (tra_radius.cu).
int tra_build_coarse_table(const uint32_t* counts, uint32_t* coarse, long long cells, int n_radii, int* status,
                           cudaStream_t stream);

// Records the first error code in the plan's device status word.
__device__ inline void tra_set_status(int* status, int code) { atomicCAS(status, 0, code); }

// Bounds-checking build (-DTRA_DEBUG): TRA_IDX(i, n, status) is true when 0 <= i < n; otherwise it
// records TRA_ERR_BOUNDS and the caller skips the access.  In the normal build it is the constant
// true and the guarded access compiles to the plain one.
#ifdef TRA_DEBUG
__device__ inline bool tra_index_ok(long long i, long long n, int* status) {
  if (i >= 0 && i < n) return true;
  tra_set_status(status, TRA_ERR_BOUNDS);
  return false;
}
#define TRA_IDX(i, n, status) tra_index_ok((long long)(i), (long long)(n), (status))
#else
#define TRA_IDX(i, n, status) true
#endif
