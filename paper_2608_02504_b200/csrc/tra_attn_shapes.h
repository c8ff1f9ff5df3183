// Arguments of one attention launch and the per-shape launchers (one translation unit per
// (head_dim, block) shape, so that the shapes compile in parallel).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "tra.h"

struct tra_attn_args {
  const tra_plan_t* plan;
  const void *Q, *K, *V;
  void* O;
  float* entropy;            // non-NULL: dense launch with the fused entropy
  float* lse;                // optional
  const int32_t* row_ptr;    // block list (NULL: dense, or list-free with ridx)
  const int32_t* col_idx;
  const uint16_t* ridx;      // non-NULL: token mask inside the blocks
  const int32_t* tile_pairs; // optional: which two query tiles share a CTA (block-sparse launches)
  long long BH;
  float sm_scale;
  cudaStream_t stream;
};

int tra_attn_launch_d128_b128(const tra_attn_args& a);
int tra_attn_launch_d64_b64(const tra_attn_args& a);
int tra_attn_launch_d64_b128(const tra_attn_args& a);
int tra_attn_launch_d128_b64(const tra_attn_args& a);
// blocks of 33 .. 128 tokens other than 64 and 128: by head_dim and key-tile width (the block size rounded up to
// a multiple of 16)
int tra_attn_launch_d128_any48(const tra_attn_args& a);
int tra_attn_launch_d128_any64(const tra_attn_args& a);
int tra_attn_launch_d128_any80(const tra_attn_args& a);
int tra_attn_launch_d128_any96(const tra_attn_args& a);
int tra_attn_launch_d128_any112(const tra_attn_args& a);
int tra_attn_launch_d128_any128(const tra_attn_args& a);
int tra_attn_launch_d64_any48(const tra_attn_args& a);
int tra_attn_launch_d64_any64(const tra_attn_args& a);
int tra_attn_launch_d64_any80(const tra_attn_args& a);
int tra_attn_launch_d64_any96(const tra_attn_args& a);
int tra_attn_launch_d64_any112(const tra_attn_args& a);
int tra_attn_launch_d64_any128(const tra_attn_args& a);
