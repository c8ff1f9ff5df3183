// Attention kernels for head_dim 64 and blocks of 113 .. 128 tokens (key tiles of 128 rows).
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_any128(const tra_attn_args& a) { return launch_shape_any<64, 128>(a); }
