// Attention kernels for head_dim 64 and blocks of 49 .. 64 tokens (key tiles of 64 rows).
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_any64(const tra_attn_args& a) { return launch_shape_any<64, 64>(a); }
