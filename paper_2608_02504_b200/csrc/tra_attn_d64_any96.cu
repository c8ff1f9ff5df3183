// Attention kernels for head_dim 64 and blocks of 81 .. 96 tokens (key tiles of 96 rows).
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_any96(const tra_attn_args& a) { return launch_shape_any<64, 96>(a); }
