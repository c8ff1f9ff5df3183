// Attention kernels for head_dim 64 and blocks of 65 .. 80 tokens (key tiles of 80 rows).
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_any80(const tra_attn_args& a) { return launch_shape_any<64, 80>(a); }
