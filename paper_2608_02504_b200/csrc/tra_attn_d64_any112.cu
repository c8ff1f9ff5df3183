// Attention kernels for head_dim 64 and blocks of 97 .. 112 tokens (key tiles of 112 rows).
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_any112(const tra_attn_args& a) { return launch_shape_any<64, 112>(a); }
