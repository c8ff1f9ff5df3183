// Attention kernels for head_dim 64 and blocks of 33 .. 48 tokens (key tiles of 48 rows).
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_any48(const tra_attn_args& a) { return launch_shape_any<64, 48>(a); }
