// Attention kernels for head_dim 64, block 64.
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d64_b64(const tra_attn_args& a) { return launch_shape<64, 64>(a); }
