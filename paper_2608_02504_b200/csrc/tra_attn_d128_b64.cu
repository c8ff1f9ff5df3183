// Attention kernels for head_dim 128, block 64.
#include "tra_attn_kernel.cuh"

int tra_attn_launch_d128_b64(const tra_attn_args& a) { return launch_shape<128, 64>(a); }
