// Entry points of the attention calls: argument checks, shape dispatch, and the self-test of the
// bounded device-side wait.  The kernels live in tra_attn_kernel.cuh, one translation unit per shape.
#include "tra_attn_kernel.cuh"

namespace {

int attn_dispatch(const tra_plan_t* plan, const void* Q, const void* K, const void* V, void* O,
                  float* entropy, float* lse, const int32_t* row_ptr, const int32_t* col_idx,
                  const uint16_t* ridx, const int32_t* tile_pairs, int B, int heads, float sm_scale,
                  void* stream_) {
  if (!plan || !Q || !K || !V || !O || B < 1 || heads < 1) return TRA_ERR_INVALID_ARG;
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 127) return TRA_ERR_INVALID_ARG;
  if (!(sm_scale > 0.f)) return TRA_ERR_INVALID_ARG;
  const long long BH = (long long)B * heads;
  if (BH > 65535 || plan->NB > 32 * kMaxBitmapWords) return TRA_ERR_UNSUPPORTED;
  if (entropy != nullptr && (row_ptr != nullptr || ridx != nullptr)) return TRA_ERR_INVALID_ARG;
  const tra_attn_args a = {plan, Q,   K,          V,  O,        entropy,
                           lse,  row_ptr, col_idx, ridx, tile_pairs, BH, sm_scale, (cudaStream_t)stream_};
  const int d = plan->cfg.head_dim, b = plan->cfg.block;
  if (d == 128 && b == 128) return tra_attn_launch_d128_b128(a);
  if (d == 64 && b == 64) return tra_attn_launch_d64_b64(a);
  if (d == 64 && b == 128) return tra_attn_launch_d64_b128(a);
  if (d == 128 && b == 64) return tra_attn_launch_d128_b64(a);
  if (b > 32 && b <= 128) {      // any other block size: key tiles of ceil(b / 16) * 16 rows
    const int w = (b + 15) / 16;
    if (d == 128)
      return w == 3 ? tra_attn_launch_d128_any48(a) : w == 4 ? tra_attn_launch_d128_any64(a)
           : w == 5 ? tra_attn_launch_d128_any80(a) : w == 6 ? tra_attn_launch_d128_any96(a)
           : w == 7 ? tra_attn_launch_d128_any112(a) : tra_attn_launch_d128_any128(a);
    if (d == 64)
      return w == 3 ? tra_attn_launch_d64_any48(a) : w == 4 ? tra_attn_launch_d64_any64(a)
           : w == 5 ? tra_attn_launch_d64_any80(a) : w == 6 ? tra_attn_launch_d64_any96(a)
           : w == 7 ? tra_attn_launch_d64_any112(a) : tra_attn_launch_d64_any128(a);
  }
  return TRA_ERR_UNSUPPORTED;
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing ever arrives on.
__global__ void tra_wait_timeout_selftest_kernel(unsigned long long limit_ns, int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) mbar_wait_slow(smem_u32(&bar), 0u, &abort_flag, status, limit_ns);
}

}  // namespace

extern "C" int tra_selftest_wait_timeout(tra_plan_t* plan, int limit_ms, void* stream) {
  if (!plan || limit_ms < 1 || limit_ms > 1000) return TRA_ERR_INVALID_ARG;
  tra_wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(
      (unsigned long long)limit_ms * 1000000ull, plan->d_status);
  TRA_CUDA_CHECK(cudaGetLastError());
  return TRA_OK;
}

extern "C" int tra_entropy_attn(const tra_plan_t* plan, const void* Q, const void* K, const void* V,
                                void* O, float* entropy, float* lse, int B, int heads, float sm_scale,
                                void* stream) {
  return attn_dispatch(plan, Q, K, V, O, entropy, lse, nullptr, nullptr, nullptr, nullptr, B, heads, sm_scale,
                       stream);
}

extern "C" int tra_sparse_attn(const tra_plan_t* plan, const void* Q, const void* K, const void* V,
                               const int32_t* row_ptr, const int32_t* col_idx, const uint16_t* ridx,
                               const int32_t* tile_pairs, void* O, float* lse, int B, int heads, float sm_scale,
                               void* stream) {
  // a block list, or (with ridx) none at all: Eq. 16 itself
  if ((row_ptr == nullptr) != (col_idx == nullptr) || (!row_ptr && !ridx)) return TRA_ERR_INVALID_ARG;
  return attn_dispatch(plan, Q, K, V, O, nullptr, lse, row_ptr, col_idx, ridx, tile_pairs, B, heads, sm_scale,
                       stream);
}
