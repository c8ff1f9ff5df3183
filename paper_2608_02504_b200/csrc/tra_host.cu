// One pass of the whole hot path over tensors in host memory, in groups of heads whose copies
// overlap the kernels of the neighbouring groups.  Heads are independent problems (Algorithm 1
// runs per head, Algorithm 2 per query row), so the pass can be cut anywhere between heads.
// Only copies, events and calls of the library's own entry points live here.
#include <stdlib.h>

#include <algorithm>
#include <vector>

#include "tra_common.cuh"

namespace {

constexpr size_t kAlign = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) & ~(kAlign - 1); }

// Device buffers of one pass, carved from the caller's workspace.
struct HostPassLayout {
  size_t stage_in[2][3], stage_out[2], qkv[3], o_dense, o_sparse, entropy, ridx, mask, row_ptr, col_idx, nnz, pairs;
  size_t total;
};

HostPassLayout make_layout(const tra_plan_t* plan, int group) {
  const size_t g = (size_t)group, S = (size_t)plan->S, d = (size_t)plan->cfg.head_dim, NB = (size_t)plan->NB;
  const size_t tensor = align_up(g * S * d * 2);
  HostPassLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += align_up(bytes);
    return at;
  };
  for (int b = 0; b < 2; ++b)
    for (int i = 0; i < 3; ++i) L.stage_in[b][i] = take(tensor);
  for (int b = 0; b < 2; ++b) L.stage_out[b] = take(tensor);
  for (int i = 0; i < 3; ++i) L.qkv[i] = take(tensor);
  L.o_dense = take(tensor);
  L.o_sparse = take(tensor);
  L.entropy = take(g * S * 4);
  L.ridx = take(g * S * 2);
  L.mask = take(g * NB * NB);
  L.row_ptr = take((g * NB + 1) * 4);
  L.col_idx = take(g * NB * NB * 4);
  L.nnz = take(8);
  const size_t G = (size_t)tra_blocks_per_tile(plan->cfg.block), NT = (NB + G - 1) / G;    // query tiles
  L.pairs = take(g * ((NT + 1) / 2) * 2 * 4);
  L.total = off;
  return L;
}

// Events of one call, drawn from a pool the plan keeps (created on first use, reused by later
// calls: recording an event again does not disturb waits that were enqueued on its earlier record).
struct EventPool {
  tra_plan_t* plan;
  int next = 0;
  cudaEvent_t make() {
    if (next == plan->n_events) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      cudaEvent_t* grown = (cudaEvent_t*)realloc(plan->events, sizeof(cudaEvent_t) * (plan->n_events + 1));
      if (!grown) {
        cudaEventDestroy(e);
        return nullptr;
      }
      plan->events = grown;
      plan->events[plan->n_events++] = e;
    }
    return plan->events[next++];
  }
};

}  // namespace

extern "C" size_t tra_hot_path_host_workspace_bytes(const tra_plan_t* plan, int group) {
  if (!plan || group < 1) return 0;
  return make_layout(plan, group).total;
}

extern "C" int tra_hot_path_host(tra_plan_t* plan, const void* Q_host, const void* K_host, const void* V_host,
                                 void* O_host, void* workspace, size_t workspace_bytes, int heads, int group,
                                 int first_group, float sm_scale, void* stream_) {
  if (!plan || !Q_host || !K_host || !V_host || !O_host || !workspace || heads < 1 || group < 1 ||
      first_group < 1 || !(sm_scale > 0.f))
    return TRA_ERR_INVALID_ARG;
  if ((uintptr_t)workspace & (kAlign - 1)) return TRA_ERR_INVALID_ARG;
  if (group > heads) group = heads;
  if (first_group > group) first_group = group;
  const HostPassLayout L = make_layout(plan, group);
  if (workspace_bytes < L.total) return TRA_ERR_CAPACITY;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return TRA_ERR_CUDA;
  if (device != plan->device) return TRA_ERR_INVALID_ARG;     // the plan's tables and streams live on its device
  cudaStream_t cs = (cudaStream_t)stream_;
  if (!plan->copy_in) {   // the two copy streams live as long as the plan
    cudaStream_t in = nullptr, out = nullptr;
    TRA_CUDA_CHECK(cudaStreamCreateWithFlags(&in, cudaStreamNonBlocking));
    if (cudaStreamCreateWithFlags(&out, cudaStreamNonBlocking) != cudaSuccess) {
      cudaStreamDestroy(in);
      return TRA_ERR_CUDA;
    }
    plan->copy_in = in;
    plan->copy_out = out;
  }
  cudaStream_t s_in = plan->copy_in, s_out = plan->copy_out;
  uint8_t* ws = (uint8_t*)workspace;
  const size_t S = (size_t)plan->S, d = (size_t)plan->cfg.head_dim, NB = (size_t)plan->NB;
  const size_t head_bytes = S * d * 2;
  const int row_bytes = (int)(d * 2);
  const void* host_in[3] = {Q_host, K_host, V_host};
  EventPool pool{plan};

  // the copy streams start after whatever the caller queued on its stream
  cudaEvent_t start = pool.make();
  if (!start) return TRA_ERR_CUDA;
  TRA_CUDA_CHECK(cudaEventRecord(start, cs));
  TRA_CUDA_CHECK(cudaStreamWaitEvent(s_in, start, 0));
  TRA_CUDA_CHECK(cudaStreamWaitEvent(s_out, start, 0));

  cudaEvent_t in_free[2] = {nullptr, nullptr};    // the gathers that read staging buffer b are done
  cudaEvent_t out_free[2] = {nullptr, nullptr};   // the copy out of output buffer b is done
  // group sizes: a small first group (the kernels start early), doubling up to `group` (a group's
  // kernels cover the copy of the next, twice as large), and a small last one (little output left to
  // copy after the last kernel)
  std::vector<int> sizes;
  for (int left = heads, ramp = first_group; left > 0; ramp = std::min(2 * ramp, group)) {
    int n = std::min(ramp, left);
    if (left - n == 0 && n > first_group && !sizes.empty()) n -= first_group;   // split the last group
    sizes.push_back(n);
    left -= n;
  }
  int h0 = 0;
  for (int i = 0; i < (int)sizes.size(); ++i) {
    const int n = sizes[i];
    const int b = i & 1;
    // inputs of this group: host -> staging buffer b
    if (in_free[b]) TRA_CUDA_CHECK(cudaStreamWaitEvent(s_in, in_free[b], 0));
    for (int t = 0; t < 3; ++t)
      TRA_CUDA_CHECK(cudaMemcpyAsync(ws + L.stage_in[b][t], (const uint8_t*)host_in[t] + (size_t)h0 * head_bytes,
                                     (size_t)n * head_bytes, cudaMemcpyHostToDevice, s_in));
    cudaEvent_t ready = pool.make();
    if (!ready) return TRA_ERR_CUDA;
    TRA_CUDA_CHECK(cudaEventRecord(ready, s_in));
    TRA_CUDA_CHECK(cudaStreamWaitEvent(cs, ready, 0));
    // the pass itself; a raster-order plan reads the staging buffers in place and writes O into the output
    // staging buffer, so the gather and scatter kernels drop out
    // (with TRA_ORDER_RASTER_QO that holds for Q and O; K and V are still gathered)
    const bool raster_kv = (plan->cfg.flags & TRA_ORDER_RASTER) != 0;
    const bool raster = raster_kv || (plan->cfg.flags & TRA_ORDER_RASTER_QO) != 0;      // Q and O
    int rc;
    for (int t = raster ? 1 : 0; t < 3 && !raster_kv; ++t)
      if ((rc = tra_tile_major_gather(plan, ws + L.stage_in[b][t], ws + L.qkv[t], n, row_bytes, cs)) != TRA_OK)
        return rc;
    if (!raster) {
      if (!(in_free[b] = pool.make())) return TRA_ERR_CUDA;
      TRA_CUDA_CHECK(cudaEventRecord(in_free[b], cs));
    }
    const void *Q = ws + (raster ? L.stage_in[b][0] : L.qkv[0]), *K = ws + (raster_kv ? L.stage_in[b][1] : L.qkv[1]),
               *V = ws + (raster_kv ? L.stage_in[b][2] : L.qkv[2]);
    if ((rc = tra_entropy_attn(plan, Q, K, V, ws + L.o_dense, (float*)(ws + L.entropy), nullptr, 1, n, sm_scale,
                               cs)) != TRA_OK)
      return rc;
    if ((rc = tra_budget_radius(plan, (const float*)(ws + L.entropy), nullptr, nullptr, (uint16_t*)(ws + L.ridx), 1,
                                n, cs)) != TRA_OK)
      return rc;
    if ((rc = tra_build_block_mask(plan, (const uint16_t*)(ws + L.ridx), ws + L.mask, (int32_t*)(ws + L.row_ptr),
                                   (int32_t*)(ws + L.col_idx), (int64_t)((size_t)n * NB * NB),
                                   (int64_t*)(ws + L.nnz), (int32_t*)(ws + L.pairs), 1, n, cs)) != TRA_OK)
      return rc;
    if (raster && out_free[b]) TRA_CUDA_CHECK(cudaStreamWaitEvent(cs, out_free[b], 0));
    if ((rc = tra_sparse_attn(plan, Q, K, V, (const int32_t*)(ws + L.row_ptr), (const int32_t*)(ws + L.col_idx),
                              nullptr, (const int32_t*)(ws + L.pairs), ws + (raster ? L.stage_out[b] : L.o_sparse),
                              nullptr, 1, n, sm_scale, cs)) != TRA_OK)
      return rc;
    if (raster) {                       // the last reader of the input staging buffer
      if (!(in_free[b] = pool.make())) return TRA_ERR_CUDA;
      TRA_CUDA_CHECK(cudaEventRecord(in_free[b], cs));
    } else {
      if (out_free[b]) TRA_CUDA_CHECK(cudaStreamWaitEvent(cs, out_free[b], 0));
      if ((rc = tra_tile_major_scatter(plan, ws + L.o_sparse, ws + L.stage_out[b], n, row_bytes, cs)) != TRA_OK)
        return rc;
    }
    cudaEvent_t done = pool.make();
    if (!done) return TRA_ERR_CUDA;
    TRA_CUDA_CHECK(cudaEventRecord(done, cs));
    // output of this group: staging buffer b -> host
    TRA_CUDA_CHECK(cudaStreamWaitEvent(s_out, done, 0));
    TRA_CUDA_CHECK(cudaMemcpyAsync((uint8_t*)O_host + (size_t)h0 * head_bytes, ws + L.stage_out[b],
                                   (size_t)n * head_bytes, cudaMemcpyDeviceToHost, s_out));
    if (!(out_free[b] = pool.make())) return TRA_ERR_CUDA;
    TRA_CUDA_CHECK(cudaEventRecord(out_free[b], s_out));
    h0 += n;
  }
  // the caller's stream ends after the last copy in either direction
  cudaEvent_t end_in = pool.make(), end_out = pool.make();
  if (!end_in || !end_out) return TRA_ERR_CUDA;
  TRA_CUDA_CHECK(cudaEventRecord(end_in, s_in));
  TRA_CUDA_CHECK(cudaEventRecord(end_out, s_out));
  TRA_CUDA_CHECK(cudaStreamWaitEvent(cs, end_in, 0));
  TRA_CUDA_CHECK(cudaStreamWaitEvent(cs, end_out, 0));
  return TRA_OK;
}
