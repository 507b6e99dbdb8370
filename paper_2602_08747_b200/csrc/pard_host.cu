/* pard_plan_host: the planner with host-resident inputs and outputs.  Copies
 * go through the caller's device workspace; the planning itself is pard_plan. */
#include <algorithm>

#include "pard_internal.h"

namespace {

struct HostLayout {
  uint64_t plan, req, pipeline_of_ctx, now, batch, free_at, q, w, workers, priority;
  uint64_t keep, est, perm, kept_idx, n_kept, seg_off, seg_kept, total;
  uint64_t plan_bytes;
};

int make_host_layout(uint64_t n, uint32_t n_ctx, int32_t S, int32_t R, HostLayout* L) {
  uint64_t plan_bytes = 0;
  int rc = pard_plan_workspace_bytes(n, n_ctx, S, &plan_bytes);
  if (rc != PARD_OK) return rc;
  if (R < 0) return PARD_EINVAL;
  auto al = [](uint64_t x) { return (x + 255) & ~(uint64_t)255; };
  const uint64_t segs = (uint64_t)n_ctx * S;
  uint64_t o = 0;
  L->plan_bytes = plan_bytes;
  L->plan = o;            o = al(o + plan_bytes);
  L->req = o;             o = al(o + 16 * n);
  L->pipeline_of_ctx = o; o = al(o + 4ull * n_ctx);
  L->now = o;             o = al(o + 8ull * n_ctx);
  L->batch = o;           o = al(o + 4 * segs);
  L->free_at = o;         o = al(o + 8 * segs);
  L->q = o;               o = al(o + 8 * segs);
  L->w = o;               o = al(o + 8ull * n_ctx * (uint64_t)R);
  L->workers = o;         o = al(o + 4 * segs);
  L->priority = o;        o = al(o + segs);
  L->keep = o;            o = al(o + n);
  L->est = o;             o = al(o + 8 * n);
  L->perm = o;            o = al(o + 4 * n);
  L->kept_idx = o;        o = al(o + 4 * n);
  L->n_kept = o;          o = al(o + 8);
  L->seg_off = o;         o = al(o + 4 * (segs + 1));
  L->seg_kept = o;        o = al(o + 4 * segs);
  L->total = o;
  return PARD_OK;
}

}  // namespace

extern "C" int pard_plan_host_workspace_bytes(uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                                              int32_t slot_stride, uint64_t* bytes) {
  if (!bytes) return PARD_EINVAL;
  HostLayout L;
  int rc = make_host_layout(n, n_ctx, stage_stride, slot_stride, &L);
  if (rc != PARD_OK) return rc;
  *bytes = L.total;
  return PARD_OK;
}

extern "C" int pard_plan_host(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                              const pard_request_t* requests, uint64_t n,
                              const pard_queue_state_t* st, uint32_t n_ctx, uint32_t mode,
                              const pard_plan_out_t* out, void* d_workspace,
                              uint64_t workspace_bytes, void* cuda_stream) {
  if (!st || !out || n_ctx < 1) return PARD_EINVAL;
  if (!st->d_now_us || !st->d_batch || !st->d_free_at_us || !st->d_q_us) return PARD_EINVAL;
  if (n > 0 && !requests) return PARD_EINVAL;
  if (!d_workspace || ((uintptr_t)d_workspace & 255)) return PARD_EINVAL;
  const int32_t R = st->d_w_us ? st->slot_stride : 0;
  HostLayout L;
  int rc = make_host_layout(n, n_ctx, st->stage_stride, R, &L);
  if (rc != PARD_OK) return rc;
  if (workspace_bytes < L.total) return PARD_EWORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* ws = (char*)d_workspace;
  const uint64_t segs = (uint64_t)n_ctx * st->stage_stride;

  auto up = [&](uint64_t off, const void* src, uint64_t bytes) -> const void* {
    if (!src) return nullptr;
    if (bytes && cudaMemcpyAsync(ws + off, src, bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
      return (const void*)-1;
    return ws + off;
  };
  pard_queue_state_t d = *st;
  const void* p;
  bool fail = false;
  p = up(L.req, requests, 16 * n);                       fail |= p == (const void*)-1;
  const pard_request_t* d_req = (const pard_request_t*)p;
  p = up(L.pipeline_of_ctx, st->d_pipeline_of_ctx, 4ull * n_ctx); fail |= p == (const void*)-1;
  d.d_pipeline_of_ctx = (const int32_t*)p;
  p = up(L.now, st->d_now_us, 8ull * n_ctx);             fail |= p == (const void*)-1;
  d.d_now_us = (const int64_t*)p;
  p = up(L.batch, st->d_batch, 4 * segs);                fail |= p == (const void*)-1;
  d.d_batch = (const int32_t*)p;
  p = up(L.free_at, st->d_free_at_us, 8 * segs);         fail |= p == (const void*)-1;
  d.d_free_at_us = (const int64_t*)p;
  p = up(L.q, st->d_q_us, 8 * segs);                     fail |= p == (const void*)-1;
  d.d_q_us = (const int64_t*)p;
  p = up(L.w, st->d_w_us, 8ull * n_ctx * (uint64_t)R);   fail |= p == (const void*)-1;
  d.d_w_us = (const int64_t*)p;
  p = up(L.workers, st->d_workers, 4 * segs);            fail |= p == (const void*)-1;
  d.d_workers = (const int32_t*)p;
  p = up(L.priority, st->d_priority, segs);              fail |= p == (const void*)-1;
  d.d_priority = (const uint8_t*)p;
  if (fail) return PARD_ECUDA;

  pard_plan_out_t dout;
  dout.d_keep = out->d_keep ? (uint8_t*)(ws + L.keep) : nullptr;
  dout.d_est_us = out->d_est_us ? (int64_t*)(ws + L.est) : nullptr;
  dout.d_perm = out->d_perm ? (uint32_t*)(ws + L.perm) : nullptr;
  dout.d_kept_idx = out->d_kept_idx ? (uint32_t*)(ws + L.kept_idx) : nullptr;
  dout.d_n_kept = (out->d_n_kept || out->d_kept_idx) ? (uint64_t*)(ws + L.n_kept) : nullptr;
  dout.d_seg_offsets = out->d_seg_offsets ? (uint32_t*)(ws + L.seg_off) : nullptr;
  dout.d_seg_kept = out->d_seg_kept ? (uint32_t*)(ws + L.seg_kept) : nullptr;

  /* this call drains the stream anyway, so the status is always read here: PARD_MODE_NOWAIT would
   * only hide a device-detected error behind the downloads */
  rc = pard_plan(pipelines, n_pipelines, d_req, n, &d, n_ctx, mode & ~PARD_MODE_NOWAIT, &dout, ws + L.plan,
                 L.plan_bytes, cuda_stream);
  if (rc != PARD_OK) return rc;

  auto down = [&](void* dst, uint64_t off, uint64_t bytes) {
    if (dst && bytes) return cudaMemcpyAsync(dst, ws + off, bytes, cudaMemcpyDeviceToHost, stream);
    return cudaSuccess;
  };
  uint64_t n_kept = 0;
  if (dout.d_n_kept) {
    PARD_CUDA_OK(cudaMemcpyAsync(&n_kept, ws + L.n_kept, 8, cudaMemcpyDeviceToHost, stream));
    PARD_CUDA_OK(cudaStreamSynchronize(stream));
    if (out->d_n_kept) *out->d_n_kept = n_kept;
  }
  PARD_CUDA_OK(down(out->d_keep, L.keep, n));
  PARD_CUDA_OK(down(out->d_est_us, L.est, 8 * n));
  PARD_CUDA_OK(down(out->d_perm, L.perm, 4 * n));
  PARD_CUDA_OK(down(out->d_kept_idx, L.kept_idx, 4 * n_kept));   /* only the filled part */
  PARD_CUDA_OK(down(out->d_seg_offsets, L.seg_off, 4 * (segs + 1)));
  PARD_CUDA_OK(down(out->d_seg_kept, L.seg_kept, 4 * segs));
  PARD_CUDA_OK(cudaStreamSynchronize(stream));
  return PARD_OK;
}
