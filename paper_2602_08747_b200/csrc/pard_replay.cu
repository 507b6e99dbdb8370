/* Carrying the queue state from one decision epoch to the next (closed-loop
 * replay): what pard_plan admitted is what the workers run.  Follows the
 * planner's own reading of paper Sec. 4.2 (t_e, the expected end of the
 * previous batch; batches run back to back) and records the queueing-delay
 * sample that pard_update_queue_delay averages.  One thread per (ctx, stage). */
#include "pard_internal.h"

namespace {

struct AdvHeader {
  uint32_t status;                               /* 0, or the positive value of a pard_status */
  uint32_t pad[63];
};
static_assert(sizeof(AdvHeader) == 256, "header is 256 bytes");

__global__ void __launch_bounds__(256)
k_advance_state(const PardPipeDev* const* __restrict__ pipes, uint32_t n_pipelines,
                const int32_t* __restrict__ pipeline_of_ctx, uint32_t n_ctx, uint32_t S,
                const long long* __restrict__ now_us, const int32_t* __restrict__ batch,
                const int32_t* __restrict__ workers, const uint32_t* __restrict__ seg_kept,
                long long* __restrict__ free_at, long long* __restrict__ sample_time,
                int32_t* __restrict__ sample_delay, uint32_t M, uint32_t slot, AdvHeader* __restrict__ hdr) {
  pdl_wait();
  const uint32_t seg = blockIdx.x * blockDim.x + threadIdx.x;
  if (seg >= n_ctx * S) return;
  const uint32_t c = seg / S, k = seg % S;
  const int32_t pi = pipeline_of_ctx ? pipeline_of_ctx[c] : 0;
  if (pi < 0 || (uint32_t)pi >= n_pipelines) {
    atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  const PardPipeDev* p = pipes[pi];
  if (k >= (uint32_t)p->n_stages) return;        /* padding column of the row: left untouched */
  const int32_t B = batch[seg];
  const long long m = workers ? workers[seg] : 1;
  const long long now = now_us[c], fa = free_at[seg];
  if (B < 1 || B > p->bmax[k] || m < 1 || now < 0 || now >= PARD_TIME_LIMIT_US || fa < 0 ||
      fa >= PARD_TIME_LIMIT_US) {
    atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  const long long d = p->lat_us[p->lat_offsets[k] + B - 1];
  const unsigned long long cap = (unsigned long long)B * (unsigned long long)m;
  const long long base = now > fa ? now : fa;                         /* t_e of the next batch */
  if (M) {
    const long long delay = base - now;                               /* queueing delay met at `now` */
    sample_time[(size_t)seg * M + slot] = now;
    sample_delay[(size_t)seg * M + slot] = (int32_t)(delay < PARD_WAIT_LIMIT_US - 1 ? delay : PARD_WAIT_LIMIT_US - 1);
  }
  const unsigned long long rounds = ((unsigned long long)seg_kept[seg] + cap - 1) / cap;   /* < 2^32 */
  const unsigned long long busy = rounds * (unsigned long long)d;     /* < 2^72 only in theory: checked */
  if (__umul64hi(rounds, (unsigned long long)d) != 0 || busy >= (unsigned long long)PARD_TIME_LIMIT_US ||
      (unsigned long long)base + busy >= (unsigned long long)PARD_TIME_LIMIT_US) {
    atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  free_at[seg] = base + (long long)busy;
}

}  // namespace

extern "C" int pard_advance_state_workspace_bytes(uint32_t n_pipelines, uint64_t* bytes) {
  if (!bytes || n_pipelines < 1) return PARD_EINVAL;
  *bytes = sizeof(AdvHeader) + ((8ull * n_pipelines + 255) & ~255ull);
  return PARD_OK;
}

extern "C" int pard_advance_state(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                                  const int32_t* d_pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                                  const int64_t* d_now_us, const int32_t* d_batch, const int32_t* d_workers,
                                  const uint32_t* d_seg_kept, int64_t* d_free_at_us,
                                  int64_t* d_sample_time_us, int32_t* d_sample_delay_us,
                                  uint32_t n_samples, uint32_t slot, uint32_t mode,
                                  void* d_workspace, uint64_t workspace_bytes, void* cuda_stream) {
  if (!pipelines || n_pipelines < 1 || n_ctx < 1 || stage_stride < 1) return PARD_EINVAL;
  if (!d_now_us || !d_batch || !d_seg_kept || !d_free_at_us) return PARD_EINVAL;
  if (n_samples > 0 && (!d_sample_time_us || !d_sample_delay_us || slot >= n_samples)) return PARD_EINVAL;
  if (mode & ~PARD_MODE_NOWAIT) return PARD_EINVAL;
  if (n_pipelines > 1 && !d_pipeline_of_ctx) return PARD_EINVAL;
  if (n_pipelines > 65536 || stage_stride > PARD_MAX_STAGES ||
      (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS || n_samples > PARD_MAX_DELAY_SAMPLES)
    return PARD_ERANGE;
  int dev = -1;
  PARD_CUDA_OK(cudaGetDevice(&dev));
  std::vector<const PardPipeDev*> h_pipes(n_pipelines);
  for (uint32_t i = 0; i < n_pipelines; ++i) {
    const pard_pipeline_t* p = pipelines[i];
    if (!p || !p->d_blob || p->device != dev) return PARD_EINVAL;
    if (p->n_stages > stage_stride) return PARD_EINVAL;
    h_pipes[i] = (const PardPipeDev*)p->d_blob;
  }
  if (!d_workspace || ((uintptr_t)d_workspace & 255)) return PARD_EINVAL;
  uint64_t need = 0;
  pard_advance_state_workspace_bytes(n_pipelines, &need);
  if (workspace_bytes < need) return PARD_EWORKSPACE;

  cudaStream_t stream = (cudaStream_t)cuda_stream;
  AdvHeader* hdr = (AdvHeader*)d_workspace;
  const PardPipeDev** d_pipes = (const PardPipeDev**)((char*)d_workspace + sizeof(AdvHeader));
  PARD_CUDA_OK(cudaMemsetAsync(hdr, 0, sizeof(AdvHeader), stream));
  PARD_CUDA_OK(cudaMemcpyAsync(d_pipes, h_pipes.data(), 8ull * n_pipelines, cudaMemcpyHostToDevice, stream));
  const uint32_t n_seg = n_ctx * (uint32_t)stage_stride;
  PARD_CUDA_OK(launch_pdl(k_advance_state, (n_seg + 255) / 256, 256, 0, stream,
                          (const PardPipeDev* const*)d_pipes, n_pipelines, d_pipeline_of_ctx, n_ctx,
                          (uint32_t)stage_stride, (const long long*)d_now_us, d_batch, d_workers, d_seg_kept,
                          (long long*)d_free_at_us, (long long*)d_sample_time_us, d_sample_delay_us, n_samples,
                          slot, hdr));
  if (mode & PARD_MODE_NOWAIT) return PARD_OK;
  uint32_t h_status = 0;
  PARD_CUDA_OK(cudaMemcpyAsync(&h_status, &hdr->status, 4, cudaMemcpyDeviceToHost, stream));
  PARD_CUDA_OK(cudaStreamSynchronize(stream));
  return h_status ? -(int)h_status : PARD_OK;
}
