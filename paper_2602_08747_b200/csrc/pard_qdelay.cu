/* Recent average queueing delay q_k of the State Planner (paper Sec. 4.2: a
 * sliding window over the monitored queueing delays, by default a 5 s linear
 * weighted one).
 *
 * One warp per (ctx, stage) row.  The lanes read the row's samples coalesced
 * (16 bytes of timestamps and 8 bytes of delays per lane and step), weigh each
 * by window - age, and the two sums are reduced by shuffles.  With the window
 * and the delays below 2^24 us and at most 2^15 samples the weighted sum stays
 * below 2^63, so one 64-bit division finishes the row. */
#include "pard_internal.h"

namespace {

struct QdHeader {
  uint32_t status;                               /* 0, or the positive value of a pard_status */
  uint32_t pad[63];
};
static_assert(sizeof(QdHeader) == 256, "header is 256 bytes");

__global__ void __launch_bounds__(256)
k_queue_delay(uint32_t n_rows, uint32_t S, const long long* __restrict__ now_us,
              const long long* __restrict__ sample_time, const int32_t* __restrict__ sample_delay,
              uint32_t M, uint32_t window_us, long long* __restrict__ q_us, QdHeader* __restrict__ hdr) {
  pdl_wait();
  const uint32_t row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t lane = threadIdx.x & 31;
  if (row >= n_rows) return;                     /* whole warps leave together */
  const long long now = now_us[row / S];
  const long long* t = sample_time + (size_t)row * M;
  const int32_t* d = sample_delay + (size_t)row * M;
  unsigned long long weighted = 0, weights = 0;
  bool bad = false;
  auto add = [&](long long tj, int32_t dj) {
    if (tj < 0) return;                          /* empty slot */
    bad |= (uint32_t)dj >= (uint32_t)PARD_WAIT_LIMIT_US;
    const long long age = now - tj;
    if (age < 0 || age >= (long long)window_us) return;
    const unsigned long long w = (unsigned long long)window_us - (unsigned long long)age;
    weighted += w * (unsigned long long)(uint32_t)dj;
    weights += w;
  };
  /* rows start on 16-byte boundaries when M is even: two samples per lane and step */
  if ((M & 1u) == 0 && (((uintptr_t)sample_time | (uintptr_t)sample_delay) & 15) == 0) {
    for (uint32_t j = 2 * lane; j < M; j += 64) {
      const longlong2 tt = __ldg(reinterpret_cast<const longlong2*>(t + j));
      const int2 dd = __ldg(reinterpret_cast<const int2*>(d + j));
      add(tt.x, dd.x);
      add(tt.y, dd.y);
    }
  } else {
    for (uint32_t j = lane; j < M; j += 32) add(__ldg(t + j), __ldg(d + j));
  }
  for (int o = 16; o; o >>= 1) {
    weighted += __shfl_xor_sync(0xffffffffu, weighted, o);
    weights += __shfl_xor_sync(0xffffffffu, weights, o);
  }
  if (__any_sync(0xffffffffu, bad)) {
    if (lane == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  if (lane == 0) q_us[row] = weights ? (long long)(weighted / weights) : 0;
}

}  // namespace

extern "C" int pard_update_queue_delay_workspace_bytes(uint64_t* bytes) {
  if (!bytes) return PARD_EINVAL;
  *bytes = sizeof(QdHeader);
  return PARD_OK;
}

extern "C" int pard_update_queue_delay(uint32_t n_ctx, int32_t stage_stride, const int64_t* d_now_us,
                                       const int64_t* d_sample_time_us, const int32_t* d_sample_delay_us,
                                       uint32_t n_samples, uint32_t window_us, uint32_t mode,
                                       int64_t* d_q_us, void* d_workspace, uint64_t workspace_bytes,
                                       void* cuda_stream) {
  if (n_ctx < 1 || stage_stride < 1 || !d_now_us || !d_q_us || window_us < 1) return PARD_EINVAL;
  if (n_samples > 0 && (!d_sample_time_us || !d_sample_delay_us)) return PARD_EINVAL;
  if (mode & ~PARD_MODE_NOWAIT) return PARD_EINVAL;
  if (stage_stride > PARD_MAX_STAGES || (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS ||
      n_samples > PARD_MAX_DELAY_SAMPLES || window_us > PARD_MAX_DELAY_WINDOW_US)
    return PARD_ERANGE;
  if (((uintptr_t)d_sample_time_us & 7) || ((uintptr_t)d_sample_delay_us & 3)) return PARD_EINVAL;
  if (!d_workspace || ((uintptr_t)d_workspace & 255)) return PARD_EINVAL;
  if (workspace_bytes < sizeof(QdHeader)) return PARD_EWORKSPACE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  QdHeader* hdr = (QdHeader*)d_workspace;
  PARD_CUDA_OK(cudaMemsetAsync(hdr, 0, sizeof(QdHeader), stream));
  const uint32_t n_rows = n_ctx * (uint32_t)stage_stride;
  PARD_CUDA_OK(launch_pdl(k_queue_delay, (n_rows + 7) / 8, 256, 0, stream, n_rows, (uint32_t)stage_stride,
                          (const long long*)d_now_us, (const long long*)d_sample_time_us, d_sample_delay_us,
                          n_samples, window_us, (long long*)d_q_us, hdr));
  if (mode & PARD_MODE_NOWAIT) return PARD_OK;
  uint32_t h_status = 0;
  PARD_CUDA_OK(cudaMemcpyAsync(&h_status, &hdr->status, 4, cudaMemcpyDeviceToHost, stream));
  PARD_CUDA_OK(cudaStreamSynchronize(stream));
  return h_status ? -(int)h_status : PARD_OK;
}
