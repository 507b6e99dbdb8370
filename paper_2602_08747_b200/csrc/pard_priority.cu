/* Adaptive request priority with delayed transition (paper Sec. 4.3): per
 * (ctx, stage) queue, the load factor mu = T_in / T_m against the band
 * [1 - eps, 1 + eps], eps = sum |T_in - T_s| / sum T_in with T_s the input
 * workload smoothed by a sliding-window average.
 *
 * One warp per queue.  The lanes walk the queue's workload samples 256 at a
 * time, eight consecutive ones per lane; the window sum of sample j is the difference of two running prefix
 * sums, one over the samples and one over the samples that have left the
 * window (the same row read `window` places back), so the work is linear in
 * the history length for any window.  All quantities are integers; the two
 * threshold tests are done cross-multiplied in 128 bits. */
#include "pard_internal.h"

namespace {

struct PrioHeader {
  uint32_t status;                               /* 0, or the positive value of a pard_status */
  uint32_t pad[63];
};
static_assert(sizeof(PrioHeader) == 256, "header is 256 bytes");

struct U128 {
  unsigned long long hi, lo;
};
__device__ __forceinline__ U128 mul128(unsigned long long a, unsigned long long b) {
  U128 r;
  r.lo = a * b;
  r.hi = __umul64hi(a, b);
  return r;
}
__device__ __forceinline__ bool less128(U128 a, U128 b) { return a.hi < b.hi || (a.hi == b.hi && a.lo < b.lo); }

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(256)
k_update_priority(const PardPipeDev* const* __restrict__ pipes, uint32_t n_pipelines,
                  const int32_t* __restrict__ pipeline_of_ctx, uint32_t n_ctx, uint32_t S,
                  const int32_t* __restrict__ batch, const int32_t* __restrict__ workers,
                  const uint32_t* __restrict__ arrivals, uint32_t H, uint32_t W, uint32_t interval_us,
                  uint8_t* __restrict__ priority, PrioHeader* __restrict__ hdr) {
  pdl_wait();
  const uint32_t seg = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t lane = threadIdx.x & 31;
  if (seg >= n_ctx * S) return;                  /* whole warps leave together */
  const uint32_t c = seg / S, k = seg % S;
  const int32_t pi = pipeline_of_ctx ? pipeline_of_ctx[c] : 0;
  if (pi < 0 || (uint32_t)pi >= n_pipelines) {
    if (lane == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  const PardPipeDev* p = pipes[pi];
  if (k >= (uint32_t)p->n_stages) return;        /* padding column of the row: left untouched */
  const int32_t B = batch[seg];
  const long long m = workers ? workers[seg] : 1;
  if (B < 1 || B > p->bmax[k] || m < 1 || (long long)B * m >= (1ll << 31)) {
    if (lane == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  const unsigned long long d = (unsigned long long)p->lat_us[p->lat_offsets[k] + B - 1];
  const unsigned long long cap = (unsigned long long)B * (unsigned long long)m;   /* T_m = cap / d */

  /* sums over the samples j >= W - 1:  sum_x = sum x_j,  dev = sum |W * x_j - (x_{j-W+1} + ... + x_j)|.
   * A lane owns kRun consecutive samples of every chunk of 32 * kRun: running sums inside the
   * lane, one warp scan of the lanes' totals per chunk. */
  constexpr uint32_t kRun = 8;
  const uint32_t* x = arrivals + (size_t)seg * H;
  const bool vec = (((uintptr_t)x) & 15) == 0;                         /* 16-byte loads of the own samples */
  unsigned long long carry_in = 0, carry_out = 0, sum_x = 0, dev = 0;
  bool bad = false;
  for (uint32_t j0 = 0; j0 < H; j0 += 32 * kRun) {
    const uint32_t jl = j0 + lane * kRun;                              /* first sample of this lane */
    uint32_t xin[kRun], xout[kRun];
    if (vec && jl + kRun <= H) {
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(x + jl));
      const uint4 b = __ldg(reinterpret_cast<const uint4*>(x + jl + 4));
      xin[0] = a.x; xin[1] = a.y; xin[2] = a.z; xin[3] = a.w;
      xin[4] = b.x; xin[5] = b.y; xin[6] = b.z; xin[7] = b.w;
    } else {
#pragma unroll
      for (uint32_t i = 0; i < kRun; ++i) xin[i] = jl + i < H ? __ldg(&x[jl + i]) : 0u;
    }
    unsigned long long tin = 0, tout = 0;
#pragma unroll
    for (uint32_t i = 0; i < kRun; ++i) {
      const uint32_t j = jl + i;
      xout[i] = (j >= W && j < H) ? __ldg(&x[j - W]) : 0u;             /* the sample that left the window */
      bad |= xin[i] >= PARD_RATE_LIMIT;
      tin += xin[i];
      tout += xout[i];
    }
    unsigned long long pin = tin, pout = tout;                         /* inclusive over the lanes' totals */
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long a = __shfl_up_sync(0xffffffffu, pin, o);
      const unsigned long long b = __shfl_up_sync(0xffffffffu, pout, o);
      if (lane >= (uint32_t)o) { pin += a; pout += b; }
    }
    unsigned long long run_in = carry_in + pin - tin, run_out = carry_out + pout - tout;   /* before this lane */
#pragma unroll
    for (uint32_t i = 0; i < kRun; ++i) {
      const uint32_t j = jl + i;
      run_in += xin[i];
      run_out += xout[i];
      if (j + 1 >= W && j < H) {
        const unsigned long long win = run_in - run_out, wx = (unsigned long long)W * xin[i];
        dev += wx > win ? wx - win : win - wx;
        sum_x += xin[i];
      }
    }
    carry_in += __shfl_sync(0xffffffffu, pin, 31);
    carry_out += __shfl_sync(0xffffffffu, pout, 31);
  }
  if (__any_sync(0xffffffffu, bad)) {
    if (lane == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  sum_x = warp_sum(sum_x);
  dev = warp_sum(dev);
  if (lane != 0) return;
  if (sum_x == 0) {                              /* nothing arrived: within capacity */
    priority[seg] = 0;
    return;
  }
  /* mu = x_now * d / (cap * interval);  eps = dev / (W * sum_x)
   * mu > 1 + eps  <=>  x_now * d * (W * sum_x) > cap * interval * (W * sum_x + dev)
   * mu < 1 - eps  <=>  x_now * d * (W * sum_x) < cap * interval * (W * sum_x - dev)
   * ranges: x_now < 2^24, d < 2^40, W * sum_x and dev < 2^48, cap and interval < 2^31 */
  const unsigned long long x_now = __ldg(&x[H - 1]);
  const unsigned long long ws = (unsigned long long)W * sum_x;
  const U128 lhs = mul128(x_now * d, ws);
  const unsigned long long scale = cap * (unsigned long long)interval_us;
  if (less128(mul128(scale, ws + dev), lhs)) priority[seg] = 1;
  else if (ws > dev && less128(lhs, mul128(scale, ws - dev))) priority[seg] = 0;
}

}  // namespace

extern "C" int pard_update_priority_workspace_bytes(uint32_t n_pipelines, uint64_t* bytes) {
  if (!bytes || n_pipelines < 1) return PARD_EINVAL;
  *bytes = sizeof(PrioHeader) + ((8ull * n_pipelines + 255) & ~255ull);
  return PARD_OK;
}

extern "C" int pard_update_priority(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                                    const int32_t* d_pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                                    const int32_t* d_batch, const int32_t* d_workers,
                                    const uint32_t* d_arrivals, uint32_t n_hist, uint32_t window,
                                    uint32_t interval_us, uint32_t mode, uint8_t* d_priority,
                                    void* d_workspace, uint64_t workspace_bytes, void* cuda_stream) {
  if (!pipelines || n_pipelines < 1 || !d_batch || !d_arrivals || !d_priority || n_ctx < 1) return PARD_EINVAL;
  if (stage_stride < 1 || window < 1 || window > n_hist || interval_us < 1) return PARD_EINVAL;
  if (mode & ~PARD_MODE_NOWAIT) return PARD_EINVAL;
  if (n_pipelines > 1 && !d_pipeline_of_ctx) return PARD_EINVAL;
  if (n_pipelines > 65536 || stage_stride > PARD_MAX_STAGES ||
      (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS || n_hist > PARD_MAX_HISTORY ||
      interval_us >= (1u << 31))
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
  pard_update_priority_workspace_bytes(n_pipelines, &need);
  if (workspace_bytes < need) return PARD_EWORKSPACE;

  cudaStream_t stream = (cudaStream_t)cuda_stream;
  PrioHeader* hdr = (PrioHeader*)d_workspace;
  const PardPipeDev** d_pipes = (const PardPipeDev**)((char*)d_workspace + sizeof(PrioHeader));
  PARD_CUDA_OK(cudaMemsetAsync(hdr, 0, sizeof(PrioHeader), stream));
  PARD_CUDA_OK(cudaMemcpyAsync(d_pipes, h_pipes.data(), 8ull * n_pipelines, cudaMemcpyHostToDevice, stream));
  const uint32_t n_seg = n_ctx * (uint32_t)stage_stride;
  PARD_CUDA_OK(launch_pdl(k_update_priority, (n_seg + 7) / 8, 256, 0, stream,
                          (const PardPipeDev* const*)d_pipes, n_pipelines, d_pipeline_of_ctx, n_ctx,
                          (uint32_t)stage_stride, d_batch, d_workers, d_arrivals, n_hist, window, interval_us,
                          d_priority, hdr));
  if (mode & PARD_MODE_NOWAIT) return PARD_OK;
  uint32_t h_status = 0;
  PARD_CUDA_OK(cudaMemcpyAsync(&h_status, &hdr->status, 4, cudaMemcpyDeviceToHost, stream));
  PARD_CUDA_OK(cudaStreamSynchronize(stream));
  return h_status ? -(int)h_status : PARD_OK;
}
