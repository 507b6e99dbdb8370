/* Batch-wait estimate w = F^{-1}(lambda) of the State Planner (paper Sec. 4.2,
 * Batch wait estimation): for every (ctx, stage, downstream path) slot, M
 * samples of the batch wait aggregated over the path's stages, and the sample
 * of rank floor(lambda * M).
 *
 * One block per (ctx, slot).  The block writes its M sums into shared memory
 * (every thread draws the recorded waits of its samples with a counter-based
 * generator, so no state is carried between samples), then finds the rank-th
 * smallest by a radix select over the sums: four rounds of 8 bits from the
 * top, each a shared-memory histogram and a scan of 256 bins by one warp. */
#include <mutex>

#include "pard_internal.h"

namespace {

constexpr int kThreads = 512;
constexpr uint32_t kSampleLimit = 1u << 24;      /* recorded waits lie in [0, 2^24) us */

struct WaitHeader {
  uint32_t status;                               /* 0, or the positive value of a pard_status */
  uint32_t pad[63];
};
static_assert(sizeof(WaitHeader) == 256, "header is 256 bytes");

/* splitmix64 (Steele, Lea, Flood 2014): the finaliser applied to counter + gamma */
__device__ __forceinline__ unsigned long long splitmix64(unsigned long long x) {
  unsigned long long z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

/* STAGED: the recorded waits of one stage at a time are copied into shared
 * memory (coalesced) and the draws gather from there, so a slot reads every
 * row of its path once instead of one 32-byte sector per draw.  Needs 8 bytes
 * of shared memory per sample; the direct form needs 4 and gathers from
 * global memory. */
template <bool STAGED>
__global__ void __launch_bounds__(kThreads)
k_estimate_w(const PardPipeDev* const* __restrict__ pipes, uint32_t n_pipelines,
             const int32_t* __restrict__ pipeline_of_ctx, uint32_t S, uint32_t R,
             const int32_t* __restrict__ samples, uint32_t M, uint32_t rank, unsigned long long seed,
             long long* __restrict__ w_out, WaitHeader* __restrict__ hdr) {
  pdl_wait();
  extern __shared__ uint32_t s_sum[];            /* [M] aggregated waits of this slot's samples, then
                                                    (STAGED) [M] recorded waits of the current stage */
  __shared__ uint32_t s_hist[256];
  __shared__ int32_t s_path[PARD_MAX_STAGES];
  __shared__ uint32_t s_prefix, s_rank, s_bad;

  const uint32_t c = blockIdx.x / R, slot = blockIdx.x % R;
  const int32_t pi = pipeline_of_ctx ? pipeline_of_ctx[c] : 0;
  if (pi < 0 || (uint32_t)pi >= n_pipelines) {
    if (threadIdx.x == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  const PardPipeDev* P = pipes[pi];
  if ((uint32_t)P->n_slots > R || (uint32_t)P->n_stages > S) {
    if (threadIdx.x == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }
  if (slot >= (uint32_t)P->n_slots) return;      /* padding of the slot stride: left untouched */
  const int32_t p0 = P->path_off[slot];
  const uint32_t L = (uint32_t)(P->path_off[slot + 1] - p0);
  if (threadIdx.x < L) s_path[threadIdx.x] = P->path_stage[p0 + threadIdx.x];
  if (threadIdx.x == 0) { s_bad = 0; s_prefix = 0; s_rank = rank; }
  __syncthreads();

  /* ---- the M samples: one recorded wait per stage of the path, picked at random ---- */
  const int32_t* ctx_samples = samples + (size_t)c * S * M;
  const unsigned long long slot_counter = ((unsigned long long)c * R + slot) * M;
  uint32_t bad = 0;
  if (STAGED) {
    uint32_t* s_stage = s_sum + M;
    for (uint32_t m = threadIdx.x; m < M; m += kThreads) s_sum[m] = 0;
    for (uint32_t j = 0; j < L; ++j) {
      const int32_t* row = ctx_samples + (size_t)s_path[j] * M;
      for (uint32_t m = threadIdx.x; m < M; m += kThreads) s_stage[m] = (uint32_t)__ldg(&row[m]);
      __syncthreads();
      for (uint32_t m = threadIdx.x; m < M; m += kThreads) {
        const uint32_t hi = (uint32_t)(splitmix64(seed + (slot_counter + m) * 64ull + j) >> 32);
        const uint32_t v = s_stage[__umulhi(hi, M)];
        bad |= v >= kSampleLimit;
        s_sum[m] += v;                           /* < 64 * 2^24 = 2^30 when no value is bad */
      }
      __syncthreads();
    }
  } else {
    for (uint32_t m = threadIdx.x; m < M; m += kThreads) {
      const unsigned long long counter = seed + (slot_counter + m) * 64ull;
      uint32_t sum = 0;
      for (uint32_t j = 0; j < L; ++j) {
        const uint32_t hi = (uint32_t)(splitmix64(counter + j) >> 32);
        const uint32_t v = (uint32_t)__ldg(&ctx_samples[(size_t)s_path[j] * M + __umulhi(hi, M)]);
        bad |= v >= kSampleLimit;
        sum += v;
      }
      s_sum[m] = sum;
    }
  }
  if (bad) s_bad = 1;
  __syncthreads();
  if (s_bad) {
    if (threadIdx.x == 0) atomicMax(&hdr->status, (uint32_t)(-PARD_EDATA));
    return;
  }

  /* ---- radix select: the element of rank s_rank among those that match s_prefix ---- */
#pragma unroll 1
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (threadIdx.x < 256) s_hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t himask = shift == 24 ? 0u : ~0u << (shift + 8);
    for (uint32_t m = threadIdx.x; m < M; m += kThreads) {
      const uint32_t v = s_sum[m];
      if ((v & himask) == prefix) atomicAdd(&s_hist[(v >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x < 32) {                      /* one warp: bin whose running count passes the rank */
      const uint32_t lane = threadIdx.x, want = s_rank;
      uint32_t cnt[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { cnt[i] = s_hist[lane * 8 + i]; tot += cnt[i]; }
      uint32_t incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= (uint32_t)o) incl += t;
      }
      uint32_t before = incl - tot;              /* elements in bins of lower lanes */
      if (want >= before && want < incl) {       /* exactly one lane holds the rank */
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (want >= before && want < before + cnt[i]) {
            s_prefix = prefix | ((uint32_t)(lane * 8 + i) << shift);
            s_rank = want - before;
          }
          before += cnt[i];
        }
      }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) w_out[(size_t)c * R + slot] = (long long)s_prefix;
}

constexpr int kStagedSmemLimit = 112 * 1024;    /* two blocks per multiprocessor */
constexpr uint32_t kDirectMaxSamples = 2048;    /* rows this short stay in the first-level cache */

std::mutex g_attr_mutex;
int g_attr_bytes[2][64];                         /* per form and device: dynamic shared memory already allowed */

int allow_wait_smem(int dev, bool staged, int bytes) {
  if (bytes <= 48 * 1024) return PARD_OK;
  std::lock_guard<std::mutex> lock(g_attr_mutex);
  if (dev >= 0 && dev < 64 && g_attr_bytes[staged][dev] >= bytes) return PARD_OK;
  if (staged)
    PARD_CUDA_OK(cudaFuncSetAttribute(k_estimate_w<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  else
    PARD_CUDA_OK(cudaFuncSetAttribute(k_estimate_w<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  if (dev >= 0 && dev < 64) g_attr_bytes[staged][dev] = bytes;
  return PARD_OK;
}

}  // namespace

extern "C" int pard_estimate_w_workspace_bytes(uint32_t n_pipelines, uint64_t* bytes) {
  if (!bytes || n_pipelines < 1) return PARD_EINVAL;
  *bytes = sizeof(WaitHeader) + ((8ull * n_pipelines + 255) & ~255ull);
  return PARD_OK;
}

extern "C" int pard_estimate_w(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                               const int32_t* d_pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                               int32_t slot_stride, const int32_t* d_wait_samples, uint32_t n_samples,
                               uint32_t lambda_num, uint32_t lambda_den, uint64_t seed, uint32_t mode,
                               int64_t* d_w_us, void* d_workspace, uint64_t workspace_bytes,
                               void* cuda_stream) {
  if (!pipelines || n_pipelines < 1 || !d_wait_samples || !d_w_us || n_ctx < 1) return PARD_EINVAL;
  if (stage_stride < 1 || slot_stride < 1 || lambda_den == 0 || lambda_num > lambda_den) return PARD_EINVAL;
  if (mode & ~PARD_MODE_NOWAIT) return PARD_EINVAL;
  if (n_pipelines > 1 && !d_pipeline_of_ctx) return PARD_EINVAL;
  if (n_pipelines > 65536) return PARD_ERANGE;
  if (stage_stride > PARD_MAX_STAGES || slot_stride > PARD_MAX_PATH_SLOTS ||
      (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS ||
      (uint64_t)n_ctx * (uint64_t)slot_stride >= (1ull << 31) || n_samples < 1 ||
      n_samples > PARD_MAX_WAIT_SAMPLES)
    return PARD_ERANGE;
  int dev = -1;
  PARD_CUDA_OK(cudaGetDevice(&dev));
  std::vector<const PardPipeDev*> h_pipes(n_pipelines);
  for (uint32_t i = 0; i < n_pipelines; ++i) {
    const pard_pipeline_t* p = pipelines[i];
    if (!p || !p->d_blob || p->device != dev) return PARD_EINVAL;
    if (p->n_stages > stage_stride || p->n_slots > slot_stride) return PARD_EINVAL;
    h_pipes[i] = (const PardPipeDev*)p->d_blob;
  }
  if (!d_workspace || ((uintptr_t)d_workspace & 255)) return PARD_EINVAL;
  uint64_t need = 0;
  pard_estimate_w_workspace_bytes(n_pipelines, &need);
  if (workspace_bytes < need) return PARD_EWORKSPACE;

  cudaStream_t stream = (cudaStream_t)cuda_stream;
  WaitHeader* hdr = (WaitHeader*)d_workspace;
  const PardPipeDev** d_pipes = (const PardPipeDev**)((char*)d_workspace + sizeof(WaitHeader));
  const bool staged = n_samples > kDirectMaxSamples && 8ull * n_samples <= (uint64_t)kStagedSmemLimit;
  const int smem = (int)((staged ? 8ull : 4ull) * n_samples);
  int rc = allow_wait_smem(dev, staged, smem);
  if (rc != PARD_OK) return rc;
  PARD_CUDA_OK(cudaMemsetAsync(hdr, 0, sizeof(WaitHeader), stream));
  PARD_CUDA_OK(cudaMemcpyAsync(d_pipes, h_pipes.data(), 8ull * n_pipelines, cudaMemcpyHostToDevice, stream));
  uint64_t rank = (uint64_t)lambda_num * n_samples / lambda_den;
  if (rank > n_samples - 1) rank = n_samples - 1;
  PARD_CUDA_OK(launch_pdl(staged ? k_estimate_w<true> : k_estimate_w<false>, n_ctx * (uint32_t)slot_stride, kThreads, (size_t)smem, stream,
                          (const PardPipeDev* const*)d_pipes, n_pipelines, d_pipeline_of_ctx,
                          (uint32_t)stage_stride, (uint32_t)slot_stride, d_wait_samples, n_samples,
                          (uint32_t)rank, (unsigned long long)seed, (long long*)d_w_us, hdr));
  if (mode & PARD_MODE_NOWAIT) return PARD_OK;
  uint32_t h_status = 0;
  PARD_CUDA_OK(cudaMemcpyAsync(&h_status, &hdr->status, 4, cudaMemcpyDeviceToHost, stream));
  PARD_CUDA_OK(cudaStreamSynchronize(stream));
  return h_status ? -(int)h_status : PARD_OK;
}
