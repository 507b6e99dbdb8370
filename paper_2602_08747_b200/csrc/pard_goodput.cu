/* Goodput counters (paper Sec. 5.1, Metrics): per ctx, queued requests and
 * requests predicted to finish within their SLO. */
#include "pard_internal.h"

namespace {

constexpr int kThreads = 256;

/* start of ctx c in service order */
__device__ __forceinline__ uint32_t ctx_start(const uint32_t* __restrict__ seg_off, uint32_t c, uint32_t S) {
  return __ldg(&seg_off[(size_t)c * S]);
}

__global__ void k_goodput_init(const uint32_t* __restrict__ seg_off, uint32_t n_ctx, uint32_t S,
                               long long* __restrict__ out_total, long long* __restrict__ out_kept) {
  pdl_wait();
  uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_ctx) return;
  out_total[c] = (long long)seg_off[(size_t)(c + 1) * S] - (long long)seg_off[(size_t)c * S];
  out_kept[c] = 0;
}

/* last ctx whose start is <= o (empty ctxs share a start; the last one owns the byte) */
__device__ __forceinline__ uint32_t ctx_of(const uint32_t* __restrict__ seg_off, uint32_t n_ctx, uint32_t S,
                                           uint64_t o) {
  uint32_t lo = 0, hi = n_ctx;                   /* start(lo) <= o; start(hi) > o or hi == n_ctx */
  while (hi - lo > 1) {
    const uint32_t mid = lo + (hi - lo) / 2;
    if (ctx_start(seg_off, mid, S) <= o) lo = mid; else hi = mid;
  }
  return lo;
}

/* A block counts the keep flags of kChunk consecutive requests, read as
 * 16-byte vectors.  If the chunk lies inside one ctx (the usual case) the
 * block reduces its count and issues one atomic; otherwise every thread finds
 * the ctx of its own 16 flags and counts per ctx. */
constexpr uint32_t kVecs = 4;                                  /* vectors per thread */
constexpr uint32_t kChunk = kThreads * kVecs * 16;             /* flags per block    */

__global__ void __launch_bounds__(kThreads)
k_goodput_count(const uint8_t* __restrict__ keep, const uint32_t* __restrict__ seg_off, uint32_t n,
                uint32_t n_ctx, uint32_t S, unsigned long long* __restrict__ out_kept) {
  pdl_wait();
  constexpr int WARPS = kThreads / 32;
  __shared__ uint32_t s_sum[WARPS];
  __shared__ uint32_t s_ctx0, s_end0;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint64_t c0 = (uint64_t)blockIdx.x * kChunk;
  const uint64_t c1 = c0 + kChunk < n ? c0 + kChunk : n;
  if (threadIdx.x == 0) {
    const uint32_t c = ctx_of(seg_off, n_ctx, S, c0);
    s_ctx0 = c;
    s_end0 = ctx_start(seg_off, c + 1, S);
  }
  __syncthreads();
  if (s_end0 >= c1) {
    /* one ctx: plain block reduction */
    uint32_t sum = 0;
#pragma unroll
    for (uint32_t k = 0; k < kVecs; ++k) {
      const uint64_t o = c0 + ((uint64_t)k * kThreads + threadIdx.x) * 16;
      if (o + 16 <= c1) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(keep + o));
        sum += __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
      } else {
        for (uint64_t b = o; b < c1; ++b) sum += keep[b] & 1u;
      }
    }
    for (int k = 16; k; k >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, k);
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t tot = 0;
      for (int w = 0; w < WARPS; ++w) tot += s_sum[w];
      if (tot) atomicAdd(&out_kept[s_ctx0], (unsigned long long)tot);
    }
    return;
  }
  /* ctx boundaries inside the chunk */
  constexpr uint32_t kNone = 0xffffffffu;
  for (uint32_t k = 0; k < kVecs; ++k) {
    const uint64_t o = c0 + ((uint64_t)k * kThreads + threadIdx.x) * 16;
    uint32_t c = kNone, run = 0;
    if (o < c1) {
      c = ctx_of(seg_off, n_ctx, S, o);
      uint32_t cend = ctx_start(seg_off, c + 1, S);
      if (o + 16 <= c1 && o + 16 <= cend) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(keep + o));
        run = __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
      } else {
        for (uint32_t b = 0; b < 16 && o + b < c1; ++b) {
          while (o + b >= cend) {
            if (run) atomicAdd(&out_kept[c], (unsigned long long)run);
            run = 0;
            ++c;
            cend = ctx_start(seg_off, c + 1, S);
          }
          run += keep[o + b] & 1u;
        }
      }
    }
    /* a warp whose 32 vectors end in one ctx adds once */
    const uint32_t w0 = __shfl_sync(0xffffffffu, c, 0);
    if (__all_sync(0xffffffffu, c == w0)) {
      for (int q = 16; q; q >>= 1) run += __shfl_xor_sync(0xffffffffu, run, q);
      if (lane == 0 && w0 != kNone && run) atomicAdd(&out_kept[w0], (unsigned long long)run);
    } else if (c != kNone && run) {
      atomicAdd(&out_kept[c], (unsigned long long)run);
    }
  }
}

/* Both counters of a ctx from the per-queue figures the planner has already produced: the
 * ctx's first and last position, and the kept counts of its queues added up.  One warp per
 * ctx, lanes over its queues; the keep flags are not read. */
__global__ void __launch_bounds__(kThreads)
k_goodput_from_queues(const uint32_t* __restrict__ seg_off, const uint32_t* __restrict__ seg_kept,
                      uint32_t n_ctx, uint32_t S, long long* __restrict__ out_total,
                      long long* __restrict__ out_kept) {
  pdl_wait();
  const uint32_t c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (c >= n_ctx) return;                          /* whole warps leave together */
  unsigned long long sum = 0;
  for (uint32_t k = lane; k < S; k += 32) sum += seg_kept[(size_t)c * S + k];
  for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    out_total[c] = (long long)seg_off[(size_t)(c + 1) * S] - (long long)seg_off[(size_t)c * S];
    out_kept[c] = (long long)sum;
  }
}

}  // namespace

extern "C" int pard_goodput(const uint8_t* d_keep, const uint32_t* d_seg_offsets,
                            const uint32_t* d_seg_kept, uint64_t n,
                            uint32_t n_ctx, int32_t stage_stride, int64_t* d_out_total,
                            int64_t* d_out_kept, void* cuda_stream) {
  if (!d_seg_offsets || !d_out_total || !d_out_kept || n_ctx < 1 || stage_stride < 1) return PARD_EINVAL;
  if (!d_seg_kept && n > 0 && (!d_keep || ((uintptr_t)d_keep & 15))) return PARD_EINVAL;
  if (n >= PARD_MAX_REQUESTS || stage_stride > PARD_MAX_STAGES ||
      (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS)
    return PARD_ERANGE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (d_seg_kept) {
    launch_pdl(k_goodput_from_queues, (n_ctx + kThreads / 32 - 1) / (kThreads / 32), kThreads, 0, stream, d_seg_offsets,
               d_seg_kept, n_ctx, (uint32_t)stage_stride, (long long*)d_out_total, (long long*)d_out_kept);
    pard_profile_extend_last(stream);
    PARD_CUDA_OK(cudaGetLastError());
    return PARD_OK;
  }
  launch_pdl(k_goodput_init, (n_ctx + 255) / 256, 256, 0, stream, d_seg_offsets, n_ctx, (uint32_t)stage_stride,
                                                          (long long*)d_out_total, (long long*)d_out_kept);
  if (n > 0) {
    uint32_t blocks = (uint32_t)((n + kChunk - 1) / kChunk);
    launch_pdl(k_goodput_count, blocks, kThreads, 0, stream, d_keep, d_seg_offsets, (uint32_t)n, n_ctx,
                                                     (uint32_t)stage_stride,
                                                     (unsigned long long*)d_out_kept);
  }
  pard_profile_extend_last(stream);
  PARD_CUDA_OK(cudaGetLastError());
  return PARD_OK;
}
