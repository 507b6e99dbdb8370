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
  uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_ctx) return;
  out_total[c] = (long long)seg_off[(size_t)(c + 1) * S] - (long long)seg_off[(size_t)c * S];
  out_kept[c] = 0;
}

/* Each thread sums 16 keep flags read as one vector; sums of one ctx are
 * combined in the warp, then in the block, before one atomic per (block, ctx). */
__global__ void __launch_bounds__(kThreads)
k_goodput_count(const uint8_t* __restrict__ keep, const uint32_t* __restrict__ seg_off, uint32_t n,
                uint32_t n_ctx, uint32_t S, unsigned long long* __restrict__ out_kept) {
  constexpr int WARPS = kThreads / 32;
  __shared__ uint32_t s_ctx[WARPS];
  __shared__ uint32_t s_sum[WARPS];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint64_t o = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) * 16;
  constexpr uint32_t kNone = 0xffffffffu;
  uint32_t my_ctx = kNone, my_sum = 0;
  if (o < n) {
    /* last ctx whose start is <= o (empty ctxs share a start; the last one owns the byte) */
    uint32_t lo = 0, hi = n_ctx;               /* invariant: start(lo) <= o, start(hi) > o or hi == n_ctx */
    while (hi - lo > 1) {
      uint32_t mid = lo + (hi - lo) / 2;
      if (ctx_start(seg_off, mid, S) <= o) lo = mid; else hi = mid;
    }
    uint32_t c = lo;
    uint32_t cend = ctx_start(seg_off, c + 1, S);
    if (o + 16 <= n && o + 16 <= cend) {
      uint4 v = __ldg(reinterpret_cast<const uint4*>(keep + o));
      my_ctx = c;
      my_sum = __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
    } else {
      /* a ctx boundary or the end of the array inside these 16 flags */
      uint32_t run = 0;
      for (uint32_t b = 0; b < 16 && o + b < n; ++b) {
        while (o + b >= cend) {
          if (run) atomicAdd(&out_kept[c], (unsigned long long)run);
          run = 0;
          ++c;
          cend = ctx_start(seg_off, c + 1, S);
        }
        run += keep[o + b] & 1u;
      }
      my_ctx = c;
      my_sum = run;
    }
  }
  /* warp: threads usually share one ctx */
  uint32_t c0 = __shfl_sync(0xffffffffu, my_ctx, 0);
  if (__all_sync(0xffffffffu, my_ctx == c0)) {
    for (int k = 16; k; k >>= 1) my_sum += __shfl_xor_sync(0xffffffffu, my_sum, k);
    if (lane == 0) { s_ctx[warp] = c0; s_sum[warp] = my_sum; }
  } else {
    if (my_ctx != kNone && my_sum) atomicAdd(&out_kept[my_ctx], (unsigned long long)my_sum);
    if (lane == 0) { s_ctx[warp] = kNone; s_sum[warp] = 0; }
  }
  __syncthreads();
  if (warp == 0) {
    uint32_t c = lane < WARPS ? s_ctx[lane] : kNone;
    uint32_t s = lane < WARPS ? s_sum[lane] : 0;
    uint32_t grp = __match_any_sync(0xffffffffu, c);
    uint32_t tot = 0;
    for (uint32_t m = grp; m; m &= m - 1) tot += __shfl_sync(grp, s, __ffs(m) - 1);
    if (c != kNone && tot && lane == (uint32_t)(__ffs(grp) - 1)) atomicAdd(&out_kept[c], (unsigned long long)tot);
  }
}

}  // namespace

extern "C" int pard_goodput(const uint8_t* d_keep, const uint32_t* d_seg_offsets, uint64_t n,
                            uint32_t n_ctx, int32_t stage_stride, int64_t* d_out_total,
                            int64_t* d_out_kept, void* cuda_stream) {
  if (!d_seg_offsets || !d_out_total || !d_out_kept || n_ctx < 1 || stage_stride < 1) return PARD_EINVAL;
  if (n > 0 && (!d_keep || ((uintptr_t)d_keep & 15))) return PARD_EINVAL;
  if (n >= PARD_MAX_REQUESTS || stage_stride > PARD_MAX_STAGES ||
      (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS)
    return PARD_ERANGE;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  k_goodput_init<<<(n_ctx + 255) / 256, 256, 0, stream>>>(d_seg_offsets, n_ctx, (uint32_t)stage_stride,
                                                          (long long*)d_out_total, (long long*)d_out_kept);
  if (n > 0) {
    uint32_t blocks = (uint32_t)((n + (uint64_t)kThreads * 16 - 1) / ((uint64_t)kThreads * 16));
    k_goodput_count<<<blocks, kThreads, 0, stream>>>(d_keep, d_seg_offsets, (uint32_t)n, n_ctx,
                                                     (uint32_t)stage_stride,
                                                     (unsigned long long*)d_out_kept);
  }
  PARD_CUDA_OK(cudaGetLastError());
  return PARD_OK;
}
