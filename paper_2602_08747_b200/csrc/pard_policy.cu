/* Decision rules that need a sequential walk of every queue.
 *
 * The planner's own rule in budget order has thresholds that only rise along a queue, which
 * turns the Request Broker's loop into a prefix minimum (pard_plan.cu).  That no longer holds
 *   - when requests carry the downstream path they will take (Sec. 5.2, dynamic-path DAGs):
 *     L_sub, and with it the threshold, differs from request to request;
 *   - in arrival order (Table 1 and Sec. 5.3, PARD-FCFS);
 *   - for Clipper++'s per-module share of the objective (Sec. 5.1, Baseline), arrival order;
 *   - for Nexus' window scan (Sec. 5.1, Baseline), a rule of its own.
 * For the first three the loop is  x <- x + [x < u_r]  with u_r the number of requests that may
 * be admitted ahead of or at r while r still makes its (own) deadline; x is the admitted count.
 * Three kernels over the sorted elements:
 *   k_policy_terms   every request on its own: gathers the request (and its arrival record),
 *                    computes u_r (Nexus: the number of batch rounds r still fits)    -> T[n]
 *   k_policy_walk    one warp per queue walks T in queue order, 32 requests per step: the
 *                    admitted positions of a step are the fixed point of
 *                    keep_i = [x + #kept among lanes below i < u_i], found by iterating from
 *                    "all kept" (bit i is final after i + 1 rounds; a few rounds in practice)
 *                                                                      -> C[n] = position | keep << 31
 *   k_policy_emit    every request on its own again: estimate from its position, outputs,
 *                    survivor lists
 * T and C live in the sort buffer that does not hold the elements. */
#include "pard_plan_internal.cuh"

using namespace pard_plan_detail;

namespace {

constexpr int kPolThreads = 128;
constexpr int kPolItems = 8;
constexpr int kPolTile = kPolThreads * kPolItems;
constexpr int kStageSegs = 4;            /* queues whose path sums a block keeps in shared memory */
constexpr int kMaskPaths = 16;           /* bits of pard_request_t.flags */
constexpr uint32_t kKeepBit = 0x80000000u;

struct SortedView {
  const unsigned long long* src;
  uint32_t* T;
  uint32_t* C;
  uint32_t kshift, imask;
};

__device__ __forceinline__ SortedView sorted_view(const PolicyArgs& a) {
  SortedView v;
  const bool odd = a.hdr->npass & 1;
  v.src = odd ? a.buf_b : a.buf_a;
  uint32_t* spare = reinterpret_cast<uint32_t*>(odd ? a.buf_a : a.buf_b);
  v.T = spare;
  v.C = spare + a.n;                     /* 8 bytes per request: two 32-bit arrays */
  v.kshift = a.ibits + a.hdr->dbits;
  v.imask = (1u << a.ibits) - 1;
  return v;
}

__device__ __forceinline__ const PardPipeDev* pipe_of(const PolicyArgs& a, uint32_t c) {
  int32_t pi = a.st.d_pipeline_of_ctx ? a.st.d_pipeline_of_ctx[c] : 0;
  if (pi < 0 || (uint32_t)pi >= a.n_pipelines) pi = 0;          /* reported by k_seg_const */
  return a.n_pipelines <= (uint32_t)kFewPipelines ? a.pipes.few[pi] : a.pipes.many[pi];
}

/* sum over the path in slot `s` of q_i + d_i(B_i), plus w of the slot (Eq. 3, State Planner part) */
__device__ long long path_sum(const PolicyArgs& a, const PardPipeDev* p, uint32_t c, int32_t s) {
  const uint32_t S = (uint32_t)a.st.stage_stride;
  long long acc = a.st.d_w_us ? a.st.d_w_us[(size_t)c * a.st.slot_stride + s] : 0;
  for (int32_t e = p->path_off[s]; e < p->path_off[s + 1]; ++e) {
    const int32_t i = p->path_stage[e];
    int32_t Bi = a.st.d_batch[(size_t)c * S + i];
    if (Bi < 1 || Bi > p->bmax[i]) Bi = 1;                      /* reported by k_seg_const */
    acc += a.st.d_q_us[(size_t)c * S + i] + p->lat_us[p->lat_offsets[i] + Bi - 1];
  }
  return acc;
}

/* Path sums of the first kStageSegs queues a block's tile touches, kept in shared memory. */
struct StagedPaths {
  long long sum[kStageSegs][kMaskPaths];
  int32_t n_paths[kStageSegs];
  uint32_t seg0;
};

__device__ void stage_paths(const PolicyArgs& a, uint32_t seg0, StagedPaths& sp) {
  const uint32_t S = (uint32_t)a.st.stage_stride;
  if (threadIdx.x == 0) sp.seg0 = seg0;
  for (uint32_t t = threadIdx.x; t < kStageSegs * kMaskPaths; t += blockDim.x) {
    const uint32_t q = t / kMaskPaths, j = t % kMaskPaths, seg = seg0 + q;
    if (seg >= a.n_seg) { if (j == 0) sp.n_paths[q] = 0; continue; }
    const uint32_t c = seg / S, k = seg % S;
    const PardPipeDev* p = pipe_of(a, c);
    int32_t np = 0;
    if (k < (uint32_t)p->n_stages) {
      const int32_t s0 = p->stage_slot_off[k];
      np = p->stage_slot_off[k + 1] - s0;
      if ((int32_t)j < np) sp.sum[q][j] = path_sum(a, p, c, s0 + (int32_t)j);
    }
    if (j == 0) sp.n_paths[q] = np;
  }
  __syncthreads();
}

/* What the rule needs of one request: with A the completion estimate at admitted position 0 and
 * D the instant it is compared with, the request at admitted position c completes (by the rule's
 * own account) at A + floor(c / cap) * d and is kept iff that is <= D. */
struct Terms {
  long long A, D;
};

__device__ Terms request_terms(const PolicyArgs& a, const StagedPaths& sp, uint32_t seg, uint32_t idx,
                               const PardSegConst& K) {
  Terms t;
  const uint4 r = __ldg(&a.req[idx]);
  t.D = (long long)(((unsigned long long)r.y << 32) | r.x);
  t.A = K.A;
  if (a.mode & (PARD_MODE_NEXUS | PARD_MODE_CLIPPER)) t.A = K.A - K.lsub;     /* the current module only: base + d */
  if (a.mode & PARD_MODE_CLIPPER) {
    /* the module's share of the request's objective, counted from its arrival at the module; the
     * request is kept iff its batch starts within the share: start <= arrive + share, i.e.
     * start + d <= arrive + share + d */
    const pard_arrival_t ar = a.arrivals[idx];
    long long share = 0;
    if (ar.arrive_us < 0 || ar.arrive_us >= PARD_TIME_LIMIT_US || ar.slo_us < 0 || ar.slo_us >= (1ll << 31) ||
        K.d >= (1ll << 32)) {
      set_status(a.hdr, PARD_EDATA);
      t.D = 0;
    } else {
      share = (long long)((unsigned long long)ar.slo_us * (unsigned long long)K.d / (unsigned long long)K.dsum);
      t.D = ar.arrive_us + share + K.d;
    }
  }
  const uint32_t flags = r.w >> 16;
  if ((a.mode & PARD_MODE_PATH_MASK) && flags != 0 && !(K.narrow & kSegNoStage)) {
    /* the request's downstream path is known: the maximum runs over the named paths only */
    const uint32_t q = seg - sp.seg0;
    long long best = -1;
    int32_t np;
    if (q < (uint32_t)kStageSegs) {
      np = sp.n_paths[q];
      for (int32_t j = 0; j < np && j < kMaskPaths; ++j)
        if ((flags >> j) & 1u) best = sp.sum[q][j] > best ? sp.sum[q][j] : best;
    } else {                                     /* a queue beyond the staged ones: straight from the tables */
      const uint32_t S = (uint32_t)a.st.stage_stride, c = seg / S, k = seg % S;
      const PardPipeDev* p = pipe_of(a, c);
      const int32_t s0 = p->stage_slot_off[k];
      np = p->stage_slot_off[k + 1] - s0;
      for (int32_t j = 0; j < np && j < kMaskPaths; ++j)
        if ((flags >> j) & 1u) {
          const long long v = path_sum(a, p, c, s0 + j);
          best = v > best ? v : best;
        }
    }
    if (np > 0) {                                /* a sink has nothing downstream whatever the mask says */
      if (best < 0) set_status(a.hdr, PARD_EDATA);   /* the mask names no path of this stage */
      else t.A = K.A - K.lsub + best;
    }
  }
  return t;
}

/* number of batch rounds b for which a request still fits, b < v: Nexus tests "base + b*d + d <= D" */
__device__ __forceinline__ uint32_t rounds_fit(long long X, const PardSegConst& K) {
  if (X < 0) return 0;
  unsigned long long q;
  if (((unsigned long long)X >> 32) == 0 && K.d_magic) q = div_magic32((uint32_t)X, K.d_magic);
  else q = (unsigned long long)X / (unsigned long long)K.d;
  return q >= kUClamp ? kUClamp : (uint32_t)q + 1;
}

__global__ void __launch_bounds__(kPolThreads)
k_policy_terms(const PolicyArgs a) {
  pdl_wait();
  __shared__ StagedPaths sp;
  if (a.hdr->wide || a.hdr->aborted) return;
  const SortedView v = sorted_view(a);
  const uint64_t tile0 = (uint64_t)blockIdx.x * kPolTile;
  if (a.mode & PARD_MODE_PATH_MASK) stage_paths(a, (uint32_t)(v.src[tile0] >> v.kshift), sp);
  else if (threadIdx.x == 0) sp.seg0 = 0;
  for (int i = 0; i < kPolItems; ++i) {
    const uint64_t j = tile0 + (uint64_t)i * kPolThreads + threadIdx.x;
    if (j >= a.n) break;
    const unsigned long long e = v.src[j];
    const uint32_t seg = (uint32_t)(e >> v.kshift), idx = (uint32_t)e & v.imask;
    const PardSegConst K = a.ktab[seg];
    if (K.narrow & kSegNoStage) { set_status(a.hdr, PARD_EDATA); v.T[j] = 0; continue; }
    const Terms t = request_terms(a, sp, seg, idx, K);
    v.T[j] = (a.mode & PARD_MODE_NEXUS) ? rounds_fit(t.D - t.A, K) : threshold_u(t.D - t.A, K);
  }
}

/* One warp per queue.  General rule: x <- x + [x < u_r]. */
__device__ void walk_admit(const uint32_t* __restrict__ T, uint32_t* __restrict__ C, uint32_t lo, uint32_t hi,
                           uint32_t lane, uint32_t* kept_out, bool raw) {
  const uint32_t below = (1u << lane) - 1;
  uint32_t x = 0;
  if (raw) {
    /* every queued request ahead takes a batch slot: a request is kept iff its own queue position
     * is below its threshold, whatever happened before it; what is walked is only the count of
     * kept requests ahead (the survivor's slot) */
    for (uint32_t b0 = lo; b0 < hi; b0 += 32) {
      const uint32_t j = b0 + lane;
      const bool keep = j < hi && (j - lo) < T[j];
      const uint32_t m = __ballot_sync(0xffffffffu, keep);
      if (j < hi) C[j] = (x + __popc(m & below)) | (keep ? kKeepBit : 0u);
      x += __popc(m);
    }
    *kept_out = x;
    return;
  }
  constexpr int kAhead = 4;                        /* steps whose thresholds are requested together */
  for (uint32_t b0 = lo; b0 < hi; b0 += 32 * kAhead) {
    uint32_t u[kAhead];
#pragma unroll
    for (int k = 0; k < kAhead; ++k) {
      const uint32_t j = b0 + 32 * k + lane;
      u[k] = j < hi ? T[j] : 0u;                   /* beyond the queue: never kept */
    }
#pragma unroll
    for (int k = 0; k < kAhead; ++k) {
      if (b0 + 32 * k >= hi) break;                /* uniform */
      uint32_t m = __ballot_sync(0xffffffffu, x < u[k]);        /* as if nobody in the step were kept before */
      for (int round = 0; round < 34; ++round) {   /* bit i is final after i + 1 rounds */
        const uint32_t m2 = __ballot_sync(0xffffffffu, x + __popc(m & below) < u[k]);
        if (m2 == m) break;
        m = m2;
      }
      const uint32_t j = b0 + 32 * k + lane;
      if (j < hi) C[j] = (x + __popc(m & below)) | (((m >> lane) & 1u) ? kKeepBit : 0u);
      x += __popc(m);
    }
  }
  *kept_out = x;
}

/* Nexus: a window of one batch round (W requests) slides over the queue; the batch is the first
 * window whose requests all still fit the round b being formed (b < v_r); everything before it
 * is dropped; b advances; the scan resumes behind the window.  A request's position is
 * b * W + its offset in the run of fitting requests it belongs to, so floor(position / W) = the
 * round it was tested against, and for the kept ones it is also the number kept before them. */
__device__ void walk_nexus(const uint32_t* __restrict__ T, uint32_t* __restrict__ C, uint32_t lo, uint32_t hi,
                           uint32_t W, uint32_t lane, uint32_t* kept_out) {
  uint32_t b = 0, run = 0;                         /* batches formed; length of the current run of fitting requests */
  for (uint32_t p0 = lo; p0 < hi; p0 += 32) {
    const uint32_t nvalid = min(32u, hi - p0);
    const uint32_t v = lane < nvalid ? T[p0 + lane] : 0u;
    const uint32_t valid = nvalid == 32 ? 0xffffffffu : ((1u << nvalid) - 1);
    uint32_t cval = 0;
    uint32_t pos = 0;
    while (pos < nvalid) {                         /* uniform */
      const uint32_t fit = __ballot_sync(0xffffffffu, b < v) & valid;
      const uint32_t from = ~((1u << pos) - 1);    /* lanes >= pos */
      const uint32_t bad = ~fit & valid & from;
      const uint32_t firstbad = bad ? (uint32_t)__ffs(bad) - 1 : nvalid;
      const uint32_t fitlen = firstbad - pos, need = W - run;
      if (fitlen >= need) {                        /* the window is full at lane pos + need - 1 */
        if (lane >= pos && lane < pos + need) cval = (b * W + run + (lane - pos)) | kKeepBit;
        ++b;
        run = 0;
        pos += need;
      } else if (firstbad < nvalid) {              /* a request that does not fit: the run before it goes too */
        if (lane >= pos && lane < firstbad) cval = b * W + run + (lane - pos);
        if (lane == firstbad) cval = b * W;
        /* the part of the run met in earlier steps (a run only grows across a step's end, so none
         * of it lies in this step): those positions lose their provisional keep */
        if (run > 0) {
          __syncwarp();
          const uint32_t first = p0 + pos - run;   /* >= lo; pos is 0 here */
          for (uint32_t q = first + lane; q < p0 + pos; q += 32) C[q] &= ~kKeepBit;
          __syncwarp();
        }
        run = 0;
        pos = firstbad + 1;
      } else {                                     /* everything up to the end of the step fits: the run goes on */
        if (lane >= pos && lane < nvalid) cval = (b * W + run + (lane - pos)) | kKeepBit;
        run += fitlen;
        pos = nvalid;
      }
    }
    if (lane < nvalid) C[p0 + lane] = cval;
  }
  *kept_out = b * W + run;                         /* a last, partly filled window runs as it is */
}

__global__ void __launch_bounds__(kPolThreads)
k_policy_walk(const PolicyArgs a) {
  pdl_wait();
  if (a.hdr->wide || a.hdr->aborted) return;
  const uint32_t s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (s >= a.n_seg) return;                        /* whole warps leave together */
  const SortedView v = sorted_view(a);
  const uint32_t lo = a.seg_off[s], hi = a.seg_off[s + 1];
  uint32_t kept = 0;
  if (hi > lo) {
    if (a.mode & PARD_MODE_NEXUS) walk_nexus(v.T, v.C, lo, hi, a.ktab[s].cap, lane, &kept);
    else walk_admit(v.T, v.C, lo, hi, lane, &kept, (a.mode & PARD_MODE_RAW) != 0);
  }
  if (lane == 0) a.seg_kept[s] = kept;
}

__global__ void __launch_bounds__(kPolThreads)
k_policy_emit(const PolicyArgs a) {
  pdl_wait();
  __shared__ StagedPaths sp;
  if (a.hdr->wide || a.hdr->aborted) return;
  const SortedView v = sorted_view(a);
  const uint64_t tile0 = (uint64_t)blockIdx.x * kPolTile;
  if (a.mode & PARD_MODE_PATH_MASK) stage_paths(a, (uint32_t)(v.src[tile0] >> v.kshift), sp);
  else if (threadIdx.x == 0) sp.seg0 = 0;
  for (int i = 0; i < kPolItems; ++i) {
    const uint64_t j = tile0 + (uint64_t)i * kPolThreads + threadIdx.x;
    if (j >= a.n) break;
    const unsigned long long e = v.src[j];
    const uint32_t seg = (uint32_t)(e >> v.kshift), idx = (uint32_t)e & v.imask;
    const PardSegConst K = a.ktab[seg];
    uint32_t c = 0, keep = 0;
    long long est = K.A;
    if (!(K.narrow & kSegNoStage)) {
      const Terms t = request_terms(a, sp, seg, idx, K);
      const uint32_t w = v.C[j];
      c = w & ~kKeepBit;                           /* kept requests ahead in the queue */
      keep = w >> 31;
      /* the batch-slot position: the kept requests ahead, or, when every request ahead takes a slot, all of them */
      const uint32_t slot = (a.mode & PARD_MODE_RAW) ? (uint32_t)j - a.seg_off[seg] : c;
      const uint32_t round = K.cap_magic ? div_magic32(slot, K.cap_magic) : slot;     /* floor(slot / cap) */
      est = t.A + (long long)round * K.d;
    }
    if (a.out_keep) a.out_keep[j] = (uint8_t)keep;
    if (a.out_est) a.out_est[j] = est;
    if (a.out_perm) a.out_perm[j] = idx;
    if (keep && a.kept_tmp) a.kept_tmp[a.seg_off[seg] + c] = idx;                /* c = kept requests ahead in the queue */
  }
}

}  // namespace

namespace pard_plan_detail {

int launch_policy_decision(const PolicyArgs& a, int sms, cudaStream_t stream) {
  (void)sms;
  const uint32_t tiles = (uint32_t)(((uint64_t)a.n + kPolTile - 1) / kPolTile);
  launch_pdl(k_policy_terms, tiles, kPolThreads, 0, stream, a);
  launch_pdl(k_policy_walk, (a.n_seg + kPolThreads / 32 - 1) / (kPolThreads / 32), kPolThreads, 0, stream, a);
  launch_pdl(k_policy_emit, tiles, kPolThreads, 0, stream, a);
  return cudaGetLastError() == cudaSuccess ? PARD_OK : PARD_ECUDA;
}

}  // namespace pard_plan_detail
