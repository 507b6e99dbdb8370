/* The planner of libpard: kernels and their orchestration.
 *
 * Steps (paper passages in pard.h):
 *   prepass   per-ctx deadline range, per-segment queue length, input checks
 *   segscan   queue lengths -> first position of every segment
 *   segconst  per-segment constants of Eq. 3: d_k(B_k), base, L_sub (max over
 *             downstream paths), folded into A = base + d + L_sub
 *   pack      request -> one 64-bit sort element (segment | deadline | index)
 *   sort      LSD radix sort, 8 bits per pass, one read and one write of the
 *             elements per pass (tile prefixes by decoupled look-back)
 *   decide    threshold u per request, segmented prefix-min scan -> admitted
 *             position c, estimate, keep flag, compaction, per-segment counts
 */
#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>

#include "pard_plan_internal.cuh"

using namespace pard_plan_detail;

namespace {

struct Layout {
  /* [hdr, zero_end) must be zero when the first kernel starts: cleared by k_clear (of the two
   * look-back arrays only the first: every sort pass clears the array of the pass after it) */
  uint64_t hdr, ctx_dmin, ctx_dmax, seg_off, seg_kept, win_done, hist, whist, hist_ctx, lookback, zero_end, tile_first,
      ctx_start, pipes, ktab, kept_base, chunk_base, tile_agg, tile_carry, win_off, win_cnt, win_own, win_big, wtab, kept_tmp,
      buf_a, buf_b, total;
  uint32_t n_seg, sort_tiles, dec_tiles, max_passes, win_capacity;
  uint32_t lb_tiles;          /* tiles the look-back arrays are sized for */
  uint32_t ctx_passes;        /* 1: the call may sort inside the contexts' ranges (contexts of more than a tile on average) */
};

__host__ __device__ inline uint32_t bit_width64(unsigned long long x) {
  uint32_t b = 0;
  while (x) { ++b; x >>= 1; }
  return b;
}

inline uint32_t ceil_log2(uint64_t x) {          /* smallest b with 2^b >= x */
  uint32_t b = 0;
  while (((uint64_t)1 << b) < x) ++b;
  return b;
}

Layout make_layout(uint64_t n, uint32_t n_ctx, int32_t stage_stride) {
  Layout L;
  auto al = [](uint64_t x) { return (x + 255) & ~(uint64_t)255; };
  L.n_seg = n_ctx * (uint32_t)stage_stride;
  L.sort_tiles = (uint32_t)((n + kSortTile - 1) / kSortTile);
  L.dec_tiles = (uint32_t)((n + kDecTile - 1) / kDecTile);
  uint32_t ibits = std::max(1u, ceil_log2(n));
  uint32_t sbits = ceil_log2(L.n_seg);
  L.max_passes = std::min<uint32_t>(kMaxPasses, (std::min(64u - ibits, sbits + 60u) + 7) / 8);
  uint64_t o = 0;
  L.hdr = o;       o = al(o + sizeof(PlanHeader));
  L.ctx_dmin = o;  o = al(o + 8ull * n_ctx);          /* complement of the minimum: starts at 0 */
  L.ctx_dmax = o;  o = al(o + 8ull * n_ctx);
  L.seg_off = o;   o = al(o + 4ull * (L.n_seg + 1));
  L.seg_kept = o;  o = al(o + 4ull * L.n_seg);
  L.win_done = o;  o = al(o + 4ull * L.n_seg);
  L.hist = o;      o = al(o + 4ull * kMaxPasses * kBins);
  L.whist = o;     o = al(o + (L.n_seg <= kHistSegs ? 4ull * kHistCap : 0ull));   /* window counts of calls with few queues */
  /* passes kept inside the contexts' ranges cut the tiles at ctx boundaries: at most one more
   * tile per ctx; they keep digit counts per ctx */
  L.ctx_passes = (n_ctx > 1 && (uint64_t)n_ctx * kSortTile < n) ? 1u : 0u;
  L.lb_tiles = L.sort_tiles + (L.ctx_passes ? n_ctx : 0u);
  L.hist_ctx = o;  o = al(o + (L.ctx_passes ? 4ull * kMaxPasses * kBins * (uint64_t)n_ctx : 0ull));
  L.lookback = o;  L.zero_end = al(o + 4ull * kBins * (uint64_t)L.lb_tiles);
  o = al(o + 2 * 4ull * kBins * (uint64_t)L.lb_tiles);                      /* two arrays, used in turn */
  L.tile_first = o; o = al(o + (L.ctx_passes ? 4ull * ((uint64_t)n_ctx + 1) : 0ull));
  L.ctx_start = o; o = al(o + 4ull * ((uint64_t)n_ctx + 1));
  L.pipes = o;     o = al(o + 8ull * kMaxPipelinesPerCall);
  L.ktab = o;      o = al(o + sizeof(PardSegConst) * (uint64_t)L.n_seg);
  L.kept_base = o; o = al(o + 4ull * (L.n_seg + 1));
  L.chunk_base = o; o = al(o + 4ull * (L.n_seg + 1));
  L.tile_agg = o;  o = al(o + 8ull * L.dec_tiles);
  L.tile_carry = o; o = al(o + 4ull * L.dec_tiles);
  L.win_capacity = (uint32_t)(n / 32 + 4ull * L.n_seg + 1024);
  if (L.n_seg <= kHistSegs) L.win_capacity = std::max(L.win_capacity, kHistCap);   /* counted tables: see k_seg_const */
  L.win_off = o;   o = al(o + 4ull * (L.n_seg + 1));
  L.win_cnt = o;   o = al(o + 4ull * (L.n_seg + 1));
  L.win_own = o;   o = al(o + 4ull * L.win_capacity);
  L.win_big = o;   o = al(o + 4ull * L.win_capacity);
  L.wtab = o;      o = al(o + 16ull * L.win_capacity);
  L.kept_tmp = o;  o = al(o + 4ull * n);
  L.buf_a = o;     o = al(o + 8ull * n);
  L.buf_b = o;     o = al(o + 8ull * n);
  L.total = o;
  return L;
}

/* A bounded wait ran out: the elements are only partly sorted from here on, so nothing after
 * this may use them as indices. */
__device__ __forceinline__ void set_aborted(PlanHeader* hdr) {
  hdr->aborted = 1;
  __threadfence();
  atomicExch(&hdr->status, (uint32_t)(-PARD_ETIMEOUT));
}

/* See k_sort_local: the call's requests come grouped by ctx and no ctx exceeds a tile. */
__device__ __forceinline__ bool sort_is_local(const PlanHeader* hdr, uint32_t candidate) {
  return candidate && !hdr->unsorted && !hdr->ctx_too_big && !hdr->wide;
}

/* True in every thread of exactly one block: the one whose arrival at `counter` is the last of
 * the grid.  Every thread's earlier global writes are visible to that block afterwards. */
__device__ __forceinline__ bool last_block_done(uint32_t* counter) {
  __shared__ uint32_t s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(counter, 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  const bool last = s_last != 0;
  if (last) __threadfence();
  return last;
}

/* Clears the part of the scratch that must start at zero.  A kernel rather than a memset: it is
 * launched like every other kernel of the call, so its blocks are placed while the previous
 * work of the stream drains. */
__global__ void __launch_bounds__(256)
k_clear(uint4* __restrict__ p, unsigned long long n16) {
  pdl_wait();
  const unsigned long long step = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += step)
    p[i] = make_uint4(0u, 0u, 0u, 0u);
}

/* ------------------------------------------------------------------------ */
/* prepass: one coalesced 16-byte read per request                           */
/* ------------------------------------------------------------------------ */
/* Range checks and the smallest / largest deadline of every ctx.  A thread
 * follows the ctx of the requests it reads and only touches global memory
 * when that ctx changes; requests of one ctx normally sit together, so this
 * is rare.  (ctx_dmin_inv holds the complement of the minimum, so that both
 * arrays start from zero and grow by atomicMax.) */
__global__ void __launch_bounds__(256)
k_prepass(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t S,
          unsigned long long* __restrict__ ctx_dmin_inv, unsigned long long* __restrict__ ctx_dmax,
          PlanHeader* hdr) {
  pdl_wait();
  constexpr uint32_t kNone = 0xffffffffu;
  const uint32_t lane = threadIdx.x & 31;
  uint32_t run_ctx = kNone;
  unsigned long long lmin = ~0ull, lmax = 0;
  bool bad_seen = false;
  auto flush = [&]() {
    if (run_ctx != kNone) {
      atomicMax(&ctx_dmin_inv[run_ctx], ~lmin);
      atomicMax(&ctx_dmax[run_ctx], lmax);
    }
  };
  /* whole warp (converged): one atomic pair if all lanes follow the same ctx, else one per lane */
  auto warp_flush = [&]() {
    const uint32_t c0 = __shfl_sync(0xffffffffu, run_ctx, 0);
    if (__all_sync(0xffffffffu, run_ctx == c0)) {
      for (int o = 16; o; o >>= 1) {
        const unsigned long long a = __shfl_xor_sync(0xffffffffu, lmin, o);
        const unsigned long long b = __shfl_xor_sync(0xffffffffu, lmax, o);
        lmin = a < lmin ? a : lmin;
        lmax = b > lmax ? b : lmax;
      }
      if (lane == 0) flush();
    } else {
      flush();
    }
    run_ctx = kNone;
    lmin = ~0ull;
    lmax = 0;
  };
  const uint64_t chunk = (uint64_t)blockDim.x * 8;
  for (uint64_t base = (uint64_t)blockIdx.x * chunk; base < n; base += (uint64_t)gridDim.x * chunk) {
    uint4 r[8];
    uint32_t have = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint64_t j = base + (uint64_t)i * blockDim.x + threadIdx.x;
      if (j < n) {
        r[i] = __ldg(&req[j]);
        have |= 1u << i;
      }
    }
    /* a new chunk usually lies in another ctx than the last one: hand the old one over together */
    if (__any_sync(0xffffffffu, (have & 1u) && run_ctx != kNone && r[0].z != run_ctx)) warp_flush();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (!((have >> i) & 1u)) continue;
      const unsigned long long D = ((unsigned long long)r[i].y << 32) | r[i].x;
      const uint32_t ctx = r[i].z, stage = r[i].w & 0xffffu;
      if (D >= (unsigned long long)PARD_TIME_LIMIT_US || ctx >= n_ctx || stage >= S) {
        bad_seen = true;
        continue;
      }
      if (ctx != run_ctx) {
        flush();
        run_ctx = ctx;
        lmin = ~0ull;
        lmax = 0;
      }
      lmin = D < lmin ? D : lmin;
      lmax = D > lmax ? D : lmax;
    }
  }
  warp_flush();
  if (bad_seen) set_status(hdr, PARD_EDATA);
}

__global__ void k_ctx_span(const unsigned long long* __restrict__ ctx_dmin_inv,
                           const unsigned long long* __restrict__ ctx_dmax, uint32_t n_ctx,
                           PlanHeader* hdr) {
  pdl_wait();
  uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
  unsigned long long span = 0;
  if (c < n_ctx && ~ctx_dmin_inv[c] <= ctx_dmax[c]) span = ctx_dmax[c] - ~ctx_dmin_inv[c];
  for (int o = 16; o; o >>= 1) {
    unsigned long long a = __shfl_xor_sync(0xffffffffu, span, o);
    span = a > span ? a : span;
  }
  if ((threadIdx.x & 31) == 0 && span) atomicMax(&hdr->span_max, span);
}

/* Width of the sort key, once the widest deadline span is known. */
/* key_sbits: the queue-id bits that the passes have to sort (all of them, or the stage bits only
 * when the passes stay inside the contexts' ranges) */
__global__ void k_key_width(uint32_t sbits, uint32_t ibits, PlanHeader* hdr, uint32_t arrival_order, uint32_t key_sbits) {
  pdl_wait();
  /* in arrival order the deadline takes no part in the key: the index alone orders a queue */
  const uint32_t dbits = arrival_order ? 0u : bit_width64(hdr->span_max);
  hdr->dbits = dbits;
  hdr->keybits = key_sbits + dbits;
  hdr->npass = (key_sbits + dbits + 7) / 8;
  if (sbits + dbits + ibits > 64) {
    hdr->npass = 0;
    hdr->wide = 1;
    set_status(hdr, PARD_ERANGE);
  }
}

/* The constants of one queue (ctx c, stage k), by one whole warp: lanes over the stage's
 * downstream paths (the path table of the pipeline lists, for every stage, each stage sequence
 * from a successor to a sink).  dmin / dmax: smallest and largest deadline of the ctx, the
 * origins of the queue's deadline offsets.  Every lane returns the same value; *bad is set in
 * the lanes that met an input out of range. */
__device__ PardSegConst seg_const_warp(const PipeTable& pipes, uint32_t n_pipelines, const pard_queue_state_t& st,
                                       uint32_t c, uint32_t k, unsigned long long dmin, unsigned long long dmax,
                                       uint32_t lane, bool* bad_out) {
  const uint32_t S = (uint32_t)st.stage_stride;
  PardSegConst out;
  out.A = 0; out.A_rel = 0; out.d = 1; out.cap = 1; out.d_magic = 0; out.cap_magic = 0;
  out.narrow = 0; out.lsub = 0; out.dsum = 1;
  int32_t pi = st.d_pipeline_of_ctx ? st.d_pipeline_of_ctx[c] : 0;
  bool bad = false;
  if (pi < 0 || (uint32_t)pi >= n_pipelines) {
    bad = true;
  } else {
    const PardPipeDev* p = n_pipelines <= (uint32_t)kFewPipelines ? pipes.few[pi] : pipes.many[pi];
    const int64_t* qrow = st.d_q_us + (size_t)c * S;
    const int32_t* brow = st.d_batch + (size_t)c * S;
    if (k >= (uint32_t)p->n_stages) {
      out.narrow = 2;            /* no such stage: a request found in this queue is an input error */
    } else {
      int32_t B = brow[k];
      int64_t m = st.d_workers ? st.d_workers[(size_t)c * S + k] : 1;
      int64_t now = st.d_now_us[c], fa = st.d_free_at_us[(size_t)c * S + k];
      if (B < 1 || B > p->bmax[k] || m < 1 || now < 0 || now >= PARD_TIME_LIMIT_US || fa < 0 ||
          fa >= PARD_TIME_LIMIT_US) {
        bad = true;
      } else {
        const int64_t d = p->lat_us[p->lat_offsets[k] + B - 1];
        const int32_t s0 = p->stage_slot_off[k], s1 = p->stage_slot_off[k + 1];
        long long lsub = -1;                              /* every path sum is >= 1 */
        for (int32_t s = s0 + (int32_t)lane; s < s1; s += 32) {
          int64_t acc = st.d_w_us ? st.d_w_us[(size_t)c * st.slot_stride + s] : 0;
          if (acc < 0 || acc >= PARD_TIME_LIMIT_US) { bad = true; acc = 0; }
          for (int32_t e = p->path_off[s]; e < p->path_off[s + 1]; ++e) {
            int32_t i = p->path_stage[e];
            int32_t Bi = brow[i];
            int64_t qi = qrow[i];
            if (Bi < 1 || Bi > p->bmax[i] || qi < 0 || qi >= PARD_TIME_LIMIT_US) { bad = true; Bi = 1; qi = 0; }
            acc += qi + p->lat_us[p->lat_offsets[i] + Bi - 1];
          }
          lsub = acc > lsub ? acc : lsub;
        }
        for (int o = 16; o; o >>= 1) {                    /* maximum over the paths */
          long long t = __shfl_xor_sync(0xffffffffu, lsub, o);
          lsub = t > lsub ? t : lsub;
        }
        if (lsub < 0) lsub = 0;                           /* a sink: nothing downstream */
        int64_t base = now > fa ? now : fa;
        int64_t cap = (int64_t)B * m;
        out.d = d;
        out.cap = (uint32_t)(cap > (int64_t)(1u << 30) ? (int64_t)(1u << 30) : cap);
        out.A = base + d + lsub;
        /* A against the origin of the queue's deadline offsets: offsets count up from the ctx's
         * smallest deadline, or, for a queue served high budget first, down from its largest */
        const bool high_first = st.d_priority && st.d_priority[(size_t)c * S + k] != 0;
        out.A_rel = high_first ? (int64_t)dmax - out.A : out.A - (int64_t)dmin;
        out.d_magic = (d >= 2 && d < ((int64_t)1 << 32)) ? magic64((uint64_t)d) : 0;
        out.cap_magic = out.cap >= 2 ? magic64(out.cap) : 0;
        const int64_t lim = (int64_t)1 << 29;
        out.narrow = (out.d_magic != 0 && d < ((int64_t)1 << 31) && out.A_rel > -lim && out.A_rel < lim) ? 1u : 0u;
        if (high_first) out.narrow |= kSegHighFirst;
        out.lsub = lsub;
        /* all stages' durations at their current batch sizes, for the rule that splits the objective
         * in proportion to them (a batch size out of range is reported by that stage's own warp) */
        long long dsum = 0;
        for (int32_t i = (int32_t)lane; i < p->n_stages; i += 32) {
          const int32_t Bi = brow[i];
          dsum += p->lat_us[p->lat_offsets[i] + ((Bi >= 1 && Bi <= p->bmax[i]) ? Bi : 1) - 1];
        }
        for (int o = 16; o; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
        out.dsum = dsum;
      }
    }
  }
  *bad_out = bad;
  return out;
}

/* Per-segment constants; one warp per (ctx, stage). */
__global__ void __launch_bounds__(128)
k_seg_const(const PipeTable pipes, uint32_t n_pipelines,
            pard_queue_state_t st, uint32_t n_ctx,
            const unsigned long long* __restrict__ ctx_dmin_inv,
            const unsigned long long* __restrict__ ctx_dmax, PardSegConst* __restrict__ ktab,
            PlanHeader* hdr, uint32_t sbits, uint32_t ibits, uint32_t with_key_width, uint32_t arrival_order,
            uint32_t win_hist, uint32_t force_scan, uint32_t* __restrict__ win_off, uint32_t* __restrict__ win_cnt,
            uint32_t key_sbits) {
  pdl_wait();
  const uint32_t S = (uint32_t)st.stage_stride;
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t seg = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (seg < n_ctx * S) {                                 /* whole warps take the same side */
    const uint32_t c = seg / S, k = seg % S;
    bool bad = false;
    const PardSegConst out = seg_const_warp(pipes, n_pipelines, st, c, k, ~ctx_dmin_inv[c], ctx_dmax[c], lane, &bad);
    if (bad) set_status(hdr, PARD_EDATA);
    if (lane == 0) ktab[seg] = out;
  }
  /* With few queues the block that finishes last also finds the widest deadline span and with
   * it the width of the sort key (the work of k_ctx_span and k_key_width, without their launches). */
  if (!with_key_width) return;
  if (!last_block_done(&hdr->seg_done)) return;
  __shared__ unsigned long long s_span[4];
  unsigned long long span = 0;
  for (uint32_t c = threadIdx.x; c < n_ctx; c += blockDim.x) {
    const unsigned long long lo = ~ctx_dmin_inv[c], hi = ctx_dmax[c];
    if (lo <= hi && hi - lo > span) span = hi - lo;
  }
  for (int o = 16; o; o >>= 1) {
    const unsigned long long a = __shfl_xor_sync(0xffffffffu, span, o);
    span = a > span ? a : span;
  }
  if (lane == 0) s_span[threadIdx.x >> 5] = span;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (uint32_t w = 1; w < blockDim.x / 32; ++w) span = s_span[w] > span ? s_span[w] : span;
    const uint32_t dbits = arrival_order ? 0u : bit_width64(span);
    hdr->span_max = span;
    hdr->dbits = dbits;
    hdr->keybits = key_sbits + dbits;
    hdr->npass = (key_sbits + dbits + 7) / 8;
    if (sbits + dbits + ibits > 64) {
      hdr->npass = 0;
      hdr->wide = 1;
      set_status(hdr, PARD_ERANGE);
    }
  }
  /* Few queues: their batch-window tables are COUNTED while the requests are packed (k_pack)
   * instead of being searched for in the sorted elements afterwards.  That needs the tables'
   * extents before any request has been looked at: a queue can have no window beyond that of its
   * ctx's latest deadline.  Entry 0 of a queue counts its requests with deadline < A, entry b + 1
   * those of window b; every queue has at least entry 0, so that the counts also give the queues'
   * lengths. */
  if (win_hist) {                                        /* still the last block, all its threads */
    __shared__ uint32_t s_w[kHistSegs];
    __shared__ uint32_t s_scan;
    const uint32_t n_seg = n_ctx * S;
    if (threadIdx.x == 0) s_scan = force_scan;
    __syncthreads();
    for (uint32_t q = threadIdx.x; q < n_seg; q += blockDim.x) {   /* every queue's number of entries, side by side */
      const PardSegConst K = ktab[q];
      const uint32_t c = q / S;
      uint32_t w = 1;
      const unsigned long long lo = ~ctx_dmin_inv[c], hi = ctx_dmax[c];
      if (!(K.narrow & kSegNoStage) && lo <= hi) {
        const long long X = (long long)hi - K.A;
        const unsigned long long nb = X < 0 ? 0ull : (unsigned long long)X / (unsigned long long)K.d + 1;
        if (nb >= 4096) s_scan = 1;                      /* kWinMaxPerSeg: too many windows for a table */
        else w = (uint32_t)nb + 1;
      }
      s_w[q] = w;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t total = 0;
      bool scan = s_scan != 0;
      for (uint32_t q = 0; q < n_seg; ++q) {
        uint32_t w = s_w[q];
        if (total + w > kHistCap) { scan = true; w = 1; }
        win_off[q] = total;
        win_cnt[q] = w;
        total += w;
      }
      hdr->win_total = total;
      if (scan) hdr->use_scan = 1;
    }
  }
}

/* request -> sort element; digit histograms of every pass */
template <bool WIN>
__global__ void __launch_bounds__(256)
k_pack(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t S,
       const unsigned long long* __restrict__ ctx_dmin_inv, const unsigned long long* __restrict__ ctx_dmax,
       const uint8_t* __restrict__ priority, uint32_t ibits,
       PlanHeader* __restrict__ hdr, unsigned long long* __restrict__ dst,
       uint32_t* __restrict__ hist, uint32_t local_candidate,
       const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ win_off,
       const uint32_t* __restrict__ win_cnt, uint32_t* __restrict__ whist) {
  pdl_wait();
  __shared__ uint32_t s_hist[kMaxPasses * kBins];
  /* WIN: the batch-window tables are counted here (few queues); per-queue constants in shared memory */
  constexpr uint32_t kWinWords = 2048;                      /* more would cost the kernel its occupancy */
  __shared__ uint32_t s_win[WIN ? kWinWords : 1];
  __shared__ long long s_A[WIN ? kHistSegs : 1], s_d[WIN ? kHistSegs : 1];
  __shared__ unsigned long long s_magic[WIN ? kHistSegs : 1];
  __shared__ uint4 s_wcon[WIN ? kHistSegs : 1];            /* per queue: A_rel, first table entry, entries, A_rel and d fit 32 bits */
  if (hdr->wide || sort_is_local(hdr, local_candidate)) return;   /* sorted block by block: k_sort_local read the requests itself */
  const uint32_t npass = hdr->npass, dbits = hdr->dbits;
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x) s_hist[i] = 0;
  /* The counters are kept in as many copies as fit (a power of two, at most one per lane), lane l
   * counting in copy l mod copies: requests of one warp that fall into the same entry -- the
   * usual case when most of a queue is expired, or lies in few windows -- then hit different words. */
  uint32_t win_total = 0, copies = 1, my_copy = 0;
  bool win_shared = false;                                  /* tables beyond kWinWords entries are counted in global memory */
  bool win_derive = false;
  if (WIN) {
    win_total = (uint32_t)hdr->win_total;
    win_shared = win_total <= kWinWords;
    while (copies < 32 && 2 * copies * win_total <= kWinWords) copies *= 2;
    my_copy = (threadIdx.x & (copies - 1)) * win_total;
    if (win_shared) for (uint32_t i = threadIdx.x; i < win_total * copies; i += blockDim.x) s_win[i] = 0;
    /* When the queue id lies inside the last pass's digit the queues' lengths can be read off that
     * pass's digit counts (see k_seg_win), and entry 0 of a queue -- its requests with deadline < A,
     * often most of an overloaded queue -- is its length minus its other entries: such requests
     * are then not counted here at all. */
    win_derive = npass > 0 && hdr->keybits - dbits <= hdr->keybits - 8 * (npass - 1);
    for (uint32_t q = threadIdx.x; q < n_ctx * S; q += blockDim.x) {
      const PardSegConst K = ktab[q];
      s_A[q] = K.A; s_d[q] = K.d; s_magic[q] = K.d_magic;
      s_wcon[q] = make_uint4((uint32_t)(int32_t)K.A_rel, win_off[q], win_cnt[q], (K.narrow & (kSegNarrow | kSegNoStage)) == kSegNarrow ? 1u : 0u);
    }
  }
  __syncthreads();
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  /* n < 2^30: positions and strides in 32 bits (the grid has at most n threads) */
  const uint32_t stride = gridDim.x * blockDim.x;
  const bool key32 = hdr->keybits <= 32;       /* the key fits one word: its digits are peeled off that word */
  const bool off32 = dbits <= 29;              /* deadline offsets fit signed 32-bit arithmetic */
  uint32_t cur_ctx = 0xffffffffu;              /* the ctx whose deadline range is at hand (requests of a ctx mostly sit together) */
  unsigned long long cmin = 0, cmax = 0;
  constexpr int kUn = 4;                       /* requests in flight per thread (measured against 1: 74 vs 78.5 us at 2^24) */
  for (uint32_t j0 = blockIdx.x * blockDim.x + threadIdx.x; j0 < n; j0 += stride * kUn) {
    uint4 rr[kUn];
#pragma unroll
    for (int u = 0; u < kUn; ++u) {
      const uint32_t j = j0 + (uint32_t)u * stride;
      if (j < n) rr[u] = __ldg(&req[j]);
    }
#pragma unroll
    for (int u = 0; u < kUn; ++u) {
      const uint32_t j = j0 + (uint32_t)u * stride;
      if (j >= n) break;
      const uint4 r = rr[u];
      const uint32_t ctx = r.z, stage = r.w & 0xffffu;
      const bool ok = ctx < n_ctx && stage < S;
      const uint32_t seg = ok ? ctx * S + stage : 0u;
      if (ok && ctx != cur_ctx) {
        cur_ctx = ctx;
        cmin = ~ctx_dmin_inv[ctx];
        cmax = ctx_dmax[ctx];
      }
      /* ascending offsets give the queue's decision order: deadlines counted up from the ctx's
       * smallest, or down from its largest when the queue is served high budget first */
      const bool high_first = ok && priority && __ldg(&priority[seg]) != 0;
      uint32_t h = 0;                            /* the request's entry in its queue's window table: 0 for deadline < A, else window + 1 */
      bool count = false;
      uint4 c = make_uint4(0u, 0u, 1u, 0u);      /* A - ctx's smallest deadline (if it fits 32 bits), first entry, entries, fits? */
      if (key32 && off32) {
        /* everything in single words: the offset is below 2^29, so the low words of the 64-bit
         * difference are the difference */
        const uint32_t off = ok ? ((high_first ? (uint32_t)cmax - r.x : r.x - (uint32_t)cmin) & (uint32_t)dmask) : 0u;
        uint32_t key = (seg << dbits) | off;
        if (WIN && ok) {
          c = s_wcon[seg];
          count = true;
          if (c.w) {
            const int32_t X = (int32_t)off - (int32_t)c.x;
            if (X >= 0) {
              const uint32_t b = div_magic32((uint32_t)X, s_magic[seg]);
              h = b + 1 < c.z ? b + 1 : c.z - 1;   /* never beyond the queue's entries (a queue decided by scanning has one) */
            }
          } else {
            const long long X = (long long)(((unsigned long long)r.y << 32) | r.x) - s_A[seg];
            if (X >= 0) {
              const unsigned long long M = s_magic[seg];
              const unsigned long long b = (((unsigned long long)X >> 32) == 0 && M) ? div_magic32((uint32_t)X, M)
                                                                                    : (unsigned long long)X / (unsigned long long)s_d[seg];
              h = b + 1 < c.z ? (uint32_t)b + 1 : c.z - 1;
            }
          }
        }
        *reinterpret_cast<uint2*>(dst + j) = make_uint2((key << ibits) | j, __funnelshift_l(key, 0u, ibits));
        uint32_t* hp = s_hist;
        for (uint32_t p = 0; p < npass; ++p, hp += kBins, key >>= 8) atomicAdd(hp + (key & 255u), 1u);
      } else {
        const unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
        const unsigned long long off = ok ? ((high_first ? cmax - D : D - cmin) & dmask) : 0ull;
        unsigned long long key = ((unsigned long long)seg << dbits) | off;
        if (WIN && ok) {
          c = s_wcon[seg];
          count = true;
          const long long X = (long long)D - s_A[seg];
          if (X >= 0) {
            const unsigned long long M = s_magic[seg];
            const unsigned long long b = (((unsigned long long)X >> 32) == 0 && M) ? div_magic32((uint32_t)X, M)
                                                                                  : (unsigned long long)X / (unsigned long long)s_d[seg];
            h = b + 1 < c.z ? (uint32_t)b + 1 : c.z - 1;
          }
        }
        dst[j] = (key << ibits) | j;
        uint32_t* hp = s_hist;
        for (uint32_t p = 0; p < npass; ++p, hp += kBins, key >>= 8) atomicAdd(hp + ((uint32_t)key & 255u), 1u);
      }
      if (WIN) {
        /* a request flagged by the prepass (its element is its index alone) sorts into queue 0 and is
         * counted there, entry 0: the counts stay the queues' lengths */
        if (!ok) { c.y = 0; h = 0; count = true; }
        if (count && (h != 0 || !win_derive)) {
          if (win_shared) atomicAdd(&s_win[my_copy + c.y + h], 1u);
          else atomicAdd(&whist[c.y + h], 1u);
        }
      }
    }
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x)
    if (s_hist[i]) atomicAdd(&hist[i], s_hist[i]);
  if (WIN && win_shared)
    for (uint32_t i = threadIdx.x; i < win_total; i += blockDim.x) {
      uint32_t sum = 0;
      for (uint32_t r = 0; r < copies; ++r) sum += s_win[r * win_total + i];
      if (sum) atomicAdd(&whist[i], sum);
    }
}

/* ------------------------------------------------------------------------ */
/* one LSD radix pass (8 bits), stable, tile prefixes by decoupled look-back */
/* ------------------------------------------------------------------------ */
/* Tile = kSortTile elements; every warp owns a run of consecutive elements
 * (kItemsLo rounds of 32 for the warps that also do the look-back, kItemsHi
 * rounds for the others) and visits it 32 at a time, so the tile order is
 * (warp, round, lane).
 *   1. every warp counts its digits (shared atomics, order irrelevant);
 *   2. thread d turns the counts of digit d into the first tile-local slot of
 *      every (warp, digit) and publishes the tile's count for the look-back;
 *   3. the lower part of the block adds up the counts of all earlier tiles
 *      (look-back, kLookBatch tiles per memory round trip) while the other
 *      warps already rank;
 *   4. ranking: the lanes that hold the same digit find each other through a
 *      shared word (atomic OR), take consecutive slots in lane order and drop
 *      their elements into the shared tile buffer, now sorted by digit;
 *   5. the buffer is written out, run by run, to the digit's global range.
 * Large tiles keep the number of tiles in flight, and with it the depth of the
 * look-back, small. */
/* loads and stores of look-back words: relaxed, device scope (other blocks write them) */
__device__ __forceinline__ uint32_t ld_relaxed(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(uint32_t* p, uint32_t v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

struct SortSmem {
  unsigned long long keys[kSortTile];
  uint32_t slot[kSortThreads / 32][kBins];    /* counts, then next free tile-local slot per (warp, digit) */
  uint32_t match[kSortThreads / 32][kBins];   /* lanes currently holding the digit */
  uint32_t dstart[kBins];
  uint32_t gofs[kBins];
  uint32_t scan[2][kSortThreads / 32];
  uint32_t tile;
  uint32_t abort;
  uint32_t ctx, lo_tile, base, limit, first;   /* the tile's ctx and range when passes stay inside the contexts */
};

/* one warp's share of step 1: ITEMS rounds of 32 consecutive elements */
template <int ITEMS>
__device__ __forceinline__ void sort_load_count(unsigned long long (&key)[kItemsHi], const unsigned long long* src,
                                                uint64_t first, uint32_t n, uint32_t shift, uint32_t* slot_row,
                                                uint32_t lane, uint32_t dig_mask = 255u) {
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const uint64_t j = first + i * 32 + lane;
    key[i] = j < n ? src[j] : ~0ull;
  }
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) atomicAdd(&slot_row[(uint32_t)(key[i] >> shift) & dig_mask], 1u);
}

/* one warp's share of step 4 */
template <int ITEMS, int CAP>
__device__ __forceinline__ void sort_rank_drop(const unsigned long long (&key)[CAP], uint32_t shift,
                                               uint32_t* slot_row, uint32_t* match_row, unsigned long long* keys,
                                               uint32_t lanebit, int items = ITEMS, uint32_t dig_mask = 255u) {
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    if (i >= items) break;                             /* the same for the whole block */
    const uint32_t d = (uint32_t)(key[i] >> shift) & dig_mask;
    atomicOr(&match_row[d], lanebit);
    __syncwarp();
    const uint32_t grp = match_row[d];
    const uint32_t below = grp & (lanebit - 1);
    const uint32_t first = slot_row[d];                /* same word for the whole group */
    __syncwarp();
    if (below == 0) {                                  /* lowest lane of the group */
      slot_row[d] = first + __popc(grp);
      match_row[d] = 0;
    }
    keys[first + __popc(below)] = key[i];
    __syncwarp();
  }
}

/* The same two steps for a pass whose digit has one or two bits (the top pass of a key of 8k + 1
 * or 8k + 2 bits): the lanes that hold the same digit find each other by one ballot per digit
 * bit, lane j keeps the warp's running count of digit j in a register, and neither the counting
 * nor the ranking touches shared memory apart from the key's own store.  Measured at 2^24
 * elements: a 1-bit pass 89 us against 120 us through the generic code (where 32 lanes hammer two
 * counters); with four ballots (a 4-bit digit) the instructions outweigh the saved shared-memory
 * traffic (16.2 us against 14.5 us at 2^20 elements), so wider digits stay on the generic code.
 * The 89 us are what a pass costs with ranking almost free: tile load, write-out, scans and
 * barriers.  Full tiles only (no padding keys). */
template <int BITS>
__device__ __forceinline__ uint32_t digit_peers(uint32_t d, const uint32_t (&bal)[BITS]) {
  uint32_t m = 0xffffffffu;
#pragma unroll
  for (int k = 0; k < BITS; ++k) m &= ((d >> k) & 1u) ? bal[k] : ~bal[k];
  return m;
}

template <int ITEMS, int BITS>
__device__ __forceinline__ void sort_load_count_few(unsigned long long (&key)[kItemsHi], const unsigned long long* src,
                                                    uint64_t first, uint32_t shift, uint32_t* slot_row, uint32_t lane) {
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) key[i] = src[first + i * 32 + lane];
  uint32_t mine = 0;                                     /* lane j: keys of this warp with digit j */
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const uint32_t d = (uint32_t)(key[i] >> shift);
    uint32_t bal[BITS];
#pragma unroll
    for (int k = 0; k < BITS; ++k) bal[k] = __ballot_sync(0xffffffffu, (d >> k) & 1u);
    mine += __popc(digit_peers<BITS>(lane, bal));
  }
  if (lane < (1u << BITS)) slot_row[lane] = mine;
}

template <int ITEMS, int CAP, int BITS>
__device__ __forceinline__ void sort_rank_drop_few(const unsigned long long (&key)[CAP], uint32_t shift,
                                                   const uint32_t* slot_row, unsigned long long* keys, uint32_t lane) {
  uint32_t next = lane < (1u << BITS) ? slot_row[lane] : 0u;   /* lane j: next free slot of digit j for this warp */
  const uint32_t below = (1u << lane) - 1;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const uint32_t d = (uint32_t)(key[i] >> shift) & ((1u << BITS) - 1);
    uint32_t bal[BITS];
#pragma unroll
    for (int k = 0; k < BITS; ++k) bal[k] = __ballot_sync(0xffffffffu, (d >> k) & 1u);
    const uint32_t grp = digit_peers<BITS>(d, bal);
    const uint32_t first = __shfl_sync(0xffffffffu, next, d);
    keys[first + __popc(grp & below)] = key[i];
    next += __popc(digit_peers<BITS>(lane, bal));
  }
}

/* digit width known at run time only: one instantiation per width */
template <int ITEMS>
__device__ __forceinline__ void sort_load_count_few_n(unsigned long long (&key)[kItemsHi], const unsigned long long* src,
                                                      uint64_t first, uint32_t shift, uint32_t bits, uint32_t* slot_row,
                                                      uint32_t lane) {
  switch (bits) {
    case 1: sort_load_count_few<ITEMS, 1>(key, src, first, shift, slot_row, lane); break;
    default: sort_load_count_few<ITEMS, 2>(key, src, first, shift, slot_row, lane); break;
  }
}
template <int ITEMS, int CAP>
__device__ __forceinline__ void sort_rank_drop_few_n(const unsigned long long (&key)[CAP], uint32_t shift, uint32_t bits,
                                                     const uint32_t* slot_row, unsigned long long* keys, uint32_t lane) {
  switch (bits) {
    case 1: sort_rank_drop_few<ITEMS, CAP, 1>(key, shift, slot_row, keys, lane); break;
    default: sort_rank_drop_few<ITEMS, CAP, 2>(key, shift, slot_row, keys, lane); break;
  }
}

/* CTX: the pass stays inside every ctx's range of the array (requests grouped by ctx, contexts of
 * more than a tile): tiles are cut at ctx boundaries (tile_first[c] = first tile of ctx c), the
 * digit counts are per ctx, a digit's range starts at the ctx's first position, and the look-back
 * stops at the ctx's first tile -- so the ctx bits of the key need no pass at all. */
struct CtxTiles {
  const uint32_t* ctx_start;     /* [n_ctx + 1] */
  const uint32_t* tile_first;    /* [n_ctx + 1] */
  const uint32_t* hist;          /* [n_ctx][kMaxPasses][kBins] */
  uint32_t n_ctx;
};

template <bool PERSIST, bool CTX>
__global__ void __launch_bounds__(kSortThreads, 2)
k_sort_pass(uint32_t pass, PlanHeader* hdr, unsigned long long* __restrict__ buf_a,
            unsigned long long* __restrict__ buf_b, const uint32_t* __restrict__ hist,
            uint32_t* __restrict__ lookback, uint32_t* __restrict__ lookback_next, uint32_t n,
            uint32_t ibits, uint32_t stall, uint32_t local_candidate, const CtxTiles ct) {
  pdl_wait();
  constexpr int WARPS = kSortThreads / 32;
  static_assert(kLoWarps * 32 == kBins, "one look-back thread per digit");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SortSmem& S = *reinterpret_cast<SortSmem*>(smem_raw);

  if (pass >= hdr->npass || hdr->aborted || sort_is_local(hdr, local_candidate)) return;
  const unsigned long long* src = (pass & 1) ? buf_b : buf_a;
  unsigned long long* dst = (pass & 1) ? buf_a : buf_b;
  hist += pass * kBins;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lanebit = 1u << lane;
  const uint32_t n_tiles = (uint32_t)(((uint64_t)n + kSortTile - 1) / kSortTile);
  /* PERSIST: a small grid whose blocks take tile after tile (used where the pass is launched
   * only as the fallback of the block-local sort and will almost always return at once);
   * otherwise one tile per block */
  for (;;) {
  if (tid == 0) {
    const uint32_t t = atomicAdd(&hdr->ticket[pass], 1u);
    S.tile = t;
    S.abort = 0;
    if (CTX) {                                           /* the ctx of the tile: last c with tile_first[c] <= t */
      uint32_t lo = 0, hi = ct.n_ctx;
      while (hi - lo > 1) {
        const uint32_t mid = lo + (hi - lo) / 2;
        if (ct.tile_first[mid] <= t) lo = mid; else hi = mid;
      }
      S.ctx = t < ct.tile_first[ct.n_ctx] ? lo : 0xffffffffu;     /* the grid may hold more blocks than there are tiles */
      S.lo_tile = ct.tile_first[lo];
      S.base = ct.ctx_start[lo] + (t - ct.tile_first[lo]) * (uint32_t)kSortTile;
      S.limit = ct.ctx_start[lo + 1];
      S.first = ct.ctx_start[lo];
    }
  }
  for (uint32_t i = tid; i < WARPS * kBins; i += kSortThreads) {
    (&S.slot[0][0])[i] = 0;
    (&S.match[0][0])[i] = 0;
  }
  uint32_t gh = (!CTX && tid < kBins) ? hist[tid] : 0; /* count of digit tid in the whole array (in the ctx), needed in step 2 */
  __syncthreads();
  const uint32_t tile = S.tile;
  if (PERSIST && tile >= n_tiles) return;
  if (CTX && S.ctx == 0xffffffffu) return;
  if (CTX && tid < kBins) gh = ct.hist[((size_t)S.ctx * kMaxPasses + pass) * kBins + tid];
  const uint64_t base = CTX ? (uint64_t)S.base : (uint64_t)tile * kSortTile;
  const uint32_t limit = CTX ? S.limit : n;            /* end of the range the tile belongs to */
  const int64_t lo_tile = CTX ? (int64_t)S.lo_tile : 0;
  const uint32_t shift = ibits + 8 * pass;

  /* 1. load and count.  The warps that will do the look-back own fewer
   * elements than the others, so that both groups finish at about the same
   * time and the look-back has registers for a wide batch. */
  unsigned long long key[kItemsHi];
  const bool lo_warp = warp < kLoWarps;
  const uint32_t wfirst = lo_warp ? warp * (32 * kItemsLo)
                                  : kLoWarps * 32 * kItemsLo + (warp - kLoWarps) * (32 * kItemsHi);
  /* a digit of one or two bits on a full tile: counted and ranked by ballots */
  const uint32_t dig_bits = min(8u, hdr->keybits - 8 * pass);
  /* inside a ctx the bits above the key (the ctx's part of the queue id) are the same everywhere
   * and take no part in the digit */
  const uint32_t dig_mask = CTX ? (1u << dig_bits) - 1 : 255u;
  const bool few = dig_bits <= 2 && base + kSortTile <= (uint64_t)limit;
  if (few) {
    if (lo_warp) sort_load_count_few_n<kItemsLo>(key, src, base + wfirst, shift, dig_bits, S.slot[warp], lane);
    else sort_load_count_few_n<kItemsHi>(key, src, base + wfirst, shift, dig_bits, S.slot[warp], lane);
  } else if (lo_warp) sort_load_count<kItemsLo>(key, src, base + wfirst, limit, shift, S.slot[warp], lane, dig_mask);
  else sort_load_count<kItemsHi>(key, src, base + wfirst, limit, shift, S.slot[warp], lane, dig_mask);
  __syncthreads();

  /* 2. thread d owns digit d */
  uint32_t cnt = 0, x = 0, g = 0;
  if (tid < kBins) {
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
      const uint32_t t = S.slot[w][tid];
      S.slot[w][tid] = cnt;                            /* exclusive over the warps */
      cnt += t;
    }
    x = cnt;
    g = gh;
    for (int o = 1; o < 32; o <<= 1) {                 /* scans over the 256 digits */
      const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
      const uint32_t z = __shfl_up_sync(0xffffffffu, g, o);
      if (lane >= (uint32_t)o) { x += y; g += z; }
    }
    if (lane == 31) { S.scan[0][warp] = x; S.scan[1][warp] = g; }
    /* the tile's count is all that later tiles need from this one for now */
    if (!(stall && tile == 0)) st_relaxed(lookback + (size_t)tile * kBins + tid, cnt | kLbAgg);
    lookback_next[(size_t)tile * kBins + tid] = 0;     /* the array of the pass after this one */
  }
  __syncthreads();
  uint32_t dstart = 0, gstart = 0;
  if (tid < kBins) {
    uint32_t wx = 0, wg = 0;
#pragma unroll
    for (int w = 0; w < kBins / 32; ++w)
      if (w < (int)warp) { wx += S.scan[0][w]; wg += S.scan[1][w]; }
    dstart = wx + x - cnt;                             /* first tile-local slot of digit tid  */
    gstart = wg + g - gh + (CTX ? S.first : 0u);       /* first global position of digit tid  */
    S.dstart[tid] = dstart;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) S.slot[w][tid] += dstart;
  }
  __syncthreads();

  /* 3. look-back by the lower part of the block; the other warps go on */
  if (tid < kBins) {
    const uint32_t* lb = lookback;
    uint32_t excl = 0, spins = 0;
    int64_t t = (int64_t)tile - 1;
    bool done = t < lo_tile;
    while (!done) {
      uint32_t v[kLookBatch];
#pragma unroll
      for (int k = 0; k < kLookBatch; ++k)
        v[k] = (t - k >= lo_tile) ? ld_relaxed(lb + (size_t)(t - k) * kBins + tid) : +kLbIncl;   /* before the first tile: nothing */
      int used = 0;
#pragma unroll
      for (int k = 0; k < kLookBatch; ++k) {
        if (!done && used == k && (v[k] >> 30) != 0) {
          excl += v[k] & kLbMask;
          used = k + 1;
          if (v[k] & kLbIncl) done = true;
        }
      }
      t -= used;
      if (!done && used < kLookBatch) {                /* met a tile that has not published yet */
        if (++spins > kSpinLimit) { S.abort = 1; break; }
        __nanosleep(40);
      }
    }
    if (!(stall && tile == 0)) st_relaxed(lookback + (size_t)tile * kBins + tid, ((excl + cnt) & kLbMask) | kLbIncl);
    S.gofs[tid] = gstart + excl - dstart;
  }

  /* 4. rank and drop into the tile buffer */
  if (few) {
    if (lo_warp) sort_rank_drop_few_n<kItemsLo, kItemsHi>(key, shift, dig_bits, S.slot[warp], S.keys, lane);
    else sort_rank_drop_few_n<kItemsHi, kItemsHi>(key, shift, dig_bits, S.slot[warp], S.keys, lane);
  } else if (lo_warp) sort_rank_drop<kItemsLo, kItemsHi>(key, shift, S.slot[warp], S.match[warp], S.keys, lanebit, kItemsLo, dig_mask);
  else sort_rank_drop<kItemsHi, kItemsHi>(key, shift, S.slot[warp], S.match[warp], S.keys, lanebit, kItemsHi, dig_mask);
  __syncthreads();
  if (S.abort) {
    if (tid == 0) set_aborted(hdr);
    return;
  }

  /* 5. write out */
  const uint32_t nvalid = (uint32_t)min((uint64_t)kSortTile, (uint64_t)limit - base);
#pragma unroll 4
  for (uint32_t pos = tid; pos < nvalid; pos += kSortThreads) {
    const unsigned long long k = S.keys[pos];
    const uint32_t d = (uint32_t)(k >> shift) & dig_mask;
    dst[S.gofs[d] + pos] = k;
  }
  if (!PERSIST) return;
  __syncthreads();                                     /* the tile buffer and the tables are reused */
  }
}

/* First tile of every ctx when the tiles are cut at ctx boundaries: the running sum of
 * ceil(requests of the ctx / kSortTile).  One block. */
__global__ void __launch_bounds__(1024)
k_tile_table(const uint32_t* __restrict__ ctx_start, uint32_t n_ctx, uint32_t* __restrict__ tile_first) {
  pdl_wait();
  __shared__ uint32_t s_w[32];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t per = (n_ctx + 1023) / 1024;          /* contexts per thread, consecutive */
  const uint32_t c0 = tid * per, c1 = min(n_ctx, c0 + per);
  uint32_t sum = 0;
  for (uint32_t c = c0; c < c1; ++c) sum += (ctx_start[c + 1] - ctx_start[c] + kSortTile - 1) / kSortTile;
  uint32_t incl = sum;
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += y;
  }
  if (lane == 31) s_w[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = s_w[lane];
    uint32_t x = w;
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= (uint32_t)o) x += y;
    }
    s_w[lane] = x - w;
  }
  __syncthreads();
  uint32_t run = s_w[warp] + incl - sum;
  for (uint32_t c = c0; c < c1; ++c) {
    tile_first[c] = run;
    run += (ctx_start[c + 1] - ctx_start[c] + kSortTile - 1) / kSortTile;
  }
  if (c1 == n_ctx && c0 < n_ctx) tile_first[n_ctx] = run;
  if (n_ctx == 0 && tid == 0) tile_first[0] = 0;
}

/* k_pack for passes that stay inside the contexts: a block packs one tile (all of one ctx) and
 * adds its digit counts to the ctx's.  The digits cover the stage and deadline bits only; a
 * request of another ctx inside the tile breaks the caller's promise. */
__global__ void __launch_bounds__(256)
k_pack_ctx(const uint4* __restrict__ req, uint32_t S, const unsigned long long* __restrict__ ctx_dmin_inv,
           const unsigned long long* __restrict__ ctx_dmax, const uint8_t* __restrict__ priority, uint32_t ibits,
           PlanHeader* __restrict__ hdr, unsigned long long* __restrict__ dst, uint32_t* __restrict__ hist_ctx,
           const CtxTiles ct) {
  pdl_wait();
  __shared__ uint32_t s_hist[kMaxPasses * kBins];
  __shared__ uint32_t s_c, s_base, s_limit;
  if (hdr->unsorted) {                                   /* k_ctx_ranges found the requests out of ctx order */
    if (blockIdx.x == 0 && threadIdx.x == 0) { hdr->aborted = 1; set_status(hdr, PARD_EDATA); }
    return;
  }
  if (hdr->wide || hdr->aborted) return;
  const uint32_t tile = blockIdx.x;
  if (threadIdx.x == 0) {
    uint32_t lo = 0, hi = ct.n_ctx;
    while (hi - lo > 1) {
      const uint32_t mid = lo + (hi - lo) / 2;
      if (ct.tile_first[mid] <= tile) lo = mid; else hi = mid;
    }
    s_c = tile < ct.tile_first[ct.n_ctx] ? lo : 0xffffffffu;
    s_base = ct.ctx_start[lo] + (tile - ct.tile_first[lo]) * (uint32_t)kSortTile;
    s_limit = ct.ctx_start[lo + 1];
  }
  const uint32_t npass = hdr->npass, dbits = hdr->dbits;
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x) s_hist[i] = 0;
  __syncthreads();
  const uint32_t c = s_c;
  if (c == 0xffffffffu) return;
  const uint32_t end = min(s_limit, s_base + (uint32_t)kSortTile);
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  const unsigned long long cmin = ~ctx_dmin_inv[c], cmax = ctx_dmax[c];
  const unsigned long long keymask = hdr->keybits >= 64 ? ~0ull : ((1ull << hdr->keybits) - 1);
  bool foreign = false;
  for (uint32_t j = s_base + threadIdx.x; j < end; j += blockDim.x) {
    const uint4 r = __ldg(&req[j]);
    const unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
    const uint32_t stage = r.w & 0xffffu;
    unsigned long long key = 0;
    if (r.z != c) foreign = true;
    else if (stage < S) {
      const uint32_t seg = c * S + stage;
      const bool high_first = priority && __ldg(&priority[seg]) != 0;
      key = ((unsigned long long)seg << dbits) | ((high_first ? cmax - D : D - cmin) & dmask);
    }
    dst[j] = (key << ibits) | j;                         /* a flagged request keeps its index alone, as in k_pack */
    key &= keymask;                                      /* the ctx's part of the queue id takes no part in the digits */
    uint32_t* hp = s_hist;
    for (uint32_t p = 0; p < npass; ++p, hp += kBins, key >>= 8) atomicAdd(hp + ((uint32_t)key & 255u), 1u);
  }
  if (__syncthreads_or(foreign)) {
    if (threadIdx.x == 0) { hdr->unsorted = 1; hdr->aborted = 1; set_status(hdr, PARD_EDATA); }
    return;
  }
  uint32_t* h = hist_ctx + (size_t)c * kMaxPasses * kBins;
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x)
    if (s_hist[i]) atomicAdd(&h[i], s_hist[i]);
}

/* ------------------------------------------------------------------------ */
/* calls whose requests come grouped by ctx, every ctx within one tile       */
/* ------------------------------------------------------------------------ */
/* Batched decision epochs and small what-if instances arrive as one array with the requests of
 * a ctx side by side.  If no ctx holds more than a tile, nothing has to move between ctxs: a
 * block sorts "its" ctx in shared memory -- radix passes over the stage and deadline bits only,
 * no global scatter, no look-back -- and the global passes do not run.  `candidate` is the
 * host's part of the test (between kSortTile / 4 and kSortTile requests per ctx on average);
 * the device adds what only it can see.  A call with a single ctx of at most kSortTile requests
 * needs no test at all: its one block is certain, and neither the range search nor the global
 * passes are launched -- the case of one module's queue planned every few milliseconds. */
/* Where every ctx would begin if the requests came in ascending ctx order: the first request
 * whose ctx is >= c, by a 32-ary search, one warp per ctx.  Whether they do come in that order
 * is settled by k_sort_local, where every block checks that its range holds requests of its ctx
 * only; that test is complete as long as the boundaries never step back and the ranges cover
 * all requests, which is checked here. */
__global__ void __launch_bounds__(256)
k_ctx_ranges(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t* __restrict__ ctx_start,
             PlanHeader* hdr, uint32_t fmt_dbits, uint32_t sbits) {
  pdl_wait();
  const uint32_t c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t lane = threadIdx.x & 31;
  if (c > n_ctx) return;                         /* whole warps leave together */
  if (c == 0 && lane == 0 && fmt_dbits) {        /* the element format is fixed by the host: no key-width step */
    hdr->dbits = fmt_dbits;
    hdr->keybits = sbits + fmt_dbits;
    hdr->npass = 0;                              /* the sorted elements are in the first buffer */
  }
  uint32_t lo[2] = {0, 0}, hi[2] = {n, n};       /* first request whose ctx is >= c, >= c + 1 */
  while (lo[0] < hi[0] || lo[1] < hi[1]) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      if (lo[q] < hi[q]) {                       /* uniform across the warp */
        const uint32_t span = hi[q] - lo[q];
        const uint32_t p = lo[q] + (uint32_t)(((unsigned long long)(lane + 1) * span) / 33u);   /* lo <= p < hi */
        const bool less = __ldg(&req[p]).z < c + q;
        const uint32_t k = __popc(__ballot_sync(0xffffffffu, less));
        const uint32_t p_below = __shfl_sync(0xffffffffu, p, k > 0 ? k - 1 : 0);
        const uint32_t p_at = __shfl_sync(0xffffffffu, p, k < 32 ? k : 31);
        if (k > 0) lo[q] = p_below + 1;
        if (k < 32) hi[q] = p_at;
      }
    }
  }
  if (lane != 0) return;
  ctx_start[c] = lo[0];
  if (c == n_ctx && lo[0] != n) hdr->unsorted = 1;      /* requests past the last ctx's range (ctx out of range) */
  if (c < n_ctx) {
    if (lo[1] < lo[0]) hdr->unsorted = 1;
    else if (lo[1] - lo[0] > (uint32_t)kSortTile) hdr->ctx_too_big = 1;
  }
}

/* One block per ctx: the ctx's requests, read from the caller's array, turned into the sort
 * elements k_pack would have made, sorted in shared memory and written to the buffer the global
 * passes would have ended in (k_pack does not run then).  Inside a ctx only the stage and the
 * deadline offset differ; the ctx's own contribution to the segment field is left out of the
 * element while it is sorted and added on the way out, so that the passes see a plain bit field. */
__global__ void __launch_bounds__(kSortThreads, 2)
k_sort_local(PlanHeader* __restrict__ hdr, uint32_t candidate, const uint4* __restrict__ req,
             const unsigned long long* __restrict__ ctx_dmin_inv, const unsigned long long* __restrict__ ctx_dmax,
             const uint8_t* __restrict__ priority, unsigned long long* __restrict__ buf_a,
             unsigned long long* __restrict__ buf_b, const uint32_t* __restrict__ ctx_start, uint32_t n,
             uint32_t S, uint32_t stage_bits, uint32_t ibits) {
  pdl_wait();
  constexpr int WARPS = kSortThreads / 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SortSmem& Sm = *reinterpret_cast<SortSmem*>(smem_raw);
  if (!sort_is_local(hdr, candidate) || hdr->aborted) return;
  const uint32_t c = blockIdx.x;
  const uint32_t first = ctx_start ? ctx_start[c] : 0u;              /* no table: the call has one ctx */
  const uint32_t cnt = ctx_start ? ctx_start[c + 1] - first : n;
  if (cnt == 0) return;
  unsigned long long* dst = (hdr->npass & 1) ? buf_b : buf_a;
  const uint32_t dbits = hdr->dbits;
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  const unsigned long long dmin = ~ctx_dmin_inv[c], dmax = ctx_dmax[c];
  const uint32_t local_bits = dbits + stage_bits;
  const uint32_t passes = (local_bits + 7) / 8;
  const unsigned long long ctx_part = (unsigned long long)c * S << (dbits + ibits);   /* < 2^64: the key fits */
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lanebit = 1u << lane;
  constexpr int kItems = kSortTile / kSortThreads;       /* every warp owns the same share here: nothing else to do meanwhile */
  static_assert(kItems * kSortThreads == kSortTile, "the tile divides evenly");
  const uint32_t wfirst = warp * (32 * kItems);

  /* the ctx's requests, straight from the caller's array, turned into sort elements without the
   * ctx's share of the segment field (k_pack's element minus ctx_part); a request of another
   * ctx inside the range means the requests are not grouped after all */
  unsigned long long key[kItems];
  bool foreign = false;
#pragma unroll
  for (int i = 0; i < kItems; ++i) {
    const uint32_t pos = wfirst + i * 32 + lane;
    key[i] = ~0ull;                                       /* padding sorts last */
    if (pos < cnt) {
      const uint32_t j = first + pos;
      const uint4 r = __ldg(&req[j]);
      const unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
      const uint32_t stage = r.w & 0xffffu;
      foreign |= ctx_start != nullptr && r.z != c;       /* with one ctx there is no other: an input error */
      if (r.z == c && stage < S) {
        const bool high_first = priority && __ldg(&priority[c * S + stage]) != 0;
        const unsigned long long off = (high_first ? dmax - D : D - dmin) & dmask;
        key[i] = ((((unsigned long long)stage << dbits) | off) << ibits) | j;
      } else {
        key[i] = (unsigned long long)j - ctx_part;        /* flagged by the prepass; k_pack's element is j */
      }
    }
  }
  if (__syncthreads_or(foreign)) {                        /* the global passes take over (k_pack, then k_sort_pass) */
    if (tid == 0) hdr->unsorted = 1;
    return;
  }
  for (uint32_t i = tid; i < WARPS * kBins; i += kSortThreads) (&Sm.match[0][0])[i] = 0;   /* ranking leaves it clear */
  for (uint32_t p = 0; p < passes; ++p) {
    const uint32_t shift = ibits + 8 * p;
    for (uint32_t i = tid; i < WARPS * kBins; i += kSortThreads) (&Sm.slot[0][0])[i] = 0;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kItems; ++i) atomicAdd(&Sm.slot[warp][(uint32_t)(key[i] >> shift) & 255u], 1u);
    __syncthreads();
    uint32_t count = 0, x = 0;
    if (tid < kBins) {                                  /* thread d owns digit d */
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        const uint32_t t = Sm.slot[w][tid];
        Sm.slot[w][tid] = count;                        /* exclusive over the warps */
        count += t;
      }
      x = count;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= (uint32_t)o) x += y;
      }
      if (lane == 31) Sm.scan[0][warp] = x;
    }
    __syncthreads();
    if (tid < kBins) {
      uint32_t wx = 0;
#pragma unroll
      for (int w = 0; w < kBins / 32; ++w)
        if (w < (int)warp) wx += Sm.scan[0][w];
      const uint32_t dstart = wx + x - count;           /* first slot of digit tid */
#pragma unroll
      for (int w = 0; w < WARPS; ++w) Sm.slot[w][tid] += dstart;
    }
    __syncthreads();
    sort_rank_drop<kItems, kItems>(key, shift, Sm.slot[warp], Sm.match[warp], Sm.keys, lanebit);
    __syncthreads();
    if (p + 1 < passes) {
#pragma unroll
      for (int i = 0; i < kItems; ++i) key[i] = Sm.keys[wfirst + i * 32 + lane];
      __syncthreads();
    }
  }
  if (passes == 0) {                                    /* nothing differs inside a ctx: index order stands */
#pragma unroll
    for (int i = 0; i < kItems; ++i) Sm.keys[wfirst + i * 32 + lane] = key[i];
    __syncthreads();
  }
  for (uint32_t pos = tid; pos < cnt; pos += kSortThreads) dst[first + pos] = Sm.keys[pos] + ctx_part;
}

/* ------------------------------------------------------------------------ */
/* decision pass over the sorted elements                                    */
/* ------------------------------------------------------------------------ */
struct SegVal {            /* value of a segmented running reduction */
  int32_t m;               /* admitted mode: minimum of u_t - t; raw mode: number of kept requests;
                              over the elements since the last queue head (or since the span's start) */
  uint32_t head;           /* a queue head lies inside the span */
};

template <bool RAW>
__device__ __forceinline__ SegVal seg_identity() {
  SegVal a;
  a.m = RAW ? 0 : 0x7fffffff;
  a.head = 0;
  return a;
}

template <bool RAW>
__device__ __forceinline__ SegVal seg_combine(SegVal left, SegVal right) {
  SegVal r;
  r.m = right.head ? right.m : (RAW ? left.m + right.m : min(left.m, right.m));
  r.head = left.head | right.head;
  return r;
}

__device__ __forceinline__ unsigned long long pack_val(SegVal a, unsigned long long state) {
  return state | ((unsigned long long)a.head << 32) | (uint32_t)a.m;
}
__device__ __forceinline__ SegVal unpack_val(unsigned long long w) {
  SegVal a;
  a.m = (int32_t)(uint32_t)w;
  a.head = (uint32_t)(w >> 32) & 1u;
  return a;
}

/* X = deadline - A of a request from its deadline offset: offsets of a queue served high
 * budget first count down from the ctx's largest deadline, and A_rel is that deadline - A */
__device__ __forceinline__ long long slack_of(unsigned long long off, const PardSegConst& K) {
  return (K.narrow & kSegHighFirst) ? K.A_rel - (long long)off : (long long)off - K.A_rel;
}

/* First half of the decision pass for one thread's kDecItems consecutive
 * sorted elements: decode, admission threshold u, position r inside the own
 * queue, and the thread's running segmented reduction (admitted mode: minimum
 * of u_t - t; raw mode: number of kept requests). */
struct TileCtx {
  const unsigned long long* src;
  const PardSegConst* ktab;
  const uint32_t* seg_off;
  uint32_t n, ibits, imask, kshift;
  unsigned long long dmask;
  bool narrow;               /* deadline offsets have at most 29 bits */
  PlanHeader* hdr;
};

template <bool RAW>
__device__ __forceinline__ void tile_first_half(const TileCtx& T, uint64_t base, unsigned long long (&e)[kDecItems],
                                                uint32_t (&idx)[kDecItems], uint32_t (&u)[kDecItems],
                                                uint32_t (&r)[kDecItems], int32_t (&lv)[kDecItems],
                                                uint32_t& lheadbits, SegVal& run, PardSegConst& K,
                                                uint32_t& sstart, uint32_t& seg_first, bool& one_seg) {
  static_assert(kDecItems == 8, "two 32-byte loads per thread");
  const bool full = base + kDecItems <= T.n;
  if (full) {
    load4(T.src + base, e);
    load4(T.src + base + 4, e + 4);
  } else {
#pragma unroll
    for (int i = 0; i < kDecItems; ++i) e[i] = base + i < T.n ? T.src[base + i] : 0;
  }
  seg_first = (uint32_t)(e[0] >> T.kshift);
  /* most threads see one queue only: its constants are then loaded once */
  one_seg = full && seg_first == (uint32_t)(e[kDecItems - 1] >> T.kshift);
  K = T.ktab[seg_first];
  sstart = T.seg_off[seg_first];
  uint32_t cur_seg = seg_first;
  lheadbits = 0;
  run = seg_identity<RAW>();
  if ((K.narrow & kSegNoStage) && base < T.n) set_status(T.hdr, PARD_EDATA);   /* queue of a stage the pipeline lacks */
  if (one_seg && T.narrow && (K.narrow & (kSegNarrow | kSegNoStage)) == kSegNarrow) {
    /* one queue, and every quantity fits 32 bits: the common case */
    const uint32_t r0 = (uint32_t)base - sstart;
    const bool high_first = K.narrow & kSegHighFirst;
#pragma unroll
    for (int i = 0; i < kDecItems; ++i) {
      const uint32_t lo = (uint32_t)e[i], hi = (uint32_t)(e[i] >> 32);
      idx[i] = lo & T.imask;
      const uint32_t off = __funnelshift_r(lo, hi, T.ibits) & (uint32_t)T.dmask;
      const int32_t X = high_first ? (int32_t)K.A_rel - (int32_t)off : (int32_t)off - (int32_t)K.A_rel;
      const unsigned long long uu = (unsigned long long)(div_magic32((uint32_t)X, K.d_magic) + 1u) * K.cap;
      u[i] = X < 0 ? 0u : (uu > kUClamp ? kUClamp : (uint32_t)uu);
      r[i] = r0 + i;
      if (r[i] == 0) { run = seg_identity<RAW>(); run.head = 1; }
      lv[i] = run.m;
      lheadbits |= run.head << i;
      if (RAW) run.m += r[i] < u[i] ? 1 : 0;
      else run.m = min(run.m, (int32_t)u[i] - (int32_t)r[i]);
    }
    return;
  }
#pragma unroll
  for (int i = 0; i < kDecItems; ++i) {
    const uint64_t j = base + i;
    if (j < T.n) {
      idx[i] = (uint32_t)e[i] & T.imask;
      const unsigned long long off = (e[i] >> T.ibits) & T.dmask;
      if (!one_seg) {
        const uint32_t sg = (uint32_t)(e[i] >> T.kshift);
        if (sg != cur_seg) {
          cur_seg = sg;
          K = T.ktab[sg];
          sstart = T.seg_off[sg];
          if (K.narrow & kSegNoStage) set_status(T.hdr, PARD_EDATA);
        }
      }
      r[i] = (uint32_t)j - sstart;
      u[i] = threshold_u(slack_of(off, K), K);
    } else {
      idx[i] = 0; r[i] = 0; u[i] = kUClamp;                    /* acts as a head, never read */
    }
    if (r[i] == 0) { run = seg_identity<RAW>(); run.head = 1; }
    lv[i] = run.m;
    lheadbits |= run.head << i;
    if (RAW) run.m += (r[i] < u[i] && j < T.n) ? 1 : 0;
    else run.m = min(run.m, (int32_t)u[i] - (int32_t)r[i]);
  }
}

__device__ __forceinline__ TileCtx make_tile_ctx(const PlanHeader* hdr, const unsigned long long* buf_a,
                                                 const unsigned long long* buf_b, uint32_t n, uint32_t ibits,
                                                 const PardSegConst* ktab, const uint32_t* seg_off) {
  TileCtx T;
  const uint32_t dbits = hdr->dbits;
  T.src = (hdr->npass & 1) ? buf_b : buf_a;
  T.ktab = ktab;
  T.seg_off = seg_off;
  T.n = n;
  T.ibits = ibits;
  T.imask = (1u << ibits) - 1;                                 /* ibits <= 30 */
  T.kshift = ibits + dbits;                                    /* < 64 */
  T.dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  /* the offsets that occur, not the field they sit in (a call whose element format is fixed by
   * the host may have a wider field than its deadline spans need) */
  T.narrow = dbits <= 29 || (hdr->span_max >> 29) == 0;
  T.hdr = const_cast<PlanHeader*>(hdr);
  return T;
}

/* Inclusive segmented warp scan of the threads' values (in lane order). */
template <bool RAW>
__device__ __forceinline__ SegVal warp_scan(SegVal v, uint32_t lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    SegVal l;
    l.m = __shfl_up_sync(0xffffffffu, v.m, o);
    l.head = __shfl_up_sync(0xffffffffu, v.head, o);
    if (lane >= (uint32_t)o) v = seg_combine<RAW>(l, v);
  }
  return v;
}

/* Exclusive segmented scan of the tile aggregates by one block, eight tiles
 * per thread and round: carry[t] is the reduction over the elements that
 * precede tile t in the queue that is open at the start of tile t. */
template <bool RAW, int THREADS>
__device__ void tile_scan_block(const unsigned long long* tile_agg, uint32_t n_tiles, int32_t* carry) {
  constexpr int PER = 8, WARPS = THREADS / 32;
  __shared__ int32_t s_wm[32];
  __shared__ uint32_t s_wh[32];
  __shared__ int32_t s_cm;
  __shared__ uint32_t s_ch;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { s_cm = seg_identity<RAW>().m; s_ch = 0; }
  __syncthreads();
  for (uint32_t b = 0; b < n_tiles; b += THREADS * PER) {
    const uint32_t t0 = b + threadIdx.x * PER;
    SegVal v[PER];
    SegVal run = seg_identity<RAW>();
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      v[k] = t0 + k < n_tiles ? unpack_val(__ldcg(&tile_agg[t0 + k])) : seg_identity<RAW>();
      run = seg_combine<RAW>(run, v[k]);
    }
    const SegVal inc = warp_scan<RAW>(run, lane);
    SegVal exc;
    exc.m = __shfl_up_sync(0xffffffffu, inc.m, 1);
    exc.head = __shfl_up_sync(0xffffffffu, inc.head, 1);
    if (lane == 0) exc = seg_identity<RAW>();
    if (lane == 31) { s_wm[warp] = inc.m; s_wh[warp] = inc.head; }
    __syncthreads();
    if (warp == 0) {                        /* scan of the warp aggregates, led by the carry */
      SegVal a = seg_identity<RAW>();
      if (lane < WARPS) { a.m = s_wm[lane]; a.head = s_wh[lane]; }
      SegVal ai = warp_scan<RAW>(a, lane);
      SegVal ae;
      ae.m = __shfl_up_sync(0xffffffffu, ai.m, 1);
      ae.head = __shfl_up_sync(0xffffffffu, ai.head, 1);
      if (lane == 0) ae = seg_identity<RAW>();
      SegVal c0; c0.m = s_cm; c0.head = s_ch;
      ae = seg_combine<RAW>(c0, ae);
      const SegVal all = seg_combine<RAW>(c0, ai);
      __syncwarp();
      s_wm[lane] = ae.m; s_wh[lane] = ae.head;
      if (lane == 31) { s_cm = all.m; s_ch = all.head; }
    }
    __syncthreads();
    SegVal pre; pre.m = s_wm[warp]; pre.head = s_wh[warp];
    pre = seg_combine<RAW>(pre, exc);
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      if (t0 + k < n_tiles) carry[t0 + k] = pre.m;
      pre = seg_combine<RAW>(pre, v[k]);
    }
    __syncthreads();
  }
}

/* Tile aggregates: the segmented reduction over each tile of kDecTile sorted
 * elements.  Tiles are independent; the block that finishes last scans the
 * aggregates into the value carried into every tile, so that the decision
 * kernel never waits on another block. */
template <bool RAW>
__device__ void tile_agg_tiles(const PlanHeader* __restrict__ hdr, const unsigned long long* __restrict__ buf_a,
                               const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits,
                               const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ seg_off,
                               unsigned long long* __restrict__ tile_agg) {
  constexpr int WARPS = kDecThreads / 32;
  __shared__ int32_t s_wm[WARPS];
  __shared__ uint32_t s_wh[WARPS];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const TileCtx T = make_tile_ctx(hdr, buf_a, buf_b, n, ibits, ktab, seg_off);
  const uint32_t n_tiles = (n + kDecTile - 1) / kDecTile;
  for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const uint64_t base = (uint64_t)tile * kDecTile + (uint64_t)tid * kDecItems;
    unsigned long long e[kDecItems];
    uint32_t idx[kDecItems], u[kDecItems], r[kDecItems], lheadbits, sstart, seg_first;
    int32_t lv[kDecItems];
    SegVal run;
    PardSegConst K;
    bool one_seg;
    tile_first_half<RAW>(T, base, e, idx, u, r, lv, lheadbits, run, K, sstart, seg_first, one_seg);
    const SegVal inc = warp_scan<RAW>(run, lane);
    if (lane == 31) { s_wm[warp] = inc.m; s_wh[warp] = inc.head; }
    __syncthreads();
    if (tid == 0) {
      SegVal agg = seg_identity<RAW>();
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        SegVal a; a.m = s_wm[w]; a.head = s_wh[w];
        agg = seg_combine<RAW>(agg, a);
      }
      tile_agg[tile] = pack_val(agg, 0);
    }
    __syncthreads();
  }
}

/* Kept requests per queue -> first output slot of every queue, the number of
 * kCompactChunk-sized copy jobs before every queue, and the total.  One block,
 * eight queues per thread and round. */
template <int THREADS>
__device__ void kept_scan_block(const uint32_t* seg_kept, uint32_t n_seg, uint32_t* kept_base,
                                uint32_t* chunk_base, uint32_t* out_seg_kept, unsigned long long* out_n_kept) {
  constexpr int PER = 8, WARPS = THREADS / 32;
  __shared__ uint32_t s_a[32], s_b[32];
  __shared__ uint32_t s_ca, s_cb;
  if (threadIdx.x == 0) { s_ca = 0; s_cb = 0; }
  __syncthreads();
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  /* a thread's eight entries as two 16-byte accesses where the arrays allow it */
  const bool vec_in = ((uintptr_t)seg_kept & 15) == 0;
  const bool vec_out = (((uintptr_t)kept_base | (uintptr_t)chunk_base) & 15) == 0;
  const bool vec_user = out_seg_kept && ((uintptr_t)out_seg_kept & 15) == 0;
  for (uint32_t base = 0; base < n_seg + 1; base += THREADS * PER) {
    const uint32_t i0 = base + threadIdx.x * PER;
    uint32_t v[PER], c[PER], x = 0, y = 0;
    if (vec_in && i0 + PER <= n_seg) {
      /* (L2 loads here and in kept_move_jobs: inside k_scan_path other blocks of the same kernel wrote these) */
      const uint4 a = __ldcg(reinterpret_cast<const uint4*>(seg_kept + i0)), b = __ldcg(reinterpret_cast<const uint4*>(seg_kept + i0 + 4));
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int k = 0; k < PER; ++k) v[k] = i0 + k < n_seg ? __ldcg(&seg_kept[i0 + k]) : 0;
    }
    if (vec_user && i0 + PER <= n_seg) {
      *reinterpret_cast<uint4*>(out_seg_kept + i0) = make_uint4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<uint4*>(out_seg_kept + i0 + 4) = make_uint4(v[4], v[5], v[6], v[7]);
    } else if (out_seg_kept) {
#pragma unroll
      for (int k = 0; k < PER; ++k) if (i0 + k < n_seg) out_seg_kept[i0 + k] = v[k];
    }
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      c[k] = (v[k] + kCompactChunk - 1) / kCompactChunk;
      x += v[k];
      y += c[k];
    }
    const uint32_t tx = x, ty = y;
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t p = __shfl_up_sync(0xffffffffu, x, o), q = __shfl_up_sync(0xffffffffu, y, o);
      if (lane >= (uint32_t)o) { x += p; y += q; }
    }
    if (lane == 31) { s_a[warp] = x; s_b[warp] = y; }
    __syncthreads();
    if (warp == 0) {
      const uint32_t a = lane < WARPS ? s_a[lane] : 0u, b = lane < WARPS ? s_b[lane] : 0u;
      uint32_t ta = a, tb = b;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t p = __shfl_up_sync(0xffffffffu, ta, o), q = __shfl_up_sync(0xffffffffu, tb, o);
        if (lane >= (uint32_t)o) { ta += p; tb += q; }
      }
      s_a[lane] = ta - a;
      s_b[lane] = tb - b;
    }
    __syncthreads();
    uint32_t ea = s_ca + s_a[warp] + x - tx, eb = s_cb + s_b[warp] + y - ty;   /* exclusive, before this thread's queues */
    uint32_t oa[PER], ob[PER];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      oa[k] = ea; ob[k] = eb;
      ea += v[k];
      eb += c[k];
    }
    if (vec_out && i0 + PER <= n_seg + 1) {
      *reinterpret_cast<uint4*>(kept_base + i0) = make_uint4(oa[0], oa[1], oa[2], oa[3]);
      *reinterpret_cast<uint4*>(kept_base + i0 + 4) = make_uint4(oa[4], oa[5], oa[6], oa[7]);
      *reinterpret_cast<uint4*>(chunk_base + i0) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
      *reinterpret_cast<uint4*>(chunk_base + i0 + 4) = make_uint4(ob[4], ob[5], ob[6], ob[7]);
    } else {
#pragma unroll
      for (int k = 0; k < PER; ++k) if (i0 + k <= n_seg) { kept_base[i0 + k] = oa[k]; chunk_base[i0 + k] = ob[k]; }
    }
    __syncthreads();
    if (threadIdx.x == THREADS - 1) { s_ca = ea; s_cb = eb; }
    __syncthreads();
  }
  if (threadIdx.x == 0 && out_n_kept) *out_n_kept = s_ca;
}

/* Decision pass; one tile of kDecTile sorted elements per block, a thread owns
 * kDecItems consecutive elements.
 *
 * Admitted mode: c_r = min(r, r-1 + min_{t<r}(u_t - t)) by a segmented
 * exclusive prefix-min; raw mode: c_r = r, and the kept requests ahead in the
 * queue are counted by a segmented exclusive prefix-sum.  Either way the
 * number k_r of kept requests ahead in the own queue is known per request, and
 * a kept request's index goes to kept_tmp[first position of its queue + k_r]:
 * every queue's survivors end up contiguous, k_kept_move packs the queues. */
template <bool RAW>
__device__ void decide_tiles(const PlanHeader* __restrict__ hdr, const unsigned long long* __restrict__ buf_a,
         const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits,
         const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ seg_off,
         const uint32_t* __restrict__ win_off, const int32_t* __restrict__ carry,
         uint8_t* __restrict__ out_keep, long long* __restrict__ out_est, uint32_t* __restrict__ out_perm,
         uint32_t* __restrict__ kept_tmp, uint32_t* __restrict__ seg_kept) {
  constexpr int WARPS = kDecThreads / 32;
  __shared__ int32_t s_wm[WARPS];
  __shared__ uint32_t s_wh[WARPS];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const TileCtx T = make_tile_ctx(hdr, buf_a, buf_b, n, ibits, ktab, seg_off);
  const uint32_t n_tiles = (n + kDecTile - 1) / kDecTile;
  for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
  const uint64_t base = (uint64_t)tile * kDecTile + (uint64_t)tid * kDecItems;
  const bool full = base + kDecItems <= n;
  const int32_t tile_carry = __ldcg(&carry[tile]);       /* written by another block of this kernel */

  unsigned long long e[kDecItems];
  uint32_t idx[kDecItems], u[kDecItems], r[kDecItems], lheadbits, sstart, seg_first;
  int32_t lv[kDecItems];     /* reduction over this thread's earlier items of the same queue */
  SegVal run;
  PardSegConst K;
  bool one_seg;
  tile_first_half<RAW>(T, base, e, idx, u, r, lv, lheadbits, run, K, sstart, seg_first, one_seg);

  /* exclusive segmented scan of the threads' aggregates: warp, block, then the tile's carry */
  const SegVal inc = warp_scan<RAW>(run, lane);
  SegVal exc;
  exc.m = __shfl_up_sync(0xffffffffu, inc.m, 1);
  exc.head = __shfl_up_sync(0xffffffffu, inc.head, 1);
  if (lane == 0) exc = seg_identity<RAW>();
  if (lane == 31) { s_wm[warp] = inc.m; s_wh[warp] = inc.head; }
  __syncthreads();
  SegVal wprefix; wprefix.m = tile_carry; wprefix.head = 0;
#pragma unroll
  for (int w = 0; w < WARPS; ++w) {
    SegVal a; a.m = s_wm[w]; a.head = s_wh[w];
    if (w < (int)warp) wprefix = seg_combine<RAW>(wprefix, a);
  }
  exc = seg_combine<RAW>(wprefix, exc);

  /* admitted position, estimate, decision */
  uint32_t keepbits = 0;
  long long est[kDecItems];
  uint32_t cur_seg = seg_first;
  uint32_t send = seg_off[seg_first + 1];
  if (!one_seg) {
    K = ktab[seg_first];
    sstart = seg_off[seg_first];
  }
  /* A queue served high budget first keeps a prefix (thresholds fall along the queue while
   * positions rise); win_off holds the length of that prefix, and the admitted position is
   * the raw one capped by it. */
  uint32_t hb_kept = (K.narrow & kSegHighFirst) ? win_off[seg_first] : 0u;
  const bool fast = one_seg && T.narrow && (K.narrow & (kSegNarrow | kSegNoStage)) == kSegNarrow;
  if (fast) {
    const bool high_first = K.narrow & kSegHighFirst;
#pragma unroll
    for (int i = 0; i < kDecItems; ++i) {
      const bool local = (lheadbits >> i) & 1u;
      const int32_t pre = local ? lv[i] : (RAW ? lv[i] + exc.m : min(lv[i], exc.m));
      uint32_t c, ahead;
      if (RAW) {
        c = r[i];
        ahead = r[i] == 0 ? 0u : (uint32_t)pre;
      } else {
        c = r[i] == 0 ? 0u : (uint32_t)min((int32_t)r[i] - 1 + pre, (int32_t)r[i]);   /* both below 2^31 */
        if (high_first) c = min(r[i], hb_kept);
        ahead = c;
      }
      const uint32_t round = K.cap_magic ? div_magic32(c, K.cap_magic) : c;
      est[i] = K.A + (long long)((unsigned long long)round * (uint32_t)K.d);
      const uint32_t kept = c < u[i] ? 1u : 0u;
      keepbits |= kept << i;
      if (kept && kept_tmp) kept_tmp[sstart + ahead] = idx[i];
      if ((uint32_t)(base + i) + 1 == send) seg_kept[cur_seg] = ahead + kept;
    }
  } else
#pragma unroll
  for (int i = 0; i < kDecItems; ++i) {
    const bool valid = base + i < n;
    if (!one_seg && valid) {
      const uint32_t sg = (uint32_t)(e[i] >> T.kshift);
      if (sg != cur_seg) {
        cur_seg = sg;
        K = ktab[sg];
        sstart = seg_off[sg];
        send = seg_off[sg + 1];
        hb_kept = (K.narrow & kSegHighFirst) ? win_off[sg] : 0u;
      }
    }
    /* reduction over the earlier requests of the same queue */
    const bool local = (lheadbits >> i) & 1u;
    const int32_t pre = local ? lv[i] : (RAW ? lv[i] + exc.m : min(lv[i], exc.m));
    uint32_t c, ahead;            /* batch-slot position; kept requests ahead in the queue */
    if (RAW) {
      c = r[i];
      ahead = r[i] == 0 ? 0u : (uint32_t)pre;
    } else {
      if (r[i] == 0) {
        c = 0;
      } else {
        const int64_t cc = (int64_t)r[i] - 1 + pre;               /* r-1 + min over t < r of (u_t - t) */
        c = cc < (int64_t)r[i] ? (uint32_t)cc : r[i];
      }
      if (K.narrow & kSegHighFirst) c = min(r[i], hb_kept);
      ahead = c;
    }
    const uint32_t round = K.cap_magic ? div_magic32(c, K.cap_magic) : c;     /* floor(c / cap) */
    est[i] = K.A + (long long)round * K.d;
    const uint32_t kept = (c < u[i] && valid) ? 1u : 0u;
    keepbits |= kept << i;
    if (kept && kept_tmp) kept_tmp[sstart + ahead] = idx[i];
    /* the last request of a queue knows the queue's kept count */
    if (valid && (uint32_t)(base + i) + 1 == send) seg_kept[cur_seg] = ahead + kept;
  }

  if (full) {
    if (out_keep) {
      /* bit k of a nibble -> byte k of a word */
      const uint32_t klo = ((keepbits & 15u) * 0x00204081u) & 0x01010101u;
      const uint32_t khi = (((keepbits >> 4) & 15u) * 0x00204081u) & 0x01010101u;
      *reinterpret_cast<uint2*>(out_keep + base) = make_uint2(klo, khi);
    }
    if (out_est) {
      store4(out_est + base, est[0], est[1], est[2], est[3]);
      store4(out_est + base + 4, est[4], est[5], est[6], est[7]);
    }
    if (out_perm)
      store4(out_perm + base, idx[0] | ((unsigned long long)idx[1] << 32),
             idx[2] | ((unsigned long long)idx[3] << 32), idx[4] | ((unsigned long long)idx[5] << 32),
             idx[6] | ((unsigned long long)idx[7] << 32));
  } else {
#pragma unroll
    for (int i = 0; i < kDecItems; ++i)
      if (base + i < n) {
        if (out_keep) out_keep[base + i] = (keepbits >> i) & 1u;
        if (out_est) out_est[base + i] = est[i];
        if (out_perm) out_perm[base + i] = idx[i];
      }
  }
  __syncthreads();
  }
}

__global__ void __launch_bounds__(1024)
k_kept_scan(const uint32_t* __restrict__ seg_kept, uint32_t n_seg, uint32_t* __restrict__ kept_base,
            uint32_t* __restrict__ chunk_base, uint32_t* __restrict__ out_seg_kept,
            unsigned long long* __restrict__ out_n_kept) {
  pdl_wait();
  kept_scan_block<1024>(seg_kept, n_seg, kept_base, chunk_base, out_seg_kept, out_n_kept);
}

/* ------------------------------------------------------------------------ */
/* window tables: the decision pass without a scan                           */
/* ------------------------------------------------------------------------ */
/* Inside one queue the threshold u is a step function of the deadline: every
 * request whose deadline falls into the same batch window
 *     b = floor((D - A) / d)
 * has u = cap * (b + 1) (requests with D < A have u = 0).  The running minimum
 * of u_t - t that fixes the admitted position therefore only changes at the
 * window boundaries: with P[b] = number of requests of the queue whose window
 * is below b, the minimum over a complete window b is u(b) - (P[b+1] - 1), and
 *     E[b] = minimum over all complete runs before window b
 * is a prefix minimum over at most a few thousand windows per queue.  A request
 * at queue position r in window b then has
 *     min_{t<r}(u_t - t) = min(E[b], u(b) - (r - 1) if r > P[b])
 * with no reference to any other request.  P comes from a search in the sorted
 * elements (one warp per window), E and the raw-mode kept counts Kp from a
 * per-queue prefix pass over the windows.  Queues with more than kWinMaxPerSeg
 * windows, or more windows in total than the table holds, make the call fall
 * back to the scan kernels (same results). */
struct __align__(16) WinEntry {
  uint32_t P;      /* requests of the queue in earlier windows (or expired)       */
  int32_t E;       /* min of u_t - t over those requests, kWinInf if there is none */
  uint32_t Kp;     /* raw mode: kept requests among them                          */
  uint32_t pad;
};
constexpr int32_t kWinInf = 0x7fffffff;
constexpr uint32_t kWinMaxPerSeg = 4096;
constexpr uint32_t kManyQueues = 8192;     /* from this many queues on a lane, not a warp, handles a queue in k_seg_win_many */
constexpr uint32_t kWinLongQueue = 8192;   /* above this a window boundary is searched by a whole warp, else by one lane */


/* u of window b (the saturation of threshold_u) */
__device__ __forceinline__ uint32_t win_u(uint32_t b, uint32_t cap) {
  const unsigned long long u = (unsigned long long)(b + 1) * cap;
  return u > kUClamp ? kUClamp : (uint32_t)u;
}

/* window of a non-negative X = D - A */
__device__ __forceinline__ unsigned long long win_of(unsigned long long X, const PardSegConst& K) {
  if ((X >> 32) == 0 && K.d_magic) return div_magic32((uint32_t)X, K.d_magic);
  return X / (unsigned long long)K.d;
}

/* One warp per queue: its first and last sorted position (a 32-ary search for
 * the segment id in the elements' upper bits), the number of its batch windows
 * (from its latest deadline), and a range of table entries for them, taken
 * from a shared counter; every entry is labelled with its queue.  If the
 * table cannot hold the windows the call falls back to the scan kernels. */
__global__ void __launch_bounds__(256)
k_seg_win(PlanHeader* hdr, const unsigned long long* __restrict__ buf_a,
          const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits, uint32_t n_seg,
          const PardSegConst* __restrict__ ktab, uint32_t* __restrict__ seg_off,
          uint32_t* __restrict__ out_seg_off, uint32_t* __restrict__ win_off, uint32_t* __restrict__ win_cnt,
          uint32_t* __restrict__ win_own, uint32_t* __restrict__ win_big, uint32_t capacity,
          uint32_t force_scan, const uint32_t* __restrict__ hist, uint32_t sbits, uint32_t local_candidate,
          uint32_t tables, uint32_t* __restrict__ seg_kept) {
  pdl_wait();
  const uint32_t s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t lane = threadIdx.x & 31;
  if (s > n_seg) return;                         /* whole warps leave together */
  if (s == 0 && lane == 0 && force_scan) hdr->use_scan = 1;
  uint32_t lo[2] = {0, 0};
  const bool wide = hdr->wide != 0 || hdr->aborted != 0;   /* nothing usable was sorted */
  const unsigned long long* src = (hdr->npass & 1) ? buf_b : buf_a;
  const uint32_t dbits = hdr->dbits;
  const uint32_t npass = hdr->npass;
  const uint32_t top_bits = npass ? hdr->keybits - 8 * (npass - 1) : 0;   /* width of the last pass's digit */
  if (!wide && n > 0 && npass && sbits <= top_bits && !sort_is_local(hdr, local_candidate)) {
    /* the segment id is the upper part of the last pass's digit: the queue starts where the
     * digits below (s << (top_bits - sbits)) end, and the digit counts of that pass are known */
    const uint32_t* h = hist + (npass - 1) * kBins;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const uint32_t limit = min((s + q) << (top_bits - sbits), (uint32_t)kBins);
      uint32_t sum = 0;
      for (uint32_t d = lane; d < limit; d += 32) sum += h[d];
      for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      lo[q] = sum;
    }
  } else if (!wide && n > 0) {
    const uint32_t kshift = ibits + dbits;
    uint32_t hi[2] = {n, n};                     /* answers: first element whose segment id is >= s, >= s+1 */
    while (lo[0] < hi[0] || lo[1] < hi[1]) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        if (lo[q] < hi[q]) {                     /* uniform across the warp */
          const uint32_t span = hi[q] - lo[q];
          const uint32_t p = lo[q] + (uint32_t)(((unsigned long long)(lane + 1) * span) / 33u);   /* lo <= p < hi */
          const bool less = (uint32_t)(__ldg(src + p) >> kshift) < s + q;
          const uint32_t k = __popc(__ballot_sync(0xffffffffu, less));   /* lanes 0..k-1 saw a smaller id */
          const uint32_t p_below = __shfl_sync(0xffffffffu, p, k > 0 ? k - 1 : 0);
          const uint32_t p_at = __shfl_sync(0xffffffffu, p, k < 32 ? k : 31);
          if (k > 0) lo[q] = p_below + 1;
          if (k < 32) hi[q] = p_at;
        }
      }
    }
  }
  if (lane == 0) {
    seg_off[s] = lo[0];
    if (out_seg_off) out_seg_off[s] = lo[0];
  }
  if (s == n_seg || !tables) return;             /* the boundaries are all the sequential rules need */
  /* A queue served high budget first needs no window table: its thresholds fall along the
   * queue while the positions rise, so the kept requests are a prefix of it.  The prefix
   * length (first position r with r >= u_r) is found by a 32-ary search and handed to the
   * decision kernels in win_off. */
  if (lo[1] > lo[0] && !wide && (ktab[s].narrow & (kSegHighFirst | kSegNoStage)) == kSegHighFirst) {
    const PardSegConst K = ktab[s];
    const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
    uint32_t a = lo[0], b = lo[1];
    while (a < b) {                                /* uniform across the warp */
      const uint32_t span = b - a;
      const uint32_t p = a + (uint32_t)(((unsigned long long)(lane + 1) * span) / 33u);   /* a <= p < b */
      const bool kept = p - lo[0] < threshold_u(slack_of((__ldg(src + p) >> ibits) & dmask, K), K);
      const uint32_t k = __popc(__ballot_sync(0xffffffffu, kept));   /* lanes 0..k-1 probe kept requests */
      const uint32_t p_below = __shfl_sync(0xffffffffu, p, k > 0 ? k - 1 : 0);
      const uint32_t p_at = __shfl_sync(0xffffffffu, p, k < 32 ? k : 31);
      if (k > 0) a = p_below + 1;
      if (k < 32) b = p_at;
    }
    if (lane == 0) { win_off[s] = a - lo[0]; win_cnt[s] = 0; seg_kept[s] = a - lo[0]; }   /* the kept prefix is the queue's kept count */
    return;
  }
  /* batch windows of the queue: 0..b_last of its requests, plus the end marker */
  uint32_t w = 0, first = 0;
  if (lane == 0 && lo[1] > lo[0] && !wide) {
    const PardSegConst K = ktab[s];
    if (K.narrow & kSegNoStage) {
      set_status(hdr, PARD_EDATA);               /* requests queued at a stage the pipeline lacks */
    } else {
      const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
      const long long X = (long long)((src[lo[1] - 1] >> ibits) & dmask) - K.A_rel;   /* latest deadline of the queue */
      const unsigned long long nb = X < 0 ? 0 : win_of((unsigned long long)X, K) + 1;
      if (nb >= kWinMaxPerSeg) {
        hdr->use_scan = 1;
      } else {
        w = (uint32_t)nb + 1;
        const unsigned long long at = atomicAdd(&hdr->win_total, (unsigned long long)w);
        if (at + w > (unsigned long long)capacity) { hdr->use_scan = 1; w = 0; }
        else first = (uint32_t)at;
      }
    }
  }
  w = __shfl_sync(0xffffffffu, w, 0);
  first = __shfl_sync(0xffffffffu, first, 0);
  if (lane == 0) { win_off[s] = first; win_cnt[s] = w; }
  for (uint32_t e = lane; e < w; e += 32) win_own[first + e] = s;
  if (w && lo[1] - lo[0] > kWinLongQueue) {      /* long queue: list its entries for the warp-wide search */
    uint32_t at = 0;
    if (lane == 0) at = atomicAdd(&hdr->big_total, w);
    at = __shfl_sync(0xffffffffu, at, 0);
    for (uint32_t e = lane; e < w; e += 32) win_big[at + e] = first + e;
  }
}

/* The same for calls with thousands of queues, where a warp per queue means more probes than a
 * pass over the elements: here a LANE owns a queue.  Lane i of a warp finds the first element
 * of queue s0 + i by a plain binary search (the lanes' early probes coincide, so they cost one
 * sector), takes the end of its queue from lane i + 1, and the warp draws its queues' table
 * entries from the shared counter with one addition. */
__global__ void __launch_bounds__(256)
k_seg_win_many(PlanHeader* hdr, const unsigned long long* __restrict__ buf_a,
               const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits, uint32_t n_seg,
               const PardSegConst* __restrict__ ktab, uint32_t* __restrict__ seg_off,
               uint32_t* __restrict__ out_seg_off, uint32_t* __restrict__ win_off, uint32_t* __restrict__ win_cnt,
               uint32_t* __restrict__ win_own, uint32_t* __restrict__ win_big, uint32_t capacity,
               uint32_t force_scan, uint32_t tables, uint32_t* __restrict__ seg_kept) {
  pdl_wait();
  const uint32_t warp_g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t s0 = warp_g * 31u;              /* queues s0 .. s0+30, boundaries s0 .. s0+31 */
  if (s0 > n_seg) return;                        /* whole warps leave together */
  if (warp_g == 0 && lane == 0 && force_scan) hdr->use_scan = 1;
  const uint32_t s = s0 + lane;
  const bool wide = hdr->wide != 0 || hdr->aborted != 0;   /* nothing usable was sorted */
  const unsigned long long* src = (hdr->npass & 1) ? buf_b : buf_a;
  const uint32_t dbits = hdr->dbits;
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  uint32_t lo = 0;                               /* first element whose segment id is >= s */
  if (!wide && n > 0 && s <= n_seg) {
    const uint32_t kshift = ibits + dbits;
    uint32_t hi = n;
    while (lo < hi) {
      const uint32_t mid = lo + (hi - lo) / 2;
      if ((uint32_t)(__ldg(src + mid) >> kshift) < s) lo = mid + 1; else hi = mid;
    }
  }
  if (lane < 31 && s <= n_seg) {                 /* boundary s0+31 belongs to the next warp */
    seg_off[s] = lo;
    if (out_seg_off) out_seg_off[s] = lo;
  }
  const uint32_t end = __shfl_down_sync(0xffffffffu, lo, 1);
  if (!tables) return;                           /* the boundaries are all the sequential rules need */
  const bool mine = lane < 31 && s < n_seg;
  uint32_t w = 0;
  bool high_first = false;
  if (mine && end > lo && !wide) {
    const PardSegConst K = ktab[s];
    if (K.narrow & kSegNoStage) {
      set_status(hdr, PARD_EDATA);               /* requests queued at a stage the pipeline lacks */
    } else if (K.narrow & kSegHighFirst) {       /* length of the kept prefix (see k_seg_win) */
      high_first = true;
      uint32_t a = lo, b = end;
      while (a < b) {
        const uint32_t mid = a + (b - a) / 2;
        if (mid - lo < threshold_u(slack_of((__ldg(src + mid) >> ibits) & dmask, K), K)) a = mid + 1; else b = mid;
      }
      win_off[s] = a - lo;
      seg_kept[s] = a - lo;                      /* the kept prefix is the queue's kept count */
      win_cnt[s] = 0;
    } else {
      const long long X = (long long)((src[end - 1] >> ibits) & dmask) - K.A_rel;   /* latest deadline of the queue */
      const unsigned long long nb = X < 0 ? 0 : win_of((unsigned long long)X, K) + 1;
      if (nb >= kWinMaxPerSeg) hdr->use_scan = 1;
      else w = (uint32_t)nb + 1;
    }
  }
  uint32_t incl = w;                             /* the warp's queues take consecutive table entries */
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= (uint32_t)o) incl += t;
  }
  unsigned long long base = 0;
  if (lane == 31 && incl) base = atomicAdd(&hdr->win_total, (unsigned long long)incl);
  base = __shfl_sync(0xffffffffu, base, 31);
  const unsigned long long first64 = base + incl - w;        /* 64 bits: the counter may pass 2^32 on legal input */
  if (w && first64 + w > (unsigned long long)capacity) { hdr->use_scan = 1; w = 0; }
  const uint32_t first = w ? (uint32_t)first64 : 0u;
  if (mine && !high_first) { win_off[s] = w ? first : 0u; win_cnt[s] = w; }
  for (uint32_t e = 0; e < w; ++e) win_own[first + e] = s;
  if (w && end - lo > kWinLongQueue) {           /* long queue: list its entries for the warp-wide search */
    const uint32_t at = atomicAdd(&hdr->big_total, w);
    for (uint32_t e = 0; e < w; ++e) win_big[at + e] = first + e;
  }
}

/* E and Kp of the table entries of one queue: the warp runs over the queue's windows, 32 at a
 * time. */
__device__ __forceinline__ uint32_t win_prefix_warp(uint32_t s, const PardSegConst* __restrict__ ktab,
                                                const uint32_t* __restrict__ win_off,
                                                const uint32_t* __restrict__ win_cnt, WinEntry* __restrict__ wtab,
                                                uint32_t lane, uint32_t raw) {
  const uint32_t w0 = win_off[s], cnt = win_cnt[s];
  if (cnt == 0) return 0xffffffffu;              /* no table (served high budget first, or no such stage) */
  const uint32_t cap = ktab[s].cap;
  WinEntry* tab = wtab + w0;
  const uint32_t P0 = __ldcg(&tab[0].P);          /* other blocks may have written the P (long queues) */
  int32_t e_carry = P0 > 0 ? -(int32_t)(P0 - 1) : kWinInf;     /* the expired run: u = 0 */
  uint32_t k_carry = 0;
  if (lane == 0) { tab[0].E = e_carry; tab[0].Kp = 0; }
  for (uint32_t b0 = 0; b0 + 1 < cnt; b0 += 32) {              /* windows b0..b0+31 -> entries b0+1.. */
    const uint32_t b = b0 + lane;
    int32_t val = kWinInf;
    uint32_t kept = 0;
    if (b + 1 < cnt) {
      const uint32_t p = __ldcg(&tab[b].P), q = __ldcg(&tab[b + 1].P);
      if (q > p) {
        const uint32_t u = win_u(b, cap);
        val = (int32_t)u - (int32_t)(q - 1);
        const uint32_t top = u < q ? u : q;
        kept = top > p ? top - p : 0;
      }
    }
    for (int o = 1; o < 32; o <<= 1) {
      const int32_t v2 = __shfl_up_sync(0xffffffffu, val, o);
      const uint32_t k2 = __shfl_up_sync(0xffffffffu, kept, o);
      if (lane >= (uint32_t)o) { val = min(val, v2); kept += k2; }
    }
    const int32_t e_inc = min(e_carry, val);
    const uint32_t k_inc = k_carry + kept;
    if (b + 1 < cnt) { tab[b + 1].E = e_inc; tab[b + 1].Kp = k_inc; }
    e_carry = __shfl_sync(0xffffffffu, e_inc, 31);
    k_carry = __shfl_sync(0xffffffffu, k_inc, 31);
  }
  /* With the table complete the queue's number of kept requests is known before any request has
   * been decided: the last entry closes the queue (P = its length n), the running Kp counts the
   * kept requests under raw positions, and the running E is the minimum of u_t - t over the whole
   * queue, so that the admitted count behind the last request is n - 1 + min(E, 1). */
  const uint32_t n_q = __ldcg(&tab[cnt - 1].P);
  return n_q == 0 ? 0u : (raw ? k_carry : (uint32_t)((int32_t)n_q - 1 + min(e_carry, 1)));
}

/* The window tables.  P of every entry: a search in the queue's sorted elements, by one lane
 * (short queue) or by a whole warp with 32 probes per step (long queue).  (Counting finished
 * entries per queue so that the last finisher could run the queue's prefix pass in the same
 * kernel was tried: the fence and the atomic per entry cost more than the launch they saved
 * once there are thousands of queues.) */
__global__ void __launch_bounds__(256)
k_win_bounds(const PlanHeader* __restrict__ hdr, const unsigned long long* __restrict__ buf_a,
             const unsigned long long* __restrict__ buf_b, uint32_t ibits, uint32_t n_seg,
             const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ seg_off,
             const uint32_t* __restrict__ win_off, const uint32_t* __restrict__ win_cnt,
             const uint32_t* __restrict__ win_own, const uint32_t* __restrict__ win_big,
             uint32_t* __restrict__ win_done, WinEntry* __restrict__ wtab, uint32_t raw, uint32_t* __restrict__ seg_kept) {
  pdl_wait();
  if (hdr->use_scan || hdr->wide || hdr->aborted) return;
  const uint32_t lane = threadIdx.x & 31;
  const unsigned long long* src = (hdr->npass & 1) ? buf_b : buf_a;
  const uint32_t dbits = hdr->dbits;
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  /* entries of short queues: one lane each, plain binary search */
  {
    /* without use_scan every request for entries was granted, so the counter is within the table */
    const uint32_t total = (uint32_t)hdr->win_total, step = gridDim.x * blockDim.x;
    for (uint32_t e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += step) {
      const uint32_t s = win_own[e];
      uint32_t lo = seg_off[s], hi = seg_off[s + 1];
      if (hi - lo > kWinLongQueue) continue;
      const uint32_t first = lo;
      const long long thr = ktab[s].A_rel + (long long)(e - win_off[s]) * ktab[s].d;
      while (lo < hi) {
        const uint32_t mid = lo + (hi - lo) / 2;
        if ((long long)((__ldg(src + mid) >> ibits) & dmask) < thr) lo = mid + 1; else hi = mid;
      }
      wtab[e].P = lo - first;
    }
  }
  /* entries of long queues: one warp each, 32 probes per step */
  const uint32_t total = hdr->big_total, step = (gridDim.x * blockDim.x) >> 5;
  for (uint32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < total; i += step) {   /* whole warps stay together */
    const uint32_t e = win_big[i];
    const uint32_t s = win_own[e], b = e - win_off[s];
    const PardSegConst K = ktab[s];
    const long long thr = K.A_rel + (long long)b * K.d;     /* window >= b  <=>  deadline offset >= thr */
    uint32_t lo = seg_off[s], hi = seg_off[s + 1];
    const uint32_t first = lo;
    while (lo < hi) {
      const uint32_t span = hi - lo;
      const uint32_t p = lo + (uint32_t)(((unsigned long long)(lane + 1) * span) / 33u);
      const bool less = (long long)((__ldg(src + p) >> ibits) & dmask) < thr;
      const uint32_t k = __popc(__ballot_sync(0xffffffffu, less));
      const uint32_t p_below = __shfl_sync(0xffffffffu, p, k > 0 ? k - 1 : 0);
      const uint32_t p_at = __shfl_sync(0xffffffffu, p, k < 32 ? k : 31);
      if (k > 0) lo = p_below + 1;
      if (k < 32) hi = p_at;
    }
    /* a long queue has few hundred entries at most, spread over as many warps: they are counted,
     * and the warp that stores the last one goes on to the queue's prefix pass */
    uint32_t last = 0;
    if (lane == 0) {
      wtab[e].P = lo - first;
      __threadfence();
      last = atomicAdd(&win_done[s], 1u) + 1 == win_cnt[s] ? 1u : 0u;
    }
    if (__shfl_sync(0xffffffffu, last, 0)) {
      __threadfence();
      const uint32_t kept = win_prefix_warp(s, ktab, win_off, win_cnt, wtab, lane, raw);
      if (lane == 0 && kept != 0xffffffffu) seg_kept[s] = kept;
    }
  }
}

/* E and Kp of the table entries of the short queues: one warp per queue runs over its windows,
 * 32 at a time. */
__global__ void __launch_bounds__(256)
k_win_prefix(const PlanHeader* __restrict__ hdr, uint32_t n_seg, const PardSegConst* __restrict__ ktab,
             const uint32_t* __restrict__ seg_off, const uint32_t* __restrict__ win_off,
             const uint32_t* __restrict__ win_cnt, WinEntry* __restrict__ wtab, uint32_t raw,
             uint32_t* __restrict__ seg_kept) {
  pdl_wait();
  if (hdr->use_scan || hdr->wide || hdr->aborted) return;
  const uint32_t s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (s >= n_seg) return;                          /* whole warps leave together */
  if (seg_off[s + 1] - seg_off[s] > kWinLongQueue) return;   /* done by k_win_bounds */
  const uint32_t kept = win_prefix_warp(s, ktab, win_off, win_cnt, wtab, threadIdx.x & 31, raw);
  if ((threadIdx.x & 31) == 0 && kept != 0xffffffffu) seg_kept[s] = kept;     /* the queue's kept count, known before the decision */
}

/* The window tables of a call with few queues, from the counts k_pack took: P is the running sum
 * of a queue's counts, E and Kp follow as in the searched tables, and the queues' first positions
 * are the running sum of their lengths.  One block; a warp per queue.  Runs before the sort: the
 * counts do not depend on the order of the elements. */
__global__ void __launch_bounds__(1024)
k_win_from_counts(PlanHeader* hdr, uint32_t n_seg, const PardSegConst* __restrict__ ktab,
                  const uint32_t* __restrict__ whist, const uint32_t* __restrict__ win_off,
                  const uint32_t* __restrict__ win_cnt, WinEntry* __restrict__ wtab,
                  uint32_t* __restrict__ seg_off, uint32_t* __restrict__ out_seg_off, uint32_t raw,
                  uint32_t* __restrict__ seg_kept, uint32_t* __restrict__ out_seg_kept,
                  uint32_t* __restrict__ kept_base, unsigned long long* __restrict__ out_n_kept,
                  const uint32_t* __restrict__ hist, uint32_t sbits) {
  pdl_wait();
  __shared__ uint32_t s_len[kHistSegs], s_kept[kHistSegs];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  /* entry 0 left uncounted by k_pack (same condition there): the queue's length, from the last
   * pass's digit counts, minus its other entries */
  const uint32_t npass = hdr->npass;
  const uint32_t top_bits = npass ? hdr->keybits - 8 * (npass - 1) : 0;
  const bool derive = npass > 0 && sbits <= top_bits;
  for (uint32_t q = warp; q < n_seg; q += blockDim.x / 32) {
    const uint32_t off = win_off[q], cnt = win_cnt[q];
    uint32_t entry0 = 0;
    if (derive) {
      const uint32_t* h = hist + (npass - 1) * kBins;
      const uint32_t d0 = min(q << (top_bits - sbits), (uint32_t)kBins), d1 = min((q + 1) << (top_bits - sbits), (uint32_t)kBins);
      uint32_t len = 0, others = 0;
      for (uint32_t d = d0 + lane; d < d1; d += 32) len += h[d];
      for (uint32_t b = 1 + lane; b < cnt; b += 32) others += whist[off + b];
      for (int o = 16; o; o >>= 1) {
        len += __shfl_xor_sync(0xffffffffu, len, o);
        others += __shfl_xor_sync(0xffffffffu, others, o);
      }
      entry0 = len - others;
    }
    uint32_t run = 0;
    for (uint32_t b0 = 0; b0 < cnt; b0 += 32) {
      const uint32_t b = b0 + lane;
      uint32_t x = b < cnt ? whist[off + b] : 0u;
      if (derive && b == 0) x = entry0;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= (uint32_t)o) x += y;
      }
      if (b < cnt) wtab[off + b].P = run + x;        /* requests of the queue up to and including entry b's */
      run += __shfl_sync(0xffffffffu, x, 31);
    }
    if (lane == 0) s_len[q] = run;
    __threadfence_block();
    __syncwarp();
    /* P as the decision reads it: entry b = requests in windows below b, i.e. the sum up to entry b */
    const uint32_t kept = win_prefix_warp(q, ktab, win_off, win_cnt, wtab, lane, raw);
    if (lane == 0) s_kept[q] = kept == 0xffffffffu ? 0u : kept;      /* the queue's kept count, known before the sort */
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool scan = hdr->use_scan != 0;                /* then the scan path counts and packs */
    uint32_t first = 0, kept = 0;
    for (uint32_t q = 0; q < n_seg; ++q) {
      seg_off[q] = first;
      if (out_seg_off) out_seg_off[q] = first;
      first += s_len[q];
      if (!scan) {
        kept_base[q] = kept;
        seg_kept[q] = s_kept[q];
        if (out_seg_kept) out_seg_kept[q] = s_kept[q];
        kept += s_kept[q];
      }
    }
    seg_off[n_seg] = first;
    if (out_seg_off) out_seg_off[n_seg] = first;
    if (!scan && out_n_kept) *out_n_kept = kept;
  }
}

/* Decision pass from the window tables: every request on its own.  HF: some
 * queue may be served high budget first (the caller gave priorities). */
template <bool RAW, bool HF>
__global__ void __launch_bounds__(kDecThreads, 8)
k_decide_win(const PlanHeader* __restrict__ hdr, const unsigned long long* __restrict__ buf_a,
             const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits,
             const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ seg_off,
             const uint32_t* __restrict__ win_off, const uint32_t* __restrict__ win_cnt,
             const WinEntry* __restrict__ wtab,
             uint8_t* __restrict__ out_keep, long long* __restrict__ out_est,
             uint32_t* __restrict__ out_perm, uint32_t* __restrict__ kept_dst, const uint32_t* __restrict__ kept_off,
             uint32_t* __restrict__ seg_kept) {
  /* kept_dst / kept_off: where the survivors of a queue go.  Normally the queue's own range of a
   * scratch array (kept_off = the queues' first positions), packed afterwards; with counted
   * tables the queues' kept counts are known beforehand and the survivors go straight to their
   * final place (kept_dst = the output, kept_off = the queues' output offsets, seg_kept = NULL). */
  pdl_wait();
  if (hdr->use_scan || hdr->wide || hdr->aborted) return;
  const TileCtx T = make_tile_ctx(hdr, buf_a, buf_b, n, ibits, ktab, seg_off);
  const uint64_t base = ((uint64_t)blockIdx.x * kDecThreads + threadIdx.x) * kDecItems;
  if (base >= n) return;
  const bool full = base + kDecItems <= n;
  unsigned long long e[kDecItems];
  if (full) {
    load4(T.src + base, e);
    load4(T.src + base + 4, e + 4);
  } else {
#pragma unroll
    for (int i = 0; i < kDecItems; ++i) e[i] = base + i < n ? T.src[base + i] : 0;
  }
  uint32_t cur_seg = (uint32_t)(e[0] >> T.kshift);
  PardSegConst K = ktab[cur_seg];
  uint32_t sstart = seg_off[cur_seg], send = seg_off[cur_seg + 1], woff = win_off[cur_seg], wcnt = win_cnt[cur_seg];
  uint32_t koff = kept_dst ? kept_off[cur_seg] : 0u;
  const bool narrow = T.narrow && (K.narrow & (kSegNarrow | kSegNoStage)) == kSegNarrow && full &&
                      cur_seg == (uint32_t)(e[kDecItems - 1] >> T.kshift);

  uint32_t keepbits = 0, idx[kDecItems];
  long long est[kDecItems];
#pragma unroll
  for (int i = 0; i < kDecItems; ++i) {
    const uint64_t j = base + i;
    const bool valid = j < n;
    uint32_t c = 0, ahead = 0, kept = 0;
    idx[i] = (uint32_t)e[i] & T.imask;
    if (valid) {
      long long X;
      if (narrow) {
        const int32_t off = (int32_t)(__funnelshift_r((uint32_t)e[i], (uint32_t)(e[i] >> 32), T.ibits) & (uint32_t)T.dmask);
        X = (HF && (K.narrow & kSegHighFirst)) ? (int32_t)K.A_rel - off : off - (int32_t)K.A_rel;
      } else {
        const uint32_t sg = (uint32_t)(e[i] >> T.kshift);
        if (sg != cur_seg) {
          cur_seg = sg;
          K = ktab[sg];
          sstart = seg_off[sg];
          koff = kept_dst ? kept_off[sg] : 0u;
          send = seg_off[sg + 1];
          woff = win_off[sg];
          wcnt = win_cnt[sg];
        }
        X = HF ? slack_of((e[i] >> T.ibits) & T.dmask, K) : (long long)((e[i] >> T.ibits) & T.dmask) - K.A_rel;
      }
      const uint32_t r = (uint32_t)j - sstart;
      uint32_t u = 0;
      if (HF && (K.narrow & kSegHighFirst)) {                 /* the kept requests are the first woff of the queue */
        u = threshold_u(X, K);
        ahead = min(r, woff);
        c = RAW ? r : ahead;
      } else if (X >= 0) {                            /* window b of the request and its table entry */
        const unsigned long long b64 = win_of((unsigned long long)X, K);
        /* The queue's table has an entry for every window up to its latest deadline's.  A queue
         * without a table (input errors: a stage its pipeline lacks, constants left at their
         * defaults) must not index one: its requests count as dropped, the call reports PARD_EDATA. */
        if (b64 >= (unsigned long long)wcnt) {
          set_status(T.hdr, PARD_EDATA);
          est[i] = K.A;
          if (seg_kept && (uint32_t)j + 1 == send) seg_kept[cur_seg] = 0;
          continue;
        }
        const uint32_t b = (uint32_t)b64;
        u = win_u(b, K.cap);
        const WinEntry w = wtab[woff + b];
        if (RAW) {
          const uint32_t top = r < u ? r : u;
          ahead = w.Kp + (top > w.P ? top - w.P : 0);
          c = r;
        } else {
          /* min over t < r of (u_t - t); values above 1 cannot lower the position */
          int32_t m = w.E;
          if (r > w.P) m = min(m, (int32_t)u - (int32_t)(r - 1));
          c = r == 0 ? 0u : r - 1 + (uint32_t)min(m, 1);
          ahead = c;
        }
      } else {                                        /* deadline before even position 0 completes */
        c = RAW ? r : 0u;
      }
      kept = c < u ? 1u : 0u;
      const uint32_t round = K.cap_magic ? div_magic32(c, K.cap_magic) : c;
      est[i] = K.A + (long long)((unsigned long long)round * (unsigned long long)K.d);
      if (kept && kept_dst) kept_dst[koff + ahead] = idx[i];
      if (seg_kept && (uint32_t)j + 1 == send) seg_kept[cur_seg] = ahead + kept;   /* the last request knows the queue's count */
    }
    keepbits |= kept << i;
  }
  if (full) {
    if (out_keep) {
      const uint32_t klo = ((keepbits & 15u) * 0x00204081u) & 0x01010101u;
      const uint32_t khi = (((keepbits >> 4) & 15u) * 0x00204081u) & 0x01010101u;
      *reinterpret_cast<uint2*>(out_keep + base) = make_uint2(klo, khi);
    }
    if (out_est) {
      store4(out_est + base, est[0], est[1], est[2], est[3]);
      store4(out_est + base + 4, est[4], est[5], est[6], est[7]);
    }
    if (out_perm)
      store4(out_perm + base, idx[0] | ((unsigned long long)idx[1] << 32),
             idx[2] | ((unsigned long long)idx[3] << 32), idx[4] | ((unsigned long long)idx[5] << 32),
             idx[6] | ((unsigned long long)idx[7] << 32));
  } else {
#pragma unroll
    for (int i = 0; i < kDecItems; ++i)
      if (base + i < n) {
        if (out_keep) out_keep[base + i] = (keepbits >> i) & 1u;
        if (out_est) out_est[base + i] = est[i];
        if (out_perm) out_perm[base + i] = idx[i];
      }
  }
}

/* Packs the queues' survivors: copy job j moves up to kCompactChunk indices of one queue; a
 * warp per job. */
__device__ __forceinline__ void kept_move_jobs(const uint32_t* __restrict__ kept_tmp, const uint32_t* __restrict__ seg_off,
                                               const uint32_t* __restrict__ seg_kept, const uint32_t* __restrict__ kept_base,
                                               const uint32_t* __restrict__ chunk_base, uint32_t n_seg,
                                               uint32_t* __restrict__ out_kept_idx) {
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t jobs = __ldcg(&chunk_base[n_seg]), step = (gridDim.x * blockDim.x) >> 5;
  for (uint32_t job = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; job < jobs; job += step) {
    uint32_t lo = 0, hi = n_seg;                 /* last queue whose first job is <= job */
    while (hi - lo > 1) {
      const uint32_t mid = lo + (hi - lo) / 2;
      if (__ldcg(&chunk_base[mid]) <= job) lo = mid; else hi = mid;
    }
    const uint32_t s = lo;
    const uint32_t first = (job - __ldcg(&chunk_base[s])) * kCompactChunk;
    const uint32_t count = min((uint32_t)kCompactChunk, __ldcg(&seg_kept[s]) - first);
    const uint32_t* src = kept_tmp + seg_off[s] + first;
    uint32_t* dst = out_kept_idx + __ldcg(&kept_base[s]) + first;
    uint32_t i = lane;
    for (; i + 224 < count; i += 256) {            /* eight loads in flight per lane */
      uint32_t v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldcg(&src[i + 32 * k]);
#pragma unroll
      for (int k = 0; k < 8; ++k) dst[i + 32 * k] = v[k];
    }
    for (; i < count; i += 32) dst[i] = __ldcg(&src[i]);
  }
}

__global__ void __launch_bounds__(256)
k_kept_move(const uint32_t* __restrict__ kept_tmp, const uint32_t* __restrict__ seg_off,
            const uint32_t* __restrict__ seg_kept, const uint32_t* __restrict__ kept_base,
            const uint32_t* __restrict__ chunk_base, uint32_t n_seg, uint32_t* __restrict__ out_kept_idx) {
  pdl_wait();
  kept_move_jobs(kept_tmp, seg_off, seg_kept, kept_base, chunk_base, n_seg, out_kept_idx);
}

/* The decision by scanning, from the sorted elements to the packed survivors, as ONE kernel: the
 * fallback for calls whose queues have too many batch windows for the tables (and what
 * PARD_MODE_SCAN asks for).  Launched on every call; returns at once when the tables did the
 * work.  Its five steps -- tile aggregates, their scan (block 0), the decision, the queues' kept
 * counts into output offsets (block 0), the packing of the survivors -- need the whole grid to
 * have finished the step before: the grid is small enough to be resident as a whole (at most two
 * blocks of 128 threads per multiprocessor), and its blocks meet at counters in the workspace
 * header, each wait bounded like the sort's (PARD_ETIMEOUT, every block gives up, nothing hangs;
 * the bound only bites when other streams keep the multiprocessors full for that long). */
__device__ bool grid_barrier(PlanHeader* hdr, int k, bool withhold = false) {
  __shared__ uint32_t s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (!withhold) atomicAdd(&hdr->bar[k], 1u);      /* (testing aid: a block that never arrives) */
    uint32_t spins = 0;
    bool ok = true;
    while (ld_relaxed(&hdr->bar[k]) < gridDim.x) {     /* up to about half a second: other work may hold multiprocessors for a while */
      if (++spins > 8 * kSpinLimit || hdr->aborted) { ok = false; break; }
      __nanosleep(200);
    }
    if (!ok) set_aborted(hdr);
    __threadfence();
    s_ok = ok ? 1u : 0u;
  }
  __syncthreads();
  return s_ok != 0;
}

template <bool RAW>
__global__ void __launch_bounds__(kDecThreads, 3)
k_scan_path(PlanHeader* hdr, const unsigned long long* __restrict__ buf_a,
            const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits, uint32_t n_seg,
            const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ seg_off,
            const uint32_t* __restrict__ win_off, unsigned long long* __restrict__ tile_agg, int32_t* __restrict__ carry,
            uint8_t* __restrict__ out_keep, long long* __restrict__ out_est, uint32_t* __restrict__ out_perm,
            uint32_t* __restrict__ kept_tmp, uint32_t* __restrict__ seg_kept, uint32_t* __restrict__ kept_base,
            uint32_t* __restrict__ chunk_base, uint32_t* __restrict__ out_seg_kept,
            unsigned long long* __restrict__ out_n_kept, uint32_t* __restrict__ out_kept_idx, uint32_t stall) {
  pdl_wait();
  if (hdr->wide || hdr->aborted || !hdr->use_scan) return;
  const uint32_t n_tiles = (n + kDecTile - 1) / kDecTile;
  tile_agg_tiles<RAW>(hdr, buf_a, buf_b, n, ibits, ktab, seg_off, tile_agg);
  if (!grid_barrier(hdr, 0, stall && blockIdx.x == 0)) return;
  if (blockIdx.x == 0) tile_scan_block<RAW, kDecThreads>(tile_agg, n_tiles, carry);
  if (!grid_barrier(hdr, 1)) return;
  decide_tiles<RAW>(hdr, buf_a, buf_b, n, ibits, ktab, seg_off, win_off, carry, out_keep, out_est, out_perm, kept_tmp, seg_kept);
  if (!grid_barrier(hdr, 2)) return;
  if (blockIdx.x == 0) kept_scan_block<kDecThreads>(seg_kept, n_seg, kept_base, chunk_base, out_seg_kept, out_n_kept);
  if (!grid_barrier(hdr, 3)) return;
  if (out_kept_idx) kept_move_jobs(kept_tmp, seg_off, seg_kept, kept_base, chunk_base, n_seg, out_kept_idx);
}

/* ------------------------------------------------------------------------ */
/* one block plans one ctx from start to end                                 */
/* ------------------------------------------------------------------------ */
/* For calls whose requests come grouped by ascending ctx with no ctx above a sort tile -- one
 * module's queue planned every few milliseconds, or many decision epochs in one call -- a block
 * does the whole job for "its" ctx without leaving shared memory: it reads the ctx's requests
 * once, finds the ctx's deadline range, computes the constants of the ctx's queues (Eq. 3),
 * sorts (radix passes over the stage and deadline bits, as k_sort_local), finds every request's
 * admitted position by a segmented scan over the sorted elements, and writes the outputs: 16
 * bytes read and 13 + 4f written per request, no element ever stored to global memory, no window
 * table, no search.  The scan runs twice over the elements, which stay in shared memory: once
 * for the warps' aggregates, once for the positions.  With a single ctx the block also packs the
 * survivors (the whole call is one launch); with several, k_kept_scan and k_kept_move follow. */
struct LocalArgs {
  const uint4* req;
  const uint32_t* ctx_start;       /* NULL: the call has one ctx */
  uint32_t n, n_ctx, ibits, raw;
  PipeTable pipes;
  uint32_t n_pipelines;
  pard_queue_state_t st;
  uint8_t* out_keep;
  long long* out_est;
  uint32_t* out_perm;
  uint32_t* out_kept_idx;          /* used directly only with one ctx */
  unsigned long long* out_n_kept;
  uint32_t* out_seg_off;
  uint32_t* out_seg_kept;
  const PardSegConst* ktab;        /* several ctx: the queues' constants, from k_seg_const */
  uint32_t* seg_off;               /* workspace copies, read by k_kept_scan / k_kept_move */
  uint32_t* seg_kept;
  uint32_t* kept_tmp;
  /* sort only (large grouped calls): the block stops behind the sort, hands the elements over in
   * the call's format -- fmt_dbits deadline bits, whatever the ctx's own span -- and publishes the
   * ctx's deadline range; the kernels of the general path take it from there */
  uint32_t sort_only, fmt_dbits;
  unsigned long long* dst;
  unsigned long long* ctx_dmin_inv;
  unsigned long long* ctx_dmax;
};

template <int THREADS>
struct LocalSmem {
  unsigned long long keys[kSortTile];
  uint32_t slot[THREADS / 32][kBins];      /* counts, then next free slot per (warp, digit) */
  uint32_t match[THREADS / 32][kBins];     /* lanes currently holding the digit */
  uint32_t scan[THREADS / 32];
  PardSegConst K[PARD_MAX_STAGES];
  uint32_t stage_cnt[PARD_MAX_STAGES];
  uint32_t stage_first[PARD_MAX_STAGES + 1];
  uint32_t stage_kept[PARD_MAX_STAGES];
  uint32_t kept_base[PARD_MAX_STAGES + 1];
  uint32_t hb_kept[PARD_MAX_STAGES];       /* high budget first: length of the kept prefix */
  unsigned long long red_min[THREADS / 32], red_max[THREADS / 32];
  int32_t wm[THREADS / 32];
  uint32_t wh[THREADS / 32];
  uint32_t flag_foreign, flag_bad;
};

/* decoded view of one sorted element inside a block of k_plan_local */
struct LocalElem {
  uint32_t stage, idx, r, u;
  bool high_first;
};

template <class SMEM>
__device__ __forceinline__ LocalElem local_decode(unsigned long long e, uint32_t pos, const SMEM& Sm,
                                                  uint32_t ibits, uint32_t dbits, unsigned long long dmask,
                                                  uint32_t imask) {
  LocalElem x;
  x.stage = (uint32_t)(e >> (ibits + dbits));
  x.idx = (uint32_t)e & imask;
  const PardSegConst& K = Sm.K[x.stage];
  x.high_first = K.narrow & kSegHighFirst;
  x.r = pos - Sm.stage_first[x.stage];
  const unsigned long long off = (e >> ibits) & dmask;
  if ((K.narrow & kSegNarrow) && dbits <= 29) {
    const int32_t X = x.high_first ? (int32_t)K.A_rel - (int32_t)off : (int32_t)off - (int32_t)K.A_rel;
    const unsigned long long uu = (unsigned long long)(div_magic32((uint32_t)X, K.d_magic) + 1u) * K.cap;
    x.u = X < 0 ? 0u : (uu > kUClamp ? kUClamp : (uint32_t)uu);
  } else {
    x.u = (K.narrow & kSegNoStage) ? 0u : threshold_u(slack_of(off, K), K);
  }
  return x;
}

/* THREADS: 512, two blocks per multiprocessor.  (1,024 threads for a call that is this one block --
 * half as many ranking rounds per warp, twice the warps -- measured the same 28 us at 4,096
 * requests: the time is the chain of barriers and dependent shared-memory steps, not the warps.) */
template <bool RAW, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 512 ? 2 : 1)
k_plan_local(PlanHeader* __restrict__ hdr, const LocalArgs a) {
  pdl_wait();
  constexpr int WARPS = THREADS / 32;
  constexpr int kItems = kSortTile / THREADS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  LocalSmem<THREADS>& Sm = *reinterpret_cast<LocalSmem<THREADS>*>(smem_raw);
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lanebit = 1u << lane;
  const uint32_t S = (uint32_t)a.st.stage_stride;
  const uint32_t c = blockIdx.x;
  const bool single = a.ctx_start == nullptr;
  if (single) {                                          /* the only kernel of the call: the header starts here */
    if (tid < sizeof(PlanHeader) / 4) reinterpret_cast<uint32_t*>(hdr)[tid] = 0;
    __syncthreads();
  } else if (hdr->unsorted || hdr->ctx_too_big) {      /* k_ctx_ranges found the promised grouping broken */
    if (tid == 0 && c == 0) { set_status(hdr, PARD_EDATA); hdr->aborted = 1; }   /* nothing is sorted: later kernels return */
    return;
  }
  const uint32_t first = single ? 0u : a.ctx_start[c];
  const uint32_t cnt = single ? a.n : a.ctx_start[c + 1] - first;
  /* every warp owns `items` rounds of 32 consecutive requests: as few as the ctx needs */
  const int items = (int)((cnt + THREADS - 1) / THREADS);
  const uint32_t wfirst = warp * (32 * (uint32_t)items);
  uint16_t* stage16 = reinterpret_cast<uint16_t*>(&Sm.slot[0][0]);     /* 16 KB: the stages until the elements are built */

  /* 1. the ctx's requests: deadlines into the tile buffer, stages beside them; deadline range,
   * queue lengths, input checks */
  for (uint32_t i = tid; i < S; i += THREADS) { Sm.stage_cnt[i] = 0; Sm.stage_kept[i] = 0; }
  if (tid == 0) { Sm.flag_foreign = 0; Sm.flag_bad = 0; }
  __syncthreads();
  unsigned long long lmin = ~0ull, lmax = 0;
  bool foreign = false, bad = false;
#pragma unroll 4
  for (int i = 0; i < kItems; ++i) {
    if (i >= items) break;
    const uint32_t pos = wfirst + i * 32 + lane;
    if (pos < cnt) {
      const uint4 r = __ldg(&a.req[first + pos]);
      const unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
      const uint32_t stage = r.w & 0xffffu;
      foreign |= r.z != c;
      const bool ok = r.z == c && stage < S && D < (unsigned long long)PARD_TIME_LIMIT_US;
      bad |= !ok;
      Sm.keys[pos] = D;
      stage16[pos] = ok ? (uint16_t)stage : (uint16_t)0xffffu;
      if (ok) {
        lmin = D < lmin ? D : lmin;
        lmax = D > lmax ? D : lmax;
        atomicAdd(&Sm.stage_cnt[stage], 1u);
      }
    }
  }
  for (int o = 16; o; o >>= 1) {
    const unsigned long long x = __shfl_xor_sync(0xffffffffu, lmin, o), y = __shfl_xor_sync(0xffffffffu, lmax, o);
    lmin = x < lmin ? x : lmin;
    lmax = y > lmax ? y : lmax;
  }
  if (lane == 0) { Sm.red_min[warp] = lmin; Sm.red_max[warp] = lmax; }
  if (foreign) Sm.flag_foreign = 1;
  if (bad) Sm.flag_bad = 1;
  __syncthreads();
  if (Sm.flag_foreign) {                                 /* not grouped by ctx after all (or, with one ctx, a request of another) */
    if (tid == 0) { hdr->unsorted = 1; set_status(hdr, PARD_EDATA); hdr->aborted = 1; }
    return;
  }
  unsigned long long dmin = ~0ull, dmax = 0;
#pragma unroll
  for (int w = 0; w < WARPS; ++w) {
    dmin = Sm.red_min[w] < dmin ? Sm.red_min[w] : dmin;
    dmax = Sm.red_max[w] > dmax ? Sm.red_max[w] : dmax;
  }
  const uint32_t dbits = dmin <= dmax ? bit_width64(dmax - dmin) : 0u;
  /* stage field of the elements: requests that failed the checks carry the value S there, so
   * that they sort behind the ctx's queues; they are reported, never decided */
  const uint32_t sb = 32u - __clz(Sm.flag_bad ? S : S - 1);    /* bit width of the largest value; __clz(0) = 32 */
  if (sb + dbits + a.ibits > 64) {                       /* the element does not fit 64 bits */
    if (tid == 0) { hdr->wide = 1; set_status(hdr, PARD_ERANGE); }
    return;
  }
  if (Sm.flag_bad && tid == 0) set_status(hdr, PARD_EDATA);

  /* 2. constants of the ctx's queues: worked out here, a warp per stage, when the call is this
   * one block; else taken from the table k_seg_const has filled for all queues at once (a chain
   * of dependent loads that every block would otherwise wait for) and completed with what hangs
   * on the ctx's deadline range */
  if (a.sort_only) {
    /* the constants come later, from k_seg_const, once every ctx's range is known */
  } else if (single) {
    for (uint32_t k = warp; k < S; k += WARPS) {
      bool kbad = false;
      const PardSegConst K = seg_const_warp(a.pipes, a.n_pipelines, a.st, c, k, dmin, dmax, lane, &kbad);
      if (kbad) set_status(hdr, PARD_EDATA);
      if (lane == 0) Sm.K[k] = K;
    }
  } else {
    for (uint32_t k = tid; k < S; k += THREADS) {
      PardSegConst K = a.ktab[(size_t)c * S + k];
      const bool high_first = K.narrow & kSegHighFirst;
      K.A_rel = high_first ? (int64_t)dmax - K.A : K.A - (int64_t)dmin;
      const int64_t lim = (int64_t)1 << 29;
      const bool fits32 = K.d_magic != 0 && K.d < ((int64_t)1 << 31) && K.A_rel > -lim && K.A_rel < lim;
      K.narrow = (K.narrow & ~kSegNarrow) | (fits32 && !(K.narrow & kSegNoStage) ? kSegNarrow : 0u);
      Sm.K[k] = K;
    }
  }
  if (warp == 0) {                                       /* first position of every queue inside the ctx */
    uint32_t run = 0;
    for (uint32_t k0 = 0; k0 < S; k0 += 32) {
      const uint32_t k = k0 + lane;
      const uint32_t v = k < S ? Sm.stage_cnt[k] : 0u;
      uint32_t x = v;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= (uint32_t)o) x += y;
      }
      if (k < S) Sm.stage_first[k] = run + x - v;
      run += __shfl_sync(0xffffffffu, x, 31);
    }
    if (lane == 0) Sm.stage_first[S] = run;
  }
  __syncthreads();
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  const uint32_t imask = (1u << a.ibits) - 1;

  /* 3. sort elements (stage | deadline offset | index), built from the tile buffer */
  unsigned long long key[kItems];
#pragma unroll
  for (int i = 0; i < kItems; ++i) {
    if (i >= items) break;
    const uint32_t pos = wfirst + i * 32 + lane;
    key[i] = ~0ull;                                      /* padding sorts last */
    if (pos < cnt) {
      const unsigned long long D = Sm.keys[pos];
      const uint32_t stage = stage16[pos];
      const uint32_t j = first + pos;
      if (stage != 0xffffu) {
        const bool high_first = a.st.d_priority && a.st.d_priority[(size_t)c * S + stage] != 0;
        const unsigned long long off = (high_first ? dmax - D : D - dmin) & dmask;
        key[i] = ((((unsigned long long)stage << dbits) | off) << a.ibits) | j;
      } else {
        key[i] = (((unsigned long long)S << dbits) << a.ibits) | j;
      }
    }
  }
  __syncthreads();                                       /* the stages have been read: their room becomes the counters again */
  const uint32_t local_bits = dbits + sb;
  const uint32_t passes = (local_bits + 7) / 8;
  for (uint32_t i = tid; i < WARPS * kBins; i += THREADS) (&Sm.match[0][0])[i] = 0;
  for (uint32_t p = 0; p < passes; ++p) {
    const uint32_t shift = a.ibits + 8 * p;
    for (uint32_t i = tid; i < WARPS * kBins; i += THREADS) (&Sm.slot[0][0])[i] = 0;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kItems; ++i)
      if (i < items) atomicAdd(&Sm.slot[warp][(uint32_t)(key[i] >> shift) & 255u], 1u);
    __syncthreads();
    uint32_t count = 0, x = 0;
    if (tid < kBins) {
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        const uint32_t t = Sm.slot[w][tid];
        Sm.slot[w][tid] = count;
        count += t;
      }
      x = count;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= (uint32_t)o) x += y;
      }
      if (lane == 31) Sm.scan[warp] = x;
    }
    __syncthreads();
    if (tid < kBins) {
      uint32_t wx = 0;
#pragma unroll
      for (int w = 0; w < kBins / 32; ++w)
        if (w < (int)warp) wx += Sm.scan[w];
      const uint32_t dstart = wx + x - count;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) Sm.slot[w][tid] += dstart;
    }
    __syncthreads();
    sort_rank_drop<kItems, kItems>(key, shift, Sm.slot[warp], Sm.match[warp], Sm.keys, lanebit, items);
    __syncthreads();
    if (p + 1 < passes) {
#pragma unroll
      for (int i = 0; i < kItems; ++i)
        if (i < items) key[i] = Sm.keys[wfirst + i * 32 + lane];
      __syncthreads();
    }
  }
  if (passes == 0) {
#pragma unroll
    for (int i = 0; i < kItems; ++i)
      if (i < items) Sm.keys[wfirst + i * 32 + lane] = key[i];
    __syncthreads();
  }

  if (a.sort_only) {
    if (Sm.flag_bad) {                                   /* a flagged request has no place in the general path's order */
      if (tid == 0) hdr->aborted = 1;
      return;
    }
    if (dbits > a.fmt_dbits) {                           /* this ctx's span does not fit the call's element */
      if (tid == 0) { hdr->wide = 1; set_status(hdr, PARD_ERANGE); }
      return;
    }
    if (tid == 0 && dmin <= dmax) {
      a.ctx_dmin_inv[c] = ~dmin;
      a.ctx_dmax[c] = dmax;
      atomicMax(&hdr->span_max, dmax - dmin);
    }
    const uint32_t kshift = a.ibits + dbits;
    for (uint32_t pos = tid; pos < cnt; pos += THREADS) {
      const unsigned long long e = Sm.keys[pos];
      const unsigned long long seg = (unsigned long long)c * S + (uint32_t)(e >> kshift);
      a.dst[first + pos] = ((seg << a.fmt_dbits | ((e >> a.ibits) & dmask)) << a.ibits) | (e & imask);
    }
    return;
  }

  /* 4. queue boundaries of the ctx */
  const uint32_t n_good = Sm.stage_first[S];             /* requests that passed the checks; the others follow them */
  for (uint32_t k = tid; k < S; k += THREADS) {
    const uint32_t v = first + Sm.stage_first[k];
    a.seg_off[(size_t)c * S + k] = v;
    if (a.out_seg_off) a.out_seg_off[(size_t)c * S + k] = v;
    Sm.hb_kept[k] = Sm.stage_cnt[k];
  }
  if (c + 1 == a.n_ctx && tid == 0) {
    a.seg_off[(size_t)a.n_ctx * S] = a.n;
    if (a.out_seg_off) a.out_seg_off[(size_t)a.n_ctx * S] = a.n;
  }
  __syncthreads();
  /* a queue served high budget first keeps a prefix: its length is the first position r with r >= u_r */
  if (a.st.d_priority) {
#pragma unroll 1
    for (int i = 0; i < kItems; ++i) {
      if (i >= items) break;
      const uint32_t pos = wfirst + i * 32 + lane;
      if (pos < n_good) {
        const LocalElem x = local_decode(Sm.keys[pos], pos, Sm, a.ibits, dbits, dmask, imask);
        if (x.high_first && x.r >= x.u) atomicMin(&Sm.hb_kept[x.stage], x.r);
      }
    }
    __syncthreads();
  }

  /* 5. segmented scan, first time: what every warp's elements add up to.  kGroup rounds are
   * scanned side by side (their shuffles do not wait for each other), then chained. */
  constexpr int kGroup = 4;
  static_assert(kItems % kGroup == 0, "whole groups");
  SegVal run = seg_identity<RAW>();
#pragma unroll 1                                         /* (see 6.) */
  for (int i0 = 0; i0 < kItems; i0 += kGroup) {
    if (i0 >= items) break;
    SegVal v[kGroup];
#pragma unroll
    for (int g = 0; g < kGroup; ++g) {
      const uint32_t pos = wfirst + (i0 + g) * 32 + lane;
      v[g] = seg_identity<RAW>();
      if (i0 + g < items && pos < n_good) {
        const LocalElem x = local_decode(Sm.keys[pos], pos, Sm, a.ibits, dbits, dmask, imask);
        v[g].head = x.r == 0 ? 1u : 0u;
        v[g].m = RAW ? (x.r < x.u ? 1 : 0) : (int32_t)x.u - (int32_t)x.r;
      }
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
      for (int g = 0; g < kGroup; ++g) {
        SegVal l;
        l.m = __shfl_up_sync(0xffffffffu, v[g].m, o);
        l.head = __shfl_up_sync(0xffffffffu, v[g].head, o);
        if (lane >= (uint32_t)o) v[g] = seg_combine<RAW>(l, v[g]);
      }
    }
#pragma unroll
    for (int g = 0; g < kGroup; ++g) {
      SegVal all;
      all.m = __shfl_sync(0xffffffffu, v[g].m, 31);
      all.head = __shfl_sync(0xffffffffu, v[g].head, 31);
      run = seg_combine<RAW>(run, all);
    }
  }
  if (lane == 0) { Sm.wm[warp] = run.m; Sm.wh[warp] = run.head; }
  __syncthreads();
  SegVal carry = seg_identity<RAW>();
#pragma unroll
  for (int w = 0; w < WARPS; ++w) {
    SegVal t; t.m = Sm.wm[w]; t.head = Sm.wh[w];
    if (w < (int)warp) carry = seg_combine<RAW>(carry, t);
  }

  /* 6. second time: every request's position, estimate and decision; outputs.  The loop is kept a
   * loop: a block that is alone on the device (one small ctx) waits for its instructions more than
   * for anything else (ncu: "no instruction" is its first stall reason), so code that runs once
   * per group is not unrolled over the groups. */
#pragma unroll 1
  for (int i0 = 0; i0 < kItems; i0 += kGroup) {
    if (i0 >= items) break;
    SegVal v[kGroup];
    LocalElem x[kGroup];
    unsigned long long e[kGroup];
#pragma unroll
    for (int g = 0; g < kGroup; ++g) {
      const uint32_t pos = wfirst + (i0 + g) * 32 + lane;
      v[g] = seg_identity<RAW>();
      x[g].stage = 0; x[g].idx = 0; x[g].r = 0; x[g].u = 0; x[g].high_first = false;
      e[g] = 0;
      if (i0 + g < items && pos < cnt) e[g] = Sm.keys[pos];
      if (i0 + g < items && pos < n_good) {
        x[g] = local_decode(e[g], pos, Sm, a.ibits, dbits, dmask, imask);
        v[g].head = x[g].r == 0 ? 1u : 0u;
        v[g].m = RAW ? (x[g].r < x[g].u ? 1 : 0) : (int32_t)x[g].u - (int32_t)x[g].r;
      }
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
      for (int g = 0; g < kGroup; ++g) {
        SegVal l;
        l.m = __shfl_up_sync(0xffffffffu, v[g].m, o);
        l.head = __shfl_up_sync(0xffffffffu, v[g].head, o);
        if (lane >= (uint32_t)o) v[g] = seg_combine<RAW>(l, v[g]);
      }
    }
#pragma unroll
    for (int g = 0; g < kGroup; ++g) {
      const uint32_t pos = wfirst + (i0 + g) * 32 + lane;
      const bool valid = i0 + g < items && pos < n_good;
      SegVal exc;
      exc.m = __shfl_up_sync(0xffffffffu, v[g].m, 1);
      exc.head = __shfl_up_sync(0xffffffffu, v[g].head, 1);
      if (lane == 0) exc = seg_identity<RAW>();
      const SegVal pre = seg_combine<RAW>(carry, exc);   /* over the earlier requests of the same queue */
      SegVal all;
      all.m = __shfl_sync(0xffffffffu, v[g].m, 31);
      all.head = __shfl_sync(0xffffffffu, v[g].head, 31);
      carry = seg_combine<RAW>(carry, all);
      if (i0 + g < items && pos < cnt) {
        const uint32_t gpos = first + pos;
        uint32_t keep = 0;
        long long est = 0;
        if (valid) {
          const PardSegConst& K = Sm.K[x[g].stage];
          uint32_t cpos, ahead;                          /* batch-slot position; kept requests ahead in the queue */
          if (RAW) {
            cpos = x[g].r;
            ahead = x[g].r == 0 ? 0u : (uint32_t)pre.m;
          } else {
            if (x[g].r == 0) cpos = 0;
            else {
              const long long cc = (long long)x[g].r - 1 + pre.m;
              cpos = cc < (long long)x[g].r ? (uint32_t)cc : x[g].r;
            }
            if (x[g].high_first) cpos = min(x[g].r, Sm.hb_kept[x[g].stage]);
            ahead = cpos;
          }
          const uint32_t round = K.cap_magic ? div_magic32(cpos, K.cap_magic) : cpos;
          est = K.A + (long long)round * K.d;
          keep = (cpos < x[g].u && !(K.narrow & kSegNoStage)) ? 1u : 0u;
          if (K.narrow & kSegNoStage) set_status(hdr, PARD_EDATA);
          if (keep && a.kept_tmp) a.kept_tmp[first + Sm.stage_first[x[g].stage] + ahead] = x[g].idx;
          if (x[g].r + 1 == Sm.stage_cnt[x[g].stage]) Sm.stage_kept[x[g].stage] = ahead + keep;   /* the queue's last request */
        }
        if (a.out_keep) a.out_keep[gpos] = (uint8_t)keep;
        if (a.out_est) a.out_est[gpos] = est;
        if (a.out_perm) a.out_perm[gpos] = (uint32_t)e[g] & imask;
      }
    }
  }
  __syncthreads();
  for (uint32_t k = tid; k < S; k += THREADS) {
    a.seg_kept[(size_t)c * S + k] = Sm.stage_kept[k];
    if (single && a.out_seg_kept) a.out_seg_kept[k] = Sm.stage_kept[k];
  }
  if (!single) return;

  /* 7. one ctx: pack the survivors here (queue after queue) and finish the call */
  if (warp == 0) {
    uint32_t run_k = 0;
    for (uint32_t k0 = 0; k0 < S; k0 += 32) {
      const uint32_t k = k0 + lane;
      const uint32_t v = k < S ? Sm.stage_kept[k] : 0u;
      uint32_t y = v;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t z = __shfl_up_sync(0xffffffffu, y, o);
        if (lane >= (uint32_t)o) y += z;
      }
      if (k < S) Sm.kept_base[k] = run_k + y - v;
      run_k += __shfl_sync(0xffffffffu, y, 31);
    }
    if (lane == 0) {
      Sm.kept_base[S] = run_k;
      if (a.out_n_kept) *a.out_n_kept = run_k;
    }
  }
  __threadfence_block();
  __syncthreads();
  if (a.out_kept_idx && a.kept_tmp)
    for (uint32_t k = 0; k < S; ++k) {
      const uint32_t nk = Sm.stage_kept[k], from = Sm.stage_first[k], to = Sm.kept_base[k];
      for (uint32_t i = tid; i < nk; i += THREADS) a.out_kept_idx[to + i] = a.kept_tmp[from + i];
    }
}

/* ------------------------------------------------------------------------ */
/* keys wider than one sort element                                          */
/* ------------------------------------------------------------------------ */
/* When segment, deadline and index bits together exceed 64 (deadline spans of years, millions
 * of queues and requests at once) the key (segment | deadline offset, up to 84 bits) is sorted
 * in chunks, least significant first, each chunk by the ordinary passes: a chunk's element is
 * chunk << ibits | current position, so every super-pass is a stable sort of the current
 * order by one more chunk, and the positions it yields are chased back to request indices.
 * The last super-pass leaves the order of the requests; the elements are then rewritten as
 * segment | index (no deadline bits) and the decision is taken by the queue walk, which looks
 * the deadlines up in the request array.  A slow path for legal but extreme inputs. */
__device__ __forceinline__ uint32_t wide_chunk_bits(const PlanHeader* hdr, uint32_t sbits, uint32_t ibits, uint32_t super) {
  const uint32_t kb = sbits + hdr->dbits, cw = 64 - ibits, lo = super * cw;
  return lo < kb ? min(cw, kb - lo) : 0u;
}

__global__ void __launch_bounds__(256)
k_wide_reset(PlanHeader* hdr, uint32_t* __restrict__ hist, uint32_t* __restrict__ lookback, unsigned long long lb_words,
             uint32_t sbits, uint32_t ibits, uint32_t super) {
  pdl_wait();
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    hdr->npass = (wide_chunk_bits(hdr, sbits, ibits, super) + 7) / 8;
    hdr->keybits = wide_chunk_bits(hdr, sbits, ibits, super);   /* what the passes of this super-pass sort */
    for (int i = 0; i <= kMaxPasses; ++i) hdr->ticket[i] = 0;
    if (super == 0) {
      hdr->wide = 2;                                      /* the chunked sort is under way */
      hdr->status = hdr->bad_input ? (uint32_t)(-PARD_EDATA) : 0u;   /* the width was not an error after all */
    }
  }
  const unsigned long long step = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < lb_words + kMaxPasses * kBins; i += step) {
    if (i < lb_words) lookback[i] = 0;
    else hist[i - lb_words] = 0;
  }
}

__global__ void __launch_bounds__(256)
k_wide_pack(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t S,
            const unsigned long long* __restrict__ ctx_dmin_inv, const unsigned long long* __restrict__ ctx_dmax,
            const uint8_t* __restrict__ priority, uint32_t sbits, uint32_t ibits, uint32_t super,
            const PlanHeader* __restrict__ hdr, const uint32_t* __restrict__ order,
            unsigned long long* __restrict__ dst, uint32_t* __restrict__ hist) {
  pdl_wait();
  __shared__ uint32_t s_hist[kMaxPasses * kBins];
  const uint32_t bits = wide_chunk_bits(hdr, sbits, ibits, super), npass = (bits + 7) / 8;
  const uint32_t dbits = hdr->dbits, lo = super * (64 - ibits);
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x) s_hist[i] = 0;
  __syncthreads();
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t p = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; p < n; p += stride) {
    const uint32_t orig = super == 0 ? (uint32_t)p : order[p];
    const uint4 r = __ldg(&req[orig]);
    const unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
    const uint32_t ctx = r.z, stage = r.w & 0xffffu;
    unsigned long long chunk = 0;
    if (ctx < n_ctx && stage < S && D < (unsigned long long)PARD_TIME_LIMIT_US && bits) {
      const uint32_t seg = ctx * S + stage;
      const bool high_first = priority && __ldg(&priority[seg]) != 0;
      const unsigned long long off = high_first ? ctx_dmax[ctx] - D : D - ~ctx_dmin_inv[ctx];
      const unsigned __int128 key = ((unsigned __int128)seg << dbits) | off;
      chunk = (unsigned long long)(key >> lo) & (bits >= 64 ? ~0ull : ((1ull << bits) - 1));
    }
    dst[p] = (chunk << ibits) | p;                        /* flagged requests sort first, into queue 0 */
    for (uint32_t q = 0; q < npass; ++q) atomicAdd(&s_hist[q * kBins + ((chunk >> (8 * q)) & 255u)], 1u);
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x)
    if (s_hist[i]) atomicAdd(&hist[i], s_hist[i]);
}

/* positions of a super-pass -> request indices, into the buffer the sort has left free */
__global__ void __launch_bounds__(256)
k_wide_chase(const PlanHeader* __restrict__ hdr, const unsigned long long* __restrict__ buf_a,
             unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits, uint32_t super,
             const uint32_t* __restrict__ order) {
  pdl_wait();
  const bool odd = hdr->npass & 1;
  const unsigned long long* sorted = odd ? buf_b : buf_a;
  uint32_t* tmp = reinterpret_cast<uint32_t*>(odd ? const_cast<unsigned long long*>(buf_a) : buf_b);
  const uint32_t imask = (1u << ibits) - 1;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n; q += stride) {
    const uint32_t pos = (uint32_t)sorted[q] & imask;
    tmp[q] = super == 0 ? pos : order[pos];
  }
}

__global__ void __launch_bounds__(256)
k_wide_keep(const PlanHeader* __restrict__ hdr, const unsigned long long* __restrict__ buf_a,
            const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t* __restrict__ order) {
  pdl_wait();
  const uint32_t* tmp = reinterpret_cast<const uint32_t*>((hdr->npass & 1) ? buf_a : buf_b);
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n; q += stride) order[q] = tmp[q];
}

/* the sorted order as elements without deadline bits: segment | request index, in buf_a */
__global__ void __launch_bounds__(256)
k_wide_final(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t S, uint32_t sbits, uint32_t ibits,
             PlanHeader* hdr, const uint32_t* __restrict__ order, unsigned long long* __restrict__ buf_a) {
  pdl_wait();
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n; q += stride) {
    const uint32_t orig = order[q];
    const uint4 r = __ldg(&req[orig]);
    const unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
    const uint32_t ctx = r.z, stage = r.w & 0xffffu;
    const bool ok = ctx < n_ctx && stage < S && D < (unsigned long long)PARD_TIME_LIMIT_US;
    buf_a[q] = ((unsigned long long)(ok ? ctx * S + stage : 0u) << ibits) | orig;
  }
}

/* after k_wide_final: the header as the kernels behind the sort expect it */
__global__ void k_wide_done(PlanHeader* hdr, uint32_t sbits) {
  pdl_wait();
  hdr->dbits = 0;
  hdr->keybits = sbits;
  hdr->npass = 0;
  hdr->wide = 0;
}

/* ---- optional phase timing (process-wide) ---- */
constexpr int kEventsPerSample = PARD_N_PHASES + 1;
static_assert(PARD_N_PHASES == 4 + kMaxPasses + 3, "phase list");
struct Profiler {
  std::mutex mu;
  cudaEvent_t* last = nullptr;       /* events of the most recent sampled call */
  std::atomic<bool> on{false};       /* read without the lock by every pard_plan call */
  bool coarse = false;
  uint32_t every = 1, max_samples = 0, calls = 0, n_samples = 0;
  std::vector<cudaEvent_t> ev;
};
Profiler g_prof;

constexpr int kPhaseTables = 4 + kMaxPasses;       /* "tables", then "decide", "compact" */

/* events of this call if it is a sampled one, else nullptr */
cudaEvent_t* profile_acquire(bool* coarse) {
  if (!g_prof.on.load(std::memory_order_acquire)) return nullptr;   /* the usual case: no lock taken */
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (!g_prof.on.load(std::memory_order_relaxed)) return nullptr;
  *coarse = g_prof.coarse;
  uint32_t call = g_prof.calls++;
  g_prof.last = nullptr;
  if (call % g_prof.every != 0 || g_prof.n_samples >= g_prof.max_samples) return nullptr;
  g_prof.last = g_prof.ev.data() + (size_t)(g_prof.n_samples++) * kEventsPerSample;
  return g_prof.last;
}

/* the sort pass needs more dynamic shared memory than the default limit: opt in once per device */
int allow_sort_smem(int dev) {
  static std::mutex mu;
  static std::atomic<bool> done[64];
  if (dev < 0 || dev >= 64) return PARD_ERANGE;
  if (done[dev].load(std::memory_order_acquire)) return PARD_OK;    /* every call but the first on a device */
  std::lock_guard<std::mutex> lock(mu);
  if (!done[dev].load(std::memory_order_relaxed)) {
    PARD_CUDA_OK(cudaFuncSetAttribute(k_sort_pass<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sizeof(SortSmem)));
    PARD_CUDA_OK(cudaFuncSetAttribute(k_sort_pass<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sizeof(SortSmem)));
    PARD_CUDA_OK(cudaFuncSetAttribute(k_sort_pass<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sizeof(SortSmem)));
    PARD_CUDA_OK(cudaFuncSetAttribute(k_sort_local, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sizeof(SortSmem)));
    PARD_CUDA_OK(cudaFuncSetAttribute(k_plan_local<false, 512>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sizeof(LocalSmem<512>)));
    PARD_CUDA_OK(cudaFuncSetAttribute(k_plan_local<true, 512>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)sizeof(LocalSmem<512>)));
    done[dev].store(true, std::memory_order_release);
  }
  return PARD_OK;
}

bool local_sort_candidate(uint64_t n, uint32_t n_ctx) {
  if (n_ctx == 1) return n > 0 && n <= (uint64_t)kSortTile;         /* certain: one ctx inside one tile */
  return n >= (uint64_t)n_ctx * (kSortTile / 4) && n <= (uint64_t)n_ctx * kSortTile;
}

int check_state(const pard_queue_state_t* st, uint32_t n_ctx) {
  if (!st) return PARD_EINVAL;
  if (st->stage_stride < 1) return PARD_EINVAL;
  if (st->stage_stride > PARD_MAX_STAGES) return PARD_ERANGE;
  if (!st->d_now_us || !st->d_batch || !st->d_free_at_us || !st->d_q_us) return PARD_EINVAL;
  if (st->d_w_us && st->slot_stride < 0) return PARD_EINVAL;
  if (n_ctx < 1) return PARD_EINVAL;
  if ((uint64_t)n_ctx * (uint64_t)st->stage_stride > PARD_MAX_SEGMENTS) return PARD_ERANGE;
  return PARD_OK;
}

}  // namespace

/* pard_goodput follows pard_plan on the same stream and belongs to the same pass over the
 * sorted queues: when the plan call just before it was a sampled one, the end of its last phase
 * moves behind the goodput kernel. */
void pard_profile_extend_last(cudaStream_t stream) {
  if (!g_prof.on.load(std::memory_order_acquire)) return;
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (g_prof.on.load(std::memory_order_relaxed) && g_prof.last) cudaEventRecord(g_prof.last[PARD_N_PHASES], stream);
}

extern "C" int pard_plan_workspace_bytes(uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                                         uint64_t* bytes) {
  if (!bytes || n_ctx < 1 || stage_stride < 1) return PARD_EINVAL;
  if (n >= PARD_MAX_REQUESTS || stage_stride > PARD_MAX_STAGES ||
      (uint64_t)n_ctx * (uint64_t)stage_stride > PARD_MAX_SEGMENTS)
    return PARD_ERANGE;
  *bytes = make_layout(n, n_ctx, stage_stride).total;
  return PARD_OK;
}

extern "C" int pard_plan(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                         const pard_request_t* d_requests, uint64_t n,
                         const pard_queue_state_t* state, uint32_t n_ctx, uint32_t mode,
                         const pard_plan_out_t* out, void* d_workspace, uint64_t workspace_bytes,
                         void* cuda_stream) {
  return pard_plan_policy(pipelines, n_pipelines, d_requests, nullptr, n, state, n_ctx, mode, out, d_workspace,
                          workspace_bytes, cuda_stream);
}

extern "C" int pard_plan_policy(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                                const pard_request_t* d_requests, const pard_arrival_t* d_arrivals, uint64_t n,
                                const pard_queue_state_t* state, uint32_t n_ctx, uint32_t mode,
                                const pard_plan_out_t* out, void* d_workspace, uint64_t workspace_bytes,
                                void* cuda_stream) {
  /* ---- host-side checks, nothing launched before they pass ---- */
  if (!pipelines || n_pipelines < 1 || !out) return PARD_EINVAL;
  if (n_pipelines > kMaxPipelinesPerCall) return PARD_ERANGE;
  constexpr uint32_t kRuleBits = PARD_MODE_PATH_MASK | PARD_MODE_FCFS | PARD_MODE_NEXUS | PARD_MODE_CLIPPER;
  if (mode & ~(PARD_MODE_RAW | PARD_MODE_NOWAIT | PARD_MODE_SCAN | PARD_MODE_TEST_STALL | PARD_MODE_GROUPED | kRuleBits))
    return PARD_EINVAL;
  /* the rules decided by a walk of every queue, and what they combine with */
  const bool rule_walk = (mode & kRuleBits) != 0;
  const bool arrival_order = (mode & (PARD_MODE_FCFS | PARD_MODE_NEXUS | PARD_MODE_CLIPPER)) != 0;
  if (rule_walk && (mode & PARD_MODE_RAW)) return PARD_EINVAL;
  if ((mode & PARD_MODE_NEXUS) && (mode & (PARD_MODE_CLIPPER | PARD_MODE_PATH_MASK))) return PARD_EINVAL;
  if ((mode & PARD_MODE_CLIPPER) && (mode & PARD_MODE_PATH_MASK)) return PARD_EINVAL;
  if ((mode & PARD_MODE_CLIPPER) && n > 0 && (!d_arrivals || ((uintptr_t)d_arrivals & 15))) return PARD_EINVAL;
  if (arrival_order && state && state->d_priority) return PARD_EINVAL;
  int rc = check_state(state, n_ctx);
  if (rc != PARD_OK) return rc;
  if (n >= PARD_MAX_REQUESTS) return PARD_ERANGE;
  if (n > 0 && !d_requests) return PARD_EINVAL;
  if ((uintptr_t)d_requests & 15) return PARD_EINVAL;
  int dev = -1;
  PARD_CUDA_OK(cudaGetDevice(&dev));
  std::vector<const PardPipeDev*> h_pipes(n_pipelines);
  int32_t max_slots = 0;
  for (uint32_t i = 0; i < n_pipelines; ++i) {
    const pard_pipeline_t* p = pipelines[i];
    if (!p || !p->d_blob || p->device != dev) return PARD_EINVAL;
    if (p->n_stages > state->stage_stride) return PARD_EINVAL;
    max_slots = std::max(max_slots, p->n_slots);
    h_pipes[i] = (const PardPipeDev*)p->d_blob;
  }
  if (state->d_w_us && state->slot_stride < max_slots) return PARD_EINVAL;
  if (!d_workspace || ((uintptr_t)d_workspace & 255)) return PARD_EINVAL;
  const Layout L = make_layout(n, n_ctx, state->stage_stride);
  if (workspace_bytes < L.total) return PARD_EWORKSPACE;
  if ((out->d_est_us && ((uintptr_t)out->d_est_us & 15)) ||
      (out->d_perm && ((uintptr_t)out->d_perm & 15)) ||
      (out->d_keep && ((uintptr_t)out->d_keep & 7)))
    return PARD_EINVAL;

  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* ws = (char*)d_workspace;
  PlanHeader* hdr = (PlanHeader*)(ws + L.hdr);
  const PardPipeDev** d_pipes = (const PardPipeDev**)(ws + L.pipes);
  unsigned long long* ctx_dmin = (unsigned long long*)(ws + L.ctx_dmin);
  unsigned long long* ctx_dmax = (unsigned long long*)(ws + L.ctx_dmax);
  uint32_t* seg_off = (uint32_t*)(ws + L.seg_off);
  PardSegConst* ktab = (PardSegConst*)(ws + L.ktab);
  uint32_t* hist = (uint32_t*)(ws + L.hist);
  uint32_t* lookback = (uint32_t*)(ws + L.lookback);
  const size_t lb_words = (size_t)L.lb_tiles * kBins;
  unsigned long long* tile_agg = (unsigned long long*)(ws + L.tile_agg);
  int32_t* tile_carry = (int32_t*)(ws + L.tile_carry);
  uint32_t* seg_kept = (uint32_t*)(ws + L.seg_kept);
  uint32_t* kept_base = (uint32_t*)(ws + L.kept_base);
  uint32_t* chunk_base = (uint32_t*)(ws + L.chunk_base);
  uint32_t* kept_tmp = (uint32_t*)(ws + L.kept_tmp);
  uint32_t* win_off = (uint32_t*)(ws + L.win_off);
  WinEntry* wtab = (WinEntry*)(ws + L.wtab);
  uint32_t* win_cnt = (uint32_t*)(ws + L.win_cnt);
  uint32_t* win_own = (uint32_t*)(ws + L.win_own);
  uint32_t* win_big = (uint32_t*)(ws + L.win_big);
  uint32_t* win_done = (uint32_t*)(ws + L.win_done);
  uint32_t* whist = (uint32_t*)(ws + L.whist);
  unsigned long long* buf_a = (unsigned long long*)(ws + L.buf_a);
  unsigned long long* buf_b = (unsigned long long*)(ws + L.buf_b);
  const uint32_t n32 = (uint32_t)n;
  const uint32_t S = (uint32_t)state->stage_stride;
  const uint32_t ibits = std::max(1u, ceil_log2(n));
  const uint32_t sbits = ceil_log2(L.n_seg);

  bool prof_coarse = false;
  /* requests grouped by ctx, no ctx beyond a tile: worth testing for when the sizes allow it */
  const uint32_t local_cand = local_sort_candidate(n, n_ctx) ? 1u : 0u;
  /* one ctx that fits a tile: the local sort is certain, no range search, no order check, no fallback passes */
  const bool local_sure = local_cand && n_ctx == 1;
  uint32_t* ctx_start = (uint32_t*)(ws + L.ctx_start);
  cudaEvent_t* evs = profile_acquire(&prof_coarse);
  int phase = 0;
  auto mark = [&]() {                      /* boundary between two phases */
    const bool inner = phase == kPhaseTables + 1 || phase == kPhaseTables + 2;   /* inside the decision pass */
    if (evs && !(prof_coarse && inner)) cudaEventRecord(evs[phase], stream);
    ++phase;
  };
  mark();
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  PipeTable pipe_table = {};
  pipe_table.many = d_pipes;
  if (n_pipelines <= (uint32_t)kFewPipelines)
    for (uint32_t i = 0; i < n_pipelines; ++i) pipe_table.few[i] = h_pipes[i];
  else
    PARD_CUDA_OK(cudaMemcpyAsync(d_pipes, h_pipes.data(), 8ull * n_pipelines, cudaMemcpyHostToDevice, stream));
  rc = allow_sort_smem(dev);
  if (rc != PARD_OK) return rc;
  const uint4* req4 = (const uint4*)d_requests;

  /* ---- keys wider than one sort element: see k_wide_reset.  Run only when a finished call has
   * reported that width (the host cannot know the deadline span beforehand), hence not for
   * PARD_MODE_NOWAIT, whose caller gets PARD_ERANGE from pard_plan_status as before. ---- */
  auto plan_wide = [&]() -> int {
    uint32_t h_wide = 0;
    PARD_CUDA_OK(cudaMemcpyAsync(&h_wide, &hdr->wide, 4, cudaMemcpyDeviceToHost, stream));
    PARD_CUDA_OK(cudaStreamSynchronize(stream));
    if (!h_wide) return PARD_ERANGE;
    const uint32_t grid_n = (uint32_t)std::min<uint64_t>((n + 255) / 256, (uint64_t)sms * 8);
    {
      const unsigned long long n16 = L.zero_end / 16;
      launch_pdl(k_clear, (uint32_t)std::min<unsigned long long>((n16 + 255) / 256, (unsigned long long)sms * 4), 256, 0,
                 stream, (uint4*)(ws + L.hdr), n16);
    }
    launch_pdl(k_prepass, (uint32_t)std::min<uint64_t>((n + 2047) / 2048, (uint64_t)sms * 8), 256, 0, stream, req4, n32, n_ctx,
               S, ctx_dmin, ctx_dmax, hdr);
    launch_pdl(k_ctx_span, (n_ctx + 255) / 256, 256, 0, stream, ctx_dmin, ctx_dmax, n_ctx, hdr);
    launch_pdl(k_key_width, 1, 1, 0, stream, sbits, ibits, hdr, 0u, sbits);
    launch_pdl(k_seg_const, (L.n_seg + 3) / 4, 128, 0, stream, pipe_table, n_pipelines, *state, n_ctx, ctx_dmin, ctx_dmax, ktab,
               hdr, sbits, ibits, 0u, 0u, 0u, 0u, win_off, win_cnt, sbits);
    const uint32_t cw = 64 - ibits;                         /* key bits per super-pass */
    const uint32_t supers = (sbits + 60 + cw - 1) / cw;     /* for the widest legal span; chunks beyond the key are empty */
    const uint32_t chunk_passes = std::min<uint32_t>(kMaxPasses, (cw + 7) / 8);
    uint32_t* order = kept_tmp;
    for (uint32_t sp = 0; sp < supers; ++sp) {
      launch_pdl(k_wide_reset, (uint32_t)std::min<uint64_t>((lb_words + kMaxPasses * kBins + 255) / 256, (uint64_t)sms * 4), 256,
                 0, stream, hdr, hist, lookback, (unsigned long long)lb_words, sbits, ibits, sp);
      launch_pdl(k_wide_pack, grid_n, 256, 0, stream, req4, n32, n_ctx, S, ctx_dmin, ctx_dmax, state->d_priority, sbits, ibits,
                 sp, (const PlanHeader*)hdr, (const uint32_t*)order, buf_a, hist);
      for (uint32_t p = 0; p < chunk_passes; ++p)
        launch_pdl(k_sort_pass<false, false>, L.sort_tiles, kSortThreads, sizeof(SortSmem), stream, p, hdr, buf_a, buf_b, hist,
                   lookback + (p & 1) * lb_words, lookback + ((p + 1) & 1) * lb_words, n32, ibits, 0u, 0u, CtxTiles{});
      launch_pdl(k_wide_chase, grid_n, 256, 0, stream, (const PlanHeader*)hdr, (const unsigned long long*)buf_a, buf_b, n32,
                 ibits, sp, (const uint32_t*)order);
      launch_pdl(k_wide_keep, grid_n, 256, 0, stream, (const PlanHeader*)hdr, (const unsigned long long*)buf_a,
                 (const unsigned long long*)buf_b, n32, order);
    }
    launch_pdl(k_wide_final, grid_n, 256, 0, stream, req4, n32, n_ctx, S, sbits, ibits, hdr, (const uint32_t*)order, buf_a);
    launch_pdl(k_wide_done, 1, 1, 0, stream, hdr, sbits);
    if (L.n_seg >= kManyQueues)
      launch_pdl(k_seg_win_many, ((L.n_seg + 31) / 31 + 7) / 8, 256, 0, stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab,
                 seg_off, out->d_seg_offsets, win_off, win_cnt, win_own, win_big, L.win_capacity, 0u, 0u, seg_kept);
    else
      launch_pdl(k_seg_win, (L.n_seg + 1 + 7) / 8, 256, 0, stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab, seg_off,
                 out->d_seg_offsets, win_off, win_cnt, win_own, win_big, L.win_capacity, 0u, (const uint32_t*)hist, sbits, 0u, 0u, seg_kept);
    PolicyArgs pa = {};
    pa.hdr = hdr; pa.buf_a = buf_a; pa.buf_b = buf_b;
    pa.n = n32; pa.ibits = ibits; pa.n_seg = L.n_seg; pa.mode = mode;
    pa.ktab = ktab; pa.seg_off = seg_off; pa.req = req4; pa.arrivals = d_arrivals;
    pa.pipes = pipe_table; pa.n_pipelines = n_pipelines; pa.st = *state;
    pa.out_keep = out->d_keep; pa.out_est = (long long*)out->d_est_us; pa.out_perm = out->d_perm;
    pa.kept_tmp = out->d_kept_idx ? kept_tmp : nullptr; pa.seg_kept = seg_kept;
    int wrc = launch_policy_decision(pa, sms, stream);
    if (wrc != PARD_OK) return wrc;
    launch_pdl(k_kept_scan, 1, 1024, 0, stream, seg_kept, L.n_seg, kept_base, chunk_base, out->d_seg_kept,
               (unsigned long long*)out->d_n_kept);
    if (out->d_kept_idx)
      launch_pdl(k_kept_move, std::min<uint32_t>(((uint32_t)((n + kCompactChunk - 1) / kCompactChunk) + L.n_seg + 7) / 8,
                                                 (uint32_t)sms * 8), 256, 0, stream,
                 kept_tmp, seg_off, seg_kept, kept_base, chunk_base, L.n_seg, out->d_kept_idx);
    PARD_CUDA_OK(cudaGetLastError());
    return pard_plan_status(d_workspace, cuda_stream);
  };

  /* ---- a block per ctx does everything (k_plan_local): a single ctx within one tile, or the
   * caller's word that the requests come grouped by ctx with no ctx beyond a tile ---- */
  const bool fused_single = n_ctx == 1 && n > 0 && n <= (uint64_t)kSortTile && !rule_walk;
  /* worth it while the blocks fit a few waves: beyond that the streaming decision kernel of the
   * general path (which finds the grouping by itself) does the positions cheaper than the blocks' scans */
  const bool fused_grouped = (mode & PARD_MODE_GROUPED) && n_ctx > 1 && n > 0 && !rule_walk && n_ctx <= 4u * (uint32_t)sms &&
                             !L.ctx_passes;
  if (fused_single || fused_grouped) {
    LocalArgs la = {};
    la.req = req4; la.ctx_start = fused_single ? nullptr : ctx_start;
    la.n = n32; la.n_ctx = n_ctx; la.ibits = ibits; la.raw = (mode & PARD_MODE_RAW) ? 1u : 0u;
    la.pipes = pipe_table; la.n_pipelines = n_pipelines; la.st = *state;
    la.out_keep = out->d_keep; la.out_est = (long long*)out->d_est_us; la.out_perm = out->d_perm;
    la.out_kept_idx = out->d_kept_idx; la.out_n_kept = (unsigned long long*)out->d_n_kept;
    la.out_seg_off = out->d_seg_offsets; la.out_seg_kept = out->d_seg_kept;
    la.ktab = ktab; la.seg_off = seg_off; la.seg_kept = seg_kept; la.kept_tmp = out->d_kept_idx ? kept_tmp : nullptr;
    if (fused_grouped) {
      launch_pdl(k_clear, 4, 256, 0, stream, (uint4*)(ws + L.hdr), (unsigned long long)(L.hist / 16));
      launch_pdl(k_ctx_ranges, (n_ctx + 1 + 7) / 8, 256, 0, stream, req4, n32, n_ctx, ctx_start, hdr, 0u, 0u);
      /* the queues' constants; what depends on a ctx's deadline range is added by the ctx's block */
      launch_pdl(k_seg_const, (L.n_seg + 3) / 4, 128, 0, stream, pipe_table, n_pipelines, *state, n_ctx, ctx_dmin, ctx_dmax,
                 ktab, hdr, sbits, ibits, 0u, 0u, 0u, 0u, win_off, win_cnt, sbits);
    }
    launch_pdl((mode & PARD_MODE_RAW) ? k_plan_local<true, 512> : k_plan_local<false, 512>, n_ctx, 512,
               sizeof(LocalSmem<512>), stream, hdr, la);
    if (fused_grouped) {
      launch_pdl(k_kept_scan, 1, 1024, 0, stream, seg_kept, L.n_seg, kept_base, chunk_base, out->d_seg_kept,
                 (unsigned long long*)out->d_n_kept);
      if (out->d_kept_idx)
        launch_pdl(k_kept_move, std::min<uint32_t>(((uint32_t)((n + kCompactChunk - 1) / kCompactChunk) + L.n_seg + 7) / 8,
                                                   (uint32_t)sms * 8), 256, 0, stream,
                   kept_tmp, seg_off, seg_kept, kept_base, chunk_base, L.n_seg, out->d_kept_idx);
    }
    while (phase <= PARD_N_PHASES) mark();             /* the phases are those of the other path: all of this counts as the first */
    PARD_CUDA_OK(cudaGetLastError());
    if (mode & PARD_MODE_NOWAIT) return PARD_OK;
    rc = pard_plan_status(d_workspace, cuda_stream);
    return rc == PARD_ERANGE ? plan_wide() : rc;
  }

  /* ---- the same promise for more contexts than that: a block per ctx still reads, checks and
   * sorts its ctx (k_plan_local, stopping behind the sort) and publishes the ctx's deadline range,
   * so that neither the prepass over all requests nor the packing and radix kernels (launched
   * otherwise in case the device finds the requests not grouped) are needed; the element format
   * is fixed here (all bits the queue id and the index leave), tables and decision as in the
   * general path ---- */
  if ((mode & PARD_MODE_GROUPED) && n_ctx > 1 && n > 0 && !rule_walk && !L.ctx_passes) {
    const uint32_t fmt_dbits = std::min(60u, 64u - ibits - sbits);
    LocalArgs la = {};
    la.req = req4; la.ctx_start = ctx_start;
    la.n = n32; la.n_ctx = n_ctx; la.ibits = ibits;
    la.pipes = pipe_table; la.n_pipelines = n_pipelines; la.st = *state;
    la.sort_only = 1; la.fmt_dbits = fmt_dbits; la.dst = buf_a; la.ctx_dmin_inv = ctx_dmin; la.ctx_dmax = ctx_dmax;
    launch_pdl(k_clear, 8, 256, 0, stream, (uint4*)(ws + L.hdr), (unsigned long long)(L.hist / 16));
    launch_pdl(k_ctx_ranges, (n_ctx + 1 + 7) / 8, 256, 0, stream, req4, n32, n_ctx, ctx_start, hdr, fmt_dbits, sbits);
    launch_pdl(k_plan_local<false, 512>, n_ctx, 512, sizeof(LocalSmem<512>), stream, hdr, la);
    launch_pdl(k_seg_const, (L.n_seg + 3) / 4, 128, 0, stream, pipe_table, n_pipelines, *state, n_ctx, ctx_dmin, ctx_dmax, ktab,
               hdr, sbits, ibits, 0u, 0u, 0u, 0u, win_off, win_cnt, sbits);
    if (L.n_seg >= kManyQueues)
      launch_pdl(k_seg_win_many, ((L.n_seg + 31) / 31 + 7) / 8, 256, 0, stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab,
                 seg_off, out->d_seg_offsets, win_off, win_cnt, win_own, win_big, L.win_capacity,
                 (mode & PARD_MODE_SCAN) ? 1u : 0u, 1u, seg_kept);
    else
      launch_pdl(k_seg_win, (L.n_seg + 1 + 7) / 8, 256, 0, stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab, seg_off,
                 out->d_seg_offsets, win_off, win_cnt, win_own, win_big, L.win_capacity,
                 (mode & PARD_MODE_SCAN) ? 1u : 0u, (const uint32_t*)hist, sbits, 1u, 1u, seg_kept);
    uint32_t* tmp = out->d_kept_idx ? kept_tmp : nullptr;
    long long* est = (long long*)out->d_est_us;
    const bool raw = mode & PARD_MODE_RAW;
    launch_pdl(k_win_bounds, std::min<uint32_t>((L.win_capacity + 7) / 8, (uint32_t)sms * 8), 256, 0, stream,
        hdr, buf_a, buf_b, ibits, L.n_seg, ktab, seg_off, win_off, win_cnt, win_own, win_big, win_done, wtab, raw ? 1u : 0u, seg_kept);
    launch_pdl(k_win_prefix, (L.n_seg + 7) / 8, 256, 0, stream, hdr, L.n_seg, ktab, seg_off, win_off, win_cnt, wtab, raw ? 1u : 0u, seg_kept);
    launch_pdl(k_kept_scan, 1, 1024, 0, stream, seg_kept, L.n_seg, kept_base, chunk_base, out->d_seg_kept,
               (unsigned long long*)out->d_n_kept);
    auto decide_win = raw ? (state->d_priority ? k_decide_win<true, true> : k_decide_win<true, false>)
                          : (state->d_priority ? k_decide_win<false, true> : k_decide_win<false, false>);
    launch_pdl(decide_win, (uint32_t)((n + (uint64_t)kDecTile - 1) / kDecTile), kDecThreads, 0, stream, hdr, buf_a, buf_b, n32,
               ibits, ktab, seg_off, win_off, win_cnt, wtab, out->d_keep, est, out->d_perm, out->d_kept_idx,
               (const uint32_t*)kept_base, (uint32_t*)nullptr);
    launch_pdl(raw ? k_scan_path<true> : k_scan_path<false>, std::min<uint32_t>(L.dec_tiles, (uint32_t)sms * 2), kDecThreads, 0,
               stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab, seg_off, win_off, tile_agg, tile_carry, out->d_keep, est,
               out->d_perm, tmp, seg_kept, kept_base, chunk_base, out->d_seg_kept, (unsigned long long*)out->d_n_kept,
               out->d_kept_idx, 0u);
    while (phase <= PARD_N_PHASES) mark();
    PARD_CUDA_OK(cudaGetLastError());
    if (mode & PARD_MODE_NOWAIT) return PARD_OK;
    rc = pard_plan_status(d_workspace, cuda_stream);
    return rc == PARD_ERANGE ? plan_wide() : rc;
  }

  /* ---- clear the scratch that must start at zero: one contiguous region ---- */
  {
    const unsigned long long n16 = (n > 0 ? L.zero_end : L.lookback) / 16;   /* offsets are multiples of 256 */
    launch_pdl(k_clear, (uint32_t)std::min<unsigned long long>((n16 + 255) / 256, (unsigned long long)sms * 4), 256, 0,
               stream, (uint4*)(ws + L.hdr), n16);
  }

  mark();
  if (n > 0) {
    uint32_t grid = (uint32_t)std::min<uint64_t>((n + 2047) / 2048, (uint64_t)sms * 8);
    launch_pdl(k_prepass, grid, 256, 0, stream, req4, n32, n_ctx, S, ctx_dmin, ctx_dmax, hdr);
  }
  mark();
  /* Requests grouped by ctx (the caller's word) with contexts of more than a tile on average: the
   * radix passes stay inside every ctx's range -- tiles cut at ctx boundaries, digit counts per
   * ctx, look-back up to the ctx's first tile -- and sort the stage and deadline bits only; the
   * ctx bits of the key need no pass (C5: four passes instead of five).  Needs the stage in the low
   * bits of the queue id: stage_stride a power of two. */
  const bool ctx_sort = (mode & PARD_MODE_GROUPED) && L.ctx_passes && (S & (S - 1)) == 0 && !rule_walk && n > 0;
  const uint32_t key_sbits = ctx_sort ? ceil_log2(S) : sbits;
  const CtxTiles ctx_tiles = {ctx_start, (const uint32_t*)(ws + L.tile_first), (const uint32_t*)(ws + L.hist_ctx), n_ctx};
  const bool fold_width = L.n_seg <= kFoldSegs;          /* few queues: k_seg_const's last block finds the key width */
  if (!fold_width) {
    if (n > 0) launch_pdl(k_ctx_span, (n_ctx + 255) / 256, 256, 0, stream, ctx_dmin, ctx_dmax, n_ctx, hdr);
    launch_pdl(k_key_width, 1, 1, 0, stream, sbits, ibits, hdr, arrival_order ? 1u : 0u, key_sbits);
  }
  /* few queues, decided by the planner's own rule in budget order from the start of every queue:
   * the window tables are counted while the requests are packed */
  const bool win_hist = n > 0 && L.n_seg <= kHistSegs && !rule_walk && !state->d_priority && !local_cand && !ctx_sort;
  launch_pdl(k_seg_const, (L.n_seg + 3) / 4, 128, 0, stream, pipe_table, n_pipelines, *state, n_ctx, ctx_dmin, ctx_dmax, ktab,
             hdr, sbits, ibits, fold_width ? 1u : 0u, arrival_order ? 1u : 0u, win_hist ? 1u : 0u,
             (mode & PARD_MODE_SCAN) ? 1u : 0u, win_off, win_cnt, key_sbits);
  if ((local_cand && !local_sure) || ctx_sort)
    launch_pdl(k_ctx_ranges, (n_ctx + 1 + 7) / 8, 256, 0, stream, req4, n32, n_ctx, ctx_start, hdr, 0u, 0u);
  if (ctx_sort) launch_pdl(k_tile_table, 1, 1024, 0, stream, (const uint32_t*)ctx_start, n_ctx, (uint32_t*)(ws + L.tile_first));
  mark();
  if (local_cand)                                /* every ctx inside one tile: sorted block by block, straight from the requests */
    launch_pdl(k_sort_local, n_ctx, kSortThreads, sizeof(SortSmem), stream, hdr, local_cand, req4, ctx_dmin, ctx_dmax,
               state->d_priority, buf_a, buf_b, local_sure ? (const uint32_t*)nullptr : (const uint32_t*)ctx_start, n32, S,
               ceil_log2(S), ibits);
  if (ctx_sort) {
    launch_pdl(k_pack_ctx, L.lb_tiles, 256, 0, stream, req4, S, ctx_dmin, ctx_dmax, state->d_priority, ibits, hdr, buf_a,
               (uint32_t*)(ws + L.hist_ctx), ctx_tiles);
  } else if (n > 0 && !local_sure) {             /* returns at once when the blocks above did the work */
    uint32_t grid = (uint32_t)std::min<uint64_t>((n + 255) / 256, (uint64_t)sms * 8);
    launch_pdl(win_hist ? k_pack<true> : k_pack<false>, grid, 256, 0, stream, req4, n32, n_ctx, S, ctx_dmin, ctx_dmax,
               state->d_priority, ibits, hdr, buf_a, hist, local_cand, (const PardSegConst*)ktab, (const uint32_t*)win_off,
               (const uint32_t*)win_cnt, whist);
    if (win_hist)
      launch_pdl(k_win_from_counts, 1, 1024, 0, stream, hdr, L.n_seg, (const PardSegConst*)ktab, (const uint32_t*)whist,
                 (const uint32_t*)win_off, (const uint32_t*)win_cnt, wtab, seg_off, out->d_seg_offsets,
                 (mode & PARD_MODE_RAW) ? 1u : 0u, seg_kept, out->d_seg_kept, kept_base, (unsigned long long*)out->d_n_kept,
                 (const uint32_t*)hist, sbits);
  }
  for (uint32_t p = 0; p < (uint32_t)kMaxPasses; ++p) {
    mark();
    if (ctx_sort) {
      if (p < std::min<uint32_t>(kMaxPasses, (key_sbits + 60 + 7) / 8))
        launch_pdl(k_sort_pass<false, true>, L.lb_tiles, kSortThreads, sizeof(SortSmem), stream, p, hdr, buf_a, buf_b, hist,
                   lookback + (p & 1) * lb_words, lookback + ((p + 1) & 1) * lb_words, n32, ibits, 0u, 0u, ctx_tiles);
    } else if (n > 0 && p < L.max_passes && !local_sure)
      launch_pdl(local_cand ? k_sort_pass<true, false> : k_sort_pass<false, false>,
                 local_cand ? std::min<uint32_t>(L.sort_tiles, 2u * (uint32_t)sms) : L.sort_tiles, kSortThreads, sizeof(SortSmem), stream,
          p, hdr, buf_a, buf_b, hist, lookback + (p & 1) * lb_words, lookback + ((p + 1) & 1) * lb_words,
          n32, ibits, (p == 0 && (mode & PARD_MODE_TEST_STALL)) ? 1u : 0u, local_cand, CtxTiles{});
  }
  mark();
  if (win_hist) {
    /* boundaries and tables are there already */
  } else if (L.n_seg >= kManyQueues)
    launch_pdl(k_seg_win_many, ((L.n_seg + 31) / 31 + 7) / 8, 256, 0, stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab,
               seg_off, out->d_seg_offsets, win_off, win_cnt, win_own, win_big, L.win_capacity,
               (mode & PARD_MODE_SCAN) ? 1u : 0u, rule_walk ? 0u : 1u, seg_kept);
  else
    launch_pdl(k_seg_win, (L.n_seg + 1 + 7) / 8, 256, 0, stream, hdr, buf_a, buf_b, n32, ibits, L.n_seg, ktab, seg_off,
               out->d_seg_offsets, win_off, win_cnt, win_own, win_big, L.win_capacity,
               (mode & PARD_MODE_SCAN) ? 1u : 0u, (const uint32_t*)hist, ctx_sort ? 64u : sbits, local_cand, rule_walk ? 0u : 1u, seg_kept);
  if (n > 0 && rule_walk) {
    /* a rule without rising thresholds: every queue is walked in order (pard_policy.cu) */
    PolicyArgs pa = {};
    pa.hdr = hdr; pa.buf_a = buf_a; pa.buf_b = buf_b;
    pa.n = n32; pa.ibits = ibits; pa.n_seg = L.n_seg; pa.mode = mode;
    pa.ktab = ktab; pa.seg_off = seg_off; pa.req = req4; pa.arrivals = d_arrivals;
    pa.pipes = pipe_table; pa.n_pipelines = n_pipelines; pa.st = *state;
    pa.out_keep = out->d_keep; pa.out_est = (long long*)out->d_est_us; pa.out_perm = out->d_perm;
    pa.kept_tmp = out->d_kept_idx ? kept_tmp : nullptr; pa.seg_kept = seg_kept;
    mark();
    rc = launch_policy_decision(pa, sms, stream);
    if (rc != PARD_OK) return rc;
  } else if (n > 0) {
    uint32_t* tmp = out->d_kept_idx ? kept_tmp : nullptr;
    long long* est = (long long*)out->d_est_us;
    const bool raw = mode & PARD_MODE_RAW;
    /* window tables, and the decision from them */
    if (!win_hist) {
      launch_pdl(k_win_bounds, std::min<uint32_t>((L.win_capacity + 7) / 8, (uint32_t)sms * 8), 256, 0, stream,
          hdr, buf_a, buf_b, ibits, L.n_seg, ktab, seg_off, win_off, win_cnt, win_own, win_big, win_done, wtab, raw ? 1u : 0u, seg_kept);
      launch_pdl(k_win_prefix, (L.n_seg + 7) / 8, 256, 0, stream, hdr, L.n_seg, ktab, seg_off, win_off, win_cnt, wtab, raw ? 1u : 0u, seg_kept);
      /* the tables give every queue's kept count: the output offsets are known before the decision */
      launch_pdl(k_kept_scan, 1, 1024, 0, stream, seg_kept, L.n_seg, kept_base, chunk_base, out->d_seg_kept,
                 (unsigned long long*)out->d_n_kept);
    }
    mark();
    const uint32_t win_grid = (uint32_t)((n + (uint64_t)kDecTile - 1) / kDecTile);
    auto decide_win = raw ? (state->d_priority ? k_decide_win<true, true> : k_decide_win<true, false>)
                          : (state->d_priority ? k_decide_win<false, true> : k_decide_win<false, false>);
    /* the survivors go straight to their place in the output */
    launch_pdl(decide_win, win_grid, kDecThreads, 0, stream, hdr, buf_a, buf_b, n32, ibits, ktab, seg_off, win_off, win_cnt, wtab,
               out->d_keep, est, out->d_perm, out->d_kept_idx, (const uint32_t*)kept_base, (uint32_t*)nullptr);
    /* fallback when a queue has too many batch windows: the same decision by scanning, one kernel
     * that returns at once otherwise */
    const uint32_t scan_grid = std::min<uint32_t>(L.dec_tiles, (uint32_t)sms * 2);
    launch_pdl(raw ? k_scan_path<true> : k_scan_path<false>, scan_grid, kDecThreads, 0, stream, hdr, buf_a, buf_b, n32, ibits,
               L.n_seg, ktab, seg_off, win_off, tile_agg, tile_carry, out->d_keep, est, out->d_perm, tmp, seg_kept, kept_base,
               chunk_base, out->d_seg_kept, (unsigned long long*)out->d_n_kept, out->d_kept_idx,
               (mode & PARD_MODE_TEST_STALL) ? 1u : 0u);
  }
  if (n == 0) mark();
  mark();
  if (rule_walk || n == 0) {                       /* the queue walk leaves per-queue lists; an empty call still owes its zeros */
    launch_pdl(k_kept_scan, 1, 1024, 0, stream, seg_kept, L.n_seg, kept_base, chunk_base, out->d_seg_kept,
               (unsigned long long*)out->d_n_kept);
    if (n > 0 && out->d_kept_idx)
      launch_pdl(k_kept_move, std::min<uint32_t>(((uint32_t)((n + kCompactChunk - 1) / kCompactChunk) + L.n_seg + 7) / 8,
                                                 (uint32_t)sms * 8), 256, 0, stream,
          kept_tmp, seg_off, seg_kept, kept_base, chunk_base, L.n_seg, out->d_kept_idx);
  }
  mark();
  PARD_CUDA_OK(cudaGetLastError());
  if (mode & PARD_MODE_NOWAIT) return PARD_OK;
  rc = pard_plan_status(d_workspace, cuda_stream);
  return (rc == PARD_ERANGE && n > 0) ? plan_wide() : rc;
}

extern "C" int pard_plan_status(const void* d_workspace, void* cuda_stream) {
  if (!d_workspace) return PARD_EINVAL;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  uint32_t h_status = 0;
  PARD_CUDA_OK(cudaMemcpyAsync(&h_status, &((const PlanHeader*)d_workspace)->status, 4,
                               cudaMemcpyDeviceToHost, stream));
  PARD_CUDA_OK(cudaStreamSynchronize(stream));
  return h_status ? -(int)h_status : PARD_OK;
}

extern "C" int pard_plan_kernel_launches(uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                                         uint32_t* launches) {
  uint64_t bytes;
  if (!launches) return PARD_EINVAL;
  int rc = pard_plan_workspace_bytes(n, n_ctx, stage_stride, &bytes);
  if (rc != PARD_OK) return rc;
  /* For the planner's own rule without priorities and without PARD_MODE_GROUPED.  One ctx of at
   * most a sort tile: one kernel.  Else always clear and seg_const; with many queues also
   * key_width (and, when n > 0, ctx_span); when n > 0: prepass, pack, the radix passes, decide_win
   * and the scan path (one kernel that returns at once); with at most 64 queues the counted window
   * tables (win_from_counts), else the queue boundaries, the searched tables and the output
   * offsets that follow from them (seg_win, win_bounds, win_prefix, kept_scan). */
  const uint64_t n_seg = (uint64_t)n_ctx * (uint64_t)stage_stride;
  const uint32_t width_kernels = n_seg <= kFoldSegs ? 0 : 1;   /* key_width (+ ctx_span when n > 0) */
  const bool local_cand = local_sort_candidate(n, n_ctx);
  const uint32_t local_kernels = local_cand ? 2 : 0;            /* ctx_ranges, sort_local */
  const uint32_t passes = make_layout(n, n_ctx, stage_stride).max_passes;
  const bool counted = n > 0 && n_seg <= kHistSegs && !local_cand;
  if (n_ctx == 1 && n > 0 && n <= (uint64_t)kSortTile) *launches = 1;
  else if (n == 0) *launches = 4 + width_kernels;               /* clear, (key_width,) seg_const, seg_win, kept_scan */
  else *launches = 2 + 2 * width_kernels + 2 + local_kernels + passes + 2 + (counted ? 1 : 4);
  return PARD_OK;
}

extern "C" int pard_profile_begin(uint32_t every, uint32_t max_samples) {
  const bool coarse = (every & PARD_PROFILE_COARSE) != 0;
  every &= ~PARD_PROFILE_COARSE;
  if (every < 1 || max_samples < 1 || max_samples > 65536) return PARD_EINVAL;
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (g_prof.on.load()) return PARD_EINVAL;
  g_prof.ev.assign((size_t)max_samples * kEventsPerSample, nullptr);
  for (auto& e : g_prof.ev)
    if (cudaEventCreate(&e) != cudaSuccess) {
      for (auto& f : g_prof.ev) if (f) cudaEventDestroy(f);
      g_prof.ev.clear();
      return PARD_ECUDA;
    }
  g_prof.every = every;
  g_prof.coarse = coarse;
  g_prof.max_samples = max_samples;
  g_prof.calls = 0;
  g_prof.n_samples = 0;
  g_prof.last = nullptr;
  g_prof.on.store(true, std::memory_order_release);
  return PARD_OK;
}

extern "C" int pard_profile_end(float* ms_sum, uint32_t* n_samples) {
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (!g_prof.on.load()) return PARD_EINVAL;
  int rc = PARD_OK;
  if (ms_sum) for (int i = 0; i < PARD_N_PHASES; ++i) ms_sum[i] = 0.f;
  for (uint32_t s = 0; s < g_prof.n_samples; ++s) {
    cudaEvent_t* e = g_prof.ev.data() + (size_t)s * kEventsPerSample;
    if (cudaEventSynchronize(e[PARD_N_PHASES]) != cudaSuccess) { rc = PARD_ECUDA; break; }
    for (int i = 0; i < PARD_N_PHASES && ms_sum; ++i) {
      float ms = 0.f;
      int to = i + 1;
      if (g_prof.coarse && i == kPhaseTables) to = PARD_N_PHASES;       /* the decision pass as one phase */
      if (g_prof.coarse && i > kPhaseTables) continue;
      if (cudaEventElapsedTime(&ms, e[i], e[to]) != cudaSuccess) rc = PARD_ECUDA;
      ms_sum[i] += ms;
    }
  }
  if (n_samples) *n_samples = g_prof.n_samples;
  for (auto& e : g_prof.ev) cudaEventDestroy(e);
  g_prof.ev.clear();
  g_prof.last = nullptr;
  g_prof.on.store(false, std::memory_order_release);
  return rc;
}

extern "C" const char* pard_profile_phase_name(uint32_t phase) {
  static const char* names[PARD_N_PHASES] = {"clear", "prepass", "segments", "pack", "sort0", "sort1",
                                              "sort2", "sort3", "sort4", "sort5", "sort6", "sort7",
                                              "tables", "decide", "compact"};
  return phase < PARD_N_PHASES ? names[phase] : "";
}
