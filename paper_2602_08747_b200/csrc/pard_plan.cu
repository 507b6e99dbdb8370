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
#include <cstring>
#include <mutex>

#include "pard_internal.h"

namespace {

constexpr int kMaxPasses = 8;
constexpr int kBins = 256;
constexpr uint32_t kUClamp = (1u << 30) - 1;       /* >= any request count      */
constexpr uint32_t kMaxPipelinesPerCall = 65536;
constexpr uint32_t kSpinLimit = 1u << 22;          /* polls before giving up    */

constexpr int kSortThreads = 256;
constexpr int kSortItems = 16;
constexpr int kSortTile = kSortThreads * kSortItems;
constexpr int kDecThreads = 256;
constexpr int kDecItems = 8;
constexpr int kDecTile = kDecThreads * kDecItems;
constexpr int kSmemSegs = 4096;                    /* segment histogram kept in shared memory up to here */

/* look-back word of the sort: [31:30] state, [29:0] count */
constexpr uint32_t kLbAgg = 1u << 30;
constexpr uint32_t kLbIncl = 2u << 30;
constexpr uint32_t kLbMask = (1u << 30) - 1;
/* look-back words of the decision pass: [63:62] state */
constexpr unsigned long long kStAgg = 1ull << 62;
constexpr unsigned long long kStIncl = 2ull << 62;

struct PlanHeader {
  uint32_t status;            /* 0, or the positive value of a pard_status */
  uint32_t dbits;             /* bits of the widest per-ctx deadline span  */
  uint32_t keybits;           /* segment bits + dbits                      */
  uint32_t npass;             /* radix passes that run                     */
  unsigned long long span_max;
  uint32_t ticket[kMaxPasses + 1];
  uint32_t wide;              /* 1: segment, deadline and index bits exceed 64; nothing is sorted */
  uint32_t pad[64 - 7 - (kMaxPasses + 1)];
};
static_assert(sizeof(PlanHeader) == 256, "header is 256 bytes");

struct Layout {
  uint64_t hdr, pipes, ctx_dmin, ctx_dmax, seg_off, ktab, hist, lookback, st_min, st_kept,
      buf_a, buf_b, total;
  uint32_t n_seg, sort_tiles, dec_tiles, max_passes;
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
  L.pipes = o;     o = al(o + 8ull * kMaxPipelinesPerCall);
  L.ctx_dmin = o;  o = al(o + 8ull * n_ctx);
  L.ctx_dmax = o;  o = al(o + 8ull * n_ctx);
  L.seg_off = o;   o = al(o + 4ull * (L.n_seg + 1));
  L.ktab = o;      o = al(o + sizeof(PardSegConst) * (uint64_t)L.n_seg);
  L.hist = o;      o = al(o + 4ull * kMaxPasses * kBins);
  L.lookback = o;  o = al(o + 4ull * kBins * (uint64_t)L.sort_tiles * L.max_passes);
  L.st_min = o;    o = al(o + 8ull * L.dec_tiles);
  L.st_kept = o;   o = al(o + 8ull * L.dec_tiles);
  L.buf_a = o;     o = al(o + 8ull * n);
  L.buf_b = o;     o = al(o + 8ull * n);
  L.total = o;
  return L;
}

__device__ __forceinline__ void set_status(PlanHeader* hdr, int status) {
  atomicCAS(&hdr->status, 0u, (uint32_t)(-status));
}

__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

/* ------------------------------------------------------------------------ */
/* prepass: one coalesced 16-byte read per request                           */
/* ------------------------------------------------------------------------ */
template <bool SMEM_HIST>
__global__ void __launch_bounds__(256)
k_prepass(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t S, uint32_t n_seg,
          unsigned long long* __restrict__ ctx_dmin, unsigned long long* __restrict__ ctx_dmax,
          uint32_t* __restrict__ seg_count, PlanHeader* hdr) {
  __shared__ uint32_t s_hist[SMEM_HIST ? kSmemSegs : 1];
  const uint32_t lane = threadIdx.x & 31;
  if (SMEM_HIST) {
    for (uint32_t s = threadIdx.x; s < n_seg; s += blockDim.x) s_hist[s] = 0;
    __syncthreads();
  }
  constexpr uint32_t kNone = 0xffffffffu;
  uint32_t run_ctx = kNone;                 /* warp-uniform */
  unsigned long long lmin = ~0ull, lmax = 0;
  bool bad_seen = false;

  auto flush = [&]() {
    if (run_ctx == kNone) return;
    for (int o = 16; o; o >>= 1) {
      unsigned long long a = __shfl_xor_sync(0xffffffffu, lmin, o);
      unsigned long long b = __shfl_xor_sync(0xffffffffu, lmax, o);
      lmin = a < lmin ? a : lmin;
      lmax = b > lmax ? b : lmax;
    }
    if (lane == 0 && lmin <= lmax) {
      atomicMin(&ctx_dmin[run_ctx], lmin);
      atomicMax(&ctx_dmax[run_ctx], lmax);
    }
    lmin = ~0ull;
    lmax = 0;
  };

  const uint64_t chunk = (uint64_t)blockDim.x * 8;
  for (uint64_t base = (uint64_t)blockIdx.x * chunk; base < n; base += (uint64_t)gridDim.x * chunk) {
#pragma unroll 4
    for (int i = 0; i < 8; ++i) {
      uint64_t j = base + (uint64_t)i * blockDim.x + threadIdx.x;
      bool ok = j < n;
      uint4 r = make_uint4(0, 0, 0, 0);
      if (ok) r = __ldg(&req[j]);
      long long D = (long long)(((unsigned long long)r.y << 32) | r.x);
      uint32_t ctx = r.z, stage = r.w & 0xffffu;
      if (ok && (D < 0 || D >= PARD_TIME_LIMIT_US || ctx >= n_ctx || stage >= S)) {
        bad_seen = true;
        ok = false;
      }
      uint32_t seg = ok ? ctx * S + stage : 0;
      if (SMEM_HIST) {
        if (ok) atomicAdd(&s_hist[seg], 1u);
      } else {
        uint32_t grp = __match_any_sync(0xffffffffu, ok ? seg : 0xffffffffu);
        if (ok && lane == (uint32_t)(__ffs(grp) - 1)) atomicAdd(&seg_count[seg], (uint32_t)__popc(grp));
      }
      uint32_t vmask = __ballot_sync(0xffffffffu, ok);
      if (vmask == 0) continue;
      uint32_t c0 = __shfl_sync(0xffffffffu, ctx, __ffs(vmask) - 1);
      bool uniform = __all_sync(0xffffffffu, !ok || ctx == c0);
      if (uniform) {
        if (run_ctx != c0) {
          flush();
          run_ctx = c0;
        }
        if (ok) {
          lmin = (unsigned long long)D < lmin ? (unsigned long long)D : lmin;
          lmax = (unsigned long long)D > lmax ? (unsigned long long)D : lmax;
        }
      } else if (ok) {
        atomicMin(&ctx_dmin[ctx], (unsigned long long)D);
        atomicMax(&ctx_dmax[ctx], (unsigned long long)D);
      }
    }
  }
  flush();
  if (bad_seen) set_status(hdr, PARD_EDATA);
  if (SMEM_HIST) {
    __syncthreads();
    for (uint32_t s = threadIdx.x; s < n_seg; s += blockDim.x)
      if (s_hist[s]) atomicAdd(&seg_count[s], s_hist[s]);
  }
}

__global__ void k_ctx_span(const unsigned long long* __restrict__ ctx_dmin,
                           const unsigned long long* __restrict__ ctx_dmax, uint32_t n_ctx,
                           PlanHeader* hdr) {
  uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
  unsigned long long span = 0;
  if (c < n_ctx && ctx_dmin[c] <= ctx_dmax[c]) span = ctx_dmax[c] - ctx_dmin[c];
  for (int o = 16; o; o >>= 1) {
    unsigned long long a = __shfl_xor_sync(0xffffffffu, span, o);
    span = a > span ? a : span;
  }
  if ((threadIdx.x & 31) == 0 && span) atomicMax(&hdr->span_max, span);
}

/* Exclusive scan of the queue lengths by one block; also fixes the key width. */
__global__ void __launch_bounds__(1024)
k_seg_scan(uint32_t* __restrict__ seg_off /* in: counts, out: offsets, [n_seg+1] */,
           uint32_t n_seg, uint32_t* __restrict__ out_seg_off, uint32_t sbits, uint32_t ibits,
           PlanHeader* hdr) {
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_carry;
  if (threadIdx.x == 0) {
    s_carry = 0;
    uint32_t dbits = bit_width64(hdr->span_max);
    hdr->dbits = dbits;
    hdr->keybits = sbits + dbits;
    hdr->npass = (sbits + dbits + 7) / 8;
    if (sbits + dbits + ibits > 64) {
      hdr->npass = 0;
      hdr->wide = 1;
      set_status(hdr, PARD_ERANGE);
    }
  }
  __syncthreads();
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (uint32_t base = 0; base < n_seg + 1; base += 1024) {
    uint32_t i = base + threadIdx.x;
    uint32_t v = (i < n_seg) ? seg_off[i] : 0;
    uint32_t x = v;
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= (uint32_t)o) x += y;
    }
    if (lane == 31) s_warp[warp] = x;
    __syncthreads();
    if (warp == 0) {
      uint32_t w = s_warp[lane], t = w;
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= (uint32_t)o) t += y;
      }
      s_warp[lane] = t - w;
    }
    __syncthreads();
    uint32_t excl = s_carry + s_warp[warp] + x - v;
    if (i <= n_seg) {
      seg_off[i] = excl;
      if (out_seg_off) out_seg_off[i] = excl;
    }
    __syncthreads();
    if (threadIdx.x == 1023) s_carry = excl + v;
    __syncthreads();
  }
}

/* Per-segment constants; one thread per (ctx, stage). */
__global__ void k_seg_const(const PardPipeDev* const* __restrict__ pipes, uint32_t n_pipelines,
                            pard_queue_state_t st, uint32_t n_ctx,
                            const unsigned long long* __restrict__ ctx_dmin,
                            const uint32_t* __restrict__ seg_off, PardSegConst* __restrict__ ktab,
                            PlanHeader* hdr) {
  const uint32_t S = (uint32_t)st.stage_stride;
  uint32_t seg = blockIdx.x * blockDim.x + threadIdx.x;
  if (seg >= n_ctx * S) return;
  uint32_t c = seg / S, k = seg % S;
  PardSegConst out;
  out.A = 0; out.A_rel = 0; out.d = 1; out.cap = 1; out.pad = 0;
  int32_t pi = st.d_pipeline_of_ctx ? st.d_pipeline_of_ctx[c] : 0;
  bool bad = false;
  if (pi < 0 || (uint32_t)pi >= n_pipelines) {
    bad = true;
  } else {
    const PardPipeDev* p = pipes[pi];
    const int64_t* qrow = st.d_q_us + (size_t)c * S;
    const int32_t* brow = st.d_batch + (size_t)c * S;
    if (k >= (uint32_t)p->n_stages) {
      if (seg_off[seg + 1] != seg_off[seg]) bad = true;   /* requests queued at a stage that does not exist */
    } else {
      int32_t B = brow[k];
      int64_t m = st.d_workers ? st.d_workers[(size_t)c * S + k] : 1;
      int64_t now = st.d_now_us[c], fa = st.d_free_at_us[(size_t)c * S + k];
      if (B < 1 || B > p->bmax[k] || m < 1 || now < 0 || now >= PARD_TIME_LIMIT_US || fa < 0 ||
          fa >= PARD_TIME_LIMIT_US) {
        bad = true;
      } else {
        int64_t d = p->lat_us[p->lat_offsets[k] + B - 1];
        int64_t lsub = 0;
        const int32_t s0 = p->stage_slot_off[k], s1 = p->stage_slot_off[k + 1];
        for (int32_t s = s0; s < s1; ++s) {             /* every downstream path */
          int64_t acc = st.d_w_us ? st.d_w_us[(size_t)c * st.slot_stride + s] : 0;
          if (acc < 0 || acc >= PARD_TIME_LIMIT_US) { bad = true; acc = 0; }
          for (int32_t e = p->path_off[s]; e < p->path_off[s + 1]; ++e) {
            int32_t i = p->path_stage[e];
            int32_t Bi = brow[i];
            int64_t qi = qrow[i];
            if (Bi < 1 || Bi > p->bmax[i] || qi < 0 || qi >= PARD_TIME_LIMIT_US) { bad = true; Bi = 1; qi = 0; }
            acc += qi + p->lat_us[p->lat_offsets[i] + Bi - 1];
          }
          lsub = (s == s0 || acc > lsub) ? acc : lsub;
        }
        int64_t base = now > fa ? now : fa;
        int64_t cap = (int64_t)B * m;
        out.d = d;
        out.cap = (uint32_t)(cap > (int64_t)(1u << 30) ? (int64_t)(1u << 30) : cap);
        out.A = base + d + lsub;
        out.A_rel = out.A - (int64_t)ctx_dmin[c];
      }
    }
  }
  if (bad) set_status(hdr, PARD_EDATA);
  ktab[seg] = out;
}

/* request -> sort element; digit histograms of every pass */
__global__ void __launch_bounds__(256)
k_pack(const uint4* __restrict__ req, uint32_t n, uint32_t n_ctx, uint32_t S,
       const unsigned long long* __restrict__ ctx_dmin, uint32_t ibits,
       const PlanHeader* __restrict__ hdr, unsigned long long* __restrict__ dst,
       uint32_t* __restrict__ hist) {
  __shared__ uint32_t s_hist[kMaxPasses * kBins];
  if (hdr->wide) return;
  const uint32_t npass = hdr->npass, dbits = hdr->dbits;
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x) s_hist[i] = 0;
  __syncthreads();
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride) {
    uint4 r = __ldg(&req[j]);
    unsigned long long D = ((unsigned long long)r.y << 32) | r.x;
    uint32_t ctx = r.z, stage = r.w & 0xffffu;
    unsigned long long e;
    if (ctx < n_ctx && stage < S) {
      unsigned long long off = (D - ctx_dmin[ctx]) & dmask;
      e = ((((unsigned long long)(ctx * S + stage) << dbits) | off) << ibits) | j;
    } else {
      e = j;                                  /* flagged by the prepass; keep indices in range */
    }
    dst[j] = e;
    unsigned long long key = e >> ibits;
    for (uint32_t p = 0; p < npass; ++p) atomicAdd(&s_hist[p * kBins + ((key >> (8 * p)) & 255u)], 1u);
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < npass * kBins; i += blockDim.x)
    if (s_hist[i]) atomicAdd(&hist[i], s_hist[i]);
}

/* ------------------------------------------------------------------------ */
/* one LSD radix pass (8 bits), stable, tile prefixes by decoupled look-back */
/* ------------------------------------------------------------------------ */
__global__ void __launch_bounds__(kSortThreads)
k_sort_pass(uint32_t pass, PlanHeader* hdr, unsigned long long* __restrict__ buf_a,
            unsigned long long* __restrict__ buf_b, const uint32_t* __restrict__ hist,
            uint32_t* __restrict__ lookback, uint32_t n, uint32_t ibits) {
  constexpr int WARPS = kSortThreads / 32;
  __shared__ unsigned long long s_keys[kSortTile];
  __shared__ uint32_t s_whist[WARPS][kBins];
  __shared__ uint32_t s_dstart[kBins];
  __shared__ uint32_t s_gofs[kBins];
  __shared__ uint32_t s_scan[WARPS];
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_abort;

  if (pass >= hdr->npass) return;
  const unsigned long long* src = (pass & 1) ? buf_b : buf_a;
  unsigned long long* dst = (pass & 1) ? buf_a : buf_b;
  hist += pass * kBins;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_tile = atomicAdd(&hdr->ticket[pass], 1u);
    s_abort = 0;
  }
  for (int w = 0; w < WARPS; ++w) s_whist[w][tid] = 0;
  __syncthreads();
  const uint32_t tile = s_tile;
  const uint64_t base = (uint64_t)tile * kSortTile;
  const uint32_t shift = ibits + 8 * pass;

  unsigned long long key[kSortItems];
  uint32_t rank[kSortItems];
#pragma unroll
  for (int i = 0; i < kSortItems; ++i) {
    uint64_t j = base + warp * (32 * kSortItems) + i * 32 + lane;
    key[i] = j < n ? src[j] : ~0ull;
  }
#pragma unroll
  for (int i = 0; i < kSortItems; ++i) {
    uint32_t d = (uint32_t)(key[i] >> shift) & 255u;
    uint32_t grp = __match_any_sync(0xffffffffu, d);
    uint32_t leader = __ffs(grp) - 1;
    uint32_t old = 0;
    if (lane == leader) {
      old = s_whist[warp][d];
      s_whist[warp][d] = old + __popc(grp);
    }
    old = __shfl_sync(0xffffffffu, old, leader);
    rank[i] = old + __popc(grp & lanemask_lt());
    __syncwarp();
  }
  __syncthreads();

  /* thread d owns digit d: counts across warps -> exclusive warp offsets */
  uint32_t cnt = 0;
#pragma unroll
  for (int w = 0; w < WARPS; ++w) {
    uint32_t t = s_whist[w][tid];
    s_whist[w][tid] = cnt;
    cnt += t;
  }
  /* exclusive scans over the 256 digits: the tile's counts and the global histogram */
  uint32_t gh = hist[tid];
  uint32_t x = cnt, g = gh;
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
    uint32_t z = __shfl_up_sync(0xffffffffu, g, o);
    if (lane >= (uint32_t)o) { x += y; g += z; }
  }
  __shared__ uint32_t s_scan_g[WARPS];
  if (lane == 31) { s_scan[warp] = x; s_scan_g[warp] = g; }
  __syncthreads();
  uint32_t wx = 0, wg = 0;
#pragma unroll
  for (int w = 0; w < WARPS; ++w)
    if (w < (int)warp) { wx += s_scan[w]; wg += s_scan_g[w]; }
  const uint32_t dstart = wx + x - cnt;        /* first local position of digit tid  */
  const uint32_t gstart = wg + g - gh;         /* first global position of digit tid */
  s_dstart[tid] = dstart;

  /* publish the tile's count, then sum the counts of all earlier tiles */
  volatile uint32_t* lb = lookback;            /* this pass's array */
  lb[(size_t)tile * kBins + tid] = cnt | kLbAgg;
  uint32_t excl = 0;
  for (int64_t t = (int64_t)tile - 1; t >= 0; --t) {
    uint32_t v, spins = 0;
    while (((v = lb[(size_t)t * kBins + tid]) >> 30) == 0) {
      if (++spins > kSpinLimit) { s_abort = 1; break; }
      __nanosleep(20);
    }
    if ((v >> 30) == 0) break;
    excl += v & kLbMask;
    if (v & kLbIncl) break;
  }
  lb[(size_t)tile * kBins + tid] = ((excl + cnt) & kLbMask) | kLbIncl;
  s_gofs[tid] = gstart + excl - dstart;
  __syncthreads();
  if (s_abort) {
    if (tid == 0) set_status(hdr, PARD_ETIMEOUT);
    return;
  }

#pragma unroll
  for (int i = 0; i < kSortItems; ++i) {
    uint32_t d = (uint32_t)(key[i] >> shift) & 255u;
    s_keys[s_dstart[d] + s_whist[warp][d] + rank[i]] = key[i];
  }
  __syncthreads();
  const uint32_t nvalid = (uint32_t)min((uint64_t)kSortTile, (uint64_t)n - base);
  for (uint32_t pos = tid; pos < nvalid; pos += kSortThreads) {
    unsigned long long k = s_keys[pos];
    uint32_t d = (uint32_t)(k >> shift) & 255u;
    dst[s_gofs[d] + pos] = k;
  }
}

/* ------------------------------------------------------------------------ */
/* decision pass over the sorted elements                                    */
/* ------------------------------------------------------------------------ */
struct SegMin {            /* value of a segmented running minimum */
  int32_t m;               /* minimum of u_t - t since the last queue head (or since the span's start) */
  uint32_t head;           /* a queue head lies inside the span */
};

__device__ __forceinline__ SegMin seg_combine(SegMin left, SegMin right) {
  SegMin r;
  r.m = right.head ? right.m : min(left.m, right.m);
  r.head = left.head | right.head;
  return r;
}

__device__ __forceinline__ unsigned long long pack_min(SegMin a, unsigned long long state) {
  return state | ((unsigned long long)a.head << 32) | (uint32_t)a.m;
}
__device__ __forceinline__ SegMin unpack_min(unsigned long long w) {
  SegMin a;
  a.m = (int32_t)(uint32_t)w;
  a.head = (uint32_t)(w >> 32) & 1u;
  return a;
}

__device__ __forceinline__ uint32_t threshold_u(int64_t X, int64_t d, uint32_t cap) {
  /* number of requests that may be admitted ahead of or at this one while it
   * still completes by its deadline: 0 if even position 0 is late, else
   * cap * (floor(X / d) + 1), saturated */
  if (X < 0) return 0;
  unsigned long long q;
  if (((unsigned long long)X | (unsigned long long)d) >> 32)
    q = (unsigned long long)X / (unsigned long long)d;
  else
    q = (uint32_t)X / (uint32_t)d;
  if (q >= kUClamp) return kUClamp;
  unsigned long long u = (q + 1) * cap;
  return u > kUClamp ? kUClamp : (uint32_t)u;
}

__global__ void __launch_bounds__(kDecThreads)
k_decide(PlanHeader* hdr, const unsigned long long* __restrict__ buf_a,
         const unsigned long long* __restrict__ buf_b, uint32_t n, uint32_t ibits, uint32_t mode,
         const PardSegConst* __restrict__ ktab, const uint32_t* __restrict__ seg_off,
         unsigned long long* st_min, unsigned long long* st_kept,
         uint8_t* __restrict__ out_keep, long long* __restrict__ out_est,
         uint32_t* __restrict__ out_perm, uint32_t* __restrict__ out_kept_idx,
         unsigned long long* __restrict__ out_n_kept, uint32_t* __restrict__ out_seg_kept) {
  constexpr int WARPS = kDecThreads / 32;
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_abort;
  __shared__ int32_t s_wm[WARPS];
  __shared__ uint32_t s_wh[WARPS];
  __shared__ uint32_t s_wk[WARPS];
  __shared__ int32_t s_carry_m;
  __shared__ uint32_t s_carry_k;

  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (hdr->wide) return;
  if (tid == 0) {
    s_tile = atomicAdd(&hdr->ticket[kMaxPasses], 1u);
    s_abort = 0;
  }
  __syncthreads();
  const uint32_t tile = s_tile;
  const uint32_t npass = hdr->npass, dbits = hdr->dbits;
  const unsigned long long* src = (npass & 1) ? buf_b : buf_a;
  const uint64_t base = (uint64_t)tile * kDecTile + (uint64_t)tid * kDecItems;
  const unsigned long long imask = (1ull << ibits) - 1;
  const unsigned long long dmask = dbits >= 64 ? ~0ull : ((1ull << dbits) - 1);
  const bool raw = mode & PARD_MODE_RAW;
  constexpr int32_t kInf = 0x7fffffff;

  uint32_t idx[kDecItems], u[kDecItems], r[kDecItems], seg[kDecItems];
  int32_t lv[kDecItems];        /* min of u_t - t over this thread's earlier items of the same queue */
  bool lhead[kDecItems];        /* the item's queue head is one of this thread's items up to it      */

  SegMin run; run.m = kInf; run.head = 0;
#pragma unroll
  for (int i = 0; i < kDecItems; ++i) {
    uint64_t j = base + i;
    if (j < n) {
      unsigned long long e = src[j];
      idx[i] = (uint32_t)(e & imask);
      unsigned long long off = (e >> ibits) & dmask;
      seg[i] = (uint32_t)((e >> ibits) >> dbits);
      const PardSegConst K = ktab[seg[i]];
      r[i] = (uint32_t)j - seg_off[seg[i]];
      u[i] = threshold_u((int64_t)off - K.A_rel, K.d, K.cap);
    } else {
      idx[i] = 0; seg[i] = 0; r[i] = 0; u[i] = kUClamp;     /* acts as a head, never read */
    }
    if (r[i] == 0) { run.m = kInf; run.head = 1; }
    lv[i] = run.m;
    lhead[i] = run.head;
    run.m = min(run.m, (int32_t)u[i] - (int32_t)r[i]);
  }

  /* exclusive segmented scan of the threads' aggregates: warp, then block, then tiles */
  SegMin inc = run;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    SegMin l;
    l.m = __shfl_up_sync(0xffffffffu, inc.m, o);
    l.head = __shfl_up_sync(0xffffffffu, inc.head, o);
    if (lane >= (uint32_t)o) inc = seg_combine(l, inc);
  }
  SegMin exc;
  exc.m = __shfl_up_sync(0xffffffffu, inc.m, 1);
  exc.head = __shfl_up_sync(0xffffffffu, inc.head, 1);
  if (lane == 0) { exc.m = kInf; exc.head = 0; }
  if (lane == 31) { s_wm[warp] = inc.m; s_wh[warp] = inc.head; }
  __syncthreads();
  SegMin wprefix; wprefix.m = kInf; wprefix.head = 0;
  SegMin tile_agg; tile_agg.m = kInf; tile_agg.head = 0;
#pragma unroll
  for (int w = 0; w < WARPS; ++w) {
    SegMin a; a.m = s_wm[w]; a.head = s_wh[w];
    if (w < (int)warp) wprefix = seg_combine(wprefix, a);
    tile_agg = seg_combine(tile_agg, a);
  }
  exc = seg_combine(wprefix, exc);

  if (!raw) {
    if (tid == 0) {
      volatile unsigned long long* st = st_min;
      st[tile] = pack_min(tile_agg, kStAgg);
      SegMin carry; carry.m = kInf; carry.head = 0;
      bool first = true;
      for (int64_t t = (int64_t)tile - 1; t >= 0; --t) {
        unsigned long long w;
        uint32_t spins = 0;
        while (((w = st[t]) >> 62) == 0) {
          if (++spins > kSpinLimit) { s_abort = 1; break; }
          __nanosleep(20);
        }
        if ((w >> 62) == 0) break;
        SegMin a = unpack_min(w);
        carry = first ? a : seg_combine(a, carry);
        first = false;
        if ((w >> 62) == 2 || carry.head) break;     /* nothing before a queue head matters */
      }
      SegMin incl = seg_combine(carry, tile_agg);
      st[tile] = pack_min(incl, kStIncl);
      s_carry_m = carry.m;
    }
    __syncthreads();
    if (s_abort) {
      if (tid == 0) set_status(hdr, PARD_ETIMEOUT);
      return;
    }
    if (!exc.head) exc.m = min(exc.m, s_carry_m);
  }

  /* admitted position, estimate, decision */
  uint32_t keepbits = 0;
  long long est[kDecItems];
  uint32_t cpos[kDecItems];
#pragma unroll
  for (int i = 0; i < kDecItems; ++i) {
    uint32_t c;
    if (raw || r[i] == 0) {
      c = r[i];
    } else {
      int32_t pm = lhead[i] ? lv[i] : min(lv[i], exc.m);   /* min over t < r of (u_t - t) */
      int64_t cc = (int64_t)r[i] - 1 + pm;
      c = cc < (int64_t)r[i] ? (uint32_t)cc : r[i];
    }
    cpos[i] = c;
    const PardSegConst K = ktab[seg[i]];
    est[i] = K.A + (long long)(c / K.cap) * K.d;
    if (c < u[i] && base + i < n) keepbits |= 1u << i;
  }

  const uint64_t nrem = base < n ? (uint64_t)n - base : 0;
  if (nrem >= kDecItems) {
    if (out_keep) {
      unsigned long long kb = 0;
#pragma unroll
      for (int i = 0; i < kDecItems; ++i) kb |= (unsigned long long)((keepbits >> i) & 1u) << (8 * i);
      *reinterpret_cast<unsigned long long*>(out_keep + base) = kb;
    }
    if (out_est) {
#pragma unroll
      for (int i = 0; i < kDecItems; i += 2)
        *reinterpret_cast<longlong2*>(out_est + base + i) = make_longlong2(est[i], est[i + 1]);
    }
    if (out_perm) {
#pragma unroll
      for (int i = 0; i < kDecItems; i += 4)
        *reinterpret_cast<uint4*>(out_perm + base + i) = make_uint4(idx[i], idx[i + 1], idx[i + 2], idx[i + 3]);
    }
  } else {
    for (int i = 0; i < (int)nrem; ++i) {
      if (out_keep) out_keep[base + i] = (keepbits >> i) & 1u;
      if (out_est) out_est[base + i] = est[i];
      if (out_perm) out_perm[base + i] = idx[i];
    }
  }
  if (out_seg_kept && !raw) {
    /* the last request of a queue knows the queue's kept count */
#pragma unroll
    for (int i = 0; i < kDecItems; ++i)
      if (base + i < n && (uint32_t)(base + i) + 1 == seg_off[seg[i] + 1])
        out_seg_kept[seg[i]] = cpos[i] + ((keepbits >> i) & 1u);
  }
  if (out_seg_kept && raw) {
    /* kept requests are not a running count here: add them up per queue */
    const bool one_seg = nrem >= kDecItems && seg[0] == seg[kDecItems - 1];
    const uint32_t s0 = __shfl_sync(0xffffffffu, seg[0], 0);
    if (__all_sync(0xffffffffu, one_seg && seg[0] == s0)) {
      uint32_t x = __popc(keepbits);
      for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
      if (lane == 0 && x) atomicAdd(&out_seg_kept[s0], x);
    } else {
      uint32_t run = 0;
      for (int i = 0; i < kDecItems && base + i < n; ++i) {
        run += (keepbits >> i) & 1u;
        if (i + 1 == kDecItems || base + i + 1 >= n || seg[i + 1] != seg[i]) {
          if (run) atomicAdd(&out_seg_kept[seg[i]], run);
          run = 0;
        }
      }
    }
  }

  /* compaction: positions of the kept requests among all kept requests */
  if (out_kept_idx || out_n_kept) {
    uint32_t mine = __popc(keepbits), x = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= (uint32_t)o) x += y;
    }
    if (lane == 31) s_wk[warp] = x;
    __syncthreads();
    uint32_t wpre = 0, total = 0;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
      if (w < (int)warp) wpre += s_wk[w];
      total += s_wk[w];
    }
    if (tid == 0) {
      volatile unsigned long long* st = st_kept;
      st[tile] = kStAgg | total;
      unsigned long long excl = 0;
      for (int64_t t = (int64_t)tile - 1; t >= 0; --t) {
        unsigned long long w;
        uint32_t spins = 0;
        while (((w = st[t]) >> 62) == 0) {
          if (++spins > kSpinLimit) { s_abort = 1; break; }
          __nanosleep(20);
        }
        if ((w >> 62) == 0) break;
        excl += w & 0xffffffffull;
        if ((w >> 62) == 2) break;
      }
      st[tile] = kStIncl | (excl + total);
      s_carry_k = (uint32_t)excl;
      if (out_n_kept && (uint64_t)(tile + 1) * kDecTile >= n) *out_n_kept = excl + total;
    }
    __syncthreads();
    if (s_abort) {
      if (tid == 0) set_status(hdr, PARD_ETIMEOUT);
      return;
    }
    if (out_kept_idx) {
      uint32_t pos = s_carry_k + wpre + x - mine;
#pragma unroll
      for (int i = 0; i < kDecItems; ++i)
        if ((keepbits >> i) & 1u) out_kept_idx[pos++] = idx[i];
    }
  }
}

/* ---- optional phase timing (process-wide) ---- */
constexpr int kEventsPerSample = PARD_N_PHASES + 1;
static_assert(PARD_N_PHASES == 4 + kMaxPasses + 1, "phase list");
struct Profiler {
  std::mutex mu;
  bool on = false;
  uint32_t every = 1, max_samples = 0, calls = 0, n_samples = 0;
  std::vector<cudaEvent_t> ev;
};
Profiler g_prof;

/* events of this call if it is a sampled one, else nullptr */
cudaEvent_t* profile_acquire() {
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (!g_prof.on) return nullptr;
  uint32_t call = g_prof.calls++;
  if (call % g_prof.every != 0 || g_prof.n_samples >= g_prof.max_samples) return nullptr;
  return g_prof.ev.data() + (size_t)(g_prof.n_samples++) * kEventsPerSample;
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
  /* ---- host-side checks, nothing launched before they pass ---- */
  if (!pipelines || n_pipelines < 1 || !out) return PARD_EINVAL;
  if (n_pipelines > kMaxPipelinesPerCall) return PARD_ERANGE;
  if (mode & ~(PARD_MODE_RAW | PARD_MODE_NOWAIT)) return PARD_EINVAL;
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
  unsigned long long* st_min = (unsigned long long*)(ws + L.st_min);
  unsigned long long* st_kept = (unsigned long long*)(ws + L.st_kept);
  unsigned long long* buf_a = (unsigned long long*)(ws + L.buf_a);
  unsigned long long* buf_b = (unsigned long long*)(ws + L.buf_b);
  const uint32_t n32 = (uint32_t)n;
  const uint32_t S = (uint32_t)state->stage_stride;
  const uint32_t ibits = std::max(1u, ceil_log2(n));
  const uint32_t sbits = ceil_log2(L.n_seg);

  cudaEvent_t* evs = profile_acquire();
  int phase = 0;
  auto mark = [&]() {                      /* boundary between two phases */
    if (evs) cudaEventRecord(evs[phase], stream);
    ++phase;
  };
  mark();
  /* ---- clear the scratch that must start at zero ---- */
  PARD_CUDA_OK(cudaMemsetAsync(ws + L.hdr, 0, sizeof(PlanHeader), stream));
  PARD_CUDA_OK(cudaMemsetAsync(ctx_dmin, 0xff, 8ull * n_ctx, stream));
  PARD_CUDA_OK(cudaMemsetAsync(ctx_dmax, 0, 8ull * n_ctx, stream));
  PARD_CUDA_OK(cudaMemsetAsync(seg_off, 0, 4ull * (L.n_seg + 1), stream));
  PARD_CUDA_OK(cudaMemsetAsync(hist, 0, 4ull * kMaxPasses * kBins, stream));
  if (n > 0) {
    PARD_CUDA_OK(cudaMemsetAsync(lookback, 0, 4ull * kBins * (uint64_t)L.sort_tiles * L.max_passes, stream));
    PARD_CUDA_OK(cudaMemsetAsync(st_min, 0, 8ull * L.dec_tiles, stream));
    PARD_CUDA_OK(cudaMemsetAsync(st_kept, 0, 8ull * L.dec_tiles, stream));
  }
  if (out->d_seg_kept) PARD_CUDA_OK(cudaMemsetAsync(out->d_seg_kept, 0, 4ull * L.n_seg, stream));
  if (out->d_n_kept) PARD_CUDA_OK(cudaMemsetAsync(out->d_n_kept, 0, 8, stream));
  PARD_CUDA_OK(cudaMemcpyAsync(d_pipes, h_pipes.data(), 8ull * n_pipelines, cudaMemcpyHostToDevice, stream));

  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const uint4* req4 = (const uint4*)d_requests;

  mark();
  if (n > 0) {
    uint32_t grid = (uint32_t)std::min<uint64_t>((n + 2047) / 2048, (uint64_t)sms * 8);
    if (L.n_seg <= (uint32_t)kSmemSegs)
      k_prepass<true><<<grid, 256, 0, stream>>>(req4, n32, n_ctx, S, L.n_seg, ctx_dmin, ctx_dmax, seg_off, hdr);
    else
      k_prepass<false><<<grid, 256, 0, stream>>>(req4, n32, n_ctx, S, L.n_seg, ctx_dmin, ctx_dmax, seg_off, hdr);
  }
  mark();
  if (n > 0) k_ctx_span<<<(n_ctx + 255) / 256, 256, 0, stream>>>(ctx_dmin, ctx_dmax, n_ctx, hdr);
  k_seg_scan<<<1, 1024, 0, stream>>>(seg_off, L.n_seg, out->d_seg_offsets, sbits, ibits, hdr);
  k_seg_const<<<(L.n_seg + 127) / 128, 128, 0, stream>>>(d_pipes, n_pipelines, *state, n_ctx, ctx_dmin,
                                                         seg_off, ktab, hdr);
  mark();
  if (n > 0) {
    uint32_t grid = (uint32_t)std::min<uint64_t>((n + 255) / 256, (uint64_t)sms * 8);
    k_pack<<<grid, 256, 0, stream>>>(req4, n32, n_ctx, S, ctx_dmin, ibits, hdr, buf_a, hist);
  }
  for (uint32_t p = 0; p < (uint32_t)kMaxPasses; ++p) {
    mark();
    if (n > 0 && p < L.max_passes)
      k_sort_pass<<<L.sort_tiles, kSortThreads, 0, stream>>>(
          p, hdr, buf_a, buf_b, hist, lookback + (size_t)p * L.sort_tiles * kBins, n32, ibits);
  }
  mark();
  if (n > 0) {
    k_decide<<<L.dec_tiles, kDecThreads, 0, stream>>>(
        hdr, buf_a, buf_b, n32, ibits, mode, ktab, seg_off, st_min, st_kept, out->d_keep,
        (long long*)out->d_est_us, out->d_perm, out->d_kept_idx,
        (unsigned long long*)out->d_n_kept, out->d_seg_kept);
  }
  mark();
  PARD_CUDA_OK(cudaGetLastError());
  if (mode & PARD_MODE_NOWAIT) return PARD_OK;
  return pard_plan_status(d_workspace, cuda_stream);
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
  /* seg_scan + seg_const always; prepass, ctx_span, pack, passes, decide when n > 0 */
  *launches = n > 0 ? 2 + 3 + make_layout(n, n_ctx, stage_stride).max_passes + 1 : 2;
  return PARD_OK;
}

extern "C" int pard_profile_begin(uint32_t every, uint32_t max_samples) {
  if (every < 1 || max_samples < 1 || max_samples > 65536) return PARD_EINVAL;
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (g_prof.on) return PARD_EINVAL;
  g_prof.ev.assign((size_t)max_samples * kEventsPerSample, nullptr);
  for (auto& e : g_prof.ev)
    if (cudaEventCreate(&e) != cudaSuccess) {
      for (auto& f : g_prof.ev) if (f) cudaEventDestroy(f);
      g_prof.ev.clear();
      return PARD_ECUDA;
    }
  g_prof.every = every;
  g_prof.max_samples = max_samples;
  g_prof.calls = 0;
  g_prof.n_samples = 0;
  g_prof.on = true;
  return PARD_OK;
}

extern "C" int pard_profile_end(float* ms_sum, uint32_t* n_samples) {
  std::lock_guard<std::mutex> lock(g_prof.mu);
  if (!g_prof.on) return PARD_EINVAL;
  int rc = PARD_OK;
  if (ms_sum) for (int i = 0; i < PARD_N_PHASES; ++i) ms_sum[i] = 0.f;
  for (uint32_t s = 0; s < g_prof.n_samples; ++s) {
    cudaEvent_t* e = g_prof.ev.data() + (size_t)s * kEventsPerSample;
    if (cudaEventSynchronize(e[PARD_N_PHASES]) != cudaSuccess) { rc = PARD_ECUDA; break; }
    for (int i = 0; i < PARD_N_PHASES && ms_sum; ++i) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, e[i], e[i + 1]) != cudaSuccess) rc = PARD_ECUDA;
      ms_sum[i] += ms;
    }
  }
  if (n_samples) *n_samples = g_prof.n_samples;
  for (auto& e : g_prof.ev) cudaEventDestroy(e);
  g_prof.ev.clear();
  g_prof.on = false;
  return rc;
}

extern "C" const char* pard_profile_phase_name(uint32_t phase) {
  static const char* names[PARD_N_PHASES] = {"clear", "prepass", "segments", "pack", "sort0", "sort1",
                                              "sort2", "sort3", "sort4", "sort5", "sort6", "sort7",
                                              "decide"};
  return phase < PARD_N_PHASES ? names[phase] : "";
}
