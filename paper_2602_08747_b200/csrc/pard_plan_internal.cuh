/* Declarations shared by the translation units that make up pard_plan: the
 * workspace header, the per-call pipeline table and a few arithmetic helpers. */
#ifndef PARD_PLAN_INTERNAL_CUH_
#define PARD_PLAN_INTERNAL_CUH_

#include "pard_internal.h"

namespace pard_plan_detail {

constexpr int kMaxPasses = 8;
constexpr int kBins = 256;
constexpr uint32_t kUClamp = (1u << 30) - 1;       /* >= any request count      */
constexpr uint32_t kMaxPipelinesPerCall = 65536;
constexpr uint32_t kSegNarrow = 1u;                /* bits of PardSegConst::narrow */
constexpr uint32_t kSegNoStage = 2u;
constexpr uint32_t kSegHighFirst = 4u;
constexpr uint32_t kFoldSegs = 1024;              /* up to this many queues the key width is found inside k_seg_const */
constexpr uint32_t kHistSegs = 64;                /* up to this many queues the batch-window tables are counted, not searched */
constexpr uint32_t kHistCap = 8192;               /* window-table entries a counted table may have in all */
constexpr uint32_t kSpinLimit = 1u << 18;          /* polling rounds (about a microsecond each) before giving up */

constexpr int kSortThreads = 512;
constexpr int kLoWarps = 8;                        /* warps 0..7 also do the look-back (one thread per digit) */
constexpr int kItemsLo = 10, kItemsHi = 22;        /* rounds of 32 elements per warp: look-back warps / others (measured best) */
constexpr int kSortTile = 32 * (kLoWarps * kItemsLo + (kSortThreads / 32 - kLoWarps) * kItemsHi);
constexpr int kDecThreads = 128;                   /* small blocks: a short tail when the grid drains (measured against 64 and 256) */
constexpr int kDecItems = 8;
constexpr int kDecTile = kDecThreads * kDecItems;
constexpr int kCompactChunk = 1024;                /* indices moved by one warp of k_kept_move */
constexpr int kLookBatch = 8;                      /* earlier tiles inspected per round trip in the sort */

/* look-back word of the sort: [31:30] state, [29:0] count */
constexpr uint32_t kLbAgg = 1u << 30;
constexpr uint32_t kLbIncl = 2u << 30;
constexpr uint32_t kLbMask = (1u << 30) - 1;

struct PlanHeader {
  uint32_t status;            /* 0, or the positive value of a pard_status */
  uint32_t dbits;             /* bits of the widest per-ctx deadline span  */
  uint32_t keybits;           /* segment bits + dbits                      */
  uint32_t npass;             /* radix passes that run                     */
  unsigned long long span_max;
  unsigned long long win_total;   /* window-table entries asked for (64 bits: 2^24 queues of up to 4,097 entries) */
  uint32_t ticket[kMaxPasses + 1];
  uint32_t wide;              /* 1: segment, deadline and index bits exceed 64; nothing is sorted */
  uint32_t use_scan;          /* 1: too many batch windows for the window tables: decide by scanning */
  uint32_t aborted;           /* 1: a bounded wait ran out; the sort is incomplete and every later kernel returns */
  uint32_t big_total;         /* window-table entries that belong to long queues */
  uint32_t agg_done;          /* blocks of k_tile_agg that have stored their aggregates */
  uint32_t seg_done;          /* blocks of k_seg_const that have stored their constants */
  uint32_t unsorted;          /* 1: some request's ctx is smaller than its predecessor's */
  uint32_t ctx_too_big;       /* 1: some ctx holds more requests than one sort tile */
  uint32_t bad_input;         /* 1: PARD_EDATA was found (kept apart from `status`, which holds the first error only) */
  uint32_t bar[4];            /* blocks of k_scan_path that have reached each of its grid-wide barriers */
  uint32_t pad[64 - 21 - (kMaxPasses + 1)];
};
static_assert(sizeof(PlanHeader) == 256, "header is 256 bytes");

__device__ __forceinline__ void set_status(PlanHeader* hdr, int status) {
  if (status == PARD_EDATA) hdr->bad_input = 1;
  atomicCAS(&hdr->status, 0u, (uint32_t)(-status));
}

/* The device tables of the call's pipelines: handed over inside the kernel arguments when they
 * are few (no copy to enqueue), else through a table in the workspace. */
constexpr int kFewPipelines = 8;
struct PipeTable {
  const PardPipeDev* few[kFewPipelines];
  const PardPipeDev* const* many;
};

/* floor(2^64 / d) + 1 for d >= 2 */
__device__ __forceinline__ unsigned long long magic64(unsigned long long d) {
  unsigned long long q = ~0ull / d;
  if (~0ull % d == d - 1) ++q;          /* d divides 2^64 */
  return q + 1;
}

/* floor(x / d) for 32-bit x, with M = floor(2^64 / d) + 1 (d >= 2): exact
 * whenever x * d < 2^64, i.e. for every 32-bit x and d */
__device__ __forceinline__ uint32_t div_magic32(uint32_t x, unsigned long long M) {
  unsigned long long p0 = (unsigned long long)x * (uint32_t)M;
  unsigned long long p1 = (unsigned long long)x * (uint32_t)(M >> 32) + (p0 >> 32);
  return (uint32_t)(p1 >> 32);
}

__device__ __forceinline__ uint32_t threshold_u(int64_t X, const PardSegConst& K) {
  /* number of requests that may be admitted ahead of or at this one while it
   * still completes by its deadline: 0 if even position 0 is late, else
   * cap * (floor(X / d) + 1), saturated */
  if (X < 0) return 0;
  unsigned long long q;
  if (((unsigned long long)X >> 32) == 0 && K.d_magic)
    q = div_magic32((uint32_t)X, K.d_magic);
  else
    q = (unsigned long long)X / (unsigned long long)K.d;    /* d == 1 or operands beyond 32 bits */
  if (q >= kUClamp) return kUClamp;
  unsigned long long u = (q + 1) * K.cap;
  return u > kUClamp ? kUClamp : (uint32_t)u;
}

/* 32 bytes with one access; p is 32-byte aligned */
__device__ __forceinline__ void load4(const unsigned long long* p, unsigned long long* v) {
  asm volatile("ld.global.nc.v4.u64 {%0, %1, %2, %3}, [%4];"
               : "=l"(v[0]), "=l"(v[1]), "=l"(v[2]), "=l"(v[3]) : "l"(p));
}
__device__ __forceinline__ void store4(void* p, unsigned long long a, unsigned long long b,
                                       unsigned long long c, unsigned long long d) {
  asm volatile("st.global.v4.u64 [%0], {%1, %2, %3, %4};" :: "l"(p), "l"(a), "l"(b), "l"(c), "l"(d) : "memory");
}


/* Decision by a sequential walk of every queue (requests whose downstream path is known, arrival
 * order, the Nexus and Clipper++ rules): defined in pard_policy.cu, enqueued by pard_plan after
 * the sort and the queue boundaries.  The sorted elements are in buf_b when hdr->npass is odd,
 * else in buf_a; the other buffer (8 bytes per request) is free by then and serves as scratch. */
struct PolicyArgs {
  PlanHeader* hdr;
  unsigned long long* buf_a;
  unsigned long long* buf_b;
  uint32_t n, ibits, n_seg, mode;
  const PardSegConst* ktab;
  const uint32_t* seg_off;
  const uint4* req;
  const pard_arrival_t* arrivals;
  PipeTable pipes;
  uint32_t n_pipelines;
  pard_queue_state_t st;
  uint8_t* out_keep;
  long long* out_est;
  uint32_t* out_perm;
  uint32_t* kept_tmp;
  uint32_t* seg_kept;
};
int launch_policy_decision(const PolicyArgs& a, int sms, cudaStream_t stream);

}  // namespace pard_plan_detail

#endif  /* PARD_PLAN_INTERNAL_CUH_ */
