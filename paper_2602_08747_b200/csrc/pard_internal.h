/* Internal declarations shared by the translation units of libpard. */
#ifndef PARD_INTERNAL_H_
#define PARD_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "pard.h"

/* Device-resident tables of one pipeline.  The struct itself is the first
 * bytes of the pipeline's single device allocation; its pointers point into
 * the same allocation. */
struct PardPipeDev {
  int32_t n_stages;
  int32_t n_slots;
  const int32_t* bmax;            /* [S]                                        */
  const int64_t* lat_offsets;     /* [S+1]                                      */
  const int64_t* lat_us;          /* profile entries                            */
  const int32_t* stage_slot_off;  /* [S+1] slots of stage k: [off[k], off[k+1]) */
  const int32_t* path_off;        /* [n_slots+1] into path_stage                */
  const int32_t* path_stage;      /* concatenated stage ids of all paths        */
};

struct pard_pipeline {
  int32_t n_stages = 0;
  int32_t n_slots = 0;
  std::vector<int32_t> bmax;
  std::vector<int64_t> lat_offsets;
  std::vector<int64_t> lat_us;
  std::vector<int32_t> stage_slot_off;          /* [S+1]                        */
  std::vector<int32_t> path_off;                /* [n_slots+1], global offsets  */
  std::vector<int32_t> path_stage;
  std::vector<std::vector<int32_t>> local_off;  /* per stage, offsets rebased to 0 */
  int device = -1;                              /* -1: host only                */
  void* d_blob = nullptr;                       /* PardPipeDev + tables         */
};

/* Per-segment constants (Eq. 3 terms that do not depend on the request). */
struct __align__(16) PardSegConst {
  int64_t A;         /* base + d_k(B_k) + L_sub : estimate of a request at position 0   */
  int64_t A_rel;     /* A - (smallest deadline of the segment's ctx)                    */
  int64_t d;         /* d_k(B_k)                                                        */
  uint64_t d_magic;  /* floor(2^64 / d) + 1, or 0 when d == 1 or d >= 2^32              */
  uint64_t cap_magic;/* floor(2^64 / cap) + 1, or 0 when cap == 1                       */
  uint32_t cap;      /* min(B_k * m_k, 2^30)                                            */
  uint32_t narrow;   /* bit 0: 2 <= d < 2^31 and |A_rel| < 2^29, so both fit 32-bit arithmetic;
                        bit 1: the ctx's pipeline has no such stage; bit 2: high budget first */
  int64_t lsub;      /* L_sub of Eq. 3 (max over all downstream paths): A - lsub = base + d_k(B_k) */
  int64_t dsum;      /* sum of d_i(B_i) over all stages of the ctx's pipeline (Clipper++ split) */
};
static_assert(sizeof(PardSegConst) == 64, "one 64-byte line per segment");

#ifdef __CUDACC__
/* Programmatic dependent launch: every kernel of the library is launched with
 * the stream-serialization attribute, so that its blocks may be scheduled while
 * the previous kernel of the stream drains, and starts with pdl_wait(), which
 * returns once that previous kernel has completed and its writes are visible.
 * No kernel touches memory or exits before the wait. */
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

/* see pard_profile_begin: lets pard_goodput count as the end of the planner's last phase */
void pard_profile_extend_last(cudaStream_t stream);

#define PARD_CUDA_OK(expr)                    \
  do {                                        \
    cudaError_t e__ = (expr);                 \
    if (e__ != cudaSuccess) return PARD_ECUDA; \
  } while (0)

#endif  /* PARD_INTERNAL_H_ */
