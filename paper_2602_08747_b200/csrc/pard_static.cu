/* pard_plan_static: the planner for callers that cannot allocate device memory.
 *
 * pard_plan needs scratch memory (sort buffers, tile look-back words, the
 * per-segment table) and leaves its allocation to the caller.  Some callers
 * have no way to provide it: a drop planner usually lives in the control loop
 * of an inference server whose runtime has claimed all device memory for
 * weights and caches at start-up, and cudaMalloc / cudaFree from that loop
 * would also take the driver's allocation lock and may synchronise the
 * device, stalling the inference kernels the planner is there to protect.
 * For them the scratch lives in the library image itself: a fixed array in
 * device global memory that exists on every GPU that loads the library, from
 * load until the process exits. */
#include <mutex>

#include "pard_internal.h"

namespace {

/* The scratch.  In host code this name is only a handle for the runtime; the
 * device address is obtained below with cudaGetSymbolAddress. */
static __device__ __align__(256) unsigned char g_static_scratch[PARD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

/* Device address of the scratch on the current device; looked up once per device. */
int scratch_address(void** out) {
  int dev = -1;
  PARD_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return PARD_ERANGE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return PARD_ECUDA;
    }
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return PARD_OK;
}

}  // namespace

extern "C" int pard_plan_static(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                                const pard_request_t* d_requests, uint64_t n,
                                const pard_queue_state_t* state, uint32_t n_ctx, uint32_t mode,
                                const pard_plan_out_t* out, void* cuda_stream) {
  if (!state) return PARD_EINVAL;
  uint64_t need = 0;
  int rc = pard_plan_workspace_bytes(n, n_ctx, state->stage_stride, &need);
  if (rc != PARD_OK) return rc;
  if (need > PARD_STATIC_SCRATCH_BYTES) return PARD_ESTATIC;   /* problem too large for the built-in scratch */
  void* scratch = nullptr;
  rc = scratch_address(&scratch);
  if (rc != PARD_OK) return rc;
  /* pard_plan clears every part of the scratch that has to start at zero, so
   * what the previous call left behind does not matter. */
  return pard_plan(pipelines, n_pipelines, d_requests, n, state, n_ctx, mode, out, scratch,
                   PARD_STATIC_SCRATCH_BYTES, cuda_stream);
}
