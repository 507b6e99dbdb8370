/*
 * pard.h -- C ABI of the PARD drop planner for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, for a snapshot of every stage queue of a DAG
 * inference pipeline, the per-request keep/drop decision of PARD's State
 * Planner and Request Broker (paper Sec. 4.2, Eq. 1-3), in the decision order
 * of the low-budget-first priority queue (Sec. 4.3), then compacts the kept
 * requests and counts goodput (Sec. 5.1, Metrics).
 *
 * Vocabulary: "stage" is the paper's module M_k; a "ctx" (context) is one
 * independent planning problem (one pipeline instance at one decision epoch);
 * a "segment" is the queue of one (ctx, stage).  segment id = ctx *
 * stage_stride + stage.  All times are int64 microseconds on one clock.
 *
 * Pointers whose name starts with d_ are DEVICE pointers; every other pointer
 * is a HOST pointer.  No function throws, aborts or prints; each returns
 * PARD_OK (0) or a negative pard_status.  Entry points may be called from
 * several host threads as long as they use distinct streams, workspaces and
 * output buffers; a pipeline handle is immutable after loading.
 */
#ifndef PARD_H_
#define PARD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- limits ------------------------------------------------------------ */
#define PARD_MAX_STAGES      64        /* stages per pipeline                       */
#define PARD_MAX_BATCH       4096      /* largest profiled batch size per stage     */
#define PARD_MAX_PATH_SLOTS  65536     /* sum over stages of downstream paths       */
#define PARD_MAX_PATH_LEN_SUM (1 << 20)/* sum of the lengths of all those paths     */
#define PARD_MAX_REQUESTS    (1ull << 30) /* requests per pard_plan call            */
#define PARD_MAX_SEGMENTS    (1u << 24)   /* n_ctx * stage_stride                   */
#define PARD_MAX_WAIT_SAMPLES (1u << 15)   /* samples per slot in pard_estimate_w      */
#define PARD_MAX_HISTORY     4096         /* workload samples per queue in pard_update_priority */
#define PARD_RATE_LIMIT      (1u << 24)   /* arrivals per sampling interval lie in [0, 2^24) */
#define PARD_MAX_DELAY_SAMPLES (1u << 15) /* queueing-delay samples per queue in pard_update_queue_delay */
#define PARD_MAX_DELAY_WINDOW_US (1u << 24) /* longest sliding window of pard_update_queue_delay */
#define PARD_WAIT_LIMIT_US   (1 << 24)    /* recorded batch waits lie in [0, 2^24)  */
#define PARD_TIME_LIMIT_US   (1ll << 60)  /* every time input lies in [0, 2^60)     */
#define PARD_LAT_LIMIT_US    (1ll << 40)  /* every profile entry lies in [1, 2^40)  */

/* ---- status codes ------------------------------------------------------ */
typedef enum pard_status {
  PARD_OK          =  0,
  PARD_EINVAL      = -1,  /* null pointer, bad count, malformed CSR, bad flag        */
  PARD_ECYCLE      = -2,  /* the stage graph has a cycle                             */
  PARD_ERANGE      = -3,  /* a host-visible value is outside the limits above; with
                             PARD_MODE_NOWAIT also: the sort key exceeds 64 bits     */
  PARD_ENOMEM      = -4,  /* host or device allocation failed (load time only)       */
  PARD_EWORKSPACE  = -5,  /* caller's workspace is smaller than required             */
  PARD_ETIMEOUT    = -6,  /* a bounded device-side wait ran out; outputs unspecified */
  PARD_ECUDA       = -7,  /* a CUDA runtime call failed                              */
  PARD_EDATA       = -8,  /* device found ctx, stage or batch size out of range, or
                             a deadline outside [0, 2^60); outputs unspecified       */
  PARD_ESTATIC     = -9   /* pard_plan_static: the problem needs more scratch than
                             the library's built-in PARD_STATIC_SCRATCH_BYTES        */
} pard_status;

const char* pard_strerror(int status);

/* ---- pipeline description (Sec. 5.1, Implementation) -------------------
 * The paper describes a pipeline as a list of modules (name, id, pres, subs).
 * Here the ids are 0..n_stages-1 and only `subs` is given, as a CSR adjacency;
 * `pres` is implied.  A stage without successors is a sink. */
typedef struct pard_dag {
  int32_t        n_stages;     /* 1..PARD_MAX_STAGES                                */
  const int32_t* sub_offsets;  /* [n_stages+1], non-decreasing, sub_offsets[0] = 0  */
  const int32_t* sub_ids;      /* [sub_offsets[n_stages]] successor ids; no self
                                  loops, no duplicate edge                          */
} pard_dag_t;

/* Offline profile d_k(b): execution duration of stage k at batch size b
 * (Sec. 4.2, State Planner, second bullet; Sec. 5.1, Implementation). */
typedef struct pard_profile {
  const int32_t* bmax;         /* [n_stages] largest profiled batch, 1..PARD_MAX_BATCH */
  const int64_t* lat_offsets;  /* [n_stages+1]; lat_offsets[s+1]-lat_offsets[s] == bmax[s] */
  const int64_t* lat_us;       /* lat_us[lat_offsets[s] + b - 1] = d_s(b), in [1, 2^40) */
} pard_profile_t;

typedef struct pard_pipeline pard_pipeline_t;   /* opaque, owned by the library */

#define PARD_LOAD_HOST_ONLY 1u  /* build the host tables only (no CUDA call); such a
                                   handle answers pard_pipeline_* queries but is
                                   rejected by pard_plan with PARD_EINVAL           */

/* Validates the graph (PARD_EINVAL / PARD_ECYCLE / PARD_ERANGE), enumerates for
 * every stage k its downstream paths -- every stage sequence that starts at a
 * successor of k and ends at a sink (Sec. 4.2: the estimate is taken along
 * each subsequent DAG path) -- ordered lexicographically by stage-id sequence,
 * and, unless PARD_LOAD_HOST_ONLY is set, copies the tables to the current
 * CUDA device (one device allocation, released by pard_free_pipeline).
 * Inputs are copied; the caller may free them on return. */
int pard_load_pipeline(const pard_dag_t* dag, const pard_profile_t* profile,
                       uint32_t flags, pard_pipeline_t** out);
int pard_free_pipeline(pard_pipeline_t* pipeline);

/* Path-slot layout.  Slot index of (stage k, its j-th downstream path) is
 * slot_base(k) + j with slot_base(k) = number of downstream paths of all
 * stages < k.  queue_state.w_us rows are indexed by slot.  */
int pard_pipeline_n_stages(const pard_pipeline_t* p, int32_t* n_stages);
int pard_pipeline_n_slots(const pard_pipeline_t* p, int32_t* n_slots);
/* Returns HOST pointers into the handle (valid until pard_free_pipeline):
 * path j of the stage is path_stage_ids[path_offsets[j] .. path_offsets[j+1]). */
int pard_pipeline_paths(const pard_pipeline_t* p, int32_t stage,
                        int32_t* n_paths, int32_t* slot_base,
                        const int32_t** path_offsets, const int32_t** path_stage_ids);

/* ---- requests and runtime state ----------------------------------------
 * One queued request.  deadline_us = t_s + SLO: the send time of Eq. 3 plus
 * the request's latency objective, so that "estimated latency exceeds the
 * SLO" becomes "estimated completion time exceeds deadline_us". */
typedef struct pard_request {
  int64_t  deadline_us;   /* in [0, 2^60)                                            */
  uint32_t ctx;           /* < n_ctx                                                 */
  uint16_t stage;         /* stage whose queue holds the request, < n_stages         */
  uint16_t flags;         /* ignored unless PARD_MODE_PATH_MASK: then the downstream
                             paths the request will take (0 = unknown, all paths)   */
} pard_request_t;         /* 16 bytes, 16-byte aligned arrays                        */

/* Runtime state the State Planner monitors and synchronises (Sec. 4.1, steps
 * 1-3; Sec. 4.2).  All arrays are DEVICE memory, row-major per ctx. */
typedef struct pard_queue_state {
  int32_t        stage_stride;     /* row length of the [n_ctx][stage] arrays; >= every
                                      used pipeline's n_stages, <= PARD_MAX_STAGES   */
  int32_t        slot_stride;      /* row length of d_w_us; >= every used pipeline's
                                      n_slots (ignored when d_w_us is NULL)          */
  const int32_t* d_pipeline_of_ctx;/* [n_ctx] index into `pipelines`; NULL => 0      */
  const int64_t* d_now_us;         /* [n_ctx] decision instant t_b of the snapshot   */
  const int32_t* d_batch;          /* [n_ctx][stage_stride] current batch size B_k in
                                      1..bmax[k]                                     */
  const int64_t* d_free_at_us;     /* [n_ctx][stage_stride] expected end of the batch
                                      now executing (t_e of the batch being formed)  */
  const int64_t* d_q_us;           /* [n_ctx][stage_stride] recent average queueing
                                      delay q_k                                      */
  const int64_t* d_w_us;           /* [n_ctx][slot_stride] batch-wait estimate w per
                                      (stage, downstream path) slot; NULL => 0       */
  const int32_t* d_workers;        /* [n_ctx][stage_stride] identical workers m_k >= 1
                                      draining the queue; NULL => 1                  */
  const uint8_t* d_priority;       /* [n_ctx][stage_stride] decision order of the queue
                                      (Sec. 4.3): 0 = low budget first, any other value =
                                      high budget first; NULL => 0.  pard_update_priority
                                      maintains such an array                        */
} pard_queue_state_t;

/* Outputs of pard_plan, all DEVICE memory owned by the caller.  Per-request
 * outputs are in service order: segments ascending, inside a segment by
 * (deadline, original index) ascending -- for a queue served high budget first
 * by deadline descending, equal deadlines still in ascending index order.  A
 * NULL member is not produced. */
typedef struct pard_plan_out {
  uint8_t*  d_keep;        /* [n]  1 = kept, 0 = dropped                             */
  int64_t*  d_est_us;      /* [n]  estimated completion time t_s + L of Eq. 3        */
  uint32_t* d_perm;        /* [n]  original index of the request at each position    */
  uint32_t* d_kept_idx;    /* [n]  capacity; first *d_n_kept entries = original
                                   indices of kept requests, in service order        */
  uint64_t* d_n_kept;      /* [1]                                                    */
  uint32_t* d_seg_offsets; /* [n_ctx*stage_stride + 1] first position of each segment */
  uint32_t* d_seg_kept;    /* [n_ctx*stage_stride] kept requests per segment         */
} pard_plan_out_t;

#define PARD_MODE_ADMITTED 0u   /* a dropped request takes no batch slot (default)   */
#define PARD_MODE_RAW      1u   /* every queued request ahead takes a batch slot     */
#define PARD_MODE_NOWAIT   2u   /* pard_plan returns once its work is enqueued and
                                   reads no status back; the status word stays in the
                                   workspace until pard_plan_status fetches it        */
#define PARD_MODE_SCAN     4u   /* take the decision by the scan path even when the
                                   batch-window tables would do (same results; the scan
                                   is otherwise the fallback for queues with thousands
                                   of batch windows).  The scan path is one kernel whose
                                   blocks (two per multiprocessor) wait for each other
                                   between its steps, each wait bounded at about half a
                                   second: a GPU that other streams keep completely full
                                   for that long makes the call return PARD_ETIMEOUT   */
#define PARD_MODE_TEST_STALL 8u /* testing aid for the bounded device-side waits: the
                                   first tile of the first sort pass withholds the word
                                   later tiles wait for, and the first block of the scan
                                   path (PARD_MODE_SCAN) never arrives at the first of its
                                   grid-wide meeting points; the waits run out (after a
                                   fraction of a second) and the call returns
                                   PARD_ETIMEOUT with unspecified outputs; the CUDA
                                   context stays usable.  Calls that the library sorts
                                   block by block (requests grouped by ctx, no ctx above
                                   8,192 requests) have no wait in the sort */
#define PARD_MODE_GROUPED 256u  /* the caller's word that d_requests is grouped by ascending
                                   ctx (batched decision epochs, many instances in one
                                   call).  What the library makes of it depends on the
                                   sizes:
                                   - contexts of at most 8,192 requests on average: the
                                     promise then includes that NO ctx holds more than
                                     8,192.  Up to a few hundred contexts one thread block
                                     plans each ctx from start to end in shared memory --
                                     constants, sort, positions, decisions -- in six
                                     kernel launches instead of about twenty, two to three
                                     times faster on small and medium calls; beyond that a
                                     block per ctx reads, checks and sorts its ctx and the
                                     rest is the general path, minus its pass over all
                                     requests for the deadline ranges and minus the
                                     kernels it launches in reserve for ungrouped input;
                                   - larger contexts (and stage_stride a power of two):
                                     the radix passes stay inside every ctx's range and
                                     sort the stage and deadline bits only -- one pass
                                     fewer whenever the ctx bits of the key cost one.
                                   The device checks the claim: a call that breaks it
                                   returns PARD_EDATA (as does, in the block-per-ctx
                                   forms, any request out of range) with unspecified
                                   outputs.  A call with a single ctx of at most 8,192
                                   requests is always planned by one block (one kernel
                                   launch).  Ignored by the rules below, which take their
                                   own path.  Same results. */

/* Other decision orders and rules on the same queues, for comparison with the
 * planner's own (which stays the default).  Their thresholds do not rise along
 * a queue, so each queue is walked in order by one warp (32 requests per step)
 * instead of being decided request by request; they cost a few times the
 * default rule on long queues.  None combines with PARD_MODE_RAW.
 *   PARD_MODE_PATH_MASK  requests whose downstream path is known (Sec. 5.2,
 *       dynamic-path DAGs, where a request takes one of several branches):
 *       pard_request_t.flags is a mask over the downstream paths of the
 *       request's stage -- bit j = the stage's j-th path in the order of
 *       pard_pipeline_paths, j < 16 -- and L_sub is the maximum over the paths
 *       named.  flags = 0 means "unknown": all paths, as without this mode; at
 *       a sink the mask is ignored; a mask naming no path of the stage gives
 *       PARD_EDATA.  Order and rule otherwise unchanged (also with priorities).
 *   PARD_MODE_FCFS       queues are decided in arrival order -- the order of the
 *       request array -- instead of budget order (Table 1 and Sec. 5.3,
 *       PARD-FCFS); estimate and rule unchanged; combines with
 *       PARD_MODE_PATH_MASK; d_priority must be NULL.
 *   PARD_MODE_NEXUS      Nexus' reactive rule (Sec. 5.1, Baseline), arrival
 *       order: a window of one batch round (B_k * m_k requests) slides over the
 *       queue; the batch is the first window whose requests can all finish the
 *       CURRENT module by their deadlines if the batch starts when the previous
 *       one ends (base + b * d for round b); all requests in front of it are
 *       dropped; the scan goes on behind it, one duration later.  A last window
 *       that the queue cannot fill runs as it is.  est_us = end of the round
 *       the request was tested against.  d_priority must be NULL.
 *   PARD_MODE_CLIPPER    Clipper++ (Sec. 5.1, Baseline), arrival order: module k
 *       gets the share SLO_k = floor(SLO * d_k / sum_i d_i) of the request's
 *       objective (d_i at the current batch sizes, all stages of the ctx's
 *       pipeline), counted from the request's arrival at the module; a request
 *       is dropped iff its batch would start later than arrive + SLO_k (a
 *       dropped request takes no batch slot).  Needs pard_plan_policy's
 *       d_arrivals; deadline_us is not read.  est_us = end of the request's
 *       batch.  arrive_us in [0, 2^60), slo_us in [0, 2^31), d_k < 2^32, else
 *       PARD_EDATA.  d_priority must be NULL. */
#define PARD_MODE_PATH_MASK 16u
#define PARD_MODE_FCFS      32u
#define PARD_MODE_NEXUS     64u
#define PARD_MODE_CLIPPER   128u

/* Per-request input of PARD_MODE_CLIPPER: when the request reached the module
 * whose queue holds it, and its end-to-end latency objective. */
typedef struct pard_arrival {
  int64_t arrive_us;
  int64_t slo_us;
} pard_arrival_t;          /* 16 bytes, 16-byte aligned arrays */

/* Device scratch pard_plan needs for n requests in n_ctx contexts. */
int pard_plan_workspace_bytes(uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                              uint64_t* bytes);

/* The planner (Sec. 4.2 Eq. 1-3; decision order of Sec. 4.3: the remaining
 * budget of a request is its deadline minus the snapshot's `now`, so low
 * budget first is deadline ascending and high budget first is deadline
 * descending).  For every segment, in its decision order, with
 *   d    = d_k(B_k)                         profile at the current batch size
 *   cap  = B_k * m_k                        requests started per batch round
 *   base = max(now, free_at_k)              start of the next batch to form
 *   Lsub = 0 for a sink, else max over downstream paths P of
 *          sum_{i in P} (q_i + d_i(B_i)) + w[slot(k,P)]
 * a request at position c (kept requests ahead of it, or all requests ahead
 * in PARD_MODE_RAW) gets est = base + floor(c/cap)*d + d + Lsub and is kept
 * iff est <= deadline.
 *
 * `pipelines` is a host array of n_pipelines handles loaded on the current
 * device.  d_requests is read only.  d_workspace must be 256-byte aligned and
 * hold pard_plan_workspace_bytes() bytes; nothing in it survives the call.
 * All work is enqueued on `cuda_stream` (a cudaStream_t, NULL = default
 * stream); the call then waits for the stream and reads back one status word,
 * so a PARD_EDATA / PARD_ETIMEOUT found on the device is returned here.  The
 * library allocates no device memory in this call.
 * Keys wider than one sort element: when the bits of the segment id, of the
 * widest per-ctx deadline span and of the request index add up to more than
 * 64 (e.g. 2^14 requests in 64 queues with deadlines 2^59 us apart), the call
 * finds that out on the device, then sorts the key in chunks and walks the
 * queues (same results, several times slower).  That second stage needs the
 * first one's report, so it only runs in the waiting form of the call; with
 * PARD_MODE_NOWAIT such a call leaves PARD_ERANGE for pard_plan_status.
 * Host-detectable errors are returned before anything is launched.
 * Performance note: requests may come in any order.  When they come grouped by
 * ascending ctx and no ctx holds more than 8,192 of them (batched decision
 * epochs, one module's queue), every ctx is sorted by one thread block in
 * shared memory, which is markedly faster; the result is the same.  A caller
 * who knows this of its requests says so with PARD_MODE_GROUPED and gets the
 * whole plan of a ctx from one thread block. */
int pard_plan(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
              const pard_request_t* d_requests, uint64_t n,
              const pard_queue_state_t* state, uint32_t n_ctx, uint32_t mode,
              const pard_plan_out_t* out,
              void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);

/* pard_plan with the per-request arrival records that PARD_MODE_CLIPPER reads
 * (DEVICE, [n], parallel to d_requests; NULL for every other mode, which makes
 * the call identical to pard_plan). */
int pard_plan_policy(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                     const pard_request_t* d_requests, const pard_arrival_t* d_arrivals,
                     uint64_t n, const pard_queue_state_t* state, uint32_t n_ctx,
                     uint32_t mode, const pard_plan_out_t* out,
                     void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);

/* For PARD_MODE_NOWAIT: waits for `cuda_stream`, then returns the status that
 * the most recent pard_plan call on this workspace left there (PARD_OK,
 * PARD_EDATA, PARD_ERANGE or PARD_ETIMEOUT).  The workspace must not have been
 * reused for anything else in between. */
int pard_plan_status(const void* d_workspace, void* cuda_stream);

/* Number of kernels one pard_plan call enqueues for these sizes under the
 * default rule, without priorities and without PARD_MODE_GROUPED (memsets and
 * copies not counted).  Radix passes beyond the key width found on the device
 * and the scan path are launched and return at once; they are included.  A
 * key wider than 64 bits adds the kernels of its second stage. */
int pard_plan_kernel_launches(uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                              uint32_t* launches);

/* The planner for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment aid).  A drop planner typically runs in
 * the control loop of an inference server: the serving runtime has often
 * claimed all device memory at start-up, and a cudaMalloc / cudaFree issued
 * from that loop takes the driver's allocation lock and may synchronise the
 * device, stalling the very inference kernels whose queues are being planned.
 * pard_plan_static computes exactly what pard_plan computes, with the same
 * arguments minus the workspace: its scratch is a fixed array of
 * PARD_STATIC_SCRATCH_BYTES of device global memory that is part of the
 * library image (every GPU that loads the library holds it until the process
 * exits).  It calls no allocation routine.
 *  - Size limit: accepted iff pard_plan_workspace_bytes(n, n_ctx, stage_stride)
 *    <= PARD_STATIC_SCRATCH_BYTES, e.g. 2^18 requests in up to 4,096 segments;
 *    anything larger returns PARD_ESTATIC and nothing is launched.
 *  - The first call on each device looks up the array's device address (a
 *    one-time set-up under a lock); make that first call before any stream
 *    capture begins on that device.
 *  - All calls on one device share the one array.  Each call clears the parts
 *    that must start at zero, so the previous call's contents do not matter,
 *    but two calls whose GPU work overlaps (different streams, or
 *    PARD_MODE_NOWAIT calls not ordered by one stream) race on it; so does a
 *    pard_plan_status on anything but this scratch.  With PARD_MODE_NOWAIT
 *    there is no way to fetch the status afterwards: use the default mode.
 * Inputs, outputs, ordering and error codes are otherwise those of pard_plan. */
#define PARD_STATIC_SCRATCH_BYTES (8u << 20)
int pard_plan_static(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                     const pard_request_t* d_requests, uint64_t n,
                     const pard_queue_state_t* state, uint32_t n_ctx, uint32_t mode,
                     const pard_plan_out_t* out, void* cuda_stream);

/* Same computation with HOST inputs and outputs: `requests`, the arrays of
 * `state` and the members of `out` are host pointers (pinned memory makes the
 * copies asynchronous).  Inputs are copied to the device, planned, and the
 * non-NULL outputs copied back, all on `cuda_stream`; the call returns after
 * the stream has drained.  d_workspace must hold
 * pard_plan_host_workspace_bytes() bytes. */
int pard_plan_host_workspace_bytes(uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                                   int32_t slot_stride, uint64_t* bytes);
int pard_plan_host(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                   const pard_request_t* requests, uint64_t n,
                   const pard_queue_state_t* state, uint32_t n_ctx, uint32_t mode,
                   const pard_plan_out_t* out,
                   void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);

/* Goodput counters (Sec. 5.1, Metrics): per ctx, the number of queued
 * requests and the number predicted to finish within their SLO (kept);
 * dropped = total - kept, drop rate = dropped / total.  Writes
 * d_out_total[n_ctx] and d_out_kept[n_ctx] (overwritten, not accumulated)
 * from pard_plan's outputs: d_seg_offsets always, and
 *   - d_seg_kept, when given: the kept counts of a ctx's queues are added up
 *     (one small kernel; d_keep is not read and may be NULL), or
 *   - d_keep, when d_seg_kept is NULL: the keep flags of every ctx are counted
 *     (16-byte aligned; a block-wide reduction and one atomic per block and
 *     ctx), for callers that did not ask pard_plan for the per-queue counts.
 * Both give the same numbers.  Enqueued on cuda_stream; does not synchronise. */
int pard_goodput(const uint8_t* d_keep, const uint32_t* d_seg_offsets,
                 const uint32_t* d_seg_kept,
                 uint64_t n, uint32_t n_ctx, int32_t stage_stride,
                 int64_t* d_out_total, int64_t* d_out_kept, void* cuda_stream);

/* Batch-wait estimate of the State Planner (Sec. 4.2, Batch wait estimation;
 * its footnote gives the default M = 10,000 samples; Sec. 5.4, Overheads: the
 * estimate is refreshed off the critical path).
 * For every ctx and every (stage k, downstream path P) slot of its pipeline,
 *   w[ctx][slot] = F^{-1}(lambda),   lambda = lambda_num / lambda_den in [0, 1],
 * where F is the empirical distribution of n_samples draws of the batch wait
 * aggregated over the stages of P: draw m adds, for the j-th stage i of P, one
 * recorded wait  d_wait_samples[(ctx * stage_stride + i) * n_samples + idx],
 *   idx = (hi32(splitmix64(seed + (((ctx*slot_stride + slot) * n_samples + m) * 64 + j)))
 *          * n_samples) >> 32,
 * (splitmix64 of Steele, Lea and Flood; 64-bit wrap-around arithmetic), and
 * F^{-1}(lambda) is the draw of rank min(n_samples - 1, floor(lambda * n_samples))
 * in ascending order: lambda = 0 gives the smallest draw, lambda = 1 the largest.
 * The result feeds pard_queue_state_t.d_w_us.
 *   d_wait_samples  DEVICE, int32 [n_ctx][stage_stride][n_samples]: for every
 *                   stage its n_samples most recent recorded batch waits in
 *                   microseconds, each in [0, PARD_WAIT_LIMIT_US); rows of
 *                   stages the pipeline lacks are not read
 *   d_w_us          DEVICE, int64 [n_ctx][slot_stride]; entries at slots the
 *                   ctx's pipeline lacks are left untouched
 *   d_workspace     DEVICE, 256-byte aligned, pard_estimate_w_workspace_bytes()
 *   mode            0 or PARD_MODE_NOWAIT (then pard_plan_status on this
 *                   workspace fetches the status later)
 * 1 <= n_samples <= PARD_MAX_WAIT_SAMPLES.  Host-detectable errors come back
 * before anything is launched; a drawn sample outside its range, a pipeline id
 * outside [0, n_pipelines) or a pipeline with more stages or slots than the
 * strides gives PARD_EDATA with unspecified outputs.  One kernel is enqueued
 * on cuda_stream; no device memory is allocated.  The caller owns all buffers. */
int pard_estimate_w_workspace_bytes(uint32_t n_pipelines, uint64_t* bytes);
int pard_estimate_w(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                    const int32_t* d_pipeline_of_ctx, uint32_t n_ctx,
                    int32_t stage_stride, int32_t slot_stride,
                    const int32_t* d_wait_samples, uint32_t n_samples,
                    uint32_t lambda_num, uint32_t lambda_den, uint64_t seed, uint32_t mode,
                    int64_t* d_w_us, void* d_workspace, uint64_t workspace_bytes,
                    void* cuda_stream);

/* Recent average queueing delay q_k of the State Planner (Sec. 4.2, first
 * bullet: monitored with a sliding window, by default a 5 s linear weighted
 * one).  For every (ctx, stage), over its recorded samples j < n_samples --
 * taken at time d_sample_time_us[(ctx * stage_stride + stage) * n_samples + j]
 * with measured queueing delay d_sample_delay_us[same index], in any order --
 *   weight_j = window_us - (now - t_j)   if 0 <= now - t_j < window_us, else 0
 *   q        = floor( sum weight_j * delay_j / sum weight_j )
 * and q = 0 when no sample has a positive weight: the newest sample weighs
 * most and the weight falls linearly to zero at the far end of the window.
 * A slot with a negative time is empty; delays lie in [0, PARD_WAIT_LIMIT_US).
 * The result, int64 [n_ctx][stage_stride], is what pard_queue_state_t.d_q_us
 * expects; d_now_us is [n_ctx] as in pard_queue_state_t.
 *   d_sample_time_us   DEVICE, int64, 8-byte aligned
 *   d_sample_delay_us  DEVICE, int32
 *   d_workspace        DEVICE, 256-byte aligned, pard_update_queue_delay_workspace_bytes()
 *   mode               0 or PARD_MODE_NOWAIT (pard_plan_status fetches the status)
 * n_samples <= PARD_MAX_DELAY_SAMPLES, 1 <= window_us <= PARD_MAX_DELAY_WINDOW_US.
 * Host-detectable errors come back before anything is launched; a delay out of
 * range gives PARD_EDATA with unspecified outputs.  One kernel is enqueued on
 * cuda_stream; nothing is allocated. */
int pard_update_queue_delay_workspace_bytes(uint64_t* bytes);
int pard_update_queue_delay(uint32_t n_ctx, int32_t stage_stride, const int64_t* d_now_us,
                            const int64_t* d_sample_time_us, const int32_t* d_sample_delay_us,
                            uint32_t n_samples, uint32_t window_us, uint32_t mode,
                            int64_t* d_q_us, void* d_workspace, uint64_t workspace_bytes,
                            void* cuda_stream);

/* Carries the queue state from one decision epoch to the next, for replaying a
 * workload in closed loop: what pard_plan admitted is what the workers will
 * run.  (The paper's system measures this state on live workers, Sec. 4.1
 * step 1; a replay has to derive it, and does so with the planner's own model
 * of Sec. 4.2: t_e is the expected end of the previous batch, and batches run
 * back to back.)  For every (ctx, stage k of its pipeline), with
 * base = max(now, free_at_k):
 *   - the queueing delay met by a request dequeued at `now`, base - now (capped
 *     at PARD_WAIT_LIMIT_US - 1), is stored with time `now` in slot `slot` of
 *     the stage's sample ring, the arrays pard_update_queue_delay reads
 *     ([n_ctx][stage_stride][n_samples]; n_samples = 0 keeps no samples);
 *   - free_at_k = base + ceil(kept / (B_k * m_k)) * d_k(B_k), with kept =
 *     d_seg_kept[ctx * stage_stride + k] as written by pard_plan.
 * d_free_at_us is read and written in place; columns of stages the ctx's
 * pipeline lacks are left untouched.  All arrays are DEVICE memory laid out as
 * in pard_queue_state_t (d_workers NULL => 1).  d_workspace: 256-byte aligned,
 * pard_advance_state_workspace_bytes().  mode: 0 or PARD_MODE_NOWAIT.
 * Host-detectable errors come back before anything is launched; a batch size,
 * worker count or time out of range (also a new free_at beyond
 * PARD_TIME_LIMIT_US) gives PARD_EDATA.  One kernel is enqueued; nothing is
 * allocated. */
int pard_advance_state_workspace_bytes(uint32_t n_pipelines, uint64_t* bytes);
int pard_advance_state(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                       const int32_t* d_pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                       const int64_t* d_now_us, const int32_t* d_batch, const int32_t* d_workers,
                       const uint32_t* d_seg_kept, int64_t* d_free_at_us,
                       int64_t* d_sample_time_us, int32_t* d_sample_delay_us,
                       uint32_t n_samples, uint32_t slot, uint32_t mode,
                       void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);

/* Adaptive request priority with delayed transition (Sec. 4.3): chooses, for
 * every (ctx, stage) queue, the decision order that pard_plan reads from
 * pard_queue_state_t.d_priority.  With
 *   T_in   the queue's input workload: d_arrivals[(ctx * stage_stride + stage)
 *          * n_hist + j], j < n_hist, requests that arrived in the j-th sampling
 *          interval of interval_us microseconds, oldest first, each in
 *          [0, PARD_RATE_LIMIT)
 *   T_s    T_in smoothed by a sliding-window average over `window` samples,
 *          defined from sample window - 1 on (earlier samples only fill the
 *          window)
 *   eps  = sum |T_in - T_s| / sum T_in           (both sums from sample window - 1 on)
 *   T_m  = B_k * m_k / d_k(B_k)                  module throughput from batch size and
 *                                                execution duration
 *   mu   = T_in / T_m                            T_in: the latest sample as a rate
 * the queue's priority becomes 1 (high budget first) when mu > 1 + eps, 0 (low
 * budget first) when mu < 1 - eps, and is left as it is in between; a queue
 * without any arrival in the summed samples gets 0.  Comparisons are exact
 * (integers, cross-multiplied).
 *   d_batch, d_workers  DEVICE, as in pard_queue_state_t (d_workers NULL => 1);
 *                       B_k * m_k must stay below 2^31
 *   d_priority          DEVICE, uint8 [n_ctx][stage_stride], read (previous
 *                       priority) and written; entries of stages the ctx's
 *                       pipeline lacks are left untouched
 *   d_workspace         DEVICE, 256-byte aligned, pard_update_priority_workspace_bytes()
 *   mode                0 or PARD_MODE_NOWAIT (pard_plan_status fetches the status)
 * 1 <= window <= n_hist <= PARD_MAX_HISTORY, 1 <= interval_us < 2^31.
 * Host-detectable errors come back before anything is launched; a batch size,
 * worker count or sample out of range gives PARD_EDATA with unspecified
 * outputs.  One kernel is enqueued on cuda_stream; nothing is allocated. */
int pard_update_priority_workspace_bytes(uint32_t n_pipelines, uint64_t* bytes);
int pard_update_priority(const pard_pipeline_t* const* pipelines, uint32_t n_pipelines,
                         const int32_t* d_pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                         const int32_t* d_batch, const int32_t* d_workers,
                         const uint32_t* d_arrivals, uint32_t n_hist, uint32_t window,
                         uint32_t interval_us, uint32_t mode, uint8_t* d_priority,
                         void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);

/* ---- optional device timing of the planner's phases ----------------------
 * For benchmarks.  Between pard_profile_begin and pard_profile_end every
 * `every`-th pard_plan call of the process (at most max_samples of them)
 * records CUDA events on its stream between its phases; the other calls are
 * untouched.  pard_profile_end waits for the sampled calls, adds up the
 * elapsed milliseconds per phase into ms_sum[PARD_N_PHASES] and returns the
 * number of sampled calls.  A pard_goodput call that follows a sampled pard_plan
 * call counts into that call's last phase.  Process-wide state: do not call begin/end while
 * another thread is inside pard_plan.  The paper has no counterpart. */
#define PARD_N_PHASES 15
/* Or-ed into `every`: no events inside the decision pass (an event between two
 * kernels costs a few microseconds and keeps the second from being scheduled
 * while the first drains); "tables" then holds the time of the whole pass --
 * window tables, decision, compaction -- and "decide", "compact" are 0. */
#define PARD_PROFILE_COARSE 0x80000000u
int pard_profile_begin(uint32_t every, uint32_t max_samples);
int pard_profile_end(float* ms_sum, uint32_t* n_samples);
/* "clear", "prepass", "segments", "pack", "sort0".."sort7", "tables", "decide", "compact" */
const char* pard_profile_phase_name(uint32_t phase);

#ifdef __cplusplus
}
#endif
#endif  /* PARD_H_ */
