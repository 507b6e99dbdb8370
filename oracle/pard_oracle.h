/*
 * pard_oracle.h -- interface of the CPU oracle for the PARD drop planner.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded statement
 * of what the planner computes, written from the paper (Sec. 4.2 Eq. 1-3,
 * Sec. 4.3, Sec. 5.1).  It exists so that tests can compare the CUDA library
 * with it; it shares no code, header or table with that library, and no
 * product path may call it.
 *
 * All pointers are host pointers.  Times are int64 microseconds.
 */
#ifndef PARD_ORACLE_H_
#define PARD_ORACLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* One pipeline: the stage graph (successor lists, CSR) and the offline
 * latency profile d_k(b), b = 1..bmax[k] (Sec. 5.1, Implementation). */
typedef struct oracle_pipeline {
  int32_t        n_stages;
  const int32_t* sub_offsets;   /* [n_stages+1] */
  const int32_t* sub_ids;       /* successors   */
  const int32_t* bmax;          /* [n_stages]   */
  const int64_t* lat_offsets;   /* [n_stages+1] */
  const int64_t* lat_us;        /* d_k(b) at lat_offsets[k] + b - 1 */
} oracle_pipeline_t;

/* A queued request: deadline = send time t_s + SLO. 16 bytes. */
typedef struct oracle_request {
  int64_t  deadline_us;
  uint32_t ctx;
  uint16_t stage;
  uint16_t flags;
} oracle_request_t;

/* Runtime state, row-major per ctx; rows have stage_stride / slot_stride
 * entries.  pipeline_of_ctx, w_us, workers and priority may be NULL
 * (=> 0, 0, 1, 0). */
typedef struct oracle_state {
  int32_t        stage_stride;
  int32_t        slot_stride;
  const int32_t* pipeline_of_ctx;
  const int64_t* now_us;
  const int32_t* batch;
  const int64_t* free_at_us;
  const int64_t* q_us;
  const int64_t* w_us;
  const int32_t* workers;
  const uint8_t* priority;      /* [n_ctx][stage_stride] decision order of each queue (Sec. 4.3):
                                   0 = low budget first, 1 = high budget first; NULL => 0 */
} oracle_state_t;

/* Number of downstream paths of `stage` (0 for a sink). */
int64_t oracle_count_paths(const oracle_pipeline_t* p, int32_t stage);

/* First w slot of `stage`: downstream paths of all stages before it. */
int64_t oracle_slot_base(const oracle_pipeline_t* p, int32_t stage);

/* L_sub of Eq. 3 for one (ctx row, stage): the maximum over the stage's
 * downstream paths of sum (q_i + d_i(B_i)) + w[slot]; 0 at a sink.
 * batch_row/q_row have n_stages entries, w_row is the ctx's slot row or NULL. */
int64_t oracle_lsub(const oracle_pipeline_t* p, int32_t stage,
                    const int32_t* batch_row, const int64_t* q_row,
                    const int64_t* w_row);

/* L_sub for a request whose downstream path is (partly) known -- the dynamic-path
 * DAGs of Sec. 5.2, where a request takes one of several branches: the maximum
 * is taken only over the stage's downstream paths j (in the lexicographic
 * enumeration, j = 0, 1, ...) whose bit j is set in `mask`.  mask = 0 means
 * "unknown": all paths, i.e. oracle_lsub.  A sink gives 0 whatever the mask.
 * Returns -1 when the mask selects no existing path. */
int64_t oracle_lsub_masked(const oracle_pipeline_t* p, int32_t stage,
                           const int32_t* batch_row, const int64_t* q_row,
                           const int64_t* w_row, uint16_t mask);

/* Decision rules and orders beside the paper's own (Sec. 5.1 Baseline, Sec. 5.2
 * dynamic paths, Table 1 / Sec. 5.3 FCFS), selected by bits of `mode`:
 *   ORACLE_MODE_PATH_MASK  request.flags is the path mask of oracle_lsub_masked
 *   ORACLE_MODE_FCFS       queues are served in arrival order, which is the order
 *                          of the request array (index order), not budget order;
 *                          estimate and drop rule unchanged  (PARD-FCFS)
 *   ORACLE_MODE_NEXUS      Nexus' reactive rule, arrival order: the queue is scanned
 *                          with a window of one batch round (B*m requests); the
 *                          batch is the first window whose requests can all finish
 *                          the CURRENT module by their deadline if the batch starts
 *                          when the previous one ends; every request before that
 *                          window is dropped; the scan resumes behind the window one
 *                          execution duration later.  A last window that the queue
 *                          cannot fill is run as it is.  est = end of the batch the
 *                          request was tested against.
 *   ORACLE_MODE_CLIPPER    Clipper++: arrival order; module k gets the share
 *                          SLO_k = floor(SLO * d_k / sum_i d_i) of the request's
 *                          objective (d_i at the current batch sizes, all stages of
 *                          the pipeline); a request is dropped iff, when its batch
 *                          starts, it has already spent more than SLO_k in the
 *                          module: start - arrive > SLO_k.  Needs `arrivals`.
 *                          est = end of that batch.
 * NEXUS and CLIPPER exclude each other, PATH_MASK and bit 0. */
#define ORACLE_MODE_PATH_MASK 16u
#define ORACLE_MODE_FCFS      32u
#define ORACLE_MODE_NEXUS     64u
#define ORACLE_MODE_CLIPPER   128u

/* when the request reached its current module, and its end-to-end objective */
typedef struct oracle_arrival {
  int64_t arrive_us;
  int64_t slo_us;
} oracle_arrival_t;

/* The planner.  mode bit 0: 0 = a dropped request takes no batch slot,
 * 1 = every request ahead takes one; further bits as above (`arrivals` is
 * [n], needed by ORACLE_MODE_CLIPPER only; oracle_plan passes NULL).
 * Outputs (any may be NULL):
 *   keep[n], est_us[n], perm[n]      in service order
 *   kept_idx[n], *n_kept             original indices of kept requests
 *   seg_offsets[n_ctx*stage_stride+1], seg_kept[n_ctx*stage_stride]
 *   ctx_total[n_ctx], ctx_kept[n_ctx]
 * Returns 0, or -1 when an input is out of range. */
int oracle_plan(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                const oracle_request_t* requests, uint64_t n,
                const oracle_state_t* state, uint32_t n_ctx, uint32_t mode,
                uint8_t* keep, int64_t* est_us, uint32_t* perm,
                uint32_t* kept_idx, uint64_t* n_kept,
                uint32_t* seg_offsets, uint32_t* seg_kept,
                int64_t* ctx_total, int64_t* ctx_kept);
int oracle_plan_policy(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                       const oracle_request_t* requests, const oracle_arrival_t* arrivals,
                       uint64_t n, const oracle_state_t* state, uint32_t n_ctx, uint32_t mode,
                       uint8_t* keep, int64_t* est_us, uint32_t* perm,
                       uint32_t* kept_idx, uint64_t* n_kept,
                       uint32_t* seg_offsets, uint32_t* seg_kept,
                       int64_t* ctx_total, int64_t* ctx_kept);

/* Batch-wait estimate w = F^{-1}(lambda) of the State Planner (Sec. 4.2, Batch
 * wait estimation): for every (ctx, stage k, downstream path P) slot, draw M
 * samples of the aggregated batch wait -- one recorded batch wait of every
 * stage on P, picked at random -- and return the sample of rank
 * floor(lambda_num * M / lambda_den) (clamped to M - 1) in ascending order.
 * wait_samples[(ctx * stage_stride + stage) * M + j], j < M, are the stage's
 * recorded batch waits in microseconds.  The random pick for sample m and the
 * j-th stage of the path is  idx = (hi32(splitmix64(counter)) * M) >> 32  with
 * counter = seed + (((ctx * slot_stride + slot) * M + m) * 64 + j)  (splitmix64
 * as published by Steele, Lea and Flood).  w_us[ctx * slot_stride + slot] is
 * written for the slots of the ctx's pipeline.  Returns 0, or -1 on bad input. */
int oracle_estimate_w(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                      const int32_t* pipeline_of_ctx, uint32_t n_ctx,
                      int32_t stage_stride, int32_t slot_stride,
                      const int32_t* wait_samples, uint32_t M,
                      uint32_t lambda_num, uint32_t lambda_den, uint64_t seed,
                      int64_t* w_us);

/* Adaptive request priority with delayed transition (Sec. 4.3).  For every
 * (ctx, stage) queue:
 *   T_in   the input workload: arrivals[(ctx * stage_stride + stage) * n_hist + j],
 *          j < n_hist, is the number of requests that arrived in the j-th
 *          sampling interval of interval_us microseconds, oldest first
 *   T_s    T_in filtered by a sliding-window average over `window` samples;
 *          defined for j >= window - 1 (the first window - 1 samples only fill
 *          the window)
 *   eps  = sum |T_in - T_s| / sum T_in          both sums over j >= window - 1
 *   T_m  = B_k * m_k / d_k(B_k)                 module throughput (requests per us)
 *   mu   = T_in / T_m, with T_in the latest sample as a rate (per us)
 * The new priority is 1 (high budget first) if mu > 1 + eps, 0 (low budget
 * first) if mu < 1 - eps, and the previous one otherwise; a queue with no
 * arrival in the summed intervals gets 0.  All comparisons are exact (integer
 * cross-multiplication).  priority[n_ctx * stage_stride] holds the previous
 * priorities on entry and the new ones on return; entries of stages the ctx's
 * pipeline lacks are left untouched.  workers may be NULL (=> 1).
 * Returns 0, or -1 on bad input. */
int oracle_update_priority(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                           const int32_t* pipeline_of_ctx, uint32_t n_ctx,
                           int32_t stage_stride, const int32_t* batch,
                           const int32_t* workers, const uint32_t* arrivals,
                           uint32_t n_hist, uint32_t window, uint32_t interval_us,
                           uint8_t* priority);

/* Recent average queueing delay q_k of the State Planner (Sec. 4.2: monitored
 * with a sliding window, by default a 5 s linear weighted one).  For every
 * (ctx, stage): over the recorded samples j < n_samples, taken at time
 * sample_time_us[..][j] with measured queueing delay sample_delay_us[..][j],
 *   weight_j = window_us - (now - t_j)   if 0 <= now - t_j < window_us, else 0
 *   q        = floor( sum weight_j * delay_j / sum weight_j ),  0 when no sample
 *              has a positive weight
 * so the newest sample weighs most and the weight falls linearly to zero at the
 * far end of the window.  A slot with a negative time is empty.  Arrays are
 * [n_ctx][stage_stride][n_samples] (samples in any order), now_us is [n_ctx],
 * q_us is [n_ctx][stage_stride].  Returns 0, or -1 on bad input. */
int oracle_queue_delay(uint32_t n_ctx, int32_t stage_stride, const int64_t* now_us,
                       const int64_t* sample_time_us, const int32_t* sample_delay_us,
                       uint32_t n_samples, uint32_t window_us, int64_t* q_us);

/* Carries the queue state from one decision epoch to the next (closed loop:
 * what the planner admitted is what the workers will run).  For every (ctx,
 * stage k of its pipeline), with base = max(now, free_at_k) the start of the
 * next batch as the planner saw it (Sec. 4.2: t_e, the expected end of the
 * previous batch):
 *   - the queueing delay a request dequeued at `now` meets, base - now
 *     (capped at 2^24 - 1), is recorded with time `now` in slot `slot` of the
 *     stage's sample ring (the samples oracle_queue_delay averages);
 *   - the seg_kept[ctx * stage_stride + k] admitted requests run back to back
 *     in rounds of B_k * m_k, each round d_k(B_k) long, so
 *     free_at_k = base + ceil(kept / (B_k * m_k)) * d_k(B_k).
 * Columns of stages the pipeline lacks are left untouched.  Returns 0 or -1. */
int oracle_advance_state(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                         const int32_t* pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                         const int64_t* now_us, const int32_t* batch, const int32_t* workers,
                         const uint32_t* seg_kept, int64_t* free_at_us,
                         int64_t* sample_time_us, int32_t* sample_delay_us,
                         uint32_t n_samples, uint32_t slot);

#ifdef __cplusplus
}
#endif
#endif  /* PARD_ORACLE_H_ */
