/*
 * pard_oracle.cpp -- CPU oracle of the PARD drop planner.
 *
 * TEST INFRASTRUCTURE ONLY: plain, slow, single-threaded, written from the
 * paper so that a reader can check it by eye.  It shares nothing with the CUDA
 * library and no product path may call it.
 *
 * What it follows:
 *   Eq. 1   L = L_pre + L_cur + L_sub                          (Sec. 4.2)
 *   Eq. 2   Lat_k = Q_k + W_k + D_k                            (Sec. 4.2)
 *   Eq. 3   L = (t_e - t_s + d_k) + (sum q_i + sum d_i + w_k)  (Sec. 4.2)
 *   DAG:    the estimate is taken along every subsequent path and the
 *           maximum is used                                     (Sec. 4.2, 5.1)
 *   Order:  low budget first = smallest remaining budget first, or high
 *           budget first = largest first, per queue                (Sec. 4.3)
 *   mu/eps: load factor, fluctuation bound, delayed transition     (Sec. 4.3)
 *   q_k:    linear weighted sliding-window average queueing delay  (Sec. 4.2)
 *   Rule:   drop when the estimate exceeds the latency objective (Sec. 5.3)
 *   Counts: goodput / drop rate                                 (Sec. 5.1)
 *   w_k:    quantile lambda of the sampled aggregated batch wait  (Sec. 4.2)
 *   Other rules on the same queues: dynamic-path requests (Sec. 5.2), arrival
 *           order (Table 1, Sec. 5.3), Nexus and Clipper++ (Sec. 5.1 Baseline)
 *
 * Readings where the paper is silent (each also listed in the design notes):
 *   - Snapshot: the Request Broker loop is run over the whole queue at the
 *     instant `now`; batches of a stage run back to back, batch j starting at
 *     base + j*d with base = max(now, free_at) (t_e chained forward).
 *   - A dropped request never enters a batch, so the position that decides the
 *     batch index counts kept requests only (mode 0).  Mode 1 counts all.
 *   - d_k is the profile at the stage's current batch size for every batch.
 *   - est == deadline is kept; equal deadlines are served in index order
 *     (under either priority).
 *   - w covers the stages after k; one value per (stage, downstream path).
 *   - m identical workers drain one queue: a batch round starts B*m requests.
 */
#include "pard_oracle.h"

#include <algorithm>
#include <vector>

namespace {

int64_t profile_at(const oracle_pipeline_t* p, int32_t stage, int32_t b) {
  return p->lat_us[p->lat_offsets[stage] + b - 1];
}

std::vector<int32_t> successors_ascending(const oracle_pipeline_t* p, int32_t stage) {
  std::vector<int32_t> s(p->sub_ids + p->sub_offsets[stage],
                         p->sub_ids + p->sub_offsets[stage + 1]);
  std::sort(s.begin(), s.end());
  return s;
}

/* Number of stage sequences that start at `stage` and end at a sink. */
int64_t count_from(const oracle_pipeline_t* p, int32_t stage) {
  std::vector<int32_t> s = successors_ascending(p, stage);
  if (s.empty()) return 1;
  int64_t c = 0;
  for (int32_t j : s) c += count_from(p, j);
  return c;
}

/* Walks every path that continues through `stage`.  `acc` is the sum of
 * q_i + d_i(B_i) over the path's stages before this one.  Each time a sink is
 * reached one complete path has been seen; paths are met in lexicographic
 * order of their stage sequence, so the running counter `slot` is the path's
 * w index. */
int64_t walk(const oracle_pipeline_t* p, int32_t stage, int64_t acc,
             const int32_t* batch_row, const int64_t* q_row,
             const int64_t* w_row, int64_t* slot) {
  acc += q_row[stage] + profile_at(p, stage, batch_row[stage]);
  std::vector<int32_t> s = successors_ascending(p, stage);
  if (s.empty()) {
    int64_t w = w_row ? w_row[*slot] : 0;
    *slot += 1;
    return acc + w;
  }
  bool first = true;
  int64_t best = 0;
  for (int32_t j : s) {
    int64_t v = walk(p, j, acc, batch_row, q_row, w_row, slot);
    if (first || v > best) best = v;
    first = false;
  }
  return best;
}

}  // namespace

extern "C" int64_t oracle_count_paths(const oracle_pipeline_t* p, int32_t stage) {
  std::vector<int32_t> s = successors_ascending(p, stage);
  int64_t c = 0;
  for (int32_t j : s) c += count_from(p, j);
  return c;
}

extern "C" int64_t oracle_slot_base(const oracle_pipeline_t* p, int32_t stage) {
  int64_t base = 0;
  for (int32_t k = 0; k < stage; ++k) base += oracle_count_paths(p, k);
  return base;
}

extern "C" int64_t oracle_lsub(const oracle_pipeline_t* p, int32_t stage,
                               const int32_t* batch_row, const int64_t* q_row,
                               const int64_t* w_row) {
  std::vector<int32_t> s = successors_ascending(p, stage);
  if (s.empty()) return 0;                       /* nothing after a sink */
  int64_t slot = oracle_slot_base(p, stage);
  bool first = true;
  int64_t best = 0;
  for (int32_t j : s) {
    int64_t v = walk(p, j, 0, batch_row, q_row, w_row, &slot);
    if (first || v > best) best = v;
    first = false;
  }
  return best;
}

namespace {

/* As walk(), but a complete path counts only if the bit of its rank among the
 * stage's downstream paths (`rank` runs 0, 1, ... in lexicographic order) is
 * set in `mask`.  Returns -1 when no path below `stage` counts (every path sum
 * is at least one execution duration, so -1 cannot be a sum). */
int64_t walk_masked(const oracle_pipeline_t* p, int32_t stage, int64_t acc,
                    const int32_t* batch_row, const int64_t* q_row, const int64_t* w_row,
                    int64_t slot_base, int64_t* rank, uint16_t mask) {
  acc += q_row[stage] + profile_at(p, stage, batch_row[stage]);
  std::vector<int32_t> s = successors_ascending(p, stage);
  if (s.empty()) {
    int64_t r = *rank;
    *rank += 1;
    if (r >= 16 || !((mask >> r) & 1)) return -1;           /* not a path this request can take */
    return acc + (w_row ? w_row[slot_base + r] : 0);
  }
  int64_t best = -1;
  for (int32_t j : s) best = std::max(best, walk_masked(p, j, acc, batch_row, q_row, w_row, slot_base, rank, mask));
  return best;
}

}  // namespace

extern "C" int64_t oracle_lsub_masked(const oracle_pipeline_t* p, int32_t stage,
                                      const int32_t* batch_row, const int64_t* q_row,
                                      const int64_t* w_row, uint16_t mask) {
  if (mask == 0) return oracle_lsub(p, stage, batch_row, q_row, w_row);   /* path unknown: all of them */
  std::vector<int32_t> s = successors_ascending(p, stage);
  if (s.empty()) return 0;
  int64_t rank = 0, best = -1;
  for (int32_t j : s)
    best = std::max(best, walk_masked(p, j, 0, batch_row, q_row, w_row, oracle_slot_base(p, stage), &rank, mask));
  return best;
}

namespace {

/* splitmix64 (Steele, Lea, Flood: "Fast splittable pseudorandom number generators") */
uint64_t splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

/* every downstream path of `stage` continuing through `cur`, in lexicographic order */
void collect_paths(const oracle_pipeline_t* p, int32_t cur, std::vector<int32_t>* prefix,
                   std::vector<std::vector<int32_t>>* out) {
  prefix->push_back(cur);
  std::vector<int32_t> s = successors_ascending(p, cur);
  if (s.empty()) out->push_back(*prefix);
  for (int32_t j : s) collect_paths(p, j, prefix, out);
  prefix->pop_back();
}

}  // namespace

extern "C" int oracle_estimate_w(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                                 const int32_t* pipeline_of_ctx, uint32_t n_ctx,
                                 int32_t stage_stride, int32_t slot_stride,
                                 const int32_t* wait_samples, uint32_t M,
                                 uint32_t lambda_num, uint32_t lambda_den, uint64_t seed,
                                 int64_t* w_us) {
  if (M == 0 || lambda_den == 0 || lambda_num > lambda_den) return -1;
  uint64_t rank = (uint64_t)lambda_num * M / lambda_den;        /* lambda = 0: smallest, lambda = 1: largest */
  if (rank > M - 1) rank = M - 1;
  for (uint32_t c = 0; c < n_ctx; ++c) {
    int32_t pi = pipeline_of_ctx ? pipeline_of_ctx[c] : 0;
    if (pi < 0 || pi >= n_pipelines) return -1;
    const oracle_pipeline_t* p = &pipelines[pi];
    int64_t slot = 0;
    for (int32_t k = 0; k < p->n_stages; ++k) {
      std::vector<std::vector<int32_t>> paths;
      std::vector<int32_t> prefix;
      for (int32_t j : successors_ascending(p, k)) collect_paths(p, j, &prefix, &paths);
      for (const std::vector<int32_t>& path : paths) {        /* one slot per (stage, downstream path) */
        if (slot >= slot_stride) return -1;
        std::vector<int64_t> sums(M);
        for (uint32_t m = 0; m < M; ++m) {
          int64_t sum = 0;                                    /* aggregated batch wait of one sampled request */
          for (size_t j = 0; j < path.size(); ++j) {
            uint64_t counter = seed + ((((uint64_t)c * (uint64_t)slot_stride + (uint64_t)slot) * M + m) * 64 + j);
            uint64_t idx = ((splitmix64(counter) >> 32) * (uint64_t)M) >> 32;
            sum += wait_samples[((size_t)c * stage_stride + path[j]) * M + idx];
          }
          sums[m] = sum;
        }
        std::sort(sums.begin(), sums.end());
        w_us[(size_t)c * slot_stride + slot] = sums[rank];    /* F^{-1}(lambda) */
        ++slot;
      }
    }
  }
  return 0;
}

extern "C" int oracle_plan(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                           const oracle_request_t* requests, uint64_t n,
                           const oracle_state_t* st, uint32_t n_ctx, uint32_t mode,
                           uint8_t* keep, int64_t* est_us, uint32_t* perm,
                           uint32_t* kept_idx, uint64_t* n_kept,
                           uint32_t* seg_offsets, uint32_t* seg_kept,
                           int64_t* ctx_total, int64_t* ctx_kept) {
  return oracle_plan_policy(pipelines, n_pipelines, requests, nullptr, n, st, n_ctx, mode, keep, est_us,
                            perm, kept_idx, n_kept, seg_offsets, seg_kept, ctx_total, ctx_kept);
}

extern "C" int oracle_plan_policy(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                                  const oracle_request_t* requests, const oracle_arrival_t* arrivals,
                                  uint64_t n, const oracle_state_t* st, uint32_t n_ctx, uint32_t mode,
                                  uint8_t* keep, int64_t* est_us, uint32_t* perm,
                                  uint32_t* kept_idx, uint64_t* n_kept,
                                  uint32_t* seg_offsets, uint32_t* seg_kept,
                                  int64_t* ctx_total, int64_t* ctx_kept) {
  const bool nexus = mode & ORACLE_MODE_NEXUS, clipper = mode & ORACLE_MODE_CLIPPER;
  const bool masked = mode & ORACLE_MODE_PATH_MASK;
  const bool arrival_order = (mode & ORACLE_MODE_FCFS) || nexus || clipper;
  if (nexus && clipper) return -1;
  if ((nexus || clipper) && (masked || (mode & 1u))) return -1;
  if (clipper && n > 0 && !arrivals) return -1;
  const int64_t S = st->stage_stride;
  /* one queue per (ctx, stage), filled in arrival (index) order */
  std::vector<std::vector<uint32_t>> queue((size_t)n_ctx * S);
  for (uint64_t i = 0; i < n; ++i) {
    const oracle_request_t& r = requests[i];
    if (r.ctx >= n_ctx) return -1;
    int32_t pi = st->pipeline_of_ctx ? st->pipeline_of_ctx[r.ctx] : 0;
    if (pi < 0 || pi >= n_pipelines) return -1;
    if (r.stage >= pipelines[pi].n_stages) return -1;
    queue[(size_t)r.ctx * S + r.stage].push_back((uint32_t)i);
  }

  uint64_t pos = 0;        /* position in service order */
  uint64_t kept_all = 0;
  for (uint32_t c = 0; c < n_ctx; ++c) {
    int32_t pi = st->pipeline_of_ctx ? st->pipeline_of_ctx[c] : 0;
    if (pi < 0 || pi >= n_pipelines) return -1;
    const oracle_pipeline_t* p = &pipelines[pi];
    const int32_t* batch_row = st->batch + (size_t)c * S;
    const int64_t* q_row = st->q_us + (size_t)c * S;
    const int64_t* free_row = st->free_at_us + (size_t)c * S;
    const int64_t* w_row = st->w_us ? st->w_us + (size_t)c * st->slot_stride : nullptr;
    const int32_t* m_row = st->workers ? st->workers + (size_t)c * S : nullptr;
    int64_t total_c = 0, kept_c = 0;

    for (int32_t k = 0; k < S; ++k) {
      std::vector<uint32_t>& qk = queue[(size_t)c * S + k];
      if (seg_offsets) seg_offsets[(size_t)c * S + k] = (uint32_t)pos;
      if (k >= p->n_stages) {                    /* padding column of the row */
        if (seg_kept) seg_kept[(size_t)c * S + k] = 0;
        continue;
      }
      int32_t B = batch_row[k];
      if (B < 1 || B > p->bmax[k]) return -1;
      int64_t m = m_row ? m_row[k] : 1;
      if (m < 1) return -1;
      int64_t d = profile_at(p, k, B);           /* D_k = d_k at the current batch size */
      int64_t cap = (int64_t)B * m;
      int64_t base = std::max(st->now_us[c], free_row[k]);   /* t_e of the next batch */
      int64_t lsub = oracle_lsub(p, k, batch_row, q_row, w_row);

      /* the remaining budget of a request is its deadline minus the same `now`
       * for the whole queue, so budget order is deadline order.
       * low budget first: smallest deadline first; high budget first: largest
       * deadline first; ties in index order either way.  Arrival order (PARD-FCFS,
       * Nexus, Clipper++) leaves the queue as it was filled. */
      bool high_first = st->priority && st->priority[(size_t)c * S + k] != 0;
      if (arrival_order) {
      } else if (high_first)
        std::stable_sort(qk.begin(), qk.end(), [&](uint32_t a, uint32_t b) {
          return requests[a].deadline_us > requests[b].deadline_us;
        });
      else
        std::stable_sort(qk.begin(), qk.end(), [&](uint32_t a, uint32_t b) {
          return requests[a].deadline_us < requests[b].deadline_us;
        });

      int64_t kept = 0, raw = 0;
      if (nexus) {
        /* Sec. 5.1 Baseline, Nexus: a window of one batch round slides over the queue in
         * arrival order; t is when the batch being formed would start */
        int64_t t = base;
        size_t window_start = 0;                 /* first request of the window being tried */
        std::vector<uint8_t> in_batch(qk.size(), 0);
        std::vector<int64_t> tested_end(qk.size(), 0);
        for (size_t r = 0; r < qk.size(); ++r) {
          const bool fits = t + d <= requests[qk[r]].deadline_us;   /* enough budget left for this module */
          tested_end[r] = t + d;
          if (!fits) {
            window_start = r + 1;                /* no window that holds r can be the batch: all before it go too */
          } else if ((int64_t)(r - window_start + 1) == cap) {
            for (size_t j = window_start; j <= r; ++j) in_batch[j] = 1;
            t += d;                              /* the next batch starts when this one ends */
            window_start = r + 1;
          }
        }
        /* what is left behind the last full batch fits and runs as a partly filled batch */
        for (size_t j = window_start; j < qk.size(); ++j) in_batch[j] = 1;
        for (size_t r = 0; r < qk.size(); ++r) {
          if (keep) keep[pos] = in_batch[r];
          if (est_us) est_us[pos] = tested_end[r];
          if (perm) perm[pos] = qk[r];
          if (in_batch[r]) {
            if (kept_idx) kept_idx[kept_all] = qk[r];
            ++kept_all;
            ++kept;
          }
          ++raw;
          ++pos;
        }
      } else {
        int64_t dsum = 0;                        /* Clipper++: sum of d_i over the pipeline's modules */
        if (clipper) for (int32_t i = 0; i < p->n_stages; ++i) {
          if (batch_row[i] < 1 || batch_row[i] > p->bmax[i]) return -1;
          dsum += profile_at(p, i, batch_row[i]);
        }
        for (uint32_t i : qk) {                    /* the Request Broker, one request at a time */
          int64_t ahead = (mode & 1u) ? raw : kept;
          int64_t t_e = base + (ahead / cap) * d;  /* its batch starts when the previous one ends */
          int64_t est;
          bool k_;
          if (clipper) {
            /* Sec. 5.1 Baseline, Clipper++: SLO_k = SLO * d_k / sum d_i; dropped iff the request has
             * already used up that share when its inference would start */
            if (arrivals[i].slo_us < 0) return -1;
            int64_t share = (int64_t)(((__int128)arrivals[i].slo_us * d) / dsum);
            est = t_e + d;
            k_ = t_e - arrivals[i].arrive_us <= share;
          } else {
            int64_t lsub_i = lsub;
            if (masked) {
              lsub_i = oracle_lsub_masked(p, k, batch_row, q_row, w_row, requests[i].flags);
              if (lsub_i < 0) return -1;
            }
            est = t_e + d + lsub_i;                /* t_s + L of Eq. 3 */
            k_ = est <= requests[i].deadline_us;
          }
          if (keep) keep[pos] = k_ ? 1 : 0;
          if (est_us) est_us[pos] = est;
          if (perm) perm[pos] = i;
          if (k_) {
            if (kept_idx) kept_idx[kept_all] = i;
            ++kept_all;
            ++kept;
          }
          ++raw;
          ++pos;
        }
      }
      if (seg_kept) seg_kept[(size_t)c * S + k] = (uint32_t)kept;
      total_c += raw;
      kept_c += kept;
    }
    if (ctx_total) ctx_total[c] = total_c;
    if (ctx_kept) ctx_kept[c] = kept_c;
  }
  if (seg_offsets) seg_offsets[(size_t)n_ctx * S] = (uint32_t)pos;
  if (n_kept) *n_kept = kept_all;
  return 0;
}

extern "C" int oracle_update_priority(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                                      const int32_t* pipeline_of_ctx, uint32_t n_ctx,
                                      int32_t stage_stride, const int32_t* batch,
                                      const int32_t* workers, const uint32_t* arrivals,
                                      uint32_t n_hist, uint32_t window, uint32_t interval_us,
                                      uint8_t* priority) {
  typedef unsigned __int128 u128;
  if (window < 1 || window > n_hist || interval_us < 1) return -1;
  for (uint32_t c = 0; c < n_ctx; ++c) {
    int32_t pi = pipeline_of_ctx ? pipeline_of_ctx[c] : 0;
    if (pi < 0 || pi >= n_pipelines) return -1;
    const oracle_pipeline_t* p = &pipelines[pi];
    for (int32_t k = 0; k < p->n_stages; ++k) {
      size_t seg = (size_t)c * stage_stride + k;
      int32_t B = batch[seg];
      if (B < 1 || B > p->bmax[k]) return -1;
      int64_t m = workers ? workers[seg] : 1;
      if (m < 1) return -1;
      int64_t d = profile_at(p, k, B);
      int64_t cap = (int64_t)B * m;                       /* T_m = cap / d requests per microsecond */
      const uint32_t* x = arrivals + seg * n_hist;        /* T_in, one sample per interval */

      /* eps = sum |T_in - T_s| / sum T_in with T_s[j] = (x[j-W+1] + ... + x[j]) / W.
       * Scaled by W to stay in integers:  eps = dev / (W * sum_x). */
      uint64_t W = window, sum_x = 0, dev = 0;
      for (uint32_t j = window - 1; j < n_hist; ++j) {
        uint64_t win = 0;
        for (uint32_t i = j + 1 - window; i <= j; ++i) win += x[i];
        uint64_t wx = W * x[j];
        dev += wx > win ? wx - win : win - wx;            /* W * |T_in[j] - T_s[j]| */
        sum_x += x[j];
      }
      if (sum_x == 0) {                                   /* nothing arrived: within capacity */
        priority[seg] = 0;
        continue;
      }
      /* mu = (x_now / interval) / (cap / d) = x_now * d / (cap * interval);
       * mu > 1 + eps  <=>  x_now * d * (W * sum_x) > cap * interval * (W * sum_x + dev)
       * mu < 1 - eps  <=>  x_now * d * (W * sum_x) < cap * interval * (W * sum_x - dev) */
      uint64_t x_now = x[n_hist - 1];
      u128 lhs = (u128)x_now * (u128)(uint64_t)d * (u128)(W * sum_x);
      u128 scale = (u128)(uint64_t)cap * (u128)interval_us;
      u128 upper = scale * (u128)(W * sum_x + dev);
      if (lhs > upper) {
        priority[seg] = 1;                                /* under-provisioned: high budget first */
      } else if (W * sum_x > dev && lhs < scale * (u128)(W * sum_x - dev)) {
        priority[seg] = 0;                                /* within capacity: low budget first */
      }                                                   /* else: inside [1 - eps, 1 + eps], unchanged */
    }
  }
  return 0;
}

extern "C" int oracle_queue_delay(uint32_t n_ctx, int32_t stage_stride, const int64_t* now_us,
                                  const int64_t* sample_time_us, const int32_t* sample_delay_us,
                                  uint32_t n_samples, uint32_t window_us, int64_t* q_us) {
  typedef unsigned __int128 u128;
  if (window_us < 1 || stage_stride < 1) return -1;
  for (uint32_t c = 0; c < n_ctx; ++c) {
    for (int32_t k = 0; k < stage_stride; ++k) {
      size_t seg = (size_t)c * stage_stride + k;
      u128 weighted = 0;                                   /* sum weight_j * delay_j */
      u128 weights = 0;                                    /* sum weight_j */
      for (uint32_t j = 0; j < n_samples; ++j) {
        int64_t t = sample_time_us[seg * n_samples + j];
        if (t < 0) continue;                               /* empty slot */
        int32_t delay = sample_delay_us[seg * n_samples + j];
        if (delay < 0) return -1;
        if (t > now_us[c]) continue;                       /* not yet happened at this snapshot */
        int64_t age = now_us[c] - t;
        if (age >= (int64_t)window_us) continue;           /* slid out of the window */
        uint64_t weight = (uint64_t)window_us - (uint64_t)age;   /* newest: window, oldest: 1 */
        weighted += (u128)weight * (u128)(uint64_t)delay;
        weights += weight;
      }
      q_us[seg] = weights == 0 ? 0 : (int64_t)(weighted / weights);
    }
  }
  return 0;
}

extern "C" int oracle_advance_state(const oracle_pipeline_t* pipelines, int32_t n_pipelines,
                                    const int32_t* pipeline_of_ctx, uint32_t n_ctx, int32_t stage_stride,
                                    const int64_t* now_us, const int32_t* batch, const int32_t* workers,
                                    const uint32_t* seg_kept, int64_t* free_at_us,
                                    int64_t* sample_time_us, int32_t* sample_delay_us,
                                    uint32_t n_samples, uint32_t slot) {
  if (n_samples > 0 && slot >= n_samples) return -1;
  for (uint32_t c = 0; c < n_ctx; ++c) {
    int32_t pi = pipeline_of_ctx ? pipeline_of_ctx[c] : 0;
    if (pi < 0 || pi >= n_pipelines) return -1;
    const oracle_pipeline_t* p = &pipelines[pi];
    for (int32_t k = 0; k < p->n_stages; ++k) {
      size_t seg = (size_t)c * stage_stride + k;
      int32_t B = batch[seg];
      if (B < 1 || B > p->bmax[k]) return -1;
      int64_t m = workers ? workers[seg] : 1;
      if (m < 1) return -1;
      int64_t cap = (int64_t)B * m;
      int64_t d = profile_at(p, k, B);
      int64_t base = std::max(now_us[c], free_at_us[seg]);        /* t_e of the next batch */
      if (n_samples > 0) {
        int64_t delay = base - now_us[c];                           /* queueing delay met at `now` */
        sample_time_us[seg * n_samples + slot] = now_us[c];
        sample_delay_us[seg * n_samples + slot] = (int32_t)std::min<int64_t>(delay, (1 << 24) - 1);
      }
      int64_t rounds = ((int64_t)seg_kept[seg] + cap - 1) / cap;    /* batches run back to back */
      free_at_us[seg] = base + rounds * d;
    }
  }
  return 0;
}
