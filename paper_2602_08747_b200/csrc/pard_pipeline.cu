/* Host side of libpard: pipeline validation, downstream-path enumeration
 * (paper Sec. 4.2 / 5.1: the estimate is taken along each subsequent DAG path)
 * and upload of the tables to the device. */
#include <algorithm>
#include <cstring>
#include <new>

#include "pard_internal.h"

namespace {

constexpr int64_t kSat = (int64_t)1 << 40;   /* saturating path counter */

int64_t sat_add(int64_t a, int64_t b) { return std::min(kSat, a + b); }

int validate(const pard_dag_t* dag, const pard_profile_t* prof) {
  if (!dag || !prof || !dag->sub_offsets || !prof->bmax || !prof->lat_offsets || !prof->lat_us)
    return PARD_EINVAL;
  const int32_t S = dag->n_stages;
  if (S < 1) return PARD_EINVAL;
  if (S > PARD_MAX_STAGES) return PARD_ERANGE;
  if (dag->sub_offsets[0] != 0) return PARD_EINVAL;
  for (int32_t k = 0; k < S; ++k)
    if (dag->sub_offsets[k + 1] < dag->sub_offsets[k]) return PARD_EINVAL;
  if (dag->sub_offsets[S] > 0 && !dag->sub_ids) return PARD_EINVAL;
  for (int32_t k = 0; k < S; ++k) {
    bool seen[PARD_MAX_STAGES] = {false};
    for (int32_t e = dag->sub_offsets[k]; e < dag->sub_offsets[k + 1]; ++e) {
      int32_t j = dag->sub_ids[e];
      if (j < 0 || j >= S || j == k || seen[j]) return PARD_EINVAL;
      seen[j] = true;
    }
  }
  if (prof->lat_offsets[0] != 0) return PARD_EINVAL;
  for (int32_t k = 0; k < S; ++k) {
    if (prof->bmax[k] < 1) return PARD_EINVAL;
    if (prof->bmax[k] > PARD_MAX_BATCH) return PARD_ERANGE;
    if (prof->lat_offsets[k + 1] - prof->lat_offsets[k] != prof->bmax[k]) return PARD_EINVAL;
    for (int64_t i = prof->lat_offsets[k]; i < prof->lat_offsets[k + 1]; ++i)
      if (prof->lat_us[i] < 1 || prof->lat_us[i] >= PARD_LAT_LIMIT_US) return PARD_ERANGE;
  }
  return PARD_OK;
}

/* Kahn's algorithm; fills `order` with a topological order or reports a cycle. */
int topo_order(const pard_dag_t* dag, std::vector<int32_t>* order) {
  const int32_t S = dag->n_stages;
  std::vector<int32_t> indeg(S, 0);
  for (int32_t e = 0; e < dag->sub_offsets[S]; ++e) indeg[dag->sub_ids[e]]++;
  std::vector<int32_t> ready;
  for (int32_t k = 0; k < S; ++k)
    if (indeg[k] == 0) ready.push_back(k);
  while (!ready.empty()) {
    int32_t k = ready.back();
    ready.pop_back();
    order->push_back(k);
    for (int32_t e = dag->sub_offsets[k]; e < dag->sub_offsets[k + 1]; ++e)
      if (--indeg[dag->sub_ids[e]] == 0) ready.push_back(dag->sub_ids[e]);
  }
  return (int32_t)order->size() == S ? PARD_OK : PARD_ECYCLE;
}

struct Enumerator {
  const std::vector<std::vector<int32_t>>& succ;
  std::vector<int32_t>& path_off;
  std::vector<int32_t>& path_stage;
  std::vector<int32_t> cur;

  /* Appends every path that extends `cur` through stage k to a sink, children
   * visited in ascending id order so that paths come out lexicographically. */
  void extend(int32_t k) {
    cur.push_back(k);
    if (succ[k].empty()) {
      path_stage.insert(path_stage.end(), cur.begin(), cur.end());
      path_off.push_back((int32_t)path_stage.size());
    } else {
      for (int32_t j : succ[k]) extend(j);
    }
    cur.pop_back();
  }
};

}  // namespace

extern "C" int pard_load_pipeline(const pard_dag_t* dag, const pard_profile_t* prof,
                                  uint32_t flags, pard_pipeline_t** out) {
  if (!out) return PARD_EINVAL;
  *out = nullptr;
  if (flags & ~PARD_LOAD_HOST_ONLY) return PARD_EINVAL;
  int rc = validate(dag, prof);
  if (rc != PARD_OK) return rc;
  const int32_t S = dag->n_stages;

  std::vector<int32_t> order;
  rc = topo_order(dag, &order);
  if (rc != PARD_OK) return rc;

  std::vector<std::vector<int32_t>> succ(S);
  for (int32_t k = 0; k < S; ++k) {
    succ[k].assign(dag->sub_ids + dag->sub_offsets[k], dag->sub_ids + dag->sub_offsets[k + 1]);
    std::sort(succ[k].begin(), succ[k].end());
  }

  /* size check before enumerating: paths and summed path length from each stage */
  std::vector<int64_t> cnt(S, 0), len(S, 0);   /* sequences starting AT k */
  for (auto it = order.rbegin(); it != order.rend(); ++it) {
    int32_t k = *it;
    if (succ[k].empty()) {
      cnt[k] = 1;
      len[k] = 1;
    } else {
      for (int32_t j : succ[k]) {
        cnt[k] = sat_add(cnt[k], cnt[j]);
        len[k] = sat_add(len[k], sat_add(len[j], cnt[j]));
      }
    }
  }
  int64_t slots = 0, total_len = 0;
  for (int32_t k = 0; k < S; ++k)
    for (int32_t j : succ[k]) {
      slots = sat_add(slots, cnt[j]);
      total_len = sat_add(total_len, len[j]);
    }
  if (slots > PARD_MAX_PATH_SLOTS || total_len > PARD_MAX_PATH_LEN_SUM) return PARD_ERANGE;

  pard_pipeline* p = new (std::nothrow) pard_pipeline();
  if (!p) return PARD_ENOMEM;
  try {
    p->n_stages = S;
    p->bmax.assign(prof->bmax, prof->bmax + S);
    p->lat_offsets.assign(prof->lat_offsets, prof->lat_offsets + S + 1);
    p->lat_us.assign(prof->lat_us, prof->lat_us + prof->lat_offsets[S]);
    p->stage_slot_off.assign(S + 1, 0);
    p->path_off.push_back(0);
    p->local_off.resize(S);
    Enumerator en{succ, p->path_off, p->path_stage, {}};
    for (int32_t k = 0; k < S; ++k) {
      for (int32_t j : succ[k]) en.extend(j);
      p->stage_slot_off[k + 1] = (int32_t)p->path_off.size() - 1;
      int32_t b = p->stage_slot_off[k], e = p->stage_slot_off[k + 1];
      for (int32_t s = b; s <= e; ++s) p->local_off[k].push_back(p->path_off[s] - p->path_off[b]);
    }
    p->n_slots = (int32_t)p->path_off.size() - 1;
  } catch (const std::bad_alloc&) {
    delete p;
    return PARD_ENOMEM;
  }

  if (!(flags & PARD_LOAD_HOST_ONLY)) {
    /* one blob: header, then the tables, each 16-byte aligned */
    auto align16 = [](size_t x) { return (x + 15) & ~(size_t)15; };
    size_t off_bmax = align16(sizeof(PardPipeDev));
    size_t off_lato = align16(off_bmax + sizeof(int32_t) * S);
    size_t off_lat = align16(off_lato + sizeof(int64_t) * (S + 1));
    size_t off_sso = align16(off_lat + sizeof(int64_t) * p->lat_us.size());
    size_t off_po = align16(off_sso + sizeof(int32_t) * (S + 1));
    size_t off_ps = align16(off_po + sizeof(int32_t) * p->path_off.size());
    size_t total = align16(off_ps + sizeof(int32_t) * std::max<size_t>(1, p->path_stage.size()));
    int dev = -1;
    char* d = nullptr;
    if (cudaGetDevice(&dev) != cudaSuccess) { delete p; return PARD_ECUDA; }
    if (cudaMalloc((void**)&d, total) != cudaSuccess) {
      cudaGetLastError();
      delete p;
      return PARD_ENOMEM;
    }
    std::vector<char> h(total, 0);
    PardPipeDev hdr;
    hdr.n_stages = S;
    hdr.n_slots = p->n_slots;
    hdr.bmax = (const int32_t*)(d + off_bmax);
    hdr.lat_offsets = (const int64_t*)(d + off_lato);
    hdr.lat_us = (const int64_t*)(d + off_lat);
    hdr.stage_slot_off = (const int32_t*)(d + off_sso);
    hdr.path_off = (const int32_t*)(d + off_po);
    hdr.path_stage = (const int32_t*)(d + off_ps);
    memcpy(h.data(), &hdr, sizeof(hdr));
    memcpy(h.data() + off_bmax, p->bmax.data(), sizeof(int32_t) * S);
    memcpy(h.data() + off_lato, p->lat_offsets.data(), sizeof(int64_t) * (S + 1));
    memcpy(h.data() + off_lat, p->lat_us.data(), sizeof(int64_t) * p->lat_us.size());
    memcpy(h.data() + off_sso, p->stage_slot_off.data(), sizeof(int32_t) * (S + 1));
    memcpy(h.data() + off_po, p->path_off.data(), sizeof(int32_t) * p->path_off.size());
    if (!p->path_stage.empty())
      memcpy(h.data() + off_ps, p->path_stage.data(), sizeof(int32_t) * p->path_stage.size());
    if (cudaMemcpy(d, h.data(), total, cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaFree(d);
      delete p;
      return PARD_ECUDA;
    }
    p->device = dev;
    p->d_blob = d;
  }
  *out = p;
  return PARD_OK;
}

extern "C" int pard_free_pipeline(pard_pipeline_t* p) {
  if (!p) return PARD_OK;
  int rc = PARD_OK;
  if (p->d_blob) {
    int cur = -1;
    cudaGetDevice(&cur);
    if (cur != p->device) cudaSetDevice(p->device);
    if (cudaFree(p->d_blob) != cudaSuccess) rc = PARD_ECUDA;
    if (cur != p->device && cur >= 0) cudaSetDevice(cur);
  }
  delete p;
  return rc;
}

extern "C" int pard_pipeline_n_stages(const pard_pipeline_t* p, int32_t* n_stages) {
  if (!p || !n_stages) return PARD_EINVAL;
  *n_stages = p->n_stages;
  return PARD_OK;
}

extern "C" int pard_pipeline_n_slots(const pard_pipeline_t* p, int32_t* n_slots) {
  if (!p || !n_slots) return PARD_EINVAL;
  *n_slots = p->n_slots;
  return PARD_OK;
}

extern "C" int pard_pipeline_paths(const pard_pipeline_t* p, int32_t stage, int32_t* n_paths,
                                   int32_t* slot_base, const int32_t** path_offsets,
                                   const int32_t** path_stage_ids) {
  if (!p || !n_paths || !slot_base || !path_offsets || !path_stage_ids) return PARD_EINVAL;
  if (stage < 0 || stage >= p->n_stages) return PARD_ERANGE;
  int32_t b = p->stage_slot_off[stage];
  *n_paths = p->stage_slot_off[stage + 1] - b;
  *slot_base = b;
  *path_offsets = p->local_off[stage].data();
  *path_stage_ids = p->path_stage.data() + p->path_off[b];
  return PARD_OK;
}

extern "C" const char* pard_strerror(int status) {
  switch (status) {
    case PARD_OK: return "ok";
    case PARD_EINVAL: return "invalid argument";
    case PARD_ECYCLE: return "stage graph has a cycle";
    case PARD_ERANGE: return "value outside the supported range";
    case PARD_ENOMEM: return "allocation failed";
    case PARD_EWORKSPACE: return "workspace too small";
    case PARD_ETIMEOUT: return "device-side wait ran out";
    case PARD_ECUDA: return "CUDA runtime call failed";
    case PARD_EDATA: return "device found out-of-range request or state data";
    case PARD_ESTATIC: return "problem exceeds the built-in scratch of pard_plan_static";
    default: return "unknown status";
  }
}
