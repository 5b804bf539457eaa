// The C ABI (include/pasta.h): argument checks, the device side of a pool, uploads and launches.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "device_common.cuh"
#include "kernels.hpp"
#include "plan.hpp"
#include "pool.hpp"

using namespace pasta;

namespace {

constexpr int kStaging = 4;           // pinned upload buffers in rotation
constexpr int kHostInflight = 3;           // host-buffer steps that may be between begin and wait
constexpr size_t kSmallPlanWords = 8192;   // plans up to this size are uploaded in the caller's stream
constexpr int kProfCalls = 512;        // timed pasta_decode_attn launches kept between two profile reads
constexpr int kRunChunk = 8192;       // tokens whose slots are uploaded at once by pasta_kv_append_run
constexpr int kTailPercent = 10;      // share of the short runs' tiles that the tensor-core kernel's CTAs share out at run time
constexpr int kTailTiles = 16;        // tiles per unit of that share; runs of up to four times as many count as short
int32_t g_last_cuda_error = 0;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Derived {
  int32_t group, max_queries, max_rows, layers_per_launch;
  int64_t max_words, staging_words;
  size_t kv_bytes, layer_stride;
  size_t off_status, off_plan, off_plan2, off_run, off_ml, off_o, ws_bytes;
};

pasta_status_t derive(const pasta_pool_config_t &c, Derived *d) {
  if (c.n_layers < 1 || c.n_kv_heads < 1 || c.n_q_heads < 1 || c.n_q_heads % c.n_kv_heads) return PASTA_ERR_INVALID_ARG;
  d->group = c.n_q_heads / c.n_kv_heads;
  if (d->group != 1 && d->group != 2 && d->group != 4 && d->group != 8) return PASTA_ERR_INVALID_ARG;
  if (c.head_dim != 64 && c.head_dim != 128) return PASTA_ERR_INVALID_ARG;
  if (c.page_size != PASTA_PAGE || c.n_pages < 1) return PASTA_ERR_INVALID_ARG;
  if (c.max_requests < 1 || c.max_threads_per_request < 1 || c.max_segments_per_thread < 1) return PASTA_ERR_INVALID_ARG;
  if (c.max_step_queries < 0 || c.max_partial_rows < 0 || c.max_layers_per_launch < 0) return PASTA_ERR_INVALID_ARG;
  const int grid = 160;   // upper bound on CTAs of the tensor-core kernel, for sizing only
  d->max_queries = c.max_step_queries ? c.max_step_queries
                                      : static_cast<int32_t>(std::min<int64_t>(int64_t(c.max_requests) * 17, 1 << 20));
  // units of the shared tail, at most: its share of all tiles in pieces of kTailTiles, plus one ragged piece per run
  const int64_t tail_units = int64_t(c.n_pages) * c.n_kv_heads / PASTA_TILE_PAGES * kTailPercent / 100 / kTailTiles +
                             int64_t(c.max_requests) * c.n_kv_heads;
  const int64_t unit_rows = std::min<int64_t>(PASTA_MAX_ROWS, int64_t(c.max_threads_per_request) * d->group);
  d->max_rows = c.max_partial_rows ? c.max_partial_rows
                                   : static_cast<int32_t>(std::min<int64_t>(
                                         int64_t(d->max_queries) * c.n_q_heads * 8 + int64_t(grid) * PASTA_MAX_ROWS +
                                             tail_units * unit_rows, 1 << 28));
  d->layers_per_launch = c.max_layers_per_launch ? std::min(c.max_layers_per_launch, c.n_layers)
                                                 : std::min(c.n_layers, 8);
  const int64_t nq = d->max_queries, nr = c.max_requests;
  d->max_words = PH_WORDS + 2 * nq + PQ_WORDS * nq + PT_WORDS * nr + 2 * nr * c.n_kv_heads +
                 PU_WORDS * (nr * c.n_kv_heads + grid) + 2 * grid + PW_WORDS * (int64_t(d->max_rows) / d->group + 1) +
                 2 * int64_t(c.n_pages) + nq * std::min(PASTA_MAX_STREAMS, c.max_threads_per_request) + nq + 64 +
                 PU_WORDS * tail_units + 2 * nr * c.n_kv_heads + 8;
  d->staging_words = std::max<int64_t>(d->max_words, 2 * kRunChunk);
  d->layer_stride = size_t(c.n_pages) * c.n_kv_heads * kv_block_bytes(c.head_dim);
  d->kv_bytes = d->layer_stride * c.n_layers;
  size_t off = 0;
  d->off_status = off; off += 256;
  d->off_plan = off;   off = align_up(off + size_t(d->max_words) * 4, 256);
  d->off_plan2 = off;  off = align_up(off + size_t(d->max_words) * 4, 256);   // plans of consecutive steps alternate
  d->off_run = off;    off = align_up(off + size_t(2 * kRunChunk) * 4, 256);
  const size_t rows = size_t(d->max_rows) * d->layers_per_launch;
  d->off_ml = off;     off = align_up(off + rows * sizeof(float2), 256);
  d->off_o = off;      off = align_up(off + rows * c.head_dim * sizeof(float), 256);
  d->ws_bytes = off;
  return PASTA_OK;
}

}  // namespace

struct pasta_pool {
  pasta_pool_config_t cfg;
  Derived d;
  HostPool host;
  bool host_only;
  int sm_count = 148;
  PoolView pv{};
  int32_t *run_slots_dev = nullptr;
  int32_t *pinned[kStaging] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t pinned_free[kStaging] = {nullptr, nullptr, nullptr, nullptr};
  int next_pinned = 0;
  int32_t *status_host = nullptr;     // pinned, one word
  std::vector<StepQuery> queries;   // of the step planned last, in entry order
  std::vector<Slot> slots;          // parallel to queries
  std::vector<int32_t> plan;
  PlanHeader hdr{};
  bool plan_valid = false;
  int64_t launches = 0;
  // the plan of step i is uploaded on a stream of its own into buffer i % 2 while step i - 1 still runs
  int32_t *plan_dev[2] = {nullptr, nullptr};
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t plan_ready[2] = {nullptr, nullptr};   // recorded on copy_stream after the upload of buffer b
  cudaEvent_t work_mark[2] = {nullptr, nullptr};    // recorded on the caller's stream at the start of step i (slot i % 2)
  int64_t step_index = 0;
  int32_t tail_percent = kTailPercent, tail_tiles = kTailTiles;
  // pasta_step_host_begin / _wait: at most two steps in flight; their copies run on streams of the pool
  cudaStream_t d2h_stream = nullptr;
  // pasta_step_host_begin / _wait: up to kHostInflight steps between begin and wait; step i uses event set i % kHostInflight
  cudaEvent_t host_inputs_ready[kHostInflight] = {};       // copy_stream: k / v / q of the step are on the device
  cudaEvent_t host_attn_done[kHostInflight] = {};          // caller's stream: the step's outputs are in the staging area
  cudaEvent_t host_out_ready[kHostInflight] = {};          // d2h_stream: the outputs are in the caller's host buffer
  int host_slot_of[kHostInflight] = {};                    // staging slot used by the step with that event set
  int64_t host_submitted = 0, host_waited = 0;
  // kernel timing (pasta_profile_*): events[4 * i .. 4 * i + 3] bracket the three kernels of call i
  bool profiling = false;
  int prof_stride = 1;                  // every prof_stride-th pasta_decode_attn launch group is timed
  int64_t prof_seen = 0;                // launch groups since profiling was enabled
  std::vector<cudaEvent_t> prof_events;
  std::vector<uint8_t> prof_mask;       // per call: bit k set if kernel k was launched
  int prof_calls = 0;

  pasta_pool(const pasta_pool_config_t &c, const Derived &dd)
      : cfg(c), d(dd),
        host(c.n_pages, c.page_size, c.free_order, c.max_requests, c.max_threads_per_request,
             c.max_segments_per_thread),
        host_only((c.flags & PASTA_FLAG_HOST_ONLY) != 0) {}
};

namespace {

pasta_status_t cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int32_t>(e);
  return PASTA_ERR_CUDA;
}
#define PASTA_CUDA(call)                                  \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(e__);        \
  } while (0)

// Copies `words` int32 from host memory to `dst` on the stream through a pinned buffer of the ring.
pasta_status_t upload(pasta_pool *p, const int32_t *src, size_t words, int32_t *dst, cudaStream_t st) {
  const int b = p->next_pinned;
  p->next_pinned = (b + 1) % kStaging;
  PASTA_CUDA(cudaEventSynchronize(p->pinned_free[b]));   // the copy that last used this buffer is done
  std::memcpy(p->pinned[b], src, words * 4);
  PASTA_CUDA(cudaMemcpyAsync(dst, p->pinned[b], words * 4, cudaMemcpyHostToDevice, st));
  PASTA_CUDA(cudaEventRecord(p->pinned_free[b], st));
  return PASTA_OK;
}

PlanLimits limits_of(const pasta_pool *p) {
  PlanLimits l;
  l.n_q_heads = p->cfg.n_q_heads;
  l.n_kv_heads = p->cfg.n_kv_heads;
  l.head_dim = p->cfg.head_dim;
  l.max_queries = p->d.max_queries;
  l.max_rows = p->d.max_rows;
  l.max_words = p->d.max_words;
  l.grid = p->sm_count;
  l.tensor_path = p->cfg.head_dim == 128 && !(p->cfg.flags & PASTA_FLAG_NO_TENSOR_PATH) && tensor_path_available();
  l.tail_percent = p->tail_percent;
  l.tail_tiles = p->tail_tiles;
  return l;
}

}  // namespace

namespace pasta {
// for entry points that live in other files
bool pool_step_view(pasta_pool_t *p, PoolView *pv, PlanHeader *hdr, int32_t *n_layers, int32_t *head_dim,
                    int32_t *device) {
  if (p->host_only || !p->plan_valid) return false;
  if (p->cfg.flags & PASTA_FLAG_OUT_BF16) return false;      // that entry point writes fp32 only
  *pv = p->pv;
  *hdr = p->hdr;
  *n_layers = p->cfg.n_layers;
  *head_dim = p->cfg.head_dim;
  *device = p->cfg.device;
  return true;
}
void pool_count_launches(pasta_pool_t *p, int n) { p->launches += n; }
}  // namespace pasta

extern "C" {

int32_t pasta_last_cuda_error(void) { return g_last_cuda_error; }

pasta_status_t pasta_kv_bytes(const pasta_pool_config_t *cfg, size_t *out) {
  if (!cfg || !out) return PASTA_ERR_INVALID_ARG;
  Derived d;
  pasta_status_t s = derive(*cfg, &d);
  if (s != PASTA_OK) return s;
  *out = d.kv_bytes;
  return PASTA_OK;
}

pasta_status_t pasta_workspace_bytes(const pasta_pool_config_t *cfg, size_t *out) {
  if (!cfg || !out) return PASTA_ERR_INVALID_ARG;
  Derived d;
  pasta_status_t s = derive(*cfg, &d);
  if (s != PASTA_OK) return s;
  *out = d.ws_bytes;
  return PASTA_OK;
}

pasta_status_t pasta_pool_create(const pasta_pool_config_t *cfg, pasta_pool_t **out) {
  if (!cfg || !out) return PASTA_ERR_INVALID_ARG;
  Derived d;
  pasta_status_t s = derive(*cfg, &d);
  if (s != PASTA_OK) return s;
  if (!HostPool::valid_free_order(cfg->n_pages, cfg->free_order)) return PASTA_ERR_INVALID_ARG;
  const bool host_only = (cfg->flags & PASTA_FLAG_HOST_ONLY) != 0;
  if (!host_only) {
    if (!cfg->kv_base || cfg->kv_bytes < d.kv_bytes || (reinterpret_cast<uintptr_t>(cfg->kv_base) & 1023))
      return PASTA_ERR_INVALID_ARG;
    if (!cfg->workspace || cfg->workspace_bytes < d.ws_bytes || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255))
      return PASTA_ERR_INVALID_ARG;
  }
  pasta_pool *p = new (std::nothrow) pasta_pool(*cfg, d);
  if (!p) return PASTA_ERR_CAPACITY;
  p->cfg.free_order = nullptr;   // read during this call only
  if (!host_only) {
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, cfg->device);
    for (int i = 0; i < kStaging && e == cudaSuccess; ++i) {
      e = cudaMallocHost(reinterpret_cast<void **>(&p->pinned[i]), size_t(d.staging_words) * 4);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->pinned_free[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaMallocHost(reinterpret_cast<void **>(&p->status_host), 64);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->d2h_stream, cudaStreamNonBlocking);
    for (int b = 0; b < 2 && e == cudaSuccess; ++b) {
      e = cudaEventCreateWithFlags(&p->plan_ready[b], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->work_mark[b], cudaEventDisableTiming);
    }
    for (int b = 0; b < kHostInflight && e == cudaSuccess; ++b) {
      e = cudaEventCreateWithFlags(&p->host_inputs_ready[b], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->host_attn_done[b], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->host_out_ready[b], cudaEventDisableTiming);
    }
    uint8_t *ws = static_cast<uint8_t *>(cfg->workspace);
    if (e == cudaSuccess) e = cudaMemset(ws, 0, 256);
    // stale bytes of a page's unused tail are multiplied by zero weights, so they must be finite
    if (e == cudaSuccess) e = cudaMemset(cfg->kv_base, 0, d.kv_bytes);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
      pasta_pool_destroy(p);
      return cuda_fail(e);
    }
    p->pv.kv_base = static_cast<uint8_t *>(cfg->kv_base);
    p->pv.layer_stride = static_cast<int64_t>(d.layer_stride);
    p->pv.n_pages = cfg->n_pages;
    p->pv.n_q_heads = cfg->n_q_heads;
    p->pv.n_kv_heads = cfg->n_kv_heads;
    p->pv.head_dim = cfg->head_dim;
    p->pv.status = reinterpret_cast<int32_t *>(ws + d.off_status);
    p->plan_dev[0] = reinterpret_cast<int32_t *>(ws + d.off_plan);
    p->plan_dev[1] = reinterpret_cast<int32_t *>(ws + d.off_plan2);
    p->pv.plan = p->plan_dev[0];
    p->run_slots_dev = reinterpret_cast<int32_t *>(ws + d.off_run);
    p->pv.part_ml = reinterpret_cast<float2 *>(ws + d.off_ml);
    p->pv.part_o = reinterpret_cast<float *>(ws + d.off_o);
    p->pv.rows_per_layer = d.max_rows;
    p->pv.wait_limit = kWaitLimitCycles;
    p->pv.debug_hold = 0;
  }
  *out = p;
  return PASTA_OK;
}

pasta_status_t pasta_pool_destroy(pasta_pool_t *p) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  for (int i = 0; i < kStaging; ++i) {
    if (p->pinned_free[i]) { cudaEventSynchronize(p->pinned_free[i]); cudaEventDestroy(p->pinned_free[i]); }
    if (p->pinned[i]) cudaFreeHost(p->pinned[i]);
  }
  if (p->status_host) cudaFreeHost(p->status_host);
  if (p->copy_stream) { cudaStreamSynchronize(p->copy_stream); cudaStreamDestroy(p->copy_stream); }
  if (p->d2h_stream) { cudaStreamSynchronize(p->d2h_stream); cudaStreamDestroy(p->d2h_stream); }
  for (int b = 0; b < 2; ++b) {
    if (p->plan_ready[b]) cudaEventDestroy(p->plan_ready[b]);
    if (p->work_mark[b]) cudaEventDestroy(p->work_mark[b]);
  }
  for (int b = 0; b < kHostInflight; ++b) {
    if (p->host_inputs_ready[b]) cudaEventDestroy(p->host_inputs_ready[b]);
    if (p->host_attn_done[b]) cudaEventDestroy(p->host_attn_done[b]);
    if (p->host_out_ready[b]) cudaEventDestroy(p->host_out_ready[b]);
  }
  for (cudaEvent_t e : p->prof_events) if (e) cudaEventDestroy(e);
  delete p;
  return PASTA_OK;
}

pasta_status_t pasta_request_begin(pasta_pool_t *p, int32_t *out_req) {
  if (!p || !out_req) return PASTA_ERR_INVALID_ARG;
  return p->host.request_begin(out_req);
}

pasta_status_t pasta_request_end(pasta_pool_t *p, int32_t req) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  pasta_status_t s = p->host.request_end(req);
  if (s == PASTA_OK) p->plan_valid = false;
  return s;
}

pasta_status_t pasta_thread_spawn(pasta_pool_t *p, int32_t req, int32_t *out_thread) {
  if (!p || !out_thread) return PASTA_ERR_INVALID_ARG;
  return p->host.thread_spawn(req, 0, 0, out_thread);
}

pasta_status_t pasta_thread_spawn_predicted(pasta_pool_t *p, int32_t req, int32_t predicted_tokens, int32_t pending,
                                            int32_t *out_thread) {
  if (!p || !out_thread) return PASTA_ERR_INVALID_ARG;
  return p->host.thread_spawn(req, predicted_tokens, pending, out_thread);
}

pasta_status_t pasta_step_positions(pasta_pool_t *p, int32_t *out_pos, int32_t capacity_entries) {
  if (!p || !out_pos) return PASTA_ERR_INVALID_ARG;
  if (!p->plan_valid) return PASTA_ERR_BAD_STATE;
  const int32_t n = p->hdr.w[PH_N_QUERIES];
  if (capacity_entries < n) return PASTA_ERR_CAPACITY;
  std::memcpy(out_pos, p->plan.data() + p->hdr.w[PH_OFF_QPOS], size_t(n) * 4);
  return PASTA_OK;
}

pasta_status_t pasta_kv_append_rope(pasta_pool_t *p, int32_t layer_begin, int32_t layer_count, const void *k_new,
                                    const void *v_new, float theta, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only || !p->plan_valid) return PASTA_ERR_BAD_STATE;
  if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > p->cfg.n_layers || !(theta > 1.f))
    return PASTA_ERR_INVALID_ARG;
  const int32_t n_app = p->hdr.w[PH_N_APPEND];
  if (n_app == 0 || layer_count == 0) return PASTA_OK;
  if (!k_new || !v_new) return PASTA_ERR_INVALID_ARG;
  PASTA_CUDA(launch_kv_append_rope(p->pv, p->pv.plan + p->hdr.w[PH_OFF_APPEND], p->pv.plan + p->hdr.w[PH_OFF_APOS], 0, n_app,
                                   layer_begin, layer_count, k_new, v_new, theta, static_cast<cudaStream_t>(stream)));
  p->launches += 1;
  return PASTA_OK;
}

pasta_status_t pasta_rope_queries(pasta_pool_t *p, int32_t layer_count, void *q, float theta, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only || !p->plan_valid) return PASTA_ERR_BAD_STATE;
  if (layer_count < 0 || layer_count > p->cfg.n_layers || !(theta > 1.f)) return PASTA_ERR_INVALID_ARG;
  const int32_t n = p->hdr.w[PH_N_QUERIES];
  if (n == 0 || layer_count == 0) return PASTA_OK;
  if (!q) return PASTA_ERR_INVALID_ARG;
  PASTA_CUDA(launch_rope_queries(p->pv, p->pv.plan + p->hdr.w[PH_OFF_QPOS], n, layer_count, q, theta,
                                 static_cast<cudaStream_t>(stream)));
  p->launches += 1;
  return PASTA_OK;
}

pasta_status_t pasta_thread_finish(pasta_pool_t *p, int32_t req, int32_t thread) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  return p->host.thread_finish(req, thread);
}

pasta_status_t pasta_sync_merge(pasta_pool_t *p, int32_t req, int32_t n_threads, const int32_t *thread_ids) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  return p->host.sync_merge(req, n_threads, thread_ids);
}

pasta_status_t pasta_step_begin(pasta_pool_t *p, int32_t n, const int32_t *req_ids, const int32_t *thread_ids,
                                const int32_t *n_new, void *stream) {
  if (!p || n < 0 || (n > 0 && (!req_ids || !thread_ids))) return PASTA_ERR_INVALID_ARG;
  std::vector<StepEntry> entries(n);
  int64_t n_queries = 0;
  for (int32_t i = 0; i < n; ++i) {
    entries[i] = StepEntry{req_ids[i], thread_ids[i], n_new ? n_new[i] : 1};
    if (entries[i].n_new < 0) return PASTA_ERR_INVALID_ARG;
    n_queries += std::max(1, entries[i].n_new);
  }
  if (n_queries > p->d.max_queries) return PASTA_ERR_CAPACITY;
  std::vector<Slot> slots;
  std::vector<StepQuery> queries;
  std::vector<StepUndo> undo;
  pasta_status_t s = p->host.reserve_step(entries, &queries, &slots, &undo);
  if (s != PASTA_OK) return s;
  p->plan_valid = false;
  p->queries.swap(queries);
  p->slots.swap(slots);
  s = build_plan(p->host, p->queries, p->slots, limits_of(p), &p->plan);
  if (s != PASTA_OK) {           // the step does not fit the pool's capacities: take the reservation back
    p->host.undo_step(undo);
    p->queries.clear();
    p->slots.clear();
    return s;
  }
  std::memcpy(p->hdr.w, p->plan.data(), sizeof(p->hdr.w));
  if (!p->host_only) {
    // Buffer b = i % 2 was last read by the kernels of step i - 2.  Everything the caller had enqueued when step
    // i - 1 began (that is, up to step i - 2) is covered by work_mark[(i - 1) % 2]; the upload waits for that mark
    // only, so it runs while step i - 1 is still executing, and the caller's stream waits for the upload.
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t i = p->step_index++;
    const int b = static_cast<int>(i & 1);
    PASTA_CUDA(cudaEventRecord(p->work_mark[b], st));
    if (p->plan.size() <= kSmallPlanWords) {
      // a small plan is copied in the caller's stream: it is ordered behind the kernels of step i - 2 there anyway,
      // and a few microseconds of copy are not worth two more events and two stream waits on the host
      s = upload(p, p->plan.data(), p->plan.size(), p->plan_dev[b], st);
      if (s != PASTA_OK) return s;
    } else {
      if (i >= 1) PASTA_CUDA(cudaStreamWaitEvent(p->copy_stream, p->work_mark[b ^ 1], 0));
      s = upload(p, p->plan.data(), p->plan.size(), p->plan_dev[b], p->copy_stream);
      if (s != PASTA_OK) return s;
      PASTA_CUDA(cudaEventRecord(p->plan_ready[b], p->copy_stream));
      PASTA_CUDA(cudaStreamWaitEvent(st, p->plan_ready[b], 0));
    }
    p->pv.plan = p->plan_dev[b];
  }
  p->plan_valid = true;
  return PASTA_OK;
}

pasta_status_t pasta_step_slots(pasta_pool_t *p, int32_t *out_slots, int32_t capacity_entries) {
  if (!p || !out_slots) return PASTA_ERR_INVALID_ARG;
  if (capacity_entries < static_cast<int32_t>(p->slots.size())) return PASTA_ERR_CAPACITY;
  for (size_t i = 0; i < p->slots.size(); ++i) {
    out_slots[2 * i] = p->slots[i].page;
    out_slots[2 * i + 1] = p->slots[i].offset;
  }
  return PASTA_OK;
}

pasta_status_t pasta_kv_append(pasta_pool_t *p, int32_t layer_begin, int32_t layer_count, const void *k_new,
                               const void *v_new, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only || !p->plan_valid) return PASTA_ERR_BAD_STATE;
  if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > p->cfg.n_layers) return PASTA_ERR_INVALID_ARG;
  const int32_t n_app = p->hdr.w[PH_N_APPEND];
  if (n_app == 0 || layer_count == 0) return PASTA_OK;
  if (!k_new || !v_new) return PASTA_ERR_INVALID_ARG;
  PASTA_CUDA(launch_kv_append(p->pv, p->pv.plan + p->hdr.w[PH_OFF_APPEND], n_app, layer_begin, layer_count, k_new, v_new,
                              static_cast<cudaStream_t>(stream)));
  p->launches += 1;
  return PASTA_OK;
}

pasta_status_t pasta_decode_attn(pasta_pool_t *p, int32_t layer_begin, int32_t layer_count, const void *q, void *out,
                                 float *lse, float scale, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only || !p->plan_valid) return PASTA_ERR_BAD_STATE;
  if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > p->cfg.n_layers) return PASTA_ERR_INVALID_ARG;
  const int32_t n = p->hdr.w[PH_N_QUERIES];
  if (n == 0 || layer_count == 0) return PASTA_OK;
  if (!q || !out || !(scale >= 0.f)) return PASTA_ERR_INVALID_ARG;
  const float sc = (scale == 0.f ? 1.0f / std::sqrt(static_cast<float>(p->cfg.head_dim)) : scale) * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t q_layer = size_t(n) * p->cfg.n_q_heads * p->cfg.head_dim;
  for (int32_t done = 0; done < layer_count; done += p->d.layers_per_launch) {
    const int32_t cnt = std::min(p->d.layers_per_launch, layer_count - done);
    const uint16_t *qg = static_cast<const uint16_t *>(q) + size_t(done) * q_layer;
    const bool out_bf16 = (p->cfg.flags & PASTA_FLAG_OUT_BF16) != 0;
    void *og = static_cast<uint8_t *>(out) + size_t(done) * q_layer * (out_bf16 ? 2 : 4);
    float *lg = lse ? lse + size_t(done) * n * p->cfg.n_q_heads : nullptr;
    const bool timed = p->profiling && p->prof_calls < kProfCalls && (p->prof_seen++ % p->prof_stride) == 0;
    cudaEvent_t *ev = timed ? &p->prof_events[4 * p->prof_calls] : nullptr;
    uint8_t mask = 0;
    if (timed) PASTA_CUDA(cudaEventRecord(ev[0], st));
    if (p->hdr.w[PH_N_TUNITS] + p->hdr.w[PH_N_DUNITS] > 0) {
      PASTA_CUDA(launch_attn_tensor(p->pv, p->hdr, layer_begin + done, cnt, qg, sc, og, lg, out_bf16, st));
      p->launches += 1;
      mask |= 1;
    }
    if (timed) PASTA_CUDA(cudaEventRecord(ev[1], st));
    if (p->hdr.w[PH_N_WUNITS] > 0) {
      PASTA_CUDA(launch_attn_warp(p->pv, p->hdr, layer_begin + done, cnt, qg, sc, st));
      p->launches += 1;
      mask |= 2;
    }
    if (timed) PASTA_CUDA(cudaEventRecord(ev[2], st));
    if (plan_needs_merge(p->hdr)) {
      PASTA_CUDA(launch_merge(p->pv, p->hdr, cnt, og, lg, st, out_bf16));
      p->launches += 1;
      mask |= 4;
    }
    if (timed) {
      PASTA_CUDA(cudaEventRecord(ev[3], st));
      p->prof_mask[p->prof_calls++] = mask;
    }
  }
  return PASTA_OK;
}

static pasta_status_t append_run_impl(pasta_pool_t *p, int32_t req, int32_t thread, int32_t m, int32_t layer_begin,
                                      int32_t layer_count, const void *k, const void *v, float theta, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > p->cfg.n_layers) return PASTA_ERR_INVALID_ARG;
  if (layer_count > 0 && p->host_only) return PASTA_ERR_BAD_STATE;
  if (layer_count > 0 && m > 0 && (!k || !v)) return PASTA_ERR_INVALID_ARG;
  std::vector<Slot> slots;
  const Request *rq = p->host.request(req);
  const int32_t pos0 = (rq && thread >= 0 && thread < static_cast<int32_t>(rq->threads.size())) ? rq->threads[thread].pos_next : 0;
  // consecutive position ids are assumed below: not so while the main thread owes a jump behind a pending promise
  if (theta > 0.f && m > 1 && thread == 0 && rq && rq->threads[0].pos_skip != 0) return PASTA_ERR_BAD_STATE;
  pasta_status_t s = p->host.reserve_run(req, thread, m, &slots);
  if (s != PASTA_OK) return s;
  p->plan_valid = false;
  if (layer_count == 0 || m == 0) return PASTA_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t tok = size_t(p->cfg.n_kv_heads) * p->cfg.head_dim;      // elements per token
  std::vector<int32_t> words;
  for (int32_t begin = 0; begin < m; begin += kRunChunk) {
    const int32_t cnt = std::min(kRunChunk, m - begin);
    words.resize(size_t(cnt) * 2);
    for (int32_t i = 0; i < cnt; ++i) { words[2 * i] = slots[begin + i].page; words[2 * i + 1] = slots[begin + i].offset; }
    s = upload(p, words.data(), words.size(), p->run_slots_dev, st);
    if (s != PASTA_OK) return s;
    for (int32_t l = 0; l < layer_count; ++l) {     // the run's layers are [layer_count, m, …]: one launch per layer and chunk
      const uint16_t *kl = static_cast<const uint16_t *>(k) + (size_t(l) * m + begin) * tok;
      const uint16_t *vl = static_cast<const uint16_t *>(v) + (size_t(l) * m + begin) * tok;
      if (theta > 0.f)
        PASTA_CUDA(launch_kv_append_rope(p->pv, p->run_slots_dev, nullptr, pos0 + begin, cnt, layer_begin + l, 1, kl, vl, theta, st));
      else
        PASTA_CUDA(launch_kv_append(p->pv, p->run_slots_dev, cnt, layer_begin + l, 1, kl, vl, st));
      p->launches += 1;
    }
  }
  return PASTA_OK;
}

pasta_status_t pasta_kv_append_run(pasta_pool_t *p, int32_t req, int32_t thread, int32_t m, int32_t layer_begin,
                                   int32_t layer_count, const void *k, const void *v, void *stream) {
  return append_run_impl(p, req, thread, m, layer_begin, layer_count, k, v, 0.f, stream);
}

pasta_status_t pasta_kv_append_run_rope(pasta_pool_t *p, int32_t req, int32_t thread, int32_t m, int32_t layer_begin,
                                        int32_t layer_count, const void *k, const void *v, float theta, void *stream) {
  if (!(theta > 1.f)) return PASTA_ERR_INVALID_ARG;
  return append_run_impl(p, req, thread, m, layer_begin, layer_count, k, v, theta, stream);
}

pasta_status_t pasta_step_device(pasta_pool_t *p, int32_t n, const int32_t *req_ids, const int32_t *thread_ids,
                                 const int32_t *n_new, const void *k_new, const void *v_new, const void *q, void *out,
                                 float *lse, float scale, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  pasta_status_t s = pasta_step_begin(p, n, req_ids, thread_ids, n_new, stream);
  if (s != PASTA_OK) return s;
  s = pasta_kv_append(p, 0, p->cfg.n_layers, k_new, v_new, stream);
  if (s != PASTA_OK) return s;
  return pasta_decode_attn(p, 0, p->cfg.n_layers, q, out, lse, scale, stream);
}

pasta_status_t pasta_step_host_bytes(pasta_pool_t *p, int32_t n, size_t *out) {
  if (!p || !out || n < 0) return PASTA_ERR_INVALID_ARG;
  const size_t L = p->cfg.n_layers, d = p->cfg.head_dim;
  const size_t kv = align_up(L * n * p->cfg.n_kv_heads * d * 2, 256);
  const size_t qb = align_up(L * n * p->cfg.n_q_heads * d * 2, 256);
  const size_t ob = align_up(L * n * p->cfg.n_q_heads * d * 4, 256);
  *out = 2 * kv + qb + ob;
  return PASTA_OK;
}

pasta_status_t pasta_step_host_begin(pasta_pool_t *p, int32_t n, const int32_t *req_ids, const int32_t *thread_ids,
                                     const int32_t *n_new, const void *k_new, const void *v_new, const void *q, void *out,
                                     void *staging, size_t staging_bytes, float scale, void *stream) {
  if (!p || !q || !out || !staging) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  size_t need = 0;
  pasta_status_t s = pasta_step_host_bytes(p, n, &need);
  if (s != PASTA_OK) return s;
  if (staging_bytes < need || (reinterpret_cast<uintptr_t>(staging) & 255)) return PASTA_ERR_INVALID_ARG;
  // A staging area of twice (three times) the size holds two (three) steps: the inputs of this step then travel while
  // the kernels of the steps before still read theirs.  Two steps may be in flight in any case (with one slot the
  // copies wait until the step before has left the area), three when the area holds three.
  const int n_slots = static_cast<int>(std::min<size_t>(kHostInflight, staging_bytes / need));
  if (p->host_submitted - p->host_waited >= std::max(2, n_slots)) return PASTA_ERR_BAD_STATE;   // no room for another step
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  size_t n_app = static_cast<size_t>(n);
  if (n_new) {
    n_app = 0;
    for (int32_t i = 0; i < n; ++i) {
      if (n_new[i] < 0 || n_new[i] > 1) return PASTA_ERR_INVALID_ARG;   // the staging layout is one query per entry
      n_app += static_cast<size_t>(n_new[i]);
    }
  }
  if (n_app > 0 && (!k_new || !v_new)) return PASTA_ERR_INVALID_ARG;
  const int64_t i = p->host_submitted;
  const int e = static_cast<int>(i % kHostInflight);
  const int slot = static_cast<int>(i % n_slots);
  const size_t L = p->cfg.n_layers, d = p->cfg.head_dim;
  const size_t kv_full = align_up(L * n * p->cfg.n_kv_heads * d * 2, 256);
  const size_t kv_bytes = L * n_app * p->cfg.n_kv_heads * d * 2;
  const size_t q_bytes = L * n * p->cfg.n_q_heads * d * 2;
  uint8_t *base = static_cast<uint8_t *>(staging) + size_t(slot) * need;
  uint8_t *k_dev = base, *v_dev = base + kv_full, *q_dev = base + 2 * kv_full;
  uint8_t *o_dev = q_dev + align_up(q_bytes, 256);
  // the input copies go first, on the pool's copy stream: the host plans the step while they are in flight.  A step
  // still in flight that uses the same slot is done with it once its outputs have reached the host.
  for (int64_t j = p->host_waited; j < i; ++j)
    if (p->host_slot_of[j % kHostInflight] == slot)
      PASTA_CUDA(cudaStreamWaitEvent(p->copy_stream, p->host_out_ready[j % kHostInflight], 0));
  if (n_app > 0) {
    PASTA_CUDA(cudaMemcpyAsync(k_dev, k_new, kv_bytes, cudaMemcpyHostToDevice, p->copy_stream));
    PASTA_CUDA(cudaMemcpyAsync(v_dev, v_new, kv_bytes, cudaMemcpyHostToDevice, p->copy_stream));
  }
  PASTA_CUDA(cudaMemcpyAsync(q_dev, q, q_bytes, cudaMemcpyHostToDevice, p->copy_stream));
  PASTA_CUDA(cudaEventRecord(p->host_inputs_ready[e], p->copy_stream));
  s = pasta_step_begin(p, n, req_ids, thread_ids, n_new, stream);
  if (s != PASTA_OK) return s;
  PASTA_CUDA(cudaStreamWaitEvent(st, p->host_inputs_ready[e], 0));
  s = pasta_kv_append(p, 0, p->cfg.n_layers, k_dev, v_dev, stream);
  if (s != PASTA_OK) return s;
  s = pasta_decode_attn(p, 0, p->cfg.n_layers, q_dev, o_dev, nullptr, scale, stream);
  if (s != PASTA_OK) return s;
  const size_t out_bytes = (p->cfg.flags & PASTA_FLAG_OUT_BF16) ? q_bytes : q_bytes * 2;
  PASTA_CUDA(cudaEventRecord(p->host_attn_done[e], st));
  PASTA_CUDA(cudaStreamWaitEvent(p->d2h_stream, p->host_attn_done[e], 0));
  PASTA_CUDA(cudaMemcpyAsync(out, o_dev, out_bytes, cudaMemcpyDeviceToHost, p->d2h_stream));
  PASTA_CUDA(cudaEventRecord(p->host_out_ready[e], p->d2h_stream));
  p->host_slot_of[e] = slot;
  p->host_submitted = i + 1;
  return PASTA_OK;
}

pasta_status_t pasta_step_host_wait(pasta_pool_t *p) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only || p->host_waited == p->host_submitted) return PASTA_ERR_BAD_STATE;
  PASTA_CUDA(cudaEventSynchronize(p->host_out_ready[p->host_waited % kHostInflight]));
  p->host_waited += 1;
  return PASTA_OK;
}

pasta_status_t pasta_step_host(pasta_pool_t *p, int32_t n, const int32_t *req_ids, const int32_t *thread_ids,
                               const int32_t *n_new, const void *k_new, const void *v_new, const void *q, void *out,
                               void *staging, size_t staging_bytes, float scale, void *stream) {
  if (p && p->host_submitted != p->host_waited) return PASTA_ERR_BAD_STATE;     // a pasta_step_host_begin is outstanding
  pasta_status_t s = pasta_step_host_begin(p, n, req_ids, thread_ids, n_new, k_new, v_new, q, out, staging, staging_bytes,
                                           scale, stream);
  if (s != PASTA_OK) return s;
  return pasta_step_host_wait(p);
}

pasta_status_t pasta_kv_read(pasta_pool_t *p, int32_t layer, int32_t req, int32_t stream_id, int32_t start, int32_t m,
                             void *k_out, void *v_out, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  const Request *r = p->host.request(req);
  if (!r || layer < 0 || layer >= p->cfg.n_layers || stream_id < 0 || stream_id >= static_cast<int32_t>(r->streams.size()))
    return PASTA_ERR_INVALID_ARG;
  const Stream &sm = r->streams[stream_id];
  if (start < 0 || m < 0 || start + m > sm.len) return PASTA_ERR_INVALID_ARG;
  if (m == 0) return PASTA_OK;
  if (!k_out || !v_out) return PASTA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t tok = size_t(p->cfg.n_kv_heads) * p->cfg.head_dim;
  std::vector<int32_t> words;
  for (int32_t begin = 0; begin < m; begin += kRunChunk) {
    const int32_t cnt = std::min(kRunChunk, m - begin);
    words.resize(size_t(cnt) * 2);
    for (int32_t i = 0; i < cnt; ++i) {
      const int32_t t = start + begin + i;
      words[2 * i] = sm.pages[t / PASTA_PAGE];
      words[2 * i + 1] = t % PASTA_PAGE;
    }
    pasta_status_t s = upload(p, words.data(), words.size(), p->run_slots_dev, st);
    if (s != PASTA_OK) return s;
    PASTA_CUDA(launch_kv_read(p->pv, p->run_slots_dev, cnt, layer, static_cast<uint16_t *>(k_out) + size_t(begin) * tok,
                              static_cast<uint16_t *>(v_out) + size_t(begin) * tok, st));
    p->launches += 1;
  }
  return PASTA_OK;
}

static pasta_status_t copy_words(const std::vector<int32_t> &w, int32_t *host_buf, size_t capacity, size_t *needed) {
  if (!needed) return PASTA_ERR_INVALID_ARG;
  *needed = w.size();
  if (host_buf && capacity >= w.size()) std::memcpy(host_buf, w.data(), w.size() * 4);
  return PASTA_OK;
}

pasta_status_t pasta_pool_dump(pasta_pool_t *p, int32_t *host_buf, size_t capacity_words, size_t *needed) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  std::vector<int32_t> w;
  p->host.dump(&w);
  return copy_words(w, host_buf, capacity_words, needed);
}

pasta_status_t pasta_plan_dump(pasta_pool_t *p, int32_t *host_buf, size_t capacity_words, size_t *needed) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (!p->plan_valid) return PASTA_ERR_BAD_STATE;
  return copy_words(p->plan, host_buf, capacity_words, needed);
}

pasta_status_t pasta_pool_status(pasta_pool_t *p, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  PASTA_CUDA(cudaMemcpyAsync(p->status_host, p->pv.status, 4, cudaMemcpyDeviceToHost, st));
  PASTA_CUDA(cudaMemsetAsync(p->pv.status, 0, 4, st));
  PASTA_CUDA(cudaStreamSynchronize(st));
  return *p->status_host;
}

pasta_status_t pasta_profile_enable(pasta_pool_t *p, int32_t on) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  if (on && p->prof_events.empty()) {
    p->prof_events.resize(4 * kProfCalls, nullptr);
    p->prof_mask.assign(kProfCalls, 0);
    for (cudaEvent_t &e : p->prof_events) PASTA_CUDA(cudaEventCreate(&e));
  }
  if (on < 0) return PASTA_ERR_INVALID_ARG;
  p->profiling = on != 0;
  p->prof_stride = on > 0 ? on : 1;
  p->prof_seen = 0;
  p->prof_calls = 0;
  return PASTA_OK;
}

pasta_status_t pasta_profile_read(pasta_pool_t *p, double *out_ms, int64_t *out_launches) {
  if (!p || !out_ms || !out_launches) return PASTA_ERR_INVALID_ARG;
  for (int k = 0; k < 3; ++k) { out_ms[k] = 0; out_launches[k] = 0; }
  for (int i = 0; i < p->prof_calls; ++i) {
    cudaEvent_t *ev = &p->prof_events[4 * i];
    PASTA_CUDA(cudaEventSynchronize(ev[3]));
    for (int k = 0; k < 3; ++k) {
      if (!(p->prof_mask[i] & (1 << k))) continue;
      float ms = 0;
      PASTA_CUDA(cudaEventElapsedTime(&ms, ev[k], ev[k + 1]));
      out_ms[k] += ms;
      out_launches[k] += 1;
    }
  }
  p->prof_calls = 0;
  return PASTA_OK;
}

pasta_status_t pasta_debug_set_wait_limit(pasta_pool_t *p, int64_t cycles) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  p->pv.wait_limit = cycles > 0 ? static_cast<long long>(cycles) : kWaitLimitCycles;
  return PASTA_OK;
}

pasta_status_t pasta_debug_stream_read(pasta_pool_t *p, const void *src, size_t bytes, int32_t mode, void *stream) {
  if (!p || mode < 0 || mode > 2) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  if (!src) { src = p->cfg.kv_base; bytes = p->d.kv_bytes; }
  if (reinterpret_cast<uintptr_t>(src) & 15) return PASTA_ERR_INVALID_ARG;
  void *sink = reinterpret_cast<uint8_t *>(p->pv.status) + 64;      // inside the 256 status bytes of the workspace
  PASTA_CUDA(launch_stream_read(src, bytes, mode, sink, p->pv.status, p->sm_count, static_cast<cudaStream_t>(stream)));
  p->launches += 1;
  return PASTA_OK;
}

pasta_status_t pasta_debug_set_tail(pasta_pool_t *p, int32_t percent, int32_t tiles) {
  if (!p || percent < 0 || percent > 50 || tiles < 2 || tiles > 1024) return PASTA_ERR_INVALID_ARG;
  p->tail_percent = percent;
  p->tail_tiles = tiles;
  return PASTA_OK;
}

void pasta_debug_set_launch_overlap(int32_t on) { set_launch_overlap(on != 0); }

pasta_status_t pasta_debug_hold_roles(pasta_pool_t *p, int32_t role_mask) {
  if (!p || role_mask < 0 || role_mask > 31) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  p->pv.debug_hold = role_mask;
  return PASTA_OK;
}

pasta_status_t pasta_debug_wait_expiry(pasta_pool_t *p, void *stream) {
  if (!p) return PASTA_ERR_INVALID_ARG;
  if (p->host_only) return PASTA_ERR_BAD_STATE;
  PASTA_CUDA(launch_wait_expiry(p->pv, static_cast<cudaStream_t>(stream)));
  p->launches += 1;
  return PASTA_OK;
}

pasta_status_t pasta_launch_count(pasta_pool_t *p, int64_t *out) {
  if (!p || !out) return PASTA_ERR_INVALID_ARG;
  *out = p->launches;
  return PASTA_OK;
}

}  // extern "C"
