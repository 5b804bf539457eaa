// pasta_decode_attn_noalloc: decode attention of one layer with the split/segment partial results
// kept in a fixed device array that is part of the library image, so that the call needs no
// workspace memory from anybody and allocates nothing.
#include <atomic>

#include "device_common.cuh"
#include "kernels.hpp"

namespace pasta {
// defined in api.cu: the device view and plan header of a pool's current step (false: no valid plan / host-only)
bool pool_step_view(pasta_pool_t *pool, PoolView *pv, PlanHeader *hdr, int32_t *n_layers, int32_t *head_dim,
                    int32_t *device);
void pool_count_launches(pasta_pool_t *pool, int n);
}  // namespace pasta

using namespace pasta;

namespace {

constexpr int kMaxRows = PASTA_NOALLOC_MAX_ROWS;                   // partial rows one call may need
constexpr size_t kMlBytes = size_t(kMaxRows) * sizeof(float2);     // (m, l) per row
constexpr size_t kScratchBytes = kMlBytes + size_t(kMaxRows) * 128 * sizeof(float);

// Lives in every GPU's memory from the moment the library is loaded there until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can use:
// the device address is looked up once per device and cached here.  The look-up gives the same answer to every
// host thread, so two threads that both find the slot empty store the same value; the atomic only keeps the
// store and the loads from tearing.  The address belongs to the device's primary context and is stale once that
// context has been destroyed (cudaDeviceReset).
constexpr int kMaxDevices = 64;
std::atomic<void *> g_scratch_addr[kMaxDevices];

}  // namespace

extern "C" pasta_status_t pasta_decode_attn_noalloc(pasta_pool_t *pool, int32_t layer, const void *q, void *out,
                                                    float *lse, float scale, void *stream) {
  if (!pool) return PASTA_ERR_INVALID_ARG;
  PoolView pv;
  PlanHeader hdr;
  int32_t n_layers = 0, head_dim = 0, device = 0;
  if (!pool_step_view(pool, &pv, &hdr, &n_layers, &head_dim, &device)) return PASTA_ERR_BAD_STATE;
  if (layer < 0 || layer >= n_layers) return PASTA_ERR_INVALID_ARG;
  if (hdr.w[PH_N_QUERIES] == 0) return PASTA_OK;                   // an empty step needs no buffers, as in pasta_decode_attn
  if (!q || !out || !(scale >= 0.f)) return PASTA_ERR_INVALID_ARG;
  if (hdr.w[PH_ROWS] > kMaxRows) return PASTA_ERR_CAPACITY;       // this step needs more partial rows than the array holds
  int current = -1;
  if (cudaGetDevice(&current) != cudaSuccess || current != device || device < 0 || device >= kMaxDevices)
    return PASTA_ERR_INVALID_ARG;                                  // the pool's device must be the current one
  void *addr = g_scratch_addr[device].load(std::memory_order_acquire);
  if (!addr) {
    const cudaError_t e = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
    if (e != cudaSuccess || !addr) return PASTA_ERR_CUDA;
    g_scratch_addr[device].store(addr, std::memory_order_release);
  }
  unsigned char *scratch = static_cast<unsigned char *>(addr);
  pv.part_ml = reinterpret_cast<float2 *>(scratch);
  pv.part_o = reinterpret_cast<float *>(scratch + kMlBytes);
  pv.rows_per_layer = kMaxRows;
  // Nothing in the array has to start at zero.  Every (m, l) pair of the step is written before the merge reads
  // it.  The output part of a row is written only when the row saw at least one token (l > 0); for a row with
  // l == 0 it keeps whatever an earlier call left there, and the merge never reads it: it skips pieces of weight 0.
  const float sc = (scale == 0.f ? rsqrtf(static_cast<float>(head_dim)) : scale) * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  int launched = 0;
  if (hdr.w[PH_N_TUNITS] + hdr.w[PH_N_DUNITS] > 0) { e = launch_attn_tensor(pv, hdr, layer, 1, q, sc, out, lse, false, st); ++launched; }
  if (e == cudaSuccess && hdr.w[PH_N_WUNITS] > 0) { e = launch_attn_warp(pv, hdr, layer, 1, q, sc, st); ++launched; }
  if (e == cudaSuccess && plan_needs_merge(hdr)) { e = launch_merge(pv, hdr, 1, static_cast<float *>(out), lse, st); ++launched; }
  pool_count_launches(pool, launched);
  return e == cudaSuccess ? PASTA_OK : PASTA_ERR_CUDA;
}
