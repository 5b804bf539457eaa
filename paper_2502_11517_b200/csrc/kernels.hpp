// Host-callable launchers of the CUDA kernels.  Each returns the cudaError_t of its launch.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace pasta {

struct PoolView;   // device_common.cuh

struct PlanHeader {            // host copy of the plan's header words
  int32_t w[32];
};

// Raises a kernel's dynamic shared-memory limit once per device of the process (the attribute belongs to the device's
// context, so a second pool on another GPU needs it again).  `done` holds one bit per device ordinal.
inline cudaError_t raise_smem_limit(const void *kernel, int bytes, uint64_t *done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && ((*done >> dev) & 1)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64) *done |= 1ull << dev;
  return cudaSuccess;
}

// Launches `kernel` so that it may start before the kernel ahead of it in the stream has drained (see
// grid_dependency_wait in device_common.cuh); with overlap switched off (pasta_debug_set_launch_overlap) an ordinary launch.
bool launch_overlap_enabled();
void set_launch_overlap(bool on);
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = launch_overlap_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// K1: copies the new tokens of `layer_count` layers into their slots.  slots: device, 2 words per token.
cudaError_t launch_kv_append(const PoolView &pv, const int32_t *slots, int32_t n_tok, int32_t layer_begin,
                             int32_t layer_count, const void *k_new, const void *v_new, cudaStream_t st);
// inverse of K1 for one layer: gathers the listed slots into dense [n_tok, Hkv, D] arrays
cudaError_t launch_kv_read(const PoolView &pv, const int32_t *slots, int32_t n_tok, int32_t layer,
                           void *k_out, void *v_out, cudaStream_t st);
// K1 with rotary embedding of K by position id (pos: device array, or NULL for consecutive ids pos0, pos0 + 1, ...)
cudaError_t launch_kv_append_rope(const PoolView &pv, const int32_t *slots, const int32_t *pos, int32_t pos0, int32_t n_tok,
                                  int32_t layer_begin, int32_t layer_count, const void *k_new, const void *v_new,
                                  double theta, cudaStream_t st);
// rotates the step's queries in place by their tokens' position ids
cudaError_t launch_rope_queries(const PoolView &pv, const int32_t *pos, int32_t n, int32_t layer_count, void *q, double theta,
                                cudaStream_t st);
// K3: warp-shuffle pass for requests the tensor-core kernel does not take (other head sizes, too many rows or streams)
cudaError_t launch_attn_warp(const PoolView &pv, const PlanHeader &h, int32_t layer_begin, int32_t layer_count,
                             const void *q, float scale_log2, cudaStream_t st);
// K2: tensor-core pass over all streams of a request whose stacked queries fit 128 rows (head_dim 128 only).  Rows of
// units the plan marks final go straight to out / lse (the layout launch_merge writes), all others to the partial rows.
cudaError_t launch_attn_tensor(const PoolView &pv, const PlanHeader &h, int32_t layer_begin, int32_t layer_count,
                               const void *q, float scale_log2, void *out, float *lse, bool out_bf16, cudaStream_t st);
bool tensor_path_available();       // false while the tensor-core kernel is compiled out
// test kernel: a bounded wait that runs out (one warp, PoolView::wait_limit cycles), reported as PASTA_ERR_TIMEOUT
cudaError_t launch_wait_expiry(const PoolView &pv, cudaStream_t st);
// measurement kernels: read `bytes` of device memory and do nothing with them (mode 0: vector loads, 1: bulk copies
// into shared memory, whole 64 KB chunks only, 2: the same with every 8 KB piece taken from a scattered place); sink: 8 bytes of device memory; status: the pool's status word
cudaError_t launch_stream_read(const void *src, size_t bytes, int mode, void *sink, int32_t *status, int sm_count,
                               cudaStream_t st);
// K4: log-sum-exp merge of all partial rows of every (query, head)
// False when every row of the step leaves the tensor-core kernel as the output (all its units final, nothing on the
// warp path): the merge then has nothing to do and is not launched.  A plan with shared units keeps its merge launch,
// which also puts their counter back to zero.
inline bool plan_needs_merge(const PlanHeader &h) { return h.w[PH_N_PARTIAL] > 0 || h.w[PH_N_DUNITS] > 0; }
// out: device fp32 [layer_count, n, Hq, D], or bf16 of the same shape when out_bf16
cudaError_t launch_merge(const PoolView &pv, const PlanHeader &h, int32_t layer_count, void *out, float *lse,
                         cudaStream_t st, bool out_bf16 = false);

}  // namespace pasta
