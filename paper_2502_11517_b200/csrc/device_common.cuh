// Device-side helpers shared by the kernels: pool layout, mbarrier / bulk-copy wrappers, bounded waits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/pasta.h"
#include "pasta_plan.h"

namespace pasta {

// ---------------------------------------------------------------------------------------------
// Layout of one (page, kv head) block of the pool: K and V of 16 tokens, D*64 bytes.
//
//   block = [token group j: 2][K, V: 2][64-element half of the head dim: D/64][8 rows x 128 bytes]
//
// Each 1024-byte atom holds 8 tokens x 64 bf16; inside it the 16-byte chunk c of row r sits at
// chunk position c ^ r (the 128-byte swizzle the tensor core reads), so that one bulk copy of a
// block lands in shared memory ready to be used as an MMA operand: K as a K-major operand with
// rows = tokens, V as an MN-major operand with the head dim along N.  The same swizzle makes
// "one token per lane" reads of shared memory bank-conflict free in the warp-shuffle kernel.
// ---------------------------------------------------------------------------------------------
__host__ __device__ constexpr int kv_block_bytes(int head_dim) { return head_dim * 64; }

// byte offset, inside a block, of the 16-byte chunk `c` (8 elements) of token row `r` (0..15);
// kv = 0 for K, 1 for V; NH = head_dim / 64
__device__ __forceinline__ int kv_chunk_offset(int NH, int kv, int r, int c) {
  const int j = r >> 3, r8 = r & 7, half = c >> 3, c8 = c & 7;
  return (((j * 2 + kv) * NH + half) << 10) + (r8 << 7) + ((c8 ^ r8) << 4);
}

struct PoolView {
  uint8_t *kv_base;
  int64_t layer_stride;      // bytes between layers
  int32_t n_pages, n_q_heads, n_kv_heads, head_dim;
  int32_t *status;           // device status word
  const int32_t *plan;       // device copy of the step plan
  float2 *part_ml;           // partial (m, l) per row; m in log2 units of the scaled score
  float *part_o;             // partial unnormalised outputs [row][D]
  int64_t rows_per_layer;    // stride of the partial arrays between layers of one launch
  long long wait_limit;      // SM cycles a role waits for another role before it gives up (kWaitLimitCycles by default)
  int32_t debug_hold;        // test hook, 0 in normal use: bit r set = role r of the tensor-core kernel never starts
};

__device__ __forceinline__ void report(int32_t *status, int32_t code) { atomicMax(status, code); }
// The status word is the first of 64 words the library keeps for itself.  Word 8 counts the shared units the CTAs of
// the tensor-core kernel have taken in the current launch (the merge that follows puts it back to zero); words 16-17
// are the sink of the read-only measurement kernels.
#define PASTA_STATUS_TAIL_COUNTER 8

// Overlap of consecutive launches of a step (programmatic dependent launch).  A kernel launched with launch_overlapped()
// may start while the kernel before it in the stream is still running, once every CTA of that kernel has called
// grid_launch_dependents() or has exited; it must call grid_dependency_wait(), in every thread and before its first
// access to anything the earlier kernel reads or writes, which returns when the earlier kernel has completed and its
// writes are visible.  What runs before that call (barrier set-up, TMEM allocation, the launch itself) is hidden behind
// the earlier kernel's last CTAs.  Each kernel waits before it lets its own successor go, so that the completion of a
// kernel implies that of all its predecessors.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Default upper bound of every wait inside a kernel, in SM clock cycles (about 1.5 s at 2 GHz).  Waits of one role
// for another take the pool's limit (PoolView::wait_limit, this value unless a test shortened it); waits for the
// hardware to finish what the CTA itself started (bulk copies, MMAs in flight when a role gives up) always take
// this constant: they end on their own.
constexpr long long kWaitLimitCycles = 3000000000ll;

// Waits for the phase with the given parity to complete, for at most `limit` cycles.
// Returns false when the wait was given up (the caller then reports PASTA_ERR_TIMEOUT and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long limit = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}

// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
// Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace pasta
