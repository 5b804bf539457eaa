// K1 (KV append), its inverse (read-back), K3 (warp-shuffle attention pass) and K4 (log-sum-exp merge).
#include <algorithm>
#include "device_common.cuh"
#include "kernels.hpp"

#include <cmath>

#include <atomic>

namespace pasta {

static std::atomic<bool> g_launch_overlap{true};
bool launch_overlap_enabled() { return g_launch_overlap.load(std::memory_order_relaxed); }
void set_launch_overlap(bool on) { g_launch_overlap.store(on, std::memory_order_relaxed); }


// =============================================================================================
// K1: KV append.  One thread moves one 16-byte chunk (8 bf16) of K or V of one token.
// =============================================================================================
__global__ void kv_append_kernel(PoolView pv, const int32_t *__restrict__ slots, int32_t n_tok,
                                 int32_t layer_begin, int32_t layer_count,
                                 const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new) {
  grid_launch_dependents();       // the attention kernel may set itself up meanwhile; it waits for this grid to finish
  const int chunks = pv.head_dim >> 3;
  const int64_t total = static_cast<int64_t>(layer_count) * n_tok * pv.n_kv_heads * 2 * chunks;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = static_cast<int>(idx % chunks);
  int64_t rest = idx / chunks;
  const int kv = static_cast<int>(rest & 1);
  rest >>= 1;
  const int g = static_cast<int>(rest % pv.n_kv_heads);
  rest /= pv.n_kv_heads;
  const int a = static_cast<int>(rest % n_tok);
  const int ll = static_cast<int>(rest / n_tok);
  const int page = slots[2 * a], off = slots[2 * a + 1];
  if (page < 0 || page >= pv.n_pages || off < 0 || off >= PASTA_PAGE) {
    report(pv.status, PASTA_ERR_DEVICE_CHECK);
    return;
  }
  const uint4 *src = (kv ? v_new : k_new) + ((static_cast<int64_t>(ll) * n_tok + a) * pv.n_kv_heads + g) * chunks + c;
  uint8_t *block = pv.kv_base + (layer_begin + ll) * pv.layer_stride +
                   (static_cast<int64_t>(page) * pv.n_kv_heads + g) * kv_block_bytes(pv.head_dim);
  *reinterpret_cast<uint4 *>(block + kv_chunk_offset(pv.head_dim >> 6, kv, off, c)) = __ldg(src);
}

__global__ void kv_read_kernel(PoolView pv, const int32_t *__restrict__ slots, int32_t n_tok, int32_t layer,
                               uint4 *__restrict__ k_out, uint4 *__restrict__ v_out) {
  const int chunks = pv.head_dim >> 3;
  const int64_t total = static_cast<int64_t>(n_tok) * pv.n_kv_heads * 2 * chunks;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = static_cast<int>(idx % chunks);
  int64_t rest = idx / chunks;
  const int kv = static_cast<int>(rest & 1);
  rest >>= 1;
  const int g = static_cast<int>(rest % pv.n_kv_heads);
  const int a = static_cast<int>(rest / pv.n_kv_heads);
  const int page = slots[2 * a], off = slots[2 * a + 1];
  if (page < 0 || page >= pv.n_pages || off < 0 || off >= PASTA_PAGE) {
    report(pv.status, PASTA_ERR_DEVICE_CHECK);
    return;
  }
  const uint8_t *block = pv.kv_base + layer * pv.layer_stride +
                         (static_cast<int64_t>(page) * pv.n_kv_heads + g) * kv_block_bytes(pv.head_dim);
  uint4 *dst = (kv ? v_out : k_out) + (static_cast<int64_t>(a) * pv.n_kv_heads + g) * chunks + c;
  *dst = *reinterpret_cast<const uint4 *>(block + kv_chunk_offset(pv.head_dim >> 6, kv, off, c));
}

// =============================================================================================
// K1 with rotary position embedding: K is rotated by its token's position id before it is stored
// (rotate-half form: element i pairs with element i + D/2; angle = pos * theta^(-2i/D)); V is copied.
// One thread handles the 16-byte chunk c of the low half together with chunk c of the high half.
// Angles are evaluated in double precision so that the stored bf16 keys agree with a float64 reference.
// =============================================================================================
// Sines and cosines of the 8 angles of chunk c (elements first_i .. first_i + 7 of the low half): they depend on
// the token's position only, so a thread evaluates them once and applies them to every head of the token.
__device__ __forceinline__ void rope_angles(int pos, int first_i, int D, double log2_theta, double *sn, double *cs) {
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const double ang = static_cast<double>(pos) * exp2(-2.0 * (first_i + e) / D * log2_theta);
    sincos(ang, &sn[e], &cs[e]);
  }
}

__device__ __forceinline__ void rope_apply(uint4 &lo, uint4 &hi, const double *sn, const double *cs) {
  uint32_t *l = reinterpret_cast<uint32_t *>(&lo), *h = reinterpret_cast<uint32_t *>(&hi);
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    float xl[2] = {bf16_lo(l[w]), bf16_hi(l[w])}, xh[2] = {bf16_lo(h[w]), bf16_hi(h[w])};
    float yl[2], yh[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const double c = cs[2 * w + e], s_ = sn[2 * w + e];
      yl[e] = static_cast<float>(static_cast<double>(xl[e]) * c - static_cast<double>(xh[e]) * s_);
      yh[e] = static_cast<float>(static_cast<double>(xh[e]) * c + static_cast<double>(xl[e]) * s_);
    }
    __nv_bfloat162 pl = __floats2bfloat162_rn(yl[0], yl[1]), ph = __floats2bfloat162_rn(yh[0], yh[1]);
    l[w] = *reinterpret_cast<uint32_t *>(&pl);
    h[w] = *reinterpret_cast<uint32_t *>(&ph);
  }
}

// Threads [0, n_k) rotate and store K: one thread per (layer, token, chunk pair), all kv heads of the token in turn.
// Threads [n_k, n_k + n_v) copy V: one thread per (layer, token, kv head, chunk pair).
__global__ void kv_append_rope_kernel(PoolView pv, const int32_t *__restrict__ slots, const int32_t *__restrict__ pos,
                                      int32_t pos0, int32_t n_tok, int32_t layer_begin, int32_t layer_count,
                                      const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new, double log2_theta) {
  grid_launch_dependents();
  const int chunks = pv.head_dim >> 3, half_chunks = chunks >> 1;
  const int64_t n_k = static_cast<int64_t>(layer_count) * n_tok * half_chunks;
  const int64_t n_v = n_k * pv.n_kv_heads;
  int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= n_k + n_v) return;
  const bool is_k = idx < n_k;
  if (!is_k) idx -= n_k;
  const int c = static_cast<int>(idx % half_chunks);
  int64_t rest = idx / half_chunks;
  int g = 0;
  if (!is_k) { g = static_cast<int>(rest % pv.n_kv_heads); rest /= pv.n_kv_heads; }
  const int a = static_cast<int>(rest % n_tok);
  const int ll = static_cast<int>(rest / n_tok);
  const int page = slots[2 * a], off = slots[2 * a + 1];
  if (page < 0 || page >= pv.n_pages || off < 0 || off >= PASTA_PAGE) {
    report(pv.status, PASTA_ERR_DEVICE_CHECK);
    return;
  }
  uint8_t *layer = pv.kv_base + (layer_begin + ll) * pv.layer_stride;
  if (is_k) {
    double sn[8], cs[8];
    rope_angles(pos ? pos[a] : pos0 + a, c * 8, pv.head_dim, log2_theta, sn, cs);
#pragma unroll 1
    for (g = 0; g < pv.n_kv_heads; ++g) {
      const uint4 *src = k_new + ((static_cast<int64_t>(ll) * n_tok + a) * pv.n_kv_heads + g) * chunks;
      uint4 lo = __ldg(src + c), hi = __ldg(src + c + half_chunks);
      rope_apply(lo, hi, sn, cs);
      uint8_t *block = layer + (static_cast<int64_t>(page) * pv.n_kv_heads + g) * kv_block_bytes(pv.head_dim);
      *reinterpret_cast<uint4 *>(block + kv_chunk_offset(pv.head_dim >> 6, 0, off, c)) = lo;
      *reinterpret_cast<uint4 *>(block + kv_chunk_offset(pv.head_dim >> 6, 0, off, c + half_chunks)) = hi;
    }
  } else {
    const uint4 *src = v_new + ((static_cast<int64_t>(ll) * n_tok + a) * pv.n_kv_heads + g) * chunks;
    uint8_t *block = layer + (static_cast<int64_t>(page) * pv.n_kv_heads + g) * kv_block_bytes(pv.head_dim);
    *reinterpret_cast<uint4 *>(block + kv_chunk_offset(pv.head_dim >> 6, 1, off, c)) = __ldg(src + c);
    *reinterpret_cast<uint4 *>(block + kv_chunk_offset(pv.head_dim >> 6, 1, off, c + half_chunks)) = __ldg(src + c + half_chunks);
  }
}

// rotates the step's queries in place: q [layer_count, n, Hq, D], positions from the plan; one thread per
// (layer, query, chunk pair), all heads of the query in turn
__global__ void rope_queries_kernel(const int32_t *__restrict__ pos, int32_t n, int32_t n_q_heads, int32_t D,
                                    int32_t layer_count, uint4 *__restrict__ q, double log2_theta) {
  grid_launch_dependents();
  const int chunks = D >> 3, half_chunks = chunks >> 1;
  const int64_t total = static_cast<int64_t>(layer_count) * n * half_chunks;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = static_cast<int>(idx % half_chunks);
  const int64_t tok = idx / half_chunks;                 // (layer, query)
  const int i = static_cast<int>(tok % n);
  double sn[8], cs[8];
  rope_angles(pos[i], c * 8, D, log2_theta, sn, cs);
#pragma unroll 1
  for (int h = 0; h < n_q_heads; ++h) {
    uint4 *row = q + (tok * n_q_heads + h) * chunks;
    uint4 lo = row[c], hi = row[c + half_chunks];
    rope_apply(lo, hi, sn, cs);
    row[c] = lo;
    row[c + half_chunks] = hi;
  }
}

// =============================================================================================
// Test kernel for the bounded waits: one warp waits, with the pool's limit, for an mbarrier phase that nobody
// completes, reports PASTA_ERR_TIMEOUT when the wait gives up (it always does) and returns.
// =============================================================================================
__global__ void wait_expiry_kernel(PoolView pv) {
  __shared__ __align__(8) uint64_t bar_mem;
  const uint32_t bar = smem_u32(&bar_mem);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    mbar_init_fence();
  }
  __syncwarp();
  const bool done = __all_sync(0xffffffffu, mbar_wait_bounded(bar, 0, pv.wait_limit));
  if (!done && threadIdx.x == 0) report(pv.status, PASTA_ERR_TIMEOUT);
}

// =============================================================================================
// Read-only streaming kernels for measurements: what this GPU delivers to a kernel that only reads, by the two
// mechanisms the attention kernels use.  Neither computes anything worth naming.
//   bulk:   one CTA per SM, a 3-stage ring of 64 KB filled by 8 KB bulk copies (the tensor-core kernel's producer
//           without its consumers); chunk c goes to CTA c % grid; its 8 KB pieces are consecutive, or scattered.
//   vector: 16-byte loads, eight in flight per thread, folded into one word so that they cannot be dropped.
// =============================================================================================
constexpr int R_STAGES = 3, R_STAGE_BYTES = 65536, R_PIECE = 8192;

__global__ void __launch_bounds__(32, 1)
stream_read_bulk_kernel(const uint8_t *__restrict__ src, int64_t n_chunks, int scattered, unsigned long long *sink,
                        int32_t *status) {
  extern __shared__ __align__(1024) uint8_t r_smem[];
  __shared__ __align__(8) uint64_t bars[R_STAGES];
  const int lane = threadIdx.x;
  const uint32_t base = smem_u32(r_smem), bar = smem_u32(bars);
  if (lane == 0) {
    for (int s = 0; s < R_STAGES; ++s) mbar_init(bar + 8 * s, 1);
    mbar_init_fence();
  }
  fence_proxy_async();
  __syncwarp();
  const int64_t mine = n_chunks > blockIdx.x ? (n_chunks - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const uint64_t n_pieces = static_cast<uint64_t>(n_chunks) * (R_STAGE_BYTES / R_PIECE);
  auto issue = [&](int64_t k) {
    const int s = static_cast<int>(k % R_STAGES);
    const uint64_t piece = static_cast<uint64_t>(blockIdx.x + k * gridDim.x) * (R_STAGE_BYTES / R_PIECE) + lane;
    // scattered: every 8 KB piece comes from a place far from its neighbours' (its number times a large prime,
    // modulo the number of pieces), the way the pages of a stream lie in a pool that hands out pages in random order
    const uint64_t from_piece = scattered ? (piece * 2654435761ull) % n_pieces : piece;   // a prime: one-to-one
    if (lane == 0) mbar_expect_tx(bar + 8 * s, R_STAGE_BYTES);
    __syncwarp();
    if (lane < R_STAGE_BYTES / R_PIECE)
      bulk_g2s(base + s * R_STAGE_BYTES + lane * R_PIECE, src + from_piece * R_PIECE, R_PIECE, bar + 8 * s);
  };
  for (int64_t k = 0; k < R_STAGES && k < mine; ++k) issue(k);
  int64_t landed = 0;
  bool ok = true;
  for (int64_t k = 0; k < mine; ++k) {
    if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar + 8 * (k % R_STAGES), (k / R_STAGES) & 1))) { ok = false; break; }
    landed = k + 1;
    if (k + R_STAGES < mine) issue(k + R_STAGES);
  }
  if (!ok) {
    if (lane == 0) report(status, PASTA_ERR_TIMEOUT);
    for (int64_t k = landed; k < mine && k < landed + R_STAGES; ++k)      // copies still in flight
      mbar_wait_bounded(bar + 8 * (k % R_STAGES), (k / R_STAGES) & 1);
    return;
  }
  if (lane == 0 && mine > 0) atomicAdd(sink, static_cast<unsigned long long>(r_smem[0]));
}

__global__ void __launch_bounds__(256)
stream_read_vector_kernel(const uint4 *__restrict__ src, int64_t n_vec, unsigned long long *sink) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  for (; i + 7 * stride < n_vec; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __ldcs(src + i + j * stride);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
  }
  for (; i < n_vec; i += stride) { const uint4 v = __ldcs(src + i); acc ^= v.x ^ v.y ^ v.z ^ v.w; }
  if (acc == 0x9e3779b9u) atomicAdd(sink, 1ull);        // practically never: the loads have to be made to find out
}

cudaError_t launch_stream_read(const void *src, size_t bytes, int mode, void *sink, int32_t *status, int sm_count,
                               cudaStream_t st) {
  if (mode == 1 || mode == 2) {
    static uint64_t prepared = 0;
    cudaError_t e = raise_smem_limit(reinterpret_cast<const void *>(stream_read_bulk_kernel), R_STAGES * R_STAGE_BYTES, &prepared);
    if (e != cudaSuccess) return e;
    const int64_t n_chunks = static_cast<int64_t>(bytes / R_STAGE_BYTES);
    if (n_chunks == 0) return cudaSuccess;
    stream_read_bulk_kernel<<<sm_count, 32, R_STAGES * R_STAGE_BYTES, st>>>(
        static_cast<const uint8_t *>(src), n_chunks, mode == 2, static_cast<unsigned long long *>(sink), status);
  } else {
    const int64_t n_vec = static_cast<int64_t>(bytes / 16);
    if (n_vec == 0) return cudaSuccess;
    stream_read_vector_kernel<<<sm_count * 8, 256, 0, st>>>(static_cast<const uint4 *>(src), n_vec,
                                                           static_cast<unsigned long long *>(sink));
  }
  return cudaGetLastError();
}

cudaError_t launch_wait_expiry(const PoolView &pv, cudaStream_t st) {
  wait_expiry_kernel<<<1, 32, 0, st>>>(pv);
  return cudaGetLastError();
}

cudaError_t launch_kv_append_rope(const PoolView &pv, const int32_t *slots, const int32_t *pos, int32_t pos0, int32_t n_tok,
                                  int32_t layer_begin, int32_t layer_count, const void *k_new, const void *v_new,
                                  double theta, cudaStream_t st) {
  const int64_t n_k = static_cast<int64_t>(layer_count) * n_tok * (pv.head_dim >> 4);
  const int64_t total = n_k * (1 + pv.n_kv_heads);        // K threads (all heads each) + V threads (one head each)
  if (total == 0) return cudaSuccess;
  const int threads = 128;
  kv_append_rope_kernel<<<static_cast<unsigned>((total + threads - 1) / threads), threads, 0, st>>>(
      pv, slots, pos, pos0, n_tok, layer_begin, layer_count, static_cast<const uint4 *>(k_new),
      static_cast<const uint4 *>(v_new), log2(theta));
  return cudaGetLastError();
}

cudaError_t launch_rope_queries(const PoolView &pv, const int32_t *pos, int32_t n, int32_t layer_count, void *q, double theta,
                                cudaStream_t st) {
  const int64_t total = static_cast<int64_t>(layer_count) * n * (pv.head_dim >> 4);
  if (total == 0) return cudaSuccess;
  const int threads = 128;
  rope_queries_kernel<<<static_cast<unsigned>((total + threads - 1) / threads), threads, 0, st>>>(
      pos, n, pv.n_q_heads, pv.head_dim, layer_count, static_cast<uint4 *>(q), log2(theta));
  return cudaGetLastError();
}

cudaError_t launch_kv_append(const PoolView &pv, const int32_t *slots, int32_t n_tok, int32_t layer_begin,
                             int32_t layer_count, const void *k_new, const void *v_new, cudaStream_t st) {
  const int64_t total = static_cast<int64_t>(layer_count) * n_tok * pv.n_kv_heads * 2 * (pv.head_dim >> 3);
  if (total == 0) return cudaSuccess;
  const int threads = 256;
  const int64_t blocks = (total + threads - 1) / threads;
  kv_append_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(
      pv, slots, n_tok, layer_begin, layer_count, static_cast<const uint4 *>(k_new),
      static_cast<const uint4 *>(v_new));
  return cudaGetLastError();
}

cudaError_t launch_kv_read(const PoolView &pv, const int32_t *slots, int32_t n_tok, int32_t layer,
                           void *k_out, void *v_out, cudaStream_t st) {
  const int64_t total = static_cast<int64_t>(n_tok) * pv.n_kv_heads * 2 * (pv.head_dim >> 3);
  if (total == 0) return cudaSuccess;
  const int threads = 256;
  const int64_t blocks = (total + threads - 1) / threads;
  kv_read_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(
      pv, slots, n_tok, layer, static_cast<uint4 *>(k_out), static_cast<uint4 *>(v_out));
  return cudaGetLastError();
}

// =============================================================================================
// K3: warp-shuffle pass.  One warp = one w-unit = (query, kv head, <= chunk tokens of one stream).
// Pages are bulk-copied into a per-warp ring of shared-memory stages.  Scores: lane (r, s) holds
// token r of the page and half s of the head dim, halves are combined with one shuffle; the
// running maximum is a shuffle reduction over the 16 tokens.  P.V: every lane owns D/32 output
// elements for each of the G heads.
// =============================================================================================
constexpr int W_WARPS = 1;            // one warp per block: the block scheduler balances the units
constexpr int W_STAGES = 2;

template <int D, int G>
struct WarpSmem {
  static constexpr int BLOCK = D * 64;
  static constexpr int Q_BYTES = G * D * 4;
  static constexpr int P_BYTES = 16 * G * 4;
  static constexpr int BAR_BYTES = 64;
  static constexpr int PER_WARP = W_STAGES * BLOCK + Q_BYTES + P_BYTES + BAR_BYTES;
  static constexpr int TOTAL = PER_WARP * W_WARPS;
};

template <int D, int G>
__global__ void __launch_bounds__(W_WARPS * 32)
attn_warp_kernel(PoolView pv, int32_t off_wunit, int32_t off_pages, int32_t n_wunits, int32_t t_rows,
                 int32_t n_queries, int32_t layer_begin, int32_t layer_count,
                 const __nv_bfloat16 *__restrict__ q, float scale_log2) {
  using S = WarpSmem<D, G>;
  constexpr int NH = D / 64;
  constexpr int E = D / 32;            // output elements per lane
  constexpr int CH = D / 16;           // 16-byte chunks of a K row handled by one lane
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  grid_dependency_wait();         // the kernel ahead in the stream (append or tensor-core pass) has completed
  grid_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t gw = static_cast<int64_t>(blockIdx.x) * W_WARPS + warp;
  if (gw >= static_cast<int64_t>(n_wunits) * layer_count) return;
  const int ll = static_cast<int>(gw / n_wunits);
  const int u = static_cast<int>(gw % n_wunits);

  uint8_t *base = smem_raw + warp * S::PER_WARP;
  uint8_t *stages = base;
  float *q_s = reinterpret_cast<float *>(base + W_STAGES * S::BLOCK);
  float *p_s = reinterpret_cast<float *>(base + W_STAGES * S::BLOCK + S::Q_BYTES);
  const uint32_t bar0 = smem_u32(base + W_STAGES * S::BLOCK + S::Q_BYTES + S::P_BYTES);

  const int4 U = *reinterpret_cast<const int4 *>(pv.plan + off_wunit + u * PW_WORDS);   // query, kv head, page offset, tokens
  const int qi = U.x, g = U.y, n_tok = U.w;
  const int32_t *pg = pv.plan + off_pages + U.z;
  const int n_pg = (n_tok + PASTA_PAGE - 1) / PASTA_PAGE;
  const uint8_t *kv_layer = pv.kv_base + (layer_begin + ll) * pv.layer_stride;

  if (lane == 0) {
    for (int s = 0; s < W_STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
    mbar_init_fence();
    fence_proxy_async();
  }
  // page ids of the unit's first 64 pages live in registers (lane i: pages i and i + 32), so that refilling a
  // stage never waits for global memory
  const int my_pg0 = lane < n_pg ? pg[lane] : 0;
  const int my_pg1 = lane + 32 < n_pg ? pg[lane + 32] : 0;
  __syncwarp();
  auto issue = [&](int i) {
    int page = i < 32 ? __shfl_sync(0xffffffffu, my_pg0, i) : i < 64 ? __shfl_sync(0xffffffffu, my_pg1, i - 32) : pg[i];
    if (lane == 0) {
      if (page < 0 || page >= pv.n_pages) { report(pv.status, PASTA_ERR_DEVICE_CHECK); page = 0; }
      const int s = i % W_STAGES;
      fence_proxy_async();            // the lanes' reads of this stage (ordered by __syncwarp) precede the refill
      mbar_expect_tx(bar0 + 8 * s, S::BLOCK);
      bulk_g2s(smem_u32(stages + s * S::BLOCK),
               kv_layer + (static_cast<int64_t>(page) * pv.n_kv_heads + g) * S::BLOCK, S::BLOCK, bar0 + 8 * s);
    }
  };
  for (int i = 0; i < W_STAGES && i < n_pg; ++i) issue(i);
  // the G query rows of this kv head, pre-multiplied by scale * log2(e) (overlaps the first copies)
  {
    const __nv_bfloat162 *qsrc = reinterpret_cast<const __nv_bfloat162 *>(
        q + ((static_cast<int64_t>(ll) * n_queries + qi) * pv.n_q_heads + g * G) * D);
#pragma unroll
    for (int i = lane; i < G * D / 2; i += 32) {
      const float2 f = __bfloat1622float2(qsrc[i]);
      q_s[2 * i] = f.x * scale_log2;
      q_s[2 * i + 1] = f.y * scale_log2;
    }
  }
  __syncwarp();

  float m[G], l[G], o[G][E];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) o[h][e] = 0.f;
  }
  const int r = lane & 15, sub = lane >> 4;
  int issued = min(W_STAGES, n_pg), consumed = 0;
  bool ok = true;

  for (int i = 0; i < n_pg; ++i) {
    const int s = i % W_STAGES;
    // the lanes poll on their own: the warp gives up as one, or the shuffles below would meet half a warp
    if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar0 + 8 * s, (i / W_STAGES) & 1, pv.wait_limit))) { ok = false; consumed = i; break; }
    const uint8_t *sp = stages + s * S::BLOCK;
    const int nv = min(PASTA_PAGE, n_tok - i * PASTA_PAGE);

    float acc[G];
#pragma unroll
    for (int h = 0; h < G; ++h) acc[h] = 0.f;
#pragma unroll
    for (int cc = 0; cc < CH; ++cc) {
      const int c = sub * CH + cc;
      const uint4 kk = *reinterpret_cast<const uint4 *>(sp + kv_chunk_offset(NH, 0, r, c));
      const float k0 = bf16_lo(kk.x), k1 = bf16_hi(kk.x), k2 = bf16_lo(kk.y), k3 = bf16_hi(kk.y);
      const float k4 = bf16_lo(kk.z), k5 = bf16_hi(kk.z), k6 = bf16_lo(kk.w), k7 = bf16_hi(kk.w);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float4 qa = *reinterpret_cast<const float4 *>(q_s + h * D + c * 8);
        const float4 qb = *reinterpret_cast<const float4 *>(q_s + h * D + c * 8 + 4);
        acc[h] = fmaf(k0, qa.x, acc[h]); acc[h] = fmaf(k1, qa.y, acc[h]);
        acc[h] = fmaf(k2, qa.z, acc[h]); acc[h] = fmaf(k3, qa.w, acc[h]);
        acc[h] = fmaf(k4, qb.x, acc[h]); acc[h] = fmaf(k5, qb.y, acc[h]);
        acc[h] = fmaf(k6, qb.z, acc[h]); acc[h] = fmaf(k7, qb.w, acc[h]);
      }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
      float sc = acc[h] + __shfl_xor_sync(0xffffffffu, acc[h], 16);
      if (r >= nv) sc = -INFINITY;
      float mx = sc;
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      const float m_new = fmaxf(m[h], mx);          // finite: nv >= 1
      const float corr = fast_exp2(m[h] - m_new);   // 0 on the first page
      const float pj = fast_exp2(sc - m_new);       // 0 for masked rows
      l[h] = l[h] * corr + (sub == 0 ? pj : 0.f);
      m[h] = m_new;
#pragma unroll
      for (int e = 0; e < E; ++e) o[h][e] *= corr;
      if (sub == 0) p_s[r * G + h] = pj;
    }
    __syncwarp();
    {
      const int c = (lane * E) >> 3;                // chunk that holds this lane's elements
      const int within = ((lane * E) & 7) * 2;      // byte offset inside the chunk
      for (int r2 = 0; r2 < nv; ++r2) {
        const uint8_t *vp = sp + kv_chunk_offset(NH, 1, r2, c) + within;
        float v[E];
        if constexpr (E == 4) {
          const uint2 vv = *reinterpret_cast<const uint2 *>(vp);
          v[0] = bf16_lo(vv.x); v[1] = bf16_hi(vv.x); v[2] = bf16_lo(vv.y); v[3] = bf16_hi(vv.y);
        } else {
          const uint32_t vv = *reinterpret_cast<const uint32_t *>(vp);
          v[0] = bf16_lo(vv); v[1] = bf16_hi(vv);
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float ph = p_s[r2 * G + h];
#pragma unroll
          for (int e = 0; e < E; ++e) o[h][e] = fmaf(ph, v[e], o[h][e]);
        }
      }
    }
    __syncwarp();                                   // every lane is done with stage s and with p_s
    if (i + W_STAGES < n_pg) { issue(i + W_STAGES); ++issued; }
  }

  if (!ok) {
    // give up: report, then wait (bounded) for the copies still in flight before leaving
    if (lane == 0) report(pv.status, PASTA_ERR_TIMEOUT);
    for (int j = consumed; j < issued; ++j) mbar_wait_bounded(bar0 + 8 * (j % W_STAGES), (j / W_STAGES) & 1);
    return;
  }

  const int64_t row0 = static_cast<int64_t>(ll) * pv.rows_per_layer + t_rows + static_cast<int64_t>(u) * G;
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float lt = l[h];
    lt += __shfl_xor_sync(0xffffffffu, lt, 16);
    lt += __shfl_xor_sync(0xffffffffu, lt, 8);
    lt += __shfl_xor_sync(0xffffffffu, lt, 4);
    lt += __shfl_xor_sync(0xffffffffu, lt, 2);
    lt += __shfl_xor_sync(0xffffffffu, lt, 1);
    if (lane == 0) pv.part_ml[row0 + h] = make_float2(m[h], lt);
    float *dst = pv.part_o + (row0 + h) * D + lane * E;
    if constexpr (E == 4) *reinterpret_cast<float4 *>(dst) = make_float4(o[h][0], o[h][1], o[h][2], o[h][3]);
    else *reinterpret_cast<float2 *>(dst) = make_float2(o[h][0], o[h][1]);
  }
}

template <int D, int G>
static cudaError_t launch_warp_t(const PoolView &pv, const PlanHeader &h, int32_t layer_begin, int32_t layer_count,
                                 const void *q, float scale_log2, cudaStream_t st) {
  using S = WarpSmem<D, G>;
  static uint64_t prepared = 0;
  {
    cudaError_t e = raise_smem_limit(reinterpret_cast<const void *>(attn_warp_kernel<D, G>), S::TOTAL, &prepared);
    if (e != cudaSuccess) return e;
  }
  const int64_t warps = static_cast<int64_t>(h.w[PH_N_WUNITS]) * layer_count;
  if (warps == 0) return cudaSuccess;
  const int64_t blocks = (warps + W_WARPS - 1) / W_WARPS;
  return launch_overlapped(attn_warp_kernel<D, G>, dim3(static_cast<unsigned>(blocks)), dim3(W_WARPS * 32), S::TOTAL, st, pv,
                           h.w[PH_OFF_WUNIT], h.w[PH_OFF_PAGES], h.w[PH_N_WUNITS], h.w[PH_T_ROWS], h.w[PH_N_QUERIES],
                           layer_begin, layer_count, static_cast<const __nv_bfloat16 *>(q), scale_log2);
}

cudaError_t launch_attn_warp(const PoolView &pv, const PlanHeader &h, int32_t layer_begin, int32_t layer_count,
                             const void *q, float scale_log2, cudaStream_t st) {
  const int G = pv.n_q_heads / pv.n_kv_heads;
#define PASTA_W(DD, GG) \
  if (pv.head_dim == DD && G == GG) return launch_warp_t<DD, GG>(pv, h, layer_begin, layer_count, q, scale_log2, st);
  PASTA_W(128, 1) PASTA_W(128, 2) PASTA_W(128, 4) PASTA_W(128, 8)
  PASTA_W(64, 1) PASTA_W(64, 2) PASTA_W(64, 4) PASTA_W(64, 8)
#undef PASTA_W
  return cudaErrorInvalidValue;
}

// =============================================================================================
// K4: log-sum-exp merge.  One warp per (query, head, group of layers), looping over its layers: m* = max m_i,
// out = sum_i 2^(m_i - m*) O_i / sum_i 2^(m_i - m*) l_i,  lse = ln2 * (m* + log2 of that sum).
// Which partial rows belong to a (query, head) is the same for every layer, so the look-ups in the plan are made
// once per warp, and the (m, l) pairs of the next layer are fetched while this layer's outputs are summed.
// =============================================================================================
template <bool kOutBf16>
__global__ void __launch_bounds__(256)
merge_kernel(PoolView pv, int32_t n_queries, int32_t layer_count, int32_t off_query, int32_t off_trange,
             int32_t off_tunit, int32_t off_drange, int32_t off_dunit, int32_t t_rows, int32_t layers_per_warp,
             void *__restrict__ out_raw, float *__restrict__ lse) {
  grid_dependency_wait();         // every partial row has been written
  // the tensor-core kernel of this launch group is over: its counter of shared units starts from zero next time
  if (blockIdx.x == 0 && threadIdx.x == 0) pv.status[PASTA_STATUS_TAIL_COUNTER] = 0;
  const int D = pv.head_dim, Hq = pv.n_q_heads, G = Hq / pv.n_kv_heads;
  const int64_t gw = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t per_group = static_cast<int64_t>(n_queries) * Hq;
  const int ll_begin = static_cast<int>(gw / per_group) * layers_per_warp;
  if (ll_begin >= layer_count) return;
  const int ll_end = min(layer_count, ll_begin + layers_per_warp);
  const int h = static_cast<int>(gw % Hq);
  const int n = static_cast<int>((gw % per_group) / Hq);
  const int g = h / G, hl = h % G;
  const int32_t *Q = pv.plan + off_query + n * PQ_WORDS;
  const int treq = Q[PQ_TREQ], tidx = Q[PQ_TIDX], w0 = Q[PQ_WUNIT0], nw = Q[PQ_NW];
  int tb = 0, nt = 0, db = 0, nd = 0;
  if (treq >= 0) {
    tb = pv.plan[off_trange + (treq * pv.n_kv_heads + g) * 2];
    nt = pv.plan[off_trange + (treq * pv.n_kv_heads + g) * 2 + 1] - tb;
    db = pv.plan[off_drange + (treq * pv.n_kv_heads + g) * 2];
    nd = pv.plan[off_drange + (treq * pv.n_kv_heads + g) * 2 + 1] - db;
  }
  if (nw == 0 && nt + nd == 1) {            // a final unit has written this pair's result itself
    const int32_t *rec = nt ? pv.plan + off_tunit + tb * PU_WORDS : pv.plan + off_dunit + db * PU_WORDS;
    if (rec[PU_FINAL]) return;
  }
  const int total = nt + nd + nw;
  auto row_of = [&](int i) -> int64_t {     // within one layer: assigned units, shared units, warp-shuffle pieces
    if (i < nt) return pv.plan[off_tunit + (tb + i) * PU_WORDS + PU_ROW_BASE] + tidx * G + hl;
    if (i < nt + nd) return pv.plan[off_dunit + (db + i - nt) * PU_WORDS + PU_ROW_BASE] + tidx * G + hl;
    return t_rows + static_cast<int64_t>(w0 + g * nw + (i - nt - nd)) * G + hl;
  };
  const int E = D >> 5;                    // 4 or 2 elements per lane
  // lane i looks up partial row i (and i + 32, ...) once; the weighted sum then takes rows and weights from the
  // lanes' registers, so that only the loads of the partial outputs are left in the loop
  const int64_t first_row = lane < total ? row_of(lane) : 0;
  float2 next_ml = make_float2(-INFINITY, 0.f);
  if (lane < total) next_ml = pv.part_ml[static_cast<int64_t>(ll_begin) * pv.rows_per_layer + first_row];
  for (int ll = ll_begin; ll < ll_end; ++ll) {
    const int64_t lbase = static_cast<int64_t>(ll) * pv.rows_per_layer;
    const float2 first_ml = next_ml;
    if (ll + 1 < ll_end && lane < total) next_ml = pv.part_ml[lbase + pv.rows_per_layer + first_row];
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float L = 0.f, mstar = -INFINITY;
    for (int base_i = 0; base_i < total; base_i += 32) {
      const int i = base_i + lane;
      int64_t my_row = lbase + first_row;
      float2 my_ml = first_ml;
      if (base_i > 0) {
        my_ml = make_float2(-INFINITY, 0.f);
        if (i < total) { my_row = lbase + row_of(i); my_ml = pv.part_ml[my_row]; }
      }
      float m_here = my_ml.y > 0.f ? my_ml.x : -INFINITY;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m_here = fmaxf(m_here, __shfl_xor_sync(0xffffffffu, m_here, o));
      if (m_here > mstar) {                  // warp-uniform: move what has been summed so far to the new maximum
        const float f = fast_exp2(mstar - m_here);    // 0 when nothing has been summed yet
        L *= f;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[e] *= f;
        mstar = m_here;
      }
      const float my_w = my_ml.y > 0.f ? fast_exp2(my_ml.x - mstar) : 0.f;
      const int cnt = min(32, total - base_i);
      for (int k = 0; k < cnt; ++k) {
        const float w = __shfl_sync(0xffffffffu, my_w, k);
        const float lk = __shfl_sync(0xffffffffu, my_ml.y, k);
        const int64_t row = __shfl_sync(0xffffffffu, my_row, k);
        if (w == 0.f) continue;              // nothing visible in that piece (warp-uniform)
        L = fmaf(w, lk, L);
        const float *src = pv.part_o + row * D + lane * E;
        if (E == 4) {
          const float4 v = *reinterpret_cast<const float4 *>(src);
          acc[0] = fmaf(w, v.x, acc[0]); acc[1] = fmaf(w, v.y, acc[1]);
          acc[2] = fmaf(w, v.z, acc[2]); acc[3] = fmaf(w, v.w, acc[3]);
        } else {
          const float2 v = *reinterpret_cast<const float2 *>(src);
          acc[0] = fmaf(w, v.x, acc[0]); acc[1] = fmaf(w, v.y, acc[1]);
        }
      }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const int64_t at = ((static_cast<int64_t>(ll) * n_queries + n) * Hq + h) * D + lane * E;
    if (kOutBf16) {
      __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(out_raw) + at;
      const __nv_bfloat162 p0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
      if (E == 4) {
        const __nv_bfloat162 p1 = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
        *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<const uint32_t *>(&p0), *reinterpret_cast<const uint32_t *>(&p1));
      } else {
        *reinterpret_cast<__nv_bfloat162 *>(dst) = p0;
      }
    } else {
      float *dst = static_cast<float *>(out_raw) + at;
      if (E == 4) *reinterpret_cast<float4 *>(dst) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
      else *reinterpret_cast<float2 *>(dst) = make_float2(acc[0] * inv, acc[1] * inv);
    }
    if (lse && lane == 0)
      lse[(static_cast<int64_t>(ll) * n_queries + n) * Hq + h] = (mstar + log2f(L)) * 0.6931471805599453f;
  }
}

cudaError_t launch_merge(const PoolView &pv, const PlanHeader &h, int32_t layer_count, void *out, float *lse,
                         cudaStream_t st, bool out_bf16) {
  const int64_t per_group = static_cast<int64_t>(h.w[PH_N_QUERIES]) * pv.n_q_heads;
  if (per_group == 0 || layer_count == 0) return cudaSuccess;
  // enough warps to fill the machine a few times over; beyond that, more layers per warp (its plan look-ups are shared)
  const int64_t want_warps = 4 * 148 * 64;
  const int64_t groups = std::min<int64_t>(layer_count, std::max<int64_t>(1, (want_warps + per_group - 1) / per_group));
  const int32_t layers_per_warp = static_cast<int32_t>((layer_count + groups - 1) / groups);
  const int64_t warps = per_group * ((layer_count + layers_per_warp - 1) / layers_per_warp);
  const int64_t blocks = (warps * 32 + 255) / 256;
  return launch_overlapped(out_bf16 ? merge_kernel<true> : merge_kernel<false>, dim3(static_cast<unsigned>(blocks)), dim3(256), 0,
                           st, pv, h.w[PH_N_QUERIES], layer_count, h.w[PH_OFF_QUERY], h.w[PH_OFF_TRANGE], h.w[PH_OFF_TUNIT],
                           h.w[PH_OFF_DRANGE], h.w[PH_OFF_DUNIT], h.w[PH_T_ROWS], layers_per_warp, out, lse);
}

}  // namespace pasta
