// Comparison layout: the paper's own (Section 3 "Efficiency", Fig. 2b/2c).  One dense, token-granular pool per
// response, filled in decode order so that the threads' tokens interleave, and one boolean mask row per thread over
// the pool's slots.  Attention is what a generic masked attention does with that: every query walks the whole pool
// and the mask decides, slot by slot, what counts.  Nothing is shared between the threads of a response and nothing
// is skipped, which is the point of the comparison with the paged pool and its per-stream visible lengths.
//
// Three plain CUDA-core kernels (this is a baseline, not the product path): append (copy the new rows, set their mask
// bits), attention (one warp per query, kv head and range of slots: 32 slots at a time staged in shared memory,
// masked online softmax, fp32), merge of the ranges' partial results.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "../../include/pasta.h"

namespace {

constexpr int kTile = 32;            // slots staged at a time, one per lane for the scores
constexpr int kMaxNew = 64;          // tokens one append call takes

struct NewRows { int32_t row[kMaxNew]; };

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// k_pool, v_pool: [max_slots][Hkv * D] bf16; mask, own: [rows][mask_stride] bytes.  Token i of the call goes to slot
// slot0 + i and becomes visible to mask row rows.row[i] (the thread that decoded it), which also owns it.
__global__ void dense_append_kernel(uint4 *k_pool, uint4 *v_pool, uint8_t *mask, uint8_t *own, int64_t mask_stride,
                                    int32_t slot0, int32_t n_new, NewRows rows, const uint4 *k_new, const uint4 *v_new,
                                    int32_t chunks_per_token) {
  const int64_t total = static_cast<int64_t>(n_new) * chunks_per_token;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int i = static_cast<int>(idx / chunks_per_token);
  const int64_t dst = static_cast<int64_t>(slot0 + i) * chunks_per_token + idx % chunks_per_token;
  k_pool[dst] = k_new[idx];
  v_pool[dst] = v_new[idx];
  if (idx % chunks_per_token == 0) {
    mask[rows.row[i] * mask_stride + slot0 + i] = 1;
    own[rows.row[i] * mask_stride + slot0 + i] = 1;
  }
}

// One warp per (query, kv head, range).  Scores: lane = slot of the tile, the key row read from padded shared memory.
// Output: lane owns D / 32 elements of each of the G heads; the weights travel by shuffle.
template <int D, int G>
__global__ void __launch_bounds__(64)
dense_mask_attn_kernel(const __nv_bfloat16 *__restrict__ k_pool, const __nv_bfloat16 *__restrict__ v_pool,
                       const uint8_t *__restrict__ mask, int64_t mask_stride, const int32_t *__restrict__ mask_row,
                       const __nv_bfloat16 *__restrict__ q, float2 *part_ml, float *part_o, int32_t n_queries,
                       int32_t n_slots, int32_t n_kv_heads, int32_t n_ranges, int32_t range_len, float scale_log2) {
  constexpr int E = D / 32;
  constexpr int ROW = D / 2 + 1;                    // 32-bit words per staged row: odd, so lanes hit different banks
  __shared__ uint32_t k_s[2][kTile * ROW];
  __shared__ uint32_t v_s[2][kTile * (D / 2)];
  __shared__ float q_s[2][G * D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t unit = static_cast<int64_t>(blockIdx.x) * 2 + warp;
  const int64_t n_units = static_cast<int64_t>(n_queries) * n_kv_heads * n_ranges;
  if (unit >= n_units) return;
  const int range = static_cast<int>(unit % n_ranges);
  const int g = static_cast<int>((unit / n_ranges) % n_kv_heads);
  const int qi = static_cast<int>(unit / n_ranges / n_kv_heads);
  const int Hq = n_kv_heads * G;
  const uint8_t *mrow = mask + mask_row[qi] * mask_stride;
  for (int i = lane; i < G * D; i += 32)
    q_s[warp][i] = __bfloat162float(q[(static_cast<int64_t>(qi) * Hq + g * G) * D + i]) * scale_log2;
  __syncwarp();
  float m[G], l[G], o[G][E];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) o[h][e] = 0.f;
  }
  const int begin = range * range_len, end = min(n_slots, begin + range_len);
  const int64_t row_elems = static_cast<int64_t>(n_kv_heads) * D;
  for (int t0 = begin; t0 < end; t0 += kTile) {
    const int nv = min(kTile, end - t0);
    // stage the tile's K and V rows of this kv head: 16-byte loads, a row's chunks on consecutive lanes
    for (int i = lane; i < nv * (D / 8); i += 32) {
      const int r = i / (D / 8), c = i % (D / 8);
      const uint4 kk = *reinterpret_cast<const uint4 *>(k_pool + (t0 + r) * row_elems + g * D + c * 8);
      const uint4 vv = *reinterpret_cast<const uint4 *>(v_pool + (t0 + r) * row_elems + g * D + c * 8);
      uint32_t *kd = &k_s[warp][r * ROW + c * 4];
      kd[0] = kk.x; kd[1] = kk.y; kd[2] = kk.z; kd[3] = kk.w;
      *reinterpret_cast<uint4 *>(&v_s[warp][r * (D / 2) + c * 4]) = vv;
    }
    __syncwarp();
    const bool seen = lane < nv && mrow[t0 + lane] != 0;
    float s[G];
#pragma unroll
    for (int h = 0; h < G; ++h) s[h] = 0.f;
    if (lane < nv) {
      for (int w = 0; w < D / 2; ++w) {
        const uint32_t kk = k_s[warp][lane * ROW + w];
        const float k0 = __uint_as_float(kk << 16), k1 = __uint_as_float(kk & 0xffff0000u);
#pragma unroll
        for (int h = 0; h < G; ++h) s[h] = fmaf(k0, q_s[warp][h * D + 2 * w], fmaf(k1, q_s[warp][h * D + 2 * w + 1], s[h]));
      }
    }
    float p[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float sc = seen ? s[h] : -INFINITY;
      float mx = sc;
#pragma unroll
      for (int d2 = 16; d2 > 0; d2 >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d2));
      const float m_new = fmaxf(m[h], mx);
      const float corr = m_new == -INFINITY ? 1.f : ex2(m[h] - m_new);     // nothing seen so far: nothing to move
      p[h] = m_new == -INFINITY ? 0.f : ex2(sc - m_new);
      float ps = p[h];
#pragma unroll
      for (int d2 = 16; d2 > 0; d2 >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, d2);
      l[h] = l[h] * corr + ps;
      m[h] = m_new;
#pragma unroll
      for (int e = 0; e < E; ++e) o[h][e] *= corr;
    }
    for (int r = 0; r < nv; ++r) {
      float vv[E];
      if constexpr (E == 4) {
        const uint2 w2 = *reinterpret_cast<const uint2 *>(&v_s[warp][r * (D / 2) + lane * 2]);
        vv[0] = __uint_as_float(w2.x << 16); vv[1] = __uint_as_float(w2.x & 0xffff0000u);
        vv[2] = __uint_as_float(w2.y << 16); vv[3] = __uint_as_float(w2.y & 0xffff0000u);
      } else {
        const uint32_t w1 = v_s[warp][r * (D / 2) + lane];
        vv[0] = __uint_as_float(w1 << 16); vv[1] = __uint_as_float(w1 & 0xffff0000u);
      }
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float ph = __shfl_sync(0xffffffffu, p[h], r);
#pragma unroll
        for (int e = 0; e < E; ++e) o[h][e] = fmaf(ph, vv[e], o[h][e]);
      }
    }
    __syncwarp();
  }
#pragma unroll
  for (int h = 0; h < G; ++h) {
    const int64_t row = (static_cast<int64_t>(qi) * Hq + g * G + h) * n_ranges + range;
    if (lane == 0) part_ml[row] = make_float2(m[h], l[h]);
#pragma unroll
    for (int e = 0; e < E; ++e) part_o[row * D + lane * E + e] = o[h][e];
  }
}

// one warp per (query, head): folds the ranges' partial rows
__global__ void dense_mask_merge_kernel(const float2 *part_ml, const float *part_o, float *out, float *lse, int32_t n_rows,
                                        int32_t n_ranges, int32_t D) {
  const int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  float ms = -INFINITY;
  for (int r = 0; r < n_ranges; ++r) {
    const float2 ml = part_ml[row * n_ranges + r];
    if (ml.y > 0.f) ms = fmaxf(ms, ml.x);
  }
  float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
  const int E = D / 32;
  for (int r = 0; r < n_ranges; ++r) {
    const float2 ml = part_ml[row * n_ranges + r];
    if (!(ml.y > 0.f)) continue;
    const float w = ex2(ml.x - ms);
    L = fmaf(w, ml.y, L);
    for (int e = 0; e < E; ++e) acc[e] = fmaf(w, part_o[(row * n_ranges + r) * D + lane * E + e], acc[e]);
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
  for (int e = 0; e < E; ++e) out[row * D + lane * E + e] = acc[e] * inv;
  if (lse && lane == 0) lse[row] = (ms + log2f(L)) * 0.6931471805599453f;
}

int ranges_for(int64_t n_queries, int n_kv_heads, int n_slots) {
  // enough warps to fill the machine a few times; ranges are whole tiles and at least 256 slots
  const int64_t want = 148 * 64;
  int64_t r = (want + n_queries * n_kv_heads - 1) / (n_queries * n_kv_heads);
  const int64_t most = (n_slots + 255) / 256;
  r = r < 1 ? 1 : (r > most ? most : r);
  return static_cast<int>(r < 1 ? 1 : r);
}

}  // namespace

extern "C" {

pasta_status_t pasta_dense_mask_scratch_bytes(int32_t n_queries, int32_t n_slots, int32_t n_q_heads, int32_t n_kv_heads,
                                              int32_t head_dim, size_t *out) {
  if (!out || n_queries < 0 || n_slots < 0 || n_q_heads < 1 || n_kv_heads < 1 || (head_dim != 64 && head_dim != 128))
    return PASTA_ERR_INVALID_ARG;
  const size_t rows = size_t(n_queries) * n_q_heads * ranges_for(n_queries > 0 ? n_queries : 1, n_kv_heads, n_slots);
  *out = rows * (sizeof(float2) + size_t(head_dim) * sizeof(float)) + 256;
  return PASTA_OK;
}

pasta_status_t pasta_dense_append(void *k_pool, void *v_pool, uint8_t *mask, uint8_t *own, int64_t mask_stride, int32_t slot0,
                                  int32_t n_new, const int32_t *rows, const void *k_new, const void *v_new,
                                  int32_t n_kv_heads, int32_t head_dim, void *stream) {
  if (n_new == 0) return PASTA_OK;
  if (!k_pool || !v_pool || !mask || !own || !rows || !k_new || !v_new || n_new < 0 || n_new > kMaxNew || slot0 < 0 ||
      slot0 + n_new > mask_stride)
    return PASTA_ERR_INVALID_ARG;
  NewRows nr;
  for (int i = 0; i < n_new; ++i) nr.row[i] = rows[i];
  const int chunks = n_kv_heads * head_dim / 8;
  const int64_t total = static_cast<int64_t>(n_new) * chunks;
  dense_append_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<uint4 *>(k_pool), static_cast<uint4 *>(v_pool), mask, own, mask_stride, slot0, n_new, nr,
      static_cast<const uint4 *>(k_new), static_cast<const uint4 *>(v_new), chunks);
  return cudaGetLastError() == cudaSuccess ? PASTA_OK : PASTA_ERR_CUDA;
}

pasta_status_t pasta_dense_mask_attn(const void *k_pool, const void *v_pool, const uint8_t *mask, int64_t mask_stride,
                                     const int32_t *mask_row, const void *q, void *out, float *lse, void *scratch,
                                     size_t scratch_bytes, int32_t n_queries, int32_t n_slots, int32_t n_q_heads,
                                     int32_t n_kv_heads, int32_t head_dim, float scale, void *stream) {
  if (n_queries == 0) return PASTA_OK;
  size_t need = 0;
  if (pasta_dense_mask_scratch_bytes(n_queries, n_slots, n_q_heads, n_kv_heads, head_dim, &need) != PASTA_OK)
    return PASTA_ERR_INVALID_ARG;
  if (!k_pool || !v_pool || !mask || !mask_row || !q || !out || !scratch || scratch_bytes < need || n_slots < 1 ||
      n_q_heads % n_kv_heads || !(scale >= 0.f) || (reinterpret_cast<uintptr_t>(scratch) & 255))
    return PASTA_ERR_INVALID_ARG;
  const int G = n_q_heads / n_kv_heads;
  const int n_ranges = ranges_for(n_queries, n_kv_heads, n_slots);
  int range_len = (n_slots + n_ranges - 1) / n_ranges;
  range_len = (range_len + kTile - 1) / kTile * kTile;
  const size_t rows = size_t(n_queries) * n_q_heads * n_ranges;
  float2 *part_ml = static_cast<float2 *>(scratch);
  float *part_o = reinterpret_cast<float *>(static_cast<uint8_t *>(scratch) + (rows * sizeof(float2) + 255) / 256 * 256);
  const float sc = (scale == 0.f ? 1.0f / std::sqrt(static_cast<float>(head_dim)) : scale) * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t units = static_cast<int64_t>(n_queries) * n_kv_heads * n_ranges;
  const unsigned blocks = static_cast<unsigned>((units + 1) / 2);
#define PASTA_DM(DD, GG)                                                                                              \
  if (head_dim == DD && G == GG) {                                                                                    \
    dense_mask_attn_kernel<DD, GG><<<blocks, 64, 0, st>>>(                                                           \
        static_cast<const __nv_bfloat16 *>(k_pool), static_cast<const __nv_bfloat16 *>(v_pool), mask, mask_stride,    \
        mask_row, static_cast<const __nv_bfloat16 *>(q), part_ml, part_o, n_queries, n_slots, n_kv_heads, n_ranges,   \
        range_len, sc);                                                                                               \
  } else
  PASTA_DM(128, 1) PASTA_DM(128, 2) PASTA_DM(128, 4) PASTA_DM(64, 1) PASTA_DM(64, 2) PASTA_DM(64, 4)
  return PASTA_ERR_INVALID_ARG;
#undef PASTA_DM
  if (cudaGetLastError() != cudaSuccess) return PASTA_ERR_CUDA;
  const int64_t n_rows = static_cast<int64_t>(n_queries) * n_q_heads;
  dense_mask_merge_kernel<<<static_cast<unsigned>((n_rows * 32 + 255) / 256), 256, 0, st>>>(
      part_ml, part_o, static_cast<float *>(out), lse, static_cast<int32_t>(n_rows), n_ranges, head_dim);
  return cudaGetLastError() == cudaSuccess ? PASTA_OK : PASTA_ERR_CUDA;
}

}  // extern "C"
