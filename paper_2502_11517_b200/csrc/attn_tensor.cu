// K2: tensor-core pass over every stream the queries of a request read (head_dim 128): the prefix they share is
// staged once for all of them; a fork's own chunk rides along with the other rows masked.
//
// One persistent CTA per SM walks its contiguous range of t-units.  A t-unit is a range of 128-token tiles
// (8 pages) of one request's page list, for one kv head.  Rows of the score matrix are the request's
// queries times the `group` query heads of that kv head (<= 128 rows, zero padded):
//
//   S[128 x 128] = Q[128 x 128] . K_tile^T            tcgen05.mma (N = 128), A and B from shared memory, D in TMEM
//   P            = 2^(S * scale*log2e - m_ref)         one thread per row and half tile, masked by visible lengths
//   O_h[128 x 128] += P_h[128 x 64] . V_half           tcgen05.mma, P (bf16) read from TMEM as the A operand
//
// The two halves h of a tile (pages 0-3 and 4-7) belong to two softmax groups.  Each group has its own running
// reference m_ref, sum l and accumulator O_h, so the groups exchange nothing until the unit's epilogue, where
// the two accumulators are folded into one row on their way out of TMEM: a partial row (m, l, O) for the merge kernel,
// or, for a unit that covers its whole (request, kv head) run, the normalised output row itself.  m_ref is raised only when a half tile's maximum exceeds
// it by more than 2^8 (then O_h and l are rescaled in TMEM).  P overwrites the first 32 columns of the scores it
// was computed from; S is double-buffered so that Q.K^T of the next tile runs during the softmax of this one.
//
// Warp roles: warp 0 producer (eight lanes issue the bulk copies of a tile's (page, kv head) blocks into a
// 3-stage ring of 64 KB), warp 1 MMA issue (one thread), warps 2-3 build the stacked, swizzled Q operand of each
// unit, warps 4-7 and 8-11 the two softmax groups (a thread owns the row held in its TMEM lane: row i is in lane i
// when the unit's MMAs have M = 128; a unit with at most 64 rows uses M = 64, which puts row i in lane
// 32 (i / 16) + i % 16).
// Every wait is bounded; on expiry the CTA reports PASTA_ERR_TIMEOUT, drains and leaves.
#include "device_common.cuh"
#include "kernels.hpp"

namespace pasta {

namespace {

constexpr int T_THREADS = 384;
constexpr int T_STAGES = 3;
constexpr int T_TILE = PASTA_TILE_PAGES * PASTA_PAGE;          // 128 tokens
constexpr int T_HALF = T_TILE / 2;                              // columns of one softmax group
constexpr int T_HALF_PAGES = PASTA_TILE_PAGES / 2;
static_assert(PASTA_TILE_PAGES == 8, "the kernel is written for 8-page tiles");
constexpr int T_BLOCK = 8192;                                  // bytes of one (page, kv head) block, d = 128
constexpr int T_STAGE_BYTES = PASTA_TILE_PAGES * T_BLOCK;      // 64 KB
constexpr int T_Q_BYTES = 128 * 128 * 2;                       // 32 KB
constexpr int OFF_Q = 0;
constexpr int OFF_STAGE = OFF_Q + T_Q_BYTES;
constexpr int OFF_BAR = OFF_STAGE + T_STAGES * T_STAGE_BYTES;
// barriers (8 bytes each)
constexpr int B_FULL = 0, B_EMPTY = B_FULL + T_STAGES, B_SFULL = B_EMPTY + T_STAGES, B_PFULL = B_SFULL + 2,
              B_QFULL = B_PFULL + 4,   // PFULL[2 * b + group]
              B_QFREE = B_QFULL + 1, B_OFULL = B_QFREE + 1,
              B_OFREE = B_OFULL + 1, B_MLFULL = B_OFREE + 1,
              B_DRAIN = B_MLFULL + 1,  // only used when a role gave up: completion of the MMAs still in flight
              B_COUNT = B_DRAIN + 1;
constexpr int OFF_META = OFF_BAR + 8 * ((B_COUNT + 1) & ~1);   // per stage: 8 page metas
constexpr int T_RING = 8;                                      // unit records the producer keeps published (64 B each)
constexpr int OFF_MISC = OFF_META + T_STAGES * 32;             // tmem base, abort flag, shared units taken, their ids
constexpr int OFF_ML1 = OFF_MISC + 16 + 64 * T_RING;           // (m_ref, l) of group 1's rows, for the epilogue
constexpr int T_SMEM_USED = OFF_ML1 + 128 * 8;
constexpr int T_SMEM_BYTES = T_SMEM_USED + 1024;               // slack to align the base to 1024
static_assert(T_SMEM_BYTES <= 232448, "shared memory budget");

constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t COL_S = 0, COL_O = 256;   // S[b] at 128 b (group g: columns 64 g .. 64 g + 63; its P reuses the first 32), O_g at 256 + 128 g

// instruction descriptors: D fp32, A/B bf16; M = 128, or M = 64 for a unit with at most 64 stacked rows (half the
// tensor-core work per tile: long runs are power-limited, and the tensor cores are what draws the power)
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10);
constexpr uint32_t IDESC_M128 = (128u >> 4) << 24, IDESC_M64 = (64u >> 4) << 24;
constexpr uint32_t IDESC_QK = IDESC_BASE | ((128u >> 3) << 17);                // N = 128, both operands K-major
constexpr uint32_t IDESC_PV = IDESC_BASE | ((128u >> 3) << 17) | (1u << 16);   // N = 128, B (= V) MN-major
constexpr int T_M64_ROWS = 64;

__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
         (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);   // version 1, 128-byte swizzle
}

__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// A operand from TMEM: row m in lane m, two bf16 per 32-bit column (16 K-elements = 8 columns)
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

#define PASTA_R32(v) \
  v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15], v[16], v[17], \
  v[18], v[19], v[20], v[21], v[22], v[23], v[24], v[25], v[26], v[27], v[28], v[29], v[30], v[31]

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
      "%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  // the wait names the registers so that nothing that uses them can be scheduled above it
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
        "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
        "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
        "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
      :: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// The same load without its wait, and the wait by itself, so that several loads can be in flight before one wait.  The
// wait (and tmem_ld_order for a second register set) names the registers so that nothing that uses them can be
// scheduled above it.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t *r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
      "%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
#define PASTA_RW32(r)                                                                                                  \
  "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),          \
  "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]),   \
  "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]),  \
  "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
__device__ __forceinline__ void tmem_ld_wait32(uint32_t *r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : PASTA_RW32(r) :: "memory");
}
__device__ __forceinline__ void tmem_ld_order32(uint32_t *r) { asm volatile("" : PASTA_RW32(r) :: "memory"); }
// 16 consecutive fp32 columns, issued without the wait
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t *r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
#define PASTA_RW16(r)                                                                                                  \
  "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),          \
  "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
// waits for every load of this thread in flight; names the registers of two of them
__device__ __forceinline__ void tmem_ld_wait16x2(uint32_t *r0, uint32_t *r1) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : PASTA_RW16(r0), PASTA_RW16(r1) :: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float *v) {
  uint32_t r[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
      "%29,%30,%31};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32_u32(uint32_t taddr, const uint32_t *r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
      "%29,%30,%31};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// two fp32 lanes at once: {x0, x1} = {a0, a1} * {b, b} + {c, c}
__device__ __forceinline__ void fma2(float &x0, float &x1, float a0, float a1, float b, float c) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(x0), "=f"(x1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
// {x0, x1} = {a0, a1} * {b, b} + {c0, c1}
__device__ __forceinline__ void fma2v(float &x0, float &x1, float a0, float a1, float b, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %6};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(x0), "=f"(x1) : "f"(a0), "f"(a1), "f"(b), "f"(c0), "f"(c1));
}
// {s0, s1} += {p0, p1}
__device__ __forceinline__ void add2(float &s0, float &s1, float p0, float p1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%0, %1};\n\tmov.b64 rb, {%2, %3};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "+f"(s0), "+f"(s1) : "f"(p0), "f"(p1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Bounded wait of one role for another that also gives up when some role of the CTA has already given up.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) { *abort_flag = 1; return false; }
  }
}
// The same for a whole warp whose lanes go on to warp-wide instructions (tcgen05.ld / st, votes, __syncwarp): the
// lanes poll on their own, so the warp takes the decision as one.
__device__ __forceinline__ bool warp_wait_or_abort(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit) {
  return __all_sync(0xffffffffu, wait_or_abort(bar, parity, abort_flag, limit));
}

// bulk copy whose lines are the first to leave L2: every page is read once per launch
__device__ __forceinline__ void bulk_g2s_stream(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}

struct UnitInfo {
  int treq, g, tile_begin, tile_end, row_base;
  int page_off, n_pages, n_threads, n_streams, vis_off, tq_off, final_rows;
};

__device__ __forceinline__ UnitInfo load_unit(const int32_t *plan, int off_tunit, int off_treq, int u) {
  (void)off_treq;
  const int4 *U = reinterpret_cast<const int4 *>(plan + off_tunit + u * PU_WORDS);   // tables start 16-byte aligned
  const int4 a = U[0], b = U[1], c = U[2];
  UnitInfo x;
  x.treq = a.x; x.g = a.y; x.tile_begin = a.z; x.tile_end = a.w;
  x.row_base = b.x; x.page_off = b.y; x.n_pages = b.z; x.n_threads = b.w;
  x.n_streams = c.x; x.vis_off = c.y; x.tq_off = c.z; x.final_rows = c.w;
  return x;
}

struct TensorArgs {
  int32_t off_tunit, off_treq, off_tcta, off_pages, off_pmeta, off_vis, off_tq;
  int32_t off_dunit, n_dunits;      // units no CTA owns in advance (per layer): taken from a counter at run time
  int32_t n_queries, layer_begin, layer_count;
  float scale_log2;
  void *out;                        // [layer_count, n_queries, Hq, 128], fp32 or bf16: rows of final units go here
  float *lse;                       // [layer_count, n_queries, Hq] or null
  int32_t out_bf16;
};

// A role's place in its CTA's sequence of units: first the units assigned to the CTA, layer by layer, whose records every
// role reads from the plan itself; then units of the shared pool (whole short runs kept back by the planner), taken from
// a counter in global memory.  Only the producer, which gets to every unit first, touches the counter: it publishes the
// record (and layer) of each shared unit it takes in a ring of T_RING slots in shared memory, and the other roles read
// the records from there in the same order, without a round trip to global memory at the start of a unit.  A record
// with tile_end = 0 ends the sequence.  The producer is at most T_STAGES tiles, hence units, ahead of the tile whose
// P.V has finished, and no role is a whole unit behind that one when it reads its next record, so a slot is not
// overwritten before everybody has read it.
struct Walk { int ll, u, k; };

template <bool kProducer, bool kShared>
__device__ __forceinline__ bool next_unit(Walk &w, const TensorArgs &a, const int32_t *plan, int u0, int u1, volatile int *ring,
                                          int32_t *counter, int lane, bool whole_warp, volatile int *abort_flag,
                                          long long limit, bool &ok, UnitInfo &x, int &ll) {
  if (u0 < u1 && w.ll < a.layer_count) {
    x = load_unit(plan, a.off_tunit, 0, w.u);
    ll = w.ll;
    if (++w.u == u1) { w.u = u0; ++w.ll; }
    return true;
  }
  if (!kShared) return false;        // this build of the kernel serves plans without shared units
  if (a.n_dunits == 0) return false;
  int32_t *slot = const_cast<int32_t *>(reinterpret_cast<volatile int32_t *>(ring)) + 2 + 16 * (w.k % T_RING);
  if (kProducer) {
    int id = -1;
    if (lane == 0) {
      id = atomicAdd(counter, 1);
      if (id >= a.n_dunits * a.layer_count) id = -1;
    }
    id = __shfl_sync(0xffffffffu, id, 0);
    if (id >= 0) {
      ll = id / a.n_dunits;
      x = load_unit(plan, a.off_dunit, 0, id - ll * a.n_dunits);
    }
    if (lane == 0) {
      int4 *s4 = reinterpret_cast<int4 *>(slot);
      s4[0] = make_int4(x.treq, x.g, x.tile_begin, id >= 0 ? x.tile_end : 0);
      s4[1] = make_int4(x.row_base, x.page_off, x.n_pages, x.n_threads);
      s4[2] = make_int4(x.n_streams, x.vis_off, x.tq_off, ll);
      s4[3] = make_int4(x.final_rows, 0, 0, 0);
      __threadfence_block();
      ring[0] = w.k + 1;
    }
    ++w.k;
    return id >= 0;
  }
  int got = 1;
  if (!whole_warp || lane == 0) {
    if (ring[0] <= w.k) {
      const long long t0 = clock64();
      while (ring[0] <= w.k) {
        if (*abort_flag) { got = 0; break; }
        if (clock64() - t0 > limit) { *abort_flag = 1; got = 0; break; }
        __nanosleep(64);
      }
    }
  }
  if (whole_warp) {
    got = __shfl_sync(0xffffffffu, got, 0);
    __syncwarp();
  }
  if (!got) { ok = false; return false; }
  const int4 *s4 = reinterpret_cast<const int4 *>(slot);
  const int4 ra = s4[0], rb = s4[1], rc = s4[2];
  x.final_rows = s4[3].x;
  ++w.k;
  if (ra.w == 0) return false;
  x.treq = ra.x; x.g = ra.y; x.tile_begin = ra.z; x.tile_end = ra.w;
  x.row_base = rb.x; x.page_off = rb.y; x.n_pages = rb.z; x.n_threads = rb.w;
  x.n_streams = rc.x; x.vis_off = rc.y; x.tq_off = rc.z; ll = rc.w;
  return true;
}

template <bool kShared>
__global__ void __launch_bounds__(T_THREADS, 1)
attn_tensor_kernel(PoolView pv, TensorArgs a, const __nv_bfloat16 *__restrict__ q) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t *sm = smem_raw + (base - raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = pv.n_q_heads / pv.n_kv_heads;
  // row / G sits between two units for every role: a shift when G is a power of two (it usually is), the division otherwise
  auto div_g = [&](int r) { return (G & (G - 1)) == 0 ? r >> (31 - __clz(G)) : r / G; };
  const uint32_t bar = base + OFF_BAR;
  int32_t *meta_s = reinterpret_cast<int32_t *>(sm + OFF_META);
  uint32_t *misc = reinterpret_cast<uint32_t *>(sm + OFF_MISC);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(misc + 1);
  const int32_t *plan = pv.plan;
  const int u0 = plan[a.off_tcta + 2 * blockIdx.x], u1 = plan[a.off_tcta + 2 * blockIdx.x + 1];

  // ---- set-up.  Operand bytes that no copy fills meet zero weights, so they only have to be finite: the Q builder
  // writes every row a unit's MMAs read (64 or 128, zeros beyond the unit's last), and the producer clears the page
  // slots a partial tile leaves empty the first time each stage is used (afterwards they hold an earlier tile's keys
  // and values).
  if (tid == 0) {
    for (int s = 0; s < T_STAGES; ++s) { mbar_init(bar + 8 * (B_FULL + s), 1); mbar_init(bar + 8 * (B_EMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar + 8 * (B_SFULL + b), 1);
      mbar_init(bar + 8 * (B_PFULL + 2 * b), 4);        // one arrival per warp: 32 arrivals of a warp on one
      mbar_init(bar + 8 * (B_PFULL + 2 * b + 1), 4);    // barrier word are served one after the other
    }
    mbar_init(bar + 8 * B_QFULL, 2);
    mbar_init(bar + 8 * B_QFREE, 1);
    mbar_init(bar + 8 * B_OFULL, 1);
    mbar_init(bar + 8 * B_OFREE, 8);       // one arrival per softmax warp, of both groups
    mbar_init(bar + 8 * B_MLFULL, 8);
    mbar_init(bar + 8 * B_DRAIN, 1);
    misc[1] = 0;
    misc[2] = 0;
    mbar_init_fence();
  }
  fence_proxy_async();
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + OFF_MISC), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];
  // everything above overlaps the end of the kernel ahead in the stream (the append of this step's tokens); from here on
  // that kernel's writes are needed, and the kernels behind this one may start their own set-up
  grid_dependency_wait();
  grid_launch_dependents();
  const long long limit = pv.wait_limit;
  uint32_t prod_it = 0;       // warp 0: tiles whose copies have been issued
  volatile int *ring = reinterpret_cast<volatile int *>(misc + 2);
  int32_t *counter = pv.status + PASTA_STATUS_TAIL_COUNTER;

  // test hook: a held role goes straight to the tear-down, so that the roles waiting for it run into their limits
  const int role = warp == 0 ? 0 : warp == 1 ? 1 : warp < 4 ? 2 : 3 + ((warp - 4) >> 2);
  if ((pv.debug_hold >> role) & 1) {
  } else if (warp == 0) {
    // ================================================================ producer
    uint32_t it = 0;
    bool ok = true;
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    {
      Walk wk{0, u0, 0};
      UnitInfo x;
      int ll = 0;
      while (ok && next_unit<true, kShared>(wk, a, plan, u0, u1, ring, counter, lane, true, abort_flag, limit, ok, x, ll)) {
        const uint8_t *kv_layer = pv.kv_base + (a.layer_begin + ll) * pv.layer_stride;
        for (int tile = x.tile_begin; tile < x.tile_end; ++tile, ++it) {
          const int s = it % T_STAGES;
          if (!warp_wait_or_abort(bar + 8 * (B_EMPTY + s), ((it / T_STAGES) & 1) ^ 1, abort_flag, limit)) { ok = false; break; }
          const int n_valid = min(PASTA_TILE_PAGES, x.n_pages - tile * PASTA_TILE_PAGES);
          int page = 0;
          if (lane < PASTA_TILE_PAGES) {
            int meta = -1;
            if (lane < n_valid) {
              page = plan[a.off_pages + x.page_off + tile * PASTA_TILE_PAGES + lane];
              meta = plan[a.off_pmeta + x.page_off + tile * PASTA_TILE_PAGES + lane];
              if (page < 0 || page >= pv.n_pages) { report(pv.status, PASTA_ERR_DEVICE_CHECK); page = 0; meta = -1; }
            }
            meta_s[s * PASTA_TILE_PAGES + lane] = meta;
          }
          if (it < T_STAGES && n_valid < PASTA_TILE_PAGES) {     // first use of this stage and some slots stay empty
            uint4 *slot = reinterpret_cast<uint4 *>(sm + OFF_STAGE + s * T_STAGE_BYTES + n_valid * T_BLOCK);
            for (int i = lane; i < (PASTA_TILE_PAGES - n_valid) * (T_BLOCK / 16); i += 32) slot[i] = make_uint4(0, 0, 0, 0);
            fence_proxy_async();
            __syncwarp();
          }
          if (lane == 0) mbar_expect_tx(bar + 8 * (B_FULL + s), n_valid * T_BLOCK);
          __syncwarp();
          if (lane < n_valid)
            bulk_g2s_stream(base + OFF_STAGE + s * T_STAGE_BYTES + lane * T_BLOCK,
                            kv_layer + (static_cast<int64_t>(page) * pv.n_kv_heads + x.g) * T_BLOCK, T_BLOCK,
                            bar + 8 * (B_FULL + s), policy);
        }
      }
    }
    prod_it = it;
  } else if (warp == 1) {
    // ================================================================ MMA issue (one thread)
    if (lane == 0) {
      uint32_t it = 0, uc = 0;
      bool ok = true;
      const uint32_t q_addr = base + OFF_Q;
      {
        Walk wk{0, u0, 0};
        UnitInfo x;
        int ll = 0;
        for (; ok && next_unit<false, kShared>(wk, a, plan, u0, u1, ring, counter, lane, false, abort_flag, limit, ok, x, ll); ++uc) {
          const int nt = x.tile_end - x.tile_begin;
          const uint32_t m_bits = x.n_threads * G <= T_M64_ROWS ? IDESC_M64 : IDESC_M128;
          if (!wait_or_abort(bar + 8 * B_QFULL, uc & 1, abort_flag, limit)) { ok = false; break; }
          tc_fence_after();
          for (int k = 0; k <= nt && ok; ++k) {
            if (k < nt) {
              // ---- S[b] = Q . K^T for tile `it` (S[b] was last used by tile it - 2, whose P.V was issued before this)
              const uint32_t s = it % T_STAGES, b = it & 1;
              if (!wait_or_abort(bar + 8 * (B_FULL + s), (it / T_STAGES) & 1, abort_flag, limit)) { ok = false; break; }
              tc_fence_after();
              const uint32_t k_addr = base + OFF_STAGE + s * T_STAGE_BYTES;
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const uint32_t half = ks >> 2, kk = ks & 3;
                mma_ss(tmem + COL_S + b * T_TILE, smem_desc(q_addr + half * 16384 + kk * 32, 16, 1024),
                       smem_desc(k_addr + half * 1024 + kk * 32, 16, 4096), IDESC_QK | m_bits, ks > 0);
              }
              mma_commit(bar + 8 * (B_SFULL + b));
              if (k == nt - 1) mma_commit(bar + 8 * B_QFREE);   // the Q operand may be replaced once these finish
            }
            if (k > 0) {
              // ---- O_g += P_g . V_g for both halves of tile `it - 1` (when k == nt, `it` already points past it)
              const uint32_t j = it - 1;
              const uint32_t s = j % T_STAGES, b = j & 1;
              if (k == 1 && uc > 0) {   // the unit's first P.V overwrites the accumulators: the previous unit's rows must be read out
                if (!wait_or_abort(bar + 8 * B_OFREE, (uc - 1) & 1, abort_flag, limit)) { ok = false; break; }
              }
              const uint32_t v_addr = base + OFF_STAGE + s * T_STAGE_BYTES + 2048;
              for (uint32_t g2 = 0; g2 < 2 && ok; ++g2) {
                if (!wait_or_abort(bar + 8 * (B_PFULL + 2 * b + g2), (j >> 1) & 1, abort_flag, limit)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int pg = 0; pg < T_HALF_PAGES; ++pg)
                  mma_ts(tmem + COL_O + g2 * 128, tmem + COL_S + b * T_TILE + g2 * T_HALF + pg * 8,
                         smem_desc(v_addr + (g2 * T_HALF_PAGES + pg) * T_BLOCK, 1024, 4096), IDESC_PV | m_bits,
                         (k > 1) || (pg > 0));
              }
              if (!ok) break;
              mma_commit(bar + 8 * (B_EMPTY + s));
              if (k == nt) mma_commit(bar + 8 * B_OFULL);
            }
            if (k < nt) ++it;
          }
        }
      }
    }
  } else if (warp < 4) {
    // ================================================================ stacked Q operand (64 threads)
    const int t64 = tid - 64;
    uint32_t uc = 0;
    bool ok = true;
    {
      Walk wk{0, u0, 0};
      UnitInfo x;
      int ll = 0;
      for (; ok && next_unit<false, kShared>(wk, a, plan, u0, u1, ring, counter, lane, true, abort_flag, limit, ok, x, ll); ++uc) {
        const int rows = x.n_threads * G;
        // thread t64 builds rows t64 and 64 + t64.  The 16 loads of a row are issued together, and those of the first
        // row before the wait for the operand buffer: the producer publishes a unit while the one before it is still
        // being worked on, so a unit of up to 64 rows has its whole operand in registers by the time the last Q.K^T of
        // its predecessor lets go of the buffer
#pragma unroll 1
        for (int rr = 0; rr < 2; ++rr) {
          const int row = rr * 64 + t64;
          if (rr == 1 && rows <= 64) break;
          uint4 val[16];
          if (row < rows) {
            const int t = div_g(row), hl = row - t * G;
            const int qn = plan[a.off_tq + x.tq_off + t];
            const uint4 *src = reinterpret_cast<const uint4 *>(
                q + ((static_cast<int64_t>(ll) * a.n_queries + qn) * pv.n_q_heads + x.g * G + hl) * 128);
#pragma unroll
            for (int c = 0; c < 16; ++c) val[c] = __ldg(src + c);
          } else {
#pragma unroll
            for (int c = 0; c < 16; ++c) val[c] = make_uint4(0, 0, 0, 0);
          }
          if (rr == 0 && uc > 0 && !warp_wait_or_abort(bar + 8 * B_QFREE, (uc - 1) & 1, abort_flag, limit)) { ok = false; break; }
          const int r8 = row & 7;
          uint8_t *dst = sm + OFF_Q + (row >> 3) * 1024 + r8 * 128;
#pragma unroll
          for (int c = 0; c < 16; ++c)
            *reinterpret_cast<uint4 *>(dst + (c >> 3) * 16384 + (((c & 7) ^ r8) << 4)) = val[c];
        }
        if (!ok) break;
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar + 8 * B_QFULL);
      }
    }
  } else {
    // ================================================================ softmax + epilogue (2 groups of 128 threads)
    const int grp = (warp - 4) >> 2;                // this group's half of every tile: pages 4 grp .. 4 grp + 3
    const int wq = warp & 3;                        // the TMEM lanes this warp reaches: 32 wq .. 32 wq + 31
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t col_o = COL_O + grp * 128;
    float2 *ml1 = reinterpret_cast<float2 *>(sm + OFF_ML1);
    uint32_t it = 0, uc = 0;
    bool ok = true;
    {
      Walk wk{0, u0, 0};
      UnitInfo x;
      int ll = 0;
      for (; ok && next_unit<false, kShared>(wk, a, plan, u0, u1, ring, counter, lane, true, abort_flag, limit, ok, x, ll); ++uc) {
        const int nt = x.tile_end - x.tile_begin;
        const int rows = x.n_threads * G;
        // M = 128: row i of the score matrix sits in TMEM lane i.  M = 64: row i sits in lane 32 (i / 16) + i % 16, so
        // a warp owns 16 rows and its upper 16 lanes hold nothing (whatever they compute is never read or written out)
        const bool m64 = rows <= T_M64_ROWS;
        const int row = m64 ? (lane < 16 ? wq * 16 + lane : 128) : wq * 32 + lane;
        const bool active = row < rows;
        const bool warp_active = (m64 ? wq * 16 : wq * 32) < rows;
        const int32_t *visrow = plan + a.off_vis + x.vis_off + (active ? div_g(row) : 0) * x.n_streams;
        // the row's visible lengths of the first four local streams stay in registers for the whole unit: a global
        // load per page would otherwise sit between two tiles of this group
        // where the unit's rows go, in one register: the first partial row, or for a final unit ~(offset of its queries)
        const int dest = x.final_rows ? ~x.tq_off : x.row_base;
        int vis0 = visrow[0];
        int vis1 = x.n_streams > 1 ? visrow[1] : 0;
        int vis2 = x.n_streams > 2 ? visrow[2] : 0;
        int vis3 = x.n_streams > 3 ? visrow[3] : 0;
        asm volatile("" : "+r"(vis0), "+r"(vis1), "+r"(vis2), "+r"(vis3));   // loaded here, once, not again at each use
        float m_ref = -INFINITY, l = 0.f;
        for (int k = 0; k < nt; ++k, ++it) {
          const uint32_t s = it % T_STAGES, b = it & 1;
          const uint32_t col_s = COL_S + b * T_TILE + grp * T_HALF;
          // the tile's page metas are in shared memory once its copies have landed: fetch the row's thresholds early
          if (!warp_wait_or_abort(bar + 8 * (B_FULL + s), (it / T_STAGES) & 1, abort_flag, limit)) { ok = false; break; }
          int thr[T_HALF_PAGES];
          bool full = true;
          const int4 m4 = *reinterpret_cast<const int4 *>(meta_s + s * PASTA_TILE_PAGES + grp * T_HALF_PAGES);
          // pages that every thread of the request sees in full need no thresholds (the same answer for the whole CTA)
          const bool no_mask = (m4.x | m4.y | m4.z | m4.w) >= 0 && ((m4.x & m4.y & m4.z & m4.w) & PASTA_PMETA_ALL_VISIBLE);
          if (warp_active && !no_mask) {
            const int base_meta = m4.x & ~PASTA_PMETA_ALL_VISIBLE;
            const bool run = m4.x >= 0 && m4.w >= 0 && (m4.y & ~PASTA_PMETA_ALL_VISIBLE) == base_meta + (1 << PASTA_PMETA_STREAM_BITS) &&
                             (m4.z & ~PASTA_PMETA_ALL_VISIBLE) == base_meta + (2 << PASTA_PMETA_STREAM_BITS) &&
                             (m4.w & ~PASTA_PMETA_ALL_VISIBLE) == base_meta + (3 << PASTA_PMETA_STREAM_BITS);
            if (run) {
              // four consecutive pages of one stream (the usual case): one look-up of the row's visible length
              const int sl = PASTA_PMETA_STREAM(base_meta);
              int vis;
              if (sl < 4) vis = sl == 0 ? vis0 : sl == 1 ? vis1 : sl == 2 ? vis2 : vis3;
              else vis = visrow[sl];
              const int rem = active ? vis - PASTA_PMETA_PAGE(base_meta) * PASTA_PAGE : 0;
#pragma unroll
              for (int pg = 0; pg < T_HALF_PAGES; ++pg) thr[pg] = min(max(rem - pg * PASTA_PAGE, 0), PASTA_PAGE);
              full = rem >= T_HALF_PAGES * PASTA_PAGE;
            } else {
              const int metas[T_HALF_PAGES] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
              for (int pg = 0; pg < T_HALF_PAGES; ++pg) {
                const int meta = metas[pg];
                int t = 0;
                if (active && meta >= 0) {
                  const int sl = PASTA_PMETA_STREAM(meta);
                  int vis;
                  if (sl < 4) vis = sl == 0 ? vis0 : sl == 1 ? vis1 : sl == 2 ? vis2 : vis3;
                  else vis = visrow[sl];
                  t = min(max(vis - PASTA_PMETA_PAGE(meta) * PASTA_PAGE, 0), PASTA_PAGE);
                }
                thr[pg] = t;
                full = full && (t == PASTA_PAGE);
              }
            }
          }
          if (!warp_wait_or_abort(bar + 8 * (B_SFULL + b), (it >> 1) & 1, abort_flag, limit)) { ok = false; break; }
          tc_fence_after();
          if (warp_active) {
            float sc[T_HALF];
            {
              uint32_t *raw_sc = reinterpret_cast<uint32_t *>(sc);      // both halves in flight before one wait
              tmem_ld32_issue(tmem + lane_addr + col_s, raw_sc);
              tmem_ld32_issue(tmem + lane_addr + col_s + 32, raw_sc + 32);
              tmem_ld_wait32(raw_sc);
              tmem_ld_order32(raw_sc + 32);
            }
            if (!full) {
#pragma unroll
              for (int j = 0; j < T_HALF; ++j)
                if ((j & 15) >= thr[j >> 4]) sc[j] = -INFINITY;
            }
            float mx[4] = {sc[0], sc[1], sc[2], sc[3]};
#pragma unroll
            for (int j = 4; j < T_HALF; j += 4) {
              mx[0] = fmaxf(mx[0], sc[j]); mx[1] = fmaxf(mx[1], sc[j + 1]);
              mx[2] = fmaxf(mx[2], sc[j + 2]); mx[3] = fmaxf(mx[3], sc[j + 3]);
            }
            const float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * a.scale_log2;
            const bool need = mt > m_ref + 8.f;       // also true for the first visible tile (m_ref = -inf)
            const bool rescale = active && need && l > 0.f;
            if (__any_sync(0xffffffffu, rescale)) {
              // O_g and l are relative to m_ref: move them to the new reference.  The accumulator is quiet once the
              // P.V of the previous tile has finished, which is what releases that tile's stage.
              if (!warp_wait_or_abort(bar + 8 * (B_EMPTY + (it - 1) % T_STAGES), ((it - 1) / T_STAGES) & 1, abort_flag, limit)) { ok = false; break; }
              tc_fence_after();
              const float f = rescale ? fast_exp2(m_ref - mt) : 1.f;
#pragma unroll 1
              for (int cb = 0; cb < 4; ++cb) {
                float ov[32];
                tmem_ld32(tmem + lane_addr + col_o + cb * 32, ov);
#pragma unroll
                for (int j = 0; j < 32; ++j) ov[j] *= f;
                tmem_st32(tmem + lane_addr + col_o + cb * 32, ov);
              }
              tmem_st_wait();
              l *= f;
            }
            if (need) m_ref = mt;
            const float ref = (m_ref == -INFINITY) ? 0.f : m_ref;
            float ls[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t pk[T_HALF / 2];
#pragma unroll
            for (int j = 0; j < T_HALF; j += 4) {
              float x0, x1, x2, x3;
              fma2(x0, x1, sc[j], sc[j + 1], a.scale_log2, -ref);
              fma2(x2, x3, sc[j + 2], sc[j + 3], a.scale_log2, -ref);
              const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = fast_exp2(x3);
              const uint32_t w0 = pack_bf16(p0, p1), w1 = pack_bf16(p2, p3);
              // l sums the weights as the MMA will read them (rounded to bf16), so that O / l stays a convex
              // combination of V rows: with one dominant key the result is that key's V row whatever m_ref is
              add2(ls[0], ls[1], bf16_lo(w0), bf16_hi(w0));
              add2(ls[2], ls[3], bf16_lo(w1), bf16_hi(w1));
              pk[j >> 1] = w0;
              pk[(j >> 1) + 1] = w1;
            }
            l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
            tmem_st32_u32(tmem + lane_addr + col_s, pk);      // P takes the place of the first 32 score columns
            tmem_st_wait();
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar + 8 * (B_PFULL + 2 * b + grp));
        }
        if (!ok) break;
        // ---- epilogue: the unit's rows leave TMEM as f0 O_0 + f1 O_1, the two groups' accumulators brought to one
        // reference.  The groups hand each other their (m_ref, l) through shared memory.  A unit of up to 64 rows
        // (`low`; its rows sit in the first 64 entries, so the table holds both groups') is written out by both groups,
        // 64 columns each: the time from a unit's last P.V to the next unit's first is mostly this epilogue.  A higher
        // unit is written out by group 0 alone.
        const bool low = m64;
        // (the query a final unit's row belongs to: asked for before the wait, which outlasts the load)
        const int qn_row = ((grp == 0 || low) && dest < 0 && active) ? __ldg(plan + a.off_tq + ~dest + div_g(row)) : 0;
        if (!warp_wait_or_abort(bar + 8 * B_OFULL, uc & 1, abort_flag, limit)) { ok = false; break; }
        tc_fence_after();
        if (active && (grp == 1 || low)) ml1[(grp == 0 ? 64 : 0) + row] = make_float2(m_ref, l);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar + 8 * B_MLFULL);
        if (grp == 1 && !low) {                 // nothing to read out of TMEM
          if (lane == 0) mbar_arrive(bar + 8 * B_OFREE);
          continue;
        }
        if (!warp_wait_or_abort(bar + 8 * B_MLFULL, uc & 1, abort_flag, limit)) { ok = false; break; }
        if (warp_active) {
          const float2 other = active ? ml1[(grp == 0 ? 0 : 64) + row] : make_float2(-INFINITY, 0.f);
          // accumulator 0 is group 0's, accumulator 1 group 1's; both groups get the same factors from the same values
          const float m0 = grp == 0 ? m_ref : other.x, l0 = grp == 0 ? l : other.y;
          const float m1 = grp == 0 ? other.x : m_ref, l1 = grp == 0 ? other.y : l;
          const float m_all = fmaxf(m0, m1);
          const float f0 = l0 > 0.f ? fast_exp2(m0 - m_all) : 0.f;
          const float f1 = l1 > 0.f ? fast_exp2(m1 - m_all) : 0.f;
          const float l_all = f0 * l0 + f1 * l1;
          const bool any0 = __any_sync(0xffffffffu, f0 != 0.f), any1 = __any_sync(0xffffffffu, f1 != 0.f);
          // a final unit's rows are the result: normalised and written to the output here, with the arithmetic the
          // merge applies to a row that has a single partial (weight 1, then times 1 / l)
          const bool fin = dest < 0;
          const int64_t prow = static_cast<int64_t>(ll) * pv.rows_per_layer + dest + row;
          int64_t orow = 0;
          float inv = 1.f;
          if (fin) {
            if (active) {
              orow = (static_cast<int64_t>(ll) * a.n_queries + qn_row) * pv.n_q_heads + x.g * G + (row - div_g(row) * G);
              inv = l_all > 0.f ? 1.f / l_all : 0.f;
              if (a.lse && grp == 0) a.lse[orow] = (m_all + log2f(l_all)) * 0.6931471805599453f;
            }
          } else if (active && grp == 0) {
            pv.part_ml[prow] = make_float2(m_all, l_all);
          }
          const bool write = active && (fin || l_all > 0.f);      // an output row with nothing visible is written as zeros
          // partial rows keep inv = 1; fp32 rows of either kind go to one address
          float *orow_f32 = fin ? static_cast<float *>(a.out) + orow * 128 : pv.part_o + prow * 128;
          // One warp per scheduler is at work here and every instruction waits for the one before it, so the epilogue
          // costs what its instruction count says.  The usual case, where every row of the warp has weights in both
          // accumulators (or all of them only in the first), takes two (one) packed instructions per pair of columns;
          // the general case guards each product: a factor of exactly 0 means that accumulator was never written for
          // this row, and whatever TMEM holds there must not be touched.
          const float g0 = f0 * inv, g1 = f1 * inv;
          const bool both = __all_sync(0xffffffffu, !active || (f0 != 0.f && f1 != 0.f));
          const bool only0 = !both && __all_sync(0xffffffffu, !active || (f0 != 0.f && f1 == 0.f));
          const int cb0 = low ? grp * 4 : 0, cb1 = low ? cb0 + 4 : 8;
#pragma unroll 1
          for (int cb = cb0; cb < cb1; ++cb) {
            // 16 columns of both accumulators in flight before one wait
            uint32_t q0[16], q1[16];
            if (any0) tmem_ld16_issue(tmem + lane_addr + COL_O + cb * 16, q0);
            if (any1) tmem_ld16_issue(tmem + lane_addr + COL_O + 128 + cb * 16, q1);
            tmem_ld_wait16x2(q0, q1);
            float r[16];
            if (both) {
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                float t0, t1;
                fma2(t0, t1, __uint_as_float(q1[j]), __uint_as_float(q1[j + 1]), g1, 0.f);
                fma2v(r[j], r[j + 1], __uint_as_float(q0[j]), __uint_as_float(q0[j + 1]), g0, t0, t1);
              }
            } else if (only0) {
#pragma unroll
              for (int j = 0; j < 16; j += 2) fma2(r[j], r[j + 1], __uint_as_float(q0[j]), __uint_as_float(q0[j + 1]), g0, 0.f);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                r[j] = (f0 != 0.f ? g0 * __uint_as_float(q0[j]) : 0.f) + (f1 != 0.f ? g1 * __uint_as_float(q1[j]) : 0.f);
            }
            if (write) {
              if (fin && a.out_bf16) {
                uint4 *dst = reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(a.out) + orow * 128 + cb * 16);
#pragma unroll
                for (int j = 0; j < 2; ++j)
                  dst[j] = make_uint4(pack_bf16(r[8 * j], r[8 * j + 1]), pack_bf16(r[8 * j + 2], r[8 * j + 3]),
                                      pack_bf16(r[8 * j + 4], r[8 * j + 5]), pack_bf16(r[8 * j + 6], r[8 * j + 7]));
              } else {
                float4 *dst = reinterpret_cast<float4 *>(orow_f32 + cb * 16);
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[j] = make_float4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar + 8 * B_OFREE);
      }
    }
  }

  // ---- tear-down
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // Some role gave up, so the others left in the middle of their work.  What the hardware still has in flight for
    // this CTA has to finish before its shared memory and TMEM are given back: the bulk copies of the last tiles
    // issued (their barriers complete whether or not anybody consumes the tiles) and the MMAs issued last (a commit
    // to a barrier of its own arrives once every earlier MMA of this thread has completed).  Both end on their own.
    if (warp == 0 && lane == 0) {
      for (uint32_t j = (prod_it > T_STAGES ? prod_it - T_STAGES : 0); j < prod_it; ++j)
        mbar_wait_bounded(bar + 8 * (B_FULL + j % T_STAGES), (j / T_STAGES) & 1);
    }
    if (warp == 1 && lane == 0) {
      mma_commit(bar + 8 * B_DRAIN);
      mbar_wait_bounded(bar + 8 * B_DRAIN, 0);
    }
    if (tid == 0) report(pv.status, PASTA_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
  }
  if (warp == 2) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace

bool tensor_path_available() { return true; }

cudaError_t launch_attn_tensor(const PoolView &pv, const PlanHeader &h, int32_t layer_begin, int32_t layer_count,
                               const void *q, float scale_log2, void *out, float *lse, bool out_bf16, cudaStream_t st) {
  if (pv.head_dim != 128) return cudaErrorInvalidValue;
  static uint64_t prepared[2] = {0, 0};
  const bool shared_units = h.w[PH_N_DUNITS] > 0;
  {
    cudaError_t e = raise_smem_limit(shared_units ? reinterpret_cast<const void *>(attn_tensor_kernel<true>)
                                                  : reinterpret_cast<const void *>(attn_tensor_kernel<false>),
                                     T_SMEM_BYTES, &prepared[shared_units]);
    if (e != cudaSuccess) return e;
  }
  const int grid = h.w[PH_T_GRID];
  if (grid == 0 || layer_count == 0) return cudaSuccess;
  TensorArgs a;
  a.off_tunit = h.w[PH_OFF_TUNIT]; a.off_treq = h.w[PH_OFF_TREQ]; a.off_tcta = h.w[PH_OFF_TCTA];
  a.off_pages = h.w[PH_OFF_PAGES]; a.off_pmeta = h.w[PH_OFF_PMETA]; a.off_vis = h.w[PH_OFF_VIS];
  a.off_tq = h.w[PH_OFF_TQ];
  a.off_dunit = h.w[PH_OFF_DUNIT]; a.n_dunits = h.w[PH_N_DUNITS];
  a.n_queries = h.w[PH_N_QUERIES]; a.layer_begin = layer_begin; a.layer_count = layer_count;
  a.scale_log2 = scale_log2;
  a.out = out; a.lse = lse; a.out_bf16 = out_bf16 ? 1 : 0;
  // two builds of the kernel: the one without the shared part of the walk is a little faster (0.7 % on long runs)
  return launch_overlapped(shared_units ? attn_tensor_kernel<true> : attn_tensor_kernel<false>, dim3(grid), dim3(T_THREADS),
                           T_SMEM_BYTES, st, pv, a, static_cast<const __nv_bfloat16 *>(q));
}

}  // namespace pasta
