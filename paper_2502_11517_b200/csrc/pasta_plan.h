// The step plan: what pasta_step_begin builds on the host and uploads, and what the kernels read.
// One array of int32 words; a header of word offsets followed by tables.  Page ids are shared by
// all layers, so one plan serves every layer of the step.
//
// Terms
//   query      one (request, thread) entry of the step, index n in entry order
//   stream     one page list: a request's main-thread tokens (id 0) or one fork's chunk (id = fork id).
//              Every thread sees a PREFIX [0, vis) of every stream (vis may be 0).
//   t-request  a request served by the tensor-core kernel: head_dim 128, its queries times `group` fit
//              PASTA_MAX_ROWS rows, at most PASTA_MAX_STREAMS streams.  The pages of every stream its queries read (the prefix
//              they share and each fork's own chunk alike) are concatenated into one page list that is cut into
//              tiles of PASTA_TILE_PAGES pages; rows of the score matrix are the request's queries
//              times the `group` query heads of one kv head: row = t_idx * group + h_local.
//   t-unit     (t-request, kv head, tile range): one CTA-sized piece of the tensor-core kernel; it
//              writes one partial result (m, l, O[d]) per row.  A unit that covers all tiles of its (t-request, kv
//              head) run, of a request none of whose queries has w-units, is FINAL: its rows are the result, the
//              kernel normalises them and writes them to the output itself, and the merge skips them.
//   d-unit     a t-unit that belongs to no CTA in advance: of the short (t-request, kv head) runs, every so often a
//              whole one is kept back; the CTAs take these from a shared counter once their own units are done, so
//              that SMs that stream faster than others end up doing more of the work.  Same record as a t-unit.
//   w-unit     (query, kv head, token range of one stream) of a request that is no t-request: one warp of
//              the warp-shuffle kernel; it writes `group` partial rows.
//   partial rows are numbered per layer: rows of the t-units and d-units first (row_base + row), then
//              t_rows + w_unit * group + h_local.
#pragma once
#include <cstdint>

#define PASTA_PLAN_MAGIC 0x50415354
#define PASTA_TILE_PAGES 8          // pages per tensor-core tile (128 tokens)
#define PASTA_PAGE 16               // tokens per page
#define PASTA_MAX_ROWS 128          // rows of the stacked-query matrix (threads * group)
// a page's meta word: bits 0-11 local stream, bits 12-29 page index within the stream, bit 30 set when every thread
// of the t-request sees the whole page (no row needs a mask there); -1 marks an unused slot of a tile
#define PASTA_PMETA_STREAM_BITS 12
#define PASTA_MAX_STREAMS ((1 << PASTA_PMETA_STREAM_BITS) - 1)      // streams one t-request may read
#define PASTA_MAX_STREAM_PAGES (1 << 18)                             // pages of one stream (4 M tokens)
#define PASTA_PMETA_ALL_VISIBLE (1 << 30)
#define PASTA_PMETA_STREAM(meta) ((meta) & PASTA_MAX_STREAMS)
#define PASTA_PMETA_PAGE(meta) (((meta) >> PASTA_PMETA_STREAM_BITS) & (PASTA_MAX_STREAM_PAGES - 1))

// header words
enum {
  PH_MAGIC = 0,
  PH_N_QUERIES,
  PH_N_APPEND,        // entries with n_new == 1
  PH_N_TREQ,
  PH_N_TUNITS,
  PH_N_WUNITS,
  PH_T_ROWS,          // partial rows written by t-units and d-units
  PH_ROWS,            // all partial rows of one layer
  PH_T_GRID,          // CTAs of the tensor-core kernel that have work
  PH_OFF_APPEND,      // 2 words per appended token: page, offset
  PH_OFF_QUERY,       // PQ_WORDS per query
  PH_OFF_TREQ,        // PT_WORDS per t-request
  PH_OFF_TRANGE,      // per (t-request, kv head): first t-unit, one past the last
  PH_OFF_TUNIT,       // PU_WORDS per t-unit
  PH_OFF_TCTA,        // per CTA: first t-unit, one past the last
  PH_OFF_WUNIT,       // PW_WORDS per w-unit
  PH_OFF_PAGES,       // page ids
  PH_OFF_PMETA,       // parallel to pages (t-request lists only): (page index in its stream << 12) | local stream
  PH_OFF_VIS,         // per t-request: [n_threads][n_streams] visible length of local stream for thread
  PH_OFF_TQ,          // per t-request: [n_threads] query index of each row-thread
  PH_OFF_APOS,        // position id of every appended token (parallel to the append table)
  PH_OFF_QPOS,        // position id of every query's token
  PH_TOTAL_WORDS,
  PH_N_DUNITS,        // d-units of one layer
  PH_OFF_DUNIT,       // PU_WORDS per d-unit
  PH_OFF_DRANGE,      // per (t-request, kv head): first d-unit, one past the last
  PH_N_PARTIAL,       // units that leave partial rows for the merge: t-units and d-units that are not final, and all w-units
  PH_WORDS = 32
};

// per query
enum {
  PQ_TREQ = 0,        // t-request index or -1
  PQ_TIDX,            // row-thread index inside the t-request
  PQ_WUNIT0,          // first w-unit of this query; w-unit of (kv head g, piece k) = WUNIT0 + g * NW + k
  PQ_NW,              // w-units per kv head
  PQ_WORDS
};

// per t-request
enum {
  PT_PAGE_OFF = 0,    // index into pages / pmeta
  PT_N_PAGES,
  PT_N_THREADS,
  PT_N_STREAMS,
  PT_VIS_OFF,         // index into vis
  PT_TQ_OFF,          // index into tq
  PT_WORDS
};

// per t-unit.  The t-request's fields are repeated here so that a kernel role learns everything about its next unit
// from one record (12 words, three 16-byte loads issued together) instead of following a second pointer.
enum {
  PU_TREQ = 0,
  PU_KV_HEAD,
  PU_TILE_BEGIN,
  PU_TILE_END,
  PU_ROW_BASE,
  PU_PAGE_OFF,        // = PT_PAGE_OFF of the t-request, and so on
  PU_N_PAGES,
  PU_N_THREADS,
  PU_N_STREAMS,
  PU_VIS_OFF,
  PU_TQ_OFF,
  PU_FINAL,           // 1: the unit's rows are the whole result of their (query, head) pairs
  PU_WORDS
};
static_assert(PU_WORDS == 12, "t-unit records are read as three int4");

// per w-unit
enum {
  PW_QUERY = 0,
  PW_KV_HEAD,
  PW_PAGE_OFF,        // index into pages of the unit's first page
  PW_N_TOKENS,        // tokens of the unit, starting at the first token of that page
  PW_WORDS
};
