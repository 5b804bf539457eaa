// Builds the step plan (see pasta_plan.h) from the pool's bookkeeping.  Host only.
#include "plan.hpp"

#include <algorithm>
#include <cmath>

namespace pasta {

// A small step's runs stay whole while the longest is at most this many tiles longer than an even share.  Measured on
// one response with 10-tile runs: a CTA that walks a run alone needs 2.9 us per tile more, the merge kernel that cutting
// brings with it 10.7 us, so cutting pays from the fourth tile on.
constexpr int32_t kWholeRunSlackTiles = 3;


namespace {

struct StreamUse {
  int32_t stream;
  int32_t n_seen;                 // queries of the step that see a non-empty prefix of it
  int32_t max_vis;
  int32_t local = -1;             // index among the t-request's shared streams
  int32_t page_off = -1;          // where its pages were put in the page table (w-units)
};

struct WPiece {                   // one stream read by one query on the warp path
  int32_t query, page_off, vis;
};

struct TReq {
  int32_t page_off, n_pages, n_threads, n_streams, vis_off, tq_off;
};

struct TUnit {
  int32_t treq, g, tile_begin, tile_end, row_base;
};

}  // namespace

// the same step planned with every tile assigned in advance: what is left when the shared tail does not fit the
// pool's capacities (it adds units, hence partial rows and plan words)
static pasta_status_t without_tail(const HostPool &pool, const std::vector<StepQuery> &entries,
                                   const std::vector<Slot> &slots, PlanLimits lim, std::vector<int32_t> *out) {
  lim.tail_percent = 0;
  return build_plan(pool, entries, slots, lim, out);
}

pasta_status_t build_plan(const HostPool &pool, const std::vector<StepQuery> &entries,
                          const std::vector<Slot> &slots, const PlanLimits &lim,
                          std::vector<int32_t> *out) {
  const int32_t n = static_cast<int32_t>(entries.size());
  const int32_t G = lim.n_q_heads / lim.n_kv_heads;
  const int32_t P = PASTA_PAGE;
  if (n > lim.max_queries) return PASTA_ERR_CAPACITY;

  // Scratch that keeps its capacity from one step to the next (a pool plans a step at a time; the planner of another
  // pool on another host thread has its own): this function runs once per decode step and most of what it does is
  // small.
  static thread_local std::vector<int32_t> req_order, slot_of, group_begin, order, vis_of, use_index, q_vis;
  static thread_local std::vector<StreamUse> uses;
  static thread_local std::vector<int32_t> pages, pmeta, vis_tab, tq_tab;

  // ---- group the queries by request, in order of first appearance: order[group_begin[g] .. group_begin[g + 1])
  req_order.clear();
  slot_of.clear();
  group_begin.clear();
  for (int32_t i = 0; i < n; ++i) {
    const int32_t r = entries[i].req;
    if (r >= static_cast<int32_t>(slot_of.size())) slot_of.resize(r + 1, -1);
    if (slot_of[r] < 0) {
      slot_of[r] = static_cast<int32_t>(req_order.size());
      req_order.push_back(r);
      group_begin.push_back(0);
    }
    group_begin[slot_of[r]] += 1;
  }
  {
    int32_t at = 0;
    for (int32_t &b : group_begin) { const int32_t c = b; b = at; at += c; }
    group_begin.push_back(at);
    order.assign(n, 0);
    std::vector<int32_t> &fill = vis_of;          // borrowed as the groups' fill counters
    fill.assign(req_order.size(), 0);
    for (int32_t i = 0; i < n; ++i) {
      const int32_t g = slot_of[entries[i].req];
      order[group_begin[g] + fill[g]++] = i;
    }
  }

  pages.clear(); pmeta.clear(); vis_tab.clear(); tq_tab.clear();
  std::vector<TReq> treqs;
  std::vector<WPiece> wpieces;
  std::vector<int32_t> q_treq(n, -1), q_tidx(n, 0);
  int64_t w_tokens = 0;

  for (size_t gi = 0; gi < req_order.size(); ++gi) {
    const Request *r = pool.request(req_order[gi]);
    const int32_t *qs = order.data() + group_begin[gi];
    const int32_t T = group_begin[gi + 1] - group_begin[gi];
    const int32_t n_streams_all = static_cast<int32_t>(r->streams.size());
    // the streams the step's threads of this request read, in order of first appearance in their views
    use_index.assign(n_streams_all, -1);
    uses.clear();
    for (int32_t ti = 0; ti < T; ++ti)
      for (const Seg &sg : r->threads[entries[qs[ti]].thread].view)
        if (use_index[sg.stream] < 0) {
          use_index[sg.stream] = static_cast<int32_t>(uses.size());
          uses.push_back(StreamUse{sg.stream, 0, 0});
        }
    const int32_t U = static_cast<int32_t>(uses.size());
    // q_vis[ti * U + u]: how much of stream uses[u] query ti sees
    q_vis.assign(static_cast<size_t>(T) * U, 0);
    for (int32_t ti = 0; ti < T; ++ti) {
      const StepQuery &e = entries[qs[ti]];
      int32_t *row = q_vis.data() + static_cast<size_t>(ti) * U;
      for (const Seg &sg : r->threads[e.thread].view) {
        int32_t &v = row[use_index[sg.stream]];
        v = std::max(v, sg.start + sg.len);
      }
      // a query for an earlier one of several tokens appended in this step does not see the later ones: they are
      // the end of the thread's own stream (stream id = thread id)
      if (e.hide && use_index[e.thread] >= 0) row[use_index[e.thread]] -= e.hide;
      for (int32_t u = 0; u < U; ++u)
        if (row[u] > 0) {
          // count each (query, stream) once: views list a stream several times only for the main stream pieces
          uses[u].n_seen += 1;
          uses[u].max_vis = std::max(uses[u].max_vis, row[u]);
        }
    }

    // A request whose stacked rows fit one MMA tile sends EVERY stream it reads through the tensor-core kernel, the
    // private chunks too: rows that may not see a page are masked there, the MMA costs the same for any number of
    // valid rows, and the pass stays bandwidth-bound; the warp kernel is left with what does not fit.
    bool tensor = lim.tensor_path && T >= 1 && T * G <= PASTA_MAX_ROWS;
    int32_t n_shared = 0;
    if (tensor) {
      bool too_long = false;                 // a page's meta word has 18 bits for its index within the stream
      for (StreamUse &u : uses)
        if (u.n_seen >= 1) { u.local = n_shared++; too_long = too_long || (u.max_vis + P - 1) / P > PASTA_MAX_STREAM_PAGES; }
      if (n_shared == 0 || n_shared > PASTA_MAX_STREAMS || too_long) {
        tensor = false;
        for (StreamUse &u : uses) u.local = -1;
      }
    }
    if (tensor) {
      TReq t;
      t.page_off = static_cast<int32_t>(pages.size());
      t.n_threads = T;
      t.n_streams = n_shared;
      t.vis_off = static_cast<int32_t>(vis_tab.size());
      t.tq_off = static_cast<int32_t>(tq_tab.size());
      for (size_t ui = 0; ui < uses.size(); ++ui) {
        const StreamUse &u = uses[ui];
        if (u.local < 0) continue;
        const std::vector<int32_t> &sp = r->streams[u.stream].pages;
        const int32_t np = (u.max_vis + P - 1) / P;
        int32_t min_vis = u.max_vis;             // what EVERY thread of the request sees of this stream
        for (int32_t ti = 0; ti < T; ++ti) min_vis = std::min(min_vis, q_vis[static_cast<size_t>(ti) * U + ui]);
        pages.insert(pages.end(), sp.begin(), sp.begin() + np);
        const size_t m0 = pmeta.size();
        pmeta.resize(m0 + np);
        int32_t *pm = pmeta.data() + m0;
        const int32_t n_all = std::min(np, min_vis / P);     // pages every thread of the request sees in full
        for (int32_t k = 0; k < n_all; ++k) pm[k] = (k << PASTA_PMETA_STREAM_BITS) | u.local | PASTA_PMETA_ALL_VISIBLE;
        for (int32_t k = n_all; k < np; ++k) pm[k] = (k << PASTA_PMETA_STREAM_BITS) | u.local;
      }
      t.n_pages = static_cast<int32_t>(pages.size()) - t.page_off;
      for (int32_t ti = 0; ti < T; ++ti) {
        for (size_t u = 0; u < uses.size(); ++u)
          if (uses[u].local >= 0) vis_tab.push_back(q_vis[static_cast<size_t>(ti) * U + u]);   // uses are in local order
        tq_tab.push_back(qs[ti]);
        q_treq[qs[ti]] = static_cast<int32_t>(treqs.size());
        q_tidx[qs[ti]] = ti;
      }
      treqs.push_back(t);
    }
    // streams that stay on the warp path: their pages are stored once per request
    for (int32_t ti = 0; ti < T; ++ti) {
      for (size_t u = 0; u < uses.size(); ++u) {
        if (uses[u].local >= 0 || q_vis[static_cast<size_t>(ti) * U + u] == 0) continue;
        if (uses[u].page_off < 0) {
          uses[u].page_off = static_cast<int32_t>(pages.size());
          const std::vector<int32_t> &sp = r->streams[uses[u].stream].pages;
          const int32_t np = (uses[u].max_vis + P - 1) / P;
          pages.insert(pages.end(), sp.begin(), sp.begin() + np);
          pmeta.insert(pmeta.end(), np, 0);
        }
        wpieces.push_back(WPiece{qs[ti], uses[u].page_off, q_vis[static_cast<size_t>(ti) * U + u]});
        w_tokens += q_vis[static_cast<size_t>(ti) * U + u];
      }
    }
  }

  // ---- t-units: cut the sequence of (t-request, kv head) tile runs into one contiguous range per CTA
  static thread_local std::vector<TUnit> tunits, dunits;
  static thread_local std::vector<int32_t> trange, drange, tcta, unit_cta, tail;
  tunits.clear(); dunits.clear(); tcta.clear(); unit_cta.clear();
  trange.assign(treqs.size() * lim.n_kv_heads * 2, 0);
  drange.assign(treqs.size() * lim.n_kv_heads * 2, 0);
  int32_t t_rows = 0;
  if (!treqs.empty()) {
    // Some of the work is kept back from the assignment below, as units which the CTAs share out among themselves at
    // run time (equal tile counts do not finish at the same time: SMs differ in the bandwidth they get).  Only when
    // there is enough work for that to matter.
    int64_t all_tiles = 0;
    for (const TReq &t : treqs) all_tiles += int64_t(lim.n_kv_heads) * ((t.n_pages + PASTA_TILE_PAGES - 1) / PASTA_TILE_PAGES);
    const bool share_tail = lim.tail_percent > 0 && lim.tail_tiles > 0 && all_tiles >= 16LL * std::max(1, lim.grid);
    // Runs of a few tiles go to the pool whole, every so often, until the pool holds its share of their tiles (`owed`
    // counts what they still owe it): a whole run is a unit anyway, so sharing it costs no extra cut and no extra
    // partial rows.  Long runs stay assigned: cutting their ends into short units cost more, in unit changes and
    // partial rows, than the evener finish gave back (measured on 8 x 32768-token prefixes).
    tail.assign(treqs.size() * lim.n_kv_heads, 0);
    if (share_tail) {
      int64_t owed = 0;
      for (size_t ti = 0; ti < treqs.size(); ++ti) {
        const int32_t n_tiles = (treqs[ti].n_pages + PASTA_TILE_PAGES - 1) / PASTA_TILE_PAGES;
        if (n_tiles > 4 * lim.tail_tiles) continue;
        for (int32_t g = 0; g < lim.n_kv_heads; ++g) {
          owed += int64_t(n_tiles) * lim.tail_percent;
          if (owed >= int64_t(n_tiles) * 100) { tail[ti * lim.n_kv_heads + g] = n_tiles; owed -= int64_t(n_tiles) * 100; }
        }
      }
    }
    const double overhead = 1.0;
    const int32_t min_piece = 1;
    double total = 0;
    for (size_t ti = 0; ti < treqs.size(); ++ti) {
      const int32_t n_tiles = (treqs[ti].n_pages + PASTA_TILE_PAGES - 1) / PASTA_TILE_PAGES;
      for (int32_t g = 0; g < lim.n_kv_heads; ++g) {
        const int32_t kept = n_tiles - tail[ti * lim.n_kv_heads + g];
        if (kept > 0) total += kept + overhead;
      }
    }
    const int32_t grid = std::max(1, lim.grid);
    const double target = std::max(total, 1.0) / grid;
    double cum = 0;
    // A small step (one response, a few threads, a context of a few hundred tokens) is not cut at all when every run can
    // have a CTA of its own and the longest run is hardly longer than an even share: a cut run leaves partial rows and
    // needs the merge kernel behind the attention kernel, whole runs are final units whose rows leave the attention
    // kernel as the output.
    bool whole_runs = false;
    {
      int64_t n_runs = 0, kept_tiles = 0;
      int32_t longest = 0;
      for (size_t ti = 0; ti < treqs.size(); ++ti) {
        const int32_t all = (treqs[ti].n_pages + PASTA_TILE_PAGES - 1) / PASTA_TILE_PAGES;
        for (int32_t g = 0; g < lim.n_kv_heads; ++g) {
          const int32_t kept = all - tail[ti * lim.n_kv_heads + g];
          if (kept > 0) { ++n_runs; kept_tiles += kept; longest = std::max(longest, kept); }
        }
      }
      whole_runs = n_runs > 0 && n_runs <= grid && longest <= kept_tiles / grid + kWholeRunSlackTiles;
    }
    int32_t run_no = 0;
    for (size_t ti = 0; ti < treqs.size(); ++ti) {
      const int32_t all = (treqs[ti].n_pages + PASTA_TILE_PAGES - 1) / PASTA_TILE_PAGES;
      const int32_t rows = treqs[ti].n_threads * G;
      for (int32_t g = 0; g < lim.n_kv_heads; ++g) {
        const int32_t n_tiles = all - tail[ti * lim.n_kv_heads + g];       // what is assigned to CTAs here
        trange[(ti * lim.n_kv_heads + g) * 2] = static_cast<int32_t>(tunits.size());
        if (n_tiles > 0) cum += overhead;
        int32_t begin = 0;
        while (begin < n_tiles) {
          const int32_t remaining = n_tiles - begin;
          if (whole_runs) {                      // one run, one unit, one CTA
            tunits.push_back(TUnit{static_cast<int32_t>(ti), g, 0, n_tiles, t_rows});
            unit_cta.push_back(run_no++);
            t_rows += rows;
            break;
          }
          int32_t c = std::min<int32_t>(grid - 1, static_cast<int32_t>(cum / target));
          if (c + 1 < grid && (c + 1) * target - cum < min_piece) ++c;   // too close to the CTA's end: next one
          int32_t take = remaining;
          if (c + 1 < grid) {
            const double room = (c + 1) * target - cum;
            take = std::min<int32_t>(remaining, std::max<int32_t>(min_piece, static_cast<int32_t>(std::lround(room))));
            if (remaining - take < min_piece) take = remaining;
          }
          tunits.push_back(TUnit{static_cast<int32_t>(ti), g, begin, begin + take, t_rows});
          unit_cta.push_back(c);
          t_rows += rows;
          begin += take;
          cum += take;
        }
        trange[(ti * lim.n_kv_heads + g) * 2 + 1] = static_cast<int32_t>(tunits.size());
        drange[(ti * lim.n_kv_heads + g) * 2] = static_cast<int32_t>(dunits.size());
        for (int32_t b2 = n_tiles; b2 < all; b2 += lim.tail_tiles) {
          dunits.push_back(TUnit{static_cast<int32_t>(ti), g, b2, std::min(all, b2 + lim.tail_tiles), t_rows});
          t_rows += rows;
        }
        drange[(ti * lim.n_kv_heads + g) * 2 + 1] = static_cast<int32_t>(dunits.size());
      }
    }
    for (size_t u = 0; u < tunits.size(); ++u) {
      if (u == 0 || unit_cta[u] != unit_cta[u - 1]) {
        if (!tcta.empty()) tcta.back() = static_cast<int32_t>(u);
        tcta.push_back(static_cast<int32_t>(u));
        tcta.push_back(static_cast<int32_t>(u));
      }
    }
    if (!tcta.empty()) tcta.back() = static_cast<int32_t>(tunits.size());
    // every CTA of the grid takes part in sharing out the tail, also those that were assigned nothing
    while (!dunits.empty() && static_cast<int32_t>(tcta.size() / 2) < grid) {
      tcta.push_back(static_cast<int32_t>(tunits.size()));
      tcta.push_back(static_cast<int32_t>(tunits.size()));
    }
  }

  // ---- w-units: pieces of at most `chunk` tokens, ordered (query, kv head, piece)
  int32_t chunk;
  {
    const double want_warps = 16.0 * std::max(1, lim.grid);
    double c = std::ceil(static_cast<double>(w_tokens) * lim.n_kv_heads / want_warps / P) * P;
    chunk = static_cast<int32_t>(std::min(1024.0, std::max(64.0, c)));
  }
  std::vector<int32_t> q_nw(n, 0), q_w0(n, 0);
  int64_t n_wunits = 0;
  for (;;) {
    std::fill(q_nw.begin(), q_nw.end(), 0);
    for (const WPiece &w : wpieces) q_nw[w.query] += (w.vis + chunk - 1) / chunk;
    n_wunits = 0;
    for (int32_t i = 0; i < n; ++i) n_wunits += static_cast<int64_t>(q_nw[i]) * lim.n_kv_heads;
    if (t_rows + n_wunits * G <= lim.max_rows) break;
    if (!dunits.empty()) return without_tail(pool, entries, slots, lim, out);    // the shared tail costs rows: do without
    if (chunk >= (1 << 24)) return PASTA_ERR_CAPACITY;
    chunk *= 2;
  }
  {
    int32_t w0 = 0;
    for (int32_t i = 0; i < n; ++i) { q_w0[i] = w0; w0 += q_nw[i] * lim.n_kv_heads; }
  }
  std::vector<int32_t> wunits(static_cast<size_t>(n_wunits) * PW_WORDS);
  {
    std::vector<int32_t> next(n, 0);       // next piece index k of each query
    // pieces of one query are contiguous in wpieces only per request group; index by query instead
    for (const WPiece &w : wpieces) {
      for (int32_t begin = 0; begin < w.vis; begin += chunk) {
        const int32_t k = next[w.query]++;
        for (int32_t g = 0; g < lim.n_kv_heads; ++g) {
          int32_t *u = &wunits[static_cast<size_t>(q_w0[w.query] + g * q_nw[w.query] + k) * PW_WORDS];
          u[PW_QUERY] = w.query;
          u[PW_KV_HEAD] = g;
          u[PW_PAGE_OFF] = w.page_off + begin / P;
          u[PW_N_TOKENS] = std::min(chunk, w.vis - begin);
        }
      }
    }
  }

  // ---- assemble
  int32_t n_app = 0;
  for (const Slot &s : slots) n_app += s.page >= 0;
  std::vector<int32_t> &w = *out;
  w.clear();
  w.reserve(PH_WORDS + pages.size() + pmeta.size() + vis_tab.size() + tq_tab.size() + trange.size() + tcta.size() +
            wunits.size() + tunits.size() * PU_WORDS + treqs.size() * PT_WORDS + static_cast<size_t>(n) * (PQ_WORDS + 4) +
            64);
  w.assign(PH_WORDS, 0);
  auto put = [&](int off_field, const std::vector<int32_t> &v) {
    w[off_field] = static_cast<int32_t>(w.size());
    w.insert(w.end(), v.begin(), v.end());
    while (w.size() % 4) w.push_back(0);   // keep every table 16-byte aligned
  };
  static thread_local std::vector<int32_t> app, apos, qpos, qtab, ttab, utab, dtab;
  app.clear(); apos.clear(); qpos.clear(); ttab.clear(); utab.clear(); dtab.clear();
  for (int32_t i = 0; i < n; ++i) {
    const int32_t pos = slots[i].pos;
    qpos.push_back(pos);
    if (slots[i].page >= 0) { app.push_back(slots[i].page); app.push_back(slots[i].offset); apos.push_back(pos); }
  }
  qtab.assign(static_cast<size_t>(n) * PQ_WORDS, 0);
  for (int32_t i = 0; i < n; ++i) {
    qtab[i * PQ_WORDS + PQ_TREQ] = q_treq[i];
    qtab[i * PQ_WORDS + PQ_TIDX] = q_tidx[i];
    qtab[i * PQ_WORDS + PQ_WUNIT0] = q_w0[i];
    qtab[i * PQ_WORDS + PQ_NW] = q_nw[i];
  }

  for (const TReq &t : treqs) {
    const int32_t rec[PT_WORDS] = {t.page_off, t.n_pages, t.n_threads, t.n_streams, t.vis_off, t.tq_off};
    ttab.insert(ttab.end(), rec, rec + PT_WORDS);
  }
  // a unit is final when nothing else contributes to its rows: it covers its whole run, and no query of its request
  // has streams on the warp path
  auto unit_record = [&](const TUnit &u, std::vector<int32_t> &tab) {
    const TReq &t = treqs[u.treq];
    bool final_rows = u.tile_begin == 0 && u.tile_end == (t.n_pages + PASTA_TILE_PAGES - 1) / PASTA_TILE_PAGES;
    for (int32_t ti = 0; final_rows && ti < t.n_threads; ++ti) final_rows = q_nw[tq_tab[t.tq_off + ti]] == 0;
    const int32_t rec[PU_WORDS] = {u.treq, u.g, u.tile_begin, u.tile_end, u.row_base, t.page_off, t.n_pages,
                                   t.n_threads, t.n_streams, t.vis_off, t.tq_off, final_rows ? 1 : 0};
    tab.insert(tab.end(), rec, rec + PU_WORDS);
  };
  for (const TUnit &u : tunits) unit_record(u, utab);
  for (const TUnit &u : dunits) unit_record(u, dtab);
  int32_t n_partial = static_cast<int32_t>(n_wunits);
  for (size_t i = PU_FINAL; i < utab.size(); i += PU_WORDS) n_partial += utab[i] == 0;
  for (size_t i = PU_FINAL; i < dtab.size(); i += PU_WORDS) n_partial += dtab[i] == 0;
  w[PH_MAGIC] = PASTA_PLAN_MAGIC;
  w[PH_N_DUNITS] = static_cast<int32_t>(dunits.size());
  w[PH_N_PARTIAL] = n_partial;
  w[PH_N_QUERIES] = n;
  w[PH_N_APPEND] = n_app;
  w[PH_N_TREQ] = static_cast<int32_t>(treqs.size());
  w[PH_N_TUNITS] = static_cast<int32_t>(tunits.size());
  w[PH_N_WUNITS] = static_cast<int32_t>(n_wunits);
  w[PH_T_ROWS] = t_rows;
  w[PH_ROWS] = t_rows + static_cast<int32_t>(n_wunits) * G;
  w[PH_T_GRID] = static_cast<int32_t>(tcta.size() / 2);
  put(PH_OFF_APPEND, app);
  put(PH_OFF_QUERY, qtab);
  put(PH_OFF_TREQ, ttab);
  put(PH_OFF_TRANGE, trange);
  put(PH_OFF_TUNIT, utab);
  put(PH_OFF_TCTA, tcta);
  put(PH_OFF_WUNIT, wunits);
  put(PH_OFF_PAGES, pages);
  put(PH_OFF_PMETA, pmeta);
  put(PH_OFF_VIS, vis_tab);
  put(PH_OFF_TQ, tq_tab);
  put(PH_OFF_APOS, apos);
  put(PH_OFF_QPOS, qpos);
  put(PH_OFF_DUNIT, dtab);
  put(PH_OFF_DRANGE, drange);
  w[PH_TOTAL_WORDS] = static_cast<int32_t>(w.size());
  if (static_cast<int64_t>(w.size()) > lim.max_words) {
    if (!dunits.empty()) return without_tail(pool, entries, slots, lim, out);
    return PASTA_ERR_CAPACITY;
  }
  return PASTA_OK;
}

}  // namespace pasta
