#include "pool.hpp"

#include <algorithm>

namespace pasta {

HostPool::HostPool(int32_t n_pages, int32_t page_size, const int32_t *free_order,
                   int32_t max_requests, int32_t max_threads, int32_t max_segments)
    : n_pages_(n_pages), page_size_(page_size), max_requests_(max_requests),
      max_threads_(max_threads), max_segments_(max_segments), requests_(max_requests) {
  for (int32_t i = 0; i < n_pages; ++i) free_.push_back(free_order ? free_order[i] : i);
}

bool HostPool::valid_free_order(int32_t n_pages, const int32_t *free_order) {
  if (!free_order) return true;
  std::vector<char> seen(n_pages, 0);
  for (int32_t i = 0; i < n_pages; ++i) {
    int32_t p = free_order[i];
    if (p < 0 || p >= n_pages || seen[p]) return false;
    seen[p] = 1;
  }
  return true;
}

Request *HostPool::live(int32_t req) {
  if (req < 0 || req >= max_requests_ || !requests_[req].live) return nullptr;
  return &requests_[req];
}

const Request *HostPool::request(int32_t req) const {
  if (req < 0 || req >= max_requests_ || !requests_[req].live) return nullptr;
  return &requests_[req];
}

pasta_status_t HostPool::request_begin(int32_t *out_req) {
  for (int32_t r = 0; r < max_requests_; ++r) {
    if (requests_[r].live) continue;
    Request &q = requests_[r];
    q.live = true;
    q.streams.assign(1, Stream());
    q.threads.assign(1, Thread());
    *out_req = r;
    return PASTA_OK;
  }
  return PASTA_ERR_CAPACITY;
}

pasta_status_t HostPool::request_end(int32_t req) {
  Request *r = live(req);
  if (!r) return PASTA_ERR_INVALID_ARG;
  for (const Stream &s : r->streams)
    for (int32_t page : s.pages) free_.push_front(page);
  r->live = false;
  r->streams.clear();
  r->threads.clear();
  return PASTA_OK;
}

pasta_status_t HostPool::thread_spawn(int32_t req, int32_t predicted_tokens, int32_t pending, int32_t *out_thread) {
  Request *r = live(req);
  if (!r || predicted_tokens < 0 || (pending != 0 && pending != 1)) return PASTA_ERR_INVALID_ARG;
  int32_t t = static_cast<int32_t>(r->threads.size());
  if (t >= max_threads_) return PASTA_ERR_CAPACITY;
  if (pending && !can_extend(*r, 0)) return PASTA_ERR_CAPACITY;
  Thread fork;
  Thread &main_thread = r->threads[0];
  const int32_t len0 = r->streams[0].len;
  fork.cutoff = len0 + pending;
  fork.view = main_thread.view;            // frozen snapshot of what the main thread sees now
  if (pending) {                           // ... plus the promise it is about to append
    if (!fork.view.empty() && fork.view.back().stream == 0 && fork.view.back().start + fork.view.back().len == len0)
      fork.view.back().len += 1;
    else
      fork.view.push_back(Seg{0, len0, 1, -1});
    fork.pos_next = main_thread.pos_next + 1;    // the promise takes pos_next, the fork continues behind it
    main_thread.pos_skip += predicted_tokens;    // the main thread jumps once the promise is in
  } else {
    fork.pos_next = main_thread.pos_next;        // the fork continues right after the promise ...
    main_thread.pos_next += predicted_tokens;    // ... and the main thread skips the predicted block
  }
  r->threads.push_back(std::move(fork));
  r->streams.push_back(Stream());
  *out_thread = t;
  return PASTA_OK;
}

pasta_status_t HostPool::thread_finish(int32_t req, int32_t thread) {
  Request *r = live(req);
  if (!r || thread <= 0 || thread >= static_cast<int32_t>(r->threads.size()))
    return PASTA_ERR_INVALID_ARG;
  if (r->threads[thread].state != PASTA_THREAD_ACTIVE) return PASTA_ERR_BAD_STATE;
  r->threads[thread].state = PASTA_THREAD_FINISHED;
  return PASTA_OK;
}

bool HostPool::can_extend(const Request &r, int32_t thread) const {
  const std::vector<Seg> &view = r.threads[thread].view;
  if (!view.empty()) {
    const Seg &last = view.back();
    if (last.stream == thread && last.start + last.len == r.streams[thread].len) return true;
  }
  return static_cast<int32_t>(view.size()) < max_segments_;
}

Slot HostPool::append_one(Request &r, int32_t thread) {
  Stream &s = r.streams[thread];
  const int32_t k = s.len;
  if (k % page_size_ == 0) {
    s.pages.push_back(free_.front());
    free_.pop_front();
  }
  Slot slot{s.pages[k / page_size_], k % page_size_, 0};
  s.len = k + 1;
  Thread &th = r.threads[thread];
  th.pos_last = th.pos_next;
  th.pos_next += 1 + th.pos_skip;
  th.pos_skip = 0;
  std::vector<Seg> &view = r.threads[thread].view;
  if (!view.empty() && view.back().stream == thread && view.back().start + view.back().len == k)
    view.back().len += 1;
  else
    view.push_back(Seg{thread, k, 1, -1});
  return slot;
}

void HostPool::undo_step(const std::vector<StepUndo> &undo) {
  for (auto it = undo.rbegin(); it != undo.rend(); ++it) {
    Request &r = requests_[it->req];
    Stream &s = r.streams[it->thread];
    while (static_cast<int32_t>(s.pages.size()) > it->n_pages) {     // last taken, first back: the old order returns
      free_.push_front(s.pages.back());
      s.pages.pop_back();
    }
    s.len = it->len;
    Thread &th = r.threads[it->thread];
    th.view.resize(it->view_size);
    if (it->view_size > 0) th.view.back().len = it->last_len;
    th.pos_next = it->pos_next; th.pos_last = it->pos_last; th.pos_skip = it->pos_skip;
  }
}

pasta_status_t HostPool::reserve_step(const std::vector<StepEntry> &entries, std::vector<StepQuery> *queries,
                                      std::vector<Slot> *slots, std::vector<StepUndo> *undo) {
  // pass 1: validate everything, count pages
  size_t need = 0;
  std::vector<std::pair<int32_t, int32_t>> seen;
  seen.reserve(entries.size());
  for (const StepEntry &e : entries) {
    Request *r = live(e.req);
    if (!r) return PASTA_ERR_INVALID_ARG;
    if (e.thread < 0 || e.thread >= static_cast<int32_t>(r->threads.size())) return PASTA_ERR_INVALID_ARG;
    if (e.n_new < 0) return PASTA_ERR_INVALID_ARG;
    seen.emplace_back(e.req, e.thread);
  }
  {
    std::vector<std::pair<int32_t, int32_t>> sorted = seen;
    std::sort(sorted.begin(), sorted.end());
    // the first duplicate in list order decides nothing about the code: any duplicate is INVALID_ARG
    if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return PASTA_ERR_INVALID_ARG;
  }
  for (const StepEntry &e : entries) {
    Request *r = live(e.req);
    const Thread &t = r->threads[e.thread];
    if (t.state != PASTA_THREAD_ACTIVE) return PASTA_ERR_INVALID_ARG;
    if (e.n_new) {   // pages opened by tokens len .. len + n_new - 1
      const int64_t len = r->streams[e.thread].len, P = page_size_;
      need += static_cast<size_t>((len + e.n_new + P - 1) / P - (len + P - 1) / P);
    }
    if (!e.n_new && t.view.empty()) return PASTA_ERR_INVALID_ARG;
    if (e.n_new && !can_extend(*r, e.thread)) return PASTA_ERR_CAPACITY;
  }
  for (const StepEntry &e : entries) {     // a fork spawned on a pending promise needs that promise in the pool
    if (e.thread == 0) continue;
    const Request *r = live(e.req);
    int32_t main_len = r->streams[0].len;
    if (r->threads[e.thread].cutoff > main_len) {
      for (const StepEntry &o : entries)
        if (o.req == e.req && o.thread == 0 && o.n_new) { main_len += o.n_new; break; }
      if (r->threads[e.thread].cutoff > main_len) return PASTA_ERR_BAD_STATE;
    }
  }
  if (need > free_.size()) return PASTA_ERR_OUT_OF_PAGES;
  // pass 2: commit
  slots->clear();
  queries->clear();
  if (undo) undo->clear();
  for (const StepEntry &e : entries) {
    Request &r = requests_[e.req];
    if (undo && e.n_new > 0) {
      const Thread &th = r.threads[e.thread];
      undo->push_back(StepUndo{e.req, e.thread, r.streams[e.thread].len, static_cast<int32_t>(r.streams[e.thread].pages.size()),
                               static_cast<int32_t>(th.view.size()), th.view.empty() ? 0 : th.view.back().len,
                               th.pos_next, th.pos_last, th.pos_skip});
    }
    if (e.n_new == 0) {
      slots->push_back(Slot{-1, -1, query_position(r.threads[e.thread])});
      queries->push_back(StepQuery{e.req, e.thread, 0});
    }
    for (int32_t j = 0; j < e.n_new; ++j) {
      Slot s = append_one(r, e.thread);
      s.pos = r.threads[e.thread].pos_last;
      slots->push_back(s);
      queries->push_back(StepQuery{e.req, e.thread, e.n_new - 1 - j});
    }
  }
  return PASTA_OK;
}

pasta_status_t HostPool::reserve_run(int32_t req, int32_t thread, int32_t m, std::vector<Slot> *slots) {
  Request *r = live(req);
  if (!r || thread < 0 || thread >= static_cast<int32_t>(r->threads.size()) || m < 0)
    return PASTA_ERR_INVALID_ARG;
  if (r->threads[thread].state != PASTA_THREAD_ACTIVE) return PASTA_ERR_INVALID_ARG;
  if (thread != 0 && r->threads[thread].cutoff > r->streams[0].len) return PASTA_ERR_BAD_STATE;
  const int64_t n = r->streams[thread].len;
  const int64_t P = page_size_;
  const int64_t need = (n + m + P - 1) / P - (n + P - 1) / P;
  if (need > static_cast<int64_t>(free_.size())) return PASTA_ERR_OUT_OF_PAGES;
  if (m > 0 && !can_extend(*r, thread)) return PASTA_ERR_CAPACITY;
  slots->clear();
  slots->reserve(m);
  for (int32_t i = 0; i < m; ++i) slots->push_back(append_one(*r, thread));
  return PASTA_OK;
}

pasta_status_t HostPool::sync_merge(int32_t req, int32_t n_threads, const int32_t *thread_ids) {
  Request *r = live(req);
  if (!r) return PASTA_ERR_INVALID_ARG;
  const int32_t n_known = static_cast<int32_t>(r->threads.size());
  std::vector<int32_t> forks;
  if (n_threads < 0) {
    for (int32_t t = 1; t < n_known; ++t)
      if (r->threads[t].state == PASTA_THREAD_FINISHED) forks.push_back(t);
  } else {
    if (n_threads > 0 && !thread_ids) return PASTA_ERR_INVALID_ARG;
    forks.assign(thread_ids, thread_ids + n_threads);
    std::sort(forks.begin(), forks.end());
    if (std::adjacent_find(forks.begin(), forks.end()) != forks.end()) return PASTA_ERR_INVALID_ARG;
    for (int32_t t : forks)
      if (t <= 0 || t >= n_known || r->threads[t].state == PASTA_THREAD_MERGED) return PASTA_ERR_INVALID_ARG;
    for (int32_t t : forks)
      if (r->threads[t].state != PASTA_THREAD_FINISHED) return PASTA_ERR_BAD_STATE;
  }
  for (int32_t t : forks)
    if (r->threads[t].cutoff > r->streams[0].len) return PASTA_ERR_BAD_STATE;   // its promise never arrived
  std::vector<Seg> view = r->threads[0].view;   // work on a copy: all or nothing
  for (int32_t t : forks) {                     // ascending id
    const int32_t len = r->streams[t].len;
    if (len == 0) continue;                     // an empty chunk leaves no entry
    const int32_t p = r->threads[t].cutoff;
    for (size_t i = 0; i < view.size(); ++i) {  // split the main piece that has p strictly inside
      const Seg s = view[i];
      if (s.stream == 0 && s.start < p && p < s.start + s.len) {
        view[i] = Seg{0, s.start, p - s.start, -1};
        view.insert(view.begin() + i + 1, Seg{0, p, s.start + s.len - p, -1});
        break;
      }
    }
    size_t at = view.size();
    for (size_t i = 0; i < view.size(); ++i) {
      const Seg &s = view[i];
      const bool behind = (s.stream == 0) ? (s.start >= p)
                                          : (s.anchor > p || (s.anchor == p && s.stream > t));
      if (behind) { at = i; break; }
    }
    view.insert(view.begin() + at, Seg{t, 0, len, p});
  }
  if (static_cast<int32_t>(view.size()) > max_segments_) return PASTA_ERR_CAPACITY;
  r->threads[0].view.swap(view);
  for (int32_t t : forks) r->threads[t].state = PASTA_THREAD_MERGED;
  return PASTA_OK;
}

void HostPool::dump(std::vector<int32_t> *w) const {
  w->clear();
  int32_t n_live = 0;
  for (const Request &r : requests_) n_live += r.live;
  w->push_back(n_live);
  for (int32_t id = 0; id < max_requests_; ++id) {
    const Request &r = requests_[id];
    if (!r.live) continue;
    w->push_back(id);
    w->push_back(static_cast<int32_t>(r.streams.size()));
    for (size_t s = 0; s < r.streams.size(); ++s) {
      w->push_back(static_cast<int32_t>(s));
      w->push_back(r.streams[s].len);
      w->push_back(static_cast<int32_t>(r.streams[s].pages.size()));
      w->insert(w->end(), r.streams[s].pages.begin(), r.streams[s].pages.end());
    }
    w->push_back(static_cast<int32_t>(r.threads.size()));
    for (size_t t = 0; t < r.threads.size(); ++t) {
      const Thread &th = r.threads[t];
      w->push_back(static_cast<int32_t>(t));
      w->push_back(th.state);
      w->push_back(th.cutoff);
      w->push_back(th.pos_next);
      w->push_back(static_cast<int32_t>(th.view.size()));
      for (const Seg &s : th.view) {
        w->push_back(s.stream);
        w->push_back(s.start);
        w->push_back(s.len);
      }
    }
  }
  w->push_back(static_cast<int32_t>(free_.size()));
  w->insert(w->end(), free_.begin(), free_.end());
}

}  // namespace pasta
