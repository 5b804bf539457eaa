// Host-side bookkeeping of the KV pool: pages, streams, threads and their segment lists.
// Pure C++ (no CUDA): everything here is integers.
//
// Rules (Section 3 "Efficiency" of the paper for what a thread may see; paging and canonical
// forms are this library's own):
//  * a stream (main thread's tokens = stream 0, a fork's chunk = stream <fork id>) takes a page
//    from the front of the free sequence whenever it appends a token whose index is a multiple of
//    the page size;
//  * a fork's view = copy of the main thread's view at spawn time + its own chunk;
//  * merging puts a chunk right after the main-stream piece ending at the fork's cut-off,
//    behind chunks with the same cut-off and a smaller id.
#pragma once
#include <cstdint>
#include <deque>
#include <vector>

#include "../../include/pasta.h"

namespace pasta {

struct Seg {
  int32_t stream, start, len;
  int32_t anchor;  // cut-off of a merged chunk; -1 for pieces of the main stream and a fork's own chunk
};

struct Stream {
  int32_t len = 0;
  std::vector<int32_t> pages;
};

struct Thread {
  int32_t state = PASTA_THREAD_ACTIVE;
  int32_t cutoff = 0;
  int32_t pos_next = 0;    // position id of the thread's next token
  int32_t pos_last = -1;   // position id of the thread's newest own token (-1: none yet)
  int32_t pos_skip = 0;    // main thread only: positions to skip once its next token is in
  std::vector<Seg> view;
};

struct Request {
  bool live = false;
  std::vector<Stream> streams;   // index = stream id = thread id
  std::vector<Thread> threads;   // index = thread id; 0 = main
};

struct StepEntry {
  int32_t req, thread, n_new;
};

// One attention query of a step.  An entry that appends m >= 1 tokens issues m queries, one per new token, each
// blind to the tokens appended after its own (`hide` = how many of the thread's newest tokens it may not see);
// an entry that appends nothing issues one query over what the thread sees already.
struct StepQuery {
  int32_t req, thread, hide;
};

// What reserve_step changed for one appending entry, so that the step can be taken back when it cannot be planned.
struct StepUndo {
  int32_t req, thread, len, n_pages, view_size, last_len, pos_next, pos_last, pos_skip;
};

struct Slot {
  int32_t page, offset;   // {-1, -1} for a query without a new token
  int32_t pos;            // position id of the query's token
};

class HostPool {
 public:
  HostPool(int32_t n_pages, int32_t page_size, const int32_t *free_order, int32_t max_requests,
           int32_t max_threads, int32_t max_segments);

  static bool valid_free_order(int32_t n_pages, const int32_t *free_order);

  pasta_status_t request_begin(int32_t *out_req);
  pasta_status_t request_end(int32_t req);
  // pending = 1: the promise is the main thread's next token, decoded but not appended yet; the fork's view
  // counts it in, and the fork may join a step only once that token is in the pool by the step's appends.
  pasta_status_t thread_spawn(int32_t req, int32_t predicted_tokens, int32_t pending, int32_t *out_thread);
  // position id of the token a query of this thread belongs to
  static int32_t query_position(const Thread &t) { return t.pos_last >= 0 ? t.pos_last : t.pos_next - 1; }
  pasta_status_t thread_finish(int32_t req, int32_t thread);
  pasta_status_t sync_merge(int32_t req, int32_t n_threads, const int32_t *thread_ids);

  // Validates the whole step first, then reserves.  Outputs one element per QUERY, in entry order (an entry with
  // n_new tokens contributes max(1, n_new) of them).
  pasta_status_t reserve_step(const std::vector<StepEntry> &entries, std::vector<StepQuery> *queries,
                              std::vector<Slot> *slots, std::vector<StepUndo> *undo = nullptr);
  // Takes a reserve_step back: lengths, page lists, views and position counters as they were, the pages back at
  // the front of the free sequence in the order they had.
  void undo_step(const std::vector<StepUndo> &undo);
  pasta_status_t reserve_run(int32_t req, int32_t thread, int32_t m, std::vector<Slot> *slots);

  const Request *request(int32_t req) const;
  int32_t page_size() const { return page_size_; }
  int32_t n_pages() const { return n_pages_; }
  void dump(std::vector<int32_t> *words) const;

 private:
  bool can_extend(const Request &r, int32_t thread) const;
  Slot append_one(Request &r, int32_t thread);
  Request *live(int32_t req);

  int32_t n_pages_, page_size_, max_requests_, max_threads_, max_segments_;
  std::deque<int32_t> free_;
  std::vector<Request> requests_;
};

}  // namespace pasta
