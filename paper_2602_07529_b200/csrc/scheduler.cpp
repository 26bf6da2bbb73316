// Frontier scheduler (host): Petri-net marking per request, the enabled-transition frontier of Eq. 1, Fork and Join as
// page-table operations with reference counts, and the mv_dag_batch of every decode step (Sec. 3.2, Sec. 3.3,
// Sec. 4.3 Phase II).  Plain C++; no device code.
#include <algorithm>
#include <cstdint>
#include <functional>
#include <new>
#include <queue>
#include <vector>

#include "medverse_sched.h"

namespace {

struct Request {
  int n = 0, words = 0;
  std::vector<int32_t> parent_off, parent_idx, tokens;
  std::vector<uint8_t> marked;        // M_k: place p_v holds its token
  std::vector<int32_t> written;       // running transitions: tokens written so far; -1 otherwise
  std::vector<int32_t> running;       // ascending
  std::vector<int32_t> active;        // the frontier being executed: running, or complete and waiting at the barrier
  std::vector<std::vector<int32_t>> pages;
  std::vector<uint64_t> view;         // [n][words]: the nodes a step reads besides itself (all its ancestors)
  int k = 0;                          // index of the marking
  bool done = false;

  bool is_root(int v) const { return parent_off[v] == parent_off[v + 1]; }
  const uint64_t* view_of(int v) const { return view.data() + size_t(v) * words; }
  bool in_view(int t, int u) const { return (view_of(t)[u >> 6] >> (u & 63)) & 1; }
};

}  // namespace

struct mv_sched {
  int32_t page_size = 16, num_pages = 0;
  std::priority_queue<int32_t, std::vector<int32_t>, std::greater<int32_t>> free_pages;  // lowest id first
  std::vector<int32_t> refs;
  std::vector<Request> requests;
  mv_sched_stats stats{};
  // the emitted step
  bool pending = false;
  std::vector<int32_t> node_off, node_len, node_new, parent_off, parent_idx, page_off, page_idx, row_req, row_node;
  std::vector<uint64_t> shown;

  int32_t alloc() {
    const int32_t p = free_pages.top();
    free_pages.pop();
    refs[size_t(p)] = 1;  // the owning node
    stats.pages_in_use++;
    stats.pages_peak = std::max(stats.pages_peak, stats.pages_in_use);
    return p;
  }
  void unref(int32_t p) {
    if (--refs[size_t(p)] == 0) {
      free_pages.push(p);
      stats.pages_in_use--;
    }
  }
  // what a transition reads is held by reference (Fork, Join): +1 / -1 on every page of every node of its view
  void hold_view(Request& rq, int t, int delta) {
    for (int u = 0; u < t; ++u) {
      if (!rq.in_view(t, u)) continue;
      for (int32_t p : rq.pages[size_t(u)]) {
        if (delta > 0) refs[size_t(p)]++;
        else unref(p);
      }
    }
  }
  // Starts the frontier of the request's current marking (Eq. 1), or, with nothing enabled, releases the request.
  void fire(Request& rq) {
    std::vector<int32_t> frontier;
    for (int t = 0; t < rq.n; ++t) {
      if (rq.is_root(t) || rq.marked[size_t(t)]) continue;  // output place must be empty
      bool enabled = true;
      for (int e = rq.parent_off[t]; e < rq.parent_off[t + 1]; ++e) enabled &= rq.marked[size_t(rq.parent_idx[e])] != 0;
      if (enabled) frontier.push_back(t);
    }
    if (frontier.empty()) {
      rq.done = true;
      stats.requests_live--;
      for (int v = 0; v < rq.n; ++v) {
        for (int32_t p : rq.pages[size_t(v)]) unref(p);
        rq.pages[size_t(v)].clear();
      }
      return;
    }
    // children of every node inside this frontier (a parent listed twice by one child counts once)
    std::vector<int32_t> kids(size_t(rq.n), 0), stamp(size_t(rq.n), -1);
    for (int32_t t : frontier)
      for (int e = rq.parent_off[t]; e < rq.parent_off[t + 1]; ++e) {
        const int32_t p = rq.parent_idx[e];
        if (stamp[size_t(p)] != t) { stamp[size_t(p)] = t; kids[size_t(p)]++; }
      }
    rq.active = frontier;
    for (int32_t t : frontier) {
      rq.written[size_t(t)] = 0;
      rq.running.push_back(t);
      stats.transitions_fired++;
      int distinct = 0;
      bool shares = false;
      const int32_t key = t + rq.n;  // distinct from every stamp of the counting pass
      for (int e = rq.parent_off[t]; e < rq.parent_off[t + 1]; ++e) {
        const int32_t p = rq.parent_idx[e];
        if (stamp[size_t(p)] == key) continue;
        stamp[size_t(p)] = key;
        ++distinct;
        shares |= kids[size_t(p)] >= 2;
      }
      if (distinct >= 2) stats.joins++;
      if (shares) stats.forks++;
      hold_view(rq, t, +1);
    }
  }
};

extern "C" mv_status mv_sched_create(int32_t page_size, int32_t num_pages, mv_sched** sched) {
  if (!sched || page_size != 16 || num_pages < 0) return MV_ERR_INVALID_ARG;
  mv_sched* s = new (std::nothrow) mv_sched();
  if (!s) return MV_ERR_INVALID_ARG;
  s->page_size = page_size;
  s->num_pages = num_pages;
  s->refs.assign(size_t(num_pages), 0);
  for (int32_t p = 0; p < num_pages; ++p) s->free_pages.push(p);
  *sched = s;
  return MV_OK;
}

extern "C" void mv_sched_destroy(mv_sched* sched) { delete sched; }

extern "C" mv_status mv_sched_add_request(mv_sched* s, int32_t n_nodes, const int32_t* parent_off, const int32_t* parent_idx,
                                          const int32_t* node_tokens, int32_t* request_id) {
  if (!s || n_nodes <= 0 || !parent_off || !node_tokens || !request_id) return MV_ERR_INVALID_ARG;
  if (parent_off[0] != 0) return MV_ERR_INVALID_ARG;
  int64_t root_pages = 0;
  for (int v = 0; v < n_nodes; ++v) {
    if (parent_off[v + 1] < parent_off[v]) return MV_ERR_INVALID_ARG;
    if (parent_off[v + 1] > parent_off[v] && !parent_idx) return MV_ERR_INVALID_ARG;
    for (int e = parent_off[v]; e < parent_off[v + 1]; ++e)
      if (parent_idx[e] < 0 || parent_idx[e] >= v) return MV_ERR_NOT_TOPOLOGICAL;
    const bool root = parent_off[v + 1] == parent_off[v];
    if (node_tokens[v] < (root ? 0 : 1)) return MV_ERR_INVALID_ARG;
    if (root) root_pages += (node_tokens[v] + s->page_size - 1) / s->page_size;
  }
  if (s->pending) return MV_ERR_INVALID_ARG;  // between a step and its commit the set of rows is fixed
  if (root_pages > int64_t(s->free_pages.size())) return MV_ERR_PAGE_CAPACITY;
  s->requests.emplace_back();
  Request& rq = s->requests.back();
  rq.n = n_nodes;
  rq.words = (n_nodes + 63) / 64;
  rq.parent_off.assign(parent_off, parent_off + n_nodes + 1);
  rq.parent_idx.assign(parent_idx, parent_idx + parent_off[n_nodes]);
  rq.tokens.assign(node_tokens, node_tokens + n_nodes);
  rq.marked.assign(size_t(n_nodes), 0);
  rq.written.assign(size_t(n_nodes), -1);
  rq.pages.assign(size_t(n_nodes), {});
  rq.view.assign(size_t(n_nodes) * rq.words, 0);
  for (int v = 0; v < n_nodes; ++v) {
    uint64_t* mine = rq.view.data() + size_t(v) * rq.words;
    for (int e = parent_off[v]; e < parent_off[v + 1]; ++e) {  // union of the predecessors' histories
      const int p = parent_idx[e];
      const uint64_t* theirs = rq.view_of(p);
      for (int w = 0; w < rq.words; ++w) mine[w] |= theirs[w];
      mine[p >> 6] |= uint64_t(1) << (p & 63);
    }
    if (rq.is_root(v)) {  // M_0: the context is in the pool already
      rq.marked[size_t(v)] = 1;
      const int np = (node_tokens[v] + s->page_size - 1) / s->page_size;
      for (int i = 0; i < np; ++i) rq.pages[size_t(v)].push_back(s->alloc());
    }
  }
  s->stats.requests_live++;
  *request_id = int32_t(s->requests.size()) - 1;
  s->fire(rq);
  return MV_OK;
}

extern "C" mv_status mv_sched_step(mv_sched* s, mv_dag_batch* b, int32_t* n_rows) {
  if (!s || !b || !n_rows) return MV_ERR_INVALID_ARG;
  if (!s->pending) {
    int64_t need = 0;
    for (const Request& rq : s->requests)
      for (int32_t t : rq.running) need += (rq.written[size_t(t)] % s->page_size) == 0;
    if (need > int64_t(s->free_pages.size())) return MV_ERR_PAGE_CAPACITY;
    s->node_off.assign(1, 0);
    s->parent_off.assign(1, 0);
    s->page_off.assign(1, 0);
    s->node_len.clear(); s->node_new.clear(); s->parent_idx.clear(); s->page_idx.clear();
    s->row_req.clear(); s->row_node.clear();
    std::vector<int32_t> local;
    for (size_t r = 0; r < s->requests.size(); ++r) {
      Request& rq = s->requests[r];
      if (rq.done || rq.running.empty()) continue;
      // a transition whose next token opens a page gets one now
      for (int32_t t : rq.running)
        if (rq.written[size_t(t)] % s->page_size == 0) rq.pages[size_t(t)].push_back(s->alloc());
      // the nodes some running transition reads, and those transitions themselves
      s->shown.assign(size_t(rq.words), 0);
      for (int32_t t : rq.running) {
        const uint64_t* v = rq.view_of(t);
        for (int w = 0; w < rq.words; ++w) s->shown[size_t(w)] |= v[w];
        s->shown[size_t(t >> 6)] |= uint64_t(1) << (t & 63);
      }
      local.assign(size_t(rq.n), -1);
      int32_t next = 0;
      for (int v = 0; v < rq.n; ++v)
        if ((s->shown[size_t(v >> 6)] >> (v & 63)) & 1) local[size_t(v)] = next++;
      for (int v = 0; v < rq.n; ++v) {
        if (local[size_t(v)] < 0) continue;
        const bool runs = rq.written[size_t(v)] >= 0;
        s->node_len.push_back(runs ? rq.written[size_t(v)] : rq.tokens[size_t(v)]);
        s->node_new.push_back(runs ? 1 : 0);
        if (runs) {
          s->row_req.push_back(int32_t(r));
          s->row_node.push_back(v);
        }
        for (int e = rq.parent_off[v]; e < rq.parent_off[v + 1]; ++e) s->parent_idx.push_back(local[size_t(rq.parent_idx[e])]);
        s->parent_off.push_back(int32_t(s->parent_idx.size()));
        s->page_idx.insert(s->page_idx.end(), rq.pages[size_t(v)].begin(), rq.pages[size_t(v)].end());
        s->page_off.push_back(int32_t(s->page_idx.size()));
      }
      s->node_off.push_back(int32_t(s->node_len.size()));
    }
    if (!s->row_req.empty()) {
      s->pending = true;
      s->stats.decode_steps++;
      s->stats.rows_emitted += int64_t(s->row_req.size());
    }
  }
  *b = mv_dag_batch{};
  b->n_req = int32_t(s->node_off.size()) - 1;
  b->node_off = s->node_off.data();
  b->node_len = s->node_len.data();
  b->node_new = s->node_new.data();
  b->parent_off = s->parent_off.data();
  b->parent_idx = s->parent_idx.data();
  b->page_off = s->page_off.data();
  b->page_idx = s->page_idx.data();
  b->page_size = s->page_size;
  b->vis_mode = MV_VIS_ANCESTORS;
  b->pos_mode = MV_POS_MAX_PARENT_END;
  *n_rows = int32_t(s->row_req.size());
  return MV_OK;
}

extern "C" mv_status mv_sched_rows(const mv_sched* s, const int32_t** request_ids, const int32_t** node_ids, int32_t* n_rows) {
  if (!s || !request_ids || !node_ids || !n_rows) return MV_ERR_INVALID_ARG;
  *request_ids = s->row_req.data();
  *node_ids = s->row_node.data();
  *n_rows = s->pending ? int32_t(s->row_req.size()) : 0;
  return MV_OK;
}

extern "C" mv_status mv_sched_commit(mv_sched* s, const uint8_t* finished) {
  if (!s || !s->pending) return MV_ERR_INVALID_ARG;
  s->pending = false;
  size_t row = 0;
  // fire() may append nothing to `requests`, so references stay valid
  for (Request& rq : s->requests) {
    if (rq.done || rq.running.empty()) continue;
    std::vector<int32_t> still;
    for (int32_t t : rq.running) {
      int32_t& w = rq.written[size_t(t)];
      ++w;
      if (w >= rq.tokens[size_t(t)] || (finished && finished[row])) {
        rq.tokens[size_t(t)] = w;
        w = -1;
        s->hold_view(rq, t, -1);  // the complete step lets go of what it read
      } else {
        still.push_back(t);
      }
      ++row;
    }
    rq.running.swap(still);
    if (rq.running.empty()) {  // the barrier: M_{k+1} marks the output places of all of F_k
      for (int32_t t : rq.active) rq.marked[size_t(t)] = 1;
      rq.active.clear();
      rq.k++;
      s->stats.markings_advanced++;
      s->fire(rq);
    }
  }
  return MV_OK;
}

extern "C" mv_status mv_sched_page_refs(const mv_sched* s, const int32_t* page_ids, int32_t n, int32_t* refs) {
  if (!s || n < 0 || (n > 0 && (!page_ids || !refs))) return MV_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i) {
    if (page_ids[i] < 0 || page_ids[i] >= s->num_pages) return MV_ERR_INVALID_ARG;
    refs[i] = s->refs[size_t(page_ids[i])];
  }
  return MV_OK;
}

extern "C" mv_status mv_sched_get_stats(const mv_sched* s, mv_sched_stats* stats) {
  if (!s || !stats) return MV_ERR_INVALID_ARG;
  *stats = s->stats;
  return MV_OK;
}
