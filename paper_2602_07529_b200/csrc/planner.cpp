// DAG -> segment planner: host only, integers only, deterministic.
//
// Turns each request's node graph into (i) frontier layers (Eq. 1: a transition fires once all of its
// input places are marked), (ii) visibility sets (Eq. 3 mask / Sec. 3.2 path history / Sec. 4.3 Join
// as a set union), (iii) adaptive position indices (Sec. 4.2), (iv) the KV index list of every active
// branch as segment + page tables (the `k` of a Petri-net token, Sec. 3.2), and (v) the private work
// lists of the decode and prefill kernels.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>

#include "plan_internal.h"
#include "trace.h"

namespace {

using mv::ItemRow;
using mv::KvRange;
using mv::QTile;
using mv::StageDesc;
using mv::WorkUnit;

struct Bits {  // dense bitset rows, n_words per node
  int n_words = 0;
  std::vector<uint64_t> w;
  void reset(int n_nodes) {
    n_words = (n_nodes + 63) / 64;
    w.assign(size_t(n_nodes) * n_words, 0);
  }
  uint64_t* row(int v) { return w.data() + size_t(v) * n_words; }
  const uint64_t* row(int v) const { return w.data() + size_t(v) * n_words; }
  void set(int v, int u) { row(v)[u >> 6] |= (uint64_t(1) << (u & 63)); }
  bool get(int v, int u) const { return (row(v)[u >> 6] >> (u & 63)) & 1; }
};

// a decode stream: one per (request, row group): a run of stages and the rows of the group
struct Seg { int32_t stage_begin, n_stages, rows_begin, n_rows; };

size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

mv_status check_batch(const mv_dag_batch* b) {
  if (!b || b->n_req < 0) return MV_ERR_INVALID_ARG;
  if (!b->node_off) return MV_ERR_INVALID_ARG;
  if (b->page_size != 16) return MV_ERR_INVALID_ARG;
  if (b->vis_mode != MV_VIS_ANCESTORS && b->vis_mode != MV_VIS_LAYERWISE) return MV_ERR_INVALID_ARG;
  if (b->pos_mode != MV_POS_MAX_PARENT_END && b->pos_mode != MV_POS_FRONTIER_ALIGNED) return MV_ERR_INVALID_ARG;
  if (b->node_off[0] != 0) return MV_ERR_INVALID_ARG;
  for (int r = 0; r < b->n_req; ++r)
    if (b->node_off[r + 1] < b->node_off[r]) return MV_ERR_INVALID_ARG;
  const int n_nodes = b->node_off[b->n_req];
  if (n_nodes > 0 && (!b->node_len || !b->node_new || !b->parent_off || !b->page_off)) return MV_ERR_INVALID_ARG;
  if (n_nodes == 0) return MV_OK;
  if (b->parent_off[0] != 0 || b->page_off[0] != 0) return MV_ERR_INVALID_ARG;
  for (int g = 0; g < n_nodes; ++g) {
    if (b->node_len[g] < 0 || b->node_new[g] < 0) return MV_ERR_INVALID_ARG;
    if (b->parent_off[g + 1] < b->parent_off[g] || b->page_off[g + 1] < b->page_off[g]) return MV_ERR_INVALID_ARG;
  }
  if (b->parent_off[n_nodes] > 0 && !b->parent_idx) return MV_ERR_INVALID_ARG;
  if (b->page_off[n_nodes] > 0 && !b->page_idx) return MV_ERR_INVALID_ARG;
  return MV_OK;
}

}  // namespace

namespace {
// kv_heads == 0: no geometry yet (canonical tables and prefill tiles only; the decode work lists are left out)
mv_status plan_impl(const mv_dag_batch* b, int kv_heads, int group, int chunk_tokens, int sched_ctas, mv_plan** out) {
  if (!out) return MV_ERR_INVALID_ARG;
  mv_status st = check_batch(b);
  if (st != MV_OK) return st;
  if (chunk_tokens < 0 || (chunk_tokens % b->page_size) != 0 || sched_ctas < 0) return MV_ERR_INVALID_ARG;

  const int ps = b->page_size;
  const int n_nodes = b->node_off[b->n_req];

  // ---- validation that needs the graph: topological numbering, page capacity, page ids
  int64_t max_page = -1;
  for (int r = 0; r < b->n_req; ++r) {
    const int lo = b->node_off[r], hi = b->node_off[r + 1];
    for (int g = lo; g < hi; ++g) {
      for (int e = b->parent_off[g]; e < b->parent_off[g + 1]; ++e) {
        const int p = b->parent_idx[e];
        if (p < 0 || p >= g - lo) return MV_ERR_NOT_TOPOLOGICAL;
      }
      const int64_t tot = int64_t(b->node_len[g]) + b->node_new[g];
      const int64_t n_pages = b->page_off[g + 1] - b->page_off[g];
      if (n_pages * ps < tot) return MV_ERR_PAGE_CAPACITY;
      for (int e = b->page_off[g]; e < b->page_off[g + 1]; ++e) {
        if (b->page_idx[e] < 0) return MV_ERR_INVALID_ARG;
        max_page = std::max<int64_t>(max_page, b->page_idx[e]);
      }
    }
  }

  mv_plan* P = *out;
  const bool created = (P == nullptr);
  if (created) {
    P = new (std::nothrow) mv_plan();
    if (!P) return MV_ERR_INVALID_ARG;
  }
  P->valid = false;
  P->device_buf = nullptr;
  P->page_size = ps;
  P->layer.assign(n_nodes, 0);
  P->pos_start.assign(n_nodes, 0);
  P->pos_id.clear(); P->slot.clear(); P->qnode.clear();
  P->qnode_tok_off.assign(1, 0);
  P->seg_off.assign(1, 0);
  P->seg_node.clear(); P->seg_len.clear(); P->kv_len.clear();
  P->units.clear(); P->cta_unit_off.clear(); P->cta_head.clear(); P->item_rows.clear(); P->rowkv_part_off.clear();
  P->q_tiles.clear(); P->kv_ranges.clear(); P->page_tab.clear(); P->k_tiles.clear(); P->q_ranges.clear();
  P->stages.clear();
  mv_plan_stats S{};
  S.n_nodes = n_nodes;
  S.max_page_id = max_page;

  bool decode_ready = true, prefill_ready = true, any_multi = false;
  int32_t max_new = 0;
  int64_t append_tiles = 0;
  for (int g = 0; g < n_nodes; ++g) {
    any_multi |= b->node_new[g] > 1;
    max_new = std::max(max_new, b->node_new[g]);
    if (b->node_new[g] > mv::kMaxAppendTokens) decode_ready = false;
    if (b->node_len[g] != 0) prefill_ready = false;
  }

  // ---- pass 1 (per request): layers, visibility, positions, canonical tables
  // scratch that keeps its capacity from one call to the next (planning runs once per decode step); bound to local
  // references once, since every access to a thread-local object of a shared library is a call
  struct Scratch {
    Bits vis;
    std::vector<int32_t> pos_end, layer_end, req_rows, row_node, row_tok, seg_rows, next_part;
    std::vector<int64_t> node_tok_start, cost_prefix;
    std::vector<char> seen_by_frontier, stage_plain;
    std::vector<Seg> segs;
  };
  static thread_local Scratch scratch;
  Scratch& sc = scratch;
  Bits& vis = sc.vis;
  std::vector<int32_t>&pos_end = sc.pos_end, &layer_end = sc.layer_end, &req_rows = sc.req_rows, &row_node = sc.row_node, &row_tok = sc.row_tok,
                      &seg_rows = sc.seg_rows, &next_part = sc.next_part;
  std::vector<int64_t>&node_tok_start = sc.node_tok_start, &cost_prefix = sc.cost_prefix;
  std::vector<char>&seen_by_frontier = sc.seen_by_frontier, &stage_plain = sc.stage_plain;
  std::vector<Seg>& segs = sc.segs;
  node_tok_start.assign(size_t(n_nodes), 0);  // flattened index of a node's first NEW token
  int64_t unique_tokens = 0, per_row_tokens = 0, visible_pairs = 0, tile_pairs = 0;
  const bool cut_lists = kv_heads > 0;  // the decode work lists need the head counts
  const int sched_kv_heads = kv_heads, sched_group = std::max(1, group);
  const int max_rows_per_item = std::max(1, 64 / sched_group);

  // decode streams: one per (request, row group): a run of stages and the rows of the group; cut into work
  // units after pass 1
  segs.clear();
  seg_rows.clear();
  stage_plain.clear();  // per stage: four full pages seen by the whole row group
  constexpr int kStage = 64;  // tokens per stage of the decode kernel's pipeline
  const int chunk = chunk_tokens;  // 0: units are cut only where a CTA's share ends

  int64_t new_tok_count = 0;
  for (int r = 0; r < b->n_req; ++r) {
    const int lo = b->node_off[r], hi = b->node_off[r + 1], n = hi - lo;
    if (n == 0) continue;
    int32_t* layer = P->layer.data() + lo;
    int32_t* pstart = P->pos_start.data() + lo;
    // Eq. 1: layer(v) = 0 for roots, else 1 + max over parents
    int max_layer = 0;
    for (int v = 0; v < n; ++v) {
      int L = 0;
      for (int e = b->parent_off[lo + v]; e < b->parent_off[lo + v + 1]; ++e)
        L = std::max(L, layer[b->parent_idx[e]] + 1);
      layer[v] = L;
      max_layer = std::max(max_layer, L);
    }
    // visibility sets
    vis.reset(n);
    if (b->vis_mode == MV_VIS_ANCESTORS) {
      for (int v = 0; v < n; ++v) {
        uint64_t* rv = vis.row(v);
        for (int e = b->parent_off[lo + v]; e < b->parent_off[lo + v + 1]; ++e) {
          const uint64_t* rp = vis.row(b->parent_idx[e]);
          for (int w = 0; w < vis.n_words; ++w) rv[w] |= rp[w];
        }
        vis.set(v, v);
      }
    } else {
      for (int v = 0; v < n; ++v) {
        for (int u = 0; u < n; ++u)
          if (layer[u] < layer[v]) vis.set(v, u);
        vis.set(v, v);
      }
    }
    // Sec. 4.2 positions
    pos_end.assign(n, 0);
    if (b->pos_mode == MV_POS_MAX_PARENT_END) {
      for (int v = 0; v < n; ++v) {
        int32_t s = 0;
        for (int e = b->parent_off[lo + v]; e < b->parent_off[lo + v + 1]; ++e)
          s = std::max(s, pos_end[b->parent_idx[e]]);
        pstart[v] = s;
        pos_end[v] = s + b->node_len[lo + v] + b->node_new[lo + v];
      }
    } else {
      layer_end.assign(max_layer + 2, 0);
      for (int L = 0; L <= max_layer; ++L) {
        int32_t e_max = 0;
        for (int v = 0; v < n; ++v) {
          if (layer[v] != L) continue;
          pstart[v] = layer_end[L];
          pos_end[v] = pstart[v] + b->node_len[lo + v] + b->node_new[lo + v];
          e_max = std::max(e_max, pos_end[v]);
        }
        layer_end[L + 1] = e_max;
      }
    }
    // canonical per-token and per-q-node tables
    seen_by_frontier.assign(size_t(n), 0);
    for (int v = 0; v < n; ++v) {
      const int g = lo + v;
      node_tok_start[g] = new_tok_count;
      const int nl = b->node_len[g], nn = b->node_new[g];
      if (nn == 0) continue;
      for (int t = nl; t < nl + nn; ++t) {
        P->pos_id.push_back(pstart[v] + t);
        const int64_t page = b->page_idx[b->page_off[g] + t / ps];
        P->slot.push_back(page * ps + t % ps);
      }
      P->qnode.push_back(g);
      int64_t kv = 0;
      for (int u = 0; u < n; ++u) {
        if (!vis.get(v, u)) continue;
        const int32_t ln = b->node_len[lo + u] + b->node_new[lo + u];
        P->seg_node.push_back(lo + u);
        P->seg_len.push_back(ln);
        kv += ln;
        seen_by_frontier[u] = 1;
      }
      P->seg_off.push_back(int32_t(P->seg_node.size()));
      P->kv_len.push_back(kv);
      per_row_tokens += kv;  // decode: exactly the row's visible tokens
      new_tok_count += nn;
      P->qnode_tok_off.push_back(int32_t(new_tok_count));
    }
    for (int u = 0; u < n; ++u)
      if (seen_by_frontier[u]) unique_tokens += b->node_len[lo + u] + b->node_new[lo + u];

    // a request in which some node receives several tokens takes the decode path only if the nodes that receive
    // tokens form one frontier: none of them sees another (single-token steps have no such condition: a row sees
    // the token another row of the step has just written whenever it sees that row's node)
    bool multi = false;
    for (int v = 0; v < n; ++v) multi |= b->node_new[lo + v] > 1;
    for (int v = 0; v < n && decode_ready && multi; ++v) {
      if (b->node_new[lo + v] == 0) continue;
      for (int u = 0; u < n; ++u)
        if (u != v && b->node_new[lo + u] > 0 && vis.get(v, u)) decode_ready = false;
    }
    // ---- decode streams of this request: per row group, the stages of every node at least one of its rows sees
    if (decode_ready && cut_lists) {
      req_rows.clear();  // rows of the request, ascending: one per new token, node after node
      row_node.clear();  // local node of each row
      row_tok.clear();   // which of its node's new tokens the row is
      for (int v = 0; v < n; ++v)
        for (int32_t j = 0; j < b->node_new[lo + v]; ++j) {
          req_rows.push_back(int32_t(node_tok_start[lo + v]) + j);
          row_node.push_back(v);
          row_tok.push_back(j);
        }
      for (size_t r0 = 0; r0 < req_rows.size(); r0 += size_t(max_rows_per_item)) {
        const size_t r1 = std::min(req_rows.size(), r0 + size_t(max_rows_per_item));
        Seg sg{int32_t(P->stages.size()), 0, int32_t(seg_rows.size()), int32_t(r1 - r0)};
        StageDesc sd{};  // the stage being filled, page slot by page slot
        const uint64_t group_rows = (r1 - r0) == 64 ? ~uint64_t(0) : ((uint64_t(1) << (r1 - r0)) - 1);
        auto flush = [&]() {
          if (sd.n_pages == 0) return;
          for (int j = sd.n_pages; j < 4; ++j) sd.page[j] = sd.page[0];
          // plain = four full pages that every row of the group sees: the kernels' unmasked softmax path
          bool plain = sd.n_pages == 4 && sd.n_tokens4 == 0x10101010u;
          for (int j = 0; j < 4 && plain; ++j) plain = ((uint64_t(sd.mask_hi[j]) << 32) | sd.mask_lo[j]) == group_rows;
          stage_plain.push_back(plain ? 1 : 0);
          P->stages.push_back(sd);
          sd = StageDesc{};
        };
        for (int u = 0; u < n; ++u) {
          const int32_t L = b->node_len[lo + u] + b->node_new[lo + u];
          if (L == 0) continue;
          uint64_t mask = 0, own = 0;  // rows that see node u; those among them that are new tokens of u itself
          for (size_t k = r0; k < r1; ++k)
            if (vis.get(row_node[k], u)) {
              mask |= uint64_t(1) << (k - r0);
              if (row_node[k] == u) own |= uint64_t(1) << (k - r0);
            }
          if (mask == 0) continue;
          const int32_t* pages = b->page_idx + b->page_off[lo + u];
          if (own != 0 && b->node_new[lo + u] > 1) {
            // Several new tokens of u in this group: token j sees u's tokens 0 .. node_len + j (causal inside the own
            // node).  A page is listed once per distinct count of visible tokens among the group's rows, each time
            // with the rows that see exactly that many (rows of other nodes cannot see u: it receives tokens).
            const int32_t old_len = b->node_len[lo + u];
            for (int32_t t0 = 0; t0 < L; t0 += ps) {
              size_t k = r0;
              while (k < r1) {
                if (row_node[k] != u) { ++k; continue; }
                const int32_t lim = std::max<int32_t>(0, std::min<int32_t>(ps, old_len + row_tok[k] + 1 - t0));
                uint64_t run = 0;
                size_t k2 = k;
                for (; k2 < r1 && row_node[k2] == u &&
                       std::max<int32_t>(0, std::min<int32_t>(ps, old_len + row_tok[k2] + 1 - t0)) == lim; ++k2)
                  run |= uint64_t(1) << (k2 - r0);
                if (lim > 0) {
                  const int j = sd.n_pages++;
                  sd.page[j] = pages[t0 / ps];
                  sd.n_tokens4 |= uint32_t(lim) << (8 * j);
                  sd.mask_lo[j] = uint32_t(run);
                  sd.mask_hi[j] = uint32_t(run >> 32);
                  if (sd.n_pages == 4) flush();
                }
                k = k2;
              }
            }
            continue;
          }
          int32_t t0 = 0;
          // open stage first, then whole stages of four full pages at once, then the tail page by page
          for (; t0 < L && sd.n_pages != 0; t0 += ps) {
            const int j = sd.n_pages++;
            sd.page[j] = pages[t0 / ps];
            sd.n_tokens4 |= uint32_t(std::min<int32_t>(ps, L - t0)) << (8 * j);
            sd.mask_lo[j] = uint32_t(mask);
            sd.mask_hi[j] = uint32_t(mask >> 32);
            if (sd.n_pages == 4) flush();
          }
          for (; t0 + 4 * ps <= L; t0 += 4 * ps) {
            StageDesc full{};
            for (int j = 0; j < 4; ++j) {
              full.page[j] = pages[t0 / ps + j];
              full.mask_lo[j] = uint32_t(mask);
              full.mask_hi[j] = uint32_t(mask >> 32);
            }
            full.n_tokens4 = 0x10101010u;
            full.n_pages = 4;
            stage_plain.push_back(mask == group_rows ? 1 : 0);
            P->stages.push_back(full);
          }
          for (; t0 < L; t0 += ps) {
            const int j = sd.n_pages++;
            sd.page[j] = pages[t0 / ps];
            sd.n_tokens4 |= uint32_t(std::min<int32_t>(ps, L - t0)) << (8 * j);
            sd.mask_lo[j] = uint32_t(mask);
            sd.mask_hi[j] = uint32_t(mask >> 32);
            if (sd.n_pages == 4) flush();
          }
        }
        flush();
        sg.n_stages = int32_t(P->stages.size()) - sg.stage_begin;
        seg_rows.insert(seg_rows.end(), req_rows.begin() + r0, req_rows.begin() + r1);
        if (sg.n_stages > 0) segs.push_back(sg);
      }
    }

    // ---- node append: paged query tiles of this request (128 new tokens of one node; one range per visible node,
    // the node's own range causal).  Built whenever some node of the batch receives several tokens; which kernel
    // runs the step is the launcher's choice.
    if (decode_ready && !prefill_ready && any_multi) {
      for (int v = 0; v < n; ++v) {
        const int g = lo + v;
        const int32_t nn = b->node_new[g], old_len = b->node_len[g];
        for (int32_t q0 = 0; q0 < nn; q0 += mv::kPrefillQTile) {
          const int32_t ql = std::min<int32_t>(mv::kPrefillQTile, nn - q0);
          QTile qt{};
          qt.q_start = int32_t(node_tok_start[g]) + q0;
          qt.q_len = ql;
          qt.range_begin = int32_t(P->kv_ranges.size());
          qt.causal_base = old_len + q0;
          for (int u = 0; u < n; ++u) {
            if (u == v) {
              P->kv_ranges.push_back(KvRange{0, old_len + q0 + ql, 1, b->page_off[g]});
            } else if (vis.get(v, u)) {
              const int32_t lu = b->node_len[lo + u] + b->node_new[lo + u];
              if (lu > 0) P->kv_ranges.push_back(KvRange{0, lu, 0, b->page_off[lo + u]});
            }
          }
          qt.range_count = int32_t(P->kv_ranges.size()) - qt.range_begin;
          P->q_tiles.push_back(qt);
          ++append_tiles;
        }
      }
    }

    // ---- prefill tiles of this request
    if (prefill_ready) {
      // flattened start of every node of the request
      for (int v = 0; v < n; ++v) {
        const int g = lo + v;
        const int32_t len_v = b->node_new[g];
        if (len_v == 0) continue;
        const int64_t v_start = node_tok_start[g];
        // visible ranges in flattened order, adjacent ones merged
        std::vector<KvRange> base;
        int64_t vis_before = 0;  // visible tokens outside the node itself
        for (int u = 0; u < n; ++u) {
          if (u == v || !vis.get(v, u) || b->node_new[lo + u] == 0) continue;
          const int32_t us = int32_t(node_tok_start[lo + u]);
          const int32_t ul = b->node_new[lo + u];
          vis_before += ul;
          if (!base.empty() && base.back().kv_start + base.back().kv_len == us) base.back().kv_len += ul;
          else base.push_back(KvRange{us, ul, 0, 0});
        }
        visible_pairs += vis_before * len_v + int64_t(len_v) * (len_v + 1) / 2;
        for (int32_t q0 = 0; q0 < len_v; q0 += mv::kPrefillQTile) {
          const int32_t ql = std::min<int32_t>(mv::kPrefillQTile, len_v - q0);
          QTile qt{};
          qt.q_start = int32_t(v_start + q0);
          qt.causal_base = qt.q_start;
          qt.q_len = ql;
          qt.range_begin = int32_t(P->kv_ranges.size());
          // own causal range [v_start, q_start + q_len), placed in flattened order.  A fully visible
          // range that ends exactly where the node starts is folded into it: every key before the
          // node start precedes every query of the tile, so the causal test is vacuous there.
          KvRange own{int32_t(v_start), q0 + ql, 1, 0};
          size_t k = 0;
          for (; k < base.size() && base[k].kv_start < own.kv_start; ++k) {
            if (base[k].kv_start + base[k].kv_len == own.kv_start) {
              own.kv_start = base[k].kv_start;
              own.kv_len += base[k].kv_len;
            } else {
              P->kv_ranges.push_back(base[k]);
            }
          }
          P->kv_ranges.push_back(own);
          for (; k < base.size(); ++k) P->kv_ranges.push_back(base[k]);
          qt.range_count = int32_t(P->kv_ranges.size()) - qt.range_begin;
          for (int i = qt.range_begin; i < qt.range_begin + qt.range_count; ++i) {
            const int64_t kl = P->kv_ranges[i].kv_len;
            tile_pairs += int64_t(mv::kPrefillQTile) * (((kl + mv::kPrefillKvTile - 1) / mv::kPrefillKvTile) * mv::kPrefillKvTile);
          }
          P->q_tiles.push_back(qt);
        }
      }
      // the transposed lists of the backward pass: per 128-key tile of node u, the runs of queries that see it
      for (int u = 0; u < n; ++u) {
        const int32_t len_u = b->node_new[lo + u];
        if (len_u == 0) continue;
        const int32_t u_start = int32_t(node_tok_start[lo + u]);
        std::vector<KvRange> seers;  // whole nodes that see u, in flattened order, adjacent ones merged
        for (int v = 0; v < n; ++v) {
          if (v == u || !vis.get(v, u) || b->node_new[lo + v] == 0) continue;
          const int32_t vs = int32_t(node_tok_start[lo + v]), vl = b->node_new[lo + v];
          if (!seers.empty() && seers.back().kv_start + seers.back().kv_len == vs) seers.back().kv_len += vl;
          else seers.push_back(KvRange{vs, vl, 0, 0});
        }
        for (int32_t k0 = 0; k0 < len_u; k0 += mv::kPrefillQTile) {
          QTile kt{};
          kt.q_start = u_start + k0;
          kt.q_len = std::min<int32_t>(mv::kPrefillQTile, len_u - k0);
          kt.causal_base = kt.q_start;
          kt.range_begin = int32_t(P->q_ranges.size());
          P->q_ranges.push_back(KvRange{u_start + k0, len_u - k0, 1, 0});  // own node: the queries from the tile's first key on
          for (const KvRange& r : seers) P->q_ranges.push_back(r);
          kt.range_count = int32_t(P->q_ranges.size()) - kt.range_begin;
          P->k_tiles.push_back(kt);
        }
      }
    }
  }

  // ---- decode: cut the stream of (row-group stream, KV head) stage runs into n_ctas shares of equal cost
  if (decode_ready && cut_lists) {
    const int64_t n_rows = new_tok_count;
    const int n_ctas = sched_ctas > 0 ? sched_ctas : 296;
    // Cost model in token equivalents, fitted to per-share times measured on the device (a full unmasked stage takes
    // about 1.4 us of a half-CTA's time = 80; a unit's q hand-over and epilogue 2.4 us; a stage whose pages are not all
    // full and seen by every row takes the masked softmax path, +0.3 us).
    constexpr int64_t kUnitOverhead = 140;
    const int max_unit_stages = chunk > 0 ? std::max(1, chunk / kStage) : (1 << 30);
    cost_prefix.assign(P->stages.size() + 1, 0);  // running stage cost over the stage table
    for (size_t i = 0; i < P->stages.size(); ++i) {
      cost_prefix[i + 1] = cost_prefix[i] + 16 * P->stages[i].n_pages + 16 + (stage_plain[i] ? 0 : 18);
    }
    int64_t remaining = 0;  // cost not yet handed out
    for (const Seg& sg : segs)
      remaining += (cost_prefix[size_t(sg.stage_begin + sg.n_stages)] - cost_prefix[size_t(sg.stage_begin)] + kUnitOverhead) * sched_kv_heads;
    // A CTA's share is recomputed from what is left whenever a CTA is opened, so that the overhead of the
    // extra units the cuts themselves create never piles up on the last CTA.
    auto share = [&](int c) {
      const int64_t left = n_ctas - c;
      return std::max<int64_t>((remaining + left * kUnitOverhead + left - 1) / left, 2 * kStage + kUnitOverhead);
    };
    P->cta_unit_off.assign(size_t(n_ctas) + 1, 0);
    P->rowkv_part_off.assign(size_t(n_rows) * sched_kv_heads + 1, 0);  // first counts, then offsets
    int cta = 0;
    int64_t acc = 0, target = share(0), max_acc = 0;
    const int64_t first_share = target;
    auto emit = [&](const Seg& sg, int kvh, int32_t st_off, int32_t take) {
      WorkUnit wu{};
      wu.stage_begin = sg.stage_begin + st_off;
      wu.n_stages = take;
      wu.row_begin = int32_t(P->item_rows.size());
      wu.n_rows = sg.n_rows;
      wu.kvh = kvh;
      uint64_t seen = 0;  // rows that see at least one stage of the unit
      const uint64_t all_rows = sg.n_rows == 64 ? ~uint64_t(0) : ((uint64_t(1) << sg.n_rows) - 1);
      for (int32_t i = 0; i < take && seen != all_rows; ++i) {
        const StageDesc& sd = P->stages[size_t(wu.stage_begin + i)];
        for (int j = 0; j < sd.n_pages; ++j) seen |= uint64_t(sd.mask_lo[j]) | (uint64_t(sd.mask_hi[j]) << 32);
      }
      for (int32_t k = 0; k < sg.n_rows; ++k) {
        const int32_t row = seg_rows[size_t(sg.rows_begin + k)];
        const bool has = (seen >> k) & 1;
        if (has) P->rowkv_part_off[size_t(row) * sched_kv_heads + kvh + 1]++;
        P->item_rows.push_back(ItemRow{row, has ? 0 : -1});  // 0: a slot is numbered below
      }
      P->units.push_back(wu);
      P->cta_unit_off[size_t(cta) + 1] = int32_t(P->units.size());
      S.max_item_rows = std::max<int64_t>(S.max_item_rows, sg.n_rows);
    };
    for (const Seg& sg : segs) {
      for (int kvh = 0; kvh < sched_kv_heads; ++kvh) {
        int32_t off = 0;
        remaining -= kUnitOverhead;  // the overhead of this run's first unit is charged below
        while (off < sg.n_stages) {
          const int64_t room = target - acc - kUnitOverhead;
          const int64_t base = cost_prefix[size_t(sg.stage_begin + off)];
          const int64_t rest = cost_prefix[size_t(sg.stage_begin + sg.n_stages)] - base;
          if (cta < n_ctas - 1 && room < kStage / 2) {  // this CTA is full
            ++cta;
            acc = 0;
            target = share(cta);
            continue;
          }
          int32_t take = sg.n_stages - off;
          if (cta < n_ctas - 1 && rest > room + kStage / 2) {
            // the run of stages whose cost comes closest to the room (at least one stage): rounding to the
            // nearest stage boundary keeps the shortfalls from drifting onto the last CTAs
            const int64_t* lo_it = cost_prefix.data() + sg.stage_begin + off;
            const int64_t* hi_it = cost_prefix.data() + sg.stage_begin + sg.n_stages + 1;
            const int64_t* it = std::upper_bound(lo_it, hi_it, base + room);  // first prefix beyond the room
            take = int32_t(it - lo_it) - 1;
            if (it != hi_it && (*it - (base + room)) < ((base + room) - *(it - 1))) ++take;
            take = std::max<int32_t>(1, std::min<int32_t>(take, sg.n_stages - off));
          }
          take = std::min(take, max_unit_stages);
          emit(sg, kvh, off, take);
          const int64_t c = cost_prefix[size_t(sg.stage_begin + off + take)] - base;
          acc += c + kUnitOverhead;
          max_acc = std::max(max_acc, acc);
          remaining -= c;
          off += take;
        }
      }
    }
    S.max_cta_cost = max_acc;
    for (int c = 1; c <= n_ctas; ++c) P->cta_unit_off[c] = std::max(P->cta_unit_off[c], P->cta_unit_off[c - 1]);
    P->cta_head.assign(size_t(n_ctas), WorkUnit{});
    for (int c = 0; c < n_ctas; ++c) {
      const int32_t ub = P->cta_unit_off[c], ue = P->cta_unit_off[c + 1];
      if (ub < ue) P->cta_head[size_t(c)] = P->units[size_t(ub)];
      P->cta_head[size_t(c)].pad[0] = ub;
      P->cta_head[size_t(c)].pad[1] = ue;
    }
    // partial slots: contiguous per (row, KV head), in unit order
    for (size_t i = 1; i < P->rowkv_part_off.size(); ++i) P->rowkv_part_off[i] += P->rowkv_part_off[i - 1];
    next_part.assign(P->rowkv_part_off.begin(), P->rowkv_part_off.end() - 1);
    for (const WorkUnit& wu : P->units) {
      ItemRow* ir = P->item_rows.data() + wu.row_begin;
      for (int32_t k = 0; k < wu.n_rows; ++k)
        if (ir[k].part == 0) ir[k].part = next_part[size_t(ir[k].row) * sched_kv_heads + wu.kvh]++;
    }
    S.n_items = int64_t(P->units.size());
    S.n_partials = int64_t(P->rowkv_part_off.back());
    S.n_ctas = n_ctas;
    S.chunk_tokens = chunk > 0 ? chunk : first_share;
  }
  if (!(decode_ready && !prefill_ready && any_multi)) append_tiles = 0;  // a later request took the batch off the decode path
  if (append_tiles > 0) P->page_tab.assign(b->page_idx, b->page_idx + b->page_off[n_nodes]);
  // ---- prefill and node append: heaviest query tiles first
  if (prefill_ready || append_tiles > 0) {
    std::vector<int64_t> cost(P->q_tiles.size(), 0);
    for (size_t i = 0; i < P->q_tiles.size(); ++i)
      for (int k = 0; k < P->q_tiles[i].range_count; ++k) cost[i] += P->kv_ranges[P->q_tiles[i].range_begin + k].kv_len;
    std::vector<int32_t> order(P->q_tiles.size());
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t c) { return cost[a] > cost[c]; });
    std::vector<QTile> sorted;
    sorted.reserve(order.size());
    for (int32_t i : order) sorted.push_back(P->q_tiles[i]);
    P->q_tiles.swap(sorted);
    if (prefill_ready) {
      std::vector<int64_t> kcost(P->k_tiles.size(), 0);
      for (size_t i = 0; i < P->k_tiles.size(); ++i)
        for (int k = 0; k < P->k_tiles[i].range_count; ++k) kcost[i] += P->q_ranges[P->k_tiles[i].range_begin + k].kv_len;
      std::vector<int32_t> korder(P->k_tiles.size());
      std::iota(korder.begin(), korder.end(), 0);
      std::stable_sort(korder.begin(), korder.end(), [&](int32_t a, int32_t c) { return kcost[a] > kcost[c]; });
      std::vector<QTile> ksorted;
      ksorted.reserve(korder.size());
      for (int32_t i : korder) ksorted.push_back(P->k_tiles[i]);
      P->k_tiles.swap(ksorted);
      S.n_q_tiles = int64_t(P->q_tiles.size());
      S.visible_pairs = visible_pairs;
      S.tile_pairs = tile_pairs;
    } else {
      S.append_tiles = int64_t(P->q_tiles.size());
    }
  }

  S.n_new_tokens = new_tok_count;
  S.n_qnodes = int64_t(P->qnode.size());
  S.n_segs = int64_t(P->seg_node.size());
  S.decode_ready = decode_ready && new_tok_count > 0;
  S.prefill_ready = prefill_ready && new_tok_count > 0;
  S.sched_kv_heads = sched_kv_heads;
  S.sched_group = cut_lists ? sched_group : 0;
  S.unique_kv_tokens = unique_tokens;
  S.per_row_kv_tokens = per_row_tokens;
  S.max_node_new = max_new;
  P->stats = S;

  // ---- device table layout
  mv::DeviceLayout L;
  size_t off = 0;
  auto place = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
  L.pos_id = place(P->pos_id.size() * sizeof(int32_t));
  L.slot = place(P->slot.size() * sizeof(int64_t));
  L.stages = place(P->stages.size() * sizeof(StageDesc));
  L.units = place(P->units.size() * sizeof(WorkUnit));
  L.cta_unit_off = place(P->cta_unit_off.size() * sizeof(int32_t));
  L.cta_head = place(P->cta_head.size() * sizeof(WorkUnit));
  L.item_rows = place(P->item_rows.size() * sizeof(ItemRow));
  L.rowkv_part_off = place(P->rowkv_part_off.size() * sizeof(int32_t));
  L.sched = place(sizeof(P->sched_zero));
  L.q_tiles = place(P->q_tiles.size() * sizeof(QTile));
  L.kv_ranges = place(P->kv_ranges.size() * sizeof(KvRange));
  L.page_tab = place(P->page_tab.size() * sizeof(int32_t));
  L.k_tiles = place(P->k_tiles.size() * sizeof(QTile));
  L.q_ranges = place(P->q_ranges.size() * sizeof(KvRange));
  L.total = std::max<size_t>(off, 256);
  P->layout = L;
  P->valid = true;
  *out = P;
  return MV_OK;
}

mv_status heads_of(const mv_attn_geom* g, int* kv_heads, int* group) {
  if (g->n_q_heads <= 0 || g->n_kv_heads <= 0) return MV_ERR_INVALID_ARG;
  if (g->n_q_heads % g->n_kv_heads != 0) return MV_ERR_UNSUPPORTED;
  *kv_heads = g->n_kv_heads;
  *group = g->n_q_heads / g->n_kv_heads;
  return MV_OK;
}
}  // namespace

extern "C" mv_status mv_plan_dag(const mv_dag_batch* b, const mv_attn_geom* geom, const mv_plan_tuning* tuning, mv_plan** out) {
  mv::NvtxRange nvtx_range("mv_plan_dag");
  int kv_heads = 0, group = 0;
  if (geom) {
    const mv_status st = heads_of(geom, &kv_heads, &group);
    if (st != MV_OK) return st;
  }
  const mv_status st = plan_impl(b, kv_heads, group, tuning ? tuning->chunk_tokens : 0, tuning ? tuning->sched_ctas : 0, out);
  if (st != MV_OK) return st;
  mv_plan::SavedBatch& sv = (*out)->saved;
  sv.kept = false;
  if (!geom) {  // keep the batch: the work lists are cut when a geometry is bound
    const int n_nodes = b->node_off[b->n_req];
    sv.n_req = b->n_req; sv.page_size = b->page_size; sv.vis_mode = b->vis_mode; sv.pos_mode = b->pos_mode;
    sv.node_off.assign(b->node_off, b->node_off + b->n_req + 1);
    auto copy = [&](std::vector<int32_t>& v, const int32_t* p, size_t n) { if (n) v.assign(p, p + n); else v.clear(); };
    copy(sv.node_len, b->node_len, size_t(n_nodes));
    copy(sv.node_new, b->node_new, size_t(n_nodes));
    copy(sv.parent_off, b->parent_off, n_nodes ? size_t(n_nodes) + 1 : 0);
    copy(sv.parent_idx, b->parent_idx, n_nodes ? size_t(b->parent_off[n_nodes]) : 0);
    copy(sv.page_off, b->page_off, n_nodes ? size_t(n_nodes) + 1 : 0);
    copy(sv.page_idx, b->page_idx, n_nodes ? size_t(b->page_off[n_nodes]) : 0);
    sv.kept = true;
  }
  return MV_OK;
}

extern "C" mv_status mv_plan_bind_geometry(mv_plan* P, const mv_attn_geom* geom, const mv_plan_tuning* tuning) {
  if (!P || !P->valid || !geom) return MV_ERR_INVALID_ARG;
  if (!P->saved.kept) return MV_ERR_UNSUPPORTED;
  int kv_heads = 0, group = 0;
  const mv_status hs = heads_of(geom, &kv_heads, &group);
  if (hs != MV_OK) return hs;
  const mv_plan::SavedBatch& sv = P->saved;
  mv_dag_batch b{};
  b.n_req = sv.n_req;
  b.node_off = sv.node_off.data();
  b.node_len = sv.node_len.data(); b.node_new = sv.node_new.data();
  b.parent_off = sv.parent_off.data(); b.parent_idx = sv.parent_idx.data();
  b.page_off = sv.page_off.data(); b.page_idx = sv.page_idx.data();
  b.page_size = sv.page_size; b.vis_mode = sv.vis_mode; b.pos_mode = sv.pos_mode;
  // planning is deterministic, so the canonical tables come out as they were; the saved batch is not touched by it
  return plan_impl(&b, kv_heads, group, tuning ? tuning->chunk_tokens : 0, tuning ? tuning->sched_ctas : 0, &P);
}

extern "C" mv_status mv_plan_table(const mv_plan* P, int which, const void** host_ptr, int64_t* count) {
  if (!P || !P->valid || !host_ptr || !count) return MV_ERR_INVALID_ARG;
  auto give32 = [&](const std::vector<int32_t>& v) { *host_ptr = v.data(); *count = int64_t(v.size()); return MV_OK; };
  auto give64 = [&](const std::vector<int64_t>& v) { *host_ptr = v.data(); *count = int64_t(v.size()); return MV_OK; };
  switch (which) {
    case MV_TAB_LAYER: return give32(P->layer);
    case MV_TAB_POS_START: return give32(P->pos_start);
    case MV_TAB_POS_ID: return give32(P->pos_id);
    case MV_TAB_SLOT: return give64(P->slot);
    case MV_TAB_QNODE: return give32(P->qnode);
    case MV_TAB_QNODE_TOK_OFF: return give32(P->qnode_tok_off);
    case MV_TAB_SEG_OFF: return give32(P->seg_off);
    case MV_TAB_SEG_NODE: return give32(P->seg_node);
    case MV_TAB_SEG_LEN: return give32(P->seg_len);
    case MV_TAB_KV_LEN: return give64(P->kv_len);
    case MV_TAB_WORK_STAGES:
      *host_ptr = P->stages.data(); *count = int64_t(P->stages.size()) * int64_t(sizeof(StageDesc) / 4); return MV_OK;
    case MV_TAB_WORK_UNITS:
      *host_ptr = P->units.data(); *count = int64_t(P->units.size()) * int64_t(sizeof(WorkUnit) / 4); return MV_OK;
    case MV_TAB_WORK_ITEM_ROWS:
      *host_ptr = P->item_rows.data(); *count = int64_t(P->item_rows.size()) * 2; return MV_OK;
    case MV_TAB_WORK_CTA_UNIT_OFF: return give32(P->cta_unit_off);
    case MV_TAB_WORK_ROWKV_PART_OFF: return give32(P->rowkv_part_off);
    default: return MV_ERR_INVALID_ARG;
  }
}

extern "C" mv_status mv_plan_get_stats(const mv_plan* P, mv_plan_stats* stats) {
  if (!P || !P->valid || !stats) return MV_ERR_INVALID_ARG;
  *stats = P->stats;
  return MV_OK;
}

extern "C" size_t mv_plan_device_bytes(const mv_plan* P) { return (P && P->valid) ? P->layout.total : 0; }

extern "C" const char* mv_status_string(mv_status s) {
  switch (s) {
    case MV_OK: return "MV_OK";
    case MV_ERR_INVALID_ARG: return "MV_ERR_INVALID_ARG: null pointer, negative size, inconsistent offsets or bad enum";
    case MV_ERR_NOT_TOPOLOGICAL: return "MV_ERR_NOT_TOPOLOGICAL: a parent index is not smaller than its child's index";
    case MV_ERR_PAGE_CAPACITY: return "MV_ERR_PAGE_CAPACITY: a node's page list is too short for its tokens";
    case MV_ERR_UNSUPPORTED: return "MV_ERR_UNSUPPORTED: geometry, dtype or batch shape not supported by this kernel";
    case MV_ERR_WORKSPACE: return "MV_ERR_WORKSPACE: workspace or table buffer missing, too small or misaligned";
    case MV_ERR_CUDA: return "MV_ERR_CUDA: a CUDA runtime call failed";
    case MV_ERR_TIMEOUT: return "MV_ERR_TIMEOUT: a bounded device-side wait ran out";
    default: return "unknown mv_status";
  }
}
