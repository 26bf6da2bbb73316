// Internal layout of an mv_plan: canonical host tables plus the packed device tables the kernels read.
// Shared by the planner (host C++) and the kernel launchers; not part of the public ABI.
#pragma once
#include <cstddef>
#include <cstdint>
#include <vector>

#include "medverse_attn.h"

namespace mv {

constexpr int kPrefillQTile = 128;   // query rows per prefill tile (tiles never straddle a node)
constexpr int kAppendTileTokens = 40;  // a node that receives at least this many tokens sends the step to the tiled kernel
                                       // (measured break-even against the row-group kernels: about 37 tokens per node)
constexpr int kMaxAppendTokens = 256;  // most new tokens per node that the decode path takes (beyond that: prefill only)
constexpr int kPrefillKvTile = 64;   // granularity used only for the executed-pairs statistic

// Decode work lists.  A request's frontier rows (at most 64 / group_size of them per row group) and all the KV
// they see form one stream of pages, node after node, packed four to a 64-token STAGE; every page slot
// carries the set of rows that see its node (the DAG mask at page granularity) and its count of valid tokens.  A work unit is a run of consecutive stages for ONE KV head; units are
// listed CTA by CTA (cta_unit_off): the planner cuts the step's whole stream into equal shares.
struct StageDesc {     // 64 bytes
  int32_t page[4];     // physical pages of the stage's four page slots (absent slots repeat page[0])
  uint32_t n_tokens4;  // valid tokens of each page slot, one byte per slot (16 except on a node's last page)
  int32_t n_pages;     // page slots in use, 1..4 (fewer than 4 only on the last stage of a stream)
  uint32_t mask_lo[4], mask_hi[4];  // per page slot: bit r set = row r of the unit's row group sees the page's node
  int32_t pad[2];
};
static_assert(sizeof(StageDesc) == 64, "stage descriptor layout");
struct WorkUnit {
  int32_t stage_begin;  // index into the stage table
  int32_t n_stages;
  int32_t row_begin;    // index into item_rows of the unit's first (row, partial slot) pair
  int32_t n_rows;       // rows of the row group
  int32_t kvh;          // KV head
  int32_t pad[3];
};
struct ItemRow {
  int32_t row;   // row index = index of the new token
  int32_t part;  // split-KV partial slot this (unit, row) pair writes (a slot holds group_size head vectors),
                 // or -1 if the row sees none of the unit's stages
};
// One prefill query tile: rows [q_start, q_start+q_len) of one node and the KV ranges they may see.
// Two forms.  Flat (prefill: every token is new, K / V come as token-ordered arrays): q and key indices are flattened
// token indices.  Paged (node append: the tile's rows are new tokens of one node, K / V come from the page pool): a
// range is one whole node, keys are counted inside the node (kv_start = 0) and `pages` is the index of the node's
// first page in the plan's page table; the causal range is the tile's own node.
struct QTile {
  int32_t q_start, q_len, range_begin, range_count;
  int32_t causal_base;  // index, in the causal range's key numbering, of the tile's first query (flat: = q_start)
  int32_t pad[3];
};
struct KvRange {
  int32_t kv_start, kv_len;
  int32_t causal;  // 1: key j is visible to query i only if j <= causal_base + i
  int32_t pages;   // paged form: index of the node's first page in the page table; flat form: 0
};

// Backward of the prefill (flat form only): the transposed lists.  A key tile is 128 keys of one node (QTile with
// q_start / q_len read as the tile's first key and key count); its ranges (KvRange with kv_start / kv_len read as a
// run of QUERY tokens) list the queries that see the tile: every token of every other node that sees the tile's node, and,
// in the tile's own node, the queries from the tile's first key on (causal = 1: query i sees key j only if j <= i).
struct DeviceLayout {  // byte offsets into the device table buffer (all multiples of 256)
  size_t pos_id = 0, slot = 0, stages = 0, units = 0, cta_unit_off = 0, cta_head = 0, item_rows = 0, rowkv_part_off = 0, sched = 0,
         q_tiles = 0, kv_ranges = 0, page_tab = 0, k_tiles = 0, q_ranges = 0, total = 0;
};

}  // namespace mv

struct mv_plan {
  // canonical tables (parity surface)
  std::vector<int32_t> layer, pos_start, pos_id, qnode, qnode_tok_off, seg_off, seg_node, seg_len;
  std::vector<int64_t> slot, kv_len;
  // kernel tables
  std::vector<mv::StageDesc> stages;
  std::vector<mv::WorkUnit> units;       // CTA by CTA
  std::vector<int32_t> cta_unit_off;     // [n_ctas + 1]
  std::vector<mv::WorkUnit> cta_head;    // [n_ctas] copy of each CTA's first unit; pad[0], pad[1] = its unit range
  std::vector<mv::ItemRow> item_rows;
  std::vector<int32_t> rowkv_part_off;   // [n_rows * n_kv_heads + 1] CSR over the partial slots of a (row, KV head)
  int32_t sched_zero[64] = {};  // device-side status words ([2] = status of bounded waits), uploaded as zeros
  std::vector<mv::QTile> q_tiles;
  std::vector<mv::KvRange> kv_ranges;
  std::vector<mv::QTile> k_tiles;        // backward: key tiles (see above), heaviest first
  std::vector<mv::KvRange> q_ranges;     // backward: the query runs that see a key tile
  std::vector<int32_t> page_tab;         // paged tiles only: the batch's page ids
  mv_plan_stats stats{};
  int32_t page_size = 16;
  bool valid = false;
  // packed image of the kernel tables in page-locked host memory
  mv::DeviceLayout layout;
  void* pinned = nullptr;
  size_t pinned_cap = 0;
  bool pinned_is_cuda = false;
  // where the last upload put the tables
  void* device_buf = nullptr;
  // a plan made without a geometry keeps its batch, so that mv_plan_bind_geometry can cut the decode work lists later
  struct SavedBatch {
    bool kept = false;
    std::vector<int32_t> node_off, node_len, node_new, parent_off, parent_idx, page_off, page_idx;
    int32_t n_req = 0, page_size = 16, vis_mode = 0, pos_mode = 0;
  } saved;
};
