// Internal layout of an mv_plan: canonical host tables plus the packed device tables the kernels read.
// Shared by the planner (host C++) and the kernel launchers; not part of the public ABI.
#pragma once
#include <cstddef>
#include <cstdint>
#include <vector>

#include "medverse_attn.h"

namespace mv {

constexpr int kPrefillQTile = 128;   // query rows per prefill tile (tiles never straddle a node)
constexpr int kPrefillKvTile = 64;   // granularity used only for the executed-pairs statistic

// One decode work item per KV head: a page-aligned chunk of one node's KV and the rows that see it.
struct WorkItem {
  int32_t page_begin;  // index into the uploaded page_idx array of the chunk's first page
  int32_t n_tokens;    // valid tokens in the chunk (the last page may be partial)
  int32_t row_begin;   // index into item_rows of the first (row, partial slot) pair
  int32_t n_rows;      // rows (new tokens) whose visible set contains this chunk
};
struct ItemRow {
  int32_t row;   // row index = index of the new token
  int32_t part;  // split-KV partial slot this (item, row) pair writes
};
// One prefill query tile: rows [q_start, q_start+q_len) of one node and the KV ranges they may see.
struct QTile {
  int32_t q_start, q_len, range_begin, range_count;
};
struct KvRange {
  int32_t kv_start, kv_len;
  int32_t causal;  // 1: key j is visible to query i only if j <= i (flattened token indices)
  int32_t pad;
};

struct DeviceLayout {  // byte offsets into the device table buffer (all multiples of 256)
  size_t pos_id = 0, slot = 0, page_idx = 0, items = 0, item_rows = 0, row_part_off = 0, sched = 0,
         q_tiles = 0, kv_ranges = 0, total = 0;
};

}  // namespace mv

struct mv_plan {
  // canonical tables (parity surface)
  std::vector<int32_t> layer, pos_start, pos_id, qnode, qnode_tok_off, seg_off, seg_node, seg_len;
  std::vector<int64_t> slot, kv_len;
  // kernel tables
  std::vector<int32_t> page_idx;
  std::vector<mv::WorkItem> items;
  std::vector<mv::ItemRow> item_rows;
  std::vector<int32_t> row_part_off;
  int32_t sched_zero[64] = {};  // device-side scheduler words (work counter, finished-CTA counter), uploaded as zeros
  std::vector<mv::QTile> q_tiles;
  std::vector<mv::KvRange> kv_ranges;
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
};
