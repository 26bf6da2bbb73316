// Plan life-cycle on the CUDA side: page-locked host image of the kernel tables, asynchronous upload,
// workspace sizing, launch counter.  The library never allocates device memory.
#include <cstdlib>
#include <cstring>

#include "common.cuh"

namespace mv {
std::atomic<int64_t> g_launches{0};
}

namespace {
bool ensure_pinned(mv_plan* P, size_t bytes) {
  if (P->pinned && P->pinned_cap >= bytes) return true;
  if (P->pinned) {
    if (P->pinned_is_cuda) cudaFreeHost(P->pinned);
    else std::free(P->pinned);
    P->pinned = nullptr;
    P->pinned_cap = 0;
  }
  const size_t cap = bytes + bytes / 2 + 4096;
  void* p = nullptr;
  if (cudaHostAlloc(&p, cap, cudaHostAllocDefault) == cudaSuccess) {
    P->pinned_is_cuda = true;
  } else {
    (void)cudaGetLastError();
    return false;
  }
  P->pinned = p;
  P->pinned_cap = cap;
  return true;
}

template <typename T>
void put(char* base, size_t off, const std::vector<T>& v) {
  if (!v.empty()) std::memcpy(base + off, v.data(), v.size() * sizeof(T));
}
}  // namespace

extern "C" mv_status mv_plan_upload(mv_plan* P, void* device_buf, size_t device_buf_bytes, void* cuda_stream) {
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  const size_t need = P->layout.total;
  if (!device_buf || device_buf_bytes < need || (reinterpret_cast<uintptr_t>(device_buf) & 255) != 0)
    return MV_ERR_WORKSPACE;
  if (!ensure_pinned(P, need)) return MV_ERR_CUDA;
  char* h = static_cast<char*>(P->pinned);
  const mv::DeviceLayout& L = P->layout;
  put(h, L.pos_id, P->pos_id);
  put(h, L.slot, P->slot);
  put(h, L.stages, P->stages);
  put(h, L.units, P->units);
  put(h, L.cta_unit_off, P->cta_unit_off);
  put(h, L.cta_head, P->cta_head);
  put(h, L.item_rows, P->item_rows);
  put(h, L.rowkv_part_off, P->rowkv_part_off);
  std::memcpy(h + L.sched, P->sched_zero, sizeof(P->sched_zero));
  put(h, L.q_tiles, P->q_tiles);
  put(h, L.kv_ranges, P->kv_ranges);
  put(h, L.page_tab, P->page_tab);
  put(h, L.k_tiles, P->k_tiles);
  put(h, L.q_ranges, P->q_ranges);
  // only the bytes in use travel (the tail of the last table)
  if (cudaMemcpyAsync(device_buf, h, need, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  P->device_buf = device_buf;
  return MV_OK;
}

extern "C" void mv_plan_destroy(mv_plan* P) {
  if (!P) return;
  if (P->pinned) {
    if (P->pinned_is_cuda) cudaFreeHost(P->pinned);
    else std::free(P->pinned);
  }
  delete P;
}

extern "C" size_t mv_workspace_bytes(const mv_plan* P, const mv_attn_geom* g, int op) {
  if (!P || !P->valid || !g) return 0;
  if (op == MV_OP_DECODE_ATTN) {
    const size_t vecs = size_t(P->stats.n_partials) * size_t(P->stats.sched_group);  // one per (partial, head of the group)
    const size_t o = (vecs * g->head_dim * sizeof(float) + 255) & ~size_t(255);
    const size_t ml = (vecs * 2 * sizeof(float) + 255) & ~size_t(255);
    return o + ml + 256;
  }
  const size_t row_heads = size_t(P->stats.n_new_tokens) * size_t(g->n_q_heads);
  // prefill: the optional per-(row, head) log-sum-exp; backward: the per-(row, head) dot products of dO and O
  if (op == MV_OP_PREFILL_ATTN || op == MV_OP_PREFILL_ATTN_BWD) return (row_heads * sizeof(float) + 255) & ~size_t(255);
  return 0;
}

extern "C" int64_t mv_launch_count(void) { return mv::g_launches.load(); }
