// End-to-end form of one frontier decode step (Sec. 4.3 Phase II) for callers whose activations live in
// host memory: copy q/k/v in, upload the plan, RoPE + KV write, multi-branch attention, copy out back.
// Everything is enqueued on the caller's stream and nothing is allocated, except in the sliced form at the end of the
// file, which keeps two streams and three events per device from its first call on.
#include "common.cuh"

#include <mutex>
#include <vector>

namespace {
size_t a256(size_t x) { return (x + 255) & ~size_t(255); }
struct Layout {
  size_t tables, q, k, v, out, ws, total, q_bytes, kv_bytes;
};
// q, k, v and out come first: their places depend on the row count and the geometry alone, so the copies can start
// before the step is planned.
Layout front(size_t n, const mv_attn_geom* g) {
  Layout L{};
  const size_t es = g->dtype == MV_BF16 ? 2 : 4;
  L.q_bytes = n * g->n_q_heads * g->head_dim * es;
  L.kv_bytes = n * g->n_kv_heads * g->head_dim * es;
  size_t off = 0;
  L.q = off;      off = a256(off + L.q_bytes);
  L.k = off;      off = a256(off + L.kv_bytes);
  L.v = off;      off = a256(off + L.kv_bytes);
  L.out = off;    off = a256(off + L.q_bytes);
  L.tables = off;
  L.total = off;
  return L;
}
Layout layout(const mv_plan* P, const mv_attn_geom* g) {
  Layout L = front(size_t(P->stats.n_new_tokens), g);
  size_t off = L.tables;
  off = a256(off + mv_plan_device_bytes(P));
  L.ws = off;     off = a256(off + mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN));
  L.total = off;
  return L;
}
bool copy_in(char* base, const Layout& L, const void* q, const void* k, const void* v, cudaStream_t s) {
  if (L.q_bytes == 0) return true;
  if (cudaMemcpyAsync(base + L.q, q, L.q_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(base + L.k, k, L.kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(base + L.v, v, L.kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  return true;
}
// table upload, RoPE + cache write, attention, copy of the result back to the host (q, k, v are in the staging buffer)
mv_status run_step(mv_plan* P, const mv_attn_geom* g, const Layout& L, char* base, void* out_host, void* k_pages, void* v_pages,
                   void* cuda_stream) {
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  mv_status st = mv_plan_upload(P, base + L.tables, mv_plan_device_bytes(P), cuda_stream);
  if (st != MV_OK) return st;
  st = mv_rope_write_kv(P, g, base + L.q, base + L.k, base + L.v, base + L.q, nullptr, k_pages, v_pages, cuda_stream);
  if (st != MV_OK) return st;
  st = mv_dag_decode_attn(P, g, base + L.q, k_pages, v_pages, base + L.out, base + L.ws,
                          mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN), cuda_stream);
  if (st != MV_OK) return st;
  if (L.q_bytes != 0 && cudaMemcpyAsync(out_host, base + L.out, L.q_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  return MV_OK;
}
}  // namespace

extern "C" size_t mv_decode_step_staging_bytes(const mv_plan* P, const mv_attn_geom* g) {
  if (!P || !P->valid || !g) return 0;
  return layout(P, g).total;
}

extern "C" mv_status mv_decode_step_host(mv_plan* P, const mv_attn_geom* g, const void* q_host, const void* k_host,
                                         const void* v_host, void* out_host, void* k_pages, void* v_pages, void* staging,
                                         size_t staging_bytes, void* cuda_stream) {
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (!q_host || !k_host || !v_host || !out_host || !k_pages || !v_pages) return MV_ERR_INVALID_ARG;
  const Layout L = layout(P, g);
  if (!staging || staging_bytes < L.total || (reinterpret_cast<uintptr_t>(staging) & 255) != 0) return MV_ERR_WORKSPACE;
  char* base = static_cast<char*>(staging);
  if (!copy_in(base, L, q_host, k_host, v_host, static_cast<cudaStream_t>(cuda_stream))) return MV_ERR_CUDA;
  return run_step(P, g, L, base, out_host, k_pages, v_pages, cuda_stream);
}

extern "C" mv_status mv_decode_step_host_batch(const mv_dag_batch* batch, mv_plan** plan, const mv_attn_geom* g, const void* q_host,
                                               const void* k_host, const void* v_host, void* out_host, void* k_pages,
                                               void* v_pages, void* staging, size_t staging_bytes, void* cuda_stream) {
  if (!batch || !plan || batch->n_req < 0 || !batch->node_off || !batch->node_new) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (!q_host || !k_host || !v_host || !out_host || !k_pages || !v_pages) return MV_ERR_INVALID_ARG;
  const int32_t n_nodes = batch->node_off[batch->n_req];
  int64_t n = 0;
  for (int32_t i = 0; i < n_nodes; ++i) {
    if (batch->node_new[i] < 0) return MV_ERR_INVALID_ARG;
    n += batch->node_new[i];
  }
  const Layout F = front(size_t(n), g);
  if (!staging || staging_bytes < F.total || (reinterpret_cast<uintptr_t>(staging) & 255) != 0) return MV_ERR_WORKSPACE;
  char* base = static_cast<char*>(staging);
  // the copies travel while the host plans the step
  if (!copy_in(base, F, q_host, k_host, v_host, static_cast<cudaStream_t>(cuda_stream))) return MV_ERR_CUDA;
  st = mv_plan_dag(batch, g, nullptr, plan);
  if (st != MV_OK) return st;
  mv_plan* P = *plan;
  if (P->stats.n_new_tokens != n) return MV_ERR_INVALID_ARG;
  const Layout L = layout(P, g);
  if (staging_bytes < L.total) return MV_ERR_WORKSPACE;
  return run_step(P, g, L, base, out_host, k_pages, v_pages, cuda_stream);
}

// ---- the same step in slices that overlap their copies with one another's kernels --------------------------
// A step with host inputs is copies in, kernels, copy out, in a row; on a large batch the copies are a good part of
// it.  Requests are independent (Sec. 4.3: each request's net advances on its own), so the batch is cut by requests
// into slices of about equal new tokens, each planned on its own and run on one of two internal streams: slice i + 1
// copies in while slice i computes, and slice i copies out while slice i + 1 computes.
namespace {
constexpr int MAX_SLICES = 8;
struct SubBatch {
  std::vector<int32_t> node_off, parent_off, page_off;
  mv_dag_batch b;
  int64_t row0, rows;
};
// requests [r0, r1) of `src` as a batch of their own (the CSR arrays rebased, everything else viewed in place)
void slice_batch(const mv_dag_batch* src, int32_t r0, int32_t r1, SubBatch* out) {
  const int32_t nb = src->node_off[r0], ne = src->node_off[r1];
  out->node_off.resize(size_t(r1 - r0) + 1);
  for (int32_t r = r0; r <= r1; ++r) out->node_off[size_t(r - r0)] = src->node_off[r] - nb;
  out->parent_off.resize(size_t(ne - nb) + 1);
  out->page_off.resize(size_t(ne - nb) + 1);
  for (int32_t i = nb; i <= ne; ++i) {
    out->parent_off[size_t(i - nb)] = src->parent_off[i] - src->parent_off[nb];
    out->page_off[size_t(i - nb)] = src->page_off[i] - src->page_off[nb];
  }
  out->b = *src;
  out->b.n_req = r1 - r0;
  out->b.node_off = out->node_off.data();
  out->b.node_len = src->node_len + nb;
  out->b.node_new = src->node_new + nb;
  out->b.parent_off = out->parent_off.data();
  out->b.parent_idx = src->parent_idx + src->parent_off[nb];
  out->b.page_off = out->page_off.data();
  out->b.page_idx = src->page_idx + src->page_off[nb];
  out->row0 = 0;
  for (int32_t i = 0; i < nb; ++i) out->row0 += src->node_new[i];
  out->rows = 0;
  for (int32_t i = nb; i < ne; ++i) out->rows += src->node_new[i];
}
// request bounds of the slices: cut where the running count of new tokens passes i / n of the total
bool slice_bounds(const mv_dag_batch* b, int32_t n_slices, int32_t* bounds) {
  if (!b || b->n_req < 1 || !b->node_off || !b->node_new || !b->parent_off || !b->page_off) return false;
  if (n_slices < 1 || n_slices > MAX_SLICES || n_slices > b->n_req) return false;
  int64_t total = 0;
  for (int32_t i = 0; i < b->node_off[b->n_req]; ++i) {
    if (b->node_new[i] < 0) return false;
    total += b->node_new[i];
  }
  bounds[0] = 0;
  int64_t run = 0;
  int32_t s = 1;
  for (int32_t r = 0; r < b->n_req && s < n_slices; ++r) {
    for (int32_t i = b->node_off[r]; i < b->node_off[r + 1]; ++i) run += b->node_new[i];
    const int32_t left_req = b->n_req - (r + 1), left_slices = n_slices - s;
    if (run * n_slices >= total * s || left_req == left_slices) bounds[s++] = r + 1;  // every slice keeps a request
  }
  bounds[n_slices] = b->n_req;
  for (int32_t i = 0; i < n_slices; ++i)
    if (bounds[i + 1] <= bounds[i]) return false;
  return true;
}
// two streams and three events per device, made on the first pipelined call on that device and kept until exit
struct Aux {
  cudaStream_t st[2] = {nullptr, nullptr};
  cudaEvent_t start = nullptr, done[2] = {nullptr, nullptr};
  bool ready = false;
};
Aux* aux_of_current_device() {
  static std::mutex mu;
  static Aux table[64];
  const int dev = mv::current_device();
  if (dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  Aux& a = table[dev];
  if (!a.ready) {
    bool ok = cudaEventCreateWithFlags(&a.start, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaStreamCreateWithFlags(&a.st[i], cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&a.done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      (void)cudaGetLastError();
      return nullptr;
    }
    a.ready = true;
  }
  return &a;
}
}  // namespace

extern "C" mv_status mv_decode_step_pipelined_plan(const mv_dag_batch* batch, mv_plan** plans, int32_t n_slices, const mv_attn_geom* g) {
  int32_t bounds[MAX_SLICES + 1];
  if (!plans || !slice_bounds(batch, n_slices, bounds)) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  for (int32_t i = 0; i < n_slices; ++i) {
    SubBatch sb;
    slice_batch(batch, bounds[i], bounds[i + 1], &sb);
    st = mv_plan_dag(&sb.b, g, nullptr, &plans[i]);
    if (st != MV_OK) return st;
  }
  return MV_OK;
}

extern "C" size_t mv_decode_step_pipelined_staging_bytes(mv_plan* const* plans, int32_t n_slices, const mv_attn_geom* g) {
  if (!plans || !g || n_slices < 1 || n_slices > MAX_SLICES) return 0;
  size_t total = 0;
  for (int32_t i = 0; i < n_slices; ++i) {
    if (!plans[i] || !plans[i]->valid) return 0;
    total += a256(layout(plans[i], g).total);
  }
  return total;
}

extern "C" mv_status mv_decode_step_host_pipelined(const mv_dag_batch* batch, mv_plan** plans, int32_t n_slices, const mv_attn_geom* g,
                                                   const void* q_host, const void* k_host, const void* v_host, void* out_host,
                                                   void* k_pages, void* v_pages, void* staging, size_t staging_bytes,
                                                   void* cuda_stream) {
  int32_t bounds[MAX_SLICES + 1];
  if (!plans || !slice_bounds(batch, n_slices, bounds)) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (!q_host || !k_host || !v_host || !out_host || !k_pages || !v_pages) return MV_ERR_INVALID_ARG;
  if (!staging || (reinterpret_cast<uintptr_t>(staging) & 255) != 0) return MV_ERR_WORKSPACE;
  Aux* aux = aux_of_current_device();
  if (!aux) return MV_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t es = g->dtype == MV_BF16 ? 2 : 4;
  const size_t q_row = size_t(g->n_q_heads) * g->head_dim * es, kv_row = size_t(g->n_kv_heads) * g->head_dim * es;
  // the internal streams start behind whatever the caller's stream holds
  if (cudaEventRecord(aux->start, s) != cudaSuccess) return MV_ERR_CUDA;
  for (int i = 0; i < 2; ++i)
    if (cudaStreamWaitEvent(aux->st[i], aux->start, 0) != cudaSuccess) return MV_ERR_CUDA;
  mv_status result = MV_OK;
  size_t used = 0;
  for (int32_t i = 0; i < n_slices && result == MV_OK; ++i) {
    cudaStream_t x = aux->st[i & 1];
    SubBatch sb;
    slice_batch(batch, bounds[i], bounds[i + 1], &sb);
    const Layout F = front(size_t(sb.rows), g);
    if (used + F.total > staging_bytes) {
      result = MV_ERR_WORKSPACE;
      break;
    }
    char* base = static_cast<char*>(staging) + used;
    const char* qh = static_cast<const char*>(q_host) + size_t(sb.row0) * q_row;
    const char* kh = static_cast<const char*>(k_host) + size_t(sb.row0) * kv_row;
    const char* vh = static_cast<const char*>(v_host) + size_t(sb.row0) * kv_row;
    // the slice's copies travel while the host plans it (and while the slice before it computes)
    if (!copy_in(base, F, qh, kh, vh, x)) {
      result = MV_ERR_CUDA;
      break;
    }
    result = mv_plan_dag(&sb.b, g, nullptr, &plans[i]);
    if (result != MV_OK) break;
    mv_plan* P = plans[i];
    const Layout L = layout(P, g);
    if (P->stats.n_new_tokens != sb.rows) result = MV_ERR_INVALID_ARG;
    else if (used + L.total > staging_bytes) result = MV_ERR_WORKSPACE;
    else result = run_step(P, g, L, base, static_cast<char*>(out_host) + size_t(sb.row0) * q_row, k_pages, v_pages, x);
    used += a256(L.total);
  }
  // the caller's stream continues behind both internal streams, also after an error (work may have been enqueued)
  for (int i = 0; i < 2; ++i)
    if (cudaEventRecord(aux->done[i], aux->st[i]) != cudaSuccess || cudaStreamWaitEvent(s, aux->done[i], 0) != cudaSuccess)
      result = result == MV_OK ? MV_ERR_CUDA : result;
  return result;
}
