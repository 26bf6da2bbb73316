// End-to-end form of one frontier decode step (Sec. 4.3 Phase II) for callers whose activations live in
// host memory: copy q/k/v in, upload the plan, RoPE + KV write, multi-branch attention, copy out back.
// Everything is enqueued on the caller's stream; nothing is allocated.
#include "common.cuh"

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
