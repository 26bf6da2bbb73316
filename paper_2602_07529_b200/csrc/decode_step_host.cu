// End-to-end form of one frontier decode step (Sec. 4.3 Phase II) for callers whose activations live in
// host memory: copy q/k/v in, upload the plan, RoPE + KV write, multi-branch attention, copy out back.
// Everything is enqueued on the caller's stream; nothing is allocated.
#include "common.cuh"

namespace {
size_t a256(size_t x) { return (x + 255) & ~size_t(255); }
struct Layout {
  size_t tables, q, k, v, out, ws, total, q_bytes, kv_bytes;
};
Layout layout(const mv_plan* P, const mv_attn_geom* g) {
  Layout L{};
  const size_t es = g->dtype == MV_BF16 ? 2 : 4;
  const size_t n = size_t(P->stats.n_new_tokens);
  L.q_bytes = n * g->n_q_heads * g->head_dim * es;
  L.kv_bytes = n * g->n_kv_heads * g->head_dim * es;
  size_t off = 0;
  L.tables = off; off = a256(off + mv_plan_device_bytes(P));
  L.q = off;      off = a256(off + L.q_bytes);
  L.k = off;      off = a256(off + L.kv_bytes);
  L.v = off;      off = a256(off + L.kv_bytes);
  L.out = off;    off = a256(off + L.q_bytes);
  L.ws = off;     off = a256(off + mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN));
  L.total = off;
  return L;
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
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(staging);
  st = mv_plan_upload(P, base + L.tables, mv_plan_device_bytes(P), cuda_stream);
  if (st != MV_OK) return st;
  if (cudaMemcpyAsync(base + L.q, q_host, L.q_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(base + L.k, k_host, L.kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(base + L.v, v_host, L.kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  st = mv_rope_write_kv(P, g, base + L.q, base + L.k, base + L.v, base + L.q, nullptr, k_pages, v_pages, cuda_stream);
  if (st != MV_OK) return st;
  st = mv_dag_decode_attn(P, g, base + L.q, k_pages, v_pages, base + L.out, base + L.ws,
                          mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN), cuda_stream);
  if (st != MV_OK) return st;
  if (cudaMemcpyAsync(out_host, base + L.out, L.q_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  return MV_OK;
}
