// Topology-masked prefill attention, float32 SIMT kernel (exact float arithmetic, no tensor cores:
// TF32 would not hold the 1e-4 tolerance).  Implements Eq. 2 with the DAG mask of Eq. 3 in its
// visibility-set form: a query tile walks only the KV ranges its node may see.
//
// One CTA = 8 warps = 8 consecutive query rows of one query tile and one query head.  Keys/values
// are staged 32 tokens at a time in shared memory and shared by the 8 rows; inside a warp lane j owns
// key j of the sub-tile (score), then the lanes switch to owning output columns (PV).
#include "common.cuh"

namespace {

constexpr int ROWS = 8;    // query rows (warps) per CTA
constexpr int SUB = 32;    // keys per shared-memory sub-tile

template <int D>
__global__ void __launch_bounds__(ROWS * 32) prefill_f32_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                                                 const float* __restrict__ v, float* __restrict__ out,
                                                                 const mv::QTile* __restrict__ q_tiles,
                                                                 const mv::KvRange* __restrict__ ranges, int Hq, int Hkv,
                                                                 float scale) {
  constexpr int GROUPS = mv::kPrefillQTile / ROWS;
  __shared__ float Ks[SUB][D + 1];
  __shared__ float Vs[SUB][D];
  __shared__ float Qs[ROWS][D];
  const mv::QTile qt = q_tiles[blockIdx.x / GROUPS];
  const int row0 = (blockIdx.x % GROUPS) * ROWS;
  if (row0 >= qt.q_len) return;
  const int h = blockIdx.y, kvh = h / (Hq / Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_rows = min(ROWS, qt.q_len - row0);
  const bool row_ok = warp < n_rows;
  const int qi = qt.q_start + row0 + warp;           // flattened index of this warp's query
  const int q_last = qt.q_start + row0 + n_rows - 1;  // last query of the CTA
  for (int c = lane; c < D; c += 32) Qs[warp][c] = row_ok ? q[(int64_t(qi) * Hq + h) * D + c] : 0.f;
  float m = -INFINITY, l = 0.f;
  float o[D / 32];
#pragma unroll
  for (int c = 0; c < D / 32; ++c) o[c] = 0.f;

  for (int ri = 0; ri < qt.range_count; ++ri) {
    const mv::KvRange rg = ranges[qt.range_begin + ri];
    const int r_end = rg.kv_start + rg.kv_len;
    for (int kv0 = rg.kv_start; kv0 < r_end; kv0 += SUB) {
      if (rg.causal && kv0 > q_last) break;  // nothing in or after this sub-tile is visible to the CTA
      const int n = min(SUB, r_end - kv0);
      __syncthreads();
      for (int i = threadIdx.x; i < SUB * (D / 4); i += blockDim.x) {
        const int r = i / (D / 4), c4 = i % (D / 4);
        float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), vv = kk;
        if (r < n) {
          kk = *reinterpret_cast<const float4*>(k + (int64_t(kv0 + r) * Hkv + kvh) * D + c4 * 4);
          vv = *reinterpret_cast<const float4*>(v + (int64_t(kv0 + r) * Hkv + kvh) * D + c4 * 4);
        }
        Ks[r][c4 * 4 + 0] = kk.x; Ks[r][c4 * 4 + 1] = kk.y; Ks[r][c4 * 4 + 2] = kk.z; Ks[r][c4 * 4 + 3] = kk.w;
        *reinterpret_cast<float4*>(&Vs[r][c4 * 4]) = vv;
      }
      __syncthreads();
      if (!row_ok) continue;
      const int kj = kv0 + lane;
      const bool valid = lane < n && (!rg.causal || kj <= qi);
      float s = 0.f;
#pragma unroll 8
      for (int c = 0; c < D; ++c) s = fmaf(Qs[warp][c], Ks[lane][c], s);
      s = valid ? s * scale : -INFINITY;
      float mx = s;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
      if (mx == -INFINITY) continue;  // the whole sub-tile is masked for this row
      const float m_new = fmaxf(m, mx);
      const float alpha = expf(m - m_new);  // m = -inf gives 0
      const float p = valid ? expf(s - m_new) : 0.f;
      float ps = p;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, d);
      l = l * alpha + ps;
      m = m_new;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) o[c] *= alpha;
      for (int j = 0; j < n; ++j) {
        const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
        for (int c = 0; c < D / 32; ++c) o[c] = fmaf(pj, Vs[j][lane + 32 * c], o[c]);
      }
    }
  }
  if (row_ok) {
    const float inv = 1.f / l;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) out[(int64_t(qi) * Hq + h) * D + lane + 32 * c] = o[c] * inv;
  }
}

}  // namespace

namespace mv {
mv_status prefill_f32(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* out,
                      cudaStream_t st) {
  const int n_tiles = int(P->stats.n_q_tiles);
  if (n_tiles == 0) return MV_OK;
  const mv::QTile* qt = mv::table<mv::QTile>(P, P->layout.q_tiles);
  const mv::KvRange* rg = mv::table<mv::KvRange>(P, P->layout.kv_ranges);
  dim3 grid(n_tiles * (mv::kPrefillQTile / ROWS), g->n_q_heads);
  const float scale = mv::softmax_scale(g);
  if (g->head_dim == 128)
    prefill_f32_kernel<128><<<grid, ROWS * 32, 0, st>>>((const float*)q, (const float*)k, (const float*)v, (float*)out, qt,
                                                        rg, g->n_q_heads, g->n_kv_heads, scale);
  else
    prefill_f32_kernel<64><<<grid, ROWS * 32, 0, st>>>((const float*)q, (const float*)k, (const float*)v, (float*)out, qt,
                                                       rg, g->n_q_heads, g->n_kv_heads, scale);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}
}  // namespace mv
