// Multi-branch decode attention over a shared paged KV cache (Eq. 2 with the DAG mask of Eq. 3; Fork =
// shared prefix pages referenced by many rows, Join = union of the predecessors' segment lists, Sec. 4.3).
//
// Segment-major: the unit of work is (a page-aligned chunk of ONE node's KV, one KV head) together with
// the set of rows (frontier tokens) that see that node.  The chunk is streamed from HBM exactly once and
// serves every sibling row and the whole GQA group: the q-vectors (rows x group) are the M dimension of
// bf16 tensor-core tiles (m16n8k16, fp32 accumulate), so that the arithmetic (16-64 flop per KV byte)
// does not throttle the HBM stream.  Each CTA keeps a multi-stage cp.async pipeline of 64-token stages
// (16-byte coalesced copies of whole 4 KB page blocks, XOR-swizzled in shared memory for conflict-free
// ldmatrix) and an online softmax; partial (max, sum, output) triples go to the split-KV workspace and a
// second kernel merges the partials of every (row, head).
#include "common.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int NTHREADS = 128;  // 4 warps
constexpr int ST = 64;         // tokens per pipeline stage (4 pages)
constexpr int NSTAGES = 3;
constexpr int MAX_CHUNK_PAGES = 256;

struct DecodeArgs {
  const bf16* q;
  const bf16* k_pages;
  const bf16* v_pages;
  const int32_t* page_idx;
  const mv::WorkItem* items;
  const mv::ItemRow* item_rows;
  float* part_o;   // [n_partials][Hq][D]
  float* part_ml;  // [n_partials][Hq][2]  (max in log2 units, sum)
  int Hq, Hkv, G;
  float scale_log2;  // softmax scale * log2(e)
};

template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {  // byte offset of 16-byte chunk `chunk` of row `row`
  return uint32_t(row) * (D * 2) + (uint32_t(chunk ^ (row & 7)) << 4);
}

template <int D>
struct Smem {
  static constexpr int STAGE_BYTES = ST * D * 2;  // one of K or V
  static constexpr int Q_BYTES = 64 * D * 2;
  static constexpr int TOTAL = NSTAGES * 2 * STAGE_BYTES + Q_BYTES + MAX_CHUNK_PAGES * 4;
};

// One pass: up to MT*16 q-vectors against the whole chunk.  Warp w: m-tile (w % MT), kv split (w / MT).
template <int D, int MT>
__device__ __forceinline__ void decode_pass(const DecodeArgs& a, const mv::WorkItem& it, int kvh, int qv0, int nqv,
                                            unsigned char* smem) {
  constexpr int KS = 4 / MT;      // kv splits inside a stage
  constexpr int WT = ST / KS;     // tokens per warp per stage
  constexpr int NT = WT / 8;      // S n-tiles per warp
  constexpr int KSTEPS = D / 16;  // k-steps of QK^T
  constexpr int DT = D / 8;       // O n-tiles
  constexpr int CPR = D / 8;      // 16-byte chunks per row
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mt = warp % MT, ks = warp / MT;
  unsigned char* k_s = smem;
  unsigned char* v_s = smem + NSTAGES * Smem<D>::STAGE_BYTES;
  unsigned char* q_s = smem + 2 * NSTAGES * Smem<D>::STAGE_BYTES;
  const int32_t* pages = reinterpret_cast<const int32_t*>(q_s + Smem<D>::Q_BYTES);
  const uint32_t k_u = mv::smem_u32(k_s), v_u = mv::smem_u32(v_s), q_u = mv::smem_u32(q_s);

  // ---- stage the pass's q-vectors (zero rows beyond nqv); q-vector x = (row x / G, head kvh*G + x % G)
  for (int i = tid; i < MT * 16 * CPR; i += NTHREADS) {
    const int x = i / CPR, c = i % CPR;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (x < nqv) {
      const int xr = (qv0 + x) / a.G, xg = (qv0 + x) % a.G;
      const int row = a.item_rows[it.row_begin + xr].row;
      val = *reinterpret_cast<const uint4*>(a.q + (int64_t(row) * a.Hq + kvh * a.G + xg) * D + c * 8);
    }
    *reinterpret_cast<uint4*>(q_s + swz<D>(x, c)) = val;
  }

  const int n_stages = (it.n_tokens + ST - 1) / ST;
  auto load_stage = [&](int s) {
    if (s < n_stages) {
      const int buf = s % NSTAGES;
      const uint32_t kd = k_u + buf * Smem<D>::STAGE_BYTES, vd = v_u + buf * Smem<D>::STAGE_BYTES;
#pragma unroll
      for (int i = tid; i < ST * CPR; i += NTHREADS) {
        const int r = i / CPR, c = i % CPR;
        const int tok = s * ST + r;
        const bool ok = tok < it.n_tokens;
        const int64_t page = ok ? pages[tok >> 4] : 0;
        const int64_t off = (((page * a.Hkv + kvh) << 4) + (tok & 15)) * D + c * 8;
        mv::cp_async_16(kd + swz<D>(r, c), a.k_pages + (ok ? off : 0), ok ? 16 : 0);
        mv::cp_async_16(vd + swz<D>(r, c), a.v_pages + (ok ? off : 0), ok ? 16 : 0);
      }
    }
    mv::cp_async_commit();
  };
#pragma unroll
  for (int s = 0; s < NSTAGES - 1; ++s) load_stage(s);
  __syncthreads();  // q_s (and the page list) visible

  uint32_t qf[KSTEPS][4];
#pragma unroll
  for (int kk = 0; kk < KSTEPS; ++kk)
    mv::ldmatrix_x4(qf[kk], q_u + swz<D>(mt * 16 + (lane & 15), kk * 2 + (lane >> 4)));

  float oacc[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // rows lane/4 and lane/4 + 8 of the m-tile

  for (int s = 0; s < n_stages; ++s) {
    mv::cp_async_wait<NSTAGES - 2>();
    __syncthreads();
    load_stage(s + NSTAGES - 1);
    const int buf = s % NSTAGES;
    const uint32_t kb = k_u + buf * Smem<D>::STAGE_BYTES, vb = v_u + buf * Smem<D>::STAGE_BYTES;
    const int tok_w = ks * WT;  // first token of this warp inside the stage
    if (s * ST + tok_w >= it.n_tokens) continue;  // warp-uniform: nothing valid for this warp

    float sacc[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t b[4];
        const int tok = tok_w + np * 16 + (lane & 7) + ((lane >> 4) << 3);
        mv::ldmatrix_x4(b, kb + swz<D>(tok, kk * 2 + ((lane >> 3) & 1)));
        mv::mma_bf16_16816(sacc[2 * np], qf[kk], b[0], b[1]);
        mv::mma_bf16_16816(sacc[2 * np + 1], qf[kk], b[2], b[3]);
      }
    }
    // scale to log2 units, mask the ragged tail, online softmax
    const int tok_lim = it.n_tokens - (s * ST + tok_w);  // tokens of this warp slice that are valid
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
        const float sv = (col < tok_lim) ? sacc[nt][e] * a.scale_log2 : -INFINITY;
        sacc[nt][e] = sv;
        if (e < 2) mx0 = fmaxf(mx0, sv);
        else mx1 = fmaxf(mx1, sv);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);  // finite: column 0 of the slice is valid
    const float al0 = mv::fast_exp2(m0 - mn0), al1 = mv::fast_exp2(m1 - mn1);
    m0 = mn0;
    m1 = mn1;
    float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      sacc[nt][0] = mv::fast_exp2(sacc[nt][0] - mn0);
      sacc[nt][1] = mv::fast_exp2(sacc[nt][1] - mn0);
      sacc[nt][2] = mv::fast_exp2(sacc[nt][2] - mn1);
      sacc[nt][3] = mv::fast_exp2(sacc[nt][3] - mn1);
      ps0 += sacc[nt][0] + sacc[nt][1];
      ps1 += sacc[nt][2] + sacc[nt][3];
    }
    l0 = l0 * al0 + ps0;  // per-thread partial sums; reduced over the quad at the end
    l1 = l1 * al1 + ps1;
#pragma unroll
    for (int i = 0; i < DT; ++i) {
      oacc[i][0] *= al0; oacc[i][1] *= al0;
      oacc[i][2] *= al1; oacc[i][3] *= al1;
    }
    // O += P V
#pragma unroll
    for (int kt = 0; kt < WT / 16; ++kt) {
      uint32_t pa[4];
      pa[0] = mv::pack_bf16(sacc[2 * kt][0], sacc[2 * kt][1]);
      pa[1] = mv::pack_bf16(sacc[2 * kt][2], sacc[2 * kt][3]);
      pa[2] = mv::pack_bf16(sacc[2 * kt + 1][0], sacc[2 * kt + 1][1]);
      pa[3] = mv::pack_bf16(sacc[2 * kt + 1][2], sacc[2 * kt + 1][3]);
#pragma unroll
      for (int dp = 0; dp < DT / 2; ++dp) {
        uint32_t b[4];
        const int tok = tok_w + kt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
        mv::ldmatrix_x4_trans(b, vb + swz<D>(tok, dp * 2 + (lane >> 4)));
        mv::mma_bf16_16816(oacc[2 * dp], pa, b[0], b[1]);
        mv::mma_bf16_16816(oacc[2 * dp + 1], pa, b[2], b[3]);
      }
    }
  }
  mv::cp_async_wait<0>();
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  __syncthreads();  // every warp is done with the stage buffers: reuse them for the cross-warp combine

  float* red_o = reinterpret_cast<float*>(smem);                 // [4 warps][16][D]
  float* red_ml = red_o + 4 * 16 * D;                             // [4 warps][16][2]
  {
    const int r0 = lane >> 2, c0 = (lane & 3) * 2;
    float* wo = red_o + warp * 16 * D;
#pragma unroll
    for (int i = 0; i < DT; ++i) {
      *reinterpret_cast<float2*>(wo + r0 * D + i * 8 + c0) = make_float2(oacc[i][0], oacc[i][1]);
      *reinterpret_cast<float2*>(wo + (r0 + 8) * D + i * 8 + c0) = make_float2(oacc[i][2], oacc[i][3]);
    }
    if ((lane & 3) == 0) {
      red_ml[(warp * 16 + r0) * 2] = m0;
      red_ml[(warp * 16 + r0) * 2 + 1] = l0;
      red_ml[(warp * 16 + r0 + 8) * 2] = m1;
      red_ml[(warp * 16 + r0 + 8) * 2 + 1] = l1;
    }
  }
  __syncthreads();
  // combine the KS kv-splits of every q-vector and write the partial (unnormalised o, max, sum)
  for (int x = 0; x < nqv; ++x) {
    const int xm = x / 16, xr = x % 16;
    float mt_ = -INFINITY;
#pragma unroll
    for (int k2 = 0; k2 < KS; ++k2) mt_ = fmaxf(mt_, red_ml[((xm + MT * k2) * 16 + xr) * 2]);
    float lsum = 0.f;
    float w[KS];
#pragma unroll
    for (int k2 = 0; k2 < KS; ++k2) {
      const float mk = red_ml[((xm + MT * k2) * 16 + xr) * 2];
      w[k2] = (mk == -INFINITY) ? 0.f : mv::fast_exp2(mk - mt_);
      lsum += w[k2] * red_ml[((xm + MT * k2) * 16 + xr) * 2 + 1];
    }
    const int xrow = (qv0 + x) / a.G, xg = (qv0 + x) % a.G;
    const mv::ItemRow ir = a.item_rows[it.row_begin + xrow];
    const int64_t pslot = int64_t(ir.part) * a.Hq + kvh * a.G + xg;
    for (int c = tid; c < D; c += NTHREADS) {
      float acc = 0.f;
#pragma unroll
      for (int k2 = 0; k2 < KS; ++k2) acc += w[k2] * red_o[((xm + MT * k2) * 16 + xr) * D + c];
      a.part_o[pslot * D + c] = acc;
    }
    if (tid == 0) {
      a.part_ml[pslot * 2] = mt_;
      a.part_ml[pslot * 2 + 1] = lsum;
    }
  }
  __syncthreads();  // the combine buffers alias the stage buffers of the next pass
}

template <int D>
__global__ void __launch_bounds__(NTHREADS) decode_attn_kernel(const DecodeArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int unit = blockIdx.x;
  const mv::WorkItem it = a.items[unit / a.Hkv];
  const int kvh = unit % a.Hkv;
  int32_t* pages = reinterpret_cast<int32_t*>(smem + 2 * NSTAGES * Smem<D>::STAGE_BYTES + Smem<D>::Q_BYTES);
  const int n_pages = (it.n_tokens + 15) >> 4;
  for (int i = threadIdx.x; i < n_pages; i += NTHREADS) pages[i] = a.page_idx[it.page_begin + i];
  __syncthreads();
  const int nq_total = it.n_rows * a.G;
  for (int qv0 = 0; qv0 < nq_total; qv0 += 64) {
    const int nqv = min(64, nq_total - qv0);
    if (nqv <= 16) decode_pass<D, 1>(a, it, kvh, qv0, nqv, smem);
    else if (nqv <= 32) decode_pass<D, 2>(a, it, kvh, qv0, nqv, smem);
    else decode_pass<D, 4>(a, it, kvh, qv0, nqv, smem);
  }
}

// Merge of the split-KV partials of one (row, head): one warp each.
template <int D>
__global__ void __launch_bounds__(128) decode_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                                                           const int32_t* __restrict__ row_part_off, bf16* __restrict__ out,
                                                           int n_rows, int Hq) {
  const int w = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (w >= n_rows * Hq) return;
  const int row = w / Hq, h = w % Hq;
  const int p0 = row_part_off[row], p1 = row_part_off[row + 1];
  float m = -INFINITY;
  for (int p = p0 + lane; p < p1; p += 32) m = fmaxf(m, part_ml[(int64_t(p) * Hq + h) * 2]);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
  constexpr int E = D / 32;
  float acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  float l = 0.f;
  for (int p = p0; p < p1; ++p) {
    const int64_t ps = int64_t(p) * Hq + h;
    const float mp = part_ml[ps * 2];
    const float wgt = (mp == -INFINITY) ? 0.f : exp2f(mp - m);
    l += wgt * part_ml[ps * 2 + 1];
    const float* po = part_o + ps * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] += wgt * po[e];
  }
  const float inv = 1.f / l;
  bf16* o = out + (int64_t(row) * Hq + h) * D + lane * E;
#pragma unroll
  for (int e = 0; e < E; e += 2) *reinterpret_cast<__nv_bfloat162*>(o + e) = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
}

template <int D>
mv_status launch(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, void* out,
                 void* ws, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(decode_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::TOTAL) != cudaSuccess) {
      (void)cudaGetLastError();
      return MV_ERR_CUDA;
    }
    attr_set = true;
  }
  const size_t parts = size_t(P->stats.n_partials);
  const size_t o_bytes = (parts * g->n_q_heads * D * sizeof(float) + 255) & ~size_t(255);
  DecodeArgs a;
  a.q = static_cast<const bf16*>(q);
  a.k_pages = static_cast<const bf16*>(kp);
  a.v_pages = static_cast<const bf16*>(vp);
  a.page_idx = mv::table<int32_t>(P, P->layout.page_idx);
  a.items = mv::table<mv::WorkItem>(P, P->layout.items);
  a.item_rows = mv::table<mv::ItemRow>(P, P->layout.item_rows);
  a.part_o = static_cast<float*>(ws);
  a.part_ml = reinterpret_cast<float*>(static_cast<char*>(ws) + o_bytes);
  a.Hq = g->n_q_heads;
  a.Hkv = g->n_kv_heads;
  a.G = g->n_q_heads / g->n_kv_heads;
  a.scale_log2 = mv::softmax_scale(g) * 1.4426950408889634f;
  const int n_units = int(P->stats.n_items) * g->n_kv_heads;
  decode_attn_kernel<D><<<n_units, NTHREADS, Smem<D>::TOTAL, st>>>(a);
  mv::g_launches++;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  const int n_rows = int(P->stats.n_new_tokens);
  const int n_warps = n_rows * g->n_q_heads;
  decode_merge_kernel<D><<<(n_warps + 3) / 4, 128, 0, st>>>(a.part_o, a.part_ml, mv::table<int32_t>(P, P->layout.row_part_off),
                                                           static_cast<bf16*>(out), n_rows, g->n_q_heads);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}

}  // namespace

extern "C" mv_status mv_dag_decode_attn(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_pages,
                                        const void* v_pages, void* out, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream) {
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (g->dtype != MV_BF16 || !P->stats.decode_ready) return MV_ERR_UNSUPPORTED;
  if (P->stats.chunk_tokens > MAX_CHUNK_PAGES * 16) return MV_ERR_UNSUPPORTED;
  if (!q_rot || !k_pages || !v_pages || !out) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  if (P->stats.max_page_id >= g->num_pages) return MV_ERR_INVALID_ARG;
  const size_t need = mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  return g->head_dim == 128 ? launch<128>(P, g, q_rot, k_pages, v_pages, out, workspace, s)
                            : launch<64>(P, g, q_rot, k_pages, v_pages, out, workspace, s);
}
