// Topology-masked prefill attention, bf16 tensor-core kernel with fp32 accumulation (Eq. 2 with the DAG
// mask of Eq. 3 in visibility-set form).  A query tile belongs to one node and walks only the KV ranges
// that node may see (tile skipping); the causal test is applied only inside the node's own range, and
// only on the tiles that touch the diagonal; ragged range ends are masked by a column bound.
//
// One CTA = 4 warps = 64 query rows (half of a planner tile) of one query head.  K/V tiles of 64 tokens
// are double-buffered with cp.async into XOR-swizzled shared memory; QK^T and PV run on m16n8k16 MMAs,
// softmax is online in log2 units.
#include "common.cuh"
#include "trace.h"

namespace {

using bf16 = __nv_bfloat16;
constexpr int NTHREADS = 128;
constexpr int BQ = 64;   // query rows per CTA
constexpr int BK = 64;   // keys per tile
constexpr int NBUF = 2;

template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return uint32_t(row) * (D * 2) + (uint32_t(chunk ^ (row & 7)) << 4);
}

template <int D>
__global__ void __launch_bounds__(NTHREADS) prefill_bf16_kernel(const bf16* __restrict__ q, const bf16* __restrict__ k,
                                                                const bf16* __restrict__ v, bf16* __restrict__ out,
                                                                const mv::QTile* __restrict__ q_tiles,
                                                                const mv::KvRange* __restrict__ ranges, int Hq, int Hkv,
                                                                float scale_log2) {
  constexpr int KSTEPS = D / 16, DT = D / 8, CPR = D / 8, NT = BK / 8;
  constexpr int TILE_BYTES = BK * D * 2;
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* q_s = smem;                       // [BQ][D]
  unsigned char* k_s = smem + BQ * D * 2;          // [NBUF][BK][D]
  unsigned char* v_s = k_s + NBUF * TILE_BYTES;    // [NBUF][BK][D]
  const uint32_t q_u = mv::smem_u32(q_s), k_u = mv::smem_u32(k_s), v_u = mv::smem_u32(v_s);

  const mv::QTile qt = q_tiles[blockIdx.x >> 1];
  const int half = blockIdx.x & 1;
  if (half * BQ >= qt.q_len) return;
  const int q0 = qt.q_start + half * BQ;                  // first query of the CTA (flattened index)
  const int nq = min(BQ, qt.q_len - half * BQ);           // valid query rows
  const int q_last = q0 + nq - 1;
  const int h = blockIdx.y, kvh = h / (Hq / Hkv);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  for (int i = tid; i < BQ * CPR; i += NTHREADS) {
    const int r = i / CPR, c = i % CPR;
    const bool ok = r < nq;
    mv::cp_async_16(q_u + swz<D>(r, c), q + (ok ? (int64_t(q0 + r) * Hq + h) * D + c * 8 : 0), ok ? 16 : 0);
  }
  mv::cp_async_commit();

  // flattened list of KV tiles: walk ranges, 64 keys at a time; causal ranges stop at the CTA's last query
  int ri = 0, kv0 = 0, r_end = 0, r_causal = 0;
  auto next_range = [&]() {
    while (ri < qt.range_count) {
      const mv::KvRange rg = ranges[qt.range_begin + ri];
      ++ri;
      kv0 = rg.kv_start;
      r_end = rg.kv_start + rg.kv_len;
      r_causal = rg.causal;
      if (r_causal) r_end = min(r_end, q_last + 1);
      if (kv0 < r_end) return true;
    }
    return false;
  };
  struct Tile { int start, n, causal; };
  auto next_tile = [&](Tile& t) {
    if (kv0 >= r_end && !next_range()) return false;
    t.start = kv0;
    t.n = min(BK, r_end - kv0);
    t.causal = r_causal;
    kv0 += BK;
    return true;
  };
  auto load_tile = [&](const Tile& t, int buf) {
    const uint32_t kd = k_u + buf * TILE_BYTES, vd = v_u + buf * TILE_BYTES;
    for (int i = tid; i < BK * CPR; i += NTHREADS) {
      const int r = i / CPR, c = i % CPR;
      const bool ok = r < t.n;
      const int64_t off = ok ? (int64_t(t.start + r) * Hkv + kvh) * D + c * 8 : 0;
      mv::cp_async_16(kd + swz<D>(r, c), k + off, ok ? 16 : 0);
      mv::cp_async_16(vd + swz<D>(r, c), v + off, ok ? 16 : 0);
    }
  };

  Tile cur, nxt;
  bool have = next_tile(cur);
  if (have) load_tile(cur, 0);
  mv::cp_async_commit();

  uint32_t qf[KSTEPS][4];
  float oacc[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const int qrow0 = q0 + warp * 16 + (lane >> 2), qrow1 = qrow0 + 8;  // flattened indices of this thread's rows
  bool q_loaded = false;
  int buf = 0;
  while (have) {
    const bool have_next = next_tile(nxt);
    if (have_next) load_tile(nxt, buf ^ 1);
    mv::cp_async_commit();
    mv::cp_async_wait<1>();
    __syncthreads();
    if (!q_loaded) {
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk)
        mv::ldmatrix_x4(qf[kk], q_u + swz<D>(warp * 16 + (lane & 15), kk * 2 + (lane >> 4)));
      q_loaded = true;
    }
    const uint32_t kb = k_u + buf * TILE_BYTES, vb = v_u + buf * TILE_BYTES;
    float sacc[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t b[4];
        const int tok = np * 16 + (lane & 7) + ((lane >> 4) << 3);
        mv::ldmatrix_x4(b, kb + swz<D>(tok, kk * 2 + ((lane >> 3) & 1)));
        mv::mma_bf16_16816(sacc[2 * np], qf[kk], b[0], b[1]);
        mv::mma_bf16_16816(sacc[2 * np + 1], qf[kk], b[2], b[3]);
      }
    }
    const bool need_mask = (cur.n < BK) || (cur.causal && cur.start + BK - 1 > q0 + warp * 16);
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float sv = sacc[nt][e] * scale_log2;
        if (need_mask) {
          const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
          const int kj = cur.start + col;
          const int qi = (e < 2) ? qrow0 : qrow1;
          if (col >= cur.n || (cur.causal && kj > qi)) sv = -INFINITY;
        }
        sacc[nt][e] = sv;
        if (e < 2) mx0 = fmaxf(mx0, sv);
        else mx1 = fmaxf(mx1, sv);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;  // fully masked so far
    const float al0 = mv::fast_exp2(m0 - mu0), al1 = mv::fast_exp2(m1 - mu1);
    m0 = mn0;
    m1 = mn1;
    float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      sacc[nt][0] = mv::fast_exp2(sacc[nt][0] - mu0);
      sacc[nt][1] = mv::fast_exp2(sacc[nt][1] - mu0);
      sacc[nt][2] = mv::fast_exp2(sacc[nt][2] - mu1);
      sacc[nt][3] = mv::fast_exp2(sacc[nt][3] - mu1);
      ps0 += sacc[nt][0] + sacc[nt][1];
      ps1 += sacc[nt][2] + sacc[nt][3];
    }
    l0 = l0 * al0 + ps0;
    l1 = l1 * al1 + ps1;
#pragma unroll
    for (int i = 0; i < DT; ++i) {
      oacc[i][0] *= al0; oacc[i][1] *= al0;
      oacc[i][2] *= al1; oacc[i][3] *= al1;
    }
#pragma unroll
    for (int kt = 0; kt < BK / 16; ++kt) {
      uint32_t pa[4];
      pa[0] = mv::pack_bf16(sacc[2 * kt][0], sacc[2 * kt][1]);
      pa[1] = mv::pack_bf16(sacc[2 * kt][2], sacc[2 * kt][3]);
      pa[2] = mv::pack_bf16(sacc[2 * kt + 1][0], sacc[2 * kt + 1][1]);
      pa[3] = mv::pack_bf16(sacc[2 * kt + 1][2], sacc[2 * kt + 1][3]);
#pragma unroll
      for (int dp = 0; dp < DT / 2; ++dp) {
        uint32_t b[4];
        const int tok = kt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
        mv::ldmatrix_x4_trans(b, vb + swz<D>(tok, dp * 2 + (lane >> 4)));
        mv::mma_bf16_16816(oacc[2 * dp], pa, b[0], b[1]);
        mv::mma_bf16_16816(oacc[2 * dp + 1], pa, b[2], b[3]);
      }
    }
    __syncthreads();  // everyone is done with `buf` before the next iteration's prefetch overwrites it
    cur = nxt;
    have = have_next;
    buf ^= 1;
  }
  mv::cp_async_wait<0>();
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float inv0 = 1.f / l0, inv1 = 1.f / l1;
  const int r0 = warp * 16 + (lane >> 2), c0 = (lane & 3) * 2;
#pragma unroll
  for (int i = 0; i < DT; ++i) {
    if (r0 < nq)
      *reinterpret_cast<__nv_bfloat162*>(out + (int64_t(q0 + r0) * Hq + h) * D + i * 8 + c0) =
          __floats2bfloat162_rn(oacc[i][0] * inv0, oacc[i][1] * inv0);
    if (r0 + 8 < nq)
      *reinterpret_cast<__nv_bfloat162*>(out + (int64_t(q0 + r0 + 8) * Hq + h) * D + i * 8 + c0) =
          __floats2bfloat162_rn(oacc[i][2] * inv1, oacc[i][3] * inv1);
  }
}

template <int D>
mv_status launch(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* out,
                 cudaStream_t st) {
  constexpr int SMEM = BQ * D * 2 + 2 * NBUF * BK * D * 2;
  static std::atomic<uint64_t> opted_in{0};  // per device
  if (!mv::opt_in_smem(prefill_bf16_kernel<D>, SMEM, opted_in)) return MV_ERR_CUDA;
  dim3 grid(int(P->stats.n_q_tiles) * 2, g->n_q_heads);
  prefill_bf16_kernel<D><<<grid, NTHREADS, SMEM, st>>>(
      static_cast<const bf16*>(q), static_cast<const bf16*>(k), static_cast<const bf16*>(v), static_cast<bf16*>(out),
      mv::table<mv::QTile>(P, P->layout.q_tiles), mv::table<mv::KvRange>(P, P->layout.kv_ranges), g->n_q_heads,
      g->n_kv_heads, mv::softmax_scale(g) * 1.4426950408889634f);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}

}  // namespace

namespace mv {
mv_status prefill_f32(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* out,
                      cudaStream_t st);
mv_status prefill_tc(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* out, float* lse,
                     cudaStream_t st);
}

extern "C" mv_status mv_dag_prefill_attn(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_rot,
                                         const void* v, void* out, void* workspace, size_t workspace_bytes,
                                         void* cuda_stream) {
  mv::NvtxRange nvtx_range("mv_dag_prefill_attn");
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (!P->stats.prefill_ready) return MV_ERR_UNSUPPORTED;
  if (!q_rot || !k_rot || !v || !out) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // head_dim 128 with an even group size runs on tcgen05 (two heads of a KV head per CTA); TMA needs 16-byte
  // aligned tensors.  Everything else takes the float32 kernel or the mma.sync kernel below.
  const bool aligned = ((reinterpret_cast<uintptr_t>(q_rot) | reinterpret_cast<uintptr_t>(k_rot) | reinterpret_cast<uintptr_t>(v)) & 15) == 0;
  const bool tc = g->dtype == MV_BF16 && g->head_dim == 128 && (g->n_q_heads / g->n_kv_heads) % 2 == 0 && aligned;
  // a workspace asks for the rows' log-sum-exp (what the backward pass needs); only the tcgen05 kernel writes it
  float* lse = nullptr;
  if (workspace) {
    if (!tc) return MV_ERR_UNSUPPORTED;
    if (workspace_bytes < mv_workspace_bytes(P, g, MV_OP_PREFILL_ATTN) || (reinterpret_cast<uintptr_t>(workspace) & 15) != 0) return MV_ERR_WORKSPACE;
    lse = static_cast<float*>(workspace);
  }
  if (g->dtype == MV_F32) return mv::prefill_f32(P, g, q_rot, k_rot, v, out, s);
  if (tc) return mv::prefill_tc(P, g, q_rot, k_rot, v, out, lse, s);
  return g->head_dim == 128 ? launch<128>(P, g, q_rot, k_rot, v, out, s) : launch<64>(P, g, q_rot, k_rot, v, out, s);
}
