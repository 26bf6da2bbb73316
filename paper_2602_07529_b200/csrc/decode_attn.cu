// Multi-branch decode attention over a shared paged KV cache (Eq. 2 with the DAG mask of Eq. 3; Fork =
// shared prefix pages referenced by many rows, Join = union of the predecessors' segment lists, Sec. 4.3).
//
// Segment-major: the unit of work is (a page-aligned chunk of ONE node's KV, one KV head) together with
// the set of rows (frontier tokens) that see that node.  The chunk is streamed from HBM exactly once and
// serves every sibling row and the whole GQA group: the q-vectors (rows x group) are the M dimension of
// bf16 tensor-core tiles (m16n8k16, fp32 accumulate), so that the arithmetic (16-64 flop per KV byte)
// does not throttle the HBM stream.
//
// Persistent CTAs (two per SM) pull units from an atomic work counter, longest first, and keep ONE
// pipeline of 64-token stages running across unit boundaries.  A stage is filled by TMA: one elected
// thread issues a [16 tokens][64 elements] box per half page block (cp.async.bulk.tensor, 128-byte
// shared-memory swizzle, completion counted on an mbarrier), so no thread spends issue slots or
// load-store-unit entries on the copy, and ldmatrix reads the tiles without bank conflicts.  Warps hand
// a consumed stage back through a second mbarrier; there is no CTA-wide barrier inside a unit.  Softmax
// is online, in log2 units; each unit leaves one partial (max, sum, unnormalised output) per q-vector in
// the split-KV workspace and a second kernel merges the partials of every (row, head).
//
// Every wait on an mbarrier is bounded: if it runs out, the CTA records MV_ERR_TIMEOUT in the plan's
// status word, stops waiting and still reaches every barrier, so the kernel always terminates.
#include <mutex>

#include "common.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int NTHREADS = 128;  // 4 warps
constexpr int ST = 64;         // tokens per pipeline stage (4 pages)
constexpr int NSTAGES = 3;

struct DecodeArgs {
  const bf16* q;
  const int32_t* page_idx;
  const mv::WorkItem* items;
  const mv::ItemRow* item_rows;
  float* part_o;   // [n_partials][Hq][D]
  float* part_ml;  // [n_partials][Hq][2]  (max in log2 units, sum)
  int32_t* sched;  // [0] next unit, [1] CTAs finished (both zero between launches), [2] status word
  int Hq, Hkv, G, n_units;
  float scale_log2;  // softmax scale * log2(e)
};

struct Unit {  // uniform across the CTA
  int page_begin, n_tokens, row_begin, n_rows, kvh, n_stages;
};

template <int D>
struct Cfg {
  static constexpr int CPR = D / 8;                 // 16-byte chunks per token row
  static constexpr int HALVES = D / 64;             // 128-byte column blocks per row (one TMA box each)
  static constexpr int HALF_BYTES = ST * 128;       // one column block of a stage: [64 tokens][128 B]
  static constexpr int KV_BYTES = ST * D * 2;       // K (or V) bytes of a stage
  static constexpr int STAGE_BYTES = 2 * KV_BYTES;  // K then V
  static constexpr int SMEM = NSTAGES * STAGE_BYTES + 1024;  // + slack to align the base to 1024 B
};

// Byte offset of 16-byte chunk `chunk` of token row `row` inside a K (or V) stage tile as TMA lays it out:
// column block h = chunk / 8 holds [64 tokens][128 B]; inside it the hardware XORs the chunk index with row % 8.
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return uint32_t(chunk >> 3) * Cfg<D>::HALF_BYTES + uint32_t(row) * 128 + (uint32_t((chunk & 7) ^ (row & 7)) << 4);
}

__device__ __forceinline__ Unit load_unit(const DecodeArgs& a, int u) {
  Unit x;
  if (u < a.n_units) {
    const int4 it = *reinterpret_cast<const int4*>(a.items + u / a.Hkv);
    x.page_begin = it.x; x.n_tokens = it.y; x.row_begin = it.z; x.n_rows = it.w;
    x.kvh = u % a.Hkv;
    x.n_stages = (it.y + ST - 1) / ST;
  } else {
    x.page_begin = 0; x.n_tokens = 0; x.row_begin = 0; x.n_rows = 0; x.kvh = 0; x.n_stages = 0;
  }
  return x;
}

struct Sync {  // shared-memory addresses of the pipeline barriers and flags
  uint32_t full, empty;  // arrays of NSTAGES mbarriers (8 bytes each)
  volatile int* abort;   // set once a bounded wait ran out
  int32_t* status;       // global status word
};

__device__ __forceinline__ void wait_or_flag(const Sync& sy, uint32_t bar, uint32_t parity) {
  if (*sy.abort) return;
  if (!mv::mbar_wait_bounded(bar, parity)) {
    *sy.abort = 1;
    atomicExch(sy.status, int(MV_ERR_TIMEOUT));
  }
}

// The producer side of the pipeline, run by thread 0: walks the stages of the current unit, then of the next.
template <int D>
struct Loader {
  int which = 0;   // 0: current unit, 1: next unit, 2: beyond (nothing to issue)
  int stage = 0;   // next stage of that unit to issue
  int issued = 0;  // stages issued so far (buffer = issued % NSTAGES)
  int pg[4] = {0, 0, 0, 0};  // prefetched page ids of the stage about to be issued

  __device__ __forceinline__ void prefetch_pages(const DecodeArgs& a, const Unit& cu, const Unit& nu) {
    const Unit& u = which == 0 ? cu : nu;
    if (which <= 1 && stage < u.n_stages) {
      const int n_pages = (u.n_tokens - stage * ST + 15) >> 4;
#pragma unroll
      for (int p = 0; p < 4; ++p) pg[p] = p < n_pages ? __ldg(a.page_idx + u.page_begin + stage * 4 + p) : 0;
    }
  }
  __device__ __forceinline__ bool issue(const DecodeArgs& a, const Unit& cu, const Unit& nu, uint32_t smem_base, const Sync& sy,
                                        const CUtensorMap* tm_k, const CUtensorMap* tm_v) {
    const Unit& u = which == 0 ? cu : nu;
    if (!(which <= 1 && stage < u.n_stages)) return false;
    const int b = issued % NSTAGES;
    wait_or_flag(sy, sy.empty + 8 * b, ((issued / NSTAGES) & 1) ^ 1);  // every warp has released the buffer
    const int n_pages = min(4, (u.n_tokens - stage * ST + 15) >> 4);
    const uint32_t bar = sy.full + 8 * b;
    mv::mbar_arrive_expect_tx(bar, uint32_t(n_pages) * 16 * D * 2 * 2);
    const uint32_t kd = smem_base + b * Cfg<D>::STAGE_BYTES, vd = kd + Cfg<D>::KV_BYTES;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      if (p < n_pages) {
        const int row = (pg[p] * a.Hkv + u.kvh) << 4;
#pragma unroll
        for (int h = 0; h < Cfg<D>::HALVES; ++h) {
          mv::tma_load_2d(kd + h * Cfg<D>::HALF_BYTES + p * 2048, tm_k, h * 64, row, bar);
          mv::tma_load_2d(vd + h * Cfg<D>::HALF_BYTES + p * 2048, tm_v, h * 64, row, bar);
        }
      }
    }
    ++stage;
    if (stage == u.n_stages) {
      ++which;
      stage = 0;
    }
    prefetch_pages(a, cu, nu);
    ++issued;
    return true;
  }
  // Keeps up to NSTAGES stages issued ahead of the consumers (as far as stages exist).
  __device__ __forceinline__ void top_up(const DecodeArgs& a, const Unit& cu, const Unit& nu, uint32_t smem_base, const Sync& sy,
                                         const CUtensorMap* tm_k, const CUtensorMap* tm_v, int consumed) {
    while (issued - consumed < NSTAGES && issue(a, cu, nu, smem_base, sy, tm_k, tm_v)) {
    }
  }
};

// merge (m, l, o) of another kv-split into mine; both in this thread's fragment layout
template <int DT>
__device__ __forceinline__ void merge_frag(float& m0, float& m1, float& l0, float& l1, float (&o)[DT][4], const float4 oml,
                                           const float4* other_o, int lane) {
  const float n0 = fmaxf(m0, oml.x), n1 = fmaxf(m1, oml.y);
  const float ws0 = (m0 == -INFINITY) ? 0.f : mv::fast_exp2(m0 - n0), wo0 = (oml.x == -INFINITY) ? 0.f : mv::fast_exp2(oml.x - n0);
  const float ws1 = (m1 == -INFINITY) ? 0.f : mv::fast_exp2(m1 - n1), wo1 = (oml.y == -INFINITY) ? 0.f : mv::fast_exp2(oml.y - n1);
  m0 = n0; m1 = n1;
  l0 = l0 * ws0 + oml.z * wo0;
  l1 = l1 * ws1 + oml.w * wo1;
#pragma unroll
  for (int i = 0; i < DT; ++i) {
    const float4 t = other_o[i * 32 + lane];
    o[i][0] = o[i][0] * ws0 + t.x * wo0;
    o[i][1] = o[i][1] * ws0 + t.y * wo0;
    o[i][2] = o[i][2] * ws1 + t.z * wo1;
    o[i][3] = o[i][3] * ws1 + t.w * wo1;
  }
}

// Consumes all stages of unit `cu` with MT m-tiles of 16 q-vectors; warp w: m-tile (w % MT), kv split (w / MT).
template <int D, int MT>
__device__ __forceinline__ void process_unit(const DecodeArgs& a, const Unit& cu, const Unit& nu, Loader<D>& ld, int& consumed,
                                             unsigned char* smem, uint32_t smem_base, const Sync& sy, const CUtensorMap* tm_k,
                                             const CUtensorMap* tm_v, int32_t pending, int32_t* s_next) {
  constexpr int KS = 4 / MT;      // kv splits inside a stage
  constexpr int WT = ST / KS;     // tokens per warp per stage
  constexpr int NT = WT / 8;      // S n-tiles per warp
  constexpr int KSTEPS = D / 16;  // k-steps of QK^T
  constexpr int DT = D / 8;       // O n-tiles
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mt = warp % MT, ks = warp / MT;
  const int nqv = cu.n_rows * a.G;

  // ---- this thread's two q rows, straight from global memory into the A-fragment layout
  uint32_t qf[KSTEPS][4];
  int part0 = -1, part1 = -1;  // partial slot (x Hq + head) of the two rows, -1 = padding row
  {
    const int x0 = mt * 16 + (lane >> 2), x1 = x0 + 8;
    const uint32_t* p0 = nullptr;
    const uint32_t* p1 = nullptr;
    if (x0 < nqv) {
      const mv::ItemRow ir = a.item_rows[cu.row_begin + x0 / a.G];
      const int head = cu.kvh * a.G + x0 % a.G;
      p0 = reinterpret_cast<const uint32_t*>(a.q + (int64_t(ir.row) * a.Hq + head) * D) + (lane & 3);
      part0 = ir.part * a.Hq + head;
    }
    if (x1 < nqv) {
      const mv::ItemRow ir = a.item_rows[cu.row_begin + x1 / a.G];
      const int head = cu.kvh * a.G + x1 % a.G;
      p1 = reinterpret_cast<const uint32_t*>(a.q + (int64_t(ir.row) * a.Hq + head) * D) + (lane & 3);
      part1 = ir.part * a.Hq + head;
    }
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      qf[kk][0] = p0 ? __ldg(p0 + kk * 8) : 0u;
      qf[kk][1] = p1 ? __ldg(p1 + kk * 8) : 0u;
      qf[kk][2] = p0 ? __ldg(p0 + kk * 8 + 4) : 0u;
      qf[kk][3] = p1 ? __ldg(p1 + kk * 8 + 4) : 0u;
    }
  }

  float oacc[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // rows lane/4 and lane/4 + 8 of the m-tile
  const int tok_w = ks * WT;                                  // first token of this warp inside a stage

  for (int s = 0; s < cu.n_stages; ++s) {
    if (tid == 0) {
      ld.top_up(a, cu, nu, smem_base, sy, tm_k, tm_v, consumed);
      if (s == 0) *s_next = pending;  // unit after `nu`; read by everyone after this unit's epilogue
    }
    const int b = consumed % NSTAGES;
    wait_or_flag(sy, sy.full + 8 * b, (consumed / NSTAGES) & 1);
    const uint32_t kb = smem_base + b * Cfg<D>::STAGE_BYTES, vb = kb + Cfg<D>::KV_BYTES;
    ++consumed;
    const bool last = (s == cu.n_stages - 1);
    const int tok_lim = cu.n_tokens - (s * ST + tok_w);  // valid tokens of this warp's slice
    if (tok_lim > 0) {                                   // warp-uniform
      if (tok_lim < WT) {
        // ragged end of the node: rows past the last token hold whatever the page (or an older stage) left
        // there; V must be zero where P is zero, or 0 * NaN would poison the output
        const int r0 = tok_w + tok_lim, nz = (WT - tok_lim) * Cfg<D>::CPR;
        for (int i = lane; i < nz; i += 32) {
          const int r = r0 + i / Cfg<D>::CPR, c = i % Cfg<D>::CPR;
          *reinterpret_cast<uint4*>(smem + (vb - smem_base) + tile_off<D>(r, c)) = make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
      }
      float sacc[NT][4];
#pragma unroll
      for (int i = 0; i < NT; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
          uint32_t bq[4];
          const int tok = tok_w + np * 16 + (lane & 7) + ((lane >> 4) << 3);
          mv::ldmatrix_x4(bq, kb + tile_off<D>(tok, kk * 2 + ((lane >> 3) & 1)));
          mv::mma_bf16_16816(sacc[2 * np], qf[kk], bq[0], bq[1]);
          mv::mma_bf16_16816(sacc[2 * np + 1], qf[kk], bq[2], bq[3]);
        }
      }
      // scale to log2 units, mask the ragged tail, online softmax
      float mx0 = -INFINITY, mx1 = -INFINITY;
      if (tok_lim >= WT) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) sacc[nt][e] *= a.scale_log2;
          mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
        }
      } else {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
            sacc[nt][e] = (col < tok_lim) ? sacc[nt][e] * a.scale_log2 : -INFINITY;
          }
          mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);  // finite: column 0 of the slice is valid
      const bool grow = (mn0 > m0) || (mn1 > m1);
      if (__any_sync(0xffffffffu, grow)) {  // rescale only when some row's maximum moved
        const float al0 = mv::fast_exp2(m0 - mn0), al1 = mv::fast_exp2(m1 - mn1);
        l0 *= al0;
        l1 *= al1;
#pragma unroll
        for (int i = 0; i < DT; ++i) {
          oacc[i][0] *= al0; oacc[i][1] *= al0;
          oacc[i][2] *= al1; oacc[i][3] *= al1;
        }
        m0 = mn0;
        m1 = mn1;
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        sacc[nt][0] = mv::fast_exp2(sacc[nt][0] - m0);
        sacc[nt][1] = mv::fast_exp2(sacc[nt][1] - m0);
        sacc[nt][2] = mv::fast_exp2(sacc[nt][2] - m1);
        sacc[nt][3] = mv::fast_exp2(sacc[nt][3] - m1);
        l0 += sacc[nt][0] + sacc[nt][1];  // per-thread partial sums; reduced over the quad at the end
        l1 += sacc[nt][2] + sacc[nt][3];
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
          uint32_t bv[4];
          const int tok = tok_w + kt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
          mv::ldmatrix_x4_trans(bv, vb + tile_off<D>(tok, dp * 2 + (lane >> 4)));
          mv::mma_bf16_16816(oacc[2 * dp], pa, bv[0], bv[1]);
          mv::mma_bf16_16816(oacc[2 * dp + 1], pa, bv[2], bv[3]);
        }
      }
    }
    if (!last) {  // hand the stage back; the unit's last stage is kept as scratch for the epilogue
      __syncwarp();
      if (lane == 0) mv::mbar_arrive(sy.empty + 8 * b);
    }
  }

  // ---- epilogue: combine the KS kv-splits through the stage buffer that was consumed last, then write one
  // partial per q-vector
  const int b_last = (consumed - 1) % NSTAGES;
  if (KS > 1) {
    float4* sc_o = reinterpret_cast<float4*>(smem + b_last * Cfg<D>::STAGE_BYTES);  // [2][DT][32]
    float4* sc_ml = sc_o + 2 * DT * 32;                                             // [2][32]
    __syncthreads();  // everyone has finished reading the last stage
    if (KS == 4) {
      if (warp >= 2) {
        float4* so = sc_o + (warp - 2) * DT * 32;
#pragma unroll
        for (int i = 0; i < DT; ++i) so[i * 32 + lane] = make_float4(oacc[i][0], oacc[i][1], oacc[i][2], oacc[i][3]);
        sc_ml[(warp - 2) * 32 + lane] = make_float4(m0, m1, l0, l1);
      }
      __syncthreads();
      if (warp < 2) merge_frag<DT>(m0, m1, l0, l1, oacc, sc_ml[warp * 32 + lane], sc_o + warp * DT * 32, lane);
      __syncthreads();
      if (warp == 1) {
#pragma unroll
        for (int i = 0; i < DT; ++i) sc_o[i * 32 + lane] = make_float4(oacc[i][0], oacc[i][1], oacc[i][2], oacc[i][3]);
        sc_ml[lane] = make_float4(m0, m1, l0, l1);
      }
      __syncthreads();
      if (warp == 0) merge_frag<DT>(m0, m1, l0, l1, oacc, sc_ml[lane], sc_o, lane);
    } else {  // KS == 2: warps 2,3 hand their state to warps 0,1 (same m-tile)
      if (ks == 1) {
        float4* so = sc_o + mt * DT * 32;
#pragma unroll
        for (int i = 0; i < DT; ++i) so[i * 32 + lane] = make_float4(oacc[i][0], oacc[i][1], oacc[i][2], oacc[i][3]);
        sc_ml[mt * 32 + lane] = make_float4(m0, m1, l0, l1);
      }
      __syncthreads();
      if (ks == 0) merge_frag<DT>(m0, m1, l0, l1, oacc, sc_ml[mt * 32 + lane], sc_o + mt * DT * 32, lane);
    }
    mv::fence_proxy_async();  // the scratch writes precede the TMA refill of this buffer
  }
  __syncwarp();
  if (lane == 0) mv::mbar_arrive(sy.empty + 8 * b_last);
  if (ks == 0) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const int c0 = (lane & 3) * 2;
    if (part0 >= 0) {
      float* po = a.part_o + int64_t(part0) * D + c0;
#pragma unroll
      for (int i = 0; i < DT; ++i) *reinterpret_cast<float2*>(po + i * 8) = make_float2(oacc[i][0], oacc[i][1]);
      if ((lane & 3) == 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(part0) * 2) = make_float2(m0, l0);
    }
    if (part1 >= 0) {
      float* po = a.part_o + int64_t(part1) * D + c0;
#pragma unroll
      for (int i = 0; i < DT; ++i) *reinterpret_cast<float2*>(po + i * 8) = make_float2(oacc[i][2], oacc[i][3]);
      if ((lane & 3) == 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(part1) * 2) = make_float2(m1, l1);
    }
  }
}

template <int D>
__global__ void __launch_bounds__(NTHREADS, 2) decode_attn_kernel(const DecodeArgs a, const __grid_constant__ CUtensorMap tm_k,
                                                                  const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_bar[2 * NSTAGES];
  __shared__ int32_t s_ids[3];
  __shared__ int s_abort;
  const int tid = threadIdx.x;
  const uint32_t raw = mv::smem_u32(smem_raw);
  const uint32_t smem_base = (raw + 1023u) & ~1023u;  // the swizzle pattern is anchored at 1024-byte boundaries
  unsigned char* smem = smem_raw + (smem_base - raw);
  Sync sy;
  sy.full = mv::smem_u32(&s_bar[0]);
  sy.empty = mv::smem_u32(&s_bar[NSTAGES]);
  sy.abort = &s_abort;
  sy.status = a.sched + 2;
  if (tid == 0) {
    s_abort = 0;
    for (int i = 0; i < NSTAGES; ++i) {
      mv::mbar_init(sy.full + 8 * i, 1);   // the producer's arrive (+ the bytes TMA reports)
      mv::mbar_init(sy.empty + 8 * i, 4);  // one arrive per consumer warp
    }
    mv::mbar_fence_init();
    mv::fence_proxy_async();
    s_ids[0] = atomicAdd(a.sched, 1);
    s_ids[1] = atomicAdd(a.sched, 1);
  }
  __syncthreads();
  Unit cu = load_unit(a, s_ids[0]);
  Unit nu = load_unit(a, s_ids[1]);
  Loader<D> ld;
  int consumed = 0;
  if (tid == 0) {
    ld.prefetch_pages(a, cu, nu);
    ld.top_up(a, cu, nu, smem_base, sy, &tm_k, &tm_v, consumed);
  }
  while (cu.n_stages > 0) {
    int32_t pending = 0;
    if (tid == 0) pending = atomicAdd(a.sched, 1);  // the unit after `nu`; published one stage later
    const int nqv = cu.n_rows * a.G;
    if (nqv <= 16) process_unit<D, 1>(a, cu, nu, ld, consumed, smem, smem_base, sy, &tm_k, &tm_v, pending, &s_ids[2]);
    else if (nqv <= 32) process_unit<D, 2>(a, cu, nu, ld, consumed, smem, smem_base, sy, &tm_k, &tm_v, pending, &s_ids[2]);
    else process_unit<D, 4>(a, cu, nu, ld, consumed, smem, smem_base, sy, &tm_k, &tm_v, pending, &s_ids[2]);
    __syncthreads();  // s_ids[2] is visible to everyone
    cu = nu;
    nu = load_unit(a, s_ids[2]);
    __syncthreads();  // s_ids[2] may be overwritten from here on
    if (tid == 0) {
      // the loader had finished the old `cu` (it was consumed), so it stands in the old `nu` or beyond it
      ld.which -= 1;
      if (ld.which == 1) ld.prefetch_pages(a, cu, nu);  // it was beyond: it now stands at the first stage of the new `nu`
      ld.top_up(a, cu, nu, smem_base, sy, &tm_k, &tm_v, consumed);
    }
  }
  // every stage that was issued has been consumed (the loader never runs past `nu`, and `nu` is empty here)
  if (tid == 0) {
    __threadfence();
    const int done = atomicAdd(a.sched + 1, 1);
    if (done == int(gridDim.x) - 1) {  // the last CTA to finish re-arms the scheduler words for the next launch
      a.sched[0] = 0;
      a.sched[1] = 0;
      __threadfence();
    }
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
    const float2 ml = *reinterpret_cast<const float2*>(part_ml + ps * 2);
    const float wgt = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - m);
    l += wgt * ml.y;
    const float* po = part_o + ps * D + lane * E;
    if (E == 4) {
      const float4 t = *reinterpret_cast<const float4*>(po);
      acc[0] += wgt * t.x; acc[1] += wgt * t.y; acc[2] += wgt * t.z; acc[3 % E] += wgt * t.w;
    } else {
      const float2 t = *reinterpret_cast<const float2*>(po);
      acc[0] += wgt * t.x; acc[1] += wgt * t.y;
    }
  }
  const float inv = 1.f / l;
  bf16* o = out + (int64_t(row) * Hq + h) * D + lane * E;
#pragma unroll
  for (int e = 0; e < E; e += 2) *reinterpret_cast<__nv_bfloat162*>(o + e) = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = 148;
    }
  }
  return n;
}

struct TmapCache {  // the pools rarely change between calls: keep the last pair of tensor maps
  const void* k = nullptr;
  const void* v = nullptr;
  int64_t rows = 0;
  int d = 0;
  CUtensorMap tm_k, tm_v;
};

template <int D>
mv_status launch(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, void* out,
                 void* ws, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(decode_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::SMEM) != cudaSuccess) {
      (void)cudaGetLastError();
      return MV_ERR_CUDA;
    }
    attr_set = true;
  }
  static thread_local TmapCache tc[4];
  static thread_local int tc_next = 0;
  const int64_t rows = g->num_pages * g->n_kv_heads * 16;
  TmapCache* hit = nullptr;
  for (auto& c : tc)
    if (c.k == kp && c.v == vp && c.rows == rows && c.d == D) hit = &c;
  if (!hit) {
    hit = &tc[tc_next];
    tc_next = (tc_next + 1) % 4;
    hit->k = nullptr;
    if (!mv::make_tmap_bf16_2d(&hit->tm_k, kp, uint64_t(rows), D, 16) || !mv::make_tmap_bf16_2d(&hit->tm_v, vp, uint64_t(rows), D, 16))
      return MV_ERR_CUDA;
    hit->k = kp; hit->v = vp; hit->rows = rows; hit->d = D;
  }
  const size_t parts = size_t(P->stats.n_partials);
  const size_t o_bytes = (parts * g->n_q_heads * D * sizeof(float) + 255) & ~size_t(255);
  DecodeArgs a;
  a.q = static_cast<const bf16*>(q);
  a.page_idx = mv::table<int32_t>(P, P->layout.page_idx);
  a.items = mv::table<mv::WorkItem>(P, P->layout.items);
  a.item_rows = mv::table<mv::ItemRow>(P, P->layout.item_rows);
  a.part_o = static_cast<float*>(ws);
  a.part_ml = reinterpret_cast<float*>(static_cast<char*>(ws) + o_bytes);
  a.sched = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched));
  a.Hq = g->n_q_heads;
  a.Hkv = g->n_kv_heads;
  a.G = g->n_q_heads / g->n_kv_heads;
  a.n_units = int(P->stats.n_items) * g->n_kv_heads;
  a.scale_log2 = mv::softmax_scale(g) * 1.4426950408889634f;
  const int grid = std::min(a.n_units, 2 * sm_count());
  decode_attn_kernel<D><<<grid, NTHREADS, Cfg<D>::SMEM, st>>>(a, hit->tm_k, hit->tm_v);
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
  if (P->stats.n_new_tokens == 0) return MV_OK;
  if (g->dtype != MV_BF16 || !P->stats.decode_ready) return MV_ERR_UNSUPPORTED;
  if (P->stats.max_item_rows * (g->n_q_heads / g->n_kv_heads) > 64) return MV_ERR_UNSUPPORTED;
  if (!q_rot || !k_pages || !v_pages || !out) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  if (P->stats.max_page_id >= g->num_pages) return MV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_pages) & 15) || (reinterpret_cast<uintptr_t>(v_pages) & 15)) return MV_ERR_INVALID_ARG;
  const size_t need = mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  return g->head_dim == 128 ? launch<128>(P, g, q_rot, k_pages, v_pages, out, workspace, s)
                            : launch<64>(P, g, q_rot, k_pages, v_pages, out, workspace, s);
}

// ---- decode attention for callers that cannot allocate device memory -------------------------------------
// The split-KV scratch lives in a file-scope device array instead of a caller-provided workspace.  In host
// code the array's name is only a stand-in for the symbol, not a device address, so the address the kernels
// receive is looked up with cudaGetSymbolAddress, once per device, with that device current.
namespace {
__device__ __align__(256) unsigned char g_static_scratch[MV_STATIC_WORKSPACE_BYTES];
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};
std::mutex g_static_scratch_mu;

mv_status static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_static_scratch_mu);
  if (!g_static_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return MV_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = p;
  }
  *out = g_static_scratch_addr[dev];
  return MV_OK;
}
}  // namespace

extern "C" size_t mv_static_workspace_bytes(void) { return size_t(MV_STATIC_WORKSPACE_BYTES); }

extern "C" mv_status mv_dag_decode_attn_static(const mv_plan* P, const mv_attn_geom* g, const void* q_rot,
                                               const void* k_pages, const void* v_pages, void* out, void* cuda_stream) {
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  // the size check comes before anything touches the device: a plan that needs more scratch than the library
  // holds is refused, never truncated
  if (mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN) > size_t(MV_STATIC_WORKSPACE_BYTES)) return MV_ERR_WORKSPACE;
  void* scratch = nullptr;
  st = static_scratch_for_current_device(&scratch);
  if (st != MV_OK) return st;
  return mv_dag_decode_attn(P, g, q_rot, k_pages, v_pages, out, scratch, size_t(MV_STATIC_WORKSPACE_BYTES), cuda_stream);
}

extern "C" mv_status mv_plan_read_status(const mv_plan* P, void* cuda_stream, int32_t* status) {
  if (!P || !P->valid || !status) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const char* src = static_cast<const char*>(P->device_buf) + P->layout.sched + 2 * sizeof(int32_t);
  if (cudaMemcpyAsync(status, src, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  return MV_OK;
}
