// Multi-branch decode attention over a shared paged KV cache (Eq. 2 with the DAG mask of Eq. 3; Fork =
// shared prefix pages referenced by many rows, Join = union of the predecessors' segment lists, Sec. 4.3).
//
// Segment-major: a request's frontier rows and all the KV they see form one stream of 64-token stages, node
// after node; a stage belongs to one node and carries the set of rows that see that node (the DAG mask at
// stage granularity).  The unit of work is a run of such stages for one KV head.  Every stage is streamed
// from HBM exactly once and serves every sibling row and the whole GQA group: the q-vectors (rows x group)
// are the M dimension of bf16 tensor-core tiles (m16n8k16, fp32 accumulate), so that the arithmetic (16-64
// flop per KV byte) does not throttle the HBM stream; rows that do not see a stage's node are masked out of
// its softmax, and a warp none of whose rows see it skips it.
//
// The planner cuts the step's whole KV stream into one equal share per CTA (two CTAs per SM), so there is
// no run-time scheduler.  A CTA is one producer warp and four consumer warps around ONE ring of 64-token
// stages that keeps running across unit boundaries.  The producer fills a stage with TMA: one box per
// contiguous (page, KV head) block of K and of V (cp.async.bulk.tensor, 128-byte shared-memory swizzle,
// completion counted on an mbarrier), eight lanes issuing one box each; it also stages the next unit's
// q-vectors and partial-slot ids in shared memory (cp.async, completion on an mbarrier) while the current
// unit is still being consumed.  Consumers hand a stage back through a second mbarrier.  Softmax is
// online, in log2 units; each unit leaves one partial (max, sum, unnormalised output) per q-vector in the
// split-KV workspace and a second kernel, launched with programmatic stream serialisation so that its
// launch overlaps this kernel's tail, merges the partials of every (row, head).
//
// Every wait on an mbarrier is bounded: if it runs out, the CTA records MV_ERR_TIMEOUT in the plan's
// status word, stops waiting and still reaches every barrier, so the kernel always terminates.
#include <mutex>

#include "common.cuh"
#include "trace.h"
#include "tmap_cache.h"

namespace mv {
mv_status append_tc(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_pages, const void* v_pages, void* out,
                    cudaStream_t st);
mv_status decode_tc(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, void* ws,
                    cudaStream_t st);
mv_status decode_fp8(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, const float* kv_scale,
                     void* ws, cudaStream_t st);
}

namespace {

using bf16 = __nv_bfloat16;
constexpr int NCONS = 128;           // consumer threads (4 warps)
constexpr int NTHREADS = NCONS + 32; // + the producer warp (warp 4)
constexpr int ST = 64;               // tokens per pipeline stage (4 pages)
constexpr int NSTAGES = 3;
constexpr int MAXQV = 64;            // q-vectors (rows x group) of one unit

struct DecodeArgs {
  const bf16* q;
  const mv::StageDesc* stages;
  const mv::WorkUnit* units;
  const int32_t* cta_unit_off;
  const mv::WorkUnit* cta_head;  // each CTA's first unit with its unit range in pad[0], pad[1]
  const mv::ItemRow* item_rows;
  float* part_o;    // [n_partials * G][D]
  float* part_ml;   // [n_partials * G][2]  (max in log2 units, sum)
  int32_t* status;  // device status word
  int Hq, Hkv, G;
  float scale_log2;  // softmax scale * log2(e)
};

template <int D>
struct Cfg {
  static constexpr int CPR = D / 8;                 // 16-byte chunks per token row
  static constexpr int HALVES = D / 64;             // 128-byte column blocks per row (one TMA box each)
  static constexpr int PAGE_BYTES = 16 * D * 2;     // K (or V) block of one (page, KV head): one TMA box
  static constexpr int KV_BYTES = ST * D * 2;       // K (or V) bytes of a stage
  static constexpr int STAGE_BYTES = 2 * KV_BYTES;  // K then V
  static constexpr int Q_BYTES = MAXQV * D * 2;     // q-vectors of one unit, [64][D] bf16, chunk-swizzled
  // dynamic shared memory: stages | q | meta (see Smem)
  static constexpr int OFF_Q = NSTAGES * STAGE_BYTES;
  static constexpr int OFF_META = OFF_Q + Q_BYTES;
  static constexpr int SMEM = OFF_META + 1024;  // D = 128: 115,712 B, the most that lets two CTAs share an SM
};

struct Meta {                       // tail of the dynamic shared memory
  float2 ml[4][16];                 // epilogue: (max, sum) of every row of every consumer warp    512 B
  int32_t pv[MAXQV];                // partial vector index (partial * G + head in group) or -1    256 B
  int32_t n_stages, n_qv;
  uint32_t st_tokens[NSTAGES];      // per stage buffer: valid tokens of the four page slots, a byte each
  uint2 st_mask[NSTAGES][4];        // per stage buffer and page slot: rows that see the slot's node (lo, hi)
  uint64_t full[NSTAGES], empty[NSTAGES], q_full, q_empty;
  int abort;
};
static_assert(sizeof(Meta) <= 1024, "meta area");

// Byte offset of 16-byte chunk `chunk` of token row `row` inside a K (or V) stage tile as TMA lays it out: a
// stage is four page blocks; a page block is [column block chunk / 8][16 tokens][128 B], and inside a
// 128-byte row the hardware XORs the chunk index with row % 8.
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return uint32_t(row >> 4) * Cfg<D>::PAGE_BYTES + uint32_t(chunk >> 3) * 2048 + uint32_t(row & 15) * 128 +
         (uint32_t((chunk & 7) ^ (row & 7)) << 4);
}
// q buffer: row x, 16-byte chunk c at x * (D*2) + ((c ^ (x & 7)) << 4)
template <int D>
__device__ __forceinline__ uint32_t q_off(int x, int c) {
  return uint32_t(x) * (D * 2) + (uint32_t(c ^ (x & 7)) << 4);
}

struct Sync {
  uint32_t full, empty, q_full, q_empty;  // shared-memory addresses
  volatile int* abort;                    // set once a bounded wait ran out
  int32_t* status;                        // global status word
};

// Bounded wait.  False once a wait of this CTA has run out (this one or an earlier one): the producer then issues no
// further copy and waits for those in flight; the consumers only read shared memory and finish their lists.
__device__ __forceinline__ bool wait_or_flag(const Sync& sy, uint32_t bar, uint32_t parity) {
  if (*sy.abort) return false;
  if (!mv::mbar_wait_bounded(bar, parity, 2000000000ull, sy.abort)) {
    if (!*sy.abort) atomicExch(sy.status, int(MV_ERR_TIMEOUT));
    *sy.abort = 1;
    return false;
  }
  return true;
}

// ---- producer warp: walks the CTA's units; per unit the q-vectors + slot ids, then the KV stages -----------------
struct UnitRegs {  // a unit's descriptor, loaded ahead of use
  int stage_begin = 0, n_stages = 0, row_begin = 0, n_rows = 0, kvh = 0;
};
struct StageRegs {  // one stage descriptor per lane (a window of 32 stages)
  int4 a = make_int4(0, 0, 0, 0), b = make_int4(0, 0, 0, 0), c = make_int4(0, 0, 0, 0), d = make_int4(0, 0, 0, 0);
};

template <int D>
__device__ __forceinline__ void producer(const DecodeArgs& a, uint32_t smem_base, Meta* meta, const Sync& sy, const CUtensorMap* tm_k,
                                         const CUtensorMap* tm_v) {
  const int lane = threadIdx.x & 31;
  // one load at a known address gives the CTA's unit range and its first unit
  UnitRegs wu;
  int u_begin, u_end;
  {
    const int4* p = reinterpret_cast<const int4*>(a.cta_head + blockIdx.x);
    const int4 x = __ldg(p), y = __ldg(p + 1);
    wu.stage_begin = x.x; wu.n_stages = x.y; wu.row_begin = x.z; wu.n_rows = x.w; wu.kvh = y.x;
    u_begin = y.y;
    u_end = y.z;
  }
  int issued = 0;  // stages issued so far (buffer = issued % NSTAGES)
  const uint64_t kv_policy = mv::l2_policy_evict_first();  // the KV stream is read once per call
  // Table reads run ahead of their use so that no load sits on the issue path: the descriptor of unit u + 2,
  // and the row list and first stage window of unit u + 1, are requested while unit u is being issued.
  auto load_unit = [&](int u) {
    UnitRegs w;
    if (u < u_end) {
      const int4* p = reinterpret_cast<const int4*>(a.units + u);
      const int4 x = __ldg(p), y = __ldg(p + 1);
      w.stage_begin = x.x; w.n_stages = x.y; w.row_begin = x.z; w.n_rows = x.w; w.kvh = y.x;
    }
    return w;
  };
  auto load_rows = [&](const UnitRegs& w, int base) {
    return base + lane < w.n_rows ? a.item_rows[w.row_begin + base + lane] : mv::ItemRow{-1, -1};
  };
  auto load_window = [&](const UnitRegs& w, int first) {  // stages first + lane of the unit
    StageRegs r;
    if (first + lane < w.n_stages) {
      const int4* p = reinterpret_cast<const int4*>(a.stages + w.stage_begin + first + lane);
      r.a = __ldg(p);      // pages
      r.b = __ldg(p + 1);  // tokens per slot, slots in use, mask_lo[0..1]
      r.c = __ldg(p + 2);  // mask_lo[2..3], mask_hi[0..1]
      r.d = __ldg(p + 3);  // mask_hi[2..3]
    }
    return r;
  };
  UnitRegs wu1 = load_unit(u_begin + 1);
  mv::ItemRow ir0 = load_rows(wu, 0), ir1 = load_rows(wu, 32);
  StageRegs win = load_window(wu, 0);
  bool ok = true;  // warp-uniform: no wait of this CTA has run out
  for (int u = u_begin; u < u_end && ok; ++u) {
    const int ui = u - u_begin;
    const UnitRegs wu2 = load_unit(u + 2);
    const mv::ItemRow nir0 = load_rows(wu1, 0), nir1 = load_rows(wu1, 32);
    const StageRegs nwin = load_window(wu1, 0);
    // ---- q-vectors and partial-slot ids of this unit
    const int n_qv = wu.n_rows * a.G;
    const int n_pad = min(MAXQV, (n_qv + 15) & ~15);
    {
      int go = 1;
      if (lane == 0) go = wait_or_flag(sy, sy.q_empty, (ui & 1) ^ 1) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, go, 0) != 0;
    }
    if (!ok) break;
    for (int x = lane; x < MAXQV; x += 32) {  // every lane takes part in the shuffles
      const int r = min(x / a.G, MAXQV - 1);
      const int p_lo = __shfl_sync(0xffffffffu, ir0.part, r & 31), p_hi = __shfl_sync(0xffffffffu, ir1.part, r & 31);
      const int part = r < 32 ? p_lo : p_hi;
      meta->pv[x] = (x < n_qv && part >= 0) ? part * a.G + x % a.G : -1;
    }
    if (lane == 0) {
      meta->n_stages = wu.n_stages;
      meta->n_qv = n_qv;
    }
    for (int i0 = 0; i0 < n_pad * Cfg<D>::CPR; i0 += 32) {  // n_pad * CPR is a multiple of 32
      const int i = i0 + lane;
      const int x = i / Cfg<D>::CPR, c = i % Cfg<D>::CPR;
      const int r = min(x / a.G, MAXQV - 1);
      const int r_lo = __shfl_sync(0xffffffffu, ir0.row, r & 31), r_hi = __shfl_sync(0xffffffffu, ir1.row, r & 31);
      const int row = r < 32 ? r_lo : r_hi;
      const bool ok = x < n_qv;
      const bf16* src = a.q + (ok ? (int64_t(row) * a.Hq + wu.kvh * a.G + x % a.G) * D + c * 8 : 0);
      mv::cp_async_16(smem_base + Cfg<D>::OFF_Q + q_off<D>(x, c), src, ok ? 16 : 0);  // padding rows are zero-filled
    }
    mv::cp_async_mbar_arrive_noinc(sy.q_full);  // 32 arrivals, each when the lane's copies have landed
    __syncwarp();                               // the lanes' meta stores precede lane 0's releasing arrive
    if (lane == 0) mv::mbar_arrive(sy.q_full);
    // ---- KV stages, 32 descriptors per window
    StageRegs nxt;
    for (int s = 0; s < wu.n_stages && ok; ++s) {
      if ((s & 31) == 0) {
        if (s > 0) win = nxt;
        nxt = load_window(wu, s + 32);
      }
      const int src = s & 31;
      const int4 da = make_int4(__shfl_sync(0xffffffffu, win.a.x, src), __shfl_sync(0xffffffffu, win.a.y, src),
                                __shfl_sync(0xffffffffu, win.a.z, src), __shfl_sync(0xffffffffu, win.a.w, src));
      const int n_pages = __shfl_sync(0xffffffffu, win.b.y, src);
      const int b = issued % NSTAGES;
      const uint32_t bar = sy.full + 8 * b;
      {
        int go = 1;
        if (lane == 0) go = wait_or_flag(sy, sy.empty + 8 * b, ((issued / NSTAGES) & 1) ^ 1) ? 1 : 0;  // every consumer warp has released the buffer
        ok = __shfl_sync(0xffffffffu, go, 0) != 0;
      }
      if (!ok) break;
      if (lane == src) {  // the lane that holds the descriptor publishes the page slots' token counts and row masks
        meta->st_tokens[b] = uint32_t(win.b.x);
        meta->st_mask[b][0] = make_uint2(uint32_t(win.b.z), uint32_t(win.c.z));
        meta->st_mask[b][1] = make_uint2(uint32_t(win.b.w), uint32_t(win.c.w));
        meta->st_mask[b][2] = make_uint2(uint32_t(win.c.x), uint32_t(win.d.x));
        meta->st_mask[b][3] = make_uint2(uint32_t(win.c.y), uint32_t(win.d.y));
      }
      __syncwarp();
      if (lane == 0) mv::mbar_arrive_expect_tx(bar, uint32_t(n_pages) * 16 * D * 2 * 2);  // releases the stores above
      // lane j < 8: page j / 2 of the stage, K or V; one box = the whole contiguous (page, head) block
      const int p = (lane >> 1) & 3, kv = lane & 1;
      const int page = p == 0 ? da.x : p == 1 ? da.y : p == 2 ? da.z : da.w;
      if (lane < 8 && p < n_pages) {
        const int row = (page * a.Hkv + wu.kvh) * (16 * Cfg<D>::HALVES);
        const uint32_t dst = smem_base + b * Cfg<D>::STAGE_BYTES + kv * Cfg<D>::KV_BYTES + p * Cfg<D>::PAGE_BYTES;
        mv::tma_load_2d_hint(dst, kv ? tm_v : tm_k, 0, row, bar, kv_policy);
      }
      ++issued;
    }
    wu = wu1;
    wu1 = wu2;
    ir0 = nir0;
    ir1 = nir1;
    win = nwin;
  }
  if (!ok) {
    // a wait ran out: what is still in flight must land before the CTA may return (a bulk copy that completes into the
    // shared memory of a CTA that has left corrupts whoever runs there next)
    mv::cp_async_wait_all();
    if (lane == 0)
      for (int k = 1; k <= min(issued, NSTAGES); ++k)
        (void)mv::mbar_wait_bounded(sy.full + 8 * ((issued - k) % NSTAGES), ((issued - k) / NSTAGES) & 1, 20000000ull);
    __syncwarp();
  }
}

// ---- consumer side ---------------------------------------------------------------------------------------
// Consumes all stages of one unit with MT m-tiles of 16 q-vectors; warp w: m-tile (w % MT), kv split (w / MT).
template <int D, int MT>
__device__ __forceinline__ void consume_unit(const DecodeArgs& a, int n_stages, int pv0, int pv1, int row0, int row1, uint64_t tile_rows,
                                             const uint32_t (&qf)[D / 16][4], int& consumed, unsigned char* smem, uint32_t smem_base,
                                             Meta* meta, const Sync& sy) {
  constexpr int KS = 4 / MT;      // kv splits inside a stage
  constexpr int WT = ST / KS;     // tokens per warp per stage
  constexpr int NT = WT / 8;      // S n-tiles per warp
  constexpr int KSTEPS = D / 16;  // k-steps of QK^T
  constexpr int DT = D / 8;       // O n-tiles
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mt = warp % MT, ks = warp / MT;
  (void)mt;

  float oacc[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // rows lane/4 and lane/4 + 8 of the m-tile
  const int tok_w = ks * WT;                                  // first token of this warp inside a stage
  int b = 0;

  for (int s = 0; s < n_stages; ++s) {
    b = consumed % NSTAGES;
    wait_or_flag(sy, sy.full + 8 * b, (consumed / NSTAGES) & 1);
    const uint32_t kb = smem_base + b * Cfg<D>::STAGE_BYTES, vb = kb + Cfg<D>::KV_BYTES;
    ++consumed;
    const bool last = (s == n_stages - 1);
    // this warp's slice of the stage is NT / 2 page slots; each has its own valid-token count and row mask
    constexpr int NS = NT / 2;
    const int slot0 = tok_w >> 4;
    const uint32_t tok4 = meta->st_tokens[b] >> (8 * slot0);
    uint64_t seen_by[NS];
    int ntok[NS];
    bool any_work = false, plain = true;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
      const uint2 mk = meta->st_mask[b][slot0 + j];
      seen_by[j] = (uint64_t(mk.y) << 32) | mk.x;
      ntok[j] = int((tok4 >> (8 * j)) & 0xffu);
      any_work |= ntok[j] > 0 && (seen_by[j] & tile_rows) != 0;
      plain &= ntok[j] == 16 && (seen_by[j] & tile_rows) == tile_rows;
    }
    if (any_work) {  // warp-uniform: some row of this m-tile sees some token of the slice
      if (!plain) {
        // rows past a page's last token hold whatever the pool (or an older stage) left there; V must be
        // zero where P is zero, or 0 * NaN would poison the output
#pragma unroll
        for (int j = 0; j < NS; ++j) {
          const int nz = (16 - ntok[j]) * Cfg<D>::CPR;
          for (int i = lane; i < nz; i += 32) {
            const int r = tok_w + j * 16 + ntok[j] + i / Cfg<D>::CPR, c = i % Cfg<D>::CPR;
            *reinterpret_cast<uint4*>(smem + (vb - smem_base) + tile_off<D>(r, c)) = make_uint4(0, 0, 0, 0);
          }
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
      if (plain) {  // every row of the m-tile sees every token of the slice
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) sacc[nt][e] *= a.scale_log2;
          mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
        }
      } else {  // the DAG mask (a row that does not see the page's node) and the ragged last page of a node
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int j = nt >> 1;
          const bool vis0 = row0 >= 0 && ((seen_by[j] >> row0) & 1), vis1 = row1 >= 0 && ((seen_by[j] >> row1) & 1);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = (nt & 1) * 8 + (lane & 3) * 2 + (e & 1);  // token inside the page
            sacc[nt][e] = (col < ntok[j] && (e < 2 ? vis0 : vis1)) ? sacc[nt][e] * a.scale_log2 : -INFINITY;
          }
          mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);  // still -inf for a row that has seen nothing yet
      const bool grow = (mn0 > m0) || (mn1 > m1);
      if (__any_sync(0xffffffffu, grow)) {  // rescale only when some row's maximum moved
        const float al0 = mv::fast_exp2(m0 - (mn0 == -INFINITY ? 0.f : mn0)), al1 = mv::fast_exp2(m1 - (mn1 == -INFINITY ? 0.f : mn1));
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
      const float e0 = (m0 == -INFINITY) ? 0.f : m0, e1 = (m1 == -INFINITY) ? 0.f : m1;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        sacc[nt][0] = mv::fast_exp2(sacc[nt][0] - e0);
        sacc[nt][1] = mv::fast_exp2(sacc[nt][1] - e0);
        sacc[nt][2] = mv::fast_exp2(sacc[nt][2] - e1);
        sacc[nt][3] = mv::fast_exp2(sacc[nt][3] - e1);
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
    if (!last || KS == 1) {  // hand the stage back; with kv splits the unit's last stage is kept as epilogue scratch
      mv::fence_proxy_async();  // a ragged page may have been patched with ordinary stores; TMA refills the buffer next
      __syncwarp();
      if (lane == 0) mv::mbar_arrive(sy.empty + 8 * b);
    }
  }

  // ---- epilogue: one partial (m, l, unnormalised o) per q-vector
  const int c0 = (lane & 3) * 2;
  if (KS == 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    if (pv0 >= 0) {
      float* po = a.part_o + int64_t(pv0) * D + c0;
#pragma unroll
      for (int i = 0; i < DT; ++i) *reinterpret_cast<float2*>(po + i * 8) = make_float2(oacc[i][0], oacc[i][1]);
      if ((lane & 3) == 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(pv0) * 2) = make_float2(m0, l0);
    }
    if (pv1 >= 0) {
      float* po = a.part_o + int64_t(pv1) * D + c0;
#pragma unroll
      for (int i = 0; i < DT; ++i) *reinterpret_cast<float2*>(po + i * 8) = make_float2(oacc[i][2], oacc[i][3]);
      if ((lane & 3) == 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(pv1) * 2) = make_float2(m1, l1);
    }
    return;
  }
  // The KS warps of an m-tile combine their states through the stage buffer that was consumed last
  // ([warp][n-tile][lane] float4, exactly one stage); each of them then finishes and stores DT / KS n-tiles.
  float4* sc_o = reinterpret_cast<float4*>(smem + b * Cfg<D>::STAGE_BYTES);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  mv::named_bar_sync(1, NCONS);  // every consumer has finished reading the last stage
#pragma unroll
  for (int i = 0; i < DT; ++i) sc_o[(warp * DT + i) * 32 + lane] = make_float4(oacc[i][0], oacc[i][1], oacc[i][2], oacc[i][3]);
  if ((lane & 3) == 0) {
    meta->ml[warp][lane >> 2] = make_float2(m0, l0);
    meta->ml[warp][(lane >> 2) + 8] = make_float2(m1, l1);
  }
  mv::named_bar_sync(1, NCONS);
  float w0[KS], w1[KS];
  float mm0 = -INFINITY, mm1 = -INFINITY;
#pragma unroll
  for (int k = 0; k < KS; ++k) {
    mm0 = fmaxf(mm0, meta->ml[mt + MT * k][lane >> 2].x);
    mm1 = fmaxf(mm1, meta->ml[mt + MT * k][(lane >> 2) + 8].x);
  }
  float ll0 = 0.f, ll1 = 0.f;
#pragma unroll
  for (int k = 0; k < KS; ++k) {
    const float2 t0 = meta->ml[mt + MT * k][lane >> 2], t1 = meta->ml[mt + MT * k][(lane >> 2) + 8];
    w0[k] = (t0.x == -INFINITY) ? 0.f : mv::fast_exp2(t0.x - mm0);
    w1[k] = (t1.x == -INFINITY) ? 0.f : mv::fast_exp2(t1.x - mm1);
    ll0 += w0[k] * t0.y;
    ll1 += w1[k] * t1.y;
  }
  constexpr int IPW = DT / KS;  // n-tiles this warp finishes
#pragma unroll
  for (int ii = 0; ii < IPW; ++ii) {
    const int i = ks * IPW + ii;
    float r0 = 0.f, r1 = 0.f, r2 = 0.f, r3 = 0.f;
#pragma unroll
    for (int k = 0; k < KS; ++k) {
      const float4 t = sc_o[((mt + MT * k) * DT + i) * 32 + lane];
      r0 += w0[k] * t.x; r1 += w0[k] * t.y;
      r2 += w1[k] * t.z; r3 += w1[k] * t.w;
    }
    if (pv0 >= 0) *reinterpret_cast<float2*>(a.part_o + int64_t(pv0) * D + i * 8 + c0) = make_float2(r0, r1);
    if (pv1 >= 0) *reinterpret_cast<float2*>(a.part_o + int64_t(pv1) * D + i * 8 + c0) = make_float2(r2, r3);
  }
  if (ks == 0) {
    if ((lane & 3) == 0) {
      if (pv0 >= 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(pv0) * 2) = make_float2(mm0, ll0);
      if (pv1 >= 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(pv1) * 2) = make_float2(mm1, ll1);
    }
  }
  mv::fence_proxy_async();  // the scratch accesses precede the TMA refill of this buffer
  __syncwarp();
  if (lane == 0) mv::mbar_arrive(sy.empty + 8 * b);
}

template <int D, int MT>
__device__ __forceinline__ void consumer_unit(const DecodeArgs& a, int n_stages, int n_qv, int& consumed, unsigned char* smem,
                                              uint32_t smem_base, Meta* meta, const Sync& sy) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mt = warp % MT;
  // this thread's two q rows of the m-tile, their partial slots and their rows of the row group
  const int x0 = mt * 16 + (lane >> 2), x1 = x0 + 8;
  const int pv0 = meta->pv[x0], pv1 = meta->pv[x1];
  const int row0 = x0 < n_qv ? x0 / a.G : -1, row1 = x1 < n_qv ? x1 / a.G : -1;
  uint64_t tile_rows = 0;  // rows of the row group that own a q-vector of this m-tile
  if (mt * 16 < n_qv) {
    const int r_lo = (mt * 16) / a.G, r_hi = (min(mt * 16 + 15, n_qv - 1)) / a.G;
    tile_rows = (r_hi - r_lo == 63 ? ~uint64_t(0) : ((uint64_t(1) << (r_hi - r_lo + 1)) - 1)) << r_lo;
  }
  uint32_t qf[D / 16][4];
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk)
    mv::ldmatrix_x4(qf[kk], smem_base + Cfg<D>::OFF_Q + q_off<D>(mt * 16 + (lane & 15), kk * 2 + (lane >> 4)));
  __syncwarp();
  if (lane == 0) mv::mbar_arrive(sy.q_empty);  // the unit's q buffer and header are free again
  consume_unit<D, MT>(a, n_stages, pv0, pv1, row0, row1, tile_rows, qf, consumed, smem, smem_base, meta, sy);
}

template <int D>
__global__ void __launch_bounds__(NTHREADS, 2) decode_attn_kernel(const DecodeArgs a, const __grid_constant__ CUtensorMap tm_k,
                                                                  const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t smem_base = mv::smem_u32(smem);
  Meta* meta = reinterpret_cast<Meta*>(smem + Cfg<D>::OFF_META);
  Sync sy;
  sy.full = mv::smem_u32(&meta->full[0]);
  sy.empty = mv::smem_u32(&meta->empty[0]);
  sy.q_full = mv::smem_u32(&meta->q_full);
  sy.q_empty = mv::smem_u32(&meta->q_empty);
  sy.abort = &meta->abort;
  sy.status = a.status;
  if ((smem_base & 1023u) != 0) {  // the swizzle pattern is anchored at 1024-byte boundaries
    if (tid == 0) atomicExch(a.status, int(MV_ERR_UNSUPPORTED));
    return;
  }
  if (tid == 0) {
    meta->abort = 0;
    for (int i = 0; i < NSTAGES; ++i) {
      mv::mbar_init(sy.full + 8 * i, 1);   // the producer's arrive (+ the bytes TMA reports)
      mv::mbar_init(sy.empty + 8 * i, 4);  // one arrive per consumer warp
    }
    mv::mbar_init(sy.q_full, 33);   // 32 copy-completion arrivals + the producer's releasing arrive
    mv::mbar_init(sy.q_empty, 4);   // one arrive per consumer warp
    mv::mbar_fence_init();
    mv::fence_proxy_async();
  }
  __syncthreads();
  if (warp == 4) {
    producer<D>(a, smem_base, meta, sy, &tm_k, &tm_v);
    mv::grid_dependency_launch_dependents();
    return;
  }
  const int u_begin = a.cta_unit_off[blockIdx.x], u_end = a.cta_unit_off[blockIdx.x + 1];
  int consumed = 0;
  for (int u = u_begin; u < u_end; ++u) {
    wait_or_flag(sy, sy.q_full, (u - u_begin) & 1);
    const int n_stages = meta->n_stages, n_qv = meta->n_qv;
    if (n_qv <= 16) consumer_unit<D, 1>(a, n_stages, n_qv, consumed, smem, smem_base, meta, sy);
    else if (n_qv <= 32) consumer_unit<D, 2>(a, n_stages, n_qv, consumed, smem, smem_base, meta, sy);
    else consumer_unit<D, 4>(a, n_stages, n_qv, consumed, smem, smem_base, meta, sy);
  }
  // this CTA's share is done: once every CTA got here (or exited) the merge kernel may become resident, so its
  // launch overlaps the tail of this grid; it still waits for the grid's completion before it reads a partial
  mv::grid_dependency_launch_dependents();
}

// Merge of the split-KV partials of one (row, head): one warp each.
template <int D>
__global__ void __launch_bounds__(128) decode_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                                                           const int32_t* __restrict__ rowkv_part_off, bf16* __restrict__ out,
                                                           int n_rows, int Hq, int G) {
  const int w = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (w >= n_rows * Hq) return;
  const int row = w / Hq, h = w % Hq, kvh = h / G, g = h % G;
  const int Hkv = Hq / G;
  const int p0 = rowkv_part_off[row * Hkv + kvh], p1 = rowkv_part_off[row * Hkv + kvh + 1];
  mv::grid_dependency_wait();  // the partials are complete and visible from here on
  // online merge, four partials per step: the loads of a step do not depend on one another, so a (row, head)
  // with up to four partials costs one round trip to L2
  constexpr int E = D / 32;
  float m = -INFINITY, l = 0.f;
  float acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  for (int pb = p0; pb < p1; pb += 4) {
    float2 ml[4];
    float t[4][E];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const bool ok = pb + k < p1;
      const int64_t ps = int64_t(ok ? pb + k : pb) * G + g;
      // through L2 (ld.global.cg), never the read-only path: the attention kernel writes the partials while this grid may
      // already be resident, so they are not read-only for this kernel's lifetime
      ml[k] = __ldcg(reinterpret_cast<const float2*>(part_ml + ps * 2));
      if (!ok) ml[k].x = -INFINITY;
      const float* po = part_o + ps * D + lane * E;
      if (E == 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(po));
        t[k][0] = v.x; t[k][1] = v.y; t[k][2 % E] = v.z; t[k][3 % E] = v.w;
      } else {
        const float2 v = __ldcg(reinterpret_cast<const float2*>(po));
        t[k][0] = v.x; t[k][1] = v.y;
      }
    }
    const float mn = fmaxf(fmaxf(m, fmaxf(ml[0].x, ml[1].x)), fmaxf(ml[2].x, ml[3].x));
    const float f = (m == -INFINITY) ? 0.f : exp2f(m - mn);
    l *= f;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] *= f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float wgt = (ml[k].x == -INFINITY) ? 0.f : exp2f(ml[k].x - mn);
      l += wgt * ml[k].y;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] += wgt * t[k][e];
    }
    m = mn;
  }
  const float inv = 1.f / l;
  bf16* o = out + (int64_t(row) * Hq + h) * D + lane * E;
#pragma unroll
  for (int e = 0; e < E; e += 2) *reinterpret_cast<__nv_bfloat162*>(o + e) = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
}

struct KvMaps {
  CUtensorMap tm_k, tm_v;
};

// The merge kernel is launched with programmatic stream serialisation: it may become resident while the attention kernel
// is still running and waits (griddepcontrol.wait) for that grid to complete.
template <int D>
mv_status launch_merge(const mv_plan* P, const mv_attn_geom* g, void* ws, void* out, cudaStream_t st) {
  const int G = g->n_q_heads / g->n_kv_heads;
  const size_t vecs = size_t(P->stats.n_partials) * size_t(G);
  const size_t o_bytes = (vecs * D * sizeof(float) + 255) & ~size_t(255);
  const int n_rows = int(P->stats.n_new_tokens);
  const int n_warps = n_rows * g->n_q_heads;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(unsigned((n_warps + 3) / 4), 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, decode_merge_kernel<D>, static_cast<const float*>(ws),
                                           reinterpret_cast<const float*>(static_cast<char*>(ws) + o_bytes),
                                           mv::table<int32_t>(P, P->layout.rowkv_part_off), static_cast<bf16*>(out), n_rows, int(g->n_q_heads), G);
  mv::g_launches++;
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  return MV_OK;
}

template <int D>
mv_status launch(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, void* out,
                 void* ws, cudaStream_t st) {
  static std::atomic<uint64_t> opted_in{0};  // per device
  if (!mv::opt_in_smem(decode_attn_kernel<D>, Cfg<D>::SMEM, opted_in)) return MV_ERR_CUDA;
  static thread_local mv::KeyedCache<KvMaps, 4> cache;  // the pools rarely change between calls
  const int64_t rows = g->num_pages * g->n_kv_heads * 16 * Cfg<D>::HALVES;  // 128-byte rows of the pool
  const mv::TmapKey key{mv::current_device(), kp, vp, nullptr, rows, D};
  KvMaps* hit = cache.find(key);
  if (!hit) {
    hit = cache.claim(key);
    if (!mv::make_tmap_bf16_2d(&hit->tm_k, kp, uint64_t(rows), 64, 16 * Cfg<D>::HALVES) ||
        !mv::make_tmap_bf16_2d(&hit->tm_v, vp, uint64_t(rows), 64, 16 * Cfg<D>::HALVES)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  const int G = g->n_q_heads / g->n_kv_heads;
  const size_t vecs = size_t(P->stats.n_partials) * size_t(G);
  const size_t o_bytes = (vecs * D * sizeof(float) + 255) & ~size_t(255);
  DecodeArgs a;
  a.q = static_cast<const bf16*>(q);
  a.stages = mv::table<mv::StageDesc>(P, P->layout.stages);
  a.units = mv::table<mv::WorkUnit>(P, P->layout.units);
  a.cta_unit_off = mv::table<int32_t>(P, P->layout.cta_unit_off);
  a.cta_head = mv::table<mv::WorkUnit>(P, P->layout.cta_head);
  a.item_rows = mv::table<mv::ItemRow>(P, P->layout.item_rows);
  a.part_o = static_cast<float*>(ws);
  a.part_ml = reinterpret_cast<float*>(static_cast<char*>(ws) + o_bytes);
  a.status = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2;
  a.Hq = g->n_q_heads;
  a.G = G;
  a.scale_log2 = mv::softmax_scale(g) * 1.4426950408889634f;
  a.Hkv = g->n_kv_heads;
  // head_dim 128 runs on the tcgen05 kernel: the tensor core reads a stage's K / V tile once for all q-vectors and the
  // products leave the warps' instruction streams (measured faster at every unit size: 54 vs 57 us at 16 q-vectors,
  // 733 vs 881 us on the serving mix at up to 64); head_dim 64 keeps the mma.sync kernel of this file
  if (D == 128) {
    const mv_status ts = mv::decode_tc(P, g, q, kp, vp, ws, st);
    if (ts != MV_OK) return ts;
  } else {
    decode_attn_kernel<D><<<unsigned(P->stats.n_ctas), NTHREADS, Cfg<D>::SMEM, st>>>(a, hit->tm_k, hit->tm_v);
    mv::g_launches++;
    if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  }
  return launch_merge<D>(P, g, ws, out, st);
}

}  // namespace

extern "C" mv_status mv_dag_decode_attn(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_pages,
                                        const void* v_pages, void* out, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream) {
  mv::NvtxRange nvtx_range("mv_dag_decode_attn");
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (P->stats.n_new_tokens == 0) return MV_OK;
  if (g->dtype != MV_BF16 || !P->stats.decode_ready) return MV_ERR_UNSUPPORTED;
  if (!q_rot || !k_pages || !v_pages || !out) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  // the work units were cut for one KV head count and one group size
  if (g->n_kv_heads != P->stats.sched_kv_heads || g->n_q_heads / g->n_kv_heads != P->stats.sched_group) return MV_ERR_UNSUPPORTED;
  if (P->stats.max_item_rows * P->stats.sched_group > MAXQV) return MV_ERR_UNSUPPORTED;
  if (P->stats.max_page_id >= g->num_pages) return MV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_pages) & 15) || (reinterpret_cast<uintptr_t>(v_pages) & 15)) return MV_ERR_INVALID_ARG;
  const size_t need = mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // Node append with long runs of new tokens: 128-row query tiles over the paged cache read a node's history once per
  // 128 rows, where the decode kernels' row groups read it once per 64 / group_size rows.
  if (P->stats.append_tiles > 0 && P->stats.max_node_new >= mv::kAppendTileTokens && g->head_dim == 128 &&
      (g->n_q_heads / g->n_kv_heads) % 2 == 0 && (reinterpret_cast<uintptr_t>(q_rot) & 15) == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0)
    return mv::append_tc(P, g, q_rot, k_pages, v_pages, out, s);
  return g->head_dim == 128 ? launch<128>(P, g, q_rot, k_pages, v_pages, out, workspace, s)
                            : launch<64>(P, g, q_rot, k_pages, v_pages, out, workspace, s);
}

// ---- decode attention over an FP8 KV cache -----------------------------------------------------------------------
extern "C" mv_status mv_dag_decode_attn_fp8(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_pages8,
                                            const void* v_pages8, const float* kv_scale, void* out, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream) {
  mv::NvtxRange nvtx_range("mv_dag_decode_attn_fp8");
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (P->stats.n_new_tokens == 0) return MV_OK;
  if (g->dtype != MV_BF16 || g->head_dim != 128 || !P->stats.decode_ready) return MV_ERR_UNSUPPORTED;
  if (P->stats.max_node_new > 1) return MV_ERR_UNSUPPORTED;  // single-token steps only: node append keeps the bf16 cache
  if (!q_rot || !k_pages8 || !v_pages8 || !kv_scale || !out) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  if (g->n_kv_heads != P->stats.sched_kv_heads || g->n_q_heads / g->n_kv_heads != P->stats.sched_group) return MV_ERR_UNSUPPORTED;
  if (P->stats.max_item_rows * P->stats.sched_group > MAXQV) return MV_ERR_UNSUPPORTED;
  if (P->stats.max_page_id >= g->num_pages) return MV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_pages8) & 15) || (reinterpret_cast<uintptr_t>(v_pages8) & 15) || (reinterpret_cast<uintptr_t>(q_rot) & 15))
    return MV_ERR_INVALID_ARG;
  const size_t need = mv_workspace_bytes(P, g, MV_OP_DECODE_ATTN);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MV_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  st = mv::decode_fp8(P, g, q_rot, k_pages8, v_pages8, kv_scale, workspace, s);
  if (st != MV_OK) return st;
  return launch_merge<128>(P, g, workspace, out, s);
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
