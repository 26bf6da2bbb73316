// Multi-branch decode attention on the 5th-generation tensor cores (head_dim 128): the same work lists, stage
// streams, partials and merge as decode_attn.cu, with the two products of a stage issued as tcgen05.mma and the
// online softmax done one thread per q-vector on scores held in tensor memory.
//
// Why a second kernel: with mma.sync every consumer warp re-reads the whole K / V tile of a stage from shared
// memory for its own 16 q-vectors, so at 64 q-vectors per unit (8 sibling rows x a GQA group of 8) shared-memory
// bandwidth and the legacy tensor pipe, not HBM, set the pace.  Here the tensor core reads each K / V tile once
// for all q-vectors, and the products leave the warps' instruction streams altogether.
//
// A CTA (one per SM, 384 threads) is two independent halves, each working through one share of the step
// (shares 2c and 2c+1): a producer warp (TMA boxes of one (page, head, column block) each, q-vectors and slot ids
// staged through shared memory one unit ahead), an issuer warp (one thread: S = Q K^T for stage s+1 is issued
// before it waits for the softmax of stage s, O += P V with P read from tensor memory) and a softmax group of
// four warps (thread r = q-vector r: page-granular DAG mask, online softmax in log2 units with lazy rescaling
// of O, P written back over S as packed bf16, at the unit's end the partial (max, sum, O) goes to the workspace).
// Every wait is bounded.  Once one has run out (or another role's has), a role issues nothing further: it leaves its
// loops, the producer waits for the copies it still has in flight, the issuer for its products, and the CTA meets at
// the final barrier, frees its tensor memory and returns with MV_ERR_TIMEOUT in the plan's status word.
// The q tile is 64 rows; the tensor core works on 128, the upper 64 being whatever follows in shared memory:
// rows are independent, and those results are never read.
#include "common.cuh"
#include "tmap_cache.h"
#include "umma.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int D = 128;
constexpr int ST = 64;       // tokens per stage (4 pages)
constexpr int NSTAGES = 3;   // per half
constexpr int MAXQV = 64;
constexpr int NTHREADS = 384;
constexpr int KV_BYTES = ST * D * 2;         // 16 KB: [2 column blocks][64 tokens][128 B]
constexpr int STAGE_BYTES = 2 * KV_BYTES;    // K then V
constexpr int Q_BYTES = MAXQV * D * 2;       // 16 KB: [2 column blocks][64 rows][128 B]
constexpr int OFF_Q = 0;                     // Q of half 0, Q of half 1
constexpr int OFF_STAGES = 2 * Q_BYTES;      // 3 stages of half 0, then 3 of half 1
constexpr int OFF_META = OFF_STAGES + 2 * NSTAGES * STAGE_BYTES;
constexpr int META_BYTES = 640;
constexpr int SMEM_BYTES = OFF_META + 2 * META_BYTES + 64;
constexpr float RESCALE_THRESHOLD = 8.f;

struct Meta {  // one per half
  int32_t pv[MAXQV];            // partial vector index of q-vector x (partial * G + head in group) or -1
  int32_t n_stages, n_qv;       // header of the unit whose q tile is staged
  uint32_t st_tokens[NSTAGES];  // per stage buffer: valid tokens of the four page slots, a byte each
  uint32_t st_pages[NSTAGES];   // per stage buffer: page slots in use
  uint2 st_mask[NSTAGES][4];    // per stage buffer and page slot: rows that see the slot's node (lo, hi)
  uint64_t full[NSTAGES], empty[NSTAGES], q_full, q_empty, s_full[2], p_full[2], o_done, o_free;
  uint64_t drained;             // issuer, after a wait ran out: its products in flight have completed
  int abort;
};
static_assert(sizeof(Meta) <= META_BYTES, "meta area");

struct TcArgs {
  const bf16* q;
  const mv::StageDesc* stages;
  const mv::WorkUnit* units;
  const mv::WorkUnit* cta_head;  // per share: its first unit, unit range in pad[0], pad[1]
  const mv::ItemRow* item_rows;
  float* part_o;
  float* part_ml;
  int32_t* status;
  int Hq, Hkv, G;
  float scale_log2;
  int n_rows;      // rows of q and out, partial vectors of the workspace: read only by the bounds checks of a debug build
  int64_t n_vecs;  // (compile with -DMV_DEBUG: an index out of range sets the status word and the access is skipped)
};

struct Half {  // what every role of one half needs
  uint32_t smem_base;    // shared-memory address of the CTA's dynamic shared memory
  unsigned char* smem;   // generic pointer to it
  uint32_t q_smem, stage_smem;  // this half's q tile and first stage
  Meta* meta;
  uint32_t tmem;         // this half's 256 tensor-memory columns: S buffers at +0 and +64, O at +128
  int lane0;             // tensor-memory lane (= row of the 128-row products) of the half's q-vector 0
  int share;             // index of the share this half works through
  int32_t* status;
};

__device__ __forceinline__ uint32_t bar(const void* p) { return mv::smem_u32(p); }

// Bounded wait.  False once a wait of this half has run out (this one or an earlier one, of any role): the caller then
// issues nothing further and leaves its loops.
__device__ __forceinline__ bool wait_or_flag(const Half& h, uint32_t b, uint32_t parity) {
  volatile int* abort = &h.meta->abort;
  if (*abort) return false;
  if (!mv::mbar_wait_bounded(b, parity, 2000000000ull, abort)) {
    if (!*abort) atomicExch(h.status, int(MV_ERR_TIMEOUT));
    *abort = 1;
    return false;
  }
  return true;
}
// The same for a whole warp whose lanes must stay together (the tensor-memory loads and stores are warp-wide).
__device__ __forceinline__ bool warp_wait(const Half& h, uint32_t b, uint32_t parity) {
  return __all_sync(0xffffffffu, wait_or_flag(h, b, parity));
}

struct UnitRegs {
  int stage_begin = 0, n_stages = 0, row_begin = 0, n_rows = 0, kvh = 0;
};
struct StageRegs {
  int4 a = make_int4(0, 0, 0, 0), b = make_int4(0, 0, 0, 0), c = make_int4(0, 0, 0, 0), d = make_int4(0, 0, 0, 0);
};

// ---- producer warp of one half ---------------------------------------------------------------------------
__device__ __forceinline__ void producer(const TcArgs& a, const Half& h, const CUtensorMap* tm_k, const CUtensorMap* tm_v) {
  const int lane = threadIdx.x & 31;
  Meta* meta = h.meta;
  UnitRegs wu;
  int u_begin, u_end;
  {
    const int4* p = reinterpret_cast<const int4*>(a.cta_head + h.share);
    const int4 x = __ldg(p), y = __ldg(p + 1);
    wu.stage_begin = x.x; wu.n_stages = x.y; wu.row_begin = x.z; wu.n_rows = x.w; wu.kvh = y.x;
    u_begin = y.y;
    u_end = y.z;
  }
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
  auto load_window = [&](const UnitRegs& w, int first) {
    StageRegs r;
    if (first + lane < w.n_stages) {
      const int4* p = reinterpret_cast<const int4*>(a.stages + w.stage_begin + first + lane);
      r.a = __ldg(p); r.b = __ldg(p + 1); r.c = __ldg(p + 2); r.d = __ldg(p + 3);
    }
    return r;
  };
  int issued = 0;
  bool ok = true;  // warp-uniform: no wait of this half has run out
  const uint64_t kv_policy = mv::l2_policy_evict_first();  // the KV stream is read once per call
  UnitRegs wu1 = load_unit(u_begin + 1);
  mv::ItemRow ir0 = load_rows(wu, 0), ir1 = load_rows(wu, 32);
  StageRegs win = load_window(wu, 0);
  for (int u = u_begin; u < u_end && ok; ++u) {
    const int ui = u - u_begin;
    const UnitRegs wu2 = load_unit(u + 2);
    const mv::ItemRow nir0 = load_rows(wu1, 0), nir1 = load_rows(wu1, 32);
    const StageRegs nwin = load_window(wu1, 0);
    // ---- KV stages, 32 descriptors per window (called with s = 0, 1, 2, ... in order); false: a wait ran out, nothing issued
    StageRegs nxt;
    auto issue_stage = [&](int s) -> bool {
      if ((s & 31) == 0) {
        if (s > 0) win = nxt;
        nxt = load_window(wu, s + 32);
      }
      const int src = s & 31;
      const int4 da = make_int4(__shfl_sync(0xffffffffu, win.a.x, src), __shfl_sync(0xffffffffu, win.a.y, src),
                                __shfl_sync(0xffffffffu, win.a.z, src), __shfl_sync(0xffffffffu, win.a.w, src));
      const int n_pages = __shfl_sync(0xffffffffu, win.b.y, src);
      const int b = issued % NSTAGES;
      const uint32_t fb = bar(&meta->full[b]);
      int go = 1;
      if (lane == 0) go = wait_or_flag(h, bar(&meta->empty[b]), ((issued / NSTAGES) & 1) ^ 1) ? 1 : 0;
      if (!__shfl_sync(0xffffffffu, go, 0)) return false;
      if (lane == src) {
        meta->st_tokens[b] = uint32_t(win.b.x);
        meta->st_pages[b] = uint32_t(win.b.y);
        meta->st_mask[b][0] = make_uint2(uint32_t(win.b.z), uint32_t(win.c.z));
        meta->st_mask[b][1] = make_uint2(uint32_t(win.b.w), uint32_t(win.c.w));
        meta->st_mask[b][2] = make_uint2(uint32_t(win.c.x), uint32_t(win.d.x));
        meta->st_mask[b][3] = make_uint2(uint32_t(win.c.y), uint32_t(win.d.y));
      }
      __syncwarp();
      if (lane == 0) mv::mbar_arrive_expect_tx(fb, uint32_t(n_pages) * 16 * D * 2 * 2);
      __syncwarp();
      // lane j < 16: page slot j / 4, K or V, column block: one 2 KB box = 16 tokens x 64 elements, contiguous
      const int p = (lane >> 2) & 3, kv = (lane >> 1) & 1, cb = lane & 1;
      const int page = p == 0 ? da.x : p == 1 ? da.y : p == 2 ? da.z : da.w;
      if (lane < 16 && p < n_pages) {
        const int row = ((page * a.Hkv + wu.kvh) * 2 + cb) * 16;
        const uint32_t dst = h.stage_smem + b * STAGE_BYTES + kv * KV_BYTES + cb * (KV_BYTES / 2) + p * 2048;
        mv::tma_load_2d_hint(dst, kv ? tm_v : tm_k, 0, row, fb, kv_policy);
      }
      ++issued;
      return true;
    };
    // Between units the first stages go out before the q tile is staged: they do not depend on it, and this keeps the ring
    // full while the producer waits for the previous unit to let go of the q tile (each stage still waits for its own
    // buffer to come free).  At the start of the share the q tile goes first: every half of the grid asks for its first
    // three stages at once (28 MB), and a q tile requested behind that burst arrives after it (measured: q ready 5.7 us
    // after kernel entry, first stage long there), while the few KB of q requested first cost the stages nothing.
    int s_next = 0;
    if (ui != 0)
      for (const int pre = min(wu.n_stages, NSTAGES); s_next < pre && ok; ++s_next) ok = issue_stage(s_next);
    if (!ok) break;
    // ---- q-vectors (K-major tile, 128-byte swizzle: what the tensor core expects) and partial-slot ids
    const int n_qv = wu.n_rows * a.G;
    {
      int go = 1;
      if (lane == 0) go = wait_or_flag(h, bar(&meta->q_empty), (ui & 1) ^ 1) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, go, 0) != 0;
    }
    if (!ok) break;
    for (int x = lane; x < MAXQV; x += 32) {
      const int r = min(x / a.G, MAXQV - 1);
      const int p_lo = __shfl_sync(0xffffffffu, ir0.part, r & 31), p_hi = __shfl_sync(0xffffffffu, ir1.part, r & 31);
      const int part = r < 32 ? p_lo : p_hi;
      meta->pv[x] = (x < n_qv && part >= 0) ? part * a.G + x % a.G : -1;
    }
    if (lane == 0) {
      meta->n_stages = wu.n_stages;
      meta->n_qv = n_qv;
    }
    // rows past n_qv are left as they are: the tensor core computes on them, nobody reads those results
    for (int i0 = 0; i0 < ((n_qv + 1) & ~1) * 16; i0 += 32) {
      const int i = i0 + lane;
      const int x = i >> 4, c = i & 15;
      const int r = min(x / a.G, MAXQV - 1);
      const int r_lo = __shfl_sync(0xffffffffu, ir0.row, r & 31), r_hi = __shfl_sync(0xffffffffu, ir1.row, r & 31);
      const int row = r < 32 ? r_lo : r_hi;
      bool okq = x < n_qv;
#ifdef MV_DEBUG
      if (okq && (row < 0 || row >= a.n_rows)) {
        atomicExch(h.status, int(MV_ERR_INVALID_ARG));
        okq = false;
      }
#endif
      const bf16* src = a.q + (okq ? (int64_t(row) * a.Hq + wu.kvh * a.G + x % a.G) * D + c * 8 : 0);
      const uint32_t dst = h.q_smem + (c >> 3) * (Q_BYTES / 2) + x * 128 + (((c & 7) ^ (x & 7)) << 4);
      mv::cp_async_16(dst, src, okq ? 16 : 0);
    }
    mv::cp_async_mbar_arrive_noinc(bar(&meta->q_full));
    __syncwarp();
    if (lane == 0) {
      mv::fence_proxy_async();  // the copies above are read by the tensor core (async proxy)
      mv::mbar_arrive(bar(&meta->q_full));
    }
    for (; s_next < wu.n_stages && ok; ++s_next) ok = issue_stage(s_next);
    wu = wu1; wu1 = wu2; ir0 = nir0; ir1 = nir1; win = nwin;
  }
  if (!ok) {
    // a wait ran out: nothing more is issued; what is still in flight must land before the CTA may return, since a
    // bulk copy that completes into the shared memory of a CTA that has left corrupts whoever runs there next
    mv::cp_async_wait_all();
    if (lane == 0)
      for (int k = 1; k <= min(issued, NSTAGES); ++k) {
        const int e = issued - k;  // the last fills of the ring
        (void)mv::mbar_wait_bounded(bar(&meta->full[e % NSTAGES]), (e / NSTAGES) & 1, 20000000ull);
      }
    __syncwarp();
  }
}

// ---- issuer warp of one half (one thread) ----------------------------------------------------------------
__device__ __forceinline__ void issuer(const TcArgs& a, const Half& h) {
  // The whole warp walks the units and waits on the barriers; one elected lane issues the products and the commits, so
  // that descriptors and tensor-memory addresses are computed in warp-uniform code.
  const bool lead = mv::um::elect_one();
  Meta* meta = h.meta;
  int u_begin, u_end;
  {
    const int4 y = __ldg(reinterpret_cast<const int4*>(a.cta_head + h.share) + 1);
    u_begin = y.y;
    u_end = y.z;
  }
  // the q tile holds 64 rows per column block: rows lane0 .. lane0 + 63 of the 128-row operand; the tensor core reads
  // the neighbouring 8 KB of shared memory as the other 64 rows, and nobody reads what it computes from them
  const uint64_t q_desc = mv::um::smem_desc(h.q_smem - uint32_t(h.lane0) * 128u, 16, 1024);
  constexpr uint32_t idesc_qk = mv::um::idesc_bf16(128, ST, 0, 0), idesc_pv = mv::um::idesc_bf16(128, D, 0, 1);
  int g = 0;  // stages consumed so far (ring position)
  int t = 0;  // stages whose scores were issued so far (S buffer = t & 1)
  bool ok = true;  // false once a wait of this half ran out: nothing more is issued (a lane that saw the barrier complete
                   // at the last moment may run on alone for a step; it issues nothing the others would not have)
  auto scores = [&](int stage_g) {  // S = Q K^T of ring entry stage_g into buffer t & 1
    const int sb = stage_g % NSTAGES;
    ok = ok && wait_or_flag(h, bar(&meta->full[sb]), (stage_g / NSTAGES) & 1);
    if (!ok) return;
    mv::um::fence_after();
    const uint64_t k_desc = mv::um::smem_desc(h.stage_smem + sb * STAGE_BYTES, 16, 1024);
    const uint32_t s_t = h.tmem + (t & 1) * 64;
    if (lead) {
      mv::um::mma_ss<false>(s_t, q_desc, k_desc, idesc_qk);
#pragma unroll
      for (int k = 1; k < D / 16; ++k) {
        const uint32_t qo = ((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4, ko = ((k >> 2) * (KV_BYTES / 2) + (k & 3) * 32) >> 4;
        mv::um::mma_ss<true>(s_t, q_desc + qo, k_desc + ko, idesc_qk);
      }
      mv::um::commit(bar(&meta->s_full[t & 1]));
    }
    ++t;
  };
  for (int u = u_begin; u < u_end && ok; ++u) {
    const int ui = u - u_begin;
    ok = wait_or_flag(h, bar(&meta->q_full), ui & 1);
    if (!ok) break;
    mv::fence_proxy_async();  // the q tile was written with ordinary asynchronous copies; the tensor core reads it
    const int n = meta->n_stages;
    const int t0 = t;  // stage s of this unit is score tile t0 + s: S / P buffer (t0 + s) & 1
    scores(g);
    if (!ok) break;
    if (n == 1 && lead) mv::um::commit(bar(&meta->q_empty));  // the unit's last scores are queued: q tile free once they ran
    for (int s = 0; s < n; ++s) {
      if (s + 1 < n) {
        scores(g + 1);
        if (!ok) break;
        if (s + 2 == n && lead) mv::um::commit(bar(&meta->q_empty));
      }
      if (s == 0 && ui > 0) ok = wait_or_flag(h, bar(&meta->o_free), (ui - 1) & 1);  // the previous unit's O has been read
      const int sb = g % NSTAGES, T = t0 + s, pb = T & 1;
      const uint32_t n_pages = meta->st_pages[sb];
      ok = ok && wait_or_flag(h, bar(&meta->p_full[pb]), (T >> 1) & 1);
      if (!ok) break;
      mv::um::fence_after();
      const uint64_t v_desc = mv::um::smem_desc(h.stage_smem + sb * STAGE_BYTES + KV_BYTES, KV_BYTES / 2, 1024);
      const uint32_t o_t = h.tmem + 128, p_t = h.tmem + pb * 64;
      if (lead) {
        if (s == 0) mv::um::mma_ts<false>(o_t, p_t, v_desc, idesc_pv);
        else mv::um::mma_ts<true>(o_t, p_t, v_desc, idesc_pv);
#pragma unroll
        for (int k = 1; k < ST / 16; ++k)
          if (uint32_t(k) < n_pages) mv::um::mma_ts<true>(o_t, p_t + k * 8, v_desc + uint32_t((k * 2048) >> 4), idesc_pv);
        mv::um::commit(bar(&meta->o_done));
        mv::um::commit(bar(&meta->empty[sb]));
      }
      ++g;
    }
  }
  __syncwarp();
  if (*reinterpret_cast<volatile int*>(&meta->abort)) {
    // products may still be in flight: they must have completed before the CTA frees its tensor memory
    if (lead) mv::um::commit(bar(&meta->drained));
    (void)mv::mbar_wait_bounded(bar(&meta->drained), 0, 20000000ull);
  }
}

// ---- softmax group of one half: the thread on tensor-memory lane lane0 + r owns q-vector r of the unit (r < 64); the
// group's other two warps idle along.  Half 0 keeps its q-vectors on lanes 0..63, half 1 on lanes 64..127, so that the
// two halves' busy warps sit on different quarters of the SM (a warp reaches the 32 lanes of its index modulo 4).
__device__ __forceinline__ void softmax_group(const TcArgs& a, const Half& h) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wb = (warp & 3) * 32 - h.lane0;  // q-vector of the warp's lane 0 (negative or >= 64: an idle warp)
  const int r = wb + lane;
  const int gt = threadIdx.x & 127;      // index inside the group
  Meta* meta = h.meta;
  const uint32_t lane_base = h.tmem + (uint32_t((warp & 3) * 32) << 16);
  const uint32_t o_t = lane_base + 128;
  int u_begin, u_end;
  {
    const int4 y = __ldg(reinterpret_cast<const int4*>(a.cta_head + h.share) + 1);
    u_begin = y.y;
    u_end = y.z;
  }
  int g = 0;  // stages consumed so far (ring position, score tile index and product index all advance together)
  bool ok = true;    // warp-uniform: false once a wait of this half ran out
  for (int u = u_begin; u < u_end && ok; ++u) {
    const int ui = u - u_begin;
    ok = warp_wait(h, bar(&meta->q_full), ui & 1);
    if (!ok) break;
    const int n = meta->n_stages, n_qv = meta->n_qv;
    const int pv = (r >= 0 && r < MAXQV) ? meta->pv[r] : -1;
    mv::mbar_arrive(bar(&meta->q_empty));  // header and slot ids are in registers
    const bool warp_active = wb >= 0 && wb < n_qv;            // some q-vector of this warp is real
    const int row = (r >= 0 && r < n_qv) ? r / a.G : -1;      // row of the unit's row group this q-vector belongs to
    uint64_t warp_rows = 0;                                   // rows that own a real q-vector of this warp
    if (warp_active) {
      const int r_lo = wb / a.G, r_hi = (min(wb + 31, n_qv - 1)) / a.G;
      warp_rows = (r_hi - r_lo == 63 ? ~uint64_t(0) : ((uint64_t(1) << (r_hi - r_lo + 1)) - 1)) << r_lo;
    }
    float m = -INFINITY, l = 0.f;
    for (int s = 0; s < n; ++s, ++g) {
      const int sb = g % NSTAGES, pb = g & 1;
      ok = warp_wait(h, bar(&meta->full[sb]), (g / NSTAGES) & 1);  // the stage's token counts and masks are visible
      if (!ok) break;
      const uint32_t tok4 = meta->st_tokens[sb], n_pages = meta->st_pages[sb];
      ok = warp_wait(h, bar(&meta->s_full[pb]), (g >> 1) & 1);
      if (!ok) break;
      mv::um::fence_after();
      const uint32_t s_t = lane_base + pb * 64;
      uint32_t sc[ST];
      float mx = -INFINITY;
      if (warp_active) {
        mv::um::ld32(s_t, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
        mv::um::ld32(s_t + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
        mv::um::wait_ld();
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        bool plain = tok4 == 0x10101010u;  // four full pages ...
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint2 mk = meta->st_mask[sb][j];
          plain &= (((uint64_t(mk.y) << 32) | mk.x) & warp_rows) == warp_rows;  // ... seen by every real q-vector of the warp
        }
        if (plain) {
#pragma unroll
          for (int c = 0; c < ST; c += 2) mx4[(c >> 1) & 3] = mv::max3(mx4[(c >> 1) & 3], __uint_as_float(sc[c]), __uint_as_float(sc[c + 1]));
          if (row < 0) mx4[0] = mx4[1] = mx4[2] = mx4[3] = -INFINITY;  // a padding q-vector of the warp
        } else {
          // the DAG mask at page granularity and the ragged last page of a node
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint2 mk = meta->st_mask[sb][j];
            const uint64_t seen_by = (uint64_t(mk.y) << 32) | mk.x;
            const bool vis = row >= 0 && j < int(n_pages) && ((seen_by >> row) & 1);
            const int lim = vis ? int((tok4 >> (8 * j)) & 0xffu) : 0;  // tokens [0, lim) of the page are visible to this q-vector
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              if (c >= lim) sc[j * 16 + c] = __float_as_uint(-INFINITY);
              mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(sc[j * 16 + c]));
            }
          }
        }
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
      }
      if (s > 0) {  // O holds stages 0 .. s-1 of the unit once the previous product is done
        ok = warp_wait(h, bar(&meta->o_done), (g - 1) & 1);
        if (!ok) break;
        mv::um::fence_after();
      }
      if (warp_active) {
        // the reference maximum moves only when it would otherwise let P grow past 2^8
        const bool move = mx > m + RESCALE_THRESHOLD || (m == -INFINITY && mx > -INFINITY);
        if (s > 0 && __any_sync(0xffffffffu, move)) {
          const float f = (move && m != -INFINITY) ? mv::fast_exp2(m - mx) : 1.f;
#pragma unroll 1
          for (int c = 0; c < D / 16; ++c) {  // sixteen columns at a time: the scores of the stage are live in registers
            uint32_t o[16];
            mv::um::ld16(o_t + c * 16, o);
            mv::um::wait_ld();
#pragma unroll
            for (int k = 0; k < 16; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * f);
            mv::um::st16(o_t + c * 16, o);
          }
          l *= f;
        }
        if (move) m = mx;
        const float mref = (m == -INFINITY) ? 0.f : m;
        // packed-pair arithmetic: one FMA and one add per two scores
        const uint64_t scale2 = mv::pack_f32x2(a.scale_log2, a.scale_log2), nmref2 = mv::pack_f32x2(-mref, -mref);
        uint64_t sum2[4] = {0, 0, 0, 0};
#pragma unroll
        for (int c = 0; c < ST / 2; ++c) {  // P over S in place: columns 2c, 2c+1 -> packed column c
          float x0, x1;
          mv::unpack_f32x2(mv::fma_f32x2(mv::pack_f32x2(__uint_as_float(sc[2 * c]), __uint_as_float(sc[2 * c + 1])), scale2, nmref2), x0, x1);
          const float p0 = mv::fast_exp2(x0), p1 = mv::fast_exp2(x1);
          sum2[c & 3] = mv::add_f32x2(sum2[c & 3], mv::pack_f32x2(p0, p1));
          sc[c] = mv::pack_bf16(p0, p1);
        }
        {
          float e, o;
          mv::unpack_f32x2(mv::add_f32x2(mv::add_f32x2(sum2[0], sum2[1]), mv::add_f32x2(sum2[2], sum2[3])), e, o);
          l += e + o;
        }
        mv::um::st32(s_t, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
        mv::um::wait_st();
      }
      // a page that is not full: its rows past the last token hold whatever the pool (or an older stage) left
      // there; V must be zero where P is zero, or 0 * NaN would poison O.  All 128 threads patch together.
      if (tok4 != 0x10101010u) {
        unsigned char* vt = h.smem + (h.stage_smem - h.smem_base) + sb * STAGE_BYTES + KV_BYTES;
        for (int j = 0; j < int(n_pages); ++j) {
          const int nt = int((tok4 >> (8 * j)) & 0xffu);
          for (int i = gt; i < (16 - nt) * 16; i += 128) {  // 16-byte pieces: row (j * 16 + nt + i / 16), column block i / 8 % 2
            const int rr = j * 16 + nt + (i >> 4), c = i & 15;
            *reinterpret_cast<uint4*>(vt + (c >> 3) * (KV_BYTES / 2) + rr * 128 + ((c & 7) << 4)) = make_uint4(0, 0, 0, 0);
          }
        }
        mv::fence_proxy_async();  // ordinary stores, read next by the tensor core
      }
      mv::um::fence_before();
      mv::mbar_arrive(bar(&meta->p_full[pb]));
    }
    if (!ok) break;
    // ---- the unit's result: (max, sum, unnormalised O) of this q-vector
    ok = warp_wait(h, bar(&meta->o_done), (g - 1) & 1);
    if (!ok) break;
    mv::um::fence_after();
#ifdef MV_DEBUG
    if (pv >= a.n_vecs) atomicExch(h.status, int(MV_ERR_INVALID_ARG));
    const int pv_checked = pv < a.n_vecs ? pv : -1;
#define pv pv_checked
#endif
    if (warp_active) {
      float* po = a.part_o + int64_t(pv >= 0 ? pv : 0) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        mv::um::ld32(o_t + c * 32, o);
        mv::um::wait_ld();
        if (pv >= 0) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            *reinterpret_cast<float4*>(po + c * 32 + k * 4) = make_float4(__uint_as_float(o[4 * k]), __uint_as_float(o[4 * k + 1]),
                                                                          __uint_as_float(o[4 * k + 2]), __uint_as_float(o[4 * k + 3]));
        }
      }
      if (pv >= 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(pv) * 2) = make_float2(m, l);
    }
#ifdef MV_DEBUG
#undef pv
#endif
    mv::um::fence_before();
    mv::mbar_arrive(bar(&meta->o_free));  // O may be overwritten by the next unit's first product
  }
}

__global__ void __launch_bounds__(NTHREADS, 1) decode_tc_kernel(const TcArgs a, const __grid_constant__ CUtensorMap tm_k,
                                                                const __grid_constant__ CUtensorMap tm_v, int n_shares) {
  extern __shared__ __align__(1024) unsigned char smem[];
  uint32_t& tmem_slot = *reinterpret_cast<uint32_t*>(smem + OFF_META + 2 * META_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t smem_base = mv::smem_u32(smem);
  if ((smem_base & 1023u) != 0) {  // the swizzle pattern is anchored at 1024-byte boundaries
    if (tid == 0) atomicExch(a.status, int(MV_ERR_UNSUPPORTED));
    return;
  }
  if (tid < 2) {
    Meta* meta = reinterpret_cast<Meta*>(smem + OFF_META + tid * META_BYTES);
    meta->abort = 0;
    for (int i = 0; i < NSTAGES; ++i) {
      mv::mbar_init(bar(&meta->full[i]), 1);   // the producer's arrive (+ the bytes TMA reports)
      mv::mbar_init(bar(&meta->empty[i]), 1);  // one tcgen05.commit after the stage's second product
    }
    mv::mbar_init(bar(&meta->q_full), 33);     // 32 copy-completion arrivals + the producer's releasing arrive
    mv::mbar_init(bar(&meta->q_empty), 129);   // the softmax group + one tcgen05.commit after the unit's last scores
    for (int i = 0; i < 2; ++i) {
      mv::mbar_init(bar(&meta->s_full[i]), 1);    // one tcgen05.commit
      mv::mbar_init(bar(&meta->p_full[i]), 128);  // the softmax group
    }
    mv::mbar_init(bar(&meta->o_done), 1);    // one tcgen05.commit
    mv::mbar_init(bar(&meta->o_free), 128);  // the softmax group
    mv::mbar_init(bar(&meta->drained), 1);   // one tcgen05.commit
    mv::mbar_fence_init();
    mv::fence_proxy_async();
  }
  if (warp == 0) {  // the SM's whole tensor memory: 256 columns per half
    mv::um::tmem_alloc(mv::smem_u32(&tmem_slot), 512);
    mv::um::tmem_relinquish();
  }
  mv::um::fence_before();
  __syncthreads();
  mv::um::fence_after();
  // launched with programmatic stream serialisation: everything above may overlap the tail of the kernel before (the
  // RoPE + cache write of the step); nothing of q or of the pools is read before that grid has completed
  mv::grid_dependency_wait();
  const int hi = warp < 4 ? (warp >> 1) : ((warp - 4) >> 2);  // which half this warp serves
  Half h;
  h.smem_base = smem_base;
  h.smem = smem;
  h.q_smem = smem_base + OFF_Q + hi * Q_BYTES;
  h.stage_smem = smem_base + OFF_STAGES + hi * NSTAGES * STAGE_BYTES;
  h.meta = reinterpret_cast<Meta*>(smem + OFF_META + hi * META_BYTES);
  h.tmem = tmem_slot + hi * 256;
  h.lane0 = hi * 64;
  h.share = blockIdx.x * 2 + hi;
  h.status = a.status;
  if (h.share < n_shares) {
    if (warp < 4) {
      if ((warp & 1) == 0) producer(a, h, &tm_k, &tm_v);
      else issuer(a, h);
    } else {
      softmax_group(a, h);
    }
  }
  mv::um::fence_before();
  __syncthreads();
  if (warp == 0) mv::um::tmem_dealloc(tmem_slot, 512);
}

struct TcMaps {
  CUtensorMap tm_k, tm_v;
};

}  // namespace

namespace mv {
// Attention kernel of mv_dag_decode_attn for head_dim 128 (the caller validated the arguments and launches the
// merge kernel afterwards).  Partials land in `ws` exactly as the mma.sync kernel leaves them.
mv_status decode_tc(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, void* ws,
                    cudaStream_t st) {
  static std::atomic<uint64_t> opted_in{0};  // per device
  if (!mv::opt_in_smem(decode_tc_kernel, SMEM_BYTES, opted_in)) return MV_ERR_CUDA;
  static thread_local mv::KeyedCache<TcMaps, 4> cache;  // the pools rarely change between calls
  const int64_t rows = g->num_pages * g->n_kv_heads * 2 * 16;  // 128-byte rows of a pool
  const mv::TmapKey key{mv::current_device(), kp, vp, nullptr, rows, 0};
  TcMaps* hit = cache.find(key);
  if (!hit) {
    hit = cache.claim(key);
    if (!mv::make_tmap_bf16_2d(&hit->tm_k, kp, uint64_t(rows), 64, 16) || !mv::make_tmap_bf16_2d(&hit->tm_v, vp, uint64_t(rows), 64, 16)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  const int G = g->n_q_heads / g->n_kv_heads;
  const size_t vecs = size_t(P->stats.n_partials) * size_t(G);
  const size_t o_bytes = (vecs * D * sizeof(float) + 255) & ~size_t(255);
  TcArgs a;
  a.q = static_cast<const bf16*>(q);
  a.stages = mv::table<mv::StageDesc>(P, P->layout.stages);
  a.units = mv::table<mv::WorkUnit>(P, P->layout.units);
  a.cta_head = mv::table<mv::WorkUnit>(P, P->layout.cta_head);
  a.item_rows = mv::table<mv::ItemRow>(P, P->layout.item_rows);
  a.part_o = static_cast<float*>(ws);
  a.part_ml = reinterpret_cast<float*>(static_cast<char*>(ws) + o_bytes);
  a.status = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2;
  a.Hq = g->n_q_heads;
  a.Hkv = g->n_kv_heads;
  a.G = G;
  a.scale_log2 = mv::softmax_scale(g) * 1.4426950408889634f;
  a.n_rows = int(P->stats.n_new_tokens);
  a.n_vecs = int64_t(vecs);
  const int n_shares = int(P->stats.n_ctas);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(unsigned((n_shares + 1) / 2), 1, 1);
  cfg.blockDim = dim3(NTHREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, decode_tc_kernel, a, hit->tm_k, hit->tm_v, n_shares);
  mv::g_launches++;
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  return MV_OK;
}
}  // namespace mv
