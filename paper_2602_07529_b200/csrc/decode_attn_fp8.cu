// Multi-branch decode attention over an FP8 KV cache (not in the paper: a storage format that halves the bytes a decode
// step streams).  K (position-embedded) and V sit in the pools as 8-bit floats with 4 exponent and 3 mantissa bits, one
// scale per KV head: value = stored * scale[head].  The kernel is the tcgen05 decode kernel (same work lists, stage
// streams, roles, partials and merge kernel) with both products issued as 8-bit-float tensor-core instructions straight
// on the pool bytes:
//   - a (page, KV head) block is 16 tokens x 128 bytes = 2 KB, one TMA box; a 64-token stage is 8 KB of K and 8 KB of V,
//     so the ring is six stages deep in the shared memory the bf16 kernel needs for three;
//   - the q-vectors of a unit are quantised by the producer warp (one scale per q-vector: its largest magnitude / 448)
//     into TWO K-major tiles of 128-byte rows: the rounded value and the rounded remainder (same scale), so that the
//     queries keep about seven bits of mantissa; S = Q_hi K^T + Q_lo K^T accumulates in tensor memory on the stored bytes;
//   - the softmax thread multiplies a score by (q-vector scale * K scale * softmax scale * log2 e); P goes back to tensor
//     memory as two 8-bit-float tiles as well (value and remainder, four per column);
//   - O += P_hi V + P_lo V reads V as an MN-major operand (32 tokens per instruction); the V scale multiplies the partial
//     once.
// What is left against the oracle (which quantises the cache with the same rule) is then of the size of the bf16 kernel's
// own rounding; the tensor pipe has the room (the kernel is bound by the HBM stream).
// Every wait is bounded, as in the bf16 kernel.
#include "common.cuh"
#include "tmap_cache.h"
#include "umma.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int D = 128;
constexpr int ST = 64;       // tokens per stage (4 pages)
constexpr int NSTAGES = 6;   // per half
constexpr int MAXQV = 64;
constexpr int NTHREADS = 384;
constexpr int KV_BYTES = ST * D;             // 8 KB: [64 tokens][128 B]
constexpr int STAGE_BYTES = 2 * KV_BYTES;    // K then V
constexpr int Q_BYTES = MAXQV * D;           // 8 KB: [64 rows][128 B]
constexpr int OFF_Q = 0;                     // Q of half 0, Q of half 1
constexpr int OFF_STAGES = 4 * Q_BYTES;      // per half: Q_hi, Q_lo; then the stages of half 0, then those of half 1
constexpr int OFF_META = OFF_STAGES + 2 * NSTAGES * STAGE_BYTES;
constexpr int META_BYTES = 1024;
constexpr int SMEM_BYTES = OFF_META + 2 * META_BYTES + 64;
constexpr float RESCALE_THRESHOLD = 8.f;

struct Meta {  // one per half
  int32_t pv[MAXQV];            // partial vector index of q-vector x (partial * G + head in group) or -1
  float qscale[MAXQV];          // scale of q-vector x: q = stored * qscale
  int32_t n_stages, n_qv, kvh;  // header of the unit whose q tile is staged
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
  const float* kv_scale;  // [2 * Hkv]: K scales, then V scales
  const mv::StageDesc* stages;
  const mv::WorkUnit* units;
  const mv::WorkUnit* cta_head;  // per share: its first unit, unit range in pad[0], pad[1]
  const mv::ItemRow* item_rows;
  float* part_o;
  float* part_ml;
  int32_t* status;
  int Hq, Hkv, G;
  float scale_log2;
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
      if (lane == 0) mv::mbar_arrive_expect_tx(fb, uint32_t(n_pages) * 16 * D * 2);
      __syncwarp();
      // lane j < 8: page slot j / 2, K or V: one 2 KB box = 16 tokens x 128 bytes, contiguous
      const int p = (lane >> 1) & 3, kv = lane & 1;
      const int page = p == 0 ? da.x : p == 1 ? da.y : p == 2 ? da.z : da.w;
      if (lane < 8 && p < n_pages) {
        const int row = (page * a.Hkv + wu.kvh) * 16;
        const uint32_t dst = h.stage_smem + b * STAGE_BYTES + kv * KV_BYTES + p * 2048;
        mv::tma_load_2d_hint(dst, kv ? tm_v : tm_k, 0, row, fb, kv_policy);
      }
      ++issued;
      return true;
    };
    // Between units the first stages go out before the q tile is staged: they do not depend on it, and this keeps the ring
    // full while the producer waits for the previous unit to let go of the q tile (each stage still waits for its own
    // buffer to come free).  At the start of the share the q-vectors go first: every half of the grid asks for its first
    // stages at once, and q-vectors requested behind that burst arrive after it, while the softmax thread, which paces
    // this kernel, cannot start before they are there.
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
      meta->kvh = wu.kvh;
    }
    // Two q-vectors per pass, sixteen lanes each (a lane holds eight elements): the q-vector's largest magnitude fixes
    // its scale, the bytes go to row x of the K-major tile (128-byte rows, 16-byte pieces XOR-swizzled with x % 8).  Rows
    // past n_qv are left as they are: the tensor core computes on them, nobody reads those results.
    constexpr int QB = 4;  // passes whose loads are in flight together
    for (int x0 = 0; x0 < n_qv; x0 += 2 * QB) {
      uint4 raw[QB];
#pragma unroll
      for (int i = 0; i < QB; ++i) {
        const int x = x0 + 2 * i + (lane >> 4), c = lane & 15;
        const int r = min(x / a.G, MAXQV - 1);
        const int r_lo = __shfl_sync(0xffffffffu, ir0.row, r & 31), r_hi = __shfl_sync(0xffffffffu, ir1.row, r & 31);
        const int row = r < 32 ? r_lo : r_hi;
        raw[i] = make_uint4(0, 0, 0, 0);
        // through L2, not the read-only path: the RoPE kernel writes q while this grid is already resident (programmatic
        // stream serialisation), so q is not read-only for this kernel's lifetime
        if (x < n_qv) raw[i] = __ldcg(reinterpret_cast<const uint4*>(a.q + (int64_t(row) * a.Hq + wu.kvh * a.G + x % a.G) * D + c * 8));
      }
#pragma unroll
      for (int i = 0; i < QB; ++i) {
        const int x = x0 + 2 * i + (lane >> 4), c = lane & 15;
        float f[8];
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw[i]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 t = __bfloat1622float2(h2[k]);
          f[2 * k] = t.x;
          f[2 * k + 1] = t.y;
        }
        float amax = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) amax = fmaxf(amax, fabsf(f[k]));
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        const float qs = amax > 0.f ? amax * (1.f / 448.f) : 1.f, inv = 1.f / qs;
        if (x < n_qv && x < MAXQV) {
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float x0 = f[2 * k] * inv, x1 = f[2 * k + 1] * inv;
            hi[k] = mv::pack_e4m3x2(x0, x1);
            const float2 back = mv::unpack_e4m3x2(hi[k]);
            lo[k] = mv::pack_e4m3x2(x0 - back.x, x1 - back.y);
          }
          unsigned char* dst = h.smem + (h.q_smem - h.smem_base) + x * 128 + ((((c >> 1) ^ (x & 7))) << 4) + (c & 1) * 8;
          *reinterpret_cast<uint2*>(dst) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
          *reinterpret_cast<uint2*>(dst + Q_BYTES) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
          if (c == 0) meta->qscale[x] = qs;
        }
      }
    }
    // ordinary stores above, read by the tensor core (async proxy): every lane that wrote fences its own stores, then one
    // lane signals
    mv::fence_proxy_async();
    __syncwarp();
    if (lane == 0) mv::mbar_arrive(bar(&meta->q_full));
    for (; s_next < wu.n_stages && ok; ++s_next) ok = issue_stage(s_next);
    wu = wu1; wu1 = wu2; ir0 = nir0; ir1 = nir1; win = nwin;
  }
  if (!ok) {
    // a wait ran out: nothing more is issued; what is still in flight must land before the CTA may return, since a
    // bulk copy that completes into the shared memory of a CTA that has left corrupts whoever runs there next
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
  const uint64_t q_desc = mv::um::smem_desc(h.q_smem - uint32_t(h.lane0) * 128u, 16, 1024);  // row lane0 of the operand = q-vector 0
  constexpr uint32_t idesc_qk = mv::um::idesc_e4m3(128, ST, 0, 0), idesc_pv = mv::um::idesc_e4m3(128, D, 0, 1);
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
      mv::um::mma8_ss<false>(s_t, q_desc, k_desc, idesc_qk);
#pragma unroll
      for (int k = 1; k < D / 32; ++k) mv::um::mma8_ss<true>(s_t, q_desc + uint32_t((k * 32) >> 4), k_desc + uint32_t((k * 32) >> 4), idesc_qk);
#pragma unroll
      for (int k = 0; k < D / 32; ++k)  // the remainders of the q-vectors
        mv::um::mma8_ss<true>(s_t, q_desc + uint32_t((Q_BYTES + k * 32) >> 4), k_desc + uint32_t((k * 32) >> 4), idesc_qk);
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
      // V as the MN-major operand: 128 contiguous bytes (the whole head vector) per token row, eight-row groups 1024 bytes
      // apart; one instruction takes 32 tokens, i.e. two page slots
      const uint64_t v_desc = mv::um::smem_desc(h.stage_smem + sb * STAGE_BYTES + KV_BYTES, KV_BYTES, 1024);
      const uint32_t o_t = h.tmem + 128, p_t = h.tmem + pb * 64;
      if (lead) {
        if (s == 0) mv::um::mma8_ts<false>(o_t, p_t, v_desc, idesc_pv);
        else mv::um::mma8_ts<true>(o_t, p_t, v_desc, idesc_pv);
        mv::um::mma8_ts<true>(o_t, p_t + 16, v_desc, idesc_pv);  // the remainders of the weights
        if (n_pages > 2) {
          mv::um::mma8_ts<true>(o_t, p_t + 8, v_desc + uint32_t(4096 >> 4), idesc_pv);
          mv::um::mma8_ts<true>(o_t, p_t + 24, v_desc + uint32_t(4096 >> 4), idesc_pv);
        }
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
    const float v_scale = __ldg(a.kv_scale + a.Hkv + meta->kvh);
    // a stored score times this is the score in log2 units
    const float mult = ((r >= 0 && r < n_qv) ? meta->qscale[r] : 0.f) * __ldg(a.kv_scale + meta->kvh) * a.scale_log2;
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
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        mx = mx == -INFINITY ? -INFINITY : mx * mult;  // (a padding q-vector has mult = 0)
      }
      if (warp_active) {
        // the reference maximum moves only when it would otherwise let P grow past 2^8
        const bool move = mx > m + RESCALE_THRESHOLD || (m == -INFINITY && mx > -INFINITY);
        if (s > 0 && __any_sync(0xffffffffu, move)) {
          // O holds stages 0 .. s-1 of the unit once the previous product is done.  Only a warp that rescales waits for it:
          // here the softmax thread, not the stream, paces a stage.  (The previous product cannot be more than one phase
          // behind this wait: the product after it needs this very thread's P.)
          ok = warp_wait(h, bar(&meta->o_done), (g - 1) & 1);
          if (!ok) break;
          mv::um::fence_after();
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
        // P as 8-bit floats, four per column (columns 4c .. 4c+3 -> packed column c): the rounded weights in packed columns
        // 0..15, their rounded remainders in packed columns 16..31
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t rem[ST / 4];
#pragma unroll
        for (int c = 0; c < ST / 4; ++c) {
          const float p0 = mv::fast_exp2(fmaf(__uint_as_float(sc[4 * c]), mult, -mref)), p1 = mv::fast_exp2(fmaf(__uint_as_float(sc[4 * c + 1]), mult, -mref));
          const float p2 = mv::fast_exp2(fmaf(__uint_as_float(sc[4 * c + 2]), mult, -mref)), p3 = mv::fast_exp2(fmaf(__uint_as_float(sc[4 * c + 3]), mult, -mref));
          sum4[0] += p0; sum4[1] += p1; sum4[2] += p2; sum4[3] += p3;
          const uint32_t w01 = mv::pack_e4m3x2(p0, p1), w23 = mv::pack_e4m3x2(p2, p3);
          const float2 r01 = mv::unpack_e4m3x2(w01), r23 = mv::unpack_e4m3x2(w23);
          sc[c] = w01 | (w23 << 16);
          rem[c] = mv::pack_e4m3x2(p0 - r01.x, p1 - r01.y) | (mv::pack_e4m3x2(p2 - r23.x, p3 - r23.y) << 16);
        }
        l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        mv::um::st16(s_t, *reinterpret_cast<uint32_t(*)[16]>(&sc[0]));
        mv::um::st16(s_t + 16, rem);
        mv::um::wait_st();
      }
      // a page that is not full: its rows past the last token hold whatever the pool (or an older stage) left there, and
      // an instruction of the second product takes two page slots, the second of which may be absent; V must be zero
      // where P is zero, or 0 * NaN would poison O.  All 128 threads patch together (a row is eight 16-byte pieces).
      if (tok4 != 0x10101010u) {
        unsigned char* vt = h.smem + (h.stage_smem - h.smem_base) + sb * STAGE_BYTES + KV_BYTES;
        const int slots = (int(n_pages) + 1) & ~1;  // page slots the instructions read
        for (int j = 0; j < slots; ++j) {
          const int nt = j < int(n_pages) ? int((tok4 >> (8 * j)) & 0xffu) : 0;
          for (int i = gt; i < (16 - nt) * 8; i += 128)
            *reinterpret_cast<uint4*>(vt + (j * 16 + nt + (i >> 3)) * 128 + ((i & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
        mv::fence_proxy_async();  // ordinary stores, read next by the tensor core
      }
      // The waits on o_done tell phases apart by parity, so a thread may never be two phases behind when it waits.  At
      // the wait above that holds: the scores of this stage were committed after the product two stages back.  At the
      // unit's final wait it would not: a warp that skipped the wait above could get there while the product of the
      // stage before the last was still in flight, take the wait for satisfied, and read O too early.  So on the last
      // stage of a unit that product (issued while this stage's weights were computed) is confirmed here, before the
      // arrival that lets the last one start.
      if (s > 0 && s + 1 == n) {
        ok = warp_wait(h, bar(&meta->o_done), (g - 1) & 1);
        if (!ok) break;
      }
      mv::um::fence_before();
      mv::mbar_arrive(bar(&meta->p_full[pb]));
    }
    if (!ok) break;
    // ---- the unit's result: (max, sum, unnormalised O) of this q-vector
    ok = warp_wait(h, bar(&meta->o_done), (g - 1) & 1);
    if (!ok) break;
    mv::um::fence_after();
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
            *reinterpret_cast<float4*>(po + c * 32 + k * 4) = make_float4(__uint_as_float(o[4 * k]) * v_scale, __uint_as_float(o[4 * k + 1]) * v_scale,
                                                                          __uint_as_float(o[4 * k + 2]) * v_scale, __uint_as_float(o[4 * k + 3]) * v_scale);
        }
      }
      if (pv >= 0) *reinterpret_cast<float2*>(a.part_ml + int64_t(pv) * 2) = make_float2(m, l);
    }
    mv::um::fence_before();
    mv::mbar_arrive(bar(&meta->o_free));  // O may be overwritten by the next unit's first product
  }
}

__global__ void __launch_bounds__(NTHREADS, 1) decode_fp8_kernel(const TcArgs a, const __grid_constant__ CUtensorMap tm_k,
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
    mv::mbar_init(bar(&meta->q_full), 1);      // the producer's releasing arrive
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
  h.q_smem = smem_base + OFF_Q + hi * 2 * Q_BYTES;  // Q_hi, then Q_lo
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
// Attention kernel of mv_dag_decode_attn_fp8 (the caller validated the arguments and launches the merge kernel
// afterwards).  Partials land in `ws` exactly as the other decode kernels leave them.
mv_status decode_fp8(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* kp, const void* vp, const float* kv_scale,
                     void* ws, cudaStream_t st) {
  static std::atomic<uint64_t> opted_in{0};  // per device
  if (!mv::opt_in_smem(decode_fp8_kernel, SMEM_BYTES, opted_in)) return MV_ERR_CUDA;
  static thread_local mv::KeyedCache<TcMaps, 4> cache;  // the pools rarely change between calls
  const int64_t rows = g->num_pages * g->n_kv_heads * 16;  // 128-byte rows of a pool
  const mv::TmapKey key{mv::current_device(), kp, vp, nullptr, rows, 8};
  TcMaps* hit = cache.find(key);
  if (!hit) {
    hit = cache.claim(key);
    if (!mv::make_tmap_u8_2d(&hit->tm_k, kp, uint64_t(rows), 16) || !mv::make_tmap_u8_2d(&hit->tm_v, vp, uint64_t(rows), 16)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  const int G = g->n_q_heads / g->n_kv_heads;
  const size_t vecs = size_t(P->stats.n_partials) * size_t(G);
  const size_t o_bytes = (vecs * D * sizeof(float) + 255) & ~size_t(255);
  TcArgs a;
  a.q = static_cast<const bf16*>(q);
  a.kv_scale = kv_scale;
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
  const cudaError_t e = cudaLaunchKernelEx(&cfg, decode_fp8_kernel, a, hit->tm_k, hit->tm_v, n_shares);
  mv::g_launches++;
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return MV_ERR_CUDA;
  }
  return MV_OK;
}
}  // namespace mv
