// Backward of the topology-masked prefill attention (the attention the model is fine-tuned through, Sec. 5.1: the
// mask of Eq. 3 at the position indices of Sec. 4.2) on the 5th-generation tensor cores: head_dim 128, bf16 in, fp32
// accumulation in tensor memory.
//
// With S = scale * Q K^T + M, P = softmax(S) and O = P V (Eq. 2 - 3), a gradient dO of the output gives
//   dV = P^T dO,  dP = dO V^T,  dS = P o (dP - delta),  delta_i = sum_j P_ij dP_ij = <dO_i, O_i>,
//   dQ = scale * dS K,  dK = scale * dS^T Q,
// a KV head collecting dK and dV from every query head of its group.  P is rebuilt from the scores and the row's
// log-sum-exp that the forward kernel leaves (no second softmax pass).  The kernels:
//   delta_kernel   delta[i][h] = <dO[i][h], O[i][h]>                                   (elementwise, one warp per row-head)
//   bwd_kernel<DQ> one CTA per (query tile, query head): walks the KV tiles the tile's node may see, exactly the
//                  forward's walk: S = Q K^T and dP = dO V^T into tensor memory, the lane threads turn them into dS
//                  (bf16, written back over S), dQ += dS K with K as the MN-major operand.
//   bwd_kernel<DK> one CTA per (key tile, KV head): walks the transposed lists (the runs of queries that see the tile's
//                  node; its own node causally) for every query head of the group: S^T = K Q^T and dP^T = V dO^T (a
//                  lane is a key, a column a query), dS^T written back over S^T, dK += dS^T Q with Q MN-major.
//   bwd_kernel<DV> the same walk: S^T = K Q^T, P^T written back over S^T, dV += P^T dO with dO MN-major.
// Every product is 128 x 128 x 16 per instruction, the shape at which the tensor cores run at their full rate
// (measured: a 128 x 64 x 16 instruction takes three quarters of the time of a 128 x 128 x 16 one).  Tensor memory
// holds two score buffers (three in DV), one dP buffer and the accumulator: while the lane threads work on step e the
// tensor cores run the accumulating product of step e - 1 and the scores of step e + 1.  The lane threads copy their
// part of dP to registers first and hand the dP buffer back at once, which is what lets one dP buffer do.  dK and dV
// come from separate CTAs because two accumulators would leave tensor memory for one score buffer only, and the
// products and the elementwise work would then run in turn.
// Masked pairs get P = 0 by selection, so nothing depends on what the padding rows or columns of a ragged tile hold.
// No atomics: every output element is written by exactly one CTA, and the result is deterministic.
// Every mbarrier wait is bounded; after one ran out a role issues nothing further, the producer and the issuer wait
// for what they have in flight, and the status word of the plan reads MV_ERR_TIMEOUT.
#include "common.cuh"
#include "trace.h"
#include "tmap_cache.h"
#include "umma.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int D = 128;
constexpr int BT = 128;                 // rows of every tile (queries or keys)
constexpr int TILE_BYTES = BT * D * 2;  // 32 KB: [2 column blocks][128 rows][128 B]
constexpr int NTHREADS = 384;           // warp 0 producer, warp 1 issuer of the scores, warp 2 issuer of the accumulating
                                        // products, warp 3 idle, warps 4..11: two threads per tensor-memory lane, each
                                        // taking 64 of a step's 128 columns
constexpr int NLANE_THREADS = 256;
enum Mode { DQ = 0, DK = 1, DV = 2 };
constexpr int NLONG = 3, NSHORT = 2;    // ring slots: tiles needed until the accumulating product / only for the scores
constexpr int OFF_FIXED = 0;            // two tiles that stay for the whole CTA (DQ: Q, dO; DK: K, V; DV: K)
constexpr int OFF_LONG = 2 * TILE_BYTES;                   // DQ: K; DK: Q; DV: dO
constexpr int OFF_SHORT = OFF_LONG + NLONG * TILE_BYTES;   // DQ: V; DK: dO; DV: Q
constexpr int OFF_VEC = OFF_SHORT + NSHORT * TILE_BYTES;   // DK, DV: two slots of -lse[128], -scale * delta[128] of a step's queries
constexpr int OFF_BAR = OFF_VEC + 2 * 2 * BT * 4;
constexpr int N_BARS = 1 + 2 * NLONG + 2 * NSHORT + 3 + 2 + 3 + 3 + 2 + 1;
constexpr int SMEM_BYTES = OFF_BAR + N_BARS * 8 + 16;
static_assert(SMEM_BYTES <= 232448, "over the shared memory of a CTA");
// tensor memory columns
constexpr uint32_t TM_S = 0;      // score buffers at 0, 128 (and 256 in DV)
constexpr uint32_t TM_DP = 256;   // dP (DQ, DK)
constexpr uint32_t TM_ACC = 384;  // dQ / dK / dV accumulator

struct BwdArgs {
  const mv::QTile* q_tiles;    // query tiles and their key ranges (DQ)
  const mv::KvRange* kv_ranges;
  const mv::QTile* k_tiles;    // key tiles and the query ranges that see them (DK, DV)
  const mv::KvRange* q_ranges;
  const float* lse;            // [T][Hq] log2-domain log-sum-exp of the forward
  const float* delta;          // [T][Hq]
  bf16* dq;                    // [T][Hq][D]
  bf16* dk;                    // [T][Hkv][D]
  bf16* dv;
  int32_t* status;
  int Hq, Hkv, G, T;
  float scale_log2, scale;
};

struct Bars {
  // lfull / lempty: NLONG consecutive barriers; sfull / sempty: NSHORT; s_full / p_full / acc_done: one per score buffer
  uint32_t fixed_full, lfull, lempty, sfull, sempty, s_full, dp_full, dp_free, p_full, acc_done, drained, vec_ready;  // drained: two, one per issuer
};

struct Waiter {
  volatile int* abort;
  int32_t* status;
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (mv::mbar_try_wait(bar, parity)) return !*abort;
    if (*abort) return false;
    if (!mv::mbar_wait_bounded(bar, parity, 2000000000ull, abort)) {
      if (!*abort) atomicExch(status, int(MV_ERR_TIMEOUT));
      *abort = 1;
      return false;
    }
    return true;
  }
  __device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) const { return __all_sync(0xffffffffu, wait(bar, parity)); }
  __device__ __forceinline__ bool aborted() const { return *abort != 0; }
};

// The steps of a CTA, in table order.  DQ: the 128-key sub-tiles of the query tile's ranges, a causal range ending
// after the tile's last query.  DK, DV: the 128-query sub-tiles of the key tile's transposed ranges (a causal range
// starts at the tile's first key and is not cut), each taken once per query head of the group.
struct Steps {
  const mv::KvRange* rg;
  int n_ranges, last_causal, heads;
  int ri = 0, pos = 0, end = 0, causal = 0, hg = 0, cur_start = 0, cur_n = 0;
  __device__ Steps(const mv::KvRange* r, int n, int lc, int h) : rg(r), n_ranges(n), last_causal(lc), heads(h), hg(h) {}
  __device__ bool next(int& start, int& n, int& c, int& head_in_group) {
    if (hg + 1 < heads) {
      ++hg;
    } else {
      while (pos >= end) {
        if (ri >= n_ranges) return false;
        const mv::KvRange r = rg[ri++];
        pos = r.kv_start;
        end = r.kv_start + r.kv_len;
        causal = r.causal;
        if (causal) end = min(end, last_causal + 1);
      }
      cur_start = pos;
      cur_n = min(BT, end - pos);
      pos += BT;
      hg = 0;
    }
    start = cur_start;
    n = cur_n;
    c = causal;
    head_in_group = hg;
    return true;
  }
};

// every tensor map's box is 64 columns x 128 rows (16 KB)
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap* tm, int col, int row, uint32_t bar) {
  for (int cb = 0; cb < 2; ++cb) mv::tma_load_2d(dst + cb * (TILE_BYTES / 2), tm, col + cb * 64, row, bar);
}

// D[tmem, 128 x 128] = A B^T with both operands K-major tiles ([128 rows][128 elements of the contraction]): eight k-steps
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t addr) { return mv::um::smem_desc(addr, 16, 1024); }
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t addr) { return mv::um::smem_desc(addr, TILE_BYTES / 2, 1024); }
__device__ __forceinline__ void issue_nt(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc) {
  constexpr uint32_t idesc = mv::um::idesc_bf16(BT, BT, 0, 0);
  mv::um::mma_ss<false>(d_tmem, a_desc, b_desc, idesc);
#pragma unroll
  for (int k = 1; k < D / 16; ++k) {
    const uint32_t off = ((k >> 2) * (TILE_BYTES / 2) + (k & 3) * 32) >> 4;
    mv::um::mma_ss<true>(d_tmem, a_desc + off, b_desc + off, idesc);
  }
}
// D[tmem, 128 x 128] (+)= A[tmem, 128 x 128 as bf16 pairs] B with B an MN-major tile ([128 contraction rows][128
// columns]): eight k-steps.  The lane threads leave A in two pieces, the pairs of a step's columns 0..63 at
// a_tmem + 0..31 and those of columns 64..127 at a_tmem + 64..95.
__device__ __forceinline__ void issue_tn(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, bool accumulate) {
  constexpr uint32_t idesc = mv::um::idesc_bf16(BT, D, 0, 1);
  if (accumulate) mv::um::mma_ts<true>(d_tmem, a_tmem, b_desc, idesc);
  else mv::um::mma_ts<false>(d_tmem, a_tmem, b_desc, idesc);
#pragma unroll
  for (int k = 1; k < BT / 16; ++k)
    mv::um::mma_ts<true>(d_tmem, a_tmem + (k >> 2) * 64 + (k & 3) * 8, b_desc + uint32_t((k * 2048) >> 4), idesc);
}

struct Ctx {
  unsigned char* smem;
  uint32_t smem_base, tmem;
  Bars br;
  Waiter w;
};

__device__ __forceinline__ bool setup(Ctx& c, unsigned char* smem, int32_t* status) {
  const int tid = threadIdx.x, warp = tid >> 5;
  c.smem = smem;
  c.smem_base = mv::smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + N_BARS * 8);
  int* abort_flag = reinterpret_cast<int*>(smem + OFF_BAR + N_BARS * 8 + 8);
  int i = 0;
  c.br.fixed_full = mv::smem_u32(&bars[i]); i += 1;
  c.br.lfull = mv::smem_u32(&bars[i]); i += NLONG;
  c.br.lempty = mv::smem_u32(&bars[i]); i += NLONG;
  c.br.sfull = mv::smem_u32(&bars[i]); i += NSHORT;
  c.br.sempty = mv::smem_u32(&bars[i]); i += NSHORT;
  c.br.s_full = mv::smem_u32(&bars[i]); i += 3;
  c.br.dp_full = mv::smem_u32(&bars[i]); i += 1;
  c.br.dp_free = mv::smem_u32(&bars[i]); i += 1;
  c.br.p_full = mv::smem_u32(&bars[i]); i += 3;
  c.br.acc_done = mv::smem_u32(&bars[i]); i += 3;
  c.br.drained = mv::smem_u32(&bars[i]); i += 2;
  c.br.vec_ready = mv::smem_u32(&bars[i]); i += 1;
  if ((c.smem_base & 1023u) != 0) {  // the swizzle pattern is anchored at 1024-byte boundaries
    if (tid == 0) atomicExch(status, int(MV_ERR_UNSUPPORTED));
    return false;
  }
  if (tid == 0) {
    *abort_flag = 0;
    for (int b = 0; b < N_BARS; ++b) {
      // one tcgen05.commit or one arrive of the producer, except the barriers on which the 256 lane threads arrive
      const uint32_t addr = mv::smem_u32(&bars[b]);
      const bool lanes = addr == c.br.dp_free || addr == c.br.vec_ready || (addr >= c.br.p_full && addr < c.br.p_full + 24);
      mv::mbar_init(addr, lanes ? NLANE_THREADS : 1);
    }
    mv::mbar_fence_init();
    mv::fence_proxy_async();
  }
  if (warp == 1) {
    mv::um::tmem_alloc(mv::smem_u32(tmem_slot), 512);
    mv::um::tmem_relinquish();
  }
  mv::um::fence_before();
  __syncthreads();
  mv::um::fence_after();
  c.tmem = *tmem_slot;
  c.w = Waiter{abort_flag, status};
  return true;
}

__device__ __forceinline__ void teardown(const Ctx& c) {
  mv::um::fence_before();
  __syncthreads();
  if ((threadIdx.x >> 5) == 1) mv::um::tmem_dealloc(c.tmem, 512);
}

// after a wait ran out: the producer's copies in flight must land before the CTA may return
__device__ __forceinline__ void drain_ring(uint32_t full, int nslots, int issued) {
  for (int k = 1; k <= min(issued, nslots); ++k)
    (void)mv::mbar_wait_bounded(full + 8 * ((issued - k) % nslots), ((issued - k) / nslots) & 1, 20000000ull);
}
__device__ __forceinline__ void drain_issuer(uint32_t drained, bool lead) {
  __syncwarp();
  if (lead) mv::um::commit(drained);
  (void)mv::mbar_wait_bounded(drained, 0, 20000000ull);
}

// ---- delta[i][h] = <dO[i][h], O[i][h]> ------------------------------------------------------------------------
__global__ void __launch_bounds__(128) delta_kernel(const bf16* __restrict__ out, const bf16* __restrict__ dout, float* __restrict__ delta,
                                                    int64_t n_row_heads) {
  const int64_t w = int64_t(blockIdx.x) * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= n_row_heads) return;
  const uint2 a = *reinterpret_cast<const uint2*>(out + w * D + lane * 4), b = *reinterpret_cast<const uint2*>(dout + w * D + lane * 4);
  const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.x)), a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a.y));
  const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.x)), b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&b.y));
  float s = a0.x * b0.x + a0.y * b0.y + a1.x * b1.x + a1.y * b1.y;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) delta[w] = s;
}

// ---- the three tensor-core kernels -----------------------------------------------------------------------------
// The lane threads' arithmetic over 32 columns: s (scores, fp32 bits) and dp (dP, fp32 bits) -> packed bf16 pairs.
// The per-pair constants (-lse, -lse) and (-scale * delta, -scale * delta) are the row's in DQ (row_nl2, row_nd2) and
// the columns' in DK and DV, read from shared memory (vs: 32 values of -lse; vs + BT: of -scale * delta) eight
// columns ahead of their use.  Columns outside [lo, hi) are masked; ALL says that none of the warp's 32 is.
template <int MODE>
__device__ __forceinline__ void lane_consts(const float* vs, int col, uint64_t (&nl)[4], uint64_t (&nd)[4], uint64_t row_nl2, uint64_t row_nd2) {
  if (MODE == DQ) {
#pragma unroll
    for (int i = 0; i < 4; ++i) nl[i] = row_nl2, nd[i] = row_nd2;
  } else {
    const float4 l0 = *reinterpret_cast<const float4*>(vs + col), l1 = *reinterpret_cast<const float4*>(vs + col + 4);
    nl[0] = mv::pack_f32x2(l0.x, l0.y), nl[1] = mv::pack_f32x2(l0.z, l0.w), nl[2] = mv::pack_f32x2(l1.x, l1.y), nl[3] = mv::pack_f32x2(l1.z, l1.w);
    if (MODE == DK) {
      const float4 d0 = *reinterpret_cast<const float4*>(vs + BT + col), d1 = *reinterpret_cast<const float4*>(vs + BT + col + 4);
      nd[0] = mv::pack_f32x2(d0.x, d0.y), nd[1] = mv::pack_f32x2(d0.z, d0.w), nd[2] = mv::pack_f32x2(d1.x, d1.y), nd[3] = mv::pack_f32x2(d1.z, d1.w);
    }
  }
}
template <int MODE, bool ALL>
__device__ __forceinline__ void lane_math(const uint32_t (&s)[32], const uint32_t* dp, uint32_t (&o)[16], float scale_log2, float scale,
                                          int j0, int lo, int hi, const float* vs, uint64_t row_nl2, uint64_t row_nd2) {
  const uint64_t sl2 = mv::pack_f32x2(scale_log2, scale_log2), sc2 = mv::pack_f32x2(scale, scale);
  uint64_t nl[2][4], nd[2][4];
  lane_consts<MODE>(vs, 0, nl[0], nd[0], row_nl2, row_nd2);
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    if (g + 1 < 4) lane_consts<MODE>(vs, (g + 1) * 8, nl[(g + 1) & 1], nd[(g + 1) & 1], row_nl2, row_nd2);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int k = g * 8 + 2 * i;
      float x0, x1;
      mv::unpack_f32x2(mv::fma_f32x2(mv::pack_u32x2(s[k], s[k + 1]), sl2, nl[g & 1][i]), x0, x1);
      float p0 = mv::fast_exp2(x0), p1 = mv::fast_exp2(x1);
      if (!ALL) {
        // a masked pair has P = 0, and with it dS = 0: dP and delta are finite whatever the padding holds
        p0 = (j0 + k >= lo && j0 + k < hi) ? p0 : 0.f;
        p1 = (j0 + k + 1 >= lo && j0 + k + 1 < hi) ? p1 : 0.f;
      }
      if (MODE == DV) {
        o[k >> 1] = mv::pack_bf16(p0, p1);
      } else {
        float d0, d1;
        mv::unpack_f32x2(mv::mul_f32x2(mv::pack_f32x2(p0, p1), mv::fma_f32x2(mv::pack_u32x2(dp[k], dp[k + 1]), sc2, nd[g & 1][i])), d0, d1);
        o[k >> 1] = mv::pack_bf16(d0, d1);
      }
    }
  }
}

template <int MODE>
__device__ __forceinline__ void bwd_body(const BwdArgs& a, const CUtensorMap* tm_q, const CUtensorMap* tm_do, const CUtensorMap* tm_k,
                                         const CUtensorMap* tm_v, unsigned char* smem) {
  constexpr int NBUF = MODE == DV ? 3 : 2;  // score buffers
  Ctx c;
  if (!setup(c, smem, a.status)) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const mv::QTile tile = MODE == DQ ? a.q_tiles[blockIdx.y] : a.k_tiles[blockIdx.y];  // DK, DV: q_start / q_len are keys
  const mv::KvRange* ranges = (MODE == DQ ? a.kv_ranges : a.q_ranges) + tile.range_begin;
  // DQ: blockIdx.x is the query head.  DK, DV: the KV head, and a step's query head is kvh * G + its index in the group.
  const int kvh = MODE == DQ ? blockIdx.x / a.G : blockIdx.x;
  const int heads = MODE == DQ ? 1 : a.G;
  const int cut = MODE == DQ ? tile.causal_base + tile.q_len - 1 : 0x3fffffff;
  const Bars& br = c.br;
  const Waiter& w = c.w;
  const uint32_t fixed0 = c.smem_base + OFF_FIXED, fixed1 = fixed0 + TILE_BYTES;
  const uint32_t ring_long = c.smem_base + OFF_LONG, ring_short = c.smem_base + OFF_SHORT;
  if (warp == 0) {
    if (lane == 0) {  // producer
      const CUtensorMap* tm_f0 = MODE == DQ ? tm_q : tm_k;
      const CUtensorMap* tm_f1 = MODE == DQ ? tm_do : tm_v;
      const CUtensorMap* tm_long = MODE == DQ ? tm_k : (MODE == DK ? tm_q : tm_do);
      const CUtensorMap* tm_short = MODE == DQ ? tm_v : (MODE == DK ? tm_do : tm_q);
      const int fixed_col = (MODE == DQ ? int(blockIdx.x) : kvh) * D;
      mv::mbar_arrive_expect_tx(br.fixed_full, (MODE == DV ? 1 : 2) * TILE_BYTES);
      load_tile(fixed0, tm_f0, fixed_col, tile.q_start, br.fixed_full);
      if (MODE != DV) load_tile(fixed1, tm_f1, fixed_col, tile.q_start, br.fixed_full);
      Steps it(ranges, tile.range_count, cut, heads);
      int start, n, cz, hg, es = 0, el = 0;  // short / long tiles issued
      bool ok = true;
      while (ok && it.next(start, n, cz, hg)) {
        const int col = (MODE == DQ ? kvh : kvh * a.G + hg) * D;
        const int ss = es % NSHORT, ls = el % NLONG;
        ok = w.wait(br.sempty + 8 * ss, ((es / NSHORT) & 1) ^ 1);
        if (!ok) break;
        mv::mbar_arrive_expect_tx(br.sfull + 8 * ss, TILE_BYTES);
        load_tile(ring_short + ss * TILE_BYTES, tm_short, col, start, br.sfull + 8 * ss);
        ++es;
        ok = w.wait(br.lempty + 8 * ls, ((el / NLONG) & 1) ^ 1);
        if (!ok) break;
        mv::mbar_arrive_expect_tx(br.lfull + 8 * ls, TILE_BYTES);
        load_tile(ring_long + ls * TILE_BYTES, tm_long, col, start, br.lfull + 8 * ls);
        ++el;
      }
      if (!ok) {
        (void)mv::mbar_wait_bounded(br.fixed_full, 0, 20000000ull);
        drain_ring(br.sfull, NSHORT, es);
        drain_ring(br.lfull, NLONG, el);
      }
    }
  } else if (warp == 1 || warp == 2) {
    // Two issuers, because a thread that issues products is held until the tensor cores take them: warp 1 issues dP
    // and the scores, warp 2 the accumulating products, and the barrier waits of one fall into the products of the
    // other.  While the lane threads work on step e, warp 2 issues the accumulating product of step e - 1 and warp 1
    // dP of step e + 1 (the lane threads have copied dP of step e to registers by then), then the scores of step e + 1,
    // whose buffer the accumulating product of step e + 1 - NBUF has read.  The whole warp walks, one elected lane issues.
    const bool lead = mv::um::elect_one();
    Steps it(ranges, tile.range_count, cut, heads);
    int start, n, cz, hg, f = 0;
    bool ok = w.wait(br.fixed_full, 0);
    // Descriptors are made before the waits, and the wait that is satisfied last comes last, so that little stands
    // between a barrier's completion and the first product.
    if (warp == 1) {
      const uint64_t f0_desc = kmajor_desc(fixed0), f1_desc = kmajor_desc(fixed1);
      for (; ok && it.next(start, n, cz, hg); ++f) {
        const int b = f % NBUF, u = f / NBUF, ss = f % NSHORT, ls = f % NLONG;
        const uint64_t short_desc = kmajor_desc(ring_short + ss * TILE_BYTES), long_desc = kmajor_desc(ring_long + ls * TILE_BYTES);
        const uint32_t s_tmem = c.tmem + TM_S + 128 * b;
        ok = w.wait(br.sfull + 8 * ss, (f / NSHORT) & 1);
        if (MODE != DV) {
          if (ok && f >= 1) ok = w.wait(br.dp_free, (f - 1) & 1);  // the lane threads hold dP of step f - 1 in registers
          if (!ok) break;
          mv::um::fence_after();
          if (lead) {
            issue_nt(c.tmem + TM_DP, f1_desc, short_desc);  // dP = dO V^T  /  dP^T = V dO^T
            mv::um::commit(br.sempty + 8 * ss);
            mv::um::commit(br.dp_full);
          }
          __syncwarp();
          ok = w.wait(br.lfull + 8 * ls, (f / NLONG) & 1);
        }
        if (ok && f >= NBUF) ok = w.wait(br.acc_done + 8 * b, (u - 1) & 1);
        if (!ok) break;
        mv::um::fence_after();
        if (lead) {
          issue_nt(s_tmem, f0_desc, MODE == DV ? short_desc : long_desc);  // S = Q K^T  /  S^T = K Q^T
          if (MODE == DV) mv::um::commit(br.sempty + 8 * ss);
          mv::um::commit(br.s_full + 8 * b);
        }
        __syncwarp();
      }
    } else {
      for (; ok && it.next(start, n, cz, hg); ++f) {
        const int b = f % NBUF, ls = f % NLONG;
        const uint64_t long_desc = mnmajor_desc(ring_long + ls * TILE_BYTES);
        const uint32_t s_tmem = c.tmem + TM_S + 128 * b;
        if (MODE == DV) ok = w.wait(br.lfull + 8 * ls, (f / NLONG) & 1);
        if (ok) ok = w.wait(br.p_full + 8 * b, (f / NBUF) & 1);  // the lane threads have left dS (P^T in DV) in the buffer
        if (!ok) break;
        mv::um::fence_after();
        if (lead) {
          issue_tn(c.tmem + TM_ACC, s_tmem, long_desc, f > 0);  // dQ += dS K, dK += dS^T Q, dV += P^T dO
          mv::um::commit(br.acc_done + 8 * b);
          mv::um::commit(br.lempty + 8 * ls);
        }
        __syncwarp();
      }
    }
    if (w.aborted()) drain_issuer(br.drained + 8 * (warp - 1), lead);
  } else if (warp >= 4) {
    // lane threads: the two threads on tensor-memory lane r own row r of the tile (a query in DQ, a key in DK and DV),
    // 64 columns of a step each
    const int tl = threadIdx.x - 128;
    const int r = (warp & 3) * 32 + lane, ch = (warp - 4) >> 2;
    const uint32_t lane_base = c.tmem + (uint32_t((warp & 3) * 32) << 16);
    const bool row_ok = r < tile.q_len;
    const int tok = tile.q_start + r, rc = tile.causal_base + r;  // the row's token, and its index in the causal numbering
    float* vec = reinterpret_cast<float*>(smem + OFF_VEC);
    uint64_t row_nl2 = 0, row_nd2 = 0;
    if (MODE == DQ) {
      const float nl = row_ok ? -a.lse[int64_t(tok) * a.Hq + blockIdx.x] : 0.f;
      const float nd = row_ok ? -a.delta[int64_t(tok) * a.Hq + blockIdx.x] * a.scale : 0.f;
      row_nl2 = mv::pack_f32x2(nl, nl);
      row_nd2 = mv::pack_f32x2(nd, nd);
    }
    // DK, DV: the step's -lse and -scale * delta per query, fetched one step ahead by the lane threads themselves
    // (thread t < 128: lse of query t; t >= 128: delta of query t - 128) into the slot of the step's parity
    auto fetch = [&](int start, int n, int hg) -> float {
      const int x = tl & (BT - 1);
      if (x >= n) return 0.f;
      const int64_t at = int64_t(start + x) * a.Hq + kvh * a.G + hg;
      return tl < BT ? a.lse[at] : a.delta[at];
    };
    const float vec_mul = tl < BT ? -1.f : -a.scale;  // applied when the value is stored, a step after it was fetched
    Steps it(ranges, tile.range_count, cut, heads), ahead(ranges, tile.range_count, cut, heads);
    int start, n, cz, hg, e = 0;
    int a_start = 0, a_n = 0, a_cz = 0, a_hg = 0;
    bool a_ok = false, ok = true;
    if (MODE != DQ) {
      if (ahead.next(a_start, a_n, a_cz, a_hg)) vec[tl] = fetch(a_start, a_n, a_hg) * vec_mul;
      mv::mbar_arrive(br.vec_ready);
      a_ok = ahead.next(a_start, a_n, a_cz, a_hg);
    }
    while (it.next(start, n, cz, hg)) {
      const int b = e % NBUF;
      float pre = 0.f;
      if (MODE != DQ && a_ok) pre = fetch(a_start, a_n, a_hg);
      // dP is complete a product before the scores.  In DQ it goes to registers at once and the buffer back to the tensor
      // cores (measured: 1.91 -> 1.83 ms); in DK, whose lane threads have more to wait for, the extra wait costs more
      // than it gains (a step 2400 -> 2660 cycles), so dP is read together with the scores.
      constexpr bool DP_EARLY = MODE == DQ;
      uint32_t s0[32], s1[32], dp0[32], dp1[32], o[16];
      if (MODE != DV && DP_EARLY) {
        ok = w.warp_wait(br.dp_full, e & 1);
        if (!ok) break;
        mv::um::fence_after();
        mv::um::ld32(lane_base + TM_DP + ch * 64, dp0);
        mv::um::ld32(lane_base + TM_DP + ch * 64 + 32, dp1);
        mv::um::wait_ld();
        mv::um::fence_before();
        mv::mbar_arrive(br.dp_free);
      }
      if (MODE != DQ) ok = w.warp_wait(br.vec_ready, e & 1);
      if (ok) ok = w.warp_wait(br.s_full + 8 * b, (e / NBUF) & 1);
      if (!ok) break;
      mv::um::fence_after();
      // columns [lo, hi) of the step are visible to this row.  DQ: the keys up to the query's own (causal range) or all
      // n; DK, DV: the queries from the key's own on (own node) or all n.
      int lo, hi;
      if (MODE == DQ) {
        lo = 0;
        hi = row_ok ? (cz ? min(n, rc - start + 1) : n) : 0;
      } else {
        lo = row_ok ? (cz ? max(0, rc - start) : 0) : n;
        hi = n;
      }
      const uint32_t sbuf = lane_base + TM_S + 128 * b + ch * 64;
      const float* vs = vec + (e & 1) * 2 * BT + ch * 64;
      // DK is short of registers (the column constants are prefetched beside dP): it reads the second half of its
      // scores after the first half's arithmetic
      constexpr bool S1_LATE = MODE == DK;
      mv::um::ld32(sbuf, s0);
      if (!S1_LATE) mv::um::ld32(sbuf + 32, s1);
      if (MODE != DV && !DP_EARLY) {
        mv::um::ld32(lane_base + TM_DP + ch * 64, dp0);
        mv::um::ld32(lane_base + TM_DP + ch * 64 + 32, dp1);
      }
      mv::um::wait_ld();
      if (MODE != DV && !DP_EARLY) {
        mv::um::fence_before();
        mv::mbar_arrive(br.dp_free);  // dP is in registers: the tensor cores may write the next step's
      }
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const int j0 = ch * 64 + cc * 32;
        if (S1_LATE && cc == 1) {
          mv::um::ld32(sbuf + 32, s1);
          mv::um::wait_ld();
        }
        const uint32_t(&s)[32] = cc == 0 ? s0 : s1;
        const uint32_t* dp = cc == 0 ? dp0 : dp1;
        const bool all = __all_sync(0xffffffffu, lo <= j0 && hi >= j0 + 32);
        if (all) lane_math<MODE, true>(s, dp, o, a.scale_log2, a.scale, j0, lo, hi, vs + cc * 32, row_nl2, row_nd2);
        else lane_math<MODE, false>(s, dp, o, a.scale_log2, a.scale, j0, lo, hi, vs + cc * 32, row_nl2, row_nd2);
        // over the thread's own score columns that it has read: 16 packed columns per 32
        mv::um::st16(sbuf + cc * 16, o);
      }
      mv::um::wait_st();
      mv::um::fence_before();
      mv::mbar_arrive(br.p_full + 8 * b);
      if (MODE != DQ) {
        // every lane thread has passed this step's vec_ready wait, so none still reads the other slot (step e - 1's)
        asm volatile("" : "+f"(pre));  // the value is consumed here, not where the load was issued
        if (a_ok) vec[((e + 1) & 1) * 2 * BT + tl] = pre * vec_mul;
        mv::mbar_arrive(br.vec_ready);
        a_ok = ahead.next(a_start, a_n, a_cz, a_hg);
      }
      ++e;
    }
    if (ok && e > 0 && w.warp_wait(br.acc_done + 8 * ((e - 1) % NBUF), ((e - 1) / NBUF) & 1)) {
      mv::um::fence_after();
      bf16* dst;
      if (MODE == DQ) dst = a.dq + (int64_t(tok) * a.Hq + blockIdx.x) * D;
      else dst = (MODE == DK ? a.dk : a.dv) + (int64_t(tok) * a.Hkv + kvh) * D;
      dst += ch * 64;
#pragma unroll 1
      for (int cb = 0; cb < 2; ++cb) {
        uint32_t acc[32];
        mv::um::ld32(lane_base + TM_ACC + ch * 64 + cb * 32, acc);
        mv::um::wait_ld();
        if (row_ok) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            uint4 v;
            v.x = mv::pack_bf16(__uint_as_float(acc[8 * k]), __uint_as_float(acc[8 * k + 1]));
            v.y = mv::pack_bf16(__uint_as_float(acc[8 * k + 2]), __uint_as_float(acc[8 * k + 3]));
            v.z = mv::pack_bf16(__uint_as_float(acc[8 * k + 4]), __uint_as_float(acc[8 * k + 5]));
            v.w = mv::pack_bf16(__uint_as_float(acc[8 * k + 6]), __uint_as_float(acc[8 * k + 7]));
            *reinterpret_cast<uint4*>(dst + cb * 32 + k * 8) = v;
          }
        }
      }
    }
  }
  teardown(c);
}

__global__ void __launch_bounds__(NTHREADS, 1) dq_kernel(const BwdArgs a, const __grid_constant__ CUtensorMap tm_q,
                                                         const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_k,
                                                         const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  bwd_body<DQ>(a, &tm_q, &tm_do, &tm_k, &tm_v, smem);
}
// blockIdx.z = 0: dK, 1: dV (the longer CTAs are scheduled first)
__global__ void __launch_bounds__(NTHREADS, 1) dkv_kernel(const BwdArgs a, const __grid_constant__ CUtensorMap tm_q,
                                                          const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_k,
                                                          const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  if (blockIdx.z == 0) bwd_body<DK>(a, &tm_q, &tm_do, &tm_k, &tm_v, smem);
  else bwd_body<DV>(a, &tm_q, &tm_do, &tm_k, &tm_v, smem);
}

struct BwdMaps {
  CUtensorMap tm_q, tm_do, tm_k, tm_v;
};

}  // namespace

extern "C" mv_status mv_dag_prefill_attn_bwd(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_rot, const void* v,
                                             const void* out, const void* dout, const void* lse, void* dq_rot, void* dk_rot, void* dv,
                                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
  mv::NvtxRange nvtx_range("mv_dag_prefill_attn_bwd");
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (!P->stats.prefill_ready) return MV_ERR_UNSUPPORTED;
  if (g->dtype != MV_BF16 || g->head_dim != 128 || (g->n_q_heads / g->n_kv_heads) % 2 != 0) return MV_ERR_UNSUPPORTED;
  if (!q_rot || !k_rot || !v || !out || !dout || !lse || !dq_rot || !dk_rot || !dv) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  const uintptr_t all = reinterpret_cast<uintptr_t>(q_rot) | reinterpret_cast<uintptr_t>(k_rot) | reinterpret_cast<uintptr_t>(v) |
                        reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(dout) | reinterpret_cast<uintptr_t>(dq_rot) |
                        reinterpret_cast<uintptr_t>(dk_rot) | reinterpret_cast<uintptr_t>(dv);
  if (all & 15) return MV_ERR_INVALID_ARG;
  const size_t need = mv_workspace_bytes(P, g, MV_OP_PREFILL_ATTN_BWD);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return MV_ERR_WORKSPACE;
  if (P->q_tiles.size() > 65535 || P->k_tiles.size() > 65535) return MV_ERR_UNSUPPORTED;  // tiles are the grid's y dimension
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  static std::atomic<uint64_t> opted_dq{0}, opted_dkv{0};  // per device
  if (!mv::opt_in_smem(dq_kernel, SMEM_BYTES, opted_dq) || !mv::opt_in_smem(dkv_kernel, SMEM_BYTES, opted_dkv)) return MV_ERR_CUDA;
  const int64_t T = P->stats.n_new_tokens;
  static thread_local mv::KeyedCache<BwdMaps, 2> cache;
  // q and dO, k and v: the key names two pointers of each pair through a mix, plus extent and head counts
  const mv::TmapKey key{mv::current_device(), q_rot, dout, k_rot, T,
                        int64_t(reinterpret_cast<uintptr_t>(v) >> 4) ^ (int64_t(g->n_q_heads) << 52) ^ (int64_t(g->n_kv_heads) << 44)};
  BwdMaps* tm = cache.find(key);
  if (!tm) {
    tm = cache.claim(key);
    if (!mv::make_tmap_bf16_2d(&tm->tm_q, q_rot, uint64_t(T), uint64_t(g->n_q_heads) * D, BT) ||
        !mv::make_tmap_bf16_2d(&tm->tm_do, dout, uint64_t(T), uint64_t(g->n_q_heads) * D, BT) ||
        !mv::make_tmap_bf16_2d(&tm->tm_k, k_rot, uint64_t(T), uint64_t(g->n_kv_heads) * D, BT) ||
        !mv::make_tmap_bf16_2d(&tm->tm_v, v, uint64_t(T), uint64_t(g->n_kv_heads) * D, BT)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  BwdArgs a;
  a.q_tiles = mv::table<mv::QTile>(P, P->layout.q_tiles);
  a.kv_ranges = mv::table<mv::KvRange>(P, P->layout.kv_ranges);
  a.k_tiles = mv::table<mv::QTile>(P, P->layout.k_tiles);
  a.q_ranges = mv::table<mv::KvRange>(P, P->layout.q_ranges);
  a.lse = static_cast<const float*>(lse);
  a.delta = static_cast<float*>(workspace);
  a.dq = static_cast<bf16*>(dq_rot);
  a.dk = static_cast<bf16*>(dk_rot);
  a.dv = static_cast<bf16*>(dv);
  a.status = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2;
  a.Hq = g->n_q_heads;
  a.Hkv = g->n_kv_heads;
  a.G = g->n_q_heads / g->n_kv_heads;
  a.T = int(T);
  a.scale = mv::softmax_scale(g);
  a.scale_log2 = a.scale * 1.4426950408889634f;
  const int64_t n_row_heads = T * g->n_q_heads;
  delta_kernel<<<unsigned((n_row_heads + 3) / 4), 128, 0, s>>>(static_cast<const bf16*>(out), static_cast<const bf16*>(dout),
                                                              static_cast<float*>(workspace), n_row_heads);
  mv::g_launches++;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  dq_kernel<<<dim3(unsigned(g->n_q_heads), unsigned(P->q_tiles.size())), NTHREADS, SMEM_BYTES, s>>>(a, tm->tm_q, tm->tm_do, tm->tm_k, tm->tm_v);
  mv::g_launches++;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  dkv_kernel<<<dim3(unsigned(g->n_kv_heads), unsigned(P->k_tiles.size()), 2), NTHREADS, SMEM_BYTES, s>>>(a, tm->tm_q, tm->tm_do, tm->tm_k, tm->tm_v);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}
