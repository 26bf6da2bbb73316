// Backward of the topology-masked prefill attention (the attention the model is fine-tuned through, Sec. 5.1: the
// mask of Eq. 3 at the position indices of Sec. 4.2) on the 5th-generation tensor cores: head_dim 128, bf16 in, fp32
// accumulation in tensor memory.
//
// With S = scale * Q K^T + M, P = softmax(S) and O = P V (Eq. 2 - 3), a gradient dO of the output gives
//   dV = P^T dO,  dP = dO V^T,  dS = P o (dP - delta),  delta_i = sum_j P_ij dP_ij = <dO_i, O_i>,
//   dQ = scale * dS K,  dK = scale * dS^T Q,
// a KV head collecting dK and dV from every query head of its group.  P is rebuilt from the scores and the row's
// log-sum-exp that the forward kernel leaves (no second softmax pass).  Three kernels:
//   delta_kernel     delta[i][h] = <dO[i][h], O[i][h]>                                   (elementwise, one warp per row-head)
//   dq_kernel        one CTA per (query tile, query head): walks the KV tiles the tile's node may see, exactly the
//                    forward's walk: S = Q K^T and dP = dO V^T into tensor memory, one thread per query row turns them
//                    into dS (bf16, written back over S), dQ += dS K with K as the MN-major operand.
//   dkv_kernel       one CTA per (key tile, KV head): walks the transposed lists (the runs of queries that see the tile's
//                    node; its own node causally) for every query head of the group: S^T = K Q^T and dP^T = V dO^T into
//                    tensor memory (a lane is a key, a column a query), one thread per key builds P^T and dS^T (bf16,
//                    written back in place), dV += P^T dO and dK += dS^T Q with dO and Q as MN-major operands.
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
constexpr int HB = 64;                  // a step is one 64-column half of a 128 x 128 score tile
constexpr int HALF_BYTES = HB * D * 2;  // 16 KB: [2 column blocks][64 rows][128 B]
constexpr int NTHREADS = 320;           // warp 0 producer, warp 1 issuer, warps 2..9: two threads per tensor-memory lane,
                                        // each taking 32 of a step's 64 columns
constexpr int OFF_FIXED = 0;            // two 128-row tiles that stay for the whole CTA (dq: Q, dO; dkv: K, V)
constexpr int OFF_RING = 2 * TILE_BYTES;  // stages of two 64-row halves (dq: K, V; dkv: Q, dO), one stage per step
constexpr int NSTAGE = 4;
constexpr int STAGE_BYTES = 2 * HALF_BYTES;
constexpr int OFF_VEC = OFF_RING + NSTAGE * STAGE_BYTES;  // dkv: per stage lse[64], delta[64] of the step's queries
constexpr int OFF_BAR = OFF_VEC + NSTAGE * 2 * HB * 4;
constexpr int N_BARS = 2 + 2 * NSTAGE + 6;
constexpr int SMEM_BYTES = OFF_BAR + N_BARS * 8 + 16;

struct BwdArgs {
  const mv::QTile* tiles;     // dq: query tiles; dkv: key tiles
  const mv::KvRange* ranges;  // dq: key ranges;  dkv: query ranges
  const float* lse;           // [T][Hq] log2-domain log-sum-exp of the forward
  const float* delta;         // [T][Hq]
  bf16* dq;                   // [T][Hq][D]
  bf16* dk;                   // [T][Hkv][D]
  bf16* dv;
  int32_t* status;
  int Hq, Hkv, G, T;
  float scale_log2, scale;
};

struct Bars {
  // full / empty: NSTAGE consecutive barriers; s_full / p_full / acc_done: one per score buffer (two)
  uint32_t fixed_full, full, empty, s_full, p_full, acc_done, drained;
};

struct Waiter {
  volatile int* abort;
  int32_t* status;
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
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

// 64-row steps of a tile's ranges, in table order.  FWD walk (dq): a causal range ends after the tile's last query.
// Transposed walk (dkv): a causal range starts at the tile's first key and is not cut.
struct Walk {
  const mv::KvRange* rg;
  int n_ranges, last_causal;  // last_causal: last index a causal range may reach (dq), or a very large number (dkv)
  int ri = 0, pos = 0, end = 0, causal = 0;
  __device__ Walk(const mv::KvRange* r, int n, int lc) : rg(r), n_ranges(n), last_causal(lc) {}
  __device__ bool next(int& start, int& n, int& c) {
    while (pos >= end) {
      if (ri >= n_ranges) return false;
      const mv::KvRange r = rg[ri++];
      pos = r.kv_start;
      end = r.kv_start + r.kv_len;
      causal = r.causal;
      if (causal) end = min(end, last_causal + 1);
    }
    start = pos;
    n = min(HB, end - pos);
    c = causal;
    pos += HB;
    return true;
  }
};

// every tensor map's box is 64 columns x 64 rows (8 KB)
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap* tm, int col, int row, uint32_t bar) {
  for (int cb = 0; cb < 2; ++cb)
    for (int rh = 0; rh < 2; ++rh) mv::tma_load_2d(dst + cb * (TILE_BYTES / 2) + rh * (HALF_BYTES / 2), tm, col + cb * 64, row + rh * HB, bar);
}
__device__ __forceinline__ void load_half(uint32_t dst, const CUtensorMap* tm, int col, int row, uint32_t bar) {
  for (int cb = 0; cb < 2; ++cb) mv::tma_load_2d(dst + cb * (HALF_BYTES / 2), tm, col + cb * 64, row, bar);
}

// D[tmem, 128 x 64] = A B^T, A a K-major 128-row tile, B a K-major 64-row half: eight k-steps over head_dim
__device__ __forceinline__ void issue_nt(uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr) {
  constexpr uint32_t idesc = mv::um::idesc_bf16(BT, HB, 0, 0);
  const uint64_t a_desc = mv::um::smem_desc(a_addr, 16, 1024), b_desc = mv::um::smem_desc(b_addr, 16, 1024);
  mv::um::mma_ss<false>(d_tmem, a_desc, b_desc, idesc);
#pragma unroll
  for (int k = 1; k < D / 16; ++k) {
    const uint32_t a_off = ((k >> 2) * (TILE_BYTES / 2) + (k & 3) * 32) >> 4, b_off = ((k >> 2) * (HALF_BYTES / 2) + (k & 3) * 32) >> 4;
    mv::um::mma_ss<true>(d_tmem, a_desc + a_off, b_desc + b_off, idesc);
  }
}
// D[tmem, 128 x 128] (+)= A[tmem, 128 x 64 as bf16 pairs] B with B a 64-row half read as the MN-major operand
// ([64 contraction rows][128 columns]): four k-steps.  The lane threads leave A in two pieces, the pairs of a step's
// columns 0..31 at a_tmem + 0..15 and those of columns 32..63 at a_tmem + 32..47.
__device__ __forceinline__ void issue_tn(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_addr, bool accumulate) {
  constexpr uint32_t idesc = mv::um::idesc_bf16(BT, D, 0, 1);
  const uint64_t b_desc = mv::um::smem_desc(b_addr, HALF_BYTES / 2, 1024);
  if (accumulate) mv::um::mma_ts<true>(d_tmem, a_tmem, b_desc, idesc);
  else mv::um::mma_ts<false>(d_tmem, a_tmem, b_desc, idesc);
#pragma unroll
  for (int k = 1; k < HB / 16; ++k)
    mv::um::mma_ts<true>(d_tmem, a_tmem + (k >> 1) * 32 + (k & 1) * 8, b_desc + uint32_t((k * 2048) >> 4), idesc);
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
  c.br.fixed_full = mv::smem_u32(&bars[0]);
  c.br.full = mv::smem_u32(&bars[1]);
  c.br.empty = mv::smem_u32(&bars[1 + NSTAGE]);
  c.br.s_full = mv::smem_u32(&bars[1 + 2 * NSTAGE]);
  c.br.p_full = mv::smem_u32(&bars[3 + 2 * NSTAGE]);
  c.br.acc_done = mv::smem_u32(&bars[5 + 2 * NSTAGE]);
  c.br.drained = mv::smem_u32(&bars[7 + 2 * NSTAGE]);
  static_assert(8 + 2 * NSTAGE <= N_BARS, "barrier table too small");
  if ((c.smem_base & 1023u) != 0) {  // the swizzle pattern is anchored at 1024-byte boundaries
    if (tid == 0) atomicExch(status, int(MV_ERR_UNSUPPORTED));
    return false;
  }
  if (tid == 0) {
    *abort_flag = 0;
    mv::mbar_init(c.br.fixed_full, 1);
    for (int i = 0; i < NSTAGE; ++i) {
      mv::mbar_init(c.br.full + 8 * i, 1);
      mv::mbar_init(c.br.empty + 8 * i, 1);  // one tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      mv::mbar_init(c.br.s_full + 8 * b, 1);     // one tcgen05.commit
      mv::mbar_init(c.br.p_full + 8 * b, 256);   // the 256 lane threads
      mv::mbar_init(c.br.acc_done + 8 * b, 1);   // one tcgen05.commit
    }
    mv::mbar_init(c.br.drained, 1);
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
__device__ __forceinline__ void drain_producer(const Ctx& c, int e) {
  (void)mv::mbar_wait_bounded(c.br.fixed_full, 0, 20000000ull);
  for (int k = 1; k <= min(e, NSTAGE); ++k)
    (void)mv::mbar_wait_bounded(c.br.full + 8 * ((e - k) % NSTAGE), ((e - k) / NSTAGE) & 1, 20000000ull);
}
__device__ __forceinline__ void drain_issuer(const Ctx& c, bool lead) {
  __syncwarp();
  if (lead) mv::um::commit(c.br.drained);
  (void)mv::mbar_wait_bounded(c.br.drained, 0, 20000000ull);
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

// ---- dQ ------------------------------------------------------------------------------------------------------
// The visible keys are taken in steps of 64, one ring stage (K, V halves) per step, alternating between two score
// buffers in tensor memory, so that the tensor cores compute the next step's S and dP while the lane threads turn this
// one's into dS.  Buffer b: S at 128 b (dS written back over its columns 0..15 and 32..47), dP at 128 b + 64; the dQ
// accumulator at +256.

__global__ void __launch_bounds__(NTHREADS, 1) dq_kernel(const BwdArgs a, const __grid_constant__ CUtensorMap tm_q,
                                                         const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_k,
                                                         const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Ctx c;
  if (!setup(c, smem, a.status)) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const mv::QTile qt = a.tiles[blockIdx.y];
  const int head = blockIdx.x, kvh = head / a.G;
  const Bars& br = c.br;
  const Waiter& w = c.w;
  const int q_last = qt.causal_base + qt.q_len - 1;
  if (warp == 0) {
    if (lane == 0) {  // producer
      mv::mbar_arrive_expect_tx(br.fixed_full, 2 * TILE_BYTES);
      load_tile(c.smem_base + OFF_FIXED, &tm_q, head * D, qt.q_start, br.fixed_full);
      load_tile(c.smem_base + OFF_FIXED + TILE_BYTES, &tm_do, head * D, qt.q_start, br.fixed_full);
      Walk it(a.ranges + qt.range_begin, qt.range_count, q_last);
      int start, n, cz, e = 0;
      bool ok = true;
      while (ok && it.next(start, n, cz)) {
        const int st = e % NSTAGE;
        ok = w.wait(br.empty + 8 * st, ((e / NSTAGE) & 1) ^ 1);
        if (!ok) break;
        mv::mbar_arrive_expect_tx(br.full + 8 * st, STAGE_BYTES);
        load_half(c.smem_base + OFF_RING + st * STAGE_BYTES, &tm_k, kvh * D, start, br.full + 8 * st);
        load_half(c.smem_base + OFF_RING + st * STAGE_BYTES + HALF_BYTES, &tm_v, kvh * D, start, br.full + 8 * st);
        ++e;
      }
      if (!ok) drain_producer(c, e);
    }
  } else if (warp == 1) {
    // issuer: the whole warp walks, one elected lane issues.  The dQ product of a step is issued after the scores of
    // the step behind it, so the tensor cores always have the next scores queued while the lane threads work.
    const bool lead = mv::um::elect_one();
    Walk it(a.ranges + qt.range_begin, qt.range_count, q_last);
    const uint32_t q_addr = c.smem_base + OFF_FIXED, do_addr = q_addr + TILE_BYTES;
    int start, n, cz, e = 0;
    // step f's dQ product: after the lane threads have left dS in buffer f & 1; it frees the buffer and the stage
    auto finish = [&](int f) -> bool {
      const int b = f & 1;
      if (!w.wait(br.p_full + 8 * b, (f >> 1) & 1)) return false;
      mv::um::fence_after();
      if (lead) {
        issue_tn(c.tmem + 256, c.tmem + 128 * b, c.smem_base + OFF_RING + (f % NSTAGE) * STAGE_BYTES, f > 0);  // dQ += dS K
        mv::um::commit(br.acc_done + 8 * b);
        mv::um::commit(br.empty + 8 * (f % NSTAGE));
      }
      __syncwarp();
      return true;
    };
    bool ok = w.wait(br.fixed_full, 0);
    while (ok && it.next(start, n, cz)) {
      const int st = e % NSTAGE, b = e & 1;
      const uint32_t kh = c.smem_base + OFF_RING + st * STAGE_BYTES, vh = kh + HALF_BYTES;
      ok = w.wait(br.full + 8 * st, (e / NSTAGE) & 1);
      // the dQ product two steps back has read dS from this buffer before the new scores overwrite it
      if (ok && e >= 2) ok = w.wait(br.acc_done + 8 * b, ((e >> 1) - 1) & 1);
      if (!ok) break;
      mv::um::fence_after();
      if (lead) {
        issue_nt(c.tmem + 128 * b, q_addr, kh);         // S = Q K^T
        issue_nt(c.tmem + 128 * b + HB, do_addr, vh);   // dP = dO V^T
        mv::um::commit(br.s_full + 8 * b);
      }
      __syncwarp();
      if (e > 0) ok = finish(e - 1);
      ++e;
    }
    if (ok && e > 0) ok = finish(e - 1);
    if (w.aborted()) drain_issuer(c, lead);
  } else {
    // lane threads: the two threads on tensor-memory lane r own query row r of the tile, 32 columns of a step each
    const int r = (warp & 3) * 32 + lane, ch = (warp - 2) >> 2;
    const uint32_t lane_base = c.tmem + (uint32_t((warp & 3) * 32) << 16);
    const int qi = qt.q_start + r, qc = qt.causal_base + r;
    const bool row_ok = r < qt.q_len;
    const float lse = row_ok ? a.lse[int64_t(qi) * a.Hq + head] : 0.f;
    const float dl = row_ok ? a.delta[int64_t(qi) * a.Hq + head] * a.scale : 0.f;
    Walk it(a.ranges + qt.range_begin, qt.range_count, q_last);
    int start, n, cz, e = 0;
    bool ok = true;
    while (it.next(start, n, cz)) {
      const int b = e & 1;
      const int lim = row_ok ? (cz ? min(n, qc - start + 1) : n) : 0;  // keys [0, lim) of the step are visible to this row
      ok = w.warp_wait(br.s_full + 8 * b, (e >> 1) & 1);
      if (!ok) break;
      mv::um::fence_after();
      const uint32_t base = lane_base + 128 * b + ch * 32;
      const int j0 = ch * 32;
      uint32_t s[32], dp[32], ds[16];
      mv::um::ld32(base, s);
      mv::um::ld32(base + HB, dp);
      mv::um::wait_ld();
#pragma unroll
      for (int k = 0; k < 32; k += 2) {
        // a masked pair has P = 0, and with it dS = 0: dP and delta are finite whatever the padding holds
        const float p0 = j0 + k < lim ? mv::fast_exp2(fmaf(__uint_as_float(s[k]), a.scale_log2, -lse)) : 0.f;
        const float p1 = j0 + k + 1 < lim ? mv::fast_exp2(fmaf(__uint_as_float(s[k + 1]), a.scale_log2, -lse)) : 0.f;
        const float d0 = p0 * fmaf(__uint_as_float(dp[k]), a.scale, -dl);
        const float d1 = p1 * fmaf(__uint_as_float(dp[k + 1]), a.scale, -dl);
        ds[k >> 1] = mv::pack_bf16(d0, d1);
      }
      mv::um::st16(base, ds);  // over the thread's own S columns, which it has read
      mv::um::wait_st();
      mv::um::fence_before();
      mv::mbar_arrive(br.p_full + 8 * b);
      ++e;
    }
    if (ok && e > 0 && w.warp_wait(br.acc_done + 8 * ((e - 1) & 1), ((e - 1) >> 1) & 1)) {
      mv::um::fence_after();
      bf16* dst = a.dq + (int64_t(qi) * a.Hq + head) * D + ch * 64;
#pragma unroll 1
      for (int cb = 0; cb < 2; ++cb) {
        uint32_t o[32];
        mv::um::ld32(lane_base + 256 + ch * 64 + cb * 32, o);
        mv::um::wait_ld();
        if (row_ok) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            uint4 v;
            v.x = mv::pack_bf16(__uint_as_float(o[8 * k]), __uint_as_float(o[8 * k + 1]));
            v.y = mv::pack_bf16(__uint_as_float(o[8 * k + 2]), __uint_as_float(o[8 * k + 3]));
            v.z = mv::pack_bf16(__uint_as_float(o[8 * k + 4]), __uint_as_float(o[8 * k + 5]));
            v.w = mv::pack_bf16(__uint_as_float(o[8 * k + 6]), __uint_as_float(o[8 * k + 7]));
            *reinterpret_cast<uint4*>(dst + cb * 32 + k * 8) = v;
          }
        }
      }
    }
  }
  teardown(c);
}

// ---- dK, dV --------------------------------------------------------------------------------------------------
// A step is (64 queries that see the tile's node, one query head of the group): one ring stage holds the Q and dO
// halves and the queries' lse and delta.  Two score buffers as in dq_kernel.  Buffer b: S^T at 128 b (P^T written
// back over its columns 0..15 and 32..47), dP^T at 128 b + 64 (dS^T likewise); the dV accumulator at +256, dK at +384.
__global__ void __launch_bounds__(NTHREADS, 1) dkv_kernel(const BwdArgs a, const __grid_constant__ CUtensorMap tm_q,
                                                          const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_k,
                                                          const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Ctx c;
  if (!setup(c, smem, a.status)) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const mv::QTile kt = a.tiles[blockIdx.y];  // q_start / q_len: the tile's first key and key count
  const int kvh = blockIdx.x;
  const Bars& br = c.br;
  const Waiter& w = c.w;
  constexpr int NO_CUT = 0x3fffffff;
  float* vec = reinterpret_cast<float*>(smem + OFF_VEC);  // [stage][lse 64 | delta * scale 64]
  if (warp == 0) {
    // producer: lane 0 issues the tile copies; all lanes fetch the stage's lse / delta vectors with plain loads
    if (lane == 0) {
      mv::mbar_arrive_expect_tx(br.fixed_full, 2 * TILE_BYTES);
      load_tile(c.smem_base + OFF_FIXED, &tm_k, kvh * D, kt.q_start, br.fixed_full);
      load_tile(c.smem_base + OFF_FIXED + TILE_BYTES, &tm_v, kvh * D, kt.q_start, br.fixed_full);
    }
    Walk it(a.ranges + kt.range_begin, kt.range_count, NO_CUT);
    int start, n, cz, e = 0;
    bool ok = true;
    while (ok && it.next(start, n, cz)) {
      for (int hg = 0; hg < a.G && ok; ++hg, ++e) {
        const int st = e % NSTAGE, head = kvh * a.G + hg;
        int go = 1;
        if (lane == 0) go = w.wait(br.empty + 8 * st, ((e / NSTAGE) & 1) ^ 1) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, go, 0) != 0;
        if (!ok) break;
        float* vs = vec + st * 2 * HB;
        for (int x = lane; x < HB; x += 32) {
          const bool in = x < n;
          vs[x] = in ? a.lse[int64_t(start + x) * a.Hq + head] : 0.f;
          vs[HB + x] = in ? a.delta[int64_t(start + x) * a.Hq + head] * a.scale : 0.f;
        }
        __syncwarp();
        if (lane == 0) {
          mv::mbar_arrive_expect_tx(br.full + 8 * st, STAGE_BYTES);  // releases the vector stores above
          load_half(c.smem_base + OFF_RING + st * STAGE_BYTES, &tm_q, head * D, start, br.full + 8 * st);
          load_half(c.smem_base + OFF_RING + st * STAGE_BYTES + HALF_BYTES, &tm_do, head * D, start, br.full + 8 * st);
        }
      }
    }
    if (!ok && lane == 0) drain_producer(c, e);
    __syncwarp();
  } else if (warp == 1) {
    const bool lead = mv::um::elect_one();
    Walk it(a.ranges + kt.range_begin, kt.range_count, NO_CUT);
    const uint32_t k_addr = c.smem_base + OFF_FIXED, v_addr = k_addr + TILE_BYTES;
    int start, n, cz, e = 0;
    // step f's accumulating products: after the lane threads have left P^T and dS^T in buffer f & 1
    auto finish = [&](int f) -> bool {
      const int b = f & 1;
      if (!w.wait(br.p_full + 8 * b, (f >> 1) & 1)) return false;
      mv::um::fence_after();
      if (lead) {
        const uint32_t qh = c.smem_base + OFF_RING + (f % NSTAGE) * STAGE_BYTES, doh = qh + HALF_BYTES;
        issue_tn(c.tmem + 256, c.tmem + 128 * b, doh, f > 0);      // dV += P^T dO
        issue_tn(c.tmem + 384, c.tmem + 128 * b + HB, qh, f > 0);  // dK += dS^T Q
        mv::um::commit(br.acc_done + 8 * b);
        mv::um::commit(br.empty + 8 * (f % NSTAGE));
      }
      __syncwarp();
      return true;
    };
    bool ok = w.wait(br.fixed_full, 0);
    while (ok && it.next(start, n, cz)) {
      for (int hg = 0; hg < a.G && ok; ++hg, ++e) {
        const int st = e % NSTAGE, b = e & 1;
        const uint32_t qh = c.smem_base + OFF_RING + st * STAGE_BYTES, doh = qh + HALF_BYTES;
        ok = w.wait(br.full + 8 * st, (e / NSTAGE) & 1);
        // the products two steps back have read P^T and dS^T from this buffer before the new scores overwrite them
        if (ok && e >= 2) ok = w.wait(br.acc_done + 8 * b, ((e >> 1) - 1) & 1);
        if (!ok) break;
        mv::um::fence_after();
        if (lead) {
          issue_nt(c.tmem + 128 * b, k_addr, qh);         // S^T = K Q^T
          issue_nt(c.tmem + 128 * b + HB, v_addr, doh);   // dP^T = V dO^T
          mv::um::commit(br.s_full + 8 * b);
        }
        __syncwarp();
        if (e > 0) ok = finish(e - 1);
      }
    }
    if (ok && e > 0) ok = finish(e - 1);
    if (w.aborted()) drain_issuer(c, lead);
  } else {
    // lane threads: the two threads on tensor-memory lane r own key r of the tile, 32 queries of a step each
    const int r = (warp & 3) * 32 + lane, ch = (warp - 2) >> 2;
    const uint32_t lane_base = c.tmem + (uint32_t((warp & 3) * 32) << 16);
    const bool key_ok = r < kt.q_len;
    const int kc = kt.causal_base + r;  // the key's flattened index
    Walk it(a.ranges + kt.range_begin, kt.range_count, NO_CUT);
    int start, n, cz, e = 0;
    bool ok = true;
    while (ok && it.next(start, n, cz)) {
      // queries [first, n) of the step see this key: all valid ones, or (own node) those not before the key
      const int first = key_ok ? (cz ? max(0, kc - start) : 0) : n;
      for (int hg = 0; hg < a.G && ok; ++hg, ++e) {
        const int st = e % NSTAGE, b = e & 1;
        ok = w.warp_wait(br.full + 8 * st, (e / NSTAGE) & 1);  // the stage's lse / delta vectors are visible
        if (ok) ok = w.warp_wait(br.s_full + 8 * b, (e >> 1) & 1);
        if (!ok) break;
        mv::um::fence_after();
        const float4* vl = reinterpret_cast<const float4*>(vec + st * 2 * HB + ch * 32);
        const float4* vd = reinterpret_cast<const float4*>(vec + st * 2 * HB + HB + ch * 32);
        const uint32_t base = lane_base + 128 * b + ch * 32;
        const int j0 = ch * 32;
        uint32_t s[32], dp[32], pt[16], ds[16];
        mv::um::ld32(base, s);
        mv::um::ld32(base + HB, dp);
        mv::um::wait_ld();
#pragma unroll
        for (int k = 0; k < 32; k += 4) {
          const float4 l4 = vl[k >> 2], d4 = vd[k >> 2];
          const float ls[4] = {l4.x, l4.y, l4.z, l4.w}, dl[4] = {d4.x, d4.y, d4.z, d4.w};
          float p[4], d[4];
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int j = j0 + k + x;
            // a masked pair has P = 0, and with it dS = 0: dP and delta are finite whatever the padding holds
            p[x] = (j >= first && j < n) ? mv::fast_exp2(fmaf(__uint_as_float(s[k + x]), a.scale_log2, -ls[x])) : 0.f;
            d[x] = p[x] * fmaf(__uint_as_float(dp[k + x]), a.scale, -dl[x]);
          }
          pt[k >> 1] = mv::pack_bf16(p[0], p[1]);
          pt[(k >> 1) + 1] = mv::pack_bf16(p[2], p[3]);
          ds[k >> 1] = mv::pack_bf16(d[0], d[1]);
          ds[(k >> 1) + 1] = mv::pack_bf16(d[2], d[3]);
        }
        mv::um::st16(base, pt);       // over the thread's own S^T columns, which it has read
        mv::um::st16(base + HB, ds);  // and over its own dP^T columns
        mv::um::wait_st();
        mv::um::fence_before();
        mv::mbar_arrive(br.p_full + 8 * b);
      }
    }
    if (ok && e > 0 && w.warp_wait(br.acc_done + 8 * ((e - 1) & 1), ((e - 1) >> 1) & 1)) {
      mv::um::fence_after();
      const int64_t tok = int64_t(kt.q_start + r);
#pragma unroll 1
      for (int which = 0; which < 2; ++which) {
        bf16* dst = (which == 0 ? a.dv : a.dk) + (tok * a.Hkv + kvh) * D + ch * 64;
#pragma unroll 1
        for (int cb = 0; cb < 2; ++cb) {
          uint32_t o[32];
          mv::um::ld32(lane_base + 256 + which * 128 + ch * 64 + cb * 32, o);
          mv::um::wait_ld();
          if (key_ok) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              uint4 v;
              v.x = mv::pack_bf16(__uint_as_float(o[8 * k]), __uint_as_float(o[8 * k + 1]));
              v.y = mv::pack_bf16(__uint_as_float(o[8 * k + 2]), __uint_as_float(o[8 * k + 3]));
              v.z = mv::pack_bf16(__uint_as_float(o[8 * k + 4]), __uint_as_float(o[8 * k + 5]));
              v.w = mv::pack_bf16(__uint_as_float(o[8 * k + 6]), __uint_as_float(o[8 * k + 7]));
              *reinterpret_cast<uint4*>(dst + cb * 32 + k * 8) = v;
            }
          }
        }
      }
    }
  }
  teardown(c);
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
    if (!mv::make_tmap_bf16_2d(&tm->tm_q, q_rot, uint64_t(T), uint64_t(g->n_q_heads) * D, HB) ||
        !mv::make_tmap_bf16_2d(&tm->tm_do, dout, uint64_t(T), uint64_t(g->n_q_heads) * D, HB) ||
        !mv::make_tmap_bf16_2d(&tm->tm_k, k_rot, uint64_t(T), uint64_t(g->n_kv_heads) * D, HB) ||
        !mv::make_tmap_bf16_2d(&tm->tm_v, v, uint64_t(T), uint64_t(g->n_kv_heads) * D, HB)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  BwdArgs a;
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
  a.tiles = mv::table<mv::QTile>(P, P->layout.q_tiles);
  a.ranges = mv::table<mv::KvRange>(P, P->layout.kv_ranges);
  dq_kernel<<<dim3(unsigned(g->n_q_heads), unsigned(P->q_tiles.size())), NTHREADS, SMEM_BYTES, s>>>(a, tm->tm_q, tm->tm_do, tm->tm_k, tm->tm_v);
  mv::g_launches++;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  a.tiles = mv::table<mv::QTile>(P, P->layout.k_tiles);
  a.ranges = mv::table<mv::KvRange>(P, P->layout.q_ranges);
  dkv_kernel<<<dim3(unsigned(g->n_kv_heads), unsigned(P->k_tiles.size())), NTHREADS, SMEM_BYTES, s>>>(a, tm->tm_q, tm->tm_do, tm->tm_k, tm->tm_v);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}
