// Topology-masked prefill attention on the 5th-generation tensor cores (Eq. 2 with the DAG mask of Eq. 3 in
// visibility-set form), head_dim 128, bf16 in, fp32 accumulation in tensor memory.
//
// A CTA owns one query tile (128 rows of one node) for TWO query heads of the same KV head, so the two
// problems walk the same KV tiles with the same mask and every K / V tile that TMA brings in feeds four
// 128 x 128 x 128 products.  Only the KV ranges the tile's node may see are walked (tile skipping); the
// causal test applies only inside the node's own range and only on tiles that touch the diagonal; ragged
// range ends are masked by a column bound.
//
// Warp roles (384 threads): warp 0 = TMA producer (Q tiles once, then a ring of K and V tiles), warp 1 =
// MMA issuer (one thread: S_i = Q_i K^T into tensor memory, O_i += P_i V with P_i read from tensor memory),
// warps 4-7 and 8-11 = softmax groups of head 0 and head 1 (one thread per query row: online softmax in
// log2 units, P written back over S as packed bf16, O rescaled in tensor memory only when the row maximum
// moved by more than 2^8, final normalisation and store).  The issuer alternates the two heads, so one
// group's softmax overlaps the other head's products.  Every mbarrier wait is bounded (status word).
//
// The same kernel in its PAGED form serves node append (several new tokens of a node against the page pool, Sec. 4.3):
// a KV range is then one whole visible node, its 128-key tiles are gathered page by page (one 2 KB box per page and
// column block, the pool layout of the decode kernels), keys are counted inside the node, and the causal range is the
// tile's own node with the first query sitting at key index causal_base.
#include "common.cuh"
#include "tmap_cache.h"
#include "umma.cuh"

namespace {

using bf16 = __nv_bfloat16;
constexpr int D = 128;
constexpr int BQ = 128;                 // query rows per tile
constexpr int BK = 128;                 // keys per KV tile
constexpr int TILE_BYTES = BK * D * 2;  // 32 KB: [2 column blocks][128 rows][128 B]
constexpr int RING = 5;                 // K and V tiles in flight (K0 V0 K1 V1 ...)
constexpr int NTHREADS = 384;
constexpr int OFF_Q = 0;                        // Q0, Q1
constexpr int OFF_RING = 2 * TILE_BYTES;        // ring entries
constexpr int OFF_BAR = OFF_RING + RING * TILE_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256;
constexpr float RESCALE_THRESHOLD = 8.f;  // log2 units: P stays below 2^8, well inside bf16 and fp32 range

struct Bars {  // shared-memory addresses
  uint32_t q_full, kv_full, kv_empty, s_full, p_full, o_done, drained;
};

struct PrefillArgs {
  const mv::QTile* q_tiles;
  const mv::KvRange* ranges;
  const int32_t* page_tab;  // paged form: page ids, indexed by KvRange::pages + key / 16
  bf16* out;
  float* lse;  // optional [T][n_q_heads]: log2 of the row's softmax denominator, in the units of scale_log2 * score
  int32_t* status;
  int Hq, Hkv, G;
  float scale_log2;
};

// The KV tiles of a query tile, in the order every role walks them: ranges in table order, 128 keys at a time;
// a causal range stops after the tile's last query (q_last: its index in the causal range's key numbering).
struct TileIter {
  const mv::KvRange* rg;
  int n_ranges, q_last;
  int ri = 0, pos = 0, end = 0, causal = 0;
  int pages = 0;    // paged form: first page-table index of the current range
  mv::KvRange nxt;  // the range after the current one, read one range ahead so that no load sits on the walk
  __device__ TileIter(const mv::KvRange* r, int n, int ql) : rg(r), n_ranges(n), q_last(ql) {
    nxt = n > 0 ? r[0] : mv::KvRange{0, 0, 0, 0};
  }
  // start key, valid keys (1..128), causal flag of the next tile; false when the walk is over
  __device__ bool next(int& start, int& n, int& c) {
    while (pos >= end) {
      if (ri >= n_ranges) return false;
      const mv::KvRange r = nxt;
      if (++ri < n_ranges) nxt = rg[ri];
      pos = r.kv_start;
      end = r.kv_start + r.kv_len;
      causal = r.causal;
      pages = r.pages;
      if (causal) end = min(end, q_last + 1);
    }
    start = pos;
    n = min(BK, end - pos);
    c = causal;
    pos += BK;
    return true;
  }
};

// Bounded waits.  wait() is false once a wait of this CTA has run out (this one or an earlier one, of any role): the
// caller then issues nothing further, leaves its loops, and the producer and the issuer wait (again bounded) for what
// they still have in flight before the CTA frees its tensor memory and returns.
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
  // for a whole warp whose lanes must stay together (tensor-memory loads and stores are warp-wide)
  __device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) const { return __all_sync(0xffffffffu, wait(bar, parity)); }
  __device__ __forceinline__ bool aborted() const { return *abort != 0; }
};

// After a wait ran out: the last fills of the ring (entries e - RING .. e - 1) and the Q tiles may still be in flight;
// a bulk copy that completes into the shared memory of a CTA that has left corrupts whoever runs there next.
__device__ __forceinline__ void drain_producer(const Bars& br, int e, int lane) {
  if (lane == 0) {
    (void)mv::mbar_wait_bounded(br.q_full, 0, 20000000ull);
    for (int k = 1; k <= min(e, RING); ++k)
      (void)mv::mbar_wait_bounded(br.kv_full + 8 * ((e - k) % RING), ((e - k) / RING) & 1, 20000000ull);
  }
  __syncwarp();
}

template <bool PAGED>
__device__ __forceinline__ void producer_warp(const mv::QTile& qt, const PrefillArgs& a, int h0, int kvh, uint32_t smem_base,
                                              const Bars& br, const Waiter& w, const CUtensorMap* tm_q, const CUtensorMap* tm_k,
                                              const CUtensorMap* tm_v) {
  const int lane = threadIdx.x & 31;
  if (!PAGED && lane != 0) return;  // flat form: one thread issues the few large boxes of a tile
  if (lane == 0) {
    mv::mbar_arrive_expect_tx(br.q_full, 2 * TILE_BYTES);
    for (int i = 0; i < 2; ++i)
      for (int h = 0; h < 2; ++h)
        mv::tma_load_2d(smem_base + OFF_Q + i * TILE_BYTES + h * (TILE_BYTES / 2), tm_q, (h0 + i) * D + h * 64, qt.q_start, br.q_full);
  }
  TileIter it(a.ranges + qt.range_begin, qt.range_count, qt.causal_base + qt.q_len - 1);
  int start, n, c, e = 0;  // e: ring entries issued so far
  if (PAGED) {
    // Paged form: a tile is gathered page by page, one 2 KB box per (page, column block).  Lane l < 16 owns page l / 2,
    // column block l % 2 of every tile; it reads its page id one tile ahead, so no load sits between two tiles.
    const int p = lane >> 1, h = lane & 1;
    auto page_of = [&](bool valid, int st_, int n_) {
      return (valid && lane < 16 && p < ((n_ + 15) >> 4)) ? __ldg(a.page_tab + it.pages + (st_ >> 4) + p) : -1;
    };
    bool more = it.next(start, n, c);
    int page = page_of(more, start, n);
    while (more) {
      int start2 = 0, n2 = 0, c2 = 0;
      const int n_pg = (n + 15) >> 4;
      const bool more2 = it.next(start2, n2, c2);
      const int page2 = page_of(more2, start2, n2);
      for (int kv = 0; kv < 2; ++kv, ++e) {
        const int slot = e % RING;
        const uint32_t bar = br.kv_full + 8 * slot;
        int go = 1;
        if (lane == 0) {
          go = w.wait(br.kv_empty + 8 * slot, ((e / RING) & 1) ^ 1) ? 1 : 0;
          if (go) mv::mbar_arrive_expect_tx(bar, uint32_t(n_pg) * 4096u);
        }
        if (!__shfl_sync(0xffffffffu, go, 0)) {
          drain_producer(br, e, lane);
          return;
        }
        if (page >= 0)
          mv::tma_load_2d(smem_base + OFF_RING + slot * TILE_BYTES + h * (TILE_BYTES / 2) + p * 2048, kv ? tm_v : tm_k, 0,
                          ((page * a.Hkv + kvh) * 2 + h) * 16, bar);
      }
      more = more2; start = start2; n = n2; c = c2; page = page2;
    }
    return;
  }
  while (it.next(start, n, c)) {
    for (int kv = 0; kv < 2; ++kv, ++e) {
      const int slot = e % RING;
      if (!w.wait(br.kv_empty + 8 * slot, ((e / RING) & 1) ^ 1)) {
        drain_producer(br, e, 0);
        return;
      }
      const uint32_t bar = br.kv_full + 8 * slot;
      mv::mbar_arrive_expect_tx(bar, TILE_BYTES);
      const uint32_t dst = smem_base + OFF_RING + slot * TILE_BYTES;
      for (int h = 0; h < 2; ++h) mv::tma_load_2d(dst + h * (TILE_BYTES / 2), kv ? tm_v : tm_k, kvh * D + h * 64, start, bar);
    }
  }
}

// S_i = Q_i K^T over the first n_cols keys of the tile (a multiple of 16): both operands K-major, eight k-steps.
// A descriptor's start address sits in its low bits in 16-byte units, so a k-step is one addition.
__device__ __forceinline__ void issue_qk(uint32_t s_tmem, uint64_t q_desc, uint64_t k_desc, int n_cols) {
  const uint32_t idesc = mv::um::idesc_bf16(BQ, n_cols, 0, 0);
  mv::um::mma_ss<false>(s_tmem, q_desc, k_desc, idesc);
#pragma unroll
  for (int k = 1; k < D / 16; ++k) {
    const uint32_t off = ((k >> 2) * (TILE_BYTES / 2) + (k & 3) * 32) >> 4;
    mv::um::mma_ss<true>(s_tmem, q_desc + off, k_desc + off, idesc);
  }
}
// O_i (+)= P_i V over the first k_steps * 16 keys: P from tensor memory (two bf16 per column), V MN-major
__device__ __forceinline__ void issue_pv(uint32_t o_tmem, uint32_t p_tmem, uint64_t v_desc, bool accumulate, int k_steps) {
  constexpr uint32_t idesc = mv::um::idesc_bf16(BQ, D, 0, 1);
  if (accumulate) mv::um::mma_ts<true>(o_tmem, p_tmem, v_desc, idesc);
  else mv::um::mma_ts<false>(o_tmem, p_tmem, v_desc, idesc);
#pragma unroll
  for (int k = 1; k < BK / 16; ++k)
    if (k < k_steps) mv::um::mma_ts<true>(o_tmem, p_tmem + k * 8, v_desc + uint32_t((k * 2048) >> 4), idesc);
}

template <bool PAGED>
__device__ __forceinline__ void mma_warp(const mv::QTile& qt, const PrefillArgs& a, unsigned char* smem, uint32_t smem_base, uint32_t tmem,
                                         const Bars& br, const Waiter& w) {
  // The whole warp walks the tiles and waits on the barriers; one elected lane issues the products and the commits.
  // Descriptors and tensor-memory addresses are then computed in warp-uniform code.
  const bool lead = mv::um::elect_one();
  TileIter it(a.ranges + qt.range_begin, qt.range_count, qt.causal_base + qt.q_len - 1);
  int start, n_cur, n_next = 0, c;
  if (!it.next(start, n_cur, c)) return;
  bool more = it.next(start, n_next, c);
  const uint64_t q0 = mv::um::smem_desc(smem_base + OFF_Q, 16, 1024), q1 = mv::um::smem_desc(smem_base + OFF_Q + TILE_BYTES, 16, 1024);
  const uint32_t s0 = tmem, s1 = tmem + 128, o0 = tmem + 256, o1 = tmem + 384;
  auto k_desc = [&](int e) { return mv::um::smem_desc(smem_base + OFF_RING + (e % RING) * TILE_BYTES, 16, 1024); };
  auto v_desc = [&](int e) { return mv::um::smem_desc(smem_base + OFF_RING + (e % RING) * TILE_BYTES, TILE_BYTES / 2, 1024); };
  bool ok = true;  // false once a wait ran out: nothing more is issued
  auto wait_full = [&](int e) { ok = ok && w.wait(br.kv_full + 8 * (e % RING), (e / RING) & 1); };
  auto drain = [&]() {  // products may still be in flight: they must have completed before the tensor memory is freed
    __syncwarp();
    if (lead) mv::um::commit(br.drained);
    (void)mv::mbar_wait_bounded(br.drained, 0, 20000000ull);
  };
  auto release = [&](int e) { if (lead) mv::um::commit(br.kv_empty + 8 * (e % RING)); };
  auto cols = [](int n) { return ((n + 15) >> 4) << 4; };  // score columns computed; the softmax groups mask the rest
  ok = w.wait(br.q_full, 0);
  wait_full(0);
  if (!ok) return drain();
  mv::um::fence_after();
  if (lead) {
    issue_qk(s0, q0, k_desc(0), cols(n_cur));
    mv::um::commit(br.s_full);
    issue_qk(s1, q1, k_desc(0), cols(n_cur));
    mv::um::commit(br.s_full + 8);
  }
  release(0);
  for (int j = 0;; ++j) {
    const int ev = 2 * j + 1, ek = 2 * j + 2;  // ring entries of V_j and K_{j+1}
    const int k_steps = (n_cur + 15) >> 4;
    wait_full(ev);
    if (!ok) break;
    if (PAGED && (n_cur & 15) && lead) {
      // the last page of a node is not full: its rows past the last key hold whatever the pool held; V must be zero
      // where P is zero, or 0 * NaN would poison O
      unsigned char* vt = smem + OFF_RING + (ev % RING) * TILE_BYTES;
      for (int rr = n_cur; rr < k_steps * 16; ++rr)
        for (int i = 0; i < 16; ++i)
          *reinterpret_cast<uint4*>(vt + (i >> 3) * (TILE_BYTES / 2) + rr * 128 + ((i & 7) << 4)) = make_uint4(0, 0, 0, 0);
      mv::fence_proxy_async();  // ordinary stores, read next by the tensor core
    }
    __syncwarp();  // the patch above is one lane's
    // the next K tile is waited for here, while P of head 0 is still being computed, not between the two products below:
    // that wait sat on head 0's chain (softmax -> P V -> next Q K^T -> softmax) in every step
    if (more) wait_full(ek);
    ok = ok && w.wait(br.p_full, j & 1);
    if (!ok) break;
    mv::um::fence_after();
    if (lead) {
      issue_pv(o0, s0, v_desc(ev), j > 0, k_steps);
      mv::um::commit(br.o_done);
      if (more) {
        issue_qk(s0, q0, k_desc(ek), cols(n_next));
        mv::um::commit(br.s_full);
      }
    }
    ok = w.wait(br.p_full + 8, j & 1);
    if (!ok) break;
    mv::um::fence_after();
    if (lead) {
      issue_pv(o1, s1, v_desc(ev), j > 0, k_steps);
      mv::um::commit(br.o_done + 8);
    }
    release(ev);
    if (!more) break;
    if (lead) {
      issue_qk(s1, q1, k_desc(ek), cols(n_next));
      mv::um::commit(br.s_full + 8);
    }
    release(ek);
    n_cur = n_next;
    more = it.next(start, n_next, c);
  }
  if (w.aborted()) drain();
}

// One softmax group = 128 threads = the 128 query rows of head `i` (0 or 1) of the CTA.
__device__ __forceinline__ void softmax_group(const mv::QTile& qt, const PrefillArgs& a, int i, int head, uint32_t tmem, const Bars& br,
                                              const Waiter& w) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = (warp & 3) * 32 + lane;                   // query row of the tile = tensor-memory lane
  const int qi = qt.q_start + r;                          // row of q and out
  const int qc = qt.causal_base + r;                      // the query's index in the causal range's key numbering
  const uint32_t lane_base = tmem + (uint32_t((warp & 3) * 32) << 16);
  const uint32_t s_t = lane_base + i * 128, o_t = lane_base + 256 + i * 128;
  const uint32_t s_full = br.s_full + 8 * i, p_full = br.p_full + 8 * i, o_done = br.o_done + 8 * i;
  TileIter it(a.ranges + qt.range_begin, qt.range_count, qt.causal_base + qt.q_len - 1);
  float m = -INFINITY, l = 0.f;  // running maximum (log2 units) and sum of this row
  int start, n, causal, j = 0;
  while (it.next(start, n, causal)) {
    if (!w.warp_wait(s_full, j & 1)) return;
    mv::um::fence_after();
    // all 128 columns are read: on a ragged tile the issuer computed only the leading ones, the rest holds an
    // older tile's scores and is masked below
    uint32_t s[BK];
#pragma unroll
    for (int c = 0; c < BK / 32; ++c) mv::um::ld32(s_t + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
    mv::um::wait_ld();
    // mask the ragged end of the range and, on diagonal tiles, keys after the query; row maximum of the raw
    // scores with four independent chains (the softmax scale is positive, so it commutes with the maximum)
    const bool need_mask = n < BK || (causal && start + BK - 1 > qt.causal_base);
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    if (!need_mask) {
#pragma unroll
      for (int c = 0; c < BK; c += 2) mx4[(c >> 1) & 3] = mv::max3(mx4[(c >> 1) & 3], __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
    } else {
      const int lim = causal ? min(n, qc - start + 1) : n;  // keys [0, lim) of the tile are visible to this row
#pragma unroll
      for (int c = 0; c < BK; ++c) {
        if (c >= lim) s[c] = __float_as_uint(-INFINITY);
        mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(s[c]));
      }
    }
    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
    // the row's reference maximum moves only when it would otherwise let P grow past 2^8
    const bool move = mx > m + RESCALE_THRESHOLD || (m == -INFINITY && mx > -INFINITY);
    if (j > 0 && __any_sync(0xffffffffu, move)) {
      const float f = (move && m != -INFINITY) ? mv::fast_exp2(m - mx) : 1.f;
      if (!w.warp_wait(o_done, (j - 1) & 1)) return;  // O_i holds tiles 0 .. j-1 and no product is writing it
      mv::um::fence_after();
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        mv::um::ld32(o_t + c * 32, o);
        mv::um::wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * f);
        mv::um::st32(o_t + c * 32, o);
      }
      l *= f;
    }
    if (move) m = mx;
    const float mref = (m == -INFINITY) ? 0.f : m;
    // packed-pair arithmetic: one FMA and one add per two scores, so that instruction issue does not pace the group
    const uint64_t scale2 = mv::pack_f32x2(a.scale_log2, a.scale_log2), nmref2 = mv::pack_f32x2(-mref, -mref);
    uint64_t sum2[4] = {0, 0, 0, 0};  // four independent chains of (even column, odd column) sums
#pragma unroll
    for (int c = 0; c < BK / 2; ++c) {  // P over S in place: columns 2c, 2c+1 -> packed column c
      float x0, x1;
      mv::unpack_f32x2(mv::fma_f32x2(mv::pack_f32x2(__uint_as_float(s[2 * c]), __uint_as_float(s[2 * c + 1])), scale2, nmref2), x0, x1);
      const float p0 = mv::fast_exp2(x0), p1 = mv::fast_exp2(x1);
      sum2[c & 3] = mv::add_f32x2(sum2[c & 3], mv::pack_f32x2(p0, p1));
      s[c] = mv::pack_bf16(p0, p1);
    }
    {
      float e, o;
      mv::unpack_f32x2(mv::add_f32x2(mv::add_f32x2(sum2[0], sum2[1]), mv::add_f32x2(sum2[2], sum2[3])), e, o);
      l += e + o;
    }
    mv::um::st32(s_t, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
    mv::um::st32(s_t + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
    mv::um::wait_st();
    mv::um::fence_before();
    mv::mbar_arrive(p_full);  // P_i (and a rescaled O_i) are in place for this tile's second product
    ++j;
  }
  if (j == 0) return;
  if (!w.warp_wait(o_done, (j - 1) & 1)) return;
  mv::um::fence_after();
  const float inv = 1.f / l;
  if (a.lse != nullptr && r < qt.q_len) a.lse[int64_t(qi) * a.Hq + head] = m + log2f(l);  // P_ij = 2^(scale_log2 * s_ij - lse)
  bf16* dst = a.out + (int64_t(qi) * a.Hq + head) * D;
#pragma unroll
  for (int c = 0; c < D / 32; ++c) {
    uint32_t o[32];
    mv::um::ld32(o_t + c * 32, o);
    mv::um::wait_ld();
    if (r < qt.q_len) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint4 v;
        v.x = mv::pack_bf16(__uint_as_float(o[8 * k]) * inv, __uint_as_float(o[8 * k + 1]) * inv);
        v.y = mv::pack_bf16(__uint_as_float(o[8 * k + 2]) * inv, __uint_as_float(o[8 * k + 3]) * inv);
        v.z = mv::pack_bf16(__uint_as_float(o[8 * k + 4]) * inv, __uint_as_float(o[8 * k + 5]) * inv);
        v.w = mv::pack_bf16(__uint_as_float(o[8 * k + 6]) * inv, __uint_as_float(o[8 * k + 7]) * inv);
        *reinterpret_cast<uint4*>(dst + c * 32 + k * 8) = v;
      }
    }
  }
}

template <bool PAGED>
__global__ void __launch_bounds__(NTHREADS, 1) prefill_tc_kernel(const PrefillArgs a, const __grid_constant__ CUtensorMap tm_q,
                                                                 const __grid_constant__ CUtensorMap tm_k,
                                                                 const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t smem_base = mv::smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 200);
  int* abort_flag = reinterpret_cast<int*>(smem + OFF_BAR + 208);
  Bars br;
  br.q_full = mv::smem_u32(&bars[0]);
  br.kv_full = mv::smem_u32(&bars[1]);
  br.kv_empty = mv::smem_u32(&bars[1 + RING]);
  br.s_full = mv::smem_u32(&bars[1 + 2 * RING]);
  br.p_full = mv::smem_u32(&bars[3 + 2 * RING]);
  br.o_done = mv::smem_u32(&bars[5 + 2 * RING]);
  br.drained = mv::smem_u32(&bars[7 + 2 * RING]);
  if ((smem_base & 1023u) != 0) {  // the swizzle pattern is anchored at 1024-byte boundaries
    if (tid == 0) atomicExch(a.status, int(MV_ERR_UNSUPPORTED));
    return;
  }
  if (tid == 0) {
    *abort_flag = 0;
    mv::mbar_init(br.q_full, 1);
    for (int i = 0; i < RING; ++i) {
      mv::mbar_init(br.kv_full + 8 * i, 1);
      mv::mbar_init(br.kv_empty + 8 * i, 1);  // one tcgen05.commit
    }
    for (int i = 0; i < 2; ++i) {
      mv::mbar_init(br.s_full + 8 * i, 1);    // one tcgen05.commit
      mv::mbar_init(br.p_full + 8 * i, 128);  // every thread of the softmax group
      mv::mbar_init(br.o_done + 8 * i, 1);    // one tcgen05.commit
    }
    mv::mbar_init(br.drained, 1);             // one tcgen05.commit, only after a wait ran out
    mv::mbar_fence_init();
    mv::fence_proxy_async();
  }
  if (warp == 2) {  // the whole tensor memory of the SM: S0 S1 O0 O1, 128 columns each
    mv::um::tmem_alloc(mv::smem_u32(tmem_slot), 512);
    mv::um::tmem_relinquish();
  }
  mv::um::fence_before();
  __syncthreads();
  mv::um::fence_after();
  const uint32_t tmem = *tmem_slot;
  // Which index of the grid is the fast one decides which CTAs are resident together.  Flat form: head pairs fast (the
  // resident CTAs cover all KV heads of a few query tiles, heaviest tiles first for every head): 1.78 -> 1.65 ms on the
  // 17K-token DAG.  Paged form: query tiles fast, so that the branches of a request, which share their prefix pages,
  // run together; the other order measures the same there (374 us either way).
  const mv::QTile qt = a.q_tiles[PAGED ? blockIdx.x : blockIdx.y];
  const int h0 = (PAGED ? blockIdx.y : blockIdx.x) * 2, kvh = h0 / a.G;
  Waiter w{abort_flag, a.status};
  if (warp < 4) {
    mv::um::reg_dec<PAGED ? 56 : 48>();
    if (warp == 0) producer_warp<PAGED>(qt, a, h0, kvh, smem_base, br, w, &tm_q, &tm_k, &tm_v);
    else if (warp == 1) mma_warp<PAGED>(qt, a, smem, smem_base, tmem, br, w);
  } else {
    mv::um::reg_inc<224>();
    const int i = (warp - 4) >> 2;
    softmax_group(qt, a, i, h0 + i, tmem, br, w);
  }
  mv::um::fence_before();
  __syncthreads();
  if (warp == 2) mv::um::tmem_dealloc(tmem, 512);
}

struct TcMaps {  // the tensor maps of one problem (pointers and token count rarely change between calls)
  CUtensorMap tm_q, tm_k, tm_v;
};

}  // namespace

namespace mv {
// Tensor-core prefill for head_dim 128 and an even group size; the caller has validated the arguments.
mv_status prefill_tc(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* out, float* lse,
                     cudaStream_t st) {
  static std::atomic<uint64_t> opted_in{0};  // per device
  if (!mv::opt_in_smem(prefill_tc_kernel<false>, SMEM_BYTES, opted_in)) return MV_ERR_CUDA;
  const int64_t T = P->stats.n_new_tokens;
  static thread_local mv::KeyedCache<TcMaps, 2> cache;
  const mv::TmapKey key{mv::current_device(), q, k, v, T, (int64_t(g->n_q_heads) << 32) | int64_t(g->n_kv_heads)};
  TcMaps* tcp = cache.find(key);
  if (!tcp) {
    tcp = cache.claim(key);
    if (!mv::make_tmap_bf16_2d(&tcp->tm_q, q, uint64_t(T), uint64_t(g->n_q_heads) * D, BQ) ||
        !mv::make_tmap_bf16_2d(&tcp->tm_k, k, uint64_t(T), uint64_t(g->n_kv_heads) * D, BK) ||
        !mv::make_tmap_bf16_2d(&tcp->tm_v, v, uint64_t(T), uint64_t(g->n_kv_heads) * D, BK)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  const TcMaps& tc = *tcp;
  PrefillArgs a;
  a.q_tiles = mv::table<mv::QTile>(P, P->layout.q_tiles);
  a.ranges = mv::table<mv::KvRange>(P, P->layout.kv_ranges);
  a.out = static_cast<bf16*>(out);
  a.lse = lse;
  a.status = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2;
  a.page_tab = nullptr;
  a.Hq = g->n_q_heads;
  a.Hkv = g->n_kv_heads;
  a.G = g->n_q_heads / g->n_kv_heads;
  a.scale_log2 = mv::softmax_scale(g) * 1.4426950408889634f;
  if (P->stats.n_q_tiles > 65535) return MV_ERR_UNSUPPORTED;  // the query tiles are the grid's y dimension
  dim3 grid(unsigned(g->n_q_heads / 2), unsigned(P->stats.n_q_tiles));
  prefill_tc_kernel<false><<<grid, NTHREADS, SMEM_BYTES, st>>>(a, tc.tm_q, tc.tm_k, tc.tm_v);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}

// Node append for head_dim 128 and an even group size: the paged form of the kernel over the plan's append tiles.
// q_rot [n_rows][n_q_heads][128]; k_pages / v_pages the page pools (the new tokens' K / V already written).  Writes
// the normalised output directly: no partials, no merge.  The caller has validated the arguments.
mv_status append_tc(const mv_plan* P, const mv_attn_geom* g, const void* q_rot, const void* k_pages, const void* v_pages, void* out,
                    cudaStream_t st) {
  static std::atomic<uint64_t> opted_in{0};  // per device
  if (!mv::opt_in_smem(prefill_tc_kernel<true>, SMEM_BYTES, opted_in)) return MV_ERR_CUDA;
  const int64_t T = P->stats.n_new_tokens;
  const int64_t pool_rows = g->num_pages * g->n_kv_heads * 2 * 16;  // 128-byte rows of a pool
  static thread_local mv::KeyedCache<TcMaps, 2> cache;
  const mv::TmapKey key{mv::current_device(), q_rot, k_pages, v_pages, T,
                        (pool_rows << 16) ^ (int64_t(g->n_q_heads) << 8) ^ int64_t(g->n_kv_heads)};
  TcMaps* tcp = cache.find(key);
  if (!tcp) {
    tcp = cache.claim(key);
    if (!mv::make_tmap_bf16_2d(&tcp->tm_q, q_rot, uint64_t(T), uint64_t(g->n_q_heads) * D, BQ) ||
        !mv::make_tmap_bf16_2d(&tcp->tm_k, k_pages, uint64_t(pool_rows), 64, 16) ||
        !mv::make_tmap_bf16_2d(&tcp->tm_v, v_pages, uint64_t(pool_rows), 64, 16)) {
      cache.drop();
      return MV_ERR_CUDA;
    }
  }
  const TcMaps& tc = *tcp;
  PrefillArgs a;
  a.q_tiles = mv::table<mv::QTile>(P, P->layout.q_tiles);
  a.ranges = mv::table<mv::KvRange>(P, P->layout.kv_ranges);
  a.page_tab = mv::table<int32_t>(P, P->layout.page_tab);
  a.out = static_cast<bf16*>(out);
  a.lse = nullptr;
  a.status = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2;
  a.Hq = g->n_q_heads;
  a.Hkv = g->n_kv_heads;
  a.G = g->n_q_heads / g->n_kv_heads;
  a.scale_log2 = mv::softmax_scale(g) * 1.4426950408889634f;
  dim3 grid(unsigned(P->stats.append_tiles), unsigned(g->n_q_heads / 2));
  prefill_tc_kernel<true><<<grid, NTHREADS, SMEM_BYTES, st>>>(a, tc.tm_q, tc.tm_k, tc.tm_v);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}
}  // namespace mv
