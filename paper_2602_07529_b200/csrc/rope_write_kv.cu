// RoPE with adaptive position indices fused into the paged KV-cache write.
//
// For every new token t: rotate q and k by the position index the planner assigned (Sec. 4.2: positions
// continue from the fork / join point), store k and v at the token's pool slot and emit the rotated q.
// P(i) of Eq. 2 is taken to be the rotary embedding with half-split pairing: element i pairs with
// i + d/2 and is rotated by pos * base^(-2i/d).  The angle and its reduction to the first octant are evaluated
// in double precision (positions reach ~2e4, where a float angle alone would already be off by ~1e-3 rad);
// cosine and sine of the reduced angle and the rotation are float.
//
// HBM-bound elementwise kernel: one or four tokens per CTA, 16-byte vector loads and stores, the cos/sin
// rows of the CTA's tokens are computed once into shared memory and reused by all heads.
#include "common.cuh"
#include "trace.h"

namespace {

template <typename T>
struct Vec16;  // 16 bytes of T
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&x)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
  __device__ static void store(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&x)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      x[2 * i] = f.x;
      x[2 * i + 1] = f.y;
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float (&x)[8]) {
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = v;
  }
};

// N floats times inv -> N bytes of 8-bit floats (N = 4 or 8), one vector store
template <int N>
__device__ __forceinline__ void store_e4m3(unsigned char* dst, const float (&x)[N], float inv) {
  uint32_t w[N / 4];
#pragma unroll
  for (int i = 0; i < N / 4; ++i)
    w[i] = mv::pack_e4m3x2(x[4 * i] * inv, x[4 * i + 1] * inv) | (mv::pack_e4m3x2(x[4 * i + 2] * inv, x[4 * i + 3] * inv) << 16);
  if (N == 8) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[N / 4 - 1]);
  else *reinterpret_cast<uint32_t*>(dst) = w[0];
}

// theta_i = base^(-2i/d) for i < d/2, evaluated once per launch on the host in double precision
struct ThetaTable {
  double theta[64];
};

// cos and sin of pos * theta.  The angle and its reduction to [-pi/4, pi/4] (two-term Cody-Waite with a 53-bit and a
// residual piece of pi/2; pos * theta stays below 2^25, so k * PIO2_HI is exact to well under 1e-12) are double
// precision; the reduced angle is rounded to float and its cosine and sine come from the accurate float routine
// (no fast-math intrinsics), so both agree with the double-precision values to within two units in the last place
// of a float.  Six double-precision instructions per (token, i) instead of a double-precision sincos: with the
// latter the arithmetic, not HBM, bounded the kernel at prefill sizes.
__device__ __forceinline__ void rope_cos_sin(int pos, double theta, float& c, float& s) {
  constexpr double TWO_OVER_PI = 0.63661977236758134308;
  constexpr double PIO2_HI = 1.57079632679489655800e+00;  // pi/2 rounded to double
  constexpr double PIO2_LO = 6.12323399573676603587e-17;  // pi/2 - PIO2_HI
  const double a = double(pos) * theta;
  const double kf = rint(a * TWO_OVER_PI);
  double r = fma(-kf, PIO2_HI, a);
  r = fma(-kf, PIO2_LO, r);
  float sr, cr;
  sincosf(float(r), &sr, &cr);
  const int k = int(kf) & 3;  // quadrant: angle = r + k * pi/2
  const float ss = (k & 1) ? cr : sr, cc = (k & 1) ? sr : cr;
  s = (k & 2) ? -ss : ss;
  c = ((k + 1) & 2) ? -cc : cc;
}

// TPC tokens per CTA.  Phase 1: the CTA's (token, i) pairs get their cos / sin, one pair per thread, while the first
// loads of phase 2 are already in flight; phase 2: 16-byte units of q, k (rotated) and v (copied) stream through.
// FP8: the pools hold 8-bit floats (4 exponent, 3 mantissa bits), [pages][KV heads][16 tokens][head_dim bytes]; a value is
// stored as round(x / scale[head]), saturating (kv_scale = the K scales of all heads, then the V scales).
template <typename T, int D, int TPC, bool FP8 = false>
// q_rot may be q and k_rot may be k (rotation in place), so those four carry no __restrict__.
__global__ void __launch_bounds__(256) rope_write_kv_kernel(const T* q, const T* k, const T* __restrict__ v, T* q_rot, T* k_rot,
                                                            T* __restrict__ k_pages,
                                                            T* __restrict__ v_pages, const int32_t* __restrict__ pos_id,
                                                            const int64_t* __restrict__ slot, int n_tok, int Hq, int Hkv,
                                                            const __grid_constant__ ThetaTable tt, const float* __restrict__ kv_scale = nullptr,
                                                            int64_t num_pages_dbg = 0, int32_t* status_dbg = nullptr) {
  constexpr int HALF = D / 2;
  constexpr int N = Vec16<T>::N;
  constexpr int CH = HALF / N;  // 16-byte chunks per half head
  constexpr int VCH = D / N;    // 16-byte chunks per head
  __shared__ float cs[TPC][HALF], sn[TPC][HALF];
  __shared__ int64_t s_slot[TPC];
  const int t0 = blockIdx.x * TPC;
  // a kernel launched behind this one with programmatic stream serialisation (the decode attention kernel) may become
  // resident and run its set-up now; it waits for this grid's completion before it reads what is written here
  mv::grid_dependency_launch_dependents();
  const int n_here = min(TPC, n_tok - t0);
  if (n_here <= 0) return;
  for (int x = threadIdx.x; x < n_here * HALF; x += blockDim.x) {
    const int tl = x / HALF, i = x % HALF;
    float c, s;
    rope_cos_sin(__ldg(pos_id + t0 + tl), tt.theta[i], c, s);
    cs[tl][i] = c;
    sn[tl][i] = s;
    if (i == 0) {
      int64_t sl = __ldg(slot + t0 + tl);
#ifdef MV_DEBUG
      // debug build: a slot outside the pool sets the status word and the token's cache write is skipped
      if ((k_pages != nullptr || v_pages != nullptr) && (sl < 0 || (sl >> 4) >= num_pages_dbg)) {
        atomicExch(status_dbg, int(MV_ERR_INVALID_ARG));
        sl = -1;
      }
#endif
      s_slot[tl] = sl;
    }
  }
  __syncthreads();
  const int n_q_units = q ? Hq * CH : 0;
  const int n_k_units = Hkv * CH;
  const int n_v_units = v_pages ? Hkv * VCH : 0;
  const int per_tok = n_q_units + n_k_units + n_v_units;
  for (int x = threadIdx.x; x < n_here * per_tok; x += blockDim.x) {
    const int tl = x / per_tok, u = x % per_tok;
    const int64_t t = t0 + tl;
    const int64_t sl = s_slot[tl];
#ifdef MV_DEBUG
    const bool pool_ok = sl >= 0;
#else
    constexpr bool pool_ok = true;
#endif
    const int64_t page = sl >> 4, off = sl & 15;
    if (u >= n_q_units + n_k_units) {  // v is stored unrotated
      const int uu = u - n_q_units - n_k_units;
      const int h = uu / VCH, c = uu % VCH;
      const int e = c * N;
      if (!pool_ok) continue;
      if (FP8) {
        float x[N];
        Vec16<T>::load(v + (t * Hkv + h) * D + e, x);
        const float inv = 1.f / __ldg(kv_scale + Hkv + h);
        unsigned char* dst = reinterpret_cast<unsigned char*>(v_pages) + (page * Hkv + h) * (16 * D) + off * D + e;
        store_e4m3<N>(dst, x, inv);
        continue;
      }
      const uint4 val = *reinterpret_cast<const uint4*>(v + (t * Hkv + h) * D + e);
      *reinterpret_cast<uint4*>(v_pages + (page * Hkv + h) * (16 * D) + (e >> 6) * 1024 + off * 64 + (e & 63)) = val;
      continue;
    }
    const bool is_q = u < n_q_units;
    const int uu = is_q ? u : u - n_q_units;
    const int h = uu / CH, c = uu % CH;
    const T* src = is_q ? q + (t * Hq + h) * D : k + (t * Hkv + h) * D;
    float lo[N], hi[N], olo[N], ohi[N];
    Vec16<T>::load(src + c * N, lo);
    Vec16<T>::load(src + HALF + c * N, hi);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float cc = cs[tl][c * N + i], ss = sn[tl][c * N + i];
      olo[i] = lo[i] * cc - hi[i] * ss;
      ohi[i] = hi[i] * cc + lo[i] * ss;
    }
    if (is_q) {
      T* dst = q_rot + (t * Hq + h) * D;
      Vec16<T>::store(dst + c * N, olo);
      Vec16<T>::store(dst + HALF + c * N, ohi);
      continue;
    }
    if (FP8 && pool_ok) {
      const float inv = 1.f / __ldg(kv_scale + h);
      unsigned char* dst = reinterpret_cast<unsigned char*>(k_pages) + (page * Hkv + h) * (16 * D) + off * D;
      store_e4m3<N>(dst + c * N, olo, inv);
      store_e4m3<N>(dst + HALF + c * N, ohi, inv);
    } else if (!FP8 && k_pages != nullptr && pool_ok) {
      // pool element (page, head, token, e) lives in 64-element column block e / 64 of the (page, head) block
      T* dst = k_pages + (page * Hkv + h) * (16 * D) + off * 64;
      const int e0 = c * N, e1 = HALF + c * N;
      Vec16<T>::store(dst + (e0 >> 6) * 1024 + (e0 & 63), olo);
      Vec16<T>::store(dst + (e1 >> 6) * 1024 + (e1 & 63), ohi);
    }
    if (k_rot != nullptr) {
      T* dst2 = k_rot + (t * Hkv + h) * D;
      Vec16<T>::store(dst2 + c * N, olo);
      Vec16<T>::store(dst2 + HALF + c * N, ohi);
    }
  }
}

inline int32_t* dbg_status(const mv_plan* P) { return const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2; }

template <typename T, int D>
mv_status launch_d(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* q_rot,
                   void* k_rot, void* k_pages, void* v_pages, cudaStream_t st) {
  const int n = int(P->stats.n_new_tokens);
  const int32_t* pos = mv::table<int32_t>(P, P->layout.pos_id);
  const int64_t* slot = mv::table<int64_t>(P, P->layout.slot);
  ThetaTable tt{};
  const double c = -2.0 * log2(g->rope_base) / double(D);
  for (int i = 0; i < D / 2; ++i) tt.theta[i] = exp2(double(i) * c);  // base^(-2i/d)
  // few tokens (a decode step): one token per CTA spreads them over the SMs; many (prefill, history): four per CTA
  // amortise the set-up and keep more 16-byte units in flight per thread
  if (n < 2048)
    rope_write_kv_kernel<T, D, 1><<<n, 256, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (T*)q_rot, (T*)k_rot, (T*)k_pages,
                                                     (T*)v_pages, pos, slot, n, g->n_q_heads, g->n_kv_heads, tt, nullptr, g->num_pages, dbg_status(P));
  else
    rope_write_kv_kernel<T, D, 4><<<(n + 3) / 4, 256, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (T*)q_rot, (T*)k_rot,
                                                               (T*)k_pages, (T*)v_pages, pos, slot, n, g->n_q_heads,
                                                               g->n_kv_heads, tt, nullptr, g->num_pages, dbg_status(P));
  mv::g_launches++;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  return MV_OK;
}

template <typename T>
mv_status launch(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* q_rot,
                 void* k_rot, void* k_pages, void* v_pages, cudaStream_t st) {
  return g->head_dim == 128 ? launch_d<T, 128>(P, g, q, k, v, q_rot, k_rot, k_pages, v_pages, st)
                            : launch_d<T, 64>(P, g, q, k, v, q_rot, k_rot, k_pages, v_pages, st);
}

template <int TPC>
void launch_fp8(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* q_rot, void* k_pages8,
                void* v_pages8, const float* kv_scale, int n, cudaStream_t st) {
  using T = __nv_bfloat16;
  constexpr int D = 128;
  ThetaTable tt{};
  const double c = -2.0 * log2(g->rope_base) / double(D);
  for (int i = 0; i < D / 2; ++i) tt.theta[i] = exp2(double(i) * c);
  rope_write_kv_kernel<T, D, TPC, true><<<(n + TPC - 1) / TPC, 256, 0, st>>>(
      (const T*)q, (const T*)k, (const T*)v, (T*)q_rot, nullptr, (T*)k_pages8, (T*)v_pages8, mv::table<int32_t>(P, P->layout.pos_id),
      mv::table<int64_t>(P, P->layout.slot), n, g->n_q_heads, g->n_kv_heads, tt, kv_scale, g->num_pages, dbg_status(P));
}

}  // namespace

extern "C" mv_status mv_rope_write_kv_fp8(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v,
                                          void* q_rot, void* k_pages8, void* v_pages8, const float* kv_scale, void* cuda_stream) {
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (g->dtype != MV_BF16 || g->head_dim != 128) return MV_ERR_UNSUPPORTED;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  if (P->stats.n_new_tokens == 0) return MV_OK;
  if (!k || !v || !k_pages8 || !v_pages8 || !kv_scale) return MV_ERR_INVALID_ARG;
  if ((q == nullptr) != (q_rot == nullptr)) return MV_ERR_INVALID_ARG;
  if (P->stats.max_page_id >= g->num_pages || g->rope_base <= 0.0) return MV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int n = int(P->stats.n_new_tokens);
  if (n < 2048) launch_fp8<1>(P, g, q, k, v, q_rot, k_pages8, v_pages8, kv_scale, n, s);
  else launch_fp8<4>(P, g, q, k, v, q_rot, k_pages8, v_pages8, kv_scale, n, s);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}

extern "C" mv_status mv_rope_write_kv(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k,
                                      const void* v, void* q_rot, void* k_rot, void* k_pages, void* v_pages,
                                      void* cuda_stream) {
  mv::NvtxRange nvtx_range("mv_rope_write_kv");
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  mv_status st = mv::check_geom(g);
  if (st != MV_OK) return st;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  if (P->stats.n_new_tokens == 0) return MV_OK;
  if (!k || !v) return MV_ERR_INVALID_ARG;
  if ((k_pages == nullptr) != (v_pages == nullptr)) return MV_ERR_INVALID_ARG;
  if (!k_pages && !k_rot) return MV_ERR_INVALID_ARG;
  if ((q == nullptr) != (q_rot == nullptr)) return MV_ERR_INVALID_ARG;
  if (k_pages && P->stats.max_page_id >= g->num_pages) return MV_ERR_INVALID_ARG;
  if (g->rope_base <= 0.0) return MV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  return g->dtype == MV_BF16 ? launch<__nv_bfloat16>(P, g, q, k, v, q_rot, k_rot, k_pages, v_pages, s)
                             : launch<float>(P, g, q, k, v, q_rot, k_rot, k_pages, v_pages, s);
}
