// RoPE with adaptive position indices fused into the paged KV-cache write.
//
// For every new token t: rotate q and k by the position index the planner assigned (Sec. 4.2: positions
// continue from the fork / join point), store k and v at the token's pool slot and emit the rotated q.
// P(i) of Eq. 2 is taken to be the rotary embedding with half-split pairing: element i pairs with
// i + d/2 and is rotated by pos * base^(-2i/d).  The angle, its cosine and sine are evaluated in double
// precision and rounded to float (positions reach ~2e4, where a float angle alone would already be off
// by ~1e-3 rad); the rotation is float.
//
// HBM-bound elementwise kernel: one CTA per token, 16-byte vector loads and stores, the cos/sin row of
// the token is computed once into shared memory and reused by all heads.
#include "common.cuh"

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

template <typename T, int D>
__global__ void __launch_bounds__(128) rope_write_kv_kernel(const T* q, const T* k,
                                                            const T* v, T* q_rot,
                                                            T* k_rot, T* k_pages,
                                                            T* v_pages,
                                                            const int32_t* pos_id,
                                                            const int64_t* slot, int n_tok, int Hq,
                                                            int Hkv, double neg_log2_base_2_over_d) {
  constexpr int HALF = D / 2;
  constexpr int N = Vec16<T>::N;
  constexpr int CH = HALF / N;  // 16-byte chunks per half head
  __shared__ float cs[HALF], sn[HALF];
  const int t = blockIdx.x;
  // a kernel launched behind this one with programmatic stream serialisation (the decode attention kernel) may become
  // resident and run its set-up now; it waits for this grid's completion before it reads what is written here
  mv::grid_dependency_launch_dependents();
  if (t >= n_tok) return;
  const int pos = pos_id[t];
  const int64_t sl = slot[t];
  for (int i = threadIdx.x; i < HALF; i += blockDim.x) {
    // theta_i = base^(-2i/d) = 2^(-(2i/d) * log2(base)), in double
    const double theta = exp2(double(i) * neg_log2_base_2_over_d);
    double s, c;
    sincos(double(pos) * theta, &s, &c);
    cs[i] = float(c);
    sn[i] = float(s);
  }
  __syncthreads();
  const int64_t page = sl >> 4, off = sl & 15;
  const int n_q_units = q ? Hq * CH : 0;
  const int n_k_units = Hkv * CH;
  // rotated q and k
  for (int u = threadIdx.x; u < n_q_units + n_k_units; u += blockDim.x) {
    const bool is_q = u < n_q_units;
    const int uu = is_q ? u : u - n_q_units;
    const int h = uu / CH, c = uu % CH;
    const T* src = is_q ? q + (int64_t(t) * Hq + h) * D : k + (int64_t(t) * Hkv + h) * D;
    // pool element (page, head, token, c) lives in 64-element column block c / 64 of the (page, head) block
    T* dst = is_q ? q_rot + (int64_t(t) * Hq + h) * D : k_pages + (page * Hkv + h) * (16 * D) + off * 64;
    T* dst2 = is_q ? nullptr : k_rot + (int64_t(t) * Hkv + h) * D;
    const bool w1 = is_q || k_pages != nullptr, w2 = !is_q && k_rot != nullptr;
    float lo[N], hi[N], olo[N], ohi[N];
    Vec16<T>::load(src + c * N, lo);
    Vec16<T>::load(src + HALF + c * N, hi);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float cc = cs[c * N + i], ss = sn[c * N + i];
      olo[i] = lo[i] * cc - hi[i] * ss;
      ohi[i] = hi[i] * cc + lo[i] * ss;
    }
    if (w1) {
      if (is_q) {
        Vec16<T>::store(dst + c * N, olo);
        Vec16<T>::store(dst + HALF + c * N, ohi);
      } else {
        const int e0 = c * N, e1 = HALF + c * N;  // element indices inside the head vector
        Vec16<T>::store(dst + (e0 >> 6) * 1024 + (e0 & 63), olo);
        Vec16<T>::store(dst + (e1 >> 6) * 1024 + (e1 & 63), ohi);
      }
    }
    if (w2) {
      Vec16<T>::store(dst2 + c * N, olo);
      Vec16<T>::store(dst2 + HALF + c * N, ohi);
    }
  }
  if (v_pages == nullptr) return;
  // v is stored unrotated
  constexpr int VCH = D / N;
  for (int u = threadIdx.x; u < Hkv * VCH; u += blockDim.x) {
    const int h = u / VCH, c = u % VCH;
    const uint4 val = *reinterpret_cast<const uint4*>(v + (int64_t(t) * Hkv + h) * D + c * N);
    const int e = c * N;
    *reinterpret_cast<uint4*>(v_pages + (page * Hkv + h) * (16 * D) + (e >> 6) * 1024 + off * 64 + (e & 63)) = val;
  }
}

template <typename T>
mv_status launch(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k, const void* v, void* q_rot,
                 void* k_rot, void* k_pages, void* v_pages, cudaStream_t st) {
  const int n = int(P->stats.n_new_tokens);
  const int32_t* pos = mv::table<int32_t>(P, P->layout.pos_id);
  const int64_t* slot = mv::table<int64_t>(P, P->layout.slot);
  const double c = -2.0 * log2(g->rope_base) / double(g->head_dim);
  if (g->head_dim == 128)
    rope_write_kv_kernel<T, 128><<<n, 128, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (T*)q_rot, (T*)k_rot,
                                                    (T*)k_pages, (T*)v_pages, pos, slot, n, g->n_q_heads,
                                                    g->n_kv_heads, c);
  else
    rope_write_kv_kernel<T, 64><<<n, 128, 0, st>>>((const T*)q, (const T*)k, (const T*)v, (T*)q_rot, (T*)k_rot,
                                                   (T*)k_pages, (T*)v_pages, pos, slot, n, g->n_q_heads,
                                                   g->n_kv_heads, c);
  mv::g_launches++;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  return MV_OK;
}

}  // namespace

extern "C" mv_status mv_rope_write_kv(const mv_plan* P, const mv_attn_geom* g, const void* q, const void* k,
                                      const void* v, void* q_rot, void* k_rot, void* k_pages, void* v_pages,
                                      void* cuda_stream) {
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
