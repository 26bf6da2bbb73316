// Self-test entry points of the library (diagnostics; nothing of the attention path runs here).
#include "common.cuh"
#include "tmap_cache.h"

namespace {

// One thread waits, with the library's bounded wait, on an mbarrier that nobody ever arrives at.  No copy and no
// tensor-core product is outstanding, so when the wait runs out the kernel has nothing to drain: it records
// MV_ERR_TIMEOUT in the status word and returns, and the context stays usable.
__global__ void bounded_wait_probe_kernel(int32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t never;
  const uint32_t bar = mv::smem_u32(&never);
  if (threadIdx.x == 0) {
    mv::mbar_init(bar, 1);
    mv::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0 && !mv::mbar_wait_bounded(bar, 0, limit_ns)) atomicExch(status, int(MV_ERR_TIMEOUT));
}

}  // namespace

extern "C" mv_status mv_selftest_bounded_wait(const mv_plan* P, uint64_t limit_ns, void* cuda_stream) {
  if (!P || !P->valid) return MV_ERR_INVALID_ARG;
  if (!P->device_buf) return MV_ERR_WORKSPACE;
  if (limit_ns == 0 || limit_ns > 100000000ull) return MV_ERR_INVALID_ARG;  // at most a tenth of a second
  int32_t* status = const_cast<int32_t*>(mv::table<int32_t>(P, P->layout.sched)) + 2;
  bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(status, limit_ns);
  mv::g_launches++;
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}

// The lookup the launchers use for their tensor maps, on an instance of its own with an integer payload: returns 1 if
// the key was already cached, 0 if it was not (and is now), so that the keying can be checked without a device.
extern "C" int32_t mv_selftest_tmap_cache(int32_t device, const void* a, const void* b, const void* c, int64_t rows, int64_t aux,
                                          int32_t reset) {
  static mv::KeyedCache<int, 4> cache;
  if (reset) cache = mv::KeyedCache<int, 4>();
  const mv::TmapKey key{device, a, b, c, rows, aux};
  if (cache.find(key)) return 1;
  *cache.claim(key) = 1;
  return 0;
}
