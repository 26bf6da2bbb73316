// Optional NVTX ranges around the library's entry points (tracing aid; off unless the environment variable MV_NVTX is
// set to a non-empty value other than "0" when the library is first used).  Header-only NVTX: nothing is linked, and
// without a profiler attached a range costs one predictable branch.
#pragma once
#include <cstdlib>

#include <nvtx3/nvToolsExt.h>

namespace mv {
inline bool nvtx_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("MV_NVTX");
    return e && e[0] != '\0' && !(e[0] == '0' && e[1] == '\0');
  }();
  return on;
}
struct NvtxRange {
  bool on;
  explicit NvtxRange(const char* name) : on(nvtx_enabled()) {
    if (on) nvtxRangePushA(name);
  }
  ~NvtxRange() {
    if (on) nvtxRangePop();
  }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};
}  // namespace mv
