// Small most-recently-made cache of tensor maps (or anything else) keyed by what a tensor map depends on.
// Host-only, no CUDA types: the launchers instantiate it with their tensor-map bundles.
#pragma once
#include <cstdint>

namespace mv {

// A tensor map encodes device addresses and extents; the device index is part of the key as well, so that two devices
// driven from one process never share an entry (a pointer value alone does not say whose memory it is once a buffer
// has been freed on one device and another allocated at the same address on the next).
struct TmapKey {
  int device = -1;
  const void* a = nullptr;
  const void* b = nullptr;
  const void* c = nullptr;
  int64_t rows = 0;  // extent of the mapped matrices
  int64_t aux = 0;   // whatever else the maps depend on (head counts, box height, ...)
  bool operator==(const TmapKey& o) const {
    return device == o.device && a == o.a && b == o.b && c == o.c && rows == o.rows && aux == o.aux;
  }
};

template <typename Payload, int N>
class KeyedCache {
 public:
  // the cached payload of `key`, or nullptr
  Payload* find(const TmapKey& key) {
    for (int i = 0; i < N; ++i)
      if (used_[i] && keys_[i] == key) return &payload_[i];
    return nullptr;
  }
  // a slot for `key` (the oldest entry is replaced); the caller fills the payload, and calls drop() if that fails
  Payload* claim(const TmapKey& key) {
    const int i = next_;
    next_ = (next_ + 1) % N;
    keys_[i] = key;
    used_[i] = true;
    last_ = i;
    return &payload_[i];
  }
  void drop() {
    if (last_ >= 0) used_[last_] = false;
  }

 private:
  TmapKey keys_[N];
  bool used_[N] = {};
  Payload payload_[N];
  int next_ = 0, last_ = -1;
};

}  // namespace mv
