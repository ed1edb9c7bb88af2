// twist_plan: the shapes of a workload and a cache of encoded tensor maps.  A tensor map is a pure function of
// (base address, dimensions, strides, box, swizzle), so a cached one never goes stale; with a plan, the calls of
// a steady-state training loop (same buffers every step) encode nothing on the host.
#pragma once
#include <cuda.h>

#include <mutex>
#include <unordered_map>

#include "common.cuh"

struct twist_plan;

namespace twist {

struct MapKey {
  const void* ptr;
  unsigned long long dims[3], strides[2];
  unsigned box[3], swizzle, promotion;
  bool operator==(const MapKey& o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    const unsigned long long* w = reinterpret_cast<const unsigned long long*>(&k);
    unsigned long long h = 0x9E3779B97F4A7C15ull;
    for (size_t i = 0; i < sizeof(MapKey) / 8; ++i) h = (h ^ w[i]) * 0xBF58476D1CE4E5B9ull + (h >> 29);
    return (size_t)h;
  }
};
static_assert(sizeof(MapKey) % 8 == 0, "the key is hashed and compared as 64-bit words");

// The plan whose cache the calling thread's tensor-map encodes go through (null: encode every time).
twist_plan* active_plan();
// Makes `plan` (may be null) the calling thread's active plan for the lifetime of the object.
struct PlanScope {
  explicit PlanScope(twist_plan* plan);
  ~PlanScope();
  twist_plan* prev;
};
// Looks the key up in the active plan's cache.  Returns true and fills *map on a hit; on a miss the caller encodes
// and calls plan_store.
bool plan_lookup(const MapKey& key, CUtensorMap* map);
void plan_store(const MapKey& key, const CUtensorMap& map);

}  // namespace twist

struct twist_plan {
  twist_config cfg;
  std::mutex mu;
  std::unordered_map<twist::MapKey, CUtensorMap, twist::MapKeyHash> maps;
  unsigned long long hits = 0, misses = 0;
};
