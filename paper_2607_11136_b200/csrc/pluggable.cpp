// Static-memory runtime as an allocator plug-in: the functions PyTorch's CUDAPluggableAllocator
// calls for every device allocation and release, with three modes.
//   pass-through  cudaMalloc / cudaFree (warm-up: one-time library workspaces get allocated here)
//   record        the same, and every request is logged with its lifetime on an event clock
//                 that ticks once per allocation: a tensor lives over [its own tick, the tick of
//                 the first allocation after its release)
//   replay        the k-th request of a step is answered with arena + offset[k] when its size
//                 equals the k-th recorded size (allocation = table lookup); releases of arena
//                 addresses do nothing.  A request that does not match falls back to cudaMalloc
//                 and is counted.
// Host code only; every entry point is serialised by one mutex.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "../../include/xema.h"
#include "kernels.h"

namespace {

struct Request {
  uint64_t bytes;        // as asked for
  uint32_t birth, death; // death == 0 while still live during recording
};

std::mutex g_mu;
int g_mode = XEMA_ALLOC_PASSTHROUGH;
std::vector<Request> g_rec;
std::unordered_map<void*, size_t> g_live;  // record mode: address -> index in g_rec
uint32_t g_clock = 0;

uint8_t* g_arena = nullptr;
uint64_t g_arena_bytes = 0;
std::vector<uint64_t> g_offsets;
size_t g_next = 0;
uint64_t g_served = 0, g_fallback = 0, g_steps = 0;

inline uint64_t round256(uint64_t n) { return (n + 255u) & ~uint64_t(255); }

void* device_malloc(size_t size) {
  void* p = nullptr;
  if (size == 0) return nullptr;
  cudaError_t e = cudaMalloc(&p, size);
  if (e != cudaSuccess) {
    xema::set_last_cuda_error((int)e);
    return nullptr;
  }
  return p;
}

}  // namespace

extern "C" {

void* xema_pluggable_malloc(ptrdiff_t size, int device, void* stream) {
  (void)device;
  (void)stream;
  std::lock_guard<std::mutex> lock(g_mu);
  if (size <= 0) return nullptr;  // empty requests carry no memory and are not part of the plan
  if (g_mode == XEMA_ALLOC_REPLAY) {
    if (g_next < g_rec.size() && g_rec[g_next].bytes == (uint64_t)size && g_arena) {
      void* p = g_arena + g_offsets[g_next];
      ++g_next;
      ++g_served;
      return p;
    }
    ++g_fallback;
    return device_malloc((size_t)size);
  }
  void* p = device_malloc((size_t)size);
  if (g_mode == XEMA_ALLOC_RECORD && p) {
    g_live[p] = g_rec.size();
    g_rec.push_back(Request{(uint64_t)size, g_clock, 0});
    ++g_clock;
  }
  return p;
}

void xema_pluggable_free(void* ptr, ptrdiff_t size, int device, void* stream) {
  (void)size;
  (void)device;
  (void)stream;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!ptr) return;
  const uint8_t* b = static_cast<const uint8_t*>(ptr);
  if (g_arena && b >= g_arena && b < g_arena + g_arena_bytes) return;  // planned memory: nothing to do
  auto it = g_live.find(ptr);
  if (it != g_live.end()) {
    g_rec[it->second].death = g_clock > g_rec[it->second].birth ? g_clock : g_rec[it->second].birth + 1;
    g_live.erase(it);
  }
  cudaError_t e = cudaFree(ptr);
  if (e != cudaSuccess) xema::set_last_cuda_error((int)e);
}

int xema_pluggable_mode(int mode) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (mode != XEMA_ALLOC_PASSTHROUGH && mode != XEMA_ALLOC_RECORD && mode != XEMA_ALLOC_REPLAY) return XEMA_EINVAL;
  if (mode == XEMA_ALLOC_RECORD) {
    g_rec.clear();
    g_live.clear();
    g_clock = 0;
    g_offsets.clear();
    g_arena = nullptr;
    g_arena_bytes = 0;
  }
  if (mode == XEMA_ALLOC_REPLAY) {
    if (!g_arena || g_offsets.size() != g_rec.size()) return XEMA_ESTATE;
    g_next = 0;
  }
  if (g_mode == XEMA_ALLOC_RECORD && mode != XEMA_ALLOC_RECORD) {
    // requests still live when recording stops live to the end of the step
    for (auto& kv : g_live) g_rec[kv.second].death = g_clock > g_rec[kv.second].birth ? g_clock : g_rec[kv.second].birth + 1;
    g_live.clear();
  }
  g_mode = mode;
  return XEMA_OK;
}

int xema_pluggable_recorded(xema_tensor* out, size_t cap, size_t* n_requests, uint32_t* n_events) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_mode == XEMA_ALLOC_RECORD) return XEMA_ESTATE;
  if (n_requests) *n_requests = g_rec.size();
  if (n_events) *n_events = g_clock;
  if (!out || cap < g_rec.size()) return XEMA_ENOSPC;
  for (size_t i = 0; i < g_rec.size(); ++i) {
    xema_tensor t;
    std::memset(&t, 0, sizeof(t));
    std::snprintf(t.name, sizeof(t.name), "req%zu", i);
    t.kind = XEMA_KIND_WORKSPACE;
    t.block = -1;
    t.chunk = -1;
    t.bytes = round256(g_rec[i].bytes ? g_rec[i].bytes : 1);
    t.birth = g_rec[i].birth;
    t.death = g_rec[i].death;
    out[i] = t;
  }
  return XEMA_OK;
}

int xema_pluggable_set_plan(void* arena_dev, uint64_t arena_bytes, const uint64_t* offsets, size_t n) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_mode != XEMA_ALLOC_PASSTHROUGH) return XEMA_ESTATE;
  if (!arena_dev || !offsets || n != g_rec.size()) return XEMA_EINVAL;
  if (reinterpret_cast<uintptr_t>(arena_dev) & 255) return XEMA_EALIGN;
  for (size_t i = 0; i < n; ++i) {
    if (offsets[i] & 255) return XEMA_EALIGN;
    if (offsets[i] + round256(g_rec[i].bytes ? g_rec[i].bytes : 1) > arena_bytes) return XEMA_ENOSPC;
  }
  g_arena = static_cast<uint8_t*>(arena_dev);
  g_arena_bytes = arena_bytes;
  g_offsets.assign(offsets, offsets + n);
  g_next = 0;
  return XEMA_OK;
}

int xema_pluggable_step_begin(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_mode != XEMA_ALLOC_REPLAY) return XEMA_ESTATE;
  g_next = 0;
  ++g_steps;
  return XEMA_OK;
}

int xema_pluggable_stats(uint64_t* served, uint64_t* fallback, uint64_t* next_index) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (served) *served = g_served;
  if (fallback) *fallback = g_fallback;
  if (next_index) *next_index = g_next;
  return XEMA_OK;
}

}  // extern "C"
