// xema_block_forward_static: the block forward for callers that cannot allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off the table -- inside a region that must
// not synchronise the device (an allocation may), in a process whose device memory is fully
// handed out to a pool the caller does not own, or in a plug-in that is only ever given its
// input and output buffers.  Such a caller has nowhere to put the block's intermediates (the
// arena that xema_block_forward expects from its caller), so this variant keeps them in a
// fixed array that is part of the library image.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "../../include/xema.h"
#include "kernels.h"

// Scratch for every intermediate of one small block.  It is allocated by the CUDA runtime when
// the library is loaded on a device and stays allocated until the process exits.
static __device__ __align__(256) unsigned char g_static_arena[XEMA_STATIC_ARENA_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_static_arena per device ordinal.  In host code the symbol's name is only
// a handle; the address a kernel can use has to be asked for, once per device.  Atomic so that
// host threads calling in at the same time either see the address or look it up themselves (the
// lookup is idempotent).  A cudaDeviceReset() by the caller invalidates the cached address.
std::atomic<unsigned char*> g_arena_ptr[kMaxDevices] = {};

int static_arena_for_current_device(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    xema::set_last_cuda_error((int)(e != cudaSuccess ? e : cudaErrorInvalidDevice));
    return XEMA_ECUDA;
  }
  unsigned char* cached = g_arena_ptr[dev].load(std::memory_order_acquire);
  if (!cached) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_arena);
    if (e != cudaSuccess || !p) {
      xema::set_last_cuda_error((int)(e != cudaSuccess ? e : cudaErrorInvalidSymbol));
      return XEMA_ECUDA;
    }
    cached = static_cast<unsigned char*>(p);
    g_arena_ptr[dev].store(cached, std::memory_order_release);
  }
  *out = cached;
  return XEMA_OK;
}

}  // namespace

extern "C" int xema_block_forward_static(const xema_config* cfg, int32_t chunks, const xema_block_weights* weights,
                                         const float* rope_dev, const void* hid_in_dev, const void* temb_dev,
                                         void* hid_out_dev, void* status_dev, void* stream) {
  if (!cfg || !weights || !rope_dev || !hid_in_dev || !temb_dev || !hid_out_dev) return XEMA_EINVAL;
  if (cfg->n_blocks != 1) return XEMA_EINVAL;
  xema_plan* plan = nullptr;
  int rc = xema_plan_create(cfg, chunks, &plan);          // host memory only
  if (rc) return rc;
  uint64_t peak = 0;
  xema_plan_info(plan, &peak, nullptr, nullptr, nullptr, nullptr);
  if (peak > XEMA_STATIC_ARENA_BYTES) {
    xema_plan_destroy(plan);
    return XEMA_ENOSPC;                                   // template too large for the fixed scratch
  }
  unsigned char* arena = nullptr;
  rc = static_arena_for_current_device(&arena);
  if (!rc) rc = xema_plan_bind(plan, arena, XEMA_STATIC_ARENA_BYTES, weights, rope_dev, status_dev);
  uint64_t off_in = 0, off_temb = 0, off_out = 0, bytes_in = 0, bytes_temb = 0, bytes_out = 0;
  if (!rc) rc = xema_plan_tensor(plan, "hid0", &off_in, &bytes_in);
  if (!rc) rc = xema_plan_tensor(plan, "temb", &off_temb, &bytes_temb);
  if (!rc) rc = xema_plan_tensor(plan, "hid1", &off_out, &bytes_out);
  if (!rc) {
    // exact sizes (the planned sizes are rounded up to 256 bytes; the caller's buffers are not)
    const uint64_t S = (uint64_t)cfg->s_text + (uint64_t)cfg->grid_t * cfg->grid_h * cfg->grid_w;
    const size_t hid_bytes = (size_t)2 * cfg->batch * S * cfg->hidden;
    const size_t temb_bytes = (size_t)2 * cfg->batch * cfg->temb_dim;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(arena + off_in, hid_in_dev, hid_bytes, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(arena + off_temb, temb_dev, temb_bytes, cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) {
      xema::set_last_cuda_error((int)e);
      rc = XEMA_ECUDA;
    }
    if (!rc) rc = xema_block_forward(plan, stream);
    if (!rc) {
      e = cudaMemcpyAsync(hid_out_dev, arena + off_out, hid_bytes, cudaMemcpyDeviceToDevice, st);
      if (e != cudaSuccess) {
        xema::set_last_cuda_error((int)e);
        rc = XEMA_ECUDA;
      }
    }
  }
  // the launches carry their TMA descriptors by value, so the host-side plan can go now
  xema_plan_destroy(plan);
  return rc;
}
