// Internal launch functions of the CUDA kernels.  All of them only enqueue work on `stream`.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include "../../include/xema.h"

namespace xema {

// Records cudaGetLastError(); returns XEMA_OK or XEMA_ECUDA.
int check_launch();
void set_last_cuda_error(int code);

// One-time launch state (function attributes, SM counts, cluster occupancy) belongs to a device,
// not to the process: these caches are indexed by the current device's ordinal and filled with
// atomic stores, so several host threads, or one process that drives several GPUs, see a
// value only after it was established on that device.  0 means "not known yet".  Ordinals at or
// beyond kMaxDevices are never cached (the value is looked up again on every call).
constexpr int kMaxDevices = 64;
struct PerDeviceInt {
  std::atomic<int> v[kMaxDevices];
  int get(int dev) const { return (dev >= 0 && dev < kMaxDevices) ? v[dev].load(std::memory_order_acquire) : 0; }
  void set(int dev, int value) {
    if (dev >= 0 && dev < kMaxDevices) v[dev].store(value, std::memory_order_release);
  }
};
// Ordinal of the calling thread's current device, or -1.
int current_device();
// Multiprocessor count of the current device (148 on a B200); cached per device.
int sm_count();
// Raises a kernel's dynamic shared-memory limit once per device.  `done` is the kernel's cache.
template <typename Kernel>
int ensure_smem_attr(Kernel kern, int bytes, PerDeviceInt& done) {
  const int dev = current_device();
  if (done.get(dev)) return XEMA_OK;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    return XEMA_ECUDA;
  }
  done.set(dev, 1);
  return XEMA_OK;
}

int launch_mod(const void* temb, const void* w_mod, const void* b_mod, float* mod, int batch, int Dt, int n_out,
               cudaStream_t stream);
int launch_ln_modulate(const void* in, int in_is_f32, long long in_batch_rows, void* out, const float* shift,
                       const float* scale, long long mod_stride, int batch, int rows, int D, float eps,
                       cudaStream_t stream);
int launch_rmsnorm_rope(void* x, long long ld, long long batch_rows, const void* g, const float* rope, int pos0,
                        int batch, int rows, int heads, int head_dim, float eps, cudaStream_t stream);

// ---- TMA descriptors (encoded on the host once per bound tensor) --------------------------
// bf16 tensor viewed as [batch][rows][cols] with row stride ld and batch stride batch_rows*ld
// (elements); box = 64 columns x box_rows rows x 1, 128-byte swizzle, out-of-range rows and
// columns read as zero.
int encode_tmap_bf16(CUtensorMap* out, const void* base, long long cols, long long rows, long long batch,
                     long long ld, long long batch_rows, int box_rows);

// ---- GEMM ------------------------------------------------------------------------------------
struct GemmLaunch {
  CUtensorMap map_a;   // [batch][rows][K], box 64 x 128
  CUtensorMap map_w;   // [1][N][K],       box 64 x block_n
  const void* bias;    // bf16 [N]
  void* out;
  long long ldo, out_batch_rows;
  const void* resid;
  long long ldr, resid_batch_rows;
  const float* gate;
  long long gate_stride;
  int batch, rows, N, K, epilogue, block_n;
  unsigned int* status;
  // XEMA_EPI_BIAS_NORM_ROPE: RMSNorm * gain + RoPE for the heads below column norm_cols
  const void* norm_gain;
  const float* rope;
  int rope_pos0, head_dim, norm_cols;
  float rms_eps;
  float norm_out_scale;   // the normalised, rotated heads are multiplied by this before rounding (1 = as they are)
};
// Fills map_a / map_w / block_n from plain pointers.
int gemm_prepare(GemmLaunch* g, const void* a, long long lda, long long a_batch_rows, const void* w, long long ldw);
int launch_gemm(const GemmLaunch& g, cudaStream_t stream);

// ---- attention -------------------------------------------------------------------------------
struct AttnLaunch {
  CUtensorMap map_q;   // [batch][rows][heads*dh], box 64 x 128
  CUtensorMap map_k;   // [batch][keys][..],       box 64 x 128
  CUtensorMap map_v;
  void* o;             // bf16 [batch][rows][heads*dh]
  float* lse;          // fp32 [batch][heads][rows] or null
  int batch, rows, keys, heads, head_dim;
  // what q k^T is multiplied by to give exponents to base 2: log2(e) / sqrt(head_dim) for a plain
  // q, 1 if q was already multiplied by that (as the fused epilogue of the Q projection does)
  float q_scale;
  unsigned int* status;
  // head_dim 64 only, both or neither: the RMSNorm gains (bf16 [head_dim], device) that q and k
  // went through before their rotation, with q multiplied by log2(e) / sqrt(head_dim) afterwards
  // (q_scale = 1).  A head of q then has norm <= max|gain_q| * log2(e) and a head of k norm <=
  // max|gain_k| * sqrt(head_dim), which bounds every score; where that bound is small the kernel
  // skips its per-score range tracking.  Null: nothing is known about the scores.
  const void* gain_q;
  const void* gain_k;
};
int attn_prepare(AttnLaunch* a, const void* q, long long ldq, long long q_batch_rows, const void* k, const void* v,
                 long long ldkv, long long kv_batch_rows);
int launch_attention(const AttnLaunch& a, cudaStream_t stream);
int launch_attention_dh64(const AttnLaunch& a, cudaStream_t stream);   // two-tile kernel for head_dim 64
constexpr int kAttnDh64KeysPerBlock = 128;                             // rows of its K/V TMA boxes

}  // namespace xema
