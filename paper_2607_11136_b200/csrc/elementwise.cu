// HBM-bound kernels of the block: adaLN modulation GEMV, LayerNorm + modulate, and
// per-head RMSNorm + RoPE.  128-bit coalesced accesses, one warp per token row, warp-shuffle
// reductions, fp32 arithmetic on bf16 storage.
#include <algorithm>

#include "kernels.h"
#include "sm100.cuh"

namespace xema {

using sm100::bf16_hi;
using sm100::bf16_lo;
using sm100::pack_bf16x2;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------------------------------
// mod[b, j] = sum_k silu(temb[b,k]) * w[j,k] + bias[j]
// One warp per output feature j; silu(temb) for all batch elements sits in shared memory.
// ---------------------------------------------------------------------------------------
constexpr int kModWarps = 8;
constexpr int kModMaxBatch = 8;

__global__ void __launch_bounds__(kModWarps * 32)
mod_gemv_kernel(const __nv_bfloat16* __restrict__ temb, const __nv_bfloat16* __restrict__ w,
                const __nv_bfloat16* __restrict__ bias, float* __restrict__ mod, int batch, int Dt, int n_out) {
  extern __shared__ float s_e[];  // [batch][Dt]
  for (int i = threadIdx.x; i < batch * Dt; i += blockDim.x) {
    float z = __bfloat162float(temb[i]);
    s_e[i] = z / (1.f + __expf(-z));
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int j = blockIdx.x * kModWarps + warp; j < n_out; j += gridDim.x * kModWarps) {
    const uint4* wr = reinterpret_cast<const uint4*>(w + (size_t)j * Dt);
    for (int b0 = 0; b0 < batch; b0 += kModMaxBatch) {
      float acc[kModMaxBatch];
#pragma unroll
      for (int b = 0; b < kModMaxBatch; ++b) acc[b] = 0.f;
      for (int k8 = lane; k8 * 8 < Dt; k8 += 32) {
        uint4 v = __ldg(wr + k8);
        float f[8] = {bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y),
                      bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w)};
#pragma unroll
        for (int b = 0; b < kModMaxBatch; ++b) {
          if (b0 + b < batch) {
            const float* e = s_e + (size_t)(b0 + b) * Dt + k8 * 8;
#pragma unroll
            for (int t = 0; t < 8; ++t) acc[b] = fmaf(f[t], e[t], acc[b]);
          }
        }
      }
#pragma unroll
      for (int b = 0; b < kModMaxBatch; ++b) {
        if (b0 + b < batch) {
          float s = warp_sum(acc[b]);
          if (lane == 0) mod[(size_t)(b0 + b) * n_out + j] = s + __bfloat162float(bias[j]);
        }
      }
    }
  }
}

int launch_mod(const void* temb, const void* w_mod, const void* b_mod, float* mod, int batch, int Dt, int n_out,
               cudaStream_t stream) {
  if (batch < 1 || Dt < 8 || (Dt & 7) || n_out < 1) return XEMA_EINVAL;
  size_t smem = (size_t)batch * Dt * sizeof(float);
  if (smem > 48 * 1024) return XEMA_EINVAL;
  int blocks = (n_out + kModWarps - 1) / kModWarps;
  mod_gemv_kernel<<<blocks, kModWarps * 32, smem, stream>>>(
      (const __nv_bfloat16*)temb, (const __nv_bfloat16*)w_mod, (const __nv_bfloat16*)b_mod, mod, batch, Dt, n_out);
  return check_launch();
}

// ---------------------------------------------------------------------------------------
// out = LN(in) * (1 + scale) + shift, one warp per row, the row held in registers.
// bf16 input: lane reads 8 elements (16 B) per step; fp32 input: 4 elements (16 B) per step.
// NV = steps per row (compile-time so the row stays in registers); NV == 0 selects the
// generic variant that re-reads the row instead.
// ---------------------------------------------------------------------------------------
constexpr int kLnWarps = 4;

template <bool IN_F32>
struct LnIo {
  static constexpr int EPV = IN_F32 ? 4 : 8;  // elements per lane per step
  __device__ static __forceinline__ void load(const void* row, int idx, float (&f)[EPV]) {
    if constexpr (IN_F32) {
      float4 v = __ldg(reinterpret_cast<const float4*>(row) + idx);
      f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    } else {
      uint4 v = __ldg(reinterpret_cast<const uint4*>(row) + idx);
      f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
      f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
    }
  }
  __device__ static __forceinline__ void store(__nv_bfloat16* row, int idx, const float (&f)[EPV]) {
    if constexpr (IN_F32) {
      uint2 v = make_uint2(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]));
      reinterpret_cast<uint2*>(row)[idx] = v;
    } else {
      uint4 v = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                           pack_bf16x2(f[6], f[7]));
      reinterpret_cast<uint4*>(row)[idx] = v;
    }
  }
};

template <bool IN_F32, int NV>
__global__ void __launch_bounds__(kLnWarps * 32)
ln_modulate_kernel(const void* __restrict__ in, long long in_batch_rows, __nv_bfloat16* __restrict__ out,
                   const float* __restrict__ shift, const float* __restrict__ scale, long long mod_stride,
                   int batch, int rows, int D, float eps) {
  using Io = LnIo<IN_F32>;
  constexpr int EPV = Io::EPV;
  const int lane = threadIdx.x & 31;
  const long long total = (long long)batch * rows;
  const long long r = (long long)blockIdx.x * kLnWarps + (threadIdx.x >> 5);
  if (r >= total) return;
  const int b = (int)(r / rows);
  const int i = (int)(r - (long long)b * rows);
  const size_t in_elem = ((size_t)b * in_batch_rows + i) * D;
  const void* src = IN_F32 ? (const void*)((const float*)in + in_elem) : (const void*)((const __nv_bfloat16*)in + in_elem);
  __nv_bfloat16* dst = out + (size_t)r * D;
  const float* sh = shift + (size_t)b * mod_stride;
  const float* sc = scale + (size_t)b * mod_stride;
  const int nv = D / (32 * EPV);
  const float inv_d = 1.f / (float)D;

  if constexpr (NV > 0) {
    float x[NV][EPV];
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      Io::load(src, v * 32 + lane, x[v]);
#pragma unroll
      for (int t = 0; t < EPV; ++t) s += x[v][t];
    }
    const float mean = warp_sum(s) * inv_d;
    float q = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
      for (int t = 0; t < EPV; ++t) {
        x[v][t] -= mean;
        q = fmaf(x[v][t], x[v][t], q);
      }
    const float rstd = rsqrtf(warp_sum(q) * inv_d + eps);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int e0 = (v * 32 + lane) * EPV;
      float y[EPV];
#pragma unroll
      for (int t4 = 0; t4 < EPV; t4 += 4) {
        float4 a = __ldg(reinterpret_cast<const float4*>(sc + e0 + t4));
        float4 c = __ldg(reinterpret_cast<const float4*>(sh + e0 + t4));
        y[t4 + 0] = fmaf(x[v][t4 + 0] * rstd, 1.f + a.x, c.x);
        y[t4 + 1] = fmaf(x[v][t4 + 1] * rstd, 1.f + a.y, c.y);
        y[t4 + 2] = fmaf(x[v][t4 + 2] * rstd, 1.f + a.z, c.z);
        y[t4 + 3] = fmaf(x[v][t4 + 3] * rstd, 1.f + a.w, c.w);
      }
      Io::store(dst, v * 32 + lane, y);
    }
  } else {
    float s = 0.f;
    for (int v = 0; v < nv; ++v) {
      float x[EPV];
      Io::load(src, v * 32 + lane, x);
#pragma unroll
      for (int t = 0; t < EPV; ++t) s += x[t];
    }
    const float mean = warp_sum(s) * inv_d;
    float q = 0.f;
    for (int v = 0; v < nv; ++v) {
      float x[EPV];
      Io::load(src, v * 32 + lane, x);
#pragma unroll
      for (int t = 0; t < EPV; ++t) {
        float c = x[t] - mean;
        q = fmaf(c, c, q);
      }
    }
    const float rstd = rsqrtf(warp_sum(q) * inv_d + eps);
    for (int v = 0; v < nv; ++v) {
      float x[EPV], y[EPV];
      Io::load(src, v * 32 + lane, x);
      const int e0 = (v * 32 + lane) * EPV;
#pragma unroll
      for (int t = 0; t < EPV; ++t) y[t] = fmaf((x[t] - mean) * rstd, 1.f + __ldg(sc + e0 + t), __ldg(sh + e0 + t));
      Io::store(dst, v * 32 + lane, y);
    }
  }
}

// Wide rows (D a multiple of 1024): one 128-thread block per row, 8 consecutive features per
// thread and step.  A thread then holds only D/128 values, so many more warps are resident and
// enough loads are in flight to cover the HBM latency; the two reductions go through shared
// memory.  Same arithmetic as above (mean, then centred sum of squares).
constexpr int kLnRowThreads = 128;

__device__ __forceinline__ float block_sum_128(float v, float* red, int phase) {
  v = warp_sum(v);
  float* slot = red + phase * 4;
  if ((threadIdx.x & 31) == 0) slot[threadIdx.x >> 5] = v;
  __syncthreads();
  return (slot[0] + slot[1]) + (slot[2] + slot[3]);
}

template <bool IN_F32, int VPT>
__global__ void __launch_bounds__(kLnRowThreads)
ln_modulate_row_kernel(const void* __restrict__ in, long long in_batch_rows, __nv_bfloat16* __restrict__ out,
                       const float* __restrict__ shift, const float* __restrict__ scale, long long mod_stride,
                       int batch, int rows, int D, float eps) {
  __shared__ float red[16];
  const long long total = (long long)batch * rows;
  const float inv_d = 1.f / (float)D;
  int parity = 0;
  for (long long r = blockIdx.x; r < total; r += gridDim.x, parity ^= 2) {
    const int b = (int)(r / rows);
    const int i = (int)(r - (long long)b * rows);
    const size_t in_elem = ((size_t)b * in_batch_rows + i) * D;
    const float* sh = shift + (size_t)b * mod_stride;
    const float* sc = scale + (size_t)b * mod_stride;
    float x[VPT][8];
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      const int e0 = (v * kLnRowThreads + threadIdx.x) * 8;
      if constexpr (IN_F32) {
        const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(in) + in_elem + e0);
        const float4 a = __ldg(p), c = __ldg(p + 1);
        x[v][0] = a.x; x[v][1] = a.y; x[v][2] = a.z; x[v][3] = a.w;
        x[v][4] = c.x; x[v][5] = c.y; x[v][6] = c.z; x[v][7] = c.w;
      } else {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(in) + in_elem + e0));
        x[v][0] = bf16_lo(u.x); x[v][1] = bf16_hi(u.x); x[v][2] = bf16_lo(u.y); x[v][3] = bf16_hi(u.y);
        x[v][4] = bf16_lo(u.z); x[v][5] = bf16_hi(u.z); x[v][6] = bf16_lo(u.w); x[v][7] = bf16_hi(u.w);
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) s += x[v][t];
    }
    const float mean = block_sum_128(s, red, parity) * inv_d;
    float q = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        x[v][t] -= mean;
        q = fmaf(x[v][t], x[v][t], q);
      }
    const float rstd = rsqrtf(block_sum_128(q, red, parity + 1) * inv_d + eps);
    __nv_bfloat16* dst = out + (size_t)r * D;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      const int e0 = (v * kLnRowThreads + threadIdx.x) * 8;
      const float4 a0 = __ldg(reinterpret_cast<const float4*>(sc + e0)), a1 = __ldg(reinterpret_cast<const float4*>(sc + e0 + 4));
      const float4 c0 = __ldg(reinterpret_cast<const float4*>(sh + e0)), c1 = __ldg(reinterpret_cast<const float4*>(sh + e0 + 4));
      const float y0 = fmaf(x[v][0] * rstd, 1.f + a0.x, c0.x), y1 = fmaf(x[v][1] * rstd, 1.f + a0.y, c0.y);
      const float y2 = fmaf(x[v][2] * rstd, 1.f + a0.z, c0.z), y3 = fmaf(x[v][3] * rstd, 1.f + a0.w, c0.w);
      const float y4 = fmaf(x[v][4] * rstd, 1.f + a1.x, c1.x), y5 = fmaf(x[v][5] * rstd, 1.f + a1.y, c1.y);
      const float y6 = fmaf(x[v][6] * rstd, 1.f + a1.z, c1.z), y7 = fmaf(x[v][7] * rstd, 1.f + a1.w, c1.w);
      *reinterpret_cast<uint4*>(dst + e0) =
          make_uint4(pack_bf16x2(y0, y1), pack_bf16x2(y2, y3), pack_bf16x2(y4, y5), pack_bf16x2(y6, y7));
    }
  }
}

template <bool IN_F32>
static int launch_ln_t(const void* in, long long in_batch_rows, void* out, const float* shift, const float* scale,
                       long long mod_stride, int batch, int rows, int D, float eps, cudaStream_t stream) {
  constexpr int EPV = LnIo<IN_F32>::EPV;
  const long long total = (long long)batch * rows;
  if (D % 1024 == 0 && D / 1024 <= 4) {
    // 16 resident blocks per SM cover the whole GPU; rows beyond that are taken in a stride loop
    const unsigned grid = (unsigned)std::min<long long>(total, 148LL * 16);
    auto* o2 = (__nv_bfloat16*)out;
#define XEMA_LNROW_CASE(N)                                                                                       \
  case N:                                                                                                        \
    ln_modulate_row_kernel<IN_F32, N><<<grid, kLnRowThreads, 0, stream>>>(in, in_batch_rows, o2, shift, scale,   \
                                                                           mod_stride, batch, rows, D, eps);     \
    break;
    switch (D / 1024) {
      XEMA_LNROW_CASE(1)
      XEMA_LNROW_CASE(2)
      XEMA_LNROW_CASE(3)
      XEMA_LNROW_CASE(4)
    }
#undef XEMA_LNROW_CASE
    return check_launch();
  }
  const unsigned blocks = (unsigned)((total + kLnWarps - 1) / kLnWarps);
  const int nv = D / (32 * EPV);
  auto* o = (__nv_bfloat16*)out;
#define XEMA_LN_CASE(N)                                                                                      \
  case N:                                                                                                    \
    ln_modulate_kernel<IN_F32, N><<<blocks, kLnWarps * 32, 0, stream>>>(in, in_batch_rows, o, shift, scale,  \
                                                                         mod_stride, batch, rows, D, eps);   \
    break;
  switch (nv) {
    XEMA_LN_CASE(2)
    XEMA_LN_CASE(4)
    XEMA_LN_CASE(12)
    XEMA_LN_CASE(24)
    default:
      ln_modulate_kernel<IN_F32, 0><<<blocks, kLnWarps * 32, 0, stream>>>(in, in_batch_rows, o, shift, scale,
                                                                           mod_stride, batch, rows, D, eps);
  }
#undef XEMA_LN_CASE
  return check_launch();
}

int launch_ln_modulate(const void* in, int in_is_f32, long long in_batch_rows, void* out, const float* shift,
                       const float* scale, long long mod_stride, int batch, int rows, int D, float eps,
                       cudaStream_t stream) {
  if (batch < 1 || rows < 0 || D < 256 || (D % 256)) return XEMA_EINVAL;
  if (rows == 0) return XEMA_OK;
  return in_is_f32 ? launch_ln_t<true>(in, in_batch_rows, out, shift, scale, mod_stride, batch, rows, D, eps, stream)
                   : launch_ln_t<false>(in, in_batch_rows, out, shift, scale, mod_stride, batch, rows, D, eps, stream);
}

// ---------------------------------------------------------------------------------------
// In place, per head: x <- RoPE(RMSNorm(x) * g).  One warp per token row; a lane owns 8
// consecutive features (four rotation pairs) of one head; DH/8 lanes share a head.
// ---------------------------------------------------------------------------------------
constexpr int kRopeWarps = 4;

template <int DH>
__global__ void __launch_bounds__(kRopeWarps * 32)
rmsnorm_rope_kernel(__nv_bfloat16* __restrict__ x, long long ld, long long batch_rows,
                    const __nv_bfloat16* __restrict__ g, const float* __restrict__ rope, int pos0, int batch,
                    int rows, int heads, float eps) {
  constexpr int LPH = DH / 8;        // lanes per head
  constexpr int HPW = 32 / LPH;      // heads per warp step
  const int lane = threadIdx.x & 31;
  const long long total = (long long)batch * rows;
  const long long r = (long long)blockIdx.x * kRopeWarps + (threadIdx.x >> 5);
  if (r >= total) return;
  const int b = (int)(r / rows);
  const int i = (int)(r - (long long)b * rows);
  __nv_bfloat16* row = x + ((size_t)b * batch_rows + i) * ld;
  const int e0 = (lane % LPH) * 8;   // first feature of this lane inside its head
  // cos/sin of this lane's four pairs and its eight gains: the same for every head
  const float4* rp = reinterpret_cast<const float4*>(rope + (size_t)(pos0 + i) * DH + e0);
  const float4 cs0 = __ldg(rp), cs1 = __ldg(rp + 1);
  const uint4 gv = __ldg(reinterpret_cast<const uint4*>(g + e0));
  const float gain[8] = {bf16_lo(gv.x), bf16_hi(gv.x), bf16_lo(gv.y), bf16_hi(gv.y),
                         bf16_lo(gv.z), bf16_hi(gv.z), bf16_lo(gv.w), bf16_hi(gv.w)};
  const float cosv[4] = {cs0.x, cs0.z, cs1.x, cs1.z};
  const float sinv[4] = {cs0.y, cs0.w, cs1.y, cs1.w};
  for (int h0 = 0; h0 < heads; h0 += HPW) {
    const int h = h0 + lane / LPH;
    const bool live = h < heads;
    uint4 v = make_uint4(0, 0, 0, 0);
    uint4* p = reinterpret_cast<uint4*>(row + (size_t)h * DH + e0);
    if (live) v = *p;
    float f[8] = {bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y),
                  bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w)};
    float ss = 0.f;
#pragma unroll
    for (int t = 0; t < 8; ++t) ss = fmaf(f[t], f[t], ss);
#pragma unroll
    for (int o = LPH / 2; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float rstd = rsqrtf(ss * (1.f / DH) + eps);
    float y[8];
#pragma unroll
    for (int pr = 0; pr < 4; ++pr) {
      const float a = f[2 * pr] * rstd * gain[2 * pr];
      const float c = f[2 * pr + 1] * rstd * gain[2 * pr + 1];
      y[2 * pr] = a * cosv[pr] - c * sinv[pr];
      y[2 * pr + 1] = a * sinv[pr] + c * cosv[pr];
    }
    if (live)
      *p = make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]),
                      pack_bf16x2(y[6], y[7]));
  }
}

int launch_rmsnorm_rope(void* x, long long ld, long long batch_rows, const void* g, const float* rope, int pos0,
                        int batch, int rows, int heads, int head_dim, float eps, cudaStream_t stream) {
  if (batch < 1 || rows < 0 || heads < 1 || (ld & 7)) return XEMA_EINVAL;
  if (rows == 0) return XEMA_OK;
  const long long total = (long long)batch * rows;
  const unsigned blocks = (unsigned)((total + kRopeWarps - 1) / kRopeWarps);
  if (head_dim == 64)
    rmsnorm_rope_kernel<64><<<blocks, kRopeWarps * 32, 0, stream>>>((__nv_bfloat16*)x, ld, batch_rows,
                                                                     (const __nv_bfloat16*)g, rope, pos0, batch, rows,
                                                                     heads, eps);
  else if (head_dim == 128)
    rmsnorm_rope_kernel<128><<<blocks, kRopeWarps * 32, 0, stream>>>((__nv_bfloat16*)x, ld, batch_rows,
                                                                      (const __nv_bfloat16*)g, rope, pos0, batch, rows,
                                                                      heads, eps);
  else
    return XEMA_EINVAL;
  return check_launch();
}

}  // namespace xema
