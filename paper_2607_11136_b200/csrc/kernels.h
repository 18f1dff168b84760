// Internal launch functions of the CUDA kernels.  All of them only enqueue work on `stream`.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/xema.h"

namespace xema {

// Records cudaGetLastError(); returns XEMA_OK or XEMA_ECUDA.
int check_launch();
void set_last_cuda_error(int code);

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
  unsigned int* status;
};
int attn_prepare(AttnLaunch* a, const void* q, long long ldq, long long q_batch_rows, const void* k, const void* v,
                 long long ldkv, long long kv_batch_rows);
int launch_attention(const AttnLaunch& a, cudaStream_t stream);
int launch_attention_dh64(const AttnLaunch& a, cudaStream_t stream);   // two-tile kernel for head_dim 64
constexpr int kAttnDh64KeysPerBlock = 64;                              // rows of its K/V TMA boxes

}  // namespace xema
