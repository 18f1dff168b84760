// Non-causal flash-style attention on tcgen05: o = softmax(q k^T / sqrt(dh)) v over all keys.
//
// One CTA owns one (batch, head, 128-query-row tile) and streams the keys in blocks of 128;
// its workspace (shared memory and TMEM) depends on the query tile only, never on the number
// of keys.  192 threads:
//   warp 0    TMA producer: Q tile once, then K and V tiles through two-stage rings
//   warp 1    owns TMEM; one thread issues S = Q K^T (TMEM, 128 fp32 columns) and
//             O += P V (TMEM, dh fp32 columns)
//   warps 2-5 softmax: thread = query row.  Read S from TMEM, running max / sum in the exp2
//             domain, write P (bf16, two per column) back into TMEM where the second MMA reads
//             it as its A operand (shared memory carries only Q, K and V: its bandwidth, not
//             the tensor pipe, bounds this kernel), rescale O in TMEM when the running max
//             moved, and at the end normalise O and store it.  The score row is held in registers, so the
//             S buffer is handed back right after the load and S(j+1) = Q K(j+1)^T runs while
//             the exponentials of block j are evaluated.
// Every decision is taken per row (the running max only moves when it grows by more than 2^8
// in the exp2 domain; multiplying the other rows by exactly 1 changes nothing), keys are
// always visited from key 0 in blocks of 128, and nothing is split or reduced across CTAs, so
// a query row's output bits do not depend on how the query rows are chunked or tiled.
#include <algorithm>

#include "kernels.h"
#include "sm100.cuh"

namespace xema {
using namespace sm100;

constexpr int ATT_BM = 128;      // query rows per CTA
constexpr int ATT_BN = 128;      // keys per block
constexpr int ATT_THREADS = 192;
constexpr int ATOM_BYTES = 128 * 128;   // 128 rows x 64 bf16, one swizzled column block
// share of the exponentials evaluated as a polynomial on the FMA pipe instead of the MUFU
#ifndef XEMA_ATT_POLY_NUM
#define XEMA_ATT_POLY_NUM 1
#endif
#ifndef XEMA_ATT_POLY_DEN
#define XEMA_ATT_POLY_DEN 4
#endif
constexpr int POLY_NUM = XEMA_ATT_POLY_NUM, POLY_DEN = XEMA_ATT_POLY_DEN;

template <int DH>
struct AttnCfg {
  static constexpr int ATOMS = DH / 64;                      // 64-wide column blocks per tile
  static constexpr int TILE_BYTES = ATOMS * ATOM_BYTES;      // Q, K or V tile
  static constexpr int KV_STAGES = (DH == 64) ? 3 : 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + TILE_BYTES;
  static constexpr int OFF_V = OFF_K + KV_STAGES * TILE_BYTES;
  static constexpr int OFF_BAR = OFF_V + KV_STAGES * TILE_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 256;
  // TMEM columns: S fp32 [0,128); P bf16, two per column [128,192); O fp32 [192, 192+DH)
  static constexpr int TMEM_P = 128;
  static constexpr int TMEM_O = 192;
  static constexpr int TMEM_COLS = (DH == 64) ? 256 : 512;
#ifdef XEMA_DBG_ONE_CTA
  static constexpr int MIN_CTAS = 1;
#else
  static constexpr int MIN_CTAS = (DH == 64) ? 2 : 1;
#endif
};

struct AttnParams {
  __nv_bfloat16* o;
  float* lse;
  int batch, rows, keys, heads;
  float scale;        // 1/sqrt(dh)
  float scale_log2;   // scale * log2(e)
  unsigned int* status;
};

template <int DH>
__global__ void __launch_bounds__(ATT_THREADS, AttnCfg<DH>::MIN_CTAS)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  using Cfg = AttnCfg<DH>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;    // [KV_STAGES <= 3]
  uint64_t* k_empty = bars + 4;
  uint64_t* v_full = bars + 7;
  uint64_t* v_empty = bars + 10;
  uint64_t* s_full = bars + 13;
  uint64_t* p_full = bars + 14;
  uint64_t* pv_done = bars + 15;
  uint64_t* s_free = bars + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int n_kv = (p.keys + ATT_BN - 1) / ATT_BN;

  // The swizzled tiles need a 1024-byte aligned base; refuse to run otherwise.
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && p.status) atomicExch(p.status, 0x54310002u);
    return;
  }

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < Cfg::KV_STAGES; ++s) {
      mbar_init(&k_full[s], 1);
      mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1);
      mbar_init(&v_empty[s], 1);
    }
    mbar_init(s_full, 1);
    mbar_init(p_full, 4);
    mbar_init(s_free, 4);
    mbar_init(pv_done, 1);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&map_q);
    prefetch_tmap(&map_k);
    prefetch_tmap(&map_v);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base;
  const uint32_t tmem_p = tmem_base + Cfg::TMEM_P;
  const uint32_t tmem_o = tmem_base + Cfg::TMEM_O;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(q_full, Cfg::TILE_BYTES);
#pragma unroll
      for (int a = 0; a < Cfg::ATOMS; ++a)
        tma_load_3d(smem + Cfg::OFF_Q + a * ATOM_BYTES, &map_q, q_full, h * DH + a * 64, qt * ATT_BM, b);
      int k_issued = 0, v_issued = 0;
      for (int j = 0; j < n_kv; ++j) {
        const int st = j % Cfg::KV_STAGES;
        const uint32_t ph = (uint32_t)(j / Cfg::KV_STAGES) & 1u;
        if (!(ok = mbar_wait(&k_empty[st], ph ^ 1, abort_flag))) break;
        mbar_expect_tx(&k_full[st], Cfg::TILE_BYTES);
#pragma unroll
        for (int a = 0; a < Cfg::ATOMS; ++a)
          tma_load_3d(smem + Cfg::OFF_K + st * Cfg::TILE_BYTES + a * ATOM_BYTES, &map_k, &k_full[st],
                      h * DH + a * 64, j * ATT_BN, b);
        k_issued = j + 1;
        if (!(ok = mbar_wait(&v_empty[st], ph ^ 1, abort_flag))) break;
        mbar_expect_tx(&v_full[st], Cfg::TILE_BYTES);
#pragma unroll
        for (int a = 0; a < Cfg::ATOMS; ++a)
          tma_load_3d(smem + Cfg::OFF_V + st * Cfg::TILE_BYTES + a * ATOM_BYTES, &map_v, &v_full[st],
                      h * DH + a * 64, j * ATT_BN, b);
        v_issued = j + 1;
      }
      if (!ok) {
        // gave up: let the copies already issued land before the CTA leaves (the latest
        // fill of each stage; older fills were consumed before their stage was reused)
        volatile uint32_t dummy = 0;
        mbar_wait(q_full, 0, &dummy);
        for (int j = max(0, k_issued - Cfg::KV_STAGES); j < k_issued; ++j) {
          dummy = 0;
          mbar_wait(&k_full[j % Cfg::KV_STAGES], (uint32_t)(j / Cfg::KV_STAGES) & 1u, &dummy);
        }
        for (int j = max(0, v_issued - Cfg::KV_STAGES); j < v_issued; ++j) {
          dummy = 0;
          mbar_wait(&v_full[j % Cfg::KV_STAGES], (uint32_t)(j / Cfg::KV_STAGES) & 1u, &dummy);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(ATT_BM, ATT_BN, false, false);   // S = Q K^T
      constexpr uint32_t idesc_o = idesc_bf16_f32(ATT_BM, DH, false, true);        // O = P V, V is N-major
      const uint32_t q_addr = smem_u32(smem + Cfg::OFF_Q);
      auto issue_s = [&](int j) -> bool {
        const int st = j % Cfg::KV_STAGES;
        const uint32_t ph = (uint32_t)(j / Cfg::KV_STAGES) & 1u;
        if (!mbar_wait(&k_full[st], ph, abort_flag)) return false;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(smem + Cfg::OFF_K + st * Cfg::TILE_BYTES);
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) {
          const uint32_t off = (k / 4) * ATOM_BYTES + (k % 4) * 32;
          mma_ss(tmem_s, smem_desc_sw128(q_addr + off, 16, 1024), smem_desc_sw128(k_addr + off, 16, 1024), idesc_s,
                 k != 0);
        }
        mma_commit(&k_empty[st]);
        mma_commit(s_full);
        return true;
      };
      bool ok = mbar_wait(q_full, 0, abort_flag);
      if (ok) ok = issue_s(0);
      for (int j = 0; ok && j < n_kv; ++j) {
        const int st = j % Cfg::KV_STAGES;
        const uint32_t ph = (uint32_t)(j / Cfg::KV_STAGES) & 1u;
        // as soon as the softmax warps hold S(j) in registers, S(j+1) may overwrite it
        if (j + 1 < n_kv) {
          if (!(ok = mbar_wait(s_free, j & 1, abort_flag))) break;
          tc_fence_after();
          if (!(ok = issue_s(j + 1))) break;
        }
        // P(j) is in shared memory (and O has been rescaled if the max moved)
        if (!(ok = mbar_wait(p_full, j & 1, abort_flag))) break;
        if (!(ok = mbar_wait(&v_full[st], ph, abort_flag))) break;
        tc_fence_after();
        const uint32_t v_addr = smem_u32(smem + Cfg::OFF_V + st * Cfg::TILE_BYTES);
#pragma unroll
        for (int kk = 0; kk < ATT_BN / 16; ++kk) {
          // P from TMEM: 16 keys = 8 packed columns per instruction.
          // V tile: rows = keys (the MMA's K), 64 dh per 128-byte row; 16 keys = 2048 bytes;
          // the second 64-wide dh block (dh = 128) starts one atom further
          const uint64_t db = smem_desc_sw128(v_addr + kk * 2048, ATOM_BYTES, 1024);
          mma_ts(tmem_o, tmem_p + kk * 8, db, idesc_o, (j | kk) != 0);
        }
        mma_commit(&v_empty[st]);
        mma_commit(pv_done);
      }
    }
  } else {
    // ---------------- softmax / correction / epilogue ----------------
    const int quad = warp & 3;
    const int r = quad * 32 + lane;                       // query row inside the tile = TMEM lane
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait(s_full, j & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      // the whole score row of this thread into registers, then hand the TMEM buffer back
      float s[ATT_BN];
#pragma unroll
      for (int ch = 0; ch < ATT_BN / 32; ++ch)
        tmem_ld32(tmem_s + lane_sel + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[ch * 32]));
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_free);
      // keys past the end exist only in the last block
      const int valid = p.keys - j * ATT_BN;
      if (valid < ATT_BN) {
#pragma unroll
        for (int t = 0; t < ATT_BN; ++t)
          if (t >= valid) s[t] = -INFINITY;
      }
      // row max: independent partial maxima, three-input max
      float mx[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) mx[u] = max3(s[16 * u], s[16 * u + 1], s[16 * u + 2]);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
#pragma unroll
        for (int t = 3; t < 15; t += 2) mx[u] = max3(mx[u], s[16 * u + t], s[16 * u + t + 1]);
        mx[u] = fmaxf(mx[u], s[16 * u + 15]);
      }
      const float m_blk = fmaxf(max3(mx[0], mx[1], mx[2]), max3(max3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
      // the running max moves only when it grows by more than 2^8 (exp2 domain); per row
      float m_new = m_run;
      if (j == 0 || (m_blk - m_run) * p.scale_log2 > 8.f) m_new = m_blk;
      const float alpha = (j == 0 || m_new == m_run) ? 1.f : ex2_approx((m_run - m_new) * p.scale_log2);
      const float neg_m = -m_new * p.scale_log2;
      // p = exp2(s * c - m * c) on pairs of columns with packed fp32x2 arithmetic; POLY_NUM of
      // every POLY_DEN pairs (fixed column positions) evaluate 2^x as a polynomial on the FMA
      // pipe, the rest on the MUFU; row sum in four independent packed partial sums
      const uint64_t c2 = pack_f32x2(p.scale_log2, p.scale_log2);
      const uint64_t nm2 = pack_f32x2(neg_m, neg_m);
      uint64_t ls2[4] = {0ull, 0ull, 0ull, 0ull};
      uint32_t pk[ATT_BN / 2];
#pragma unroll
      for (int t = 0; t < ATT_BN; t += 2) {
        const int pair = t >> 1;
        uint64_t e2 = fma_f32x2(pack_f32x2(s[t], s[t + 1]), c2, nm2);
        float e0, e1;
        if ((pair % POLY_DEN) < POLY_NUM) {
          e2 = exp2_poly_f32x2(e2);
          unpack_f32x2(e2, e0, e1);
        } else {
          unpack_f32x2(e2, e0, e1);
#ifdef XEMA_DBG_NOEXP
          e0 = e0 * 0.001f + 1.f;
          e1 = e1 * 0.001f + 1.f;
#else
          e0 = ex2_approx(e0);
          e1 = ex2_approx(e1);
#endif
          e2 = pack_f32x2(e0, e1);
        }
        ls2[pair & 3] = add_f32x2(ls2[pair & 3], e2);
        pk[pair] = pack_bf16x2(e0, e1);
      }
      float ls[4];
      {
        float a, b;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          unpack_f32x2(ls2[u], a, b);
          ls[u] = a + b;
        }
      }
      l_run = fmaf(l_run, alpha, (ls[0] + ls[1]) + (ls[2] + ls[3]));
      m_run = m_new;
      // P(j) overwrites the buffer PV(j-1) reads, and O must be at rest before it is rescaled
      if (j > 0) {
        ok = mbar_wait(pv_done, (j - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
      }
      // P(j) into TMEM: this thread's row, two bf16 per column, 64 columns
#pragma unroll
      for (int ch = 0; ch < ATT_BN / 64; ++ch)
        tmem_st32(tmem_p + lane_sel + ch * 32, *reinterpret_cast<const uint32_t(*)[32]>(&pk[ch * 32]));
      // rescale O where the max moved (rows that kept their max multiply by exactly 1)
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
        for (int ch = 0; ch < DH / 32; ++ch) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_sel + ch * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int t = 0; t < 32; ++t) o[t] = __float_as_uint(__uint_as_float(o[t]) * alpha);
          tmem_st32(tmem_o + lane_sel + ch * 32, o);
        }
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full);
    }
    if (ok) {
      ok = mbar_wait(pv_done, (n_kv - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const int row = qt * ATT_BM + r;
      const float inv_l = 1.f / l_run;
      __nv_bfloat16* orow = p.o + ((size_t)b * p.rows + row) * ((size_t)p.heads * DH) + (size_t)h * DH;
#pragma unroll 1
      for (int ch = 0; ch < DH / 32; ++ch) {
        uint32_t o[32];
        tmem_ld32(tmem_o + lane_sel + ch * 32, o);
        tmem_ld_wait();
        if (row < p.rows) {
          uint4* dst = reinterpret_cast<uint4*>(orow + ch * 32);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            dst[q] = make_uint4(pack_bf16x2(__uint_as_float(o[8 * q + 0]) * inv_l, __uint_as_float(o[8 * q + 1]) * inv_l),
                                pack_bf16x2(__uint_as_float(o[8 * q + 2]) * inv_l, __uint_as_float(o[8 * q + 3]) * inv_l),
                                pack_bf16x2(__uint_as_float(o[8 * q + 4]) * inv_l, __uint_as_float(o[8 * q + 5]) * inv_l),
                                pack_bf16x2(__uint_as_float(o[8 * q + 6]) * inv_l, __uint_as_float(o[8 * q + 7]) * inv_l));
        }
      }
      if (p.lse && row < p.rows)
        p.lse[((size_t)b * p.heads + h) * p.rows + row] = fmaf(m_run, p.scale, logf(l_run));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicExch(p.status, STATUS_TIMEOUT_MBARRIER);
}

template <int DH>
static int launch_attention_t(const AttnLaunch& a, cudaStream_t stream) {
  using Cfg = AttnCfg<DH>;
  static bool attr_set = false;
  auto kern = attention_kernel<DH>;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) {
      set_last_cuda_error((int)e);
      return XEMA_ECUDA;
    }
    attr_set = true;
  }
  AttnParams p;
  p.o = (__nv_bfloat16*)a.o;
  p.lse = a.lse;
  p.batch = a.batch;
  p.rows = a.rows;
  p.keys = a.keys;
  p.heads = a.heads;
  p.scale = 1.0f / sqrtf((float)DH);
  p.scale_log2 = p.scale * 1.4426950408889634f;
  p.status = a.status;
  dim3 grid((a.rows + ATT_BM - 1) / ATT_BM, a.heads, a.batch);
  kern<<<grid, ATT_THREADS, Cfg::SMEM_BYTES, stream>>>(a.map_q, a.map_k, a.map_v, p);
  return check_launch();
}

int launch_attention(const AttnLaunch& a, cudaStream_t stream) {
  if (a.rows == 0 || a.batch == 0) return XEMA_OK;
  if (a.head_dim == 64) return launch_attention_t<64>(a, stream);
  if (a.head_dim == 128) return launch_attention_t<128>(a, stream);
  return XEMA_EINVAL;
}

int attn_prepare(AttnLaunch* a, const void* q, long long ldq, long long q_batch_rows, const void* k, const void* v,
                 long long ldkv, long long kv_batch_rows) {
  if (a->batch < 1 || a->rows < 0 || a->keys < 1 || a->heads < 1) return XEMA_EINVAL;
  if (a->head_dim != 64 && a->head_dim != 128) return XEMA_EINVAL;
  if (a->heads > 65535 || a->batch > 65535) return XEMA_EINVAL;
  if (!q || !k || !v || !a->o) return XEMA_EINVAL;
  if ((ldq & 7) || (ldkv & 7)) return XEMA_EALIGN;
  auto mis = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; };
  if (mis(q) || mis(k) || mis(v) || mis(a->o)) return XEMA_EALIGN;
  const long long width = (long long)a->heads * a->head_dim;
  int rc = encode_tmap_bf16(&a->map_q, q, width, a->rows > 0 ? a->rows : 1, a->batch, ldq, q_batch_rows, ATT_BM);
  if (rc) return rc;
  rc = encode_tmap_bf16(&a->map_k, k, width, a->keys, a->batch, ldkv, kv_batch_rows, ATT_BN);
  if (rc) return rc;
  return encode_tmap_bf16(&a->map_v, v, width, a->keys, a->batch, ldkv, kv_batch_rows, ATT_BN);
}

}  // namespace xema
