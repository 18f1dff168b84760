// Attention for head_dim 64: two 128-row query tiles per CTA, two CTAs per SM.
//
// With 64-wide heads the kernel is bound by the softmax warps (one exponential per 256 flop),
// not by the tensor pipe, and a softmax warp spends a good part of each key block in
// latencies (TMEM round trips, barrier hand-offs).  Sixteen softmax warps per SM -- four per
// scheduler -- keep the MUFU and issue slots busy through those gaps.  To fit 2 x 2 tiles into
// the 512 TMEM columns each tile has ONE 64-column score buffer (P(j) overwrites S(j) in
// place and S(j+1) is queued right behind PV(j)) and a 64-column output accumulator; both
// tiles of a CTA share the K and V tiles in shared memory.
//
//   warp 0     TMA producer: both Q tiles once, then K and V tiles through a ring of stages
//   warp 1     owns TMEM; converged warp, one elected lane issues, per tile and key block:
//              O += P(j) V(j), then S(j+1) = Q K(j+1)^T
//   warps 2-9  softmax: warps 2-5 own tile 0, warps 6-9 tile 1; thread = query row
//
// Keys are visited from key 0 in blocks of 64 and every decision is per row, exactly as in the
// general kernel, so the two kernels give the same bits for a row however rows are tiled.
#include <algorithm>

#include "kernels.h"
#include "sm100.cuh"

namespace xema {
using namespace sm100;

namespace {
constexpr int BM = 128;          // rows per tile
constexpr int TILES = 2;
constexpr int BN = kAttnDh64KeysPerBlock;   // keys per block (64)
constexpr int DH = 64;
constexpr int THREADS = 64 + 128 * TILES;
constexpr int Q_TILE_BYTES = BM * 128;
constexpr int KV_TILE_BYTES = BN * 128;
constexpr int STAGES = 4;
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILES * Q_TILE_BYTES;
constexpr int OFF_V = OFF_K + STAGES * KV_TILE_BYTES;
constexpr int OFF_BAR = OFF_V + STAGES * KV_TILE_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256;
constexpr int TMEM_COLS = 256;   // per tile: S/P [0,64), O [64,128)
#ifndef XEMA_ATT_POLY_NUM
#define XEMA_ATT_POLY_NUM 1
#endif
#ifndef XEMA_ATT_POLY_DEN
#define XEMA_ATT_POLY_DEN 4
#endif
constexpr int POLY_NUM = XEMA_ATT_POLY_NUM, POLY_DEN = XEMA_ATT_POLY_DEN;
}  // namespace

struct Attn64Params {
  __nv_bfloat16* o;
  float* lse;
  int batch, rows, keys, heads;
  float scale, scale_log2;
  unsigned int* status;
};

__global__ void __launch_bounds__(THREADS, 2)
attention_dh64_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v, const Attn64Params p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;    // [STAGES]
  uint64_t* k_empty = bars + 5;
  uint64_t* v_full = bars + 9;
  uint64_t* v_empty = bars + 13;
  uint64_t* s_full = bars + 17;   // [TILES]
  uint64_t* p_full = bars + 19;   // [TILES]
  uint64_t* pv_done = bars + 21;  // [TILES]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 23);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int n_kv = (p.keys + BN - 1) / BN;

  // The swizzled tiles need a 1024-byte aligned base; refuse to run otherwise.
  if ((smem_u32(smem) & 1023u) != 0) {
    if (threadIdx.x == 0 && p.status) atomicExch(p.status, 0x54310002u);
    return;
  }
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&k_full[s], 1);
      mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1);
      mbar_init(&v_empty[s], 1);
    }
    for (int t = 0; t < TILES; ++t) {
      mbar_init(&s_full[t], 1);
      mbar_init(&p_full[t], 128);   // every softmax thread of the tile arrives (no divergent single-lane arrive)
      mbar_init(&pv_done[t], 1);
    }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&map_q);
    prefetch_tmap(&map_k);
    prefetch_tmap(&map_v);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(q_full, TILES * Q_TILE_BYTES);
#pragma unroll
      for (int t = 0; t < TILES; ++t)
        tma_load_3d(smem + OFF_Q + t * Q_TILE_BYTES, &map_q, q_full, h * DH, (qt * TILES + t) * BM, b);
      int k_issued = 0, v_issued = 0;
      int st = 0;
      uint32_t ph = 0;
      for (int j = 0; j < n_kv; ++j) {
        if (!(ok = mbar_wait(&k_empty[st], ph ^ 1, abort_flag))) break;
        mbar_expect_tx(&k_full[st], KV_TILE_BYTES);
        tma_load_3d(smem + OFF_K + st * KV_TILE_BYTES, &map_k, &k_full[st], h * DH, j * BN, b);
        k_issued = j + 1;
        if (!(ok = mbar_wait(&v_empty[st], ph ^ 1, abort_flag))) break;
        mbar_expect_tx(&v_full[st], KV_TILE_BYTES);
        tma_load_3d(smem + OFF_V + st * KV_TILE_BYTES, &map_v, &v_full[st], h * DH, j * BN, b);
        v_issued = j + 1;
        if (++st == STAGES) { st = 0; ph ^= 1; }
      }
      if (!ok) {
        // gave up: let the copies already issued land before the CTA leaves (the latest
        // fill of each stage; older fills were consumed before their stage was reused)
        volatile uint32_t dummy = 0;
        mbar_wait(q_full, 0, &dummy);
        for (int j = max(0, k_issued - STAGES); j < k_issued; ++j) {
          dummy = 0;
          mbar_wait(&k_full[j % STAGES], (uint32_t)(j / STAGES) & 1u, &dummy);
        }
        for (int j = max(0, v_issued - STAGES); j < v_issued; ++j) {
          dummy = 0;
          mbar_wait(&v_full[j % STAGES], (uint32_t)(j / STAGES) & 1u, &dummy);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (converged warp, one elected lane issues) ----------------
    constexpr uint32_t idesc_s = idesc_bf16_f32(BM, BN, false, false);   // S = Q K^T
    constexpr uint32_t idesc_o = idesc_bf16_f32(BM, DH, false, true);    // O = P V, V is N-major
    const uint64_t q_desc0 = smem_desc_sw128(smem_u32(smem + OFF_Q), 16, 1024);
    const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + OFF_K), 16, 1024);
    const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + OFF_V), KV_TILE_BYTES, 1024);
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    auto issue_s = [&](int t, uint64_t k_desc) {   // elected lane only
      const uint32_t d = tmem_base + t * 128;
      const uint64_t q_desc = q_desc0 + (uint64_t)(t * (Q_TILE_BYTES >> 4));
#pragma unroll
      for (int k = 0; k < DH / 16; ++k) mma_ss(d, q_desc + (uint64_t)(2 * k), k_desc + (uint64_t)(2 * k), idesc_s, k != 0);
      mma_commit(&s_full[t]);
    };
    int k_st = 0, v_st = 0;
    uint32_t k_ph = 0, v_ph = 0;
    bool ok = wait_all(q_full, 0) && wait_all(&k_full[0], 0);
    if (ok) {
      tc_fence_after();
      if (elect_one()) {
        for (int t = 0; t < TILES; ++t) issue_s(t, k_desc0);
        mma_commit(&k_empty[0]);
      }
      __syncwarp();
      k_st = 1;
    }
    for (int j = 0; ok && j < n_kv; ++j) {
      const uint32_t par = (uint32_t)j & 1u;
      const bool more = j + 1 < n_kv;
      // K(j+1) and V(j) were requested stages ahead; check them before the hand-over of P(j)
      if (more && !(ok = wait_all(&k_full[k_st], k_ph))) break;
      if (!(ok = wait_all(&v_full[v_st], v_ph))) break;
      const uint64_t v_desc = v_desc0 + (uint64_t)(v_st * (KV_TILE_BYTES >> 4));
      const uint64_t k_desc = k_desc0 + (uint64_t)(k_st * (KV_TILE_BYTES >> 4));
#pragma unroll
      for (int t = 0; t < TILES; ++t) {
        // P(j) of this tile sits in TMEM over S(j) (and O was rescaled if a running max moved)
        if (!(ok = wait_all(&p_full[t], par))) break;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t sp = tmem_base + t * 128;
#pragma unroll
          for (int kk = 0; kk < BN / 16; ++kk)               // 16 keys = 8 packed P columns
            mma_ts(sp + 64, sp + kk * 8, v_desc + (uint64_t)(kk * (2048 >> 4)), idesc_o, (j | kk) != 0);
          mma_commit(&pv_done[t]);
          if (t == TILES - 1) mma_commit(&v_empty[v_st]);
          // S(j+1) goes into the same columns; it is queued behind PV(j), which reads P(j) there
          if (more) {
            issue_s(t, k_desc);
            if (t == TILES - 1) mma_commit(&k_empty[k_st]);
          }
        }
        __syncwarp();
      }
      if (++v_st == STAGES) { v_st = 0; v_ph ^= 1; }
      if (more && ++k_st == STAGES) { k_st = 0; k_ph ^= 1; }
    }
  } else {
    // ---------------- softmax / correction / epilogue ----------------
    const int tile = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int r = quad * 32 + lane;                       // query row inside the tile = TMEM lane
    const uint32_t s_tmem = tmem_base + ((uint32_t)(quad * 32) << 16) + tile * 128;
    const uint32_t o_tmem = s_tmem + 64;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      const uint32_t par = (uint32_t)j & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(&s_full[tile], par, abort_flag));
      if (!ok) break;
      tc_fence_after();
      float s[BN];
#pragma unroll
      for (int ch = 0; ch < BN / 32; ++ch)
        tmem_ld32(s_tmem + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[ch * 32]));
      tmem_ld_wait();
      // keys past the end exist only in the last block
      const int valid = p.keys - j * BN;
      if (valid < BN) {
#pragma unroll
        for (int t = 0; t < BN; ++t)
          if (t >= valid) s[t] = -INFINITY;
      }
      // row max: independent chains of three-input max
      float mx[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        mx[u] = max3(s[16 * u], s[16 * u + 1], s[16 * u + 2]);
#pragma unroll
        for (int t = 3; t < 15; t += 2) mx[u] = max3(mx[u], s[16 * u + t], s[16 * u + t + 1]);
        mx[u] = fmaxf(mx[u], s[16 * u + 15]);
      }
      const float m_blk = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      // the running max moves only when it grows by more than 2^8 (exp2 domain); per row
      float m_new = m_run;
      if (j == 0 || (m_blk - m_run) * p.scale_log2 > 8.f) m_new = m_blk;
      const float alpha = (j == 0 || m_new == m_run) ? 1.f : ex2_approx((m_run - m_new) * p.scale_log2);
      const float neg_m = -m_new * p.scale_log2;
      // p = exp2(s * c - m * c) on pairs of columns with packed fp32x2 arithmetic; POLY_NUM of
      // every POLY_DEN pairs (fixed column positions) evaluate 2^x as a polynomial on the FMA
      // pipe, the rest on the MUFU; row sum in four independent packed partial sums
      const f32x2 c2 = pack_f32x2(p.scale_log2, p.scale_log2);
      const f32x2 nm2 = pack_f32x2(neg_m, neg_m);
      f32x2 ls2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      uint32_t pk[BN / 2];
#pragma unroll
      for (int t = 0; t < BN; t += 2) {
        const int pair = t >> 1;
        f32x2 e2 = fma_f32x2(pack_f32x2(s[t], s[t + 1]), c2, nm2);
        float e0, e1;
        if ((pair % POLY_DEN) < POLY_NUM) {
          e2 = exp2_poly_f32x2(e2);
          unpack_f32x2(e2, e0, e1);
        } else {
          unpack_f32x2(e2, e0, e1);
          e0 = ex2_approx(e0);
          e1 = ex2_approx(e1);
          e2 = pack_f32x2(e0, e1);
        }
        ls2[pair & 3] = add_f32x2(ls2[pair & 3], e2);
        pk[pair] = pack_bf16x2(e0, e1);
      }
      float ls[4];
      {
        float a0, a1;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          unpack_f32x2(ls2[u], a0, a1);
          ls[u] = a0 + a1;
        }
      }
      l_run = fmaf(l_run, alpha, (ls[0] + ls[1]) + (ls[2] + ls[3]));
      m_run = m_new;
      // rescale O where the max moved (rows that kept their max multiply by exactly 1); only
      // then must PV(j-1) have finished
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
        ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[tile], (uint32_t)(j - 1) & 1u, abort_flag));
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int ch = 0; ch < DH / 32; ++ch) {
          uint32_t o[32];
          tmem_ld32(o_tmem + ch * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int t = 0; t < 32; ++t) o[t] = __float_as_uint(__uint_as_float(o[t]) * alpha);
          tmem_st32(o_tmem + ch * 32, o);
        }
      }
      // P(j) in place over this thread's score row: two bf16 per column, 32 columns
      tmem_st32(s_tmem, pk);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&p_full[tile]);
    }
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[tile], (uint32_t)(n_kv - 1) & 1u, abort_flag));
    if (ok) {
      tc_fence_after();
      const int row = (qt * TILES + tile) * BM + r;
      const float inv_l = 1.f / l_run;
      __nv_bfloat16* orow = p.o + ((size_t)b * p.rows + row) * ((size_t)p.heads * DH) + (size_t)h * DH;
#pragma unroll 1
      for (int ch = 0; ch < DH / 32; ++ch) {
        uint32_t o[32];
        tmem_ld32(o_tmem + ch * 32, o);
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
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicExch(p.status, STATUS_TIMEOUT_MBARRIER);
}

int launch_attention_dh64(const AttnLaunch& a, cudaStream_t stream) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attention_dh64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) {
      set_last_cuda_error((int)e);
      return XEMA_ECUDA;
    }
    attr_set = true;
  }
  Attn64Params p;
  p.o = (__nv_bfloat16*)a.o;
  p.lse = a.lse;
  p.batch = a.batch;
  p.rows = a.rows;
  p.keys = a.keys;
  p.heads = a.heads;
  p.scale = 0.125f;
  p.scale_log2 = p.scale * 1.4426950408889634f;
  p.status = a.status;
  dim3 grid((a.rows + TILES * BM - 1) / (TILES * BM), a.heads, a.batch);
  attention_dh64_kernel<<<grid, THREADS, SMEM_BYTES, stream>>>(a.map_q, a.map_k, a.map_v, p);
  return check_launch();
}

}  // namespace xema
