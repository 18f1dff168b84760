// Non-causal flash-style attention on tcgen05: o = softmax(q k^T / sqrt(dh)) v over all keys.
//
// One CTA owns one (batch, head, 128-query-row tile) and streams the keys in blocks of 64; its
// workspace (shared memory and TMEM) depends on the query tile only, never on the number of
// keys.  Two CTAs share an SM.  192 threads:
//   warp 0    TMA producer: Q tile once, then K and V tiles through a ring of stages
//   warp 1    owns TMEM; one thread issues S(j) = Q K(j)^T into one of two TMEM score buffers
//             and O += P(j) V(j) with P read from TMEM
//   warps 2-5 softmax: thread = query row.  Reads its score row from TMEM into registers,
//             keeps the running max / sum in the exp2 domain, writes P(j) (bf16, two per
//             column) in place over the score buffer it came from, rescales O in TMEM when the
//             running max moved, and at the end normalises O and stores it.
// Pipeline: the issuing thread's tcgen05 operations execute in order, so after P(j) is ready
// it queues PV(j) and then S(j+2) into the buffer PV(j) frees; the softmax warps therefore
// find S(j+1) waiting and depend on the tensor pipe again only in the rare iterations in which
// a row's running max moved (O must then be at rest).  Shared memory carries only Q, K, V.
//
// Every decision is taken per row (the running max only moves when it grows by more than 2^8
// in the exp2 domain; multiplying the other rows by exactly 1 changes nothing), keys are
// always visited from key 0 in blocks of 64, and nothing is split or reduced across CTAs, so
// a query row's output bits do not depend on how the query rows are chunked or tiled.
#include <algorithm>

#include "kernels.h"
#include "sm100.cuh"

namespace xema {
using namespace sm100;

constexpr int ATT_BM = 128;      // query rows per CTA
constexpr int ATT_BN = 64;       // keys per block
constexpr int ATT_THREADS = 192;
constexpr int Q_ATOM_BYTES = ATT_BM * 128;    // 128 rows x 64 bf16, one swizzled column block
constexpr int KV_ATOM_BYTES = ATT_BN * 128;   // 64 keys x 64 bf16
// Share of the exponentials evaluated as a polynomial on the FMA pipe instead of the MUFU: none
// in this kernel (with 128-wide heads a share of 1/8 or 1/4 measured 4-7 % slower: the shape is
// not bound by the exponent rate).
constexpr int POLY_NUM = 0, POLY_DEN = 4;

template <int DH>
struct AttnCfg {
  static constexpr int ATOMS = DH / 64;                        // 64-wide column blocks per tile
  static constexpr int Q_BYTES = ATOMS * Q_ATOM_BYTES;
  static constexpr int KV_BYTES = ATOMS * KV_ATOM_BYTES;       // one K or V tile
  static constexpr int KV_STAGES = (DH == 64) ? 4 : 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + KV_STAGES * KV_BYTES;
  static constexpr int OFF_BAR = OFF_V + KV_STAGES * KV_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 256;
  // TMEM columns: two score buffers S0 [0,64), S1 [64,128) (P(j) overwrites the first 32
  // columns of the buffer S(j) came from); O fp32 [128, 128+DH)
  static constexpr int TMEM_O = 128;
  static constexpr int TMEM_COLS = 256;
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
__global__ void __launch_bounds__(ATT_THREADS, 2)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  using Cfg = AttnCfg<DH>;
  constexpr int STAGES = Cfg::KV_STAGES;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;    // [STAGES <= 4]
  uint64_t* k_empty = bars + 5;
  uint64_t* v_full = bars + 9;
  uint64_t* v_empty = bars + 13;
  uint64_t* s_full = bars + 17;   // [2] one per score buffer
  uint64_t* p_full = bars + 19;   // [2]
  uint64_t* pv_done = bars + 21;  // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 23);
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
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&k_full[s], 1);
      mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1);
      mbar_init(&v_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&p_full[s], 4);
      mbar_init(&pv_done[s], 1);
    }
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
  const uint32_t tmem_o = tmem_base + Cfg::TMEM_O;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(q_full, Cfg::Q_BYTES);
#pragma unroll
      for (int a = 0; a < Cfg::ATOMS; ++a)
        tma_load_3d(smem + Cfg::OFF_Q + a * Q_ATOM_BYTES, &map_q, q_full, h * DH + a * 64, qt * ATT_BM, b);
      int k_issued = 0, v_issued = 0;
      int st = 0;
      uint32_t ph = 0;
      for (int j = 0; j < n_kv; ++j) {
        if (!(ok = mbar_wait(&k_empty[st], ph ^ 1, abort_flag))) break;
        mbar_expect_tx(&k_full[st], Cfg::KV_BYTES);
#pragma unroll
        for (int a = 0; a < Cfg::ATOMS; ++a)
          tma_load_3d(smem + Cfg::OFF_K + st * Cfg::KV_BYTES + a * KV_ATOM_BYTES, &map_k, &k_full[st],
                      h * DH + a * 64, j * ATT_BN, b);
        k_issued = j + 1;
        if (!(ok = mbar_wait(&v_empty[st], ph ^ 1, abort_flag))) break;
        mbar_expect_tx(&v_full[st], Cfg::KV_BYTES);
#pragma unroll
        for (int a = 0; a < Cfg::ATOMS; ++a)
          tma_load_3d(smem + Cfg::OFF_V + st * Cfg::KV_BYTES + a * KV_ATOM_BYTES, &map_v, &v_full[st],
                      h * DH + a * 64, j * ATT_BN, b);
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
    // ---------------- MMA issuer ----------------
    // The whole warp runs this loop converged and one elected lane issues: descriptors and
    // barrier addresses then stay warp-uniform values (a lone divergent thread would have to
    // move every operand into the uniform datapath one by one, and its dependent instruction
    // stream, not the tensor pipe, would bound the kernel).
    constexpr uint32_t idesc_s = idesc_bf16_f32(ATT_BM, ATT_BN, false, false);   // S = Q K^T
    constexpr uint32_t idesc_o = idesc_bf16_f32(ATT_BM, DH, false, true);        // O = P V, V is N-major
    const uint64_t q_desc = smem_desc_sw128(smem_u32(smem + Cfg::OFF_Q), 16, 1024);
    const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + Cfg::OFF_K), 16, 1024);
    // V tile: rows = keys (the MMA's K), 64 dh per 128-byte row, 16 keys = 2048 bytes; the
    // second 64-wide dh block (dh = 128) starts one atom further (leading byte offset)
    const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + Cfg::OFF_V), KV_ATOM_BYTES, 1024);
    int k_st = 0, v_st = 0;
    uint32_t k_ph = 0, v_ph = 0;
    auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    auto issue_s = [&](int buf) -> bool {
      if (!wait_all(&k_full[k_st], k_ph)) return false;
      tc_fence_after();
      if (elect_one()) {
        const uint64_t k_desc = k_desc0 + (uint64_t)(k_st * (Cfg::KV_BYTES >> 4));
        const uint32_t d = tmem_base + buf * ATT_BN;
#pragma unroll
        for (int k = 0; k < DH / 16; ++k)
          mma_ss(d, q_desc + (uint64_t)(((k / 4) * Q_ATOM_BYTES + (k % 4) * 32) >> 4),
                 k_desc + (uint64_t)(((k / 4) * KV_ATOM_BYTES + (k % 4) * 32) >> 4), idesc_s, k != 0);
        mma_commit(&k_empty[k_st]);
        mma_commit(&s_full[buf]);
      }
      __syncwarp();
      if (++k_st == STAGES) { k_st = 0; k_ph ^= 1; }
      return true;
    };
    bool ok = wait_all(q_full, 0);
    if (ok) ok = issue_s(0);
    if (ok && n_kv > 1) ok = issue_s(1);
    for (int j = 0; ok && j < n_kv; ++j) {
      const int buf = j & 1;
      const uint32_t par = (uint32_t)(j >> 1) & 1u;
      const bool more = j + 2 < n_kv;
      // K(j+2) and V(j) were loaded stages ahead: check them while P(j) is still being made,
      // so that nothing stands between P(j) becoming ready and the two products being queued
      // (only with a deep ring: with two stages K(j+2) is requested too late for that)
      constexpr bool kEarlyK = STAGES >= 4;
      if (kEarlyK && more && !(ok = wait_all(&k_full[k_st], k_ph))) break;
      if (!(ok = wait_all(&v_full[v_st], v_ph))) break;
      // P(j) sits in TMEM over S(j) (and O has been rescaled if a running max moved)
      if (!(ok = wait_all(&p_full[buf], par))) break;
      tc_fence_after();
      if (elect_one()) {
        const uint64_t v_desc = v_desc0 + (uint64_t)(v_st * (Cfg::KV_BYTES >> 4));
        const uint32_t sp_tmem = tmem_base + buf * ATT_BN;
#pragma unroll
        for (int kk = 0; kk < ATT_BN / 16; ++kk)             // 16 keys = 8 packed P columns
          mma_ts(tmem_o, sp_tmem + kk * 8, v_desc + (uint64_t)(kk * (2048 >> 4)), idesc_o, (j | kk) != 0);
        mma_commit(&v_empty[v_st]);
        mma_commit(&pv_done[buf]);
      }
      if (!kEarlyK && more) {
        if (!(ok = wait_all(&k_full[k_st], k_ph))) break;
        tc_fence_after();
      }
      if (elect_one()) {
        const uint32_t sp_tmem = tmem_base + buf * ATT_BN;
        // S(j+2) reuses the buffer; it is queued behind PV(j), which reads P(j) from it
        if (more) {
          const uint64_t k_desc = k_desc0 + (uint64_t)(k_st * (Cfg::KV_BYTES >> 4));
#pragma unroll
          for (int k = 0; k < DH / 16; ++k)
            mma_ss(sp_tmem, q_desc + (uint64_t)(((k / 4) * Q_ATOM_BYTES + (k % 4) * 32) >> 4),
                   k_desc + (uint64_t)(((k / 4) * KV_ATOM_BYTES + (k % 4) * 32) >> 4), idesc_s, k != 0);
          mma_commit(&k_empty[k_st]);
          mma_commit(&s_full[buf]);
        }
      }
      __syncwarp();
      if (++v_st == STAGES) { v_st = 0; v_ph ^= 1; }
      if (more && ++k_st == STAGES) { k_st = 0; k_ph ^= 1; }
    }
  } else {
    // ---------------- softmax / correction / epilogue ----------------
    const int quad = warp & 3;
    const int r = quad * 32 + lane;                       // query row inside the tile = TMEM lane
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    // The score row of block j+1 is requested from TMEM at the end of iteration j, right after
    // P(j) has been handed over; s[] always holds the block that is being worked on.
    float s[ATT_BN];
    ok = __all_sync(0xffffffffu, mbar_wait(&s_full[0], 0, abort_flag));
    if (ok) {
      tc_fence_after();
#pragma unroll
      for (int ch = 0; ch < ATT_BN / 32; ++ch)
        tmem_ld32(tmem_base + lane_sel + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[ch * 32]));
    }
    for (int j = 0; ok && j < n_kv; ++j) {
      const int buf = j & 1;
      const uint32_t s_tmem = tmem_base + lane_sel + buf * ATT_BN;
      const uint32_t next_par = (uint32_t)((j + 1) >> 1) & 1u;
      tmem_ld_wait();
      // keys past the end exist only in the last block
      const int valid = p.keys - j * ATT_BN;
      if (valid < ATT_BN) {
#pragma unroll
        for (int t = 0; t < ATT_BN; ++t)
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
      uint32_t pk[ATT_BN / 2];
#pragma unroll
      for (int t = 0; t < ATT_BN; t += 2) {
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
        ok = mbar_wait(&pv_done[(j - 1) & 1], (uint32_t)((j - 1) >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
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
      // P(j) in place over this thread's score row: two bf16 per column, 32 columns
      tmem_st32(s_tmem, pk);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[buf]);
      // request the next score row (S(j+1) was queued while this block was being worked on)
      if (j + 1 < n_kv) {
        ok = __all_sync(0xffffffffu, mbar_wait(&s_full[buf ^ 1], next_par, abort_flag));
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < ATT_BN / 32; ++ch)
          tmem_ld32(tmem_base + lane_sel + (buf ^ 1) * ATT_BN + ch * 32,
                    *reinterpret_cast<uint32_t(*)[32]>(&s[ch * 32]));
      }
    }
    if (ok) {
      ok = mbar_wait(&pv_done[(n_kv - 1) & 1], (uint32_t)((n_kv - 1) >> 1) & 1u, abort_flag);
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
  static PerDeviceInt attr_done;
  auto kern = attention_kernel<DH>;
  if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES, attr_done)) return rc;
  AttnParams p;
  p.o = (__nv_bfloat16*)a.o;
  p.lse = a.lse;
  p.batch = a.batch;
  p.rows = a.rows;
  p.keys = a.keys;
  p.heads = a.heads;
  p.scale_log2 = a.q_scale;                         // scores times this = exponents to base 2
  p.scale = a.q_scale * 0.6931471805599453f;        // ... and times this = natural exponents (for lse)
  p.status = a.status;
  dim3 grid((a.rows + ATT_BM - 1) / ATT_BM, a.heads, a.batch);
  kern<<<grid, ATT_THREADS, Cfg::SMEM_BYTES, stream>>>(a.map_q, a.map_k, a.map_v, p);
  return check_launch();
}

int launch_attention(const AttnLaunch& a, cudaStream_t stream) {
  if (a.rows == 0 || a.batch == 0) return XEMA_OK;
  if (a.head_dim == 64) return launch_attention_dh64(a, stream);
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
  // keys per block (= rows of a K/V box): 128 in the head_dim 64 kernel, 64 in the general one
  const int kv_box = (a->head_dim == 64) ? kAttnDh64KeysPerBlock : ATT_BN;
  rc = encode_tmap_bf16(&a->map_k, k, width, a->keys, a->batch, ldkv, kv_batch_rows, kv_box);
  if (rc) return rc;
  return encode_tmap_bf16(&a->map_v, v, width, a->keys, a->batch, ldkv, kv_batch_rows, kv_box);
}

}  // namespace xema
