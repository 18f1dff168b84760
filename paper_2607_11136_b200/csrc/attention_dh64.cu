// Attention for head_dim 64: o = softmax(q k^T / 8) v over all keys, non-causal.
//
// One CTA per SM owns two 128-row query tiles of one (batch, head) and streams the keys in
// blocks of 128 from key 0.  With 64-wide heads there is one exponential per 256 flop: the kernel
// is bound by the softmax threads (MUFU and issue slots), so everything else is arranged to stay
// out of their way and their own instruction count is kept down:
//
//   * per tile the scores S (128 fp32 columns of TMEM), the probabilities P (64 columns, bf16
//     pairs) and the output accumulator O (64 columns) are separate: S(j+1) = Q K(j+1)^T is
//     issued as soon as the tile's softmax threads hold S(j) in registers (half-way through
//     their block) and runs while they work; P(j) is stored in one piece at the end of the
//     block, when O += P(j-1) V(j-1), which reads the same columns, has long finished;
//   * 128-key blocks halve the number of tensor-core instructions and barrier hand-offs per key
//     (an MMA of 128 x 64 x 16 is bound by its shared-memory operand reads, 128 x 128 x 16 is
//     not), and the two MMA streams have a warp each: one warp for both spent as long in its
//     barrier waits as in issuing, and every wait of one stream held up the other;
//   * a score row is split between two threads (64 keys each): 16 softmax warps per SM, four per
//     scheduler, each working through its 64 scores in chunks of 16 with the next chunk on its
//     way from TMEM;
//   * no running maximum and, in the normal pass, no reference at all.  q arrives multiplied by
//     log2(e) / sqrt(64) (the Q projection's epilogue does that before its one rounding to bf16;
//     a plain q is multiplied here, in shared memory), so a score leaves the tensor core as the
//     exponent to base 2 of its unnormalised probability and p = 2^s is formed whatever its size
//     -- fp32 sums and bf16 probabilities keep their relative precision from 2^-90 to 2^90 -- so
//     nothing is ever rescaled, the two threads of a row need not talk to each other inside the
//     loop, and a softmax thread's work per pair of scores is the exponential, one packed add
//     for the row sum and one pack.  A row that leaves that range (a probability of 2^90 or more,
//     a row sum of 2^-90 or less), or that hands the exponential polynomial an argument outside
//     its range, is flagged, and its CTA runs two more sweeps: one that only takes the true row
//     maximum, one that repeats the pass with that maximum as the reference of the flagged rows
//     and with the polynomial's arguments clamped.  In that repeat the reference is taken off
//     inside the tensor core: the contraction gets a fifth 16-wide step over
//     [-reference, 0, ...] x [1, 0, ...] -- two small constant-shaped operands next to Q and K in
//     shared memory, the reference (as a bf16 number, zero for the rows that were fine) written
//     there by the row's thread.  Rows that were not flagged repeat exactly what they did
//     before, bit for bit;
//
//   warp 0      TMA producer: both Q tiles once, then K and V tiles through a ring of stages
//   warp 1      owns TMEM; converged warp, one elected lane issues S(j+1) of a tile as soon as
//               its S(j) is released
//   warp 2      the same for O += P(j) V(j) as soon as a tile's P(j) is complete
//   warps 3-18  softmax: warp = (tile, half of the key block, 32-row quarter); thread = query row
//
// Every decision is per row and keys are always visited in the same order, so a row's bits do not
// depend on how rows are tiled or chunked.
#include <algorithm>
#include <type_traits>

#include "kernels.h"
#include "sm100.cuh"

namespace xema {
using namespace sm100;

namespace {
constexpr int BM = 128;          // rows per tile
constexpr int TILES = 2;
constexpr int BN = kAttnDh64KeysPerBlock;   // keys per block (128)
constexpr int HALF = BN / 2;     // keys per softmax thread and block
constexpr int DH = 64;
constexpr int SOFTMAX_WARPS = 8 * TILES;
constexpr int THREADS = 96 + 32 * SOFTMAX_WARPS;
constexpr int Q_TILE_BYTES = BM * 128;
constexpr int KV_TILE_BYTES = BN * 128;
constexpr int STAGES = 4;
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILES * Q_TILE_BYTES;
constexpr int OFF_V = OFF_K + STAGES * KV_TILE_BYTES;
constexpr int OFF_QX = OFF_V + STAGES * KV_TILE_BYTES;       // per tile: 128 rows x 128 B, column 0 = -reference
constexpr int OFF_KX = OFF_QX + TILES * Q_TILE_BYTES;        // 128 keys x 128 B, column 0 = 1
constexpr int OFF_XCH = OFF_KX + KV_TILE_BYTES;              // float [2 slots][TILES][2 halves][BM]
constexpr int OFF_BAR = OFF_XCH + 2 * TILES * 2 * BM * 4;
constexpr int SMEM_BYTES = OFF_BAR + 512;
constexpr int TMEM_COLS = 512;   // per tile 256: S [0,128), P [128,192), O [192,256)
constexpr int TM_P = 128, TM_O = 192, TM_TILE = 256;
constexpr float DANGER = 1.2379400392853803e27f;   // 2^90
constexpr float TINY = 8.077935669463161e-28f;     // 2^-90
// Share of the exponentials evaluated as a polynomial on the FMA pipe instead of the MUFU: three
// column pairs of every eight (fixed positions).  Measured on B200 at 17776 x 17776 x 48 heads:
// none 753, 1/8 808, 1/4 870, 3/8 929, 1/2 790 TFLOP/s (before later changes that added ~6 %).
constexpr int POLY_NUM = 3, POLY_DEN = 8;
static_assert(BN == 128, "the kernel is written for 128-key blocks");
}  // namespace

// 2^x for two values on the FMA pipe, as exp2_poly_f32x2 but without its clamp: the caller
// guarantees -125 <= x <= 126.
__device__ __forceinline__ f32x2 exp2_poly_unclamped(f32x2 x2) {
  const f32x2 magic = make_float2(12582912.f, 12582912.f);
  const f32x2 neg_magic = make_float2(-12582912.f, -12582912.f);
  const f32x2 neg_one = make_float2(-1.f, -1.f);
  const f32x2 t2 = add_f32x2(x2, magic);                 // integer part lands in the low mantissa bits
  const f32x2 n2 = add_f32x2(t2, neg_magic);             // nearest integer as a float
  const f32x2 r2 = fma_f32x2(n2, neg_one, x2);           // r = x - n
  f32x2 p2 = fma_f32x2(make_float2(0.0551716685f, 0.0551716685f), r2, make_float2(0.242611125f, 0.242611125f));
  p2 = fma_f32x2(p2, r2, make_float2(0.693260968f, 0.693260968f));
  p2 = fma_f32x2(p2, r2, make_float2(0.999928057f, 0.999928057f));
  return make_float2(__uint_as_float(__float_as_uint(p2.x) + (__float_as_uint(t2.x) << 23)),
                     __uint_as_float(__float_as_uint(p2.y) + (__float_as_uint(t2.y) << 23)));
}

// p = 2^s for 16 consecutive score columns: 8 packed bf16x2 words, the values added
// into four packed partial sums.  POLY_NUM of every POLY_DEN column pairs (fixed positions)
// evaluate 2^x as a polynomial on the FMA pipe, the others on the MUFU.  The polynomial is only
// valid for arguments in [-125, 126].  SAFE = false: it is used as it is and, with TRACK,
// `poly_abs` collects the largest magnitude handed to it, for the caller to check afterwards
// (without TRACK the caller knows a bound on every score beforehand).  SAFE = true:
// arguments are clamped from below first (2^-125 stands in for zero); wherever the unclamped
// form was valid the result has the same bits.
template <bool SAFE, bool TRACK>
__device__ __forceinline__ void exp16(const float (&s)[16], uint32_t (&pk)[8], f32x2 (&ls2)[4], float& poly_abs) {
#pragma unroll
  for (int t = 0; t < 16; t += 2) {
    const int pair = t >> 1;
    f32x2 e2 = pack_f32x2(s[t], s[t + 1]);   // the scores come out of the tensor core as exponents
    float e0, e1;
    if ((pair % POLY_DEN) < POLY_NUM) {
      if (SAFE) {
        e2 = exp2_poly_f32x2(e2);
      } else {
        if (TRACK) poly_abs = max3(poly_abs, fabsf(e2.x), fabsf(e2.y));
        e2 = exp2_poly_unclamped(e2);
      }
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
}
__device__ __forceinline__ void mask_tail16(float (&s)[16], int valid) {
#pragma unroll
  for (int t = 0; t < 16; ++t)
    if (t >= valid) s[t] = -INFINITY;
}
__device__ __forceinline__ float sum_partials(const f32x2 (&ls2)[4]) {
  const f32x2 a = add_f32x2(ls2[0], ls2[1]), b = add_f32x2(ls2[2], ls2[3]);
  const f32x2 c = add_f32x2(a, b);
  return c.x + c.y;
}
// columns at or beyond `valid` (keys past the end of the sequence) count as minus infinity
__device__ __forceinline__ void mask_tail(float (&s)[32], int valid) {
#pragma unroll
  for (int t = 0; t < 32; ++t)
    if (t >= valid) s[t] = -INFINITY;
}
__device__ __forceinline__ float row_max32(const float (&s)[32]) {
  float mx[2];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    mx[u] = max3(s[16 * u], s[16 * u + 1], s[16 * u + 2]);
#pragma unroll
    for (int t = 3; t < 15; t += 2) mx[u] = max3(mx[u], s[16 * u + t], s[16 * u + t + 1]);
    mx[u] = fmaxf(mx[u], s[16 * u + 15]);
  }
  return fmaxf(mx[0], mx[1]);
}

struct Attn64Params {
  __nv_bfloat16* o;
  float* lse;
  int batch, rows, keys, heads;
  float q_scale;      // q k^T times this = exponents to base 2 (1: q arrives already multiplied)
  unsigned int* status;
  const __nv_bfloat16 *gain_q, *gain_k;   // RMSNorm gains behind q and k, or null (see AttnLaunch)
};

__global__ void __launch_bounds__(THREADS, 1)
attention_dh64_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v, const Attn64Params p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;     // [STAGES]
  uint64_t* k_empty = bars + 5;
  uint64_t* v_full = bars + 9;
  uint64_t* v_empty = bars + 13;
  uint64_t* s_full = bars + 17;    // [TILES] S(j) of the tile is complete in TMEM
  uint64_t* s_free = bars + 19;    // [TILES] every softmax thread of the tile holds S(j) in registers
  uint64_t* p_full = bars + 21;    // [TILES] P(j) of the tile is complete in TMEM
  uint64_t* pv_done = bars + 23;   // [TILES] O += P(j) V(j) has finished
  uint64_t* xch_bar = bars + 25;   // [TILES * 4] the two warps that share 32 rows exchange a value
  uint64_t* q_ready = bars + 33;   // the Q tiles are scaled and the extension operands are set up
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 34);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* danger_any = tmem_slot + 2;
  uint32_t* gain_max = tmem_slot + 3;          // [2] bit patterns of max|gain_q|, max|gain_k|
  volatile float* xch = reinterpret_cast<volatile float*>(smem + OFF_XCH);

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
      mbar_init(&s_free[t], 256);   // every softmax thread of the tile arrives
      mbar_init(&p_full[t], 256);
      mbar_init(&pv_done[t], 1);
    }
    for (int i = 0; i < TILES * 4; ++i) mbar_init(&xch_bar[i], 64);
    mbar_init(q_ready, 32 * SOFTMAX_WARPS);
    *abort_flag = 0;
    *danger_any = 0;
    gain_max[0] = gain_max[1] = 0;
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

  // ---- per-role state that lives across the sweeps ------------------------------------------
  // producer and MMA warp: rings of K and V stages
  int k_st = 0, v_st = 0;
  uint32_t k_ph = 0, v_ph = 0;
  // MMA warp: phases of the per-tile hand-over barriers it waits on
  uint32_t sfree_ph[TILES] = {0, 0}, pfull_ph[TILES] = {0, 0};
  // producer: what it has issued (for the drain after a give-up)
  int k_issued = 0, v_issued = 0;
  // softmax threads
  const int sw = warp - 3;
  const int quad = warp & 3;                               // TMEM lanes [32 * quad, 32 * quad + 32)
  const int tile = (sw >> 3) & 1;
  const int half = (sw >> 2) & 1;
  const int r = quad * 32 + lane;                          // query row inside the tile = TMEM lane
  const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + tile * TM_TILE;
  const uint32_t s_tmem = t_lane + half * HALF;
  const uint32_t p_tmem = t_lane + TM_P + half * (HALF / 2);
  const uint32_t o_tmem = t_lane + TM_O + half * (DH / 2);
  uint32_t sfull_ph = 0, pv_ph = 0, xch_ph = 0;
  int xch_slot = 0;
  float m_ref = 0.f, l_half = 0.f, m_true = -INFINITY;
  bool danger = false, danger_row = false;
  bool bounded = false;      // every score is known to lie well inside the polynomial's range
  bool ok = true;

  // One value from each of the two threads that share a row; returns the partner's.
  auto exchange = [&](float mine) -> float {
    volatile float* base = xch + ((xch_slot * TILES + tile) * 2) * BM;
    base[half * BM + r] = mine;
    uint64_t* bar = &xch_bar[tile * 4 + quad];
    mbar_arrive(bar);
    const bool got = __all_sync(0xffffffffu, mbar_wait(bar, xch_ph, abort_flag));
    xch_ph ^= 1;
    xch_slot ^= 1;
    return got ? base[(half ^ 1) * BM + r] : mine;
  };

  // Sweep 0: the pass itself (no reference).  If a row left the safe range: sweep 1 takes the
  // true maximum of every row (scores only), sweep 2 repeats the pass against it.
  for (int sweep = 0; sweep < 3; ++sweep) {
    const bool scores_only = (sweep == 1);
    if (warp == 0) {
      // ---------------- TMA producer ----------------
      if (lane == 0 && ok) {
        if (sweep == 0) {
          mbar_expect_tx(q_full, TILES * Q_TILE_BYTES);
#pragma unroll
          for (int t = 0; t < TILES; ++t)
            tma_load_3d(smem + OFF_Q + t * Q_TILE_BYTES, &map_q, q_full, h * DH, (qt * TILES + t) * BM, b);
        }
        for (int j = 0; j < n_kv; ++j) {
          if (!(ok = mbar_wait(&k_empty[k_st], k_ph ^ 1, abort_flag))) break;
          mbar_expect_tx(&k_full[k_st], KV_TILE_BYTES);
          tma_load_3d(smem + OFF_K + k_st * KV_TILE_BYTES, &map_k, &k_full[k_st], h * DH, j * BN, b);
          ++k_issued;
          if (++k_st == STAGES) { k_st = 0; k_ph ^= 1; }
          if (scores_only) continue;
          if (!(ok = mbar_wait(&v_empty[v_st], v_ph ^ 1, abort_flag))) break;
          mbar_expect_tx(&v_full[v_st], KV_TILE_BYTES);
          tma_load_3d(smem + OFF_V + v_st * KV_TILE_BYTES, &map_v, &v_full[v_st], h * DH, j * BN, b);
          ++v_issued;
          if (++v_st == STAGES) { v_st = 0; v_ph ^= 1; }
        }
        if (!ok) {
          // gave up: let the copies already issued land before the CTA leaves (the latest
          // fill of each stage; older fills were consumed before their stage was reused)
          volatile uint32_t dummy = 0;
          mbar_wait(q_full, 0, &dummy);
          for (int i = max(0, k_issued - STAGES); i < k_issued; ++i) {
            dummy = 0;
            mbar_wait(&k_full[i % STAGES], (uint32_t)(i / STAGES) & 1u, &dummy);
          }
          for (int i = max(0, v_issued - STAGES); i < v_issued; ++i) {
            dummy = 0;
            mbar_wait(&v_full[i % STAGES], (uint32_t)(i / STAGES) & 1u, &dummy);
          }
        }
      }
    } else if (warp == 1) {
      // ---------------- score issuer: S = Q K^T (converged warp, one elected lane issues) -------
      constexpr uint32_t idesc_s = idesc_bf16_f32(BM, BN, false, false);
      const uint64_t q_desc0 = smem_desc_sw128(smem_u32(smem + OFF_Q), 16, 1024);
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + OFF_K), 16, 1024);
      const uint64_t qx_desc0 = smem_desc_sw128(smem_u32(smem + OFF_QX), 16, 1024);
      const uint64_t kx_desc = smem_desc_sw128(smem_u32(smem + OFF_KX), 16, 1024);
      // with_ref (the repeat after a flag): one more 16-wide step of the contraction, over
      // [-reference, 0, ...] x [1, 0, ...]: the scores arrive with the row's reference taken off
      auto issue_s = [&](int t, uint64_t k_desc, bool with_ref) {   // elected lane only
        const uint32_t d = tmem_base + t * TM_TILE;
        const uint64_t q_desc = q_desc0 + (uint64_t)(t * (Q_TILE_BYTES >> 4));
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) mma_ss(d, q_desc + (uint64_t)(2 * k), k_desc + (uint64_t)(2 * k), idesc_s, k != 0);
        if (with_ref) mma_ss(d, qx_desc0 + (uint64_t)(t * (Q_TILE_BYTES >> 4)), kx_desc, idesc_s, 1);
        mma_commit(&s_full[t]);
      };
      if (ok && sweep == 0) ok = mbar_wait_warp(q_full, 0, abort_flag) && mbar_wait_warp(q_ready, 0, abort_flag);
      // S(0) of both tiles at once (the softmax threads are done with the previous sweep's scores:
      // the sweeps are separated by a CTA-wide barrier); S(j+1) of a tile as soon as its threads
      // hold S(j) in registers
      for (int j = 0; ok && j < n_kv; ++j) {
        ok = mbar_wait_warp(&k_full[k_st], k_ph, abort_flag); if (!ok) break;
        const uint64_t k_desc = k_desc0 + (uint64_t)(k_st * (KV_TILE_BYTES >> 4));
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
          if (j > 0) {
            ok = mbar_wait_warp(&s_free[t], sfree_ph[t], abort_flag); if (!ok) break;
            sfree_ph[t] ^= 1;
          }
          tc_fence_after();
          if (elect_one()) {
            issue_s(t, k_desc, sweep == 2);
            if (t == TILES - 1) mma_commit(&k_empty[k_st]);
          }
          __syncwarp();
        }
        if (!ok) break;
        if (++k_st == STAGES) { k_st = 0; k_ph ^= 1; }
      }
#pragma unroll
      for (int t = 0; t < TILES; ++t) sfree_ph[t] ^= 1;   // the release after the last block is not waited for
    } else if (warp == 2) {
      // ---------------- product issuer: O += P V (converged warp, one elected lane issues) ------
      constexpr uint32_t idesc_o = idesc_bf16_f32(BM, DH, false, true);    // V is N-major
      const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + OFF_V), KV_TILE_BYTES, 1024);
      for (int j = 0; ok && !scores_only && j < n_kv; ++j) {
        ok = mbar_wait_warp(&v_full[v_st], v_ph, abort_flag); if (!ok) break;
        const uint64_t v_desc = v_desc0 + (uint64_t)(v_st * (KV_TILE_BYTES >> 4));
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
          ok = mbar_wait_warp(&p_full[t], pfull_ph[t], abort_flag); if (!ok) break;
          pfull_ph[t] ^= 1;
          tc_fence_after();
          if (elect_one()) {
            const uint32_t tb = tmem_base + t * TM_TILE;
#pragma unroll
            for (int kk = 0; kk < BN / 16; ++kk)               // 16 keys = 8 packed P columns
              mma_ts(tb + TM_O, tb + TM_P + kk * 8, v_desc + (uint64_t)(kk * (2048 >> 4)), idesc_o, (j | kk) != 0);
            mma_commit(&pv_done[t]);
            if (t == TILES - 1) mma_commit(&v_empty[v_st]);
          }
          __syncwarp();
        }
        if (!ok) break;
        if (++v_st == STAGES) { v_st = 0; v_ph ^= 1; }
      }
    } else if (ok) {
      // ---------------- softmax ----------------
      // where a row's reference sits in the extension operand of its tile (128-byte swizzle:
      // the 16-byte chunk holding column 0 of row r is chunk r % 8 of the row)
      __nv_bfloat16* ref_slot = reinterpret_cast<__nv_bfloat16*>(smem + OFF_QX + tile * Q_TILE_BYTES + r * 128 + (r & 7) * 16);
      auto publish_ref = [&]() {
        // the reference as a bf16 number (any value near the maximum serves, as long as the same
        // one is used everywhere), negated, into column 0 of the extension operand
        const __nv_bfloat16 q = __float2bfloat16_rn(m_ref);
        m_ref = __bfloat162float(q);
        if (half == 0) *ref_slot = __float2bfloat16_rn(-m_ref);
        fence_proxy_async_smem();
      };
      if (sweep == 0) {
        // One-time set-up by the 512 softmax threads: the extension operands (zeros, and a one in
        // column 0 of every key row), and and, for a q that does not arrive in exponent
        // units, its tiles multiplied so that scores are exponents to base 2.
        const int ts = threadIdx.x - 96;
        uint4* zx = reinterpret_cast<uint4*>(smem + OFF_QX);
        for (int i = ts; i < (TILES * Q_TILE_BYTES + KV_TILE_BYTES) / 16; i += 32 * SOFTMAX_WARPS) {
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          const int k = i - TILES * Q_TILE_BYTES / 16;       // 16-byte chunk index inside the key operand
          if (k >= 0 && (k & 7) == ((k >> 3) & 7)) v.x = 0x3F80u;   // bf16 1.0 in column 0 of key row k / 8
          zx[i] = v;
        }
        if (p.q_scale != 1.f) {
          // a plain q: its tiles are multiplied here (a second rounding to bf16)
          ok = mbar_wait_warp(q_full, 0, abort_flag);
          if (ok) {
            uint4* qv = reinterpret_cast<uint4*>(smem + OFF_Q);
            for (int i = ts; i < TILES * Q_TILE_BYTES / 16; i += 32 * SOFTMAX_WARPS) {
              uint4 v = qv[i];
              uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
              for (int e = 0; e < 4; ++e) w[e] = pack_bf16x2(bf16_lo(w[e]) * p.q_scale, bf16_hi(w[e]) * p.q_scale);
              qv[i] = v;
            }
          }
        }
        if (ok) {
          fence_proxy_async_smem();
          mbar_arrive(q_ready);
        }
        // With q and k out of an RMSNorm (gains g), a rotation and, for q, the factor log2(e) / 8,
        // a head of q has norm <= max|g_q| * log2(e) and a head of k norm <= 8 * max|g_k|: every
        // score lies within +-11.55 * max|g_q| * max|g_k| (plus the bf16 roundings, under half a
        // percent).  Far inside the polynomial's range nothing needs to be tracked per score.
        if (p.gain_q && p.gain_k && p.q_scale == 1.f) {
          if (ts < DH) {
            atomicMax(&gain_max[0], __float_as_uint(fabsf(__bfloat162float(p.gain_q[ts]))));
            atomicMax(&gain_max[1], __float_as_uint(fabsf(__bfloat162float(p.gain_k[ts]))));
          }
          asm volatile("bar.sync 1, %0;" ::"n"(32 * SOFTMAX_WARPS) : "memory");
          const float gq = __uint_as_float(*(volatile uint32_t*)&gain_max[0]);
          const float gk = __uint_as_float(*(volatile uint32_t*)&gain_max[1]);
          bounded = gq * gk * 11.55f * 1.01f < 100.f;    // false for a NaN gain
        }
      }
      auto u16 = [](float(&a)[16]) -> uint32_t(&)[16] { return *reinterpret_cast<uint32_t(*)[16]>(&a[0]); };
      auto u32 = [](float(&a)[32]) -> uint32_t(&)[32] { return *reinterpret_cast<uint32_t(*)[32]>(&a[0]); };
      // the largest score of this thread's half of block j
      auto half_max = [&](int j) -> float {
        float sa[32], sb[32];
        tmem_ld32(s_tmem, u32(sa));
        tmem_ld32(s_tmem + 32, u32(sb));
        tmem_ld_wait_on(u32(sa));
        tmem_ld_wait_on(u32(sb));
        const int valid = p.keys - j * BN - half * HALF;
        if (valid < 32) mask_tail(sa, valid);
        if (valid < HALF) mask_tail(sb, valid - 32);
        return fmaxf(row_max32(sa), row_max32(sb));
      };
      if (scores_only) {
        for (int j = 0; j < n_kv; ++j) {
          ok = mbar_wait_warp(&s_full[tile], sfull_ph, abort_flag);
          sfull_ph ^= 1;
          if (!ok) break;
          tc_fence_after();
          const float mine = half_max(j);
          tc_fence_before();
          mbar_arrive(&s_free[tile]);
          m_true = fmaxf(m_true, mine);
        }
      } else {
        // (the reference of a flagged row was published at the end of the second sweep)
        // partial row sums and the largest polynomial argument of the whole sweep
        f32x2 ls2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        float poly_abs = 0.f;
        // One key block.  16 columns at a time: three chunks are requested at once and the fourth
        // as soon as the first has been worked on, so the whole of S(j) sits in registers -- and
        // S(j+1) may land -- when half of the block is done.  P(j) goes to TMEM in one piece at
        // the end: O += P(j-1) V(j-1), which reads the same columns, was only issued when the
        // previous block ended and has had this block's arithmetic to finish.
        auto run_block = [&](int j, auto masked_tag, auto first_tag, auto safe_tag, auto track_tag) {
          constexpr bool TRACK = decltype(track_tag)::value;
          constexpr bool MASKED = decltype(masked_tag)::value;
          constexpr bool FIRST = decltype(first_tag)::value;   // no earlier product to wait for
          // the ragged last block masks with minus infinity, which the unclamped polynomial cannot take
          constexpr bool SAFE = decltype(safe_tag)::value || MASKED;
          ok = mbar_wait_warp(&s_full[tile], sfull_ph, abort_flag);
          if (!ok) return;
          tc_fence_after();
          sfull_ph ^= 1;
          const int valid = MASKED ? p.keys - j * BN - half * HALF : HALF;
          uint32_t pk[32];
          auto pk8 = [&](int q) -> uint32_t(&)[8] { return *reinterpret_cast<uint32_t(*)[8]>(&pk[8 * q]); };
          float b0[16], b1[16], b2[16];
          tmem_ld16(s_tmem, u16(b0));
          tmem_ld16(s_tmem + 16, u16(b1));
          tmem_ld16(s_tmem + 32, u16(b2));
          tmem_ld_wait_on(u16(b0));
          tmem_ld_wait_on(u16(b1));
          tmem_ld_wait_on(u16(b2));
          if (MASKED && valid < 16) mask_tail16(b0, valid);
          exp16<SAFE, TRACK>(b0, pk8(0), ls2, poly_abs);
          tmem_ld16(s_tmem + 48, u16(b0));
          if (MASKED && valid < 32) mask_tail16(b1, valid - 16);
          exp16<SAFE, TRACK>(b1, pk8(1), ls2, poly_abs);
          tmem_ld_wait_on(u16(b0));
          tc_fence_before();
          mbar_arrive(&s_free[tile]);                       // S(j) is in registers: S(j+1) may land
          if (MASKED && valid < 48) mask_tail16(b2, valid - 32);
          exp16<SAFE, TRACK>(b2, pk8(2), ls2, poly_abs);
          if (MASKED) mask_tail16(b0, valid - 48);
          exp16<SAFE, TRACK>(b0, pk8(3), ls2, poly_abs);
          if (!FIRST) {
            if (!mbar_peek(&pv_done[tile], pv_ph)) ok = mbar_wait_warp(&pv_done[tile], pv_ph, abort_flag);
            pv_ph ^= 1;
            if (!ok) return;
            tc_fence_after();
          }
          tmem_st32(p_tmem, pk);
          tmem_st_wait();
          tc_fence_before();
          mbar_arrive(&p_full[tile]);
        };
        const int n_full = p.keys / BN;                     // blocks without keys past the end
        auto run_all = [&](auto safe_tag, auto track_tag) {
          if (ok) {
            if (n_full > 0) run_block(0, std::false_type{}, std::true_type{}, safe_tag, track_tag);
            else run_block(0, std::true_type{}, std::true_type{}, safe_tag, track_tag);
          }
          for (int j = 1; ok && j < n_full; ++j) run_block(j, std::false_type{}, std::false_type{}, safe_tag, track_tag);
          if (ok && n_full > 0 && n_full < n_kv) run_block(n_full, std::true_type{}, std::false_type{}, safe_tag, track_tag);
        };
        // the repeat after an overflow clamps the polynomial's arguments (rows that were fine get
        // the same bits from either form)
        if (sweep != 0) run_all(std::true_type{}, std::false_type{});
        else if (bounded) run_all(std::false_type{}, std::false_type{});
        else run_all(std::false_type{}, std::true_type{});
        // the accumulator is final once the last products have finished
        if (ok) {
          ok = mbar_wait_warp(&pv_done[tile], pv_ph, abort_flag);
          pv_ph ^= 1;
        }
        // Any probability of 2^90 or more shows in the sum: the sums only ever grow, and an
        // overflowed one is infinite or not a number.  An argument outside the polynomial's
        // range shows in poly_abs.
        l_half = sum_partials(ls2);
        danger = !(l_half < DANGER) || poly_abs > 120.f;
      }
      if (ok && sweep == 0) {
        // The row's sum (an infinity stands for a thread's own flag): above 2^90 a probability
        // overflowed or came close; at or below 2^-90 the row's scores lie so far below zero that
        // the small terms were flushed away.  Both threads of the row decide the same.
        const float mine = danger ? INFINITY : l_half;
        const float l_row = mine + exchange(mine);
        danger_row = !(l_row < DANGER) || !(l_row > TINY);
        if (danger_row) *danger_any = 1;
      }
      if (ok && sweep == 1) {
        m_true = fmaxf(m_true, exchange(m_true));
        if (danger_row) {
          m_ref = m_true;
          publish_ref();
        }
      }
    }
    // every role is done with this sweep; the softmax threads' flags are visible after the barrier
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*abort_flag) ok = false;
    if (sweep == 0 && (!*danger_any || !ok)) break;
  }

  if (warp >= 3 && ok) {
    // ---------------- epilogue: each of the row's two threads normalises and stores 32 columns ---
    const float l_row = l_half + exchange(l_half);
    tc_fence_after();
    const int row = (qt * TILES + tile) * BM + r;
    const float inv_l = 1.f / l_row;
    uint32_t o[32];
    tmem_ld32(o_tmem, o);
    tmem_ld_wait();
    if (row < p.rows) {
      __nv_bfloat16* orow = p.o + ((size_t)b * p.rows + row) * ((size_t)p.heads * DH) + (size_t)h * DH + half * (DH / 2);
      uint4* dst = reinterpret_cast<uint4*>(orow);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        dst[q] = make_uint4(pack_bf16x2(__uint_as_float(o[8 * q + 0]) * inv_l, __uint_as_float(o[8 * q + 1]) * inv_l),
                            pack_bf16x2(__uint_as_float(o[8 * q + 2]) * inv_l, __uint_as_float(o[8 * q + 3]) * inv_l),
                            pack_bf16x2(__uint_as_float(o[8 * q + 4]) * inv_l, __uint_as_float(o[8 * q + 5]) * inv_l),
                            pack_bf16x2(__uint_as_float(o[8 * q + 6]) * inv_l, __uint_as_float(o[8 * q + 7]) * inv_l));
      if (p.lse && half == 0) p.lse[((size_t)b * p.heads + h) * p.rows + row] = fmaf(m_ref, 0.6931471805599453f, logf(l_row));
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
  static PerDeviceInt attr_done;
  if (int rc = ensure_smem_attr(attention_dh64_kernel, SMEM_BYTES, attr_done)) return rc;
  Attn64Params p;
  p.o = (__nv_bfloat16*)a.o;
  p.lse = a.lse;
  p.batch = a.batch;
  p.rows = a.rows;
  p.keys = a.keys;
  p.heads = a.heads;
  p.q_scale = a.q_scale;
  p.status = a.status;
  p.gain_q = (const __nv_bfloat16*)a.gain_q;
  p.gain_k = (const __nv_bfloat16*)a.gain_k;
  dim3 grid((a.rows + TILES * BM - 1) / (TILES * BM), a.heads, a.batch);
  attention_dh64_kernel<<<grid, THREADS, SMEM_BYTES, stream>>>(a.map_q, a.map_k, a.map_v, p);
  return check_launch();
}

}  // namespace xema
