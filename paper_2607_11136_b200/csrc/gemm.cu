// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores (tcgen05) with the four fused
// epilogues of the DiT block.
//
//   acc[b, i, n] = sum_k A[b, i, k] * W[n, k]          (both operands K-major)
//
// Structure of one CTA (persistent, one per SM, 192 threads):
//   warp 0    TMA producer: 128 x 64 tiles of A and BN x 64 tiles of W into a ring of
//             shared-memory stages (128-byte swizzle), completion on mbarriers
//   warp 1    owns TMEM; one thread issues tcgen05.mma (M = 128, N = BN, K = 16) into one of
//             two fp32 accumulators in TMEM and commits stage releases / accumulator-ready
//   warps 2-5 epilogue: tcgen05.ld the finished accumulator (thread = output row), apply the
//             epilogue in fp32 and store; runs while the next tile's main loop fills the
//             other accumulator
// A row's result depends only on (row, N, K): the K loop always runs in the same order and the
// tile shape is chosen from N alone, so outputs are bit-identical however rows are chunked.
#include <type_traits>

#include "kernels.h"
#include "sm100.cuh"

namespace xema {
using namespace sm100;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int GEMM_THREADS = 192;
constexpr int GROUP_M = 8;
constexpr int A_TILE_BYTES = BM * BK * 2;

template <int BN>
struct GemmCfg {
  static constexpr int B_TILE_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + BAR_BYTES;
};

struct GemmParams {
  const __nv_bfloat16* bias;
  void* out;
  long long ldo, out_batch_rows;
  const void* resid;
  long long ldr, resid_batch_rows;
  const float* gate;
  long long gate_stride;
  int batch, rows, N, K;
  unsigned int* status;
  // XEMA_EPI_BIAS_NORM_ROPE only: heads that start below column norm_cols get RMSNorm * gain
  // and RoPE in the epilogue (a thread owns whole rows, hence whole heads, of the tile)
  const __nv_bfloat16* norm_gain;   // [head_dim]
  const float* rope;                // [token][head_dim/2][cos, sin]
  int rope_pos0, head_dim, norm_cols;
  float rms_eps, norm_out_scale;
};

__device__ __forceinline__ float gelu_tanh_f(float z) {
  const float u = 0.7978845608028654f * fmaf(0.044715f * z * z, z, z);
  return 0.5f * z * (1.f + tanh_approx(u));
}

template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, int b, int row, int n0, const uint32_t (&r)[32]) {
  // bias and gate are the same for every row of the tile: broadcast loads
  float v[32];
  const uint4* bp = reinterpret_cast<const uint4*>(p.bias + n0);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 bb = __ldg(bp + q);
    v[8 * q + 0] = __uint_as_float(r[8 * q + 0]) + bf16_lo(bb.x);
    v[8 * q + 1] = __uint_as_float(r[8 * q + 1]) + bf16_hi(bb.x);
    v[8 * q + 2] = __uint_as_float(r[8 * q + 2]) + bf16_lo(bb.y);
    v[8 * q + 3] = __uint_as_float(r[8 * q + 3]) + bf16_hi(bb.y);
    v[8 * q + 4] = __uint_as_float(r[8 * q + 4]) + bf16_lo(bb.z);
    v[8 * q + 5] = __uint_as_float(r[8 * q + 5]) + bf16_hi(bb.z);
    v[8 * q + 6] = __uint_as_float(r[8 * q + 6]) + bf16_lo(bb.w);
    v[8 * q + 7] = __uint_as_float(r[8 * q + 7]) + bf16_hi(bb.w);
  }
  if (row >= p.rows) return;
  const size_t orow = ((size_t)b * p.out_batch_rows + row) * p.ldo + n0;
  if constexpr (EPI == XEMA_EPI_BIAS || EPI == XEMA_EPI_BIAS_GELU) {
    if constexpr (EPI == XEMA_EPI_BIAS_GELU) {
#pragma unroll
      for (int t = 0; t < 32; ++t) v[t] = gelu_tanh_f(v[t]);
    }
    uint4* op = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      op[q] = make_uint4(pack_bf16x2(v[8 * q], v[8 * q + 1]), pack_bf16x2(v[8 * q + 2], v[8 * q + 3]),
                         pack_bf16x2(v[8 * q + 4], v[8 * q + 5]), pack_bf16x2(v[8 * q + 6], v[8 * q + 7]));
  } else {
    const float4* gp = reinterpret_cast<const float4*>(p.gate + (size_t)b * p.gate_stride + n0);
    const size_t rrow = ((size_t)b * p.resid_batch_rows + row) * p.ldr + n0;
    if constexpr (EPI == XEMA_EPI_GATE_RES_F32) {
      // out fp32 = resid(bf16) + gate * v
      const uint4* rp = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.resid) + rrow);
      float4* op = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + orow);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 x = __ldg(rp + q);
        const float4 g0 = __ldg(gp + 2 * q), g1 = __ldg(gp + 2 * q + 1);
        op[2 * q] = make_float4(fmaf(g0.x, v[8 * q + 0], bf16_lo(x.x)), fmaf(g0.y, v[8 * q + 1], bf16_hi(x.x)),
                                fmaf(g0.z, v[8 * q + 2], bf16_lo(x.y)), fmaf(g0.w, v[8 * q + 3], bf16_hi(x.y)));
        op[2 * q + 1] = make_float4(fmaf(g1.x, v[8 * q + 4], bf16_lo(x.z)), fmaf(g1.y, v[8 * q + 5], bf16_hi(x.z)),
                                    fmaf(g1.z, v[8 * q + 6], bf16_lo(x.w)), fmaf(g1.w, v[8 * q + 7], bf16_hi(x.w)));
      }
    } else {
      // out bf16 = resid(fp32) + gate * v
      const float4* rp = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.resid) + rrow);
      uint4* op = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 x0 = __ldg(rp + 2 * q), x1 = __ldg(rp + 2 * q + 1);
        const float4 g0 = __ldg(gp + 2 * q), g1 = __ldg(gp + 2 * q + 1);
        op[q] = make_uint4(
            pack_bf16x2(fmaf(g0.x, v[8 * q + 0], x0.x), fmaf(g0.y, v[8 * q + 1], x0.y)),
            pack_bf16x2(fmaf(g0.z, v[8 * q + 2], x0.z), fmaf(g0.w, v[8 * q + 3], x0.w)),
            pack_bf16x2(fmaf(g1.x, v[8 * q + 4], x1.x), fmaf(g1.y, v[8 * q + 5], x1.y)),
            pack_bf16x2(fmaf(g1.z, v[8 * q + 6], x1.z), fmaf(g1.w, v[8 * q + 7], x1.w)));
      }
    }
  }
}

// The two gated epilogues for one 32-column chunk of a warp's 32 rows, with coalesced global
// accesses.  In the accumulator a thread owns a row, so a warp-wide 16-byte access would touch 32
// different rows -- 32 separate lines per instruction, eight store instructions and four to eight
// residual loads per chunk; the load/store unit then takes longer over a tile's epilogue (30 000
// cycles measured) than the tensor pipe over the next tile's main loop (22 000).  Here the accumulator
// goes through a per-warp shared-memory tile (rows padded to 36 floats) and comes back
// transposed: eight lanes cover the 32 columns of one row, a warp instruction covers four whole
// rows, and residual, gate and output are accessed a full row segment at a time.
constexpr int STAGE_LD = 36;                         // floats per staged row (16-byte aligned, conflict-light)
constexpr int STAGE_FLOATS = 32 * STAGE_LD;          // per warp
template <int EPI>
struct GatedResid {
  typename std::conditional<EPI == XEMA_EPI_GATE_RES_F32, uint2, float4>::type x[8];
  float4 gate;   // of the lane's four columns
  uint2 bias;    // four bf16
};
// Requests what a lane needs for one chunk besides the accumulator: the residual values of its
// four columns in eight rows, and the gate and bias of those columns.
template <int EPI>
__device__ __forceinline__ void gated_load_resid(const GemmParams& p, int b, int row0, int n0, int lane, GatedResid<EPI>& rs) {
  const int c4 = (lane & 7) * 4;
  const int rbase = row0 + (lane >> 3);
  rs.gate = __ldg(reinterpret_cast<const float4*>(p.gate + (size_t)b * p.gate_stride + n0 + c4));
  rs.bias = __ldg(reinterpret_cast<const uint2*>(p.bias + n0 + c4));
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = rbase + 4 * i;
    if (row < p.rows) {
      const size_t rrow = ((size_t)b * p.resid_batch_rows + row) * p.ldr + n0 + c4;
      if constexpr (EPI == XEMA_EPI_GATE_RES_F32)
        rs.x[i] = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p.resid) + rrow));
      else
        rs.x[i] = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.resid) + rrow));
    }
  }
}
template <int EPI>
__device__ __forceinline__ void epilogue_chunk_gated(const GemmParams& p, int b, int row0, int n0, const uint32_t (&r)[32],
                                                     float* stage, int lane, const GatedResid<EPI>& rs) {
  {
    // the raw accumulator row of this thread into the tile
    uint4* sp = reinterpret_cast<uint4*>(stage + lane * STAGE_LD);
#pragma unroll
    for (int q = 0; q < 8; ++q) sp[q] = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
  }
  __syncwarp();
  const int c4 = (lane & 7) * 4;                     // this lane's four columns of the chunk
  const float4 g = rs.gate;
  const float4 bs = make_float4(bf16_lo(rs.bias.x), bf16_hi(rs.bias.x), bf16_lo(rs.bias.y), bf16_hi(rs.bias.y));
  const int rbase = row0 + (lane >> 3);
  float4 v[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 a = *reinterpret_cast<const float4*>(stage + (4 * i + (lane >> 3)) * STAGE_LD + c4);
    v[i] = make_float4(a.x + bs.x, a.y + bs.y, a.z + bs.z, a.w + bs.w);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = rbase + 4 * i;
    if (row < p.rows) {
      const size_t orow = ((size_t)b * p.out_batch_rows + row) * p.ldo + n0 + c4;
      if constexpr (EPI == XEMA_EPI_GATE_RES_F32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + orow) =
            make_float4(fmaf(g.x, v[i].x, bf16_lo(rs.x[i].x)), fmaf(g.y, v[i].y, bf16_hi(rs.x[i].x)),
                        fmaf(g.z, v[i].z, bf16_lo(rs.x[i].y)), fmaf(g.w, v[i].w, bf16_hi(rs.x[i].y)));
      } else {
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow) =
            make_uint2(pack_bf16x2(fmaf(g.x, v[i].x, rs.x[i].x), fmaf(g.y, v[i].y, rs.x[i].y)),
                       pack_bf16x2(fmaf(g.z, v[i].z, rs.x[i].z), fmaf(g.w, v[i].w, rs.x[i].w)));
      }
    }
  }
  __syncwarp();                                      // the tile is free for the next chunk
}

// One head (DH columns starting at n0) of this thread's row: acc + bias, RMSNorm over the head,
// gain, rotation of adjacent pairs by the token's angles, bf16 store.
template <int DH>
__device__ __forceinline__ void epilogue_head_norm_rope(const GemmParams& p, int b, int row, int n0, uint32_t t_cols) {
  float v[DH];
#pragma unroll
  for (int ch = 0; ch < DH / 32; ++ch)
    tmem_ld32(t_cols + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[ch * 32]));
  tmem_ld_wait();
  if (row >= p.rows) return;
  float ss = 0.f;
#pragma unroll
  for (int q = 0; q < DH / 8; ++q) {
    const uint4 bb = __ldg(reinterpret_cast<const uint4*>(p.bias + n0) + q);
    v[8 * q + 0] += bf16_lo(bb.x); v[8 * q + 1] += bf16_hi(bb.x);
    v[8 * q + 2] += bf16_lo(bb.y); v[8 * q + 3] += bf16_hi(bb.y);
    v[8 * q + 4] += bf16_lo(bb.z); v[8 * q + 5] += bf16_hi(bb.z);
    v[8 * q + 6] += bf16_lo(bb.w); v[8 * q + 7] += bf16_hi(bb.w);
#pragma unroll
    for (int t = 0; t < 8; ++t) ss = fmaf(v[8 * q + t], v[8 * q + t], ss);
  }
  const float rstd = rsqrtf(ss * (1.f / DH) + p.rms_eps) * p.norm_out_scale;
  const float4* rp = reinterpret_cast<const float4*>(p.rope + (size_t)(p.rope_pos0 + row) * DH);
  uint4* op = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) +
                                       ((size_t)b * p.out_batch_rows + row) * p.ldo + n0);
#pragma unroll
  for (int q = 0; q < DH / 8; ++q) {
    const uint4 gg = __ldg(reinterpret_cast<const uint4*>(p.norm_gain) + q);
    const float gn[8] = {bf16_lo(gg.x), bf16_hi(gg.x), bf16_lo(gg.y), bf16_hi(gg.y),
                         bf16_lo(gg.z), bf16_hi(gg.z), bf16_lo(gg.w), bf16_hi(gg.w)};
    const float4 cs0 = __ldg(rp + 2 * q), cs1 = __ldg(rp + 2 * q + 1);
    const float cosv[4] = {cs0.x, cs0.z, cs1.x, cs1.z};
    const float sinv[4] = {cs0.y, cs0.w, cs1.y, cs1.w};
    float y[8];
#pragma unroll
    for (int pr = 0; pr < 4; ++pr) {
      const float a = v[8 * q + 2 * pr] * rstd * gn[2 * pr];
      const float c = v[8 * q + 2 * pr + 1] * rstd * gn[2 * pr + 1];
      y[2 * pr] = a * cosv[pr] - c * sinv[pr];
      y[2 * pr + 1] = a * sinv[pr] + c * cosv[pr];
    }
    op[q] = make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
  }
}

// The finished BN-wide accumulator row of one thread (TMEM address t_addr) -> global memory.
// `stage`: the warp's shared-memory tile for the coalesced form of the gated epilogues, or null
// (every thread then reads and writes its own row directly).
template <int BN, int EPI>
__device__ __forceinline__ void epilogue_row(const GemmParams& p, int b, int row, int n_base, uint32_t t_addr,
                                             float* stage = nullptr) {
  if constexpr (EPI == XEMA_EPI_BIAS_NORM_ROPE) {
    // head by head; heads at or beyond norm_cols (the V half of a KV product) get the bias only
#pragma unroll 1
    for (int hc = 0; hc < BN; hc += p.head_dim) {
      const int n0 = n_base + hc;
      if (n0 < p.norm_cols) {
        if (p.head_dim == 64) epilogue_head_norm_rope<64>(p, b, row, n0, t_addr + hc);
        else epilogue_head_norm_rope<128>(p, b, row, n0, t_addr + hc);
      } else {
#pragma unroll 1
        for (int ch = 0; ch < p.head_dim / 32; ++ch) {
          uint32_t r[32];
          tmem_ld32(t_addr + hc + ch * 32, r);
          tmem_ld_wait();
          epilogue_chunk<XEMA_EPI_BIAS>(p, b, row, n0 + ch * 32, r);
        }
      }
    }
  } else {
    if constexpr (EPI == XEMA_EPI_GATE_RES_F32 || EPI == XEMA_EPI_GATE_RES_BF16) {
      if (stage) {
        // coalesced form; the residual of chunk c+1 is requested before chunk c is worked on, and
        // all loads of a chunk are in flight together (one memory round trip per chunk, covered)
        const int lane = threadIdx.x & 31;
        const int row0 = row - lane;
        GatedResid<EPI> ra, rb;
        gated_load_resid<EPI>(p, b, row0, n_base, lane, ra);
#pragma unroll 1
        for (int ch = 0; ch < BN / 32; ch += 2) {
          uint32_t r[32];
          gated_load_resid<EPI>(p, b, row0, n_base + (ch + 1) * 32, lane, rb);
          tmem_ld32(t_addr + ch * 32, r);
          tmem_ld_wait();
          epilogue_chunk_gated<EPI>(p, b, row0, n_base + ch * 32, r, stage, lane, ra);
          if (ch + 2 < BN / 32) gated_load_resid<EPI>(p, b, row0, n_base + (ch + 2) * 32, lane, ra);
          tmem_ld32(t_addr + (ch + 1) * 32, r);
          tmem_ld_wait();
          epilogue_chunk_gated<EPI>(p, b, row0, n_base + (ch + 1) * 32, r, stage, lane, rb);
        }
        return;
      }
    }
#pragma unroll 1
    for (int ch = 0; ch < BN / 32; ++ch) {
      uint32_t r[32];
      tmem_ld32(t_addr + ch * 32, r);
      tmem_ld_wait();
      epilogue_chunk<EPI>(p, b, row, n_base + ch * 32, r);
    }
  }
}

struct TileCoord {
  int b, mt, nt;
};
__device__ __forceinline__ TileCoord tile_coord(int tile, int m_tiles, int n_tiles) {
  const int per_batch = m_tiles * n_tiles;
  TileCoord c;
  c.b = tile / per_batch;
  const int t = tile - c.b * per_batch;
  const int group_size = GROUP_M * n_tiles;
  const int g = t / group_size;
  const int first_m = g * GROUP_M;
  const int gm = min(GROUP_M, m_tiles - first_m);
  const int in_group = t - g * group_size;
  c.mt = first_m + in_group % gm;
  c.nt = in_group / gm;
  return c;
}

template <int BN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                 const GemmParams p) {
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* bar_base = smem + STAGES * Cfg::STAGE_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(bar_base);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (p.rows + BM - 1) / BM;
  const int n_tiles = p.N / BN;
  const int k_blocks = p.K / BK;
  const int total_tiles = p.batch * m_tiles * n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tmem_full[s], 1);
      mbar_init(&tmem_empty[s], 4);
    }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_w);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const TileCoord c = tile_coord(tile, m_tiles, n_tiles);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag))) break;
          uint8_t* sa = smem + stage * Cfg::STAGE_BYTES;
          uint8_t* sb = sa + A_TILE_BYTES;
          mbar_expect_tx(&full[stage], Cfg::STAGE_BYTES);
          tma_load_3d(sa, &map_a, &full[stage], kb * BK, c.mt * BM, c.b);
          tma_load_3d(sb, &map_w, &full[stage], kb * BK, c.nt * BN, 0);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        // gave up: let the copies already issued land before the CTA leaves
        for (int s = 0; s < STAGES; ++s) {
          const int st = (stage + s) % STAGES;                 // oldest outstanding first
          const uint32_t ph = (st < stage) ? phase : (phase ^ 1);
          volatile uint32_t dummy = 0;
          mbar_wait(&full[st], ph, &dummy);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    // The whole warp walks the loop and waits together; one elected lane issues.  (A lone
    // thread of a diverged warp issues MMAs markedly slower than the tensor pipe retires them.)
    {
      constexpr uint32_t idesc = idesc_bf16_f32(BM, BN, false, false);
      // Descriptors are built once and advanced by adding constants (the start-address field
      // counts 16-byte units and never carries out of its 14 bits inside shared memory).
      const uint64_t a_desc0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
      const uint64_t b_desc0 = smem_desc_sw128(smem_u32(smem + A_TILE_BYTES), 16, 1024);
      auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        if (!(ok = wait_all(&tmem_empty[acc], acc_phase ^ 1))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        uint32_t accumulate = 0;
#pragma unroll 1
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = wait_all(&full[stage], phase))) break;
          tc_fence_after();
          if (elect_one()) {
            const uint64_t soff = (uint64_t)(stage * (Cfg::STAGE_BYTES >> 4));
            const uint64_t da = a_desc0 + soff, db = b_desc0 + soff;
            mma_ss(d_tmem, da, db, idesc, accumulate);
            mma_ss(d_tmem, da + 2, db + 2, idesc, 1);
            mma_ss(d_tmem, da + 4, db + 4, idesc, 1);
            mma_ss(d_tmem, da + 6, db + 6, idesc, 1);
            mma_commit(&empty[stage]);
          }
          __syncwarp();
          accumulate = 1;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if (elect_one()) mma_commit(&tmem_full[acc]);
        __syncwarp();
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ---------------- epilogue ----------------
    const int quad = warp & 3;           // TMEM lanes [32*quad, 32*quad + 32) belong to this warp
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
      const TileCoord c = tile_coord(tile, m_tiles, n_tiles);
      ok = mbar_wait(&tmem_full[acc], acc_phase, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = c.mt * BM + quad * 32 + lane;
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BN;
      epilogue_row<BN, EPI>(p, c.b, row, c.nt * BN, t_addr);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1; }
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


// ---------------------------------------------------------------------------------------------
// CTA-pair variant (N a multiple of 256): two CTAs on neighbouring SMs share one 256 x 256
// output tile.  Each CTA loads its own 128 rows of A and one half (128 rows) of the W tile, so a
// stage costs 32 KB of shared-memory fill per SM instead of 48 KB and every MMA reads 8 KB of
// operands per SM instead of 12 KB; the even CTA issues tcgen05.mma.cta_group::2 (M = 256),
// which accumulates 128 rows x 256 columns in the TMEM of each CTA.
//   full[s]        barrier of the even CTA: its producer expects the bytes of both CTAs, and
//                  both CTAs' loads complete on it (an expect-tx arrival sent from the peer
//                  CTA for every stage halved the speed of the whole loop)
//   empty[s]       one barrier per CTA, released for both by a multicast commit
//   tmem_full[a]   one barrier per CTA, same commit form
//   tmem_empty[a]  barrier of the even CTA: the four epilogue warps of both CTAs arrive
// The K loop and the per-instruction summation are the same for every row, so results do not
// depend on how rows are chunked.
constexpr int PAIR_BN = 256;
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_B_HALF_BYTES = (PAIR_BN / 2) * BK * 2;
constexpr int PAIR_STAGE_BYTES = A_TILE_BYTES + PAIR_B_HALF_BYTES;
constexpr int PAIR_STAGE_TILE_BYTES = 4 * STAGE_FLOATS * 4;      // one transposition tile per epilogue warp
constexpr int PAIR_SMEM_BYTES = 1024 + PAIR_STAGES * PAIR_STAGE_BYTES + 256 + PAIR_STAGE_TILE_BYTES;
constexpr int PAIR_TMEM_COLS = 2 * PAIR_BN;
// Limit of one drain wait after a give-up (about 50 ms): long enough for any copy in flight,
// short enough that six of them in a row stay far below the limit of a regular wait.
constexpr long long kDrainLimitCycles = 100000000ll;

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                      const GemmParams p) {
  constexpr int STAGES = PAIR_STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* bar_base = smem + STAGES * PAIR_STAGE_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(bar_base);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();            // 0: even CTA (issues the MMAs), 1: its peer
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles = (p.rows + 2 * BM - 1) / (2 * BM);   // tiles of 256 rows
  const int n_tiles = p.N / PAIR_BN;
  const int k_blocks = p.K / BK;
  const int total_tiles = p.batch * m_tiles * n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tmem_full[s], 1);
      mbar_init(&tmem_empty[s], 8);
    }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_w);
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, PAIR_TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();      // both CTAs' barriers exist before anything arrives on them remotely
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer (one per CTA) ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        const TileCoord c = tile_coord(tile, m_tiles, n_tiles);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag))) break;
          uint8_t* sa = smem + stage * PAIR_STAGE_BYTES;
          uint8_t* sb = sa + A_TILE_BYTES;
          const uint32_t full0 = mapa_shared(smem_u32(&full[stage]), 0);
          if (rank == 0) mbar_expect_tx(&full[stage], 2 * PAIR_STAGE_BYTES);
          tma_load_3d_pair(sa, &map_a, full0, kb * BK, (c.mt * 2 + (int)rank) * BM, c.b);
          tma_load_3d_pair(sb, &map_w, full0, kb * BK, c.nt * PAIR_BN + (int)rank * (PAIR_BN / 2), 0);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      // Tail: the same waits as for STAGES further fills, without filling.  They return once the
      // commits that release this CTA's last fills (arrivals multicast by the even CTA) have
      // landed here, so none of them can reach this CTA's barriers after it has left.
      for (int s = 0; ok && s < STAGES; ++s) {
        ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag);
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
      if (!ok) {
        // Gave up.  Copies already issued must land before either CTA leaves: all of them
        // complete on the even CTA's full[] barriers, so the even CTA waits (bounded, and
        // without looking at the abort flag) for the latest fill of every stage, which covers
        // the bytes of both CTAs wherever both issued; the closing cluster barrier then keeps
        // the peer until that is done.  A short settling time on both CTAs covers loads of a
        // stage that only one of the two CTAs still issued.
        if (rank == 0) {
          for (int s = 0; s < STAGES; ++s) {
            const int st = (stage + s) % STAGES;                 // oldest outstanding first
            const uint32_t ph = (st < stage) ? phase : (phase ^ 1);
            volatile uint32_t dummy = 0;
            mbar_wait_slow(&full[st], ph, &dummy, kDrainLimitCycles);
          }
        }
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (even CTA only; converged warp, one elected lane) ----------------
    if (rank == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(2 * BM, PAIR_BN, false, false);
      const uint64_t a_desc0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
      const uint64_t b_desc0 = smem_desc_sw128(smem_u32(smem + A_TILE_BYTES), 16, 1024);
      auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
      };
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        // the peer's epilogue warps arrive on this barrier from their own CTA: cluster-scope acquire
        if (!(ok = __all_sync(0xffffffffu, mbar_wait_cluster(&tmem_empty[acc], acc_phase ^ 1, abort_flag)))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * PAIR_BN;
        uint32_t accumulate = 0;
#pragma unroll 1
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = wait_all(&full[stage], phase))) break;
          tc_fence_after();
          if (elect_one()) {
            const uint64_t soff = (uint64_t)(stage * (PAIR_STAGE_BYTES >> 4));
            const uint64_t da = a_desc0 + soff, db = b_desc0 + soff;
            mma_ss_pair(d_tmem, da, db, idesc, accumulate);
            mma_ss_pair(d_tmem, da + 2, db + 2, idesc, 1);
            mma_ss_pair(d_tmem, da + 4, db + 4, idesc, 1);
            mma_ss_pair(d_tmem, da + 6, db + 6, idesc, 1);
            mma_commit_pair(&empty[stage]);
          }
          __syncwarp();
          accumulate = 1;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if (elect_one()) mma_commit_pair(&tmem_full[acc]);
        __syncwarp();
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ---------------- epilogue (both CTAs, each its own 128 rows) ----------------
    const int quad = warp & 3;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = pair; ok && tile < total_tiles; tile += n_pairs) {
      const TileCoord c = tile_coord(tile, m_tiles, n_tiles);
      ok = mbar_wait(&tmem_full[acc], acc_phase, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = (c.mt * 2 + (int)rank) * BM + quad * 32 + lane;
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * PAIR_BN;
      epilogue_row<PAIR_BN, EPI>(p, c.b, row, c.nt * PAIR_BN, t_addr,
                                 reinterpret_cast<float*>(bar_base + 256) + quad * STAGE_FLOATS);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&tmem_empty[acc]), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1; }
    }
  }

  // Neither CTA leaves (or frees TMEM) while the other may still read its shared memory, write
  // its TMEM or arrive on its barriers.
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, PAIR_TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) atomicExch(p.status, STATUS_TIMEOUT_MBARRIER);
}

// ---------------------------------------------------------------------------------------------
static GemmParams make_params(const GemmLaunch& g) {
  GemmParams p;
  p.bias = (const __nv_bfloat16*)g.bias;
  p.out = g.out;
  p.ldo = g.ldo;
  p.out_batch_rows = g.out_batch_rows;
  p.resid = g.resid;
  p.ldr = g.ldr;
  p.resid_batch_rows = g.resid_batch_rows;
  p.gate = g.gate;
  p.gate_stride = g.gate_stride;
  p.batch = g.batch;
  p.rows = g.rows;
  p.N = g.N;
  p.K = g.K;
  p.status = g.status;
  p.norm_gain = (const __nv_bfloat16*)g.norm_gain;
  p.rope = g.rope;
  p.rope_pos0 = g.rope_pos0;
  p.head_dim = g.head_dim;
  p.norm_cols = g.norm_cols;
  p.rms_eps = g.rms_eps;
  p.norm_out_scale = g.norm_out_scale > 0.f ? g.norm_out_scale : 1.f;
  return p;
}

template <int BN, int EPI>
static int launch_gemm_t(const GemmLaunch& g, cudaStream_t stream) {
  using Cfg = GemmCfg<BN>;
  static PerDeviceInt attr_done;
  auto kern = gemm_bf16_kernel<BN, EPI>;
  if (int rc = ensure_smem_attr(kern, Cfg::SMEM_BYTES, attr_done)) return rc;
  const GemmParams p = make_params(g);
  const int m_tiles = (g.rows + BM - 1) / BM;
  const long long tiles = (long long)g.batch * m_tiles * (g.N / BN);
  const int grid = (int)std::min<long long>(tiles, sm_count());
  kern<<<grid, GEMM_THREADS, Cfg::SMEM_BYTES, stream>>>(g.map_a, g.map_w, p);
  return check_launch();
}

template <int EPI>
static int launch_gemm_pair_t(const GemmLaunch& g, cudaStream_t stream) {
  static PerDeviceInt attr_done;
  auto kern = gemm_bf16_pair_kernel<EPI>;
  if (int rc = ensure_smem_attr(kern, PAIR_SMEM_BYTES, attr_done)) return rc;
  // A persistent grid must be resident all at once: ask how many CTA pairs fit on the device
  // (SMs are handed out to clusters in hardware groups, so it can be fewer than SMs / 2).
  static PerDeviceInt pairs_cache;
  const int dev = current_device();
  int max_pairs = pairs_cache.get(dev);
  if (max_pairs == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (sm_count() / 2), 1, 1);
    cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = PAIR_SMEM_BYTES;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess || n <= 0) {
      set_last_cuda_error((int)e);
      return XEMA_ECUDA;
    }
    max_pairs = std::min(n, sm_count() / 2);
    pairs_cache.set(dev, max_pairs);
  }
  const GemmParams p = make_params(g);
  const int m_tiles = (g.rows + 2 * BM - 1) / (2 * BM);
  const long long tiles = (long long)g.batch * m_tiles * (g.N / PAIR_BN);
  const int pairs = (int)std::min<long long>(tiles, max_pairs);
  kern<<<2 * pairs, GEMM_THREADS, PAIR_SMEM_BYTES, stream>>>(g.map_a, g.map_w, p);
  return check_launch();
}

static int launch_gemm_pair(const GemmLaunch& g, cudaStream_t stream) {
  switch (g.epilogue) {
    case XEMA_EPI_BIAS: return launch_gemm_pair_t<XEMA_EPI_BIAS>(g, stream);
    case XEMA_EPI_BIAS_GELU: return launch_gemm_pair_t<XEMA_EPI_BIAS_GELU>(g, stream);
    case XEMA_EPI_GATE_RES_F32: return launch_gemm_pair_t<XEMA_EPI_GATE_RES_F32>(g, stream);
    case XEMA_EPI_GATE_RES_BF16: return launch_gemm_pair_t<XEMA_EPI_GATE_RES_BF16>(g, stream);
    case XEMA_EPI_BIAS_NORM_ROPE: return launch_gemm_pair_t<XEMA_EPI_BIAS_NORM_ROPE>(g, stream);
    default: return XEMA_EINVAL;
  }
}

template <int BN>
static int launch_gemm_bn(const GemmLaunch& g, cudaStream_t stream) {
  switch (g.epilogue) {
    case XEMA_EPI_BIAS: return launch_gemm_t<BN, XEMA_EPI_BIAS>(g, stream);
    case XEMA_EPI_BIAS_GELU: return launch_gemm_t<BN, XEMA_EPI_BIAS_GELU>(g, stream);
    case XEMA_EPI_GATE_RES_F32: return launch_gemm_t<BN, XEMA_EPI_GATE_RES_F32>(g, stream);
    case XEMA_EPI_GATE_RES_BF16: return launch_gemm_t<BN, XEMA_EPI_GATE_RES_BF16>(g, stream);
    case XEMA_EPI_BIAS_NORM_ROPE: return launch_gemm_t<BN, XEMA_EPI_BIAS_NORM_ROPE>(g, stream);
    default: return XEMA_EINVAL;
  }
}

int launch_gemm(const GemmLaunch& g, cudaStream_t stream) {
  if (g.rows == 0 || g.batch == 0) return XEMA_OK;
  if (g.block_n == 256) return launch_gemm_pair(g, stream);
  if (g.block_n == 128) return launch_gemm_bn<128>(g, stream);
  return XEMA_EINVAL;
}

int gemm_prepare(GemmLaunch* g, const void* a, long long lda, long long a_batch_rows, const void* w, long long ldw) {
  if (g->batch < 1 || g->rows < 0 || g->N < 128 || (g->N % 128) || g->K < 64 || (g->K % 64)) return XEMA_EINVAL;
  if (g->epilogue < XEMA_EPI_BIAS || g->epilogue > XEMA_EPI_BIAS_NORM_ROPE) return XEMA_EINVAL;
  if (!a || !w || !g->bias || !g->out) return XEMA_EINVAL;
  const bool gated = g->epilogue == XEMA_EPI_GATE_RES_F32 || g->epilogue == XEMA_EPI_GATE_RES_BF16;
  if (gated && (!g->resid || !g->gate)) return XEMA_EINVAL;
  if (g->epilogue == XEMA_EPI_BIAS_NORM_ROPE) {
    if (!g->norm_gain || !g->rope || (g->head_dim != 64 && g->head_dim != 128)) return XEMA_EINVAL;
    if (g->norm_cols < 0 || g->norm_cols > g->N || g->norm_cols % g->head_dim || g->N % 256 || g->rope_pos0 < 0)
      return XEMA_EINVAL;
    if ((reinterpret_cast<uintptr_t>(g->norm_gain) & 15) || (reinterpret_cast<uintptr_t>(g->rope) & 15)) return XEMA_EALIGN;
  }
  if ((lda & 7) || (ldw & 7) || (g->ldo & 7) || (gated && (g->ldr & 7))) return XEMA_EALIGN;
  auto mis = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; };
  if (mis(a) || mis(w) || mis(g->bias) || mis(g->out) || (g->resid && mis(g->resid)) || (g->gate && mis(g->gate)))
    return XEMA_EALIGN;
  // tile width from N alone, so the arithmetic of a row never depends on how rows are chunked
  g->block_n = (g->N % 256 == 0) ? 256 : 128;
  int rc = encode_tmap_bf16(&g->map_a, a, g->K, g->rows > 0 ? g->rows : 1, g->batch, lda, a_batch_rows, BM);
  if (rc) return rc;
  // the pair kernel (N % 256 == 0) loads the W tile as two 128-row halves, one per CTA
  return encode_tmap_bf16(&g->map_w, w, g->K, g->N, 1, ldw, g->N, 128);
}

}  // namespace xema
