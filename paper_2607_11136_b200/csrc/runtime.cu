// Executor and C ABI: binds a plan to arena memory, pre-encodes the TMA descriptors, and
// replays the block's launch list on the caller's stream.  Nothing here allocates, frees or
// synchronises device memory.
#include <cuda_bf16.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <unordered_map>
#include <vector>

#include "kernels.h"
#include "planner.h"

namespace xema {

static thread_local int t_last_cuda_error = 0;
void set_last_cuda_error(int code) { t_last_cuda_error = code; }

int current_device() {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

int sm_count() {
  static PerDeviceInt cache;
  const int dev = current_device();
  int n = cache.get(dev);
  if (n > 0) return n;
  if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  cache.set(dev, n);
  return n;
}

int check_launch() {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    t_last_cuda_error = (int)e;
    return XEMA_ECUDA;
  }
  return XEMA_OK;
}

// cuTensorMapEncodeTiled is fetched from the driver at run time so the library has no link
// dependency on libcuda and loads on machines without a driver.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !p) {
      t_last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorUnknown);
      return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int encode_tmap_bf16(CUtensorMap* out, const void* base, long long cols, long long rows, long long batch,
                     long long ld, long long batch_rows, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return XEMA_ECUDA;
  if (cols < 64 || rows < 1 || batch < 1 || ld < cols || box_rows < 1 || box_rows > 256) return XEMA_EINVAL;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (ld & 7)) return XEMA_EALIGN;
  if (batch > 1 && batch_rows < rows) return XEMA_EINVAL;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)batch};
  long long bstride = (batch_rows > 0 ? batch_rows : rows) * ld * 2;
  cuuint64_t strides[2] = {(cuuint64_t)(ld * 2), (cuuint64_t)bstride};
  cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    t_last_cuda_error = (int)r;
    return XEMA_ECUDA;
  }
  return XEMA_OK;
}

// ---------------------------------------------------------------------------------------------
enum OpKind { OP_MOD, OP_LN, OP_ROPE, OP_GEMM, OP_ATTN, OP_FUSED };  // OP_FUSED: done by the previous launch

struct Op {
  OpKind kind;
  char name[8];       // logical op: MOD, LN1A, KV, KROPE, LN1B, Q, QROPE, ATTN, PROJ, LN2, FFN1, FFN2
  int block, chunk;
  double flops;       // algorithmic floating-point operations of this launch
  double bytes;       // algorithmic HBM bytes of this launch (operands read once, results written once)
  // OP_MOD
  const void *temb, *w_mod, *b_mod;
  float* mod;
  // OP_LN
  const void* ln_in;
  int ln_in_f32;
  long long ln_in_batch_rows;
  void* ln_out;
  const float *shift, *scale;
  // OP_ROPE
  void* rope_x;
  long long rope_ld, rope_batch_rows;
  const void* rope_g;
  int pos0;
  // shared
  int rows;
  int batch;          // batch elements this launch covers (OP_LN, OP_ROPE)
  GemmLaunch gemm;
  AttnLaunch attn;
};

}  // namespace xema

using namespace xema;

struct xema_plan {
  xema_config cfg;
  int32_t chunks[3];  // key/value, attention, feed-forward phase
  int32_t axes[3];    // XEMA_SPLIT_ROWS or XEMA_SPLIT_BATCH per phase
  Shard shard;        // sequence-parallel shard this plan covers ({0, 1}: the whole sequence)
  uint64_t guard;     // debug layout: bytes kept free after every tensor (0 in a normal plan)
  std::vector<xema_tensor> tensors;
  std::vector<uint64_t> offsets;
  std::unordered_map<std::string, size_t> index;
  uint64_t peak, live;
  uint32_t n_ops;
  bool bound;
  uint8_t* arena;     // as given to xema_plan_bind
  const float* rope;
  std::vector<Op> ops;
  // xema_forward_host: a second stream and one event per piece of the first and last phase, so
  // that the copies of one piece overlap the launches of its neighbours (made at the first call;
  // concurrent calls on one plan share the arena and are the caller's error anyway)
  mutable cudaStream_t copy_stream = nullptr;
  mutable std::vector<cudaEvent_t> copy_events;
  ~xema_plan() {
    for (cudaEvent_t e : copy_events) cudaEventDestroy(e);
    if (copy_stream) cudaStreamDestroy(copy_stream);
  }
};

static int issue(const xema_plan* pl, const Op& op, cudaStream_t st) {
  const xema_config& c = pl->cfg;
  switch (op.kind) {
    case OP_MOD:
      return launch_mod(op.temb, op.w_mod, op.b_mod, op.mod, c.batch, c.temb_dim, 6 * c.hidden, st);
    case OP_LN:
      return launch_ln_modulate(op.ln_in, op.ln_in_f32, op.ln_in_batch_rows, op.ln_out, op.shift, op.scale,
                                6LL * c.hidden, op.batch, op.rows, c.hidden, c.ln_eps, st);
    case OP_ROPE:
      return launch_rmsnorm_rope(op.rope_x, op.rope_ld, op.rope_batch_rows, op.rope_g, pl->rope, op.pos0, op.batch,
                                 op.rows, c.heads, c.head_dim, c.rms_eps, st);
    case OP_GEMM:
      return launch_gemm(op.gemm, st);
    case OP_ATTN:
      return launch_attention(op.attn, st);
    case OP_FUSED:
      return XEMA_OK;
  }
  return XEMA_EINVAL;
}

static int run_ops(const xema_plan* pl, size_t first, size_t n, void* stream) {
  if (!pl) return XEMA_EINVAL;
  if (!pl->bound) return XEMA_ESTATE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  n = std::min(n, pl->ops.size());
  for (size_t i = first; i < n; ++i) {
    int rc = issue(pl, pl->ops[i], st);
    if (rc) return rc;
  }
  return XEMA_OK;
}

extern "C" {

int xema_plan_create(const xema_config* cfg, int32_t chunks, xema_plan** out) {
  const int32_t c3[3] = {chunks, chunks, chunks};
  return xema_plan_create_phases(cfg, c3, out);
}

int xema_plan_create_phases(const xema_config* cfg, const int32_t chunks[3], xema_plan** out) {
  if (!chunks) return XEMA_EINVAL;
  xema_mitigation m;
  for (int i = 0; i < 3; ++i) {
    m.chunks[i] = chunks[i];
    m.axis[i] = XEMA_SPLIT_ROWS;
  }
  return xema_plan_create_mitigated(cfg, &m, out);
}

int xema_plan_create_mitigated(const xema_config* cfg, const xema_mitigation* m, xema_plan** out) {
  return xema_plan_create_sharded(cfg, m, 0, 1, out);
}

int xema_plan_create_sharded(const xema_config* cfg, const xema_mitigation* m, int32_t shard, int32_t shards,
                             xema_plan** out) {
  return xema_plan_create_guarded(cfg, m, shard, shards, 0, out);
}

int xema_plan_create_guarded(const xema_config* cfg, const xema_mitigation* m, int32_t shard, int32_t shards,
                             uint64_t guard_bytes, xema_plan** out) {
  if (!cfg || !out || !m) return XEMA_EINVAL;
  if (guard_bytes % 256 || guard_bytes > (1ull << 30)) return XEMA_EINVAL;
  *out = nullptr;
  xema_plan* pl = new (std::nothrow) xema_plan();
  if (!pl) return XEMA_ENOSPC;
  pl->cfg = *cfg;
  const int32_t* chunks = m->chunks;
  for (int i = 0; i < 3; ++i) {
    pl->chunks[i] = m->chunks[i];
    pl->axes[i] = m->axis[i];
  }
  pl->bound = false;
  pl->arena = nullptr;
  pl->rope = nullptr;
  pl->shard.p = shard;
  pl->shard.P = shards;
  int rc = build_trace(*cfg, chunks, pl->axes, pl->shard, pl->tensors, &pl->n_ops);
  pl->guard = guard_bytes;
  if (!rc) {
    pl->offsets.assign(pl->tensors.size(), 0);
    if (guard_bytes == 0) {
      rc = plan_arena(pl->tensors.data(), pl->tensors.size(), pl->offsets.data(), &pl->peak, &pl->live);
    } else {
      // lay out tensors that are guard_bytes larger than they are: the bytes after every tensor
      // then belong to nobody for as long as the tensor lives
      std::vector<xema_tensor> padded(pl->tensors);
      for (xema_tensor& t : padded) t.bytes += guard_bytes;
      uint64_t padded_live = 0;
      rc = plan_arena(padded.data(), padded.size(), pl->offsets.data(), &pl->peak, &padded_live);
      pl->live = max_live(pl->tensors.data(), pl->tensors.size());
    }
  }
  if (rc) {
    delete pl;
    return rc;
  }
  for (size_t i = 0; i < pl->tensors.size(); ++i) pl->index[pl->tensors[i].name] = i;
  *out = pl;
  return XEMA_OK;
}

void xema_plan_destroy(xema_plan* plan) { delete plan; }

int xema_plan_info(const xema_plan* plan, uint64_t* peak_bytes, uint64_t* max_live_bytes, size_t* n_tensors,
                   uint32_t* n_ops, int32_t* chunks) {
  if (!plan) return XEMA_EINVAL;
  if (peak_bytes) *peak_bytes = plan->peak;
  if (max_live_bytes) *max_live_bytes = plan->live;
  if (n_tensors) *n_tensors = plan->tensors.size();
  if (n_ops) *n_ops = plan->n_ops;
  if (chunks) *chunks = std::max(plan->chunks[0], std::max(plan->chunks[1], plan->chunks[2]));
  return XEMA_OK;
}

int xema_plan_phase_chunks(const xema_plan* plan, int32_t chunks[3]) {
  if (!plan || !chunks) return XEMA_EINVAL;
  for (int i = 0; i < 3; ++i) chunks[i] = plan->chunks[i];
  return XEMA_OK;
}

int xema_plan_mitigation(const xema_plan* plan, xema_mitigation* m) {
  if (!plan || !m) return XEMA_EINVAL;
  for (int i = 0; i < 3; ++i) {
    m->chunks[i] = plan->chunks[i];
    m->axis[i] = plan->axes[i];
  }
  return XEMA_OK;
}

int xema_plan_shard(const xema_plan* plan, int32_t* shard, int32_t* shards, int64_t* row0, int64_t* rows) {
  if (!plan) return XEMA_EINVAL;
  if (shard) *shard = plan->shard.p;
  if (shards) *shards = plan->shard.P;
  return shard_rows(plan->cfg, plan->shard, row0, rows);
}

uint64_t xema_plan_guard_bytes(const xema_plan* plan) { return plan ? plan->guard : 0; }

int xema_plan_gather_point(const xema_plan* plan, int32_t block, uint32_t* first_op, uint64_t* kv_offset) {
  if (!plan || block < 0 || block >= plan->cfg.n_blocks) return XEMA_EINVAL;
  const uint32_t per_block = 1 + 3 * (uint32_t)plan->chunks[0] + 5 * (uint32_t)plan->chunks[1] + 3 * (uint32_t)plan->chunks[2];
  if (first_op) *first_op = (uint32_t)block * per_block + 1 + 3 * (uint32_t)plan->chunks[0];
  if (kv_offset) {
    auto it = plan->index.find("kv" + std::to_string(block));
    if (it == plan->index.end()) return XEMA_EINVAL;
    *kv_offset = plan->offsets[it->second];
  }
  return XEMA_OK;
}

int xema_plan_tensor(const xema_plan* plan, const char* name, uint64_t* offset, uint64_t* bytes) {
  if (!plan || !name) return XEMA_EINVAL;
  auto it = plan->index.find(name);
  if (it == plan->index.end()) return XEMA_EINVAL;
  if (offset) *offset = plan->offsets[it->second];
  if (bytes) *bytes = plan->tensors[it->second].bytes;
  return XEMA_OK;
}

int xema_plan_tensor_at(const xema_plan* plan, size_t i, xema_tensor* tensor, uint64_t* offset) {
  if (!plan || i >= plan->tensors.size()) return XEMA_EINVAL;
  if (tensor) *tensor = plan->tensors[i];
  if (offset) *offset = plan->offsets[i];
  return XEMA_OK;
}

int xema_plan_bind(xema_plan* plan, void* arena_dev, uint64_t arena_bytes, const xema_block_weights* weights,
                   const float* rope_dev, void* status_dev) {
  if (!plan || !arena_dev || !weights || !rope_dev) return XEMA_EINVAL;
  if (arena_bytes < plan->peak) return XEMA_ENOSPC;
  if (reinterpret_cast<uintptr_t>(arena_dev) & 255) return XEMA_EALIGN;
  if (reinterpret_cast<uintptr_t>(rope_dev) & 15) return XEMA_EALIGN;
  const xema_config& c = plan->cfg;
  if (c.hidden % 256 || c.ffn % 256 || c.temb_dim % 8 || (c.head_dim != 64 && c.head_dim != 128))
    return XEMA_EINVAL;
  plan->bound = false;
  plan->ops.clear();
  plan->rope = rope_dev;
  plan->arena = static_cast<uint8_t*>(arena_dev);
  uint8_t* arena = static_cast<uint8_t*>(arena_dev);
  unsigned int* status = static_cast<unsigned int*>(status_dev);

  auto at = [&](const char* stem, int block, int chunk) -> uint8_t* {
    char name[32];
    if (block < 0)
      std::snprintf(name, sizeof(name), "%s", stem);
    else if (chunk < 0)
      std::snprintf(name, sizeof(name), "%s%d", stem, block);
    else
      std::snprintf(name, sizeof(name), "%s%d_%d", stem, block, chunk);
    auto it = plan->index.find(name);
    if (it == plan->index.end()) return nullptr;
    const size_t i = it->second;
    if (plan->offsets[i] + plan->tensors[i].bytes > arena_bytes) return nullptr;
    return arena + plan->offsets[i];
  };

  // S: the token rows this plan covers (the owned rows of its shard; all of them without
  // sharding), row0: the first of them; S_all: every row -- the keys and values of all shards
  const long long S_all = seq_len(c), D = c.hidden, F = c.ffn;
  int64_t row0_ = 0, rows_ = 0;
  if (shard_rows(c, plan->shard, &row0_, &rows_)) return XEMA_EINVAL;
  const long long S = rows_, row0 = row0_;
  const int CA = plan->chunks[0], CB = plan->chunks[1], CC = plan->chunks[2];
  for (int l = 0; l < c.n_blocks; ++l) {
    const xema_block_weights& w = weights[l];
    const void* wp[12] = {w.w_mod, w.b_mod, w.w_qkv, w.b_qkv, w.g_q, w.g_k, w.w_o, w.b_o, w.w_1, w.b_1, w.w_2, w.b_2};
    for (const void* p : wp) {
      if (!p) return XEMA_EINVAL;
      if (reinterpret_cast<uintptr_t>(p) & 15) return XEMA_EALIGN;
    }
    const __nv_bfloat16* w_qkv = static_cast<const __nv_bfloat16*>(w.w_qkv);
    const __nv_bfloat16* b_qkv = static_cast<const __nv_bfloat16*>(w.b_qkv);
    uint8_t* hid = at("hid", l, -1);
    uint8_t* hid_next = at("hid", l + 1, -1);
    float* mod = reinterpret_cast<float*>(at("mod", l, -1));
    uint8_t* kv = at("kv", l, -1);
    uint8_t* res = at("res", l, -1);
    uint8_t* temb = at("temb", -1, -1);
    if (!hid || !hid_next || !mod || !kv || !res || !temb) return XEMA_EINVAL;

    Op op{};
    op.kind = OP_MOD;
    op.temb = temb; op.w_mod = w.w_mod; op.b_mod = w.b_mod; op.mod = mod;
    const double Bd = c.batch, Dd = (double)D, Fd = (double)F, Sd = (double)S_all;
    auto tag = [&](Op& o, const char* nm, int chunk, double flops, double bytes) {
      std::snprintf(o.name, sizeof(o.name), "%s", nm);
      o.block = l; o.chunk = chunk; o.flops = flops; o.bytes = bytes;
    };
    tag(op, "MOD", -1, 2.0 * Bd * 6 * Dd * c.temb_dim, 2.0 * 6 * Dd * c.temb_dim + 24.0 * Bd * Dd);
    plan->ops.push_back(op);

    // A piece of a phase: batch elements [b0, b0 + nb) x rows [r0, r0 + n).
    struct Piece {
      long long b0, r0;
      int nb, n;
    };
    auto piece_of = [&](int phase, int ci) {
      const int C = plan->chunks[phase];
      Piece pc;
      if (plan->axes[phase] == XEMA_SPLIT_BATCH) {
        pc.b0 = (long long)ci * c.batch / C;
        pc.nb = (int)((long long)(ci + 1) * c.batch / C - pc.b0);
        pc.r0 = 0;
        pc.n = (int)S;
      } else {
        pc.b0 = 0;
        pc.nb = c.batch;
        pc.r0 = (long long)ci * S / C;
        pc.n = (int)((long long)(ci + 1) * S / C - pc.r0);
      }
      return pc;
    };
    // byte offset of (batch b0, row r0) in a [B, S, width] tensor over the plan's rows, and in the
    // [B, S_all, 2D] keys-and-values tensor, whose rows are global
    auto at_row = [&](const Piece& pc, long long width, int elem_bytes) { return (pc.b0 * S + pc.r0) * width * elem_bytes; };
    auto at_kv_row = [&](const Piece& pc) { return (pc.b0 * S_all + row0 + pc.r0) * 2 * D * 2; };
    auto ln_op = [&](const void* in, int f32, void* out, const Piece& pc, int which, const char* nm, int chunk) {
      Op o{};
      o.kind = OP_LN;
      const double elems = (double)pc.nb * pc.n;
      tag(o, nm, chunk, 8.0 * elems * Dd, elems * Dd * (f32 ? 6.0 : 4.0));
      o.ln_in = in; o.ln_in_f32 = f32; o.ln_in_batch_rows = S; o.ln_out = out;
      o.shift = mod + pc.b0 * 6 * D + (which == 1 ? 0 : 3 * D);
      o.scale = mod + pc.b0 * 6 * D + (which == 1 ? D : 4 * D);
      o.rows = pc.n;
      o.batch = pc.nb;
      plan->ops.push_back(o);
    };
    auto gemm_op = [&](const void* a, long long lda, long long a_batch_rows, const void* wt, long long ldw,
                       const void* bias, void* out, long long ldo, long long out_batch_rows, const void* resid,
                       long long ldr, long long resid_batch_rows, const float* gate, const Piece& pc, int N, int K,
                       int epi, const char* nm, int chunk, const void* norm_gain = nullptr, int norm_cols = 0,
                       int pos0 = 0, float norm_out_scale = 1.f) -> int {
      const int rows = pc.n;
      const double Bd = (double)pc.nb;
      Op o{};
      o.kind = OP_GEMM;
      o.gemm.norm_gain = norm_gain; o.gemm.rope = rope_dev; o.gemm.rope_pos0 = pos0; o.gemm.head_dim = c.head_dim;
      o.gemm.norm_cols = norm_cols; o.gemm.rms_eps = c.rms_eps; o.gemm.norm_out_scale = norm_out_scale;
      {
        const double out_b = (epi == XEMA_EPI_GATE_RES_F32) ? 4.0 : 2.0;
        const double res_b = (epi == XEMA_EPI_GATE_RES_F32) ? 2.0 : (epi == XEMA_EPI_GATE_RES_BF16 ? 4.0 : 0.0);
        tag(o, nm, chunk, 2.0 * Bd * rows * (double)N * K,
            2.0 * Bd * rows * K + 2.0 * (double)N * K + (out_b + res_b) * Bd * rows * N);
      }
      GemmLaunch& g = o.gemm;
      g.bias = bias; g.out = out; g.ldo = ldo; g.out_batch_rows = out_batch_rows;
      g.resid = resid; g.ldr = ldr; g.resid_batch_rows = resid_batch_rows;
      g.gate = gate; g.gate_stride = 6 * D;
      g.batch = pc.nb; g.rows = rows; g.N = N; g.K = K; g.epilogue = epi; g.status = status;
      int rc = gemm_prepare(&g, a, lda, a_batch_rows, wt, ldw);
      if (rc) return rc;
      plan->ops.push_back(o);
      return XEMA_OK;
    };

    // phase A: keys and values of every piece
    for (int ci = 0; ci < CA; ++ci) {
      const Piece pc = piece_of(0, ci);
      const int n = pc.n;
      uint8_t* h1a = at("h1a", l, ci);
      if (!h1a) return XEMA_EINVAL;
      uint8_t* kv_pc = kv + at_kv_row(pc);
      ln_op(hid + at_row(pc, D, 2), 0, h1a, pc, 1, "LN1A", ci);
      // K half: RMSNorm * g_k + RoPE in the GEMM epilogue; the KROPE op of the trace is then
      // a placeholder (the fused kernel touches a subset of what the trace says is live)
      int rc = gemm_op(h1a, D, n, w_qkv + D * D, D, b_qkv + D, kv_pc, 2 * D, S_all, nullptr, 0, 0, nullptr,
                       pc, (int)(2 * D), (int)D, XEMA_EPI_BIAS_NORM_ROPE, "KV", ci, w.g_k, (int)D, (int)(row0 + pc.r0));
      if (rc) return rc;
      Op o{};
      o.kind = OP_FUSED;
      tag(o, "KROPE", ci, 0.0, 0.0);
      o.rope_x = kv_pc; o.rope_ld = 2 * D; o.rope_batch_rows = S_all; o.rope_g = w.g_k;
      o.pos0 = (int)(row0 + pc.r0); o.rows = n; o.batch = pc.nb;
      plan->ops.push_back(o);
    }
    // The queries leave their projection already multiplied by log2(e) / sqrt(head_dim), inside the
    // epilogue that rounds them to bf16 (one rounding, as before): the attention's scores are then
    // exponents to base 2 as they come out of the tensor core.
    const float q_scale = 1.4426950408889634f / std::sqrt((float)c.head_dim);
    // phase B: queries, attention and the gated output projection of every piece
    for (int ci = 0; ci < CB; ++ci) {
      const Piece pc = piece_of(1, ci);
      const int n = pc.n;
      const double Bd = (double)pc.nb;
      uint8_t* h1b = at("h1b", l, ci);
      uint8_t* q = at("q", l, ci);
      uint8_t* o_t = at("o", l, ci);
      float* lse = reinterpret_cast<float*>(at("lse", l, ci));
      if (!h1b || !q || !o_t || !lse) return XEMA_EINVAL;
      const uint8_t* hid_pc = hid + at_row(pc, D, 2);
      const uint8_t* kv_b = kv + pc.b0 * S_all * 2 * D * 2;      // keys and values of these batch elements
      ln_op(hid_pc, 0, h1b, pc, 1, "LN1B", ci);
      // With one piece in both phases LN1B recomputes what LN1A wrote.  When the layout put h1b
      // at h1a's address and nothing was born in between (KROPE allocates nothing, so the only
      // births since the KV op are h1b's own), those bytes are still there: the launch is elided.
      if (CA == 1 && CB == 1 && h1b == at("h1a", l, 0)) {
        bool untouched = true;
        const size_t ia = plan->index.at(std::string("h1a") + std::to_string(l) + "_0");
        const size_t ib = plan->index.at(std::string("h1b") + std::to_string(l) + "_0");
        const xema_tensor& ta = plan->tensors[ia];
        const xema_tensor& tb = plan->tensors[ib];
        for (size_t i = 0; i < plan->tensors.size() && untouched; ++i) {
          if (i == ia || i == ib) continue;
          const xema_tensor& tt = plan->tensors[i];
          const bool born_between = tt.birth >= ta.death && tt.birth <= tb.birth;
          const bool overlaps = plan->offsets[i] < plan->offsets[ia] + ta.bytes && plan->offsets[ia] < plan->offsets[i] + tt.bytes;
          if (born_between && overlaps) untouched = false;
        }
        if (untouched && ta.bytes == tb.bytes) {
          plan->ops.back().kind = OP_FUSED;
          plan->ops.back().flops = 0.0;
          plan->ops.back().bytes = 0.0;
        }
      }
      int rc = gemm_op(h1b, D, n, w_qkv, D, b_qkv, q, D, n, nullptr, 0, 0, nullptr, pc, (int)D, (int)D,
                       XEMA_EPI_BIAS_NORM_ROPE, "Q", ci, w.g_q, (int)D, (int)(row0 + pc.r0), q_scale);
      if (rc) return rc;
      Op o{};
      o.kind = OP_FUSED;
      tag(o, "QROPE", ci, 0.0, 0.0);
      o.rope_x = q; o.rope_ld = D; o.rope_batch_rows = n; o.rope_g = w.g_q; o.pos0 = (int)(row0 + pc.r0); o.rows = n;
      o.batch = pc.nb;
      plan->ops.push_back(o);
      Op a{};
      a.kind = OP_ATTN;
      // q and o once, k and v once per launch, lse
      tag(a, "ATTN", ci, 4.0 * Bd * n * Sd * Dd, 4.0 * Bd * n * Dd + 4.0 * Bd * Sd * Dd + 4.0 * Bd * c.heads * n);
      a.attn.o = o_t; a.attn.lse = lse; a.attn.batch = pc.nb; a.attn.rows = n; a.attn.keys = (int)S_all;
      a.attn.heads = c.heads; a.attn.head_dim = c.head_dim; a.attn.status = status; a.attn.q_scale = 1.f;
      a.attn.gain_q = w.g_q; a.attn.gain_k = w.g_k;     // q and k come out of the fused RMSNorm + RoPE epilogues
      rc = attn_prepare(&a.attn, q, D, n, kv_b, kv_b + D * 2, 2 * D, S_all);
      if (rc) return rc;
      plan->ops.push_back(a);
      rc = gemm_op(o_t, D, n, w.w_o, D, w.b_o, res + at_row(pc, D, 4), D, S, hid_pc, D, S,
                   mod + pc.b0 * 6 * D + 2 * D, pc, (int)D, (int)D, XEMA_EPI_GATE_RES_F32, "PROJ", ci);
      if (rc) return rc;
    }
    // phase C: feed-forward of every piece
    for (int ci = 0; ci < CC; ++ci) {
      const Piece pc = piece_of(2, ci);
      const int n = pc.n;
      uint8_t* h2 = at("h2", l, ci);
      uint8_t* g = at("g", l, ci);
      if (!h2 || !g) return XEMA_EINVAL;
      uint8_t* res_pc = res + at_row(pc, D, 4);
      ln_op(res_pc, 1, h2, pc, 2, "LN2", ci);
      int rc = gemm_op(h2, D, n, w.w_1, D, w.b_1, g, F, n, nullptr, 0, 0, nullptr, pc, (int)F, (int)D,
                       XEMA_EPI_BIAS_GELU, "FFN1", ci);
      if (rc) return rc;
      rc = gemm_op(g, F, n, w.w_2, F, w.b_2, hid_next + at_row(pc, D, 2), D, S, res_pc, D, S,
                   mod + pc.b0 * 6 * D + 5 * D, pc, (int)D, (int)F, XEMA_EPI_GATE_RES_BF16, "FFN2", ci);
      if (rc) return rc;
    }
  }
  if (plan->ops.size() != plan->n_ops) return XEMA_EINVAL;
  plan->bound = true;
  return XEMA_OK;
}

int xema_block_forward(const xema_plan* plan, void* stream) {
  if (!plan) return XEMA_EINVAL;
  if (plan->cfg.n_blocks != 1) return XEMA_ESTATE;
  return run_ops(plan, 0, plan->ops.size(), stream);
}

int xema_step_forward(const xema_plan* plan, void* stream) {
  if (!plan) return XEMA_EINVAL;
  return run_ops(plan, 0, plan->ops.size(), stream);
}

// One piece of a [B, rows, D] bf16 tensor (rows [r0, r0 + rows) of `batch` consecutive batch
// elements, the first at `dev`) between the arena and the host copy of the whole tensor.
static cudaError_t copy_piece(uint8_t* tensor_dev, uint8_t* tensor_host, const uint8_t* dev, int batch, int rows,
                              long long row_elems, long long batch_rows, bool to_host, cudaStream_t st) {
  const size_t off = (size_t)(dev - tensor_dev), pitch = (size_t)batch_rows * row_elems * 2,
               width = (size_t)rows * row_elems * 2;
  if (to_host)
    return cudaMemcpy2DAsync(tensor_host + off, pitch, tensor_dev + off, pitch, width, batch, cudaMemcpyDeviceToHost, st);
  return cudaMemcpy2DAsync(tensor_dev + off, pitch, tensor_host + off, pitch, width, batch, cudaMemcpyHostToDevice, st);
}

int xema_forward_host(const xema_plan* plan, const void* hid_in_host, const void* temb_host, void* hid_out_host,
                      void* stream) {
  if (!plan || !hid_in_host || !temb_host || !hid_out_host) return XEMA_EINVAL;
  if (!plan->bound) return XEMA_ESTATE;
  const xema_config& c = plan->cfg;
  char out_name[32];
  std::snprintf(out_name, sizeof(out_name), "hid%d", c.n_blocks);
  auto i_in = plan->index.find("hid0"), i_temb = plan->index.find("temb"), i_out = plan->index.find(out_name);
  if (i_in == plan->index.end() || i_temb == plan->index.end() || i_out == plan->index.end()) return XEMA_EINVAL;
  // exact sizes (the planned sizes are rounded up to 256 bytes; the caller's buffers are not)
  int64_t own_rows = 0;
  if (shard_rows(c, plan->shard, nullptr, &own_rows)) return XEMA_EINVAL;
  if (plan->shard.P != 1) return XEMA_ESTATE;   // a shard's step needs the caller's exchange in the middle
  const size_t hid_bytes = (size_t)2 * c.batch * (size_t)own_rows * c.hidden;
  const size_t temb_bytes = (size_t)2 * c.batch * c.temb_dim;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* in_dev = plan->arena + plan->offsets[i_in->second];
  uint8_t* out_dev = plan->arena + plan->offsets[i_out->second];
  uint8_t* in_host = static_cast<uint8_t*>(const_cast<void*>(hid_in_host));
  uint8_t* out_host = static_cast<uint8_t*>(hid_out_host);
  const std::vector<Op>& ops = plan->ops;
  const size_t n = ops.size();
  cudaError_t e = cudaSuccess;
  auto fail = [&](cudaError_t err) {
    t_last_cuda_error = (int)err;
    return XEMA_ECUDA;
  };

  // The pieces of the first block's key/value phase read the input piece by piece (LN1A of piece c
  // reads the rows of piece c only), and the pieces of the last block's feed-forward phase finish
  // the output piece by piece (FFN2 of piece c).  With more than one piece in either phase the
  // copies run on a second stream, ordered by events: the input of piece c + 1 arrives while
  // piece c is worked on, the output of piece c leaves while piece c + 1 is worked on.  Bits do
  // not depend on it.  With one piece the copy is a plain one on the caller's stream.
  std::vector<size_t> in_ops, out_ops;      // LN1A launches of block 0, FFN2 launches of the last block
  for (size_t i = 0; i < n; ++i) {
    if (ops[i].kind == OP_LN && ops[i].block == 0 && !std::strcmp(ops[i].name, "LN1A")) in_ops.push_back(i);
    if (ops[i].kind == OP_GEMM && ops[i].block == c.n_blocks - 1 && !std::strcmp(ops[i].name, "FFN2")) out_ops.push_back(i);
  }
  const bool row_major_out = !out_ops.empty() && ops[out_ops[0]].gemm.ldo == c.hidden;
  const bool split_in = in_ops.size() > 1, split_out = out_ops.size() > 1 && row_major_out;
  const size_t n_events = (split_in ? in_ops.size() : 0) + (split_out ? out_ops.size() : 0) + 1;
  if (split_in || split_out) {
    if (!plan->copy_stream && (e = cudaStreamCreateWithFlags(&plan->copy_stream, cudaStreamNonBlocking)) != cudaSuccess)
      return fail(e);
    while (plan->copy_events.size() < n_events) {
      cudaEvent_t ev;
      if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return fail(e);
      plan->copy_events.push_back(ev);
    }
  }
  size_t next_event = 0;
  cudaStream_t cs = plan->copy_stream;

  // ---- input
  if ((e = cudaMemcpyAsync(plan->arena + plan->offsets[i_temb->second], temb_host, temb_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return fail(e);
  std::vector<cudaEvent_t> in_ready(in_ops.size(), nullptr);
  if (!split_in) {
    if ((e = cudaMemcpyAsync(in_dev, in_host, hid_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail(e);
  } else {
    // the copy stream starts where the caller's stream stands (the arena may still be in use by
    // work enqueued before this call)
    cudaEvent_t start = plan->copy_events[next_event++];
    if ((e = cudaEventRecord(start, st)) != cudaSuccess || (e = cudaStreamWaitEvent(cs, start, 0)) != cudaSuccess) return fail(e);
    for (size_t k = 0; k < in_ops.size(); ++k) {
      const Op& o = ops[in_ops[k]];
      e = copy_piece(in_dev, in_host, static_cast<const uint8_t*>(o.ln_in), o.batch, o.rows, c.hidden, o.ln_in_batch_rows,
                     false, k == 0 ? st : cs);
      if (e != cudaSuccess) return fail(e);
      if (k > 0) {
        in_ready[k] = plan->copy_events[next_event++];
        if ((e = cudaEventRecord(in_ready[k], cs)) != cudaSuccess) return fail(e);
      }
    }
  }

  // ---- launches, with the waits for input pieces and the copies of finished output pieces
  size_t k_in = 0, k_out = 0;
  for (size_t i = 0; i < n; ++i) {
    if (split_in && k_in < in_ops.size() && i == in_ops[k_in]) {
      if (in_ready[k_in] && (e = cudaStreamWaitEvent(st, in_ready[k_in], 0)) != cudaSuccess) return fail(e);
      ++k_in;
    }
    int rc = issue(plan, ops[i], st);
    if (rc) return rc;
    if (split_out && k_out < out_ops.size() && i == out_ops[k_out]) {
      const Op& o = ops[i];
      const bool last = (k_out + 1 == out_ops.size());
      if (!last) {
        cudaEvent_t ev = plan->copy_events[next_event++];
        if ((e = cudaEventRecord(ev, st)) != cudaSuccess || (e = cudaStreamWaitEvent(cs, ev, 0)) != cudaSuccess) return fail(e);
      }
      e = copy_piece(out_dev, out_host, static_cast<const uint8_t*>(o.gemm.out), o.gemm.batch, o.gemm.rows, c.hidden,
                     o.gemm.out_batch_rows, true, last ? st : cs);
      if (e != cudaSuccess) return fail(e);
      ++k_out;
    }
  }
  if (!split_out) {
    if ((e = cudaMemcpyAsync(out_host, out_dev, hid_bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return fail(e);
  }
  if (split_in || split_out) {
    // the caller's stream ends after everything the copy stream was given
    cudaEvent_t ev = plan->copy_events[next_event++];
    if ((e = cudaEventRecord(ev, cs)) != cudaSuccess || (e = cudaStreamWaitEvent(st, ev, 0)) != cudaSuccess) return fail(e);
  }
  return XEMA_OK;
}

int xema_forward_prefix(const xema_plan* plan, uint32_t n_logical_ops, void* stream) {
  return run_ops(plan, 0, n_logical_ops, stream);
}

int xema_forward_range(const xema_plan* plan, uint32_t first_op, uint32_t end_op, void* stream) {
  if (first_op > end_op) return XEMA_EINVAL;
  return run_ops(plan, first_op, end_op, stream);
}

int xema_plan_op(const xema_plan* plan, uint32_t i, char* name8, int32_t* block, int32_t* chunk, double* flops,
                 double* bytes) {
  if (!plan) return XEMA_EINVAL;
  if (!plan->bound) return XEMA_ESTATE;
  if (i >= plan->ops.size()) return XEMA_EINVAL;
  const Op& o = plan->ops[i];
  if (name8) std::memcpy(name8, o.name, 8);
  if (block) *block = o.block;
  if (chunk) *chunk = o.chunk;
  if (flops) *flops = o.flops;
  if (bytes) *bytes = o.bytes;
  return XEMA_OK;
}

int xema_plan_launch_count(const xema_plan* plan) {
  if (!plan || !plan->bound) return 0;
  int n = 0;
  for (const Op& o : plan->ops) n += o.kind != OP_FUSED;
  return n;
}

int xema_op_mod(const void* temb, const void* w_mod, const void* b_mod, float* mod, int32_t batch, int32_t temb_dim,
                int32_t n_out, void* stream) {
  if (!temb || !w_mod || !b_mod || !mod) return XEMA_EINVAL;
  return launch_mod(temb, w_mod, b_mod, mod, batch, temb_dim, n_out, reinterpret_cast<cudaStream_t>(stream));
}

int xema_op_ln_modulate(const void* in, int32_t in_is_f32, int64_t in_batch_rows, void* out, const float* shift,
                        const float* scale, int64_t mod_stride, int32_t batch, int32_t rows, int32_t D, float eps,
                        void* stream) {
  if (!in || !out || !shift || !scale) return XEMA_EINVAL;
  return launch_ln_modulate(in, in_is_f32, in_batch_rows, out, shift, scale, mod_stride, batch, rows, D, eps,
                            reinterpret_cast<cudaStream_t>(stream));
}

int xema_op_rmsnorm_rope(void* x, int64_t ld, int64_t batch_rows, const void* g, const float* rope, int32_t pos0,
                         int32_t batch, int32_t rows, int32_t heads, int32_t head_dim, float eps, void* stream) {
  if (!x || !g || !rope) return XEMA_EINVAL;
  return launch_rmsnorm_rope(x, ld, batch_rows, g, rope, pos0, batch, rows, heads, head_dim, eps,
                             reinterpret_cast<cudaStream_t>(stream));
}

int xema_op_gemm(const xema_gemm_args* a, void* status_dev, void* stream) {
  if (!a) return XEMA_EINVAL;
  GemmLaunch g{};
  g.bias = a->bias; g.out = a->out; g.ldo = a->ldo; g.out_batch_rows = a->out_batch_rows;
  g.resid = a->resid; g.ldr = a->ldr; g.resid_batch_rows = a->resid_batch_rows;
  g.gate = a->gate; g.gate_stride = a->gate_stride;
  g.batch = a->batch; g.rows = a->rows; g.N = a->N; g.K = a->K; g.epilogue = a->epilogue;
  g.norm_gain = a->norm_gain; g.rope = a->rope; g.rope_pos0 = a->rope_pos0; g.head_dim = a->head_dim;
  g.norm_cols = a->norm_cols; g.rms_eps = a->rms_eps; g.norm_out_scale = a->norm_out_scale;
  g.status = static_cast<unsigned int*>(status_dev);
  int rc = gemm_prepare(&g, a->a, a->lda, a->a_batch_rows, a->w, a->ldw);
  if (rc) return rc;
  return launch_gemm(g, reinterpret_cast<cudaStream_t>(stream));
}

int xema_op_attention(const void* q, int64_t ldq, int64_t q_batch_rows, const void* k, const void* v, int64_t ldkv,
                      int64_t kv_batch_rows, void* o, float* lse, int32_t batch, int32_t rows, int32_t keys,
                      int32_t heads, int32_t head_dim, float q_scale, void* status_dev, void* stream) {
  if (!(q_scale > 0.f)) return XEMA_EINVAL;
  AttnLaunch a{};
  a.o = o; a.lse = lse; a.batch = batch; a.rows = rows; a.keys = keys; a.heads = heads; a.head_dim = head_dim;
  a.q_scale = q_scale;
  a.status = static_cast<unsigned int*>(status_dev);
  int rc = attn_prepare(&a, q, ldq, q_batch_rows, k, v, ldkv, kv_batch_rows);
  if (rc) return rc;
  return launch_attention(a, reinterpret_cast<cudaStream_t>(stream));
}

int xema_last_cuda_error(void) { return t_last_cuda_error; }

}  // extern "C"
