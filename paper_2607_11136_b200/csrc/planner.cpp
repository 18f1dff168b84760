// Host-side planner: lifetime trace of the chunked DiT block template, Algorithm 1
// (offline static memory layout) and the smallest-chunk-count search.  Pure integer code.
#include "planner.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>

namespace xema {

static inline uint64_t align256(uint64_t n) { return (n + 255u) & ~uint64_t(255); }

int validate_config(const xema_config& c) {
  if (c.batch < 1 || c.s_text < 0 || c.grid_t < 1 || c.grid_h < 1 || c.grid_w < 1) return XEMA_EINVAL;
  if (c.hidden < 1 || c.heads < 1 || c.head_dim < 1 || c.ffn < 1 || c.temb_dim < 1) return XEMA_EINVAL;
  if ((int64_t)c.heads * c.head_dim != c.hidden) return XEMA_EINVAL;
  if (c.rope_dim_t < 0 || c.rope_dim_h < 0 || c.rope_dim_w < 0) return XEMA_EINVAL;
  if ((c.rope_dim_t | c.rope_dim_h | c.rope_dim_w) & 1) return XEMA_EINVAL;
  if (c.rope_dim_t + c.rope_dim_h + c.rope_dim_w != c.head_dim) return XEMA_EINVAL;
  if (c.n_blocks < 1) return XEMA_EINVAL;
  if (!(c.rope_base > 0.f) || !(c.ln_eps >= 0.f) || !(c.rms_eps >= 0.f)) return XEMA_EINVAL;
  int64_t s = (int64_t)c.s_text + (int64_t)c.grid_t * c.grid_h * c.grid_w;
  if (s < 1 || s > (int64_t)1 << 30) return XEMA_EINVAL;
  return XEMA_OK;
}

int64_t seq_len(const xema_config& c) {
  return (int64_t)c.s_text + (int64_t)c.grid_t * c.grid_h * c.grid_w;
}

// Index of a logical op inside block l.  Phase A holds 3 ops per chunk, phase B 5, phase C 3.
struct OpIndex {
  uint32_t base;  // index of MOD of this block
  uint32_t CA, CB, CC;  // chunks of the key/value, attention and feed-forward phases
  uint32_t mod() const { return base; }
  uint32_t ln1a(uint32_t c) const { return base + 1 + 3 * c; }
  uint32_t kv(uint32_t c) const { return ln1a(c) + 1; }
  uint32_t krope(uint32_t c) const { return ln1a(c) + 2; }
  uint32_t ln1b(uint32_t c) const { return base + 1 + 3 * CA + 5 * c; }
  uint32_t q(uint32_t c) const { return ln1b(c) + 1; }
  uint32_t qrope(uint32_t c) const { return ln1b(c) + 2; }
  uint32_t attn(uint32_t c) const { return ln1b(c) + 3; }
  uint32_t proj(uint32_t c) const { return ln1b(c) + 4; }
  uint32_t ln2(uint32_t c) const { return base + 1 + 3 * CA + 5 * CB + 3 * c; }
  uint32_t ffn1(uint32_t c) const { return ln2(c) + 1; }
  uint32_t ffn2(uint32_t c) const { return ln2(c) + 2; }
};

static xema_tensor make(const char* stem, int block, int chunk, uint32_t kind, uint32_t dtype,
                        uint64_t bytes, uint32_t birth, uint32_t death) {
  xema_tensor t;
  std::memset(&t, 0, sizeof(t));
  if (block < 0)
    std::snprintf(t.name, sizeof(t.name), "%s", stem);
  else if (chunk < 0)
    std::snprintf(t.name, sizeof(t.name), "%s%d", stem, block);
  else
    std::snprintf(t.name, sizeof(t.name), "%s%d_%d", stem, block, chunk);
  t.kind = kind;
  t.dtype = dtype;
  t.block = block;
  t.chunk = chunk;
  t.bytes = align256(bytes);
  t.birth = birth;
  t.death = death;
  return t;
}

int build_trace(const xema_config& cfg, int32_t chunks, std::vector<xema_tensor>& out, uint32_t* n_ops) {
  const int32_t c3[3] = {chunks, chunks, chunks};
  return build_trace(cfg, c3, out, n_ops);
}

int build_trace(const xema_config& cfg, const int32_t chunks[3], std::vector<xema_tensor>& out, uint32_t* n_ops) {
  const int32_t axes[3] = {XEMA_SPLIT_ROWS, XEMA_SPLIT_ROWS, XEMA_SPLIT_ROWS};
  return build_trace(cfg, chunks, axes, out, n_ops);
}

int build_trace(const xema_config& cfg, const int32_t chunks[3], const int32_t axes[3], std::vector<xema_tensor>& out,
                uint32_t* n_ops) {
  return build_trace(cfg, chunks, axes, Shard{}, out, n_ops);
}

int shard_rows(const xema_config& cfg, Shard sh, int64_t* row0, int64_t* rows) {
  const int64_t S = seq_len(cfg);
  if (sh.P < 1 || sh.p < 0 || sh.p >= sh.P || sh.P > S) return XEMA_EINVAL;
  const int64_t r0 = (int64_t)sh.p * S / sh.P;
  if (row0) *row0 = r0;
  if (rows) *rows = (int64_t)(sh.p + 1) * S / sh.P - r0;
  return XEMA_OK;
}

int build_trace(const xema_config& cfg, const int32_t chunks[3], const int32_t axes[3], Shard sh,
                std::vector<xema_tensor>& out, uint32_t* n_ops) {
  int rc = validate_config(cfg);
  if (rc) return rc;
  const int64_t S_all = seq_len(cfg);
  int64_t S = 0;                       // rows this trace covers: the owned rows of the shard
  rc = shard_rows(cfg, sh, nullptr, &S);
  if (rc) return rc;
  for (int i = 0; i < 3; ++i) {
    if (axes[i] != XEMA_SPLIT_ROWS && axes[i] != XEMA_SPLIT_BATCH) return XEMA_EINVAL;
    if (chunks[i] < 1 || chunks[i] > (axes[i] == XEMA_SPLIT_BATCH ? (int64_t)cfg.batch : S)) return XEMA_EINVAL;
  }
  const uint64_t B = cfg.batch, D = cfg.hidden, H = cfg.heads, F = cfg.ffn, Dt = cfg.temb_dim;
  const uint32_t CA = (uint32_t)chunks[0], CB = (uint32_t)chunks[1], CC = (uint32_t)chunks[2];
  const uint32_t L = (uint32_t)cfg.n_blocks;
  const uint32_t ops_per_block = 1 + 3 * CA + 5 * CB + 3 * CC;
  const uint32_t total_ops = L * ops_per_block;
  const uint64_t u = 2 * B * (uint64_t)S * D;           // one bf16 hidden tensor over the owned rows
  const uint64_t u_all = 2 * B * (uint64_t)S_all * D;   // ... over every row: keys and values of all shards
  // rows x batch elements of piece c of a phase split C ways along its axis
  auto elems_of = [&](uint32_t c, uint32_t C, int phase) {
    if (axes[phase] == XEMA_SPLIT_BATCH)
      return (uint64_t)((int64_t)(c + 1) * (int64_t)B / C - (int64_t)c * (int64_t)B / C) * (uint64_t)S;
    return B * (uint64_t)((int64_t)(c + 1) * S / C - (int64_t)c * S / C);
  };

  out.clear();
  out.reserve((size_t)L * (4 + 2 * CA + 4 * CB + 2 * CC) + 2);
  // Emitted directly in id order: ascending birth; tensors born at the same op follow the
  // order temb, hid, mod, kv, h1a, h1b, q, o, lse, res, h2, g.
  OpIndex last{(L - 1) * ops_per_block, CA, CB, CC};
  out.push_back(make("temb", -1, -1, XEMA_KIND_INPUT, XEMA_DTYPE_BF16, 2 * B * Dt, 0, last.mod() + 1));
  for (uint32_t l = 0; l < L; ++l) {
    OpIndex op{l * ops_per_block, CA, CB, CC};
    if (l == 0) {
      // the block input is read by LN1A/LN1B and as the residual of PROJ
      uint32_t kind = XEMA_KIND_INPUT;
      out.push_back(make("hid", 0, -1, kind, XEMA_DTYPE_BF16, u, 0, op.proj(CB - 1) + 1));
    }
    out.push_back(make("mod", l, -1, XEMA_KIND_FULL, XEMA_DTYPE_F32, 24 * B * D, op.mod(), op.ffn2(CC - 1) + 1));
    for (uint32_t c = 0; c < CA; ++c) {
      uint64_t n = elems_of(c, CA, 0);
      out.push_back(make("h1a", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_BF16, 2 * n * D, op.ln1a(c), op.kv(c) + 1));
      if (c == 0)
        out.push_back(make("kv", l, -1, XEMA_KIND_FULL, XEMA_DTYPE_BF16, 2 * u_all, op.kv(0), op.attn(CB - 1) + 1));
    }
    for (uint32_t c = 0; c < CB; ++c) {
      uint64_t n = elems_of(c, CB, 1);
      out.push_back(make("h1b", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_BF16, 2 * n * D, op.ln1b(c), op.q(c) + 1));
      out.push_back(make("q", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_BF16, 2 * n * D, op.q(c), op.attn(c) + 1));
      out.push_back(make("o", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_BF16, 2 * n * D, op.attn(c), op.proj(c) + 1));
      out.push_back(make("lse", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_F32, 4 * H * n, op.attn(c), op.attn(c) + 1));
      if (c == 0)
        out.push_back(make("res", l, -1, XEMA_KIND_FULL, XEMA_DTYPE_F32, 2 * u, op.proj(0), op.ffn2(CC - 1) + 1));
    }
    for (uint32_t c = 0; c < CC; ++c) {
      uint64_t n = elems_of(c, CC, 2);
      out.push_back(make("h2", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_BF16, 2 * n * D, op.ln2(c), op.ffn1(c) + 1));
      out.push_back(make("g", l, c, XEMA_KIND_CHUNK, XEMA_DTYPE_BF16, 2 * n * F, op.ffn1(c), op.ffn2(c) + 1));
      if (c == 0) {
        // the next hidden state: written chunk by chunk from FFN2_0 on; read by the next
        // block up to its last PROJ, or kept to the end if it is the output
        bool is_out = (l + 1 == L);
        OpIndex nx{(l + 1) * ops_per_block, CA, CB, CC};
        uint32_t death = is_out ? total_ops : nx.proj(CB - 1) + 1;
        out.push_back(make("hid", l + 1, -1, is_out ? XEMA_KIND_OUTPUT : XEMA_KIND_FULL, XEMA_DTYPE_BF16, u,
                           op.ffn2(0), death));
      }
    }
  }
  if (n_ops) *n_ops = total_ops;
  return XEMA_OK;
}

uint64_t max_live(const xema_tensor* t, size_t n) {
  // sweep over birth/death events; deaths at an index are applied before births
  std::vector<std::pair<uint32_t, int64_t>> ev;
  ev.reserve(2 * n);
  for (size_t i = 0; i < n; ++i) {
    if (t[i].death <= t[i].birth) continue;
    ev.emplace_back(t[i].birth, (int64_t)t[i].bytes);
    ev.emplace_back(t[i].death, -(int64_t)t[i].bytes);
  }
  std::sort(ev.begin(), ev.end(), [](const auto& a, const auto& b) {
    return a.first != b.first ? a.first < b.first : a.second < b.second;
  });
  int64_t live = 0, best = 0;
  for (auto& e : ev) {
    live += e.second;
    best = std::max(best, live);
  }
  return (uint64_t)best;
}

int plan_arena(const xema_tensor* t, size_t n, uint64_t* offsets, uint64_t* peak, uint64_t* live) {
  if (n && (!t || !offsets)) return XEMA_EINVAL;
  for (size_t i = 0; i < n; ++i)
    if (t[i].death <= t[i].birth) return XEMA_EINVAL;
  std::vector<uint32_t> order(n);
  for (size_t i = 0; i < n; ++i) order[i] = (uint32_t)i;
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
    if (t[a].bytes != t[b].bytes) return t[a].bytes > t[b].bytes;
    if (t[a].birth != t[b].birth) return t[a].birth < t[b].birth;
    if (t[a].death != t[b].death) return t[a].death < t[b].death;
    return a < b;
  });
  // `placed` is kept sorted by (offset, index) so the conflicting subset comes out in
  // address order without a per-tensor sort.
  std::vector<uint32_t> placed;
  placed.reserve(n);
  uint64_t top = 0;
  for (uint32_t i : order) {
    const xema_tensor& ti = t[i];
    uint64_t cursor = 0, best_size = 0, best_at = 0;
    bool have = false;
    for (uint32_t j : placed) {
      const xema_tensor& tj = t[j];
      if (!(ti.birth < tj.death && tj.birth < ti.death)) continue;
      if (offsets[j] > cursor) {
        uint64_t hole = offsets[j] - cursor;
        if (hole >= ti.bytes && (!have || hole < best_size)) {
          have = true;
          best_size = hole;
          best_at = cursor;
        }
      }
      cursor = std::max(cursor, offsets[j] + tj.bytes);
    }
    offsets[i] = have ? best_at : cursor;
    top = std::max(top, offsets[i] + ti.bytes);
    auto pos = std::lower_bound(placed.begin(), placed.end(), i, [&](uint32_t a, uint32_t b) {
      return offsets[a] != offsets[b] ? offsets[a] < offsets[b] : a < b;
    });
    placed.insert(pos, i);
  }
  if (peak) *peak = top;
  if (live) *live = max_live(t, n);
  return XEMA_OK;
}

int chunks_for_budget(const xema_config& cfg, uint64_t budget, int32_t max_chunks, int32_t* chunks,
                      uint64_t* peak_out) {
  int rc = validate_config(cfg);
  if (rc) return rc;
  if (max_chunks < 1) return XEMA_EINVAL;
  int64_t S = seq_len(cfg);
  int32_t hi = (int32_t)std::min<int64_t>(max_chunks, S);
  uint64_t smallest = ~uint64_t(0);
  std::vector<xema_tensor> ts;
  std::vector<uint64_t> offs;
  for (int32_t C = 1; C <= hi; ++C) {
    uint32_t n_ops = 0;
    rc = build_trace(cfg, C, ts, &n_ops);
    if (rc) return rc;
    offs.assign(ts.size(), 0);
    uint64_t peak = 0;
    rc = plan_arena(ts.data(), ts.size(), offs.data(), &peak, nullptr);
    if (rc) return rc;
    if (peak <= budget) {
      if (chunks) *chunks = C;
      if (peak_out) *peak_out = peak;
      return XEMA_OK;
    }
    smallest = std::min(smallest, peak);
  }
  if (chunks) *chunks = 0;
  if (peak_out) *peak_out = smallest;
  return XEMA_EBUDGET;
}

// Chunking only where the active-memory trace exceeds the budget: raise the chunk count of
// exactly the phases that hold an over-budget op, one step at a time; if the laid-out peak still
// exceeds the budget afterwards, raise the phase that holds the op with the most live bytes.
int phase_chunks_for_budget(const xema_config& cfg, uint64_t budget, int32_t max_chunks, int32_t chunks[3],
                            uint64_t* peak_out) {
  int32_t axes[3];
  return mitigation_for_budget(cfg, budget, max_chunks, false, chunks, axes, peak_out);
}

// The same search; with `serialize` a phase split C > 1 ways is split into sub-batches while
// C <= B (temporary serialization) and into row chunks otherwise.
int mitigation_for_budget(const xema_config& cfg, uint64_t budget, int32_t max_chunks, bool serialize,
                          int32_t chunks[3], int32_t axes[3], uint64_t* peak_out) {
  int rc = validate_config(cfg);
  if (rc) return rc;
  if (max_chunks < 1) return XEMA_EINVAL;
  const int32_t limit = (int32_t)std::min<int64_t>(max_chunks, seq_len(cfg));
  int32_t c[3] = {1, 1, 1};
  uint64_t smallest = ~uint64_t(0);
  std::vector<xema_tensor> ts;
  std::vector<uint64_t> offs, live;
  while (true) {
    uint32_t n_ops = 0;
    int32_t ax[3];
    for (int i = 0; i < 3; ++i)
      ax[i] = (serialize && c[i] > 1 && c[i] <= cfg.batch) ? XEMA_SPLIT_BATCH : XEMA_SPLIT_ROWS;
    rc = build_trace(cfg, c, ax, ts, &n_ops);
    if (rc) return rc;
    offs.assign(ts.size(), 0);
    uint64_t peak = 0;
    rc = plan_arena(ts.data(), ts.size(), offs.data(), &peak, nullptr);
    if (rc) return rc;
    smallest = std::min(smallest, peak);
    // active-memory trace by difference array
    std::vector<int64_t> delta(n_ops + 1, 0);
    for (const xema_tensor& t : ts) {
      delta[t.birth] += (int64_t)t.bytes;
      delta[t.death] -= (int64_t)t.bytes;
    }
    const uint32_t per_block = 1 + 3 * c[0] + 5 * c[1] + 3 * c[2];
    auto phase_of = [&](uint32_t op) {
      const uint32_t k = op % per_block;
      return k < 1u + 3 * c[0] ? 0 : (k < 1u + 3 * c[0] + 5 * c[1] ? 1 : 2);
    };
    bool over[3] = {false, false, false};
    int64_t cur = 0, best = -1;
    uint32_t best_op = 0;
    for (uint32_t op = 0; op < n_ops; ++op) {
      cur += delta[op];
      if ((uint64_t)cur > budget) over[phase_of(op)] = true;
      if (cur > best) { best = cur; best_op = op; }
    }
    if (!over[0] && !over[1] && !over[2]) {
      if (peak <= budget) {
        for (int i = 0; i < 3; ++i) {
          chunks[i] = c[i];
          axes[i] = ax[i];
        }
        if (peak_out) *peak_out = peak;
        return XEMA_OK;
      }
      over[phase_of(best_op)] = true;
    }
    for (int i = 0; i < 3; ++i) {
      if (!over[i]) continue;
      if (++c[i] > limit) {
        chunks[0] = chunks[1] = chunks[2] = 0;
        axes[0] = axes[1] = axes[2] = XEMA_SPLIT_ROWS;
        if (peak_out) *peak_out = smallest;
        return XEMA_EBUDGET;
      }
    }
  }
}

int rope_table(const xema_config& cfg, float* out) {
  int rc = validate_config(cfg);
  if (rc) return rc;
  if (!out) return XEMA_EINVAL;
  const int64_t S = seq_len(cfg);
  const int half = cfg.head_dim / 2;
  const int dims[3] = {cfg.rope_dim_t, cfg.rope_dim_h, cfg.rope_dim_w};
  std::vector<double> inv_freq(half);
  std::vector<int> axis_of(half);
  int p = 0;
  for (int a = 0; a < 3; ++a)
    for (int j = 0; j < dims[a] / 2; ++j, ++p) {
      inv_freq[p] = std::pow((double)cfg.rope_base, -2.0 * j / dims[a]);
      axis_of[p] = a;
    }
  const int64_t hw = (int64_t)cfg.grid_h * cfg.grid_w;
  for (int64_t i = 0; i < S; ++i) {
    int64_t pos[3] = {0, 0, 0};
    if (i >= cfg.s_text) {
      int64_t nn = i - cfg.s_text;
      pos[0] = nn / hw;
      pos[1] = (nn / cfg.grid_w) % cfg.grid_h;
      pos[2] = nn % cfg.grid_w;
    }
    float* row = out + i * half * 2;
    for (int j = 0; j < half; ++j) {
      double ang = (double)pos[axis_of[j]] * inv_freq[j];
      row[2 * j] = (float)std::cos(ang);
      row[2 * j + 1] = (float)std::sin(ang);
    }
  }
  return XEMA_OK;
}

}  // namespace xema

extern "C" {

int xema_trace(const xema_config* cfg, int32_t chunks, xema_tensor* out, size_t cap, size_t* n_tensors,
               uint32_t* n_ops) {
  if (!cfg) return XEMA_EINVAL;
  std::vector<xema_tensor> ts;
  uint32_t ops = 0;
  int rc = xema::build_trace(*cfg, chunks, ts, &ops);
  if (rc) return rc;
  if (n_tensors) *n_tensors = ts.size();
  if (n_ops) *n_ops = ops;
  if (cap < ts.size() || !out) return XEMA_ENOSPC;
  std::memcpy(out, ts.data(), ts.size() * sizeof(xema_tensor));
  return XEMA_OK;
}

int xema_trace_phases(const xema_config* cfg, const int32_t chunks[3], xema_tensor* out, size_t cap,
                      size_t* n_tensors, uint32_t* n_ops) {
  if (!cfg || !chunks) return XEMA_EINVAL;
  std::vector<xema_tensor> ts;
  uint32_t ops = 0;
  int rc = xema::build_trace(*cfg, chunks, ts, &ops);
  if (rc) return rc;
  if (n_tensors) *n_tensors = ts.size();
  if (n_ops) *n_ops = ops;
  if (cap < ts.size() || !out) return XEMA_ENOSPC;
  std::memcpy(out, ts.data(), ts.size() * sizeof(xema_tensor));
  return XEMA_OK;
}

int xema_phase_chunks_for_budget(const xema_config* cfg, uint64_t budget_bytes, int32_t max_chunks,
                                 int32_t chunks[3], uint64_t* peak_bytes) {
  if (!cfg || !chunks) return XEMA_EINVAL;
  return xema::phase_chunks_for_budget(*cfg, budget_bytes, max_chunks, chunks, peak_bytes);
}

int xema_trace_mitigated(const xema_config* cfg, const xema_mitigation* m, xema_tensor* out, size_t cap,
                         size_t* n_tensors, uint32_t* n_ops) {
  if (!cfg || !m) return XEMA_EINVAL;
  std::vector<xema_tensor> ts;
  uint32_t ops = 0;
  int rc = xema::build_trace(*cfg, m->chunks, m->axis, ts, &ops);
  if (rc) return rc;
  if (n_tensors) *n_tensors = ts.size();
  if (n_ops) *n_ops = ops;
  if (cap < ts.size() || !out) return XEMA_ENOSPC;
  std::memcpy(out, ts.data(), ts.size() * sizeof(xema_tensor));
  return XEMA_OK;
}

int xema_trace_sharded(const xema_config* cfg, const xema_mitigation* m, int32_t shard, int32_t shards,
                       xema_tensor* out, size_t cap, size_t* n_tensors, uint32_t* n_ops) {
  if (!cfg || !m) return XEMA_EINVAL;
  std::vector<xema_tensor> ts;
  uint32_t ops = 0;
  xema::Shard sh;
  sh.p = shard;
  sh.P = shards;
  int rc = xema::build_trace(*cfg, m->chunks, m->axis, sh, ts, &ops);
  if (rc) return rc;
  if (n_tensors) *n_tensors = ts.size();
  if (n_ops) *n_ops = ops;
  if (cap < ts.size() || !out) return XEMA_ENOSPC;
  std::memcpy(out, ts.data(), ts.size() * sizeof(xema_tensor));
  return XEMA_OK;
}

int xema_shard_rows(const xema_config* cfg, int32_t shard, int32_t shards, int64_t* row0, int64_t* rows) {
  if (!cfg) return XEMA_EINVAL;
  int rc = xema::validate_config(*cfg);
  if (rc) return rc;
  xema::Shard sh;
  sh.p = shard;
  sh.P = shards;
  return xema::shard_rows(*cfg, sh, row0, rows);
}

int xema_mitigation_for_budget(const xema_config* cfg, uint64_t budget_bytes, int32_t max_chunks,
                               xema_mitigation* m, uint64_t* peak_bytes) {
  if (!cfg || !m) return XEMA_EINVAL;
  return xema::mitigation_for_budget(*cfg, budget_bytes, max_chunks, true, m->chunks, m->axis, peak_bytes);
}

int xema_pressure_ranges(const xema_tensor* tensors, size_t n, uint32_t n_ops, uint64_t budget_bytes,
                         uint32_t* ranges, size_t cap, size_t* n_ranges) {
  if (n && !tensors) return XEMA_EINVAL;
  std::vector<int64_t> delta((size_t)n_ops + 1, 0);
  for (size_t i = 0; i < n; ++i) {
    if (tensors[i].death <= tensors[i].birth || tensors[i].death > n_ops) return XEMA_EINVAL;
    delta[tensors[i].birth] += (int64_t)tensors[i].bytes;
    delta[tensors[i].death] -= (int64_t)tensors[i].bytes;
  }
  std::vector<uint32_t> out;
  int64_t live = 0;
  bool open = false;
  for (uint32_t op = 0; op < n_ops; ++op) {
    live += delta[op];
    const bool over = (uint64_t)live > budget_bytes;
    if (over && !open) out.push_back(op);
    if (!over && open) out.push_back(op);
    open = over;
  }
  if (open) out.push_back(n_ops);
  if (n_ranges) *n_ranges = out.size() / 2;
  if (out.size() / 2 > cap || (!ranges && !out.empty())) return XEMA_ENOSPC;
  for (size_t i = 0; i < out.size(); ++i) ranges[i] = out[i];
  return XEMA_OK;
}

int xema_plan_arena(const xema_tensor* tensors, size_t n, uint64_t* offsets, uint64_t* peak_bytes,
                    uint64_t* max_live_bytes) {
  return xema::plan_arena(tensors, n, offsets, peak_bytes, max_live_bytes);
}

int xema_chunks_for_budget(const xema_config* cfg, uint64_t budget_bytes, int32_t max_chunks, int32_t* chunks,
                           uint64_t* peak_bytes) {
  if (!cfg) return XEMA_EINVAL;
  return xema::chunks_for_budget(*cfg, budget_bytes, max_chunks, chunks, peak_bytes);
}

int xema_rope_table(const xema_config* cfg, float* host_out) {
  if (!cfg) return XEMA_EINVAL;
  return xema::rope_table(*cfg, host_out);
}

const char* xema_strerror(int status) {
  switch (status) {
    case XEMA_OK: return "ok";
    case XEMA_EINVAL: return "invalid argument or configuration";
    case XEMA_ENOSPC: return "output array or arena too small";
    case XEMA_EBUDGET: return "no chunk count within max_chunks fits the byte budget";
    case XEMA_EALIGN: return "device pointer not aligned as required";
    case XEMA_ECUDA: return "CUDA call failed (see xema_last_cuda_error)";
    case XEMA_ETIMEOUT: return "a kernel gave up a bounded wait";
    case XEMA_ESTATE: return "plan not bound or wrong call for this plan";
    default: return "unknown status";
  }
}

const char* xema_version(void) { return "xema-b200 0.1 (sm_100a)"; }

}  // extern "C"
