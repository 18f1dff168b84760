// Internal C++ view of the host planner (trace, Algorithm 1 layout, chunk search).
#pragma once
#include <vector>

#include "../../include/xema.h"

namespace xema {

int validate_config(const xema_config& cfg);
int64_t seq_len(const xema_config& cfg);
int build_trace(const xema_config& cfg, int32_t chunks, std::vector<xema_tensor>& out, uint32_t* n_ops);
// chunks[3]: key/value phase, attention phase, feed-forward phase
int build_trace(const xema_config& cfg, const int32_t chunks[3], std::vector<xema_tensor>& out, uint32_t* n_ops);
// axes[3]: XEMA_SPLIT_ROWS or XEMA_SPLIT_BATCH per phase
int build_trace(const xema_config& cfg, const int32_t chunks[3], const int32_t axes[3], std::vector<xema_tensor>& out,
                uint32_t* n_ops);
// Sequence-parallel shard p of P: token rows [floor(p S / P), floor((p+1) S / P)).
struct Shard {
  int32_t p = 0, P = 1;
};
int shard_rows(const xema_config& cfg, Shard sh, int64_t* row0, int64_t* rows);
// The trace of one shard: every tensor over the owned rows, except the full-size kv.
int build_trace(const xema_config& cfg, const int32_t chunks[3], const int32_t axes[3], Shard sh,
                std::vector<xema_tensor>& out, uint32_t* n_ops);
int mitigation_for_budget(const xema_config& cfg, uint64_t budget, int32_t max_chunks, bool serialize,
                          int32_t chunks[3], int32_t axes[3], uint64_t* peak_out);
int phase_chunks_for_budget(const xema_config& cfg, uint64_t budget, int32_t max_chunks, int32_t chunks[3],
                            uint64_t* peak_out);
uint64_t max_live(const xema_tensor* t, size_t n);
int plan_arena(const xema_tensor* t, size_t n, uint64_t* offsets, uint64_t* peak, uint64_t* live);
int chunks_for_budget(const xema_config& cfg, uint64_t budget, int32_t max_chunks, int32_t* chunks,
                      uint64_t* peak_out);
int rope_table(const xema_config& cfg, float* out);

}  // namespace xema
