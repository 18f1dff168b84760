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
