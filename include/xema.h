/*
 * xema.h -- C ABI of the B200 (sm_100a) library for memory-budgeted DiT blocks.
 *
 * The library implements the single-GPU hot path of Xema's fine-grained memory
 * management for diffusion serving: a DiT denoising block (or a stack of blocks, one
 * denoising step) is run sequence-chunked so that its activation peak fits a byte
 * budget, and every intermediate tensor lives at a precomputed offset of one static
 * arena derived from an offline lifetime trace instead of a caching allocator.
 *
 *   xema_trace              template + chunk count -> tensor sizes and lifetimes
 *                           (the paper's Memory Analyzer; section "Memory Analysis and
 *                           Latency Profiling" and "Offline Static Layout")
 *   xema_plan_arena         lifetimes -> arena offsets (Algorithm 1, "Offline static
 *                           memory layout") + reserved peak + max-live bytes
 *   xema_chunks_for_budget  smallest chunk count whose reserved peak fits the budget
 *                           (section "Applying Only as Much Mitigation as Needed", with the
 *                           chunk count as the mitigation intensity; "Localized chunking")
 *   xema_phase_chunks_for_budget  one chunk count per phase of the block, raised only in
 *                           the phases whose trace exceeds the budget (section "Applying
 *                           Mitigation Only Where Needed")
 *   xema_block_forward /    run one block / all n_blocks blocks on a caller-given CUDA
 *   xema_step_forward       stream over caller-owned arena memory ("Static memory
 *                           runtime": allocation at run time is a table lookup)
 *
 * Conventions
 *   - All functions return 0 (XEMA_OK) or a negative xema_status; nothing throws, aborts,
 *     allocates device memory, frees device memory or synchronises a stream or device
 *     (one stated exception: the allocator plug-in's malloc / free entry points).
 *   - "host" / "device" is stated for every pointer.  Device pointers must belong to the
 *     CUDA device that is current when the function is called.
 *   - Linear layers are y = x W^T + b with W stored [out, in] row-major, bf16.
 *   - Token rows: text tokens first, then the video/image tokens in (t, h, w) raster order.
 *   - Chunk c of C covers token rows [floor(c*S/C), floor((c+1)*S/C)).
 *   - Every tensor size is rounded up to 256 bytes, so every arena offset is 256-aligned.
 */
#ifndef XEMA_H_
#define XEMA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum xema_status {
  XEMA_OK = 0,
  XEMA_EINVAL = -1,   /* bad argument or configuration                                   */
  XEMA_ENOSPC = -2,   /* an output array or the arena is too small                        */
  XEMA_EBUDGET = -3,  /* no chunk count up to max_chunks fits the budget                  */
  XEMA_EALIGN = -4,   /* a device pointer is not aligned as required                      */
  XEMA_ECUDA = -5,    /* a CUDA runtime/driver call failed; see xema_last_cuda_error()    */
  XEMA_ETIMEOUT = -6, /* a kernel gave up a bounded wait (read back from the status word) */
  XEMA_ESTATE = -7    /* the plan is not bound, or is bound for a different kind of call  */
} xema_status;

/* Request template.  Plain data, caller-owned, copied by the library. */
typedef struct xema_config {
  int32_t batch;      /* B >= 1; every chunk carries all B batch elements                 */
  int32_t s_text;     /* text tokens (>= 0)                                               */
  int32_t grid_t, grid_h, grid_w; /* latent grid; S = s_text + grid_t*grid_h*grid_w       */
  int32_t hidden;     /* D = heads * head_dim; multiple of 256                            */
  int32_t heads;      /* H                                                                */
  int32_t head_dim;   /* dh: 64 or 128                                                    */
  int32_t ffn;        /* F, multiple of 256                                               */
  int32_t temb_dim;   /* Dt, multiple of 8                                                */
  int32_t rope_dim_t, rope_dim_h, rope_dim_w; /* even, sum == head_dim                    */
  float rope_base;    /* 10000                                                            */
  float ln_eps;       /* LayerNorm epsilon (1e-6)                                         */
  float rms_eps;      /* QK RMSNorm epsilon (1e-6)                                        */
  int32_t n_blocks;   /* 1 = block template, 42 = CogVideoX-shaped denoising step         */
} xema_config;

enum { XEMA_KIND_INPUT = 0, XEMA_KIND_OUTPUT = 1, XEMA_KIND_FULL = 2, XEMA_KIND_CHUNK = 3,
       XEMA_KIND_WORKSPACE = 4 };
enum { XEMA_DTYPE_BF16 = 0, XEMA_DTYPE_F32 = 1 };

/* One traced tensor.  Lifetime is the half-open interval [birth, death) of logical-op
 * indices, as Algorithm 1 takes it. */
typedef struct xema_tensor {
  char name[24];   /* "hid0", "kv3", "q0_2", ... NUL-terminated                           */
  uint32_t kind;   /* XEMA_KIND_*                                                         */
  uint32_t dtype;  /* XEMA_DTYPE_*                                                        */
  int32_t block;   /* block index, -1 for temb                                            */
  int32_t chunk;   /* chunk index, -1 for full-sequence tensors                           */
  uint64_t bytes;  /* rounded up to 256                                                   */
  uint32_t birth;  /* first op that writes it (0 for inputs)                              */
  uint32_t death;  /* 1 + last op that reads or writes it (n_ops for the output)          */
} xema_tensor;

/* Device pointers to one block's bf16 parameters. */
typedef struct xema_block_weights {
  const void* w_mod;  /* [6D, Dt]  adaLN modulation (shift1, scale1, gate1, shift2, ...)  */
  const void* b_mod;  /* [6D]                                                             */
  const void* w_qkv;  /* [3D, D]   rows 0..D-1 -> q, D..2D-1 -> k, 2D..3D-1 -> v          */
  const void* b_qkv;  /* [3D]                                                             */
  const void* g_q;    /* [dh]      RMSNorm gain of q                                      */
  const void* g_k;    /* [dh]      RMSNorm gain of k                                      */
  const void* w_o;    /* [D, D]                                                           */
  const void* b_o;    /* [D]                                                              */
  const void* w_1;    /* [F, D]                                                           */
  const void* b_1;    /* [F]                                                              */
  const void* w_2;    /* [D, F]                                                           */
  const void* b_2;    /* [D]                                                              */
} xema_block_weights;

/* ---- host-only planner (pure integer code; no CUDA call) -------------------------------- */

/* Tensor lifetimes of the template run with `chunks` sequence chunks (the offline,
 * shape-only analysis of "Offline Static Layout").  Op order per block, 1 + 11*chunks ops:
 * MOD; per chunk LN1A, KV, KROPE; per chunk LN1B, Q, QROPE, ATTN, PROJ; per chunk LN2,
 * FFN1, FFN2.  Tensors are written to `out` (host, capacity `cap`) in id order = order of
 * first birth.  *n_tensors (host) always receives the number of tensors, *n_ops (host) the
 * number of ops, so a first call with cap = 0 sizes the array (returns XEMA_ENOSPC).
 * XEMA_EINVAL: bad config or chunks outside [1, S]. */
int xema_trace(const xema_config* cfg, int32_t chunks, xema_tensor* out, size_t cap,
               size_t* n_tensors, uint32_t* n_ops);

/* Algorithm 1 ("Offline static memory layout"): tensors in descending size (ties: birth,
 * death, index); for each, the already placed tensors with an intersecting lifetime define
 * address gaps; take the smallest gap that fits (ties: lowest address), else the address
 * above all of them.  offsets (host, n entries) receives one byte offset per tensor;
 * *peak_bytes = max(offset + bytes) is the reserved peak; *max_live_bytes is the largest sum
 * of bytes live at one op (the active peak the reserved peak is compared with).  Either
 * output pointer may be NULL. */
int xema_plan_arena(const xema_tensor* tensors, size_t n, uint64_t* offsets,
                    uint64_t* peak_bytes, uint64_t* max_live_bytes);

/* Minimum mitigation that fits (section "Applying Only as Much Mitigation as Needed"):
 * scans chunks = 1, 2, ..., max_chunks and returns the first whose reserved peak
 * (xema_trace -> xema_plan_arena) is <= budget_bytes.  On XEMA_EBUDGET *chunks is 0 and
 * *peak_bytes is the smallest peak seen. */
int xema_chunks_for_budget(const xema_config* cfg, uint64_t budget_bytes, int32_t max_chunks,
                           int32_t* chunks, uint64_t* peak_bytes);

/* The memory-pressure set (section "Applying Mitigation Only Where Needed"; planner stage
 * "locate where memory exceeds the budget"): the maximal half-open op ranges [first, end) in
 * which the live bytes of the trace exceed budget_bytes.  ranges (host) receives up to cap
 * pairs (first, end) in ascending order; *n_ranges (host) always receives their number, so a
 * call with cap = 0 sizes the array (XEMA_ENOSPC when there is at least one range).
 * XEMA_EINVAL: a tensor with death <= birth or death > n_ops. */
int xema_pressure_ranges(const xema_tensor* tensors, size_t n, uint32_t n_ops,
                         uint64_t budget_bytes, uint32_t* ranges, size_t cap, size_t* n_ranges);

/* Per-phase chunk counts (section "Applying Mitigation Only Where Needed": the planner
 * locates, on the memory trace, where the budget is exceeded and mitigates only there).
 * A block has three phases: 0 = keys/values (LN1A, KV, KROPE per chunk), 1 = queries,
 * attention, output projection (LN1B, Q, QROPE, ATTN, PROJ per chunk), 2 = feed-forward
 * (LN2, FFN1, FFN2 per chunk).  chunks[3] (host) holds one count per phase; phase p splits
 * the S rows into chunks[p] pieces by the rule above; a block then has
 * 1 + 3*chunks[0] + 5*chunks[1] + 3*chunks[2] ops.  Otherwise as xema_trace, which is the
 * case chunks[0] = chunks[1] = chunks[2]. */
int xema_trace_phases(const xema_config* cfg, const int32_t chunks[3], xema_tensor* out,
                      size_t cap, size_t* n_tensors, uint32_t* n_ops);

/* Search for per-phase counts that fit: start at (1, 1, 1); on the trace of the current
 * counts, every phase that holds an op whose live bytes exceed budget_bytes gets one more
 * chunk; repeat.  When no op is over, the trace is laid out (Algorithm 1); if the reserved
 * peak still exceeds the budget, the phase holding the op with the most live bytes (lowest
 * op index on ties) gets one more chunk.  chunks (host, 3 entries) receives the counts and
 * *peak_bytes the reserved peak.  XEMA_EBUDGET when a phase would need more than
 * min(max_chunks, S) chunks: chunks is then zeroed and *peak_bytes is the smallest reserved
 * peak seen. */
int xema_phase_chunks_for_budget(const xema_config* cfg, uint64_t budget_bytes,
                                 int32_t max_chunks, int32_t chunks[3], uint64_t* peak_bytes);

/* Temporary serialization (section "Applying Mitigation Only Where Needed", paragraph
 * "Temporary serialization"; "Memory mitigation primitives": only the planned steps are split
 * into sub-batches, which rejoin afterwards).  A phase can be split along the batch instead of
 * along the rows: piece c of C then covers batch elements [floor(c*B/C), floor((c+1)*B/C)) and
 * all S rows (1 <= C <= B); the full-size tensors kv, res and hid are where the sub-batches
 * rejoin.  chunks[p] pieces along axis[p] for phase p. */
enum { XEMA_SPLIT_ROWS = 0, XEMA_SPLIT_BATCH = 1 };
typedef struct xema_mitigation {
  int32_t chunks[3]; /* pieces of the key/value, attention and feed-forward phase            */
  int32_t axis[3];   /* XEMA_SPLIT_ROWS or XEMA_SPLIT_BATCH per phase                         */
} xema_mitigation;

/* xema_trace_phases with a split axis per phase (all XEMA_SPLIT_ROWS gives the same trace).
 * XEMA_EINVAL: a count outside [1, S] (rows) or [1, B] (batch), or an unknown axis. */
int xema_trace_mitigated(const xema_config* cfg, const xema_mitigation* m, xema_tensor* out,
                         size_t cap, size_t* n_tensors, uint32_t* n_ops);

/* The search of xema_phase_chunks_for_budget where, at every step, a phase that is split
 * C > 1 ways is split into sub-batches while C <= B and into row chunks beyond that.  *m
 * (host) receives counts and axes (axis of an unsplit phase: XEMA_SPLIT_ROWS); on
 * XEMA_EBUDGET the counts are zeroed and *peak_bytes is the smallest reserved peak seen. */
int xema_mitigation_for_budget(const xema_config* cfg, uint64_t budget_bytes, int32_t max_chunks,
                               xema_mitigation* m, uint64_t* peak_bytes);

/* ---- sequence parallelism (the paper's SP, section "Execution Configurations": the latent
 * sequence is split across GPUs; the planner enumerates the SP degree in stage 1 of "Planning
 * Workflow") ---------------------------------------------------------------------------------
 * GPU `shard` of `shards` owns token rows [floor(shard*S/shards), floor((shard+1)*S/shards)).
 * Its block has the same ops.  Every tensor holds the owned rows only (chunks then cut the owned
 * rows: chunk c of C covers owned rows [floor(c*n/C), floor((c+1)*n/C)) of the n owned), except
 * kv<l>, which stays [B, S, 2D] over ALL rows: phase A (LN1A, KV, KROPE) fills the owned rows,
 * the keys and values of the other GPUs must be in place (one all-gather, done by the caller
 * into its own arena) before the first op of phase B.  Nothing in the library communicates. */

/* First row and number of rows shard `shard` of `shards` owns.  XEMA_EINVAL unless
 * 0 <= shard < shards <= S. */
int xema_shard_rows(const xema_config* cfg, int32_t shard, int32_t shards, int64_t* row0, int64_t* rows);
/* xema_trace_mitigated for one shard (shard 0 of 1 gives the same trace).  Counts are limited by
 * the owned rows. */
int xema_trace_sharded(const xema_config* cfg, const xema_mitigation* m, int32_t shard, int32_t shards,
                       xema_tensor* out, size_t cap, size_t* n_tensors, uint32_t* n_ops);

/* RoPE table for the template: host_out (host) receives S * (dh/2) * 2 floats laid out
 * [token][pair][cos, sin]; angle = position * rope_base^(-2j/d) inside each of the three
 * sections (t, h, w), evaluated in double precision and rounded once.  Text tokens sit at
 * position (0, 0, 0).  The table is template-static parameter memory, not an arena tensor. */
int xema_rope_table(const xema_config* cfg, float* host_out);

/* ---- plan objects ----------------------------------------------------------------------- */

typedef struct xema_plan xema_plan; /* opaque; host memory owned by the library */

/* Traces and lays out the template for `chunks` chunks.  No CUDA call. */
int xema_plan_create(const xema_config* cfg, int32_t chunks, xema_plan** out);
/* The same with one chunk count per phase (see xema_trace_phases). */
int xema_plan_create_phases(const xema_config* cfg, const int32_t chunks[3], xema_plan** out);
void xema_plan_destroy(xema_plan* plan);

/* Plan figures: any output pointer may be NULL.  *chunks is the largest of the plan's three
 * per-phase counts (the count itself for a plan made by xema_plan_create). */
int xema_plan_info(const xema_plan* plan, uint64_t* peak_bytes, uint64_t* max_live_bytes,
                   size_t* n_tensors, uint32_t* n_ops, int32_t* chunks);
/* The plan's per-phase chunk counts; chunks: host, 3 entries. */
int xema_plan_phase_chunks(const xema_plan* plan, int32_t chunks[3]);
/* Plan with a split axis per phase (see xema_trace_mitigated), and the plan's counts and axes. */
int xema_plan_create_mitigated(const xema_config* cfg, const xema_mitigation* m, xema_plan** out);
int xema_plan_mitigation(const xema_plan* plan, xema_mitigation* m);
/* Plan for one sequence-parallel shard (see xema_trace_sharded).  Its hid<l> / res<l> tensors and
 * its input and output are [B, rows owned, D]; token positions (RoPE) stay global.  The forward
 * calls run as usual; the caller splits them at the gather points:
 *   for every block l: xema_forward_range(plan, previous point, first_op(l)); all-gather of
 *   kv<l>'s rows; ... and xema_forward_range(plan, first_op(last), n_ops) at the end.
 * xema_forward_host refuses a sharded plan (XEMA_ESTATE). */
int xema_plan_create_sharded(const xema_config* cfg, const xema_mitigation* m, int32_t shard, int32_t shards,
                             xema_plan** out);
/* Debug layout with guard bands (a stand-in for a memory checker): every tensor is laid out as
 * if it were guard_bytes (a multiple of 256) larger, so the guard_bytes after it -- [offset +
 * bytes, offset + bytes + guard_bytes) -- belong to no tensor for as long as it lives.  A caller
 * fills those bytes with a pattern when the tensor is born and checks them after every op until it
 * dies (tensor lifetimes: xema_plan_tensor_at; one op at a time: xema_forward_range): a kernel
 * that writes past the end of its own tensor shows up at once, with the op that did it.  The
 * reported tensor sizes and max-live bytes are the real ones; the peak includes the guards.
 * Outputs are the same bits as with any other layout. */
int xema_plan_create_guarded(const xema_config* cfg, const xema_mitigation* m, int32_t shard, int32_t shards,
                             uint64_t guard_bytes, xema_plan** out);
/* guard_bytes of the plan (0 for a plan made any other way). */
uint64_t xema_plan_guard_bytes(const xema_plan* plan);
/* The plan's shard and the rows it owns (0 of 1 and all rows for an unsharded plan). */
int xema_plan_shard(const xema_plan* plan, int32_t* shard, int32_t* shards, int64_t* row0, int64_t* rows);
/* Gather point of block `block`: *first_op = index of the first op of its phase B (every op
 * before it may run before the exchange, none from it on); *kv_offset = arena offset of kv<block>,
 * laid out [B, S, 2D] bf16 with row (b, r) at ((b*S + r) * 2D) elements, K half first. */
int xema_plan_gather_point(const xema_plan* plan, int32_t block, uint32_t* first_op, uint64_t* kv_offset);
/* Offset and (256-rounded) size of a tensor by name, e.g. "hid0", "temb", "hid1", "res0". */
int xema_plan_tensor(const xema_plan* plan, const char* name, uint64_t* offset, uint64_t* bytes);
/* Copy of the plan's tensor i and its offset. */
int xema_plan_tensor_at(const xema_plan* plan, size_t i, xema_tensor* tensor, uint64_t* offset);

/* Binds the plan to memory and pre-encodes every TMA descriptor (all addresses are static,
 * so nothing is encoded at launch time).  arena_dev: device, 256-byte aligned, arena_bytes >=
 * the plan's peak (XEMA_ENOSPC otherwise).  weights: host array of n_blocks structs holding
 * device pointers (16-byte aligned).  rope_dev: device copy of xema_rope_table's output.
 * status_dev: device, 4 bytes, zeroed by the caller, or NULL; kernels that give up a bounded
 * wait store a non-zero code there.  Launches nothing.  The arena, weights and table stay
 * owned by the caller and must outlive the forward calls. */
int xema_plan_bind(xema_plan* plan, void* arena_dev, uint64_t arena_bytes,
                   const xema_block_weights* weights, const float* rope_dev, void* status_dev);

/* Enqueues the block (n_blocks must be 1) / all n_blocks blocks on `stream` (a cudaStream_t
 * passed as void*).  Input: the caller has written hid0 [B,S,D] bf16 and temb [B,Dt] bf16 at
 * their plan offsets; output: hid<n_blocks> [B,S,D] bf16 at its plan offset once the stream
 * reaches the end of the enqueued work.  Every byte written lies inside [arena, arena+peak).
 * Returns XEMA_ECUDA if a launch is rejected; asynchronous faults surface at the caller's
 * own synchronisation. */
int xema_block_forward(const xema_plan* plan, void* stream);
int xema_step_forward(const xema_plan* plan, void* stream);

/* The same forward with HOST buffers (the end-to-end form of the paper's serving runtime,
 * section "Static memory runtime": a request's latent goes in, the denoised latent comes out).
 * Enqueues on `stream`: a host-to-device copy of hid_in_host [B,S,D] bf16 and temb_host [B,Dt]
 * bf16 into their arena slots, all n_blocks blocks, and a device-to-host copy of the output
 * hidden state into hid_out_host [B,S,D] bf16.  The arena is the one given to xema_plan_bind;
 * no other device memory is touched or allocated.  Where the first block's key/value phase or
 * the last block's feed-forward phase runs in more than one piece, the copies of all pieces but
 * one go through a second stream owned by the plan (created at the first such call, destroyed
 * with the plan) and are ordered against `stream` by events in both directions: the input of
 * piece c + 1 arrives while piece c is worked on, the output of piece c leaves while piece
 * c + 1 is worked on, and `stream` does not pass the call before the last copy has finished.
 * The results do not depend on it.  The host buffers are the caller's and
 * must stay valid until the stream has passed the call; they should be page-locked (the copies
 * of pageable memory are staged by the CUDA runtime and may block the calling thread).  Does
 * not synchronise.  XEMA_ESTATE if the plan is unbound, XEMA_ECUDA if a copy or launch is
 * rejected. */
int xema_forward_host(const xema_plan* plan, const void* hid_in_host, const void* temb_host,
                      void* hid_out_host, void* stream);

/* The block forward for callers that cannot allocate device memory (the paper has no
 * counterpart: its runtime always has PyTorch's allocator behind it).  Some callers can call
 * neither cudaMalloc nor a framework allocator: code inside a region that must not
 * synchronise the device, a process whose device memory already belongs to a pool it does not
 * own, a plug-in that is handed nothing but its input and output buffers.  xema_block_forward
 * needs a caller-allocated arena for the block's intermediates; this variant keeps them in a
 * fixed array of XEMA_STATIC_ARENA_BYTES inside the library image instead (every GPU that
 * loads the library holds that much memory until the process exits).
 *
 * One block (cfg->n_blocks must be 1) with `chunks` sequence chunks.  weights: host pointer to
 * one struct of device pointers; rope_dev: device copy of xema_rope_table's output;
 * hid_in_dev [B,S,D] bf16, temb_dev [B,Dt] bf16 (device, read); hid_out_dev [B,S,D] bf16
 * (device, written; may not overlap the inputs); status_dev: device, 4 zeroed bytes, or NULL.
 * Enqueues two device-to-device copies in, the block's launches, and one copy out on `stream`.
 * Calls no cudaMalloc/cudaFree and no allocating library routine; host memory for the plan is
 * taken from the C++ heap and released before returning.  Every call derives the trace and
 * its layout again and encodes all TMA descriptors on the host (tens of microseconds for a
 * small template): a caller that can hold a plan should use xema_plan_bind once and
 * xema_block_forward per call instead.  Host threads may call in concurrently as far as the
 * host side goes (the cached device address is atomic); the shared scratch array is what
 * limits them, see below.
 *
 * XEMA_ENOSPC: the template's arena peak for this chunk count exceeds XEMA_STATIC_ARENA_BYTES
 * (the tiny template needs 2 076 672 bytes at chunks = 1); use xema_block_forward with your own
 * arena instead.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress); make that first call before any stream capture begins.  All calls
 * share the one array and it keeps the previous call's contents (the block writes every
 * intermediate before reading it, so nothing has to be cleared); two calls whose work overlaps
 * on the GPU -- different streams, or different host threads -- race on it. */
#define XEMA_STATIC_ARENA_BYTES (4u << 20)
int xema_block_forward_static(const xema_config* cfg, int32_t chunks, const xema_block_weights* weights,
                              const float* rope_dev, const void* hid_in_dev, const void* temb_dev,
                              void* hid_out_dev, void* status_dev, void* stream);

/* Number of kernel launches one forward call enqueues (0 if unbound). */
int xema_plan_launch_count(const xema_plan* plan);

/* Debug aid: enqueue only the first n_logical_ops logical ops of the trace order. */
int xema_forward_prefix(const xema_plan* plan, uint32_t n_logical_ops, void* stream);
/* Enqueue logical ops [first_op, end_op) of the trace order (one launch each); lets a caller
 * put its own events between ops to time them. */
int xema_forward_range(const xema_plan* plan, uint32_t first_op, uint32_t end_op, void* stream);
/* Describes launch i of a bound plan: name8 (host, 8 bytes) receives "MOD", "LN1A", "KV",
 * "KROPE", "LN1B", "Q", "QROPE", "ATTN", "PROJ", "LN2", "FFN1" or "FFN2"; *flops the algorithmic
 * floating-point operations (2 per multiply-add; attention 4*B*rows*S*D), *bytes the
 * algorithmic HBM bytes (each operand read once, each result written once).  Any output
 * pointer may be NULL. */
int xema_plan_op(const xema_plan* plan, uint32_t i, char* name8, int32_t* block, int32_t* chunk,
                 double* flops, double* bytes);

/* ---- single operators (the kernels behind the forward calls, on plain device pointers) --- */

/* mod[b, j] = sum_k silu(temb[b,k]) w_mod[j,k] + b_mod[j]; temb [B,Dt] bf16, w_mod [n_out,Dt]
 * bf16, b_mod [n_out] bf16 -> mod [B,n_out] fp32 (all device). */
int xema_op_mod(const void* temb, const void* w_mod, const void* b_mod, float* mod, int32_t batch,
                int32_t temb_dim, int32_t n_out, void* stream);

/* out[b,i,:] = LN(in[b,i,:]) * (1 + scale[b,:]) + shift[b,:]; LayerNorm without affine,
 * biased variance.  in: device, bf16 (in_is_f32 = 0) or fp32 (1), row (b,i) at element
 * (b*in_batch_rows + i)*D; out: device bf16 [B,rows,D] contiguous; shift/scale: device fp32,
 * batch stride mod_stride elements. */
int xema_op_ln_modulate(const void* in, int32_t in_is_f32, int64_t in_batch_rows, void* out,
                        const float* shift, const float* scale, int64_t mod_stride, int32_t batch,
                        int32_t rows, int32_t D, float eps, void* stream);

/* In place, per head: x <- RoPE(x / sqrt(mean(x^2) + eps) * g).  x: device bf16, row (b,i) at
 * element (b*batch_rows + i)*ld, heads*head_dim leading features of each row are touched.
 * rope: device fp32 [*, head_dim/2, 2] indexed by token = pos0 + i.  g: device bf16 [head_dim]. */
int xema_op_rmsnorm_rope(void* x, int64_t ld, int64_t batch_rows, const void* g, const float* rope,
                         int32_t pos0, int32_t batch, int32_t rows, int32_t heads, int32_t head_dim,
                         float eps, void* stream);

/* Epilogues of the tensor-core GEMM acc = A[b] (rows x K) * W^T (N x K), fp32 accumulate. */
enum {
  XEMA_EPI_BIAS = 0,       /* out bf16 = acc + bias                                        */
  XEMA_EPI_BIAS_GELU = 1,  /* out bf16 = gelu_tanh(acc + bias)                             */
  XEMA_EPI_GATE_RES_F32 = 2,  /* out fp32 = resid(bf16) + gate[b,:] * (acc + bias)         */
  XEMA_EPI_GATE_RES_BF16 = 3, /* out bf16 = resid(fp32) + gate[b,:] * (acc + bias)         */
  XEMA_EPI_BIAS_NORM_ROPE = 4 /* out bf16 = acc + bias; heads that start below column
                                 norm_cols additionally get RoPE(RMSNorm(.) * norm_gain), the
                                 same arithmetic as xema_op_rmsnorm_rope but on the fp32
                                 accumulator (one rounding less).  Needs N % 256 == 0.        */
};
typedef struct xema_gemm_args {
  const void* a;        /* device bf16, row (b,i) at element (b*a_batch_rows + i)*lda      */
  int64_t lda, a_batch_rows;
  const void* w;        /* device bf16 [N, K], row stride ldw                              */
  int64_t ldw;
  const void* bias;     /* device bf16 [N]                                                 */
  void* out;            /* device, row (b,i) at element (b*out_batch_rows + i)*ldo         */
  int64_t ldo, out_batch_rows;
  const void* resid;    /* device, same row addressing with ldr / resid_batch_rows; or NULL */
  int64_t ldr, resid_batch_rows;
  const float* gate;    /* device fp32, gate[b*gate_stride + n]; or NULL                   */
  int64_t gate_stride;
  int32_t batch, rows, N, K; /* N % 128 == 0, K % 64 == 0                                  */
  int32_t epilogue;     /* XEMA_EPI_*                                                      */
  /* XEMA_EPI_BIAS_NORM_ROPE only (ignored otherwise): */
  int32_t head_dim;     /* 64 or 128                                                       */
  int32_t norm_cols;    /* multiple of head_dim, <= N: columns [0, norm_cols) are heads to
                           normalise and rotate (D for a K|V product, N for a Q product)   */
  int32_t rope_pos0;    /* token index of row 0: row i uses table row rope_pos0 + i        */
  float rms_eps;
  float norm_out_scale; /* the normalised, rotated heads are multiplied by this before the
                           rounding to bf16; 0 means 1 (the other columns are never scaled)   */
  const void* norm_gain; /* device bf16 [head_dim]                                          */
  const float* rope;     /* device fp32 [tokens][head_dim/2][cos, sin]                      */
} xema_gemm_args;
int xema_op_gemm(const xema_gemm_args* args, void* status_dev, void* stream);

/* Non-causal attention of `rows` query rows against all `keys` keys, per (batch, head):
 * o = softmax(q k^T / sqrt(head_dim)) v, lse = log sum exp (natural log).
 * q: device bf16, row (b,i) at (b*q_batch_rows + i)*ldq, head h at feature h*head_dim.
 * k, v: device bf16, key (b,j) at (b*kv_batch_rows + j)*ldkv (k and v are separate base
 * pointers into the same rows).  o: device bf16 [B,rows,heads*head_dim] contiguous.
 * lse: device fp32 [B,heads,rows] or NULL.
 * q_scale (> 0): what q k^T is multiplied by to give exponents to base 2.  For a plain q pass
 * log2(e) / sqrt(head_dim).  Pass 1 if q was already multiplied by that -- the block does this in
 * the fused epilogue of the Q projection (norm_out_scale), where it costs no extra rounding: the
 * head_dim 64 kernel takes the exponents straight from the tensor core.  Given any other q_scale
 * that kernel multiplies its copy of the q tiles in shared memory first, which rounds q to bf16 a
 * second time (relative 2^-9 per element; visible where |q k^T| / sqrt(head_dim) reaches the
 * hundreds). */
int xema_op_attention(const void* q, int64_t ldq, int64_t q_batch_rows, const void* k, const void* v,
                      int64_t ldkv, int64_t kv_batch_rows, void* o, float* lse, int32_t batch,
                      int32_t rows, int32_t keys, int32_t heads, int32_t head_dim, float q_scale,
                      void* status_dev, void* stream);

/* ---- allocator plug-in ------------------------------------------------------------------ */
/* The paper's run-time mechanism for code that is not this library's own kernels (section
 * "Static memory runtime"; implementation: PyTorch's CUDAPluggableAllocator): a framework hands
 * every device allocation and release to xema_pluggable_malloc / xema_pluggable_free; one
 * step is recorded, its requests are laid out by xema_plan_arena, and from then on the k-th
 * request of a step is answered by a table lookup, arena + offset[k].
 *
 * These are the only entry points of the library that call cudaMalloc / cudaFree (in the
 * pass-through and record modes, and for requests that do not match the plan); they never
 * synchronise.  All state is process-wide and guarded by one mutex.
 *
 * Lifetimes are measured on a clock that ticks once per allocation: request i is born at its
 * own tick and dies at the tick of the first allocation after its release (at the end of the
 * recording if it was never released).  Everything a recorded step allocates must be released
 * before the next replayed step starts, because the next step gets the same addresses. */
enum { XEMA_ALLOC_PASSTHROUGH = 0, XEMA_ALLOC_RECORD = 1, XEMA_ALLOC_REPLAY = 2 };

/* Signatures CUDAPluggableAllocator expects.  size in bytes; device and stream are ignored
 * (the current device is used).  malloc returns NULL on failure (see xema_last_cuda_error)
 * and for size 0 (empty requests are not part of a recording); free of an address inside the
 * planned arena does nothing. */
void* xema_pluggable_malloc(ptrdiff_t size, int device, void* stream);
void xema_pluggable_free(void* ptr, ptrdiff_t size, int device, void* stream);

/* Switches mode.  -> RECORD clears the previous recording and plan; leaving RECORD closes the
 * lifetimes of requests still live; -> REPLAY needs a plan (XEMA_ESTATE otherwise) and starts
 * at request 0. */
int xema_pluggable_mode(int mode);
/* The recording as tensors (bytes rounded up to 256, birth, death; name "req<i>") in request
 * order, for xema_plan_arena.  out: host, capacity cap; *n_requests and *n_events (host) are
 * always written; XEMA_ENOSPC when cap is too small; XEMA_ESTATE while still recording. */
int xema_pluggable_recorded(xema_tensor* out, size_t cap, size_t* n_requests, uint32_t* n_events);
/* Installs the plan: arena_dev (device, 256-aligned, caller-owned, must outlive replay),
 * offsets (host, one per recorded request, multiples of 256).  Only in pass-through mode. */
int xema_pluggable_set_plan(void* arena_dev, uint64_t arena_bytes, const uint64_t* offsets, size_t n);
/* Replay mode: the next request is request 0 again. */
int xema_pluggable_step_begin(void);
/* Counters since load: requests served from the arena, requests that fell back to cudaMalloc
 * in replay mode, and the index the next request will be matched against.  Any may be NULL. */
int xema_pluggable_stats(uint64_t* served, uint64_t* fallback, uint64_t* next_index);

/* ---- diagnostics ------------------------------------------------------------------------ */
/* Every wait inside the kernels (on an mbarrier fed by TMA, by the tensor pipe or by another
 * warp) is bounded: when the limit runs out the CTA stops, frees its TMEM, stores
 * XEMA_DEVICE_STATUS_TIMEOUT in the caller's status word and returns; the forward call's work
 * is then incomplete but the context stays usable.  This self-test launches one small kernel
 * that waits, with `limit_cycles` (1 .. 4e9 SM clock cycles) as its limit, on a barrier nothing
 * completes, so the mechanism can be exercised without faulting or hanging a GPU.
 * status_dev: device, 4 zeroed bytes, receives XEMA_DEVICE_STATUS_TIMEOUT.  waited_cycles_dev:
 * device int64 or NULL, receives the cycles the wait took. */
#define XEMA_DEVICE_STATUS_TIMEOUT 0x54310001u
int xema_selftest_wait_timeout(void* status_dev, int64_t limit_cycles, int64_t* waited_cycles_dev,
                               void* stream);

const char* xema_strerror(int status);
/* Last cudaError_t / CUresult seen by this thread's most recent failing call (0 if none). */
int xema_last_cuda_error(void);
/* Library version string, e.g. "xema-b200 0.1 (sm_100a)". */
const char* xema_version(void);

#ifdef __cplusplus
}
#endif
#endif /* XEMA_H_ */
