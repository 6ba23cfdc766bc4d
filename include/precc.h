/*
 * precc -- shared base KV cache + per-agent low-rank (LR) KV cache path for
 * multi-LoRA agents, hand-written for NVIDIA B200 (sm_100a).
 *
 * The library implements, for ONE decoder layer, the cache path of PReCache:
 *
 *   Eq. 1            Y_i = X (W0 + A_i B_i) = X W0 + (X A_i) B_i
 *   Section 2.2      base cache X W0 (shared by all agents) + LR cache X A_i (width r, per agent)
 *   Section 3.1      PreLRShared: when a segment is first processed, X A_k is built for EVERY agent k
 *   Section 3.2      ReBaseShared: the base cache is rebuilt as X_neut W0 from adapter-free hidden states
 *   Section 4.1 /    attention of the current agent over the base cache plus its own LR cache without
 *   Appendix D.2     materialising the agent's K or V (the adapter is folded into the query side and
 *                    into the output side by associativity)
 *
 * with the usual LoRA scale s = alpha / r:  K_a = K_base + s_k (H A_a^K) B_a^K,  V_a likewise.
 * The main path is position-free (no rotary embedding is applied).  The *_rope entry points at the
 * end of this header are the rotary-key variant of Appendix D.2.
 *
 * Conventions
 *   - All tensors are bf16 in DEVICE memory unless stated; all accumulation is fp32; stores round to
 *     nearest even.  Index arrays are int32 in DEVICE memory unless stated.
 *   - Every buffer is owned by the caller.  Apart from the 8 bytes (status word, wait limit) that precc_create obtains
 *     (and precc_destroy releases) the library allocates no device memory; it keeps no pointer after the
 *     work it enqueued on `stream` has completed.  `stream` is a cudaStream_t passed as void* (NULL = the
 *     default stream).  The compute calls are asynchronous with respect to the host and can be captured
 *     into a CUDA graph (they neither synchronise nor allocate; precc_poll_status synchronises).
 *   - Return value: PRECC_OK or an error code.  On a host-detected error nothing is launched and no
 *     output is touched.  Text for the last error of a context: precc_last_error().
 *   - A context may be used from one host thread at a time; different contexts may be used from
 *     different threads (kernel launch limits shared by all contexts of a device are kept under a lock).
 *
 * HBM layouts (PRECC_PAGE = 16 tokens per block; token slot s lives in block s / 16 at offset s % 16)
 *   base K, base V : [n_blocks][n_kv_heads][16][head_dim]
 *   LR K, LR V     : [n_agents][n_blocks][16][rank]          (one row per token, shared by all kv heads)
 *   q, out         : [rows][n_q_heads][head_dim]
 *   B_k, B_v       : [n_agents][rank][n_kv_heads*head_dim]   (the paper's B_i, r x d_out)
 *   packed A       : [n_agents*(rank_k+rank_v)][d_model]      rows ordered [projection K,V][agent][r]
 *   packed W       : [2*n_kv_heads*head_dim][d_model]         rows ordered [projection K,V][kv head][c]
 *   A "contiguous" cache is the same layout addressed without a block table (logical block i of a
 *   sequence = physical block first_block + i).
 *
 * Supported shapes (anything else returns PRECC_ERR_UNSUPPORTED):
 *   head_dim in {64,128}; n_q_heads % n_kv_heads == 0 with group size <= 8;
 *   (rank_k, rank_v) in {(0,0), (0,r), (r,r)} with r in {8,16,32,64}; d_model % 64 == 0;
 *   n_agents <= 64.
 */
#ifndef PRECC_H_
#define PRECC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PRECC_PAGE 16

enum {
  PRECC_OK = 0,
  PRECC_ERR_INVALID_ARG = 1,   /* null pointer, negative size, inconsistent sizes */
  PRECC_ERR_UNSUPPORTED = 2,   /* shape outside the supported set above */
  PRECC_ERR_MISALIGNED = 3,    /* a tensor pointer is not 16-byte aligned */
  PRECC_ERR_WORKSPACE = 4,     /* workspace missing or too small */
  PRECC_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed (text in precc_last_error) */
  PRECC_ERR_DEVICE_STATUS = 6  /* a kernel recorded a problem (see precc_poll_status) */
};

/* Bits of the device status word read by precc_poll_status(). */
#define PRECC_STATUS_BAD_INDEX 1u /* an agent id / block id / slot was out of range and was skipped  */
#define PRECC_STATUS_TIMEOUT 2u   /* a bounded wait inside a kernel expired (results are invalid)    */

typedef struct precc_ctx precc_ctx;

/* One decoder layer's KV-path geometry (host struct, read during the call only). */
typedef struct {
  int32_t d_model;
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t n_agents;
  int32_t rank_k, rank_v;      /* 0 = that projection carries no adapter (the paper's default adapts Q,V: rank_k = 0) */
  float lora_scale_k;          /* s for the key side; 1.0 is Eq. 1 literally */
  float lora_scale_v;          /* s for the value side */
  float softmax_scale;         /* <= 0 selects 1/sqrt(head_dim) */
} precc_layer_desc;

/* Caller-owned caches of one layer (device pointers, layouts above). lr_k / lr_v may be NULL when
 * the corresponding rank is 0. */
typedef struct {
  void* k_base;
  void* v_base;
  void* lr_k;
  void* lr_v;
  int64_t n_blocks;            /* physical blocks in each of the four arrays */
} precc_cache;

/* Create a context for CUDA device `device` (host allocation only, plus 8 bytes of device memory - the status
 * word and the wait limit - obtained with cudaMalloc here and released in precc_destroy). */
int32_t precc_create(precc_ctx** out, int32_t device);
int32_t precc_destroy(precc_ctx* ctx);
/* Text of the last error seen by `ctx` (owned by ctx, valid until the next call on it). */
const char* precc_last_error(const precc_ctx* ctx);
const char* precc_error_name(int32_t code);
/* Number of SMs of the context's device (the split schedule of decode depends on it). */
int32_t precc_sm_count(const precc_ctx* ctx);

/* Tracing (optional).  Give the context a caller-owned DEVICE buffer of n_blocks * 16 uint64 entries;
 * while it is set, each thread block of precc_lr_attend_decode whose grid has at most n_blocks blocks
 * records the GPU nanosecond timer at points of its life at entry [block][point]: 0 start, 1 indices
 * read, 2 stream issued, 3 query fold ready, 4 first tile landed, 5 stream done, 7 done, 8 / 9 just before and after
 * the wait for the preceding kernel, 11 all warps of the block have left the stream, 13 warp records written, 14 block
 * merge done.  Ticket schedule: 6 record published, and the merging block reuses 8 and 9 - partials gathered, weights
 * ready - and records 10 merged.  Cluster schedule: 6 sends issued, 12 everything addressed to the block received, and the id of the SM
 * the block runs on at entry 15.  Entries not written stay as they were.  Pass NULL to switch tracing off (the
 * default).  There is no paper counterpart. */
int32_t precc_set_trace_buffer(precc_ctx* ctx, void* buffer, size_t n_blocks);

/* Read the device status word accumulated by kernels launched through `ctx`, then clear it.
 * Synchronises `stream`.  *status_out receives an OR of PRECC_STATUS_* bits.  Returns PRECC_OK when the
 * word is zero, PRECC_ERR_DEVICE_STATUS otherwise. */
int32_t precc_poll_status(precc_ctx* ctx, void* stream, uint32_t* status_out);

/* Bounded waits (no paper counterpart).  Every wait inside a kernel of this library - on an mbarrier that a TMA
 * copy or a tensor-core commit completes - gives up after a limit, records PRECC_STATUS_TIMEOUT and lets the kernel
 * run to its end (freeing its tensor memory); results of that launch are void, the context stays usable.  The limit
 * is a number of SM clock cycles, about one second by default (sm_cycles == 0 restores the default); it is rounded
 * up to a multiple of 1024 cycles.  The call synchronises with nothing: set it while no kernel of this context runs. */
int32_t precc_set_wait_limit(precc_ctx* ctx, uint64_t sm_cycles);
/* Self-test of that mechanism: one tiny kernel waits on a barrier that is never completed.  It must end by itself
 * after the wait limit; *done_flag (device uint32) then holds 2 and precc_poll_status reports
 * PRECC_STATUS_TIMEOUT.  With the default limit this takes about a second of GPU time: lower the limit first. */
int32_t precc_selftest_wait_timeout(precc_ctx* ctx, uint32_t* done_flag, void* stream);

/* Pack a row-major [d_model][n_cols] matrix (paper layout d_in x d_out) as rows [dst_row0, dst_row0 +
 * n_cols) of a packed matrix of dst_rows rows, the operand format of the projection kernels: k-blocked
 * K-major, element (row, i) at ((i / 64) * dst_rows + row) * 64 + i % 64, holding src[i][row - dst_row0]
 * (the 64-deep k step of any run of rows is contiguous, one TMA box).  dst has dst_rows * d_model
 * elements and must be packed with the dst_rows it is later used with.  Used to build the packed A (all
 * agents' down-projections side by side, Section 3.1), the packed W and the two together.  src, dst
 * device; d_model % 64 == 0.
 * Packed matrices are constants of the projection calls: a projection of up to 64 rows is a programmatic
 * dependent launch and requests its first weight boxes before it waits for the kernel ahead of it on the stream
 * (H, the slot and mask arrays and every store come after that wait).  precc_pack_kmajor itself never lets a
 * dependent launch start early, so packing and projecting back to back on one stream is ordered as usual. */
int32_t precc_pack_kmajor(precc_ctx* ctx, const void* src, int32_t d_model, int32_t n_cols,
                          void* dst, int32_t dst_rows, int32_t dst_row0, void* stream);

/* LR-cache precompute (Section 3.1, PreLRShared): L_k^p = H A_k^p for every agent k whose bit is set
 * in agent_mask and both projections p, written to the LR caches at the tokens' slots.
 *   H            [M][d_model]
 *   A_packed     n_agents*(rank_k+rank_v) packed rows (precc_pack_kmajor output): agent-major K rows, then V rows
 *   slot_mapping [M] physical token slots, or NULL for slots start_slot .. start_slot+M-1
 *   agent_mask   bit k = write agent k (all agents: PreLRShared; all but the current one: the
 *                adapter-free pass of ReBaseShared; only the current one: its adapted pass)
 * Slots outside [0, 16*n_blocks) are skipped and PRECC_STATUS_BAD_INDEX is recorded.  M == 0 is a no-op. */
int32_t precc_lr_precompute(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M,
                            const void* A_packed, const int32_t* slot_mapping, int64_t start_slot,
                            uint64_t agent_mask, const precc_cache* cache, void* stream);

/* Base-cache (re-)projection (Section 3.2, ReBaseShared; also the in-turn append): K_base[slot] = H W_k,
 * V_base[slot] = H W_v for each of the M rows; existing slots are overwritten.
 *   H [M][d_model];  W_packed: 2*n_kv_heads*head_dim packed rows (W_k columns, then W_v columns);
 *   slot_mapping / start_slot as above. */
int32_t precc_rebase_project(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M,
                             const void* W_packed, const int32_t* slot_mapping, int64_t start_slot,
                             const precc_cache* cache, void* stream);

/* Both of the above in one pass over H (Section 3.1: the hidden states of a newly processed segment
 * feed the base cache and every agent's LR cache; Section 3.2: the adapter-free pass writes the neutral
 * base rows and the other agents' LR rows).  H is read from HBM once and one kernel runs instead of two.
 *   WA_packed  2*n_kv_heads*head_dim + n_agents*(rank_k+rank_v) packed rows: the W rows followed by the A
 *              rows (precc_pack_kmajor into one buffer of that many rows)
 *   agent_mask selects the LR caches written; the base rows are always written.
 * Results are bit-identical to precc_rebase_project followed by precc_lr_precompute with the same M (the
 * three calls pick their kernel from M, d_model and the layer's fused width alone, so they agree).  The same
 * row projected in calls of different M may differ in the last bf16 bit: few rows (a decode step), a short
 * turn and a long segment run on three kernels whose fp32 summation orders differ. */
int32_t precc_turn_project(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M,
                           const void* WA_packed, const int32_t* slot_mapping, int64_t start_slot,
                           uint64_t agent_mask, const precc_cache* cache, void* stream);

/* precc_turn_project with one agent mask per row (double batching, Section 3.2: the adapted and the
 * adapter-free sequence of a turn ride in one batch — the adapted rows write only the current agent's LR
 * rows, the adapter-free rows write the other agents').  Every row writes its base rows at its own slot, so
 * the two sequences must map to different slots (e.g. private blocks for the adapted one).
 *   slot_mapping     [M] required;  row_agent_masks  device uint64 [M], bit k = write agent k for that row
 *   lr_copy_slots    optional device int32 [M] (NULL = none): a second slot that also receives the LR rows the
 *                    row writes (entry < 0: none for that row).  The adapted sequence keeps its base rows in
 *                    private blocks, which are dropped after the turn, but its own LR rows (built from the
 *                    adapted hidden states, Section 3.2) belong to the shared trajectory for good: they are
 *                    written at the private slot, where this turn's attention finds them through the adapted
 *                    block table, and at the token's shared slot.  A slot >= 16*n_blocks raises
 *                    PRECC_STATUS_BAD_INDEX. */
int32_t precc_turn_project_rows(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M,
                                const void* WA_packed, const int32_t* slot_mapping,
                                const uint64_t* row_agent_masks, const int32_t* lr_copy_slots,
                                const precc_cache* cache, void* stream);

/* Workspace size for precc_lr_attend_decode with at most max_batch requests of at most max_ctx tokens
 * on a device with `sm_count` SMs: an upper bound over every such call (a smaller batch splits each request
 * further, so the bound is taken over all batch sizes up to max_batch).  The workspace must be zeroed once (precc_workspace_init) before its
 * first use; calls leave it ready for the next call.  Two calls that may run concurrently need
 * separate workspaces. */
size_t precc_decode_workspace_bytes(const precc_layer_desc* desc, int32_t max_batch, int32_t max_ctx,
                                    int32_t sm_count);
int32_t precc_workspace_init(precc_ctx* ctx, void* workspace, size_t workspace_bytes, void* stream);

/* LR-reconstructed decode attention (Sections 3.1, 4.1): for request b with agent a = agent_id[b] and
 * every q head h (kv head g = h / (n_q_heads/n_kv_heads)):
 *   z_t  = softmax_scale * ( q_h . K_base[t,g] + s_k (q_h B^K_{a,g}^T) . L^K_a[t] ),   t < ctx_len[b]
 *   out_h = sum_t softmax(z)_t V_base[t,g] + s_v (sum_t softmax(z)_t L^V_a[t]) B^V_{a,g}
 * which equals plain attention with K_a = K_base + s_k L^K_a B^K_a and V_a likewise (Eq. 1).
 *   q, out        [B][n_q_heads][head_dim]
 *   agent_id      [B] in [0, n_agents), or -1 for the adapter-free view of Section 3.2 (double batching:
 *                 the request attends to its base cache only; no LR row and no B matrix is touched);
 *                 ctx_len [B] >= 1 (a request with ctx_len < 1 gets zeros)
 *   block_table   [B][table_stride] logical block -> physical block, or NULL
 *   first_block   [B] physical block of logical block 0 when block_table is NULL (NULL = 0 for all)
 *   max_ctx       HOST upper bound on every ctx_len[b]; with B and the SM count it fixes the split of
 *                 the context across thread blocks, so results are bit-identical for any block
 *                 placement given the same (B, max_ctx)
 *   B_k, B_v      [n_agents][rank][n_kv_heads*head_dim]
 * A request whose ctx_len exceeds max_ctx is rejected on the device: zeros, PRECC_STATUS_BAD_INDEX.
 * B == 0 is a no-op.
 * Overlap with the kernel before it on the stream.  The launch is a programmatic dependent launch: where the
 * preceding kernel permits it (of this library: another decode or combine launch, and the few-row projection
 * that serves calls of at most 64 rows; kernels of other libraries normally do not) the decode kernel starts
 * while that kernel still runs and, before it waits for it to finish, already reads ctx_len, agent_id, the block
 * table / first_block, B_k, B_v and every cache page that holds none of the request's last 64 tokens (logical
 * positions ctx_len-64 .. ctx_len-1).  q, the pages holding those last 64 tokens and every store come after the
 * wait.  So the immediately preceding kernel may produce q and may append or overwrite the request's newest
 * tokens (the in-turn append of Section 3.1, the ReBaseShared overwrite of a just-appended short segment), but
 * if it is one of the kernels named above it must not write the index arrays, the B matrices or older cache
 * rows of the attended requests; put any other kernel or an event between the two otherwise. */
int32_t precc_lr_attend_decode(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                               const int32_t* agent_id, const int32_t* ctx_len,
                               const int32_t* block_table, int32_t table_stride,
                               const int32_t* first_block, int32_t max_ctx,
                               const void* B_k, const void* B_v, const precc_cache* cache,
                               void* out, void* workspace, size_t workspace_bytes, void* stream);

/* The same decode attention for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a property of the library, not of the method).  Some users of this library run
 * where cudaMalloc is off limits: a serving engine that handed every free byte of HBM to its KV-cache
 * pool at start-up, code running while a stream is being captured (allocation is illegal there), or a
 * latency-critical decode loop that must not take cudaMalloc's device-wide synchronisation.  For them the
 * split-merge scratch of precc_lr_attend_decode lives in an array compiled into the library
 * (PRECC_STATIC_SCRATCH_BYTES of device memory, held by every GPU that loads the library until the
 * process exits) instead of a caller workspace.  Arguments and results are those of
 * precc_lr_attend_decode without `workspace`.
 *   - If precc_decode_workspace_bytes(desc, B, max_ctx, sm_count) exceeds PRECC_STATIC_SCRATCH_BYTES the
 *     call returns PRECC_ERR_WORKSPACE (the message names both sizes) and launches nothing.
 *   - The call allocates nothing: no cudaMalloc / cudaFree, no allocating library routine.
 *   - The first call on a device looks up the device address of the array (the context's device must be
 *     the current device).  Make that first call outside any stream capture.
 *   - Every call on a device shares the one array.  The part that must start at zero is cleared on
 *     `stream` at the start of each call; the rest keeps the previous call's contents.  Two calls that
 *     may overlap on the GPU (different streams, or different contexts on the same device) race on it:
 *     serialise them, or give one of them precc_lr_attend_decode with its own workspace. */
#define PRECC_STATIC_SCRATCH_BYTES (8u << 20)
int32_t precc_lr_attend_decode_static(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                                      const int32_t* agent_id, const int32_t* ctx_len,
                                      const int32_t* block_table, int32_t table_stride,
                                      const int32_t* first_block, int32_t max_ctx,
                                      const void* B_k, const void* B_v, const precc_cache* cache,
                                      void* out, void* stream);

/* LR-reconstructed attention for the S new tokens of a turn (Section 3.1: the current agent computes
 * only over the newly added context and reuses base + own LR cache for the rest).  The caches must
 * already cover the new tokens (precc_rebase_project + precc_lr_precompute on them first).  Query i
 * (0 <= i < S) attends logical positions 0 .. ctx_len + i: the old context fully, the new tokens
 * causally.  Same formula as decode.
 *   q, out       [S][n_q_heads][head_dim]
 *   agent        the current agent, or -1 for the adapter-free pass over the neutral base cache (host
 *                value);  ctx_len  T, tokens before the new ones (host value)
 *   block_table  [table_stride] logical -> physical block for this sequence, or NULL
 *   first_block  physical block of logical block 0 when block_table is NULL
 * No workspace is needed.  S == 0 is a no-op. */
int32_t precc_lr_attend_prefill(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S,
                                int32_t agent, int32_t ctx_len, const int32_t* block_table,
                                int32_t table_stride, int32_t first_block,
                                const void* B_k, const void* B_v, const precc_cache* cache,
                                void* out, void* stream);

/* precc_lr_attend_prefill with a caller-provided workspace (Section 3.1; the workspace has no counterpart
 * in the paper).  A turn whose (row tile, kv head) blocks fill more than half of the SMs but not all of
 * them - 512 new tokens of 8 kv heads are 128 blocks on 148 SMs - runs in one wave that leaves SMs idle.
 * With a workspace each block stops some way before the end of its context and helper blocks on the idle
 * SMs take the remaining steps of all tiles; the pieces of a tile are written to the workspace as fp32
 * partial results (maximum, denominator, numerator) and merged, in a fixed order, by whichever block
 * finishes last.  Same arguments and errors as precc_lr_attend_prefill, plus
 *   ws, ws_bytes  device, 256-byte aligned (PRECC_ERR_MISALIGNED otherwise); precc_prefill_ws_bytes(ctx,
 *                 desc, S) bytes are always enough; contents on entry do not matter, the call clears what
 *                 must start at zero on `stream`; the caller owns it and may reuse it for the next call on
 *                 the same stream.  Two calls that may overlap on the GPU need separate workspaces.
 * With ws == NULL, a workspace that is too small, a turn length for which precc_prefill_ws_bytes returns 0,
 * a short context, or where the tensor-memory kernel does not take the call, the call behaves exactly like
 * precc_lr_attend_prefill.  Where helper blocks are used the result differs from precc_lr_attend_prefill
 * in rounding only (another summation order over the context); it is the same from run to run. */
size_t precc_prefill_ws_bytes(const precc_ctx* ctx, const precc_layer_desc* desc, int32_t S);
int32_t precc_lr_attend_prefill_ws(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S,
                                   int32_t agent, int32_t ctx_len, const int32_t* block_table,
                                   int32_t table_stride, int32_t first_block,
                                   const void* B_k, const void* B_v, const precc_cache* cache,
                                   void* out, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------- rotary keys (Appendix D.2)
 * With a rotary position embedding the agent's key row of token t is RoPE_t(H_t (W_k + s_k A B)): the
 * rotation sits between the rank-r term and the query, so the rank-r term must be expanded to full
 * width and rotated before it meets q.  In this variant
 *   - the base K cache holds ROTATED rows RoPE_t(H_t W_k) (written by the *_project_rope calls),
 *   - the LR-K cache holds UNROTATED rows H_t A_a^K (precc_lr_precompute / the LR columns of
 *     precc_turn_project_rope, unchanged),
 *   - decode expands L^K B^K_{a,g} page by page on chip, rotates it by the tokens' positions and adds it
 *     to the rotated base rows; K_a is never written to memory.  V is not rotated.
 *   - q must already be rotated by the caller (the query projection is outside this library).
 * Convention: rotate-half pairing, coordinates (c, c + head_dim/2) of a head turn by angle(t, c):
 *   x'[c] = x[c] cos - x[c + hd/2] sin,   x'[c + hd/2] = x[c + hd/2] cos + x[c] sin.
 * Cached token t sits at position t in decode and prefill (the new tokens of a turn at ctx_len + i). */
typedef struct precc_rope {
  const float* table;        /* device fp32 [max_pos][head_dim/2][2]: (cos, sin) of angle(t, c); 16-byte aligned */
  int32_t max_pos;           /* rows of `table` */
  const int32_t* positions;  /* projection calls: device [M] position of each projected row, or NULL for
                                start_pos + i.  Ignored by decode, where cached token t sits at position t. */
  int64_t start_pos;
} precc_rope;

/* precc_rebase_project with the key columns rotated by each row's position before the store.  A
 * position outside [0, max_pos) raises PRECC_STATUS_BAD_INDEX and that row is not written. */
int32_t precc_rebase_project_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M,
                                  const void* W_packed, const int32_t* slot_mapping, int64_t start_slot,
                                  const precc_rope* rope, const precc_cache* cache, void* stream);

/* precc_turn_project with rotated base K rows; the LR rows are written unrotated. */
int32_t precc_turn_project_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* H, int32_t M,
                                const void* WA_packed, const int32_t* slot_mapping, int64_t start_slot,
                                uint64_t agent_mask, const precc_rope* rope, const precc_cache* cache,
                                void* stream);

/* precc_lr_attend_decode over rotated base keys.  Same arguments plus `rope` (max_pos >= max_ctx; a
 * context longer than max_pos raises PRECC_STATUS_BAD_INDEX and clamps the position).  The workspace
 * of precc_decode_workspace_bytes suffices.  With rank_k == 0, or for agent id -1, the result equals
 * precc_lr_attend_decode (the rotated base cache is all there is). */
int32_t precc_lr_attend_decode_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                                    const int32_t* agent_id, const int32_t* ctx_len,
                                    const int32_t* block_table, int32_t table_stride,
                                    const int32_t* first_block, int32_t max_ctx,
                                    const void* B_k, const void* B_v, const precc_rope* rope,
                                    const precc_cache* cache, void* out, void* workspace,
                                    size_t workspace_bytes, void* stream);

/* precc_lr_attend_prefill over rotated base keys (rope->max_pos >= ctx_len + S).  The rank-r key term of
 * every 64-token tile is expanded, rotated and added to the tile in shared memory before the scores are
 * taken.  With rank_k == 0, or for agent -1, the result equals precc_lr_attend_prefill. */
int32_t precc_lr_attend_prefill_rope(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S,
                                     int32_t agent, int32_t ctx_len, const int32_t* block_table,
                                     int32_t table_stride, int32_t first_block,
                                     const void* B_k, const void* B_v, const precc_rope* rope,
                                     const precc_cache* cache, void* out, void* stream);

/* The same attention as precc_lr_attend_prefill_rope, computed the fast way at the price of a scratch area
 * (Appendix D.2 leaves the mechanics open; the paper's own path never materialises adapted keys).  The adapted rotary
 * keys of THIS sequence - K_base_rot[t] + s_k RoPE_t(L^K_a[t] B^K_a) for its ctx_len + S tokens, all kv heads - are
 * written once into `key_scratch` (device, 128-byte aligned, at least precc_prefill_rope_scratch_bytes(desc, ctx_len,
 * S) bytes = the sequence's base-key bytes rounded up to whole 128-token steps), in logical block order, and the
 * tensor-core prefill kernel then streams them as its key operand; values and the value-side adapter are used from
 * the caches as usual.  The scratch is transient: its contents are unspecified after the call and it can be reused
 * by the next layer or sequence on the same stream.  Results agree with precc_lr_attend_prefill_rope within the
 * attention tolerance (the key term is rounded to bf16 once here, twice there).  With rank_k == 0, for agent -1,
 * or where the tensor-core kernel does not apply (unaligned caches), the call behaves exactly like
 * precc_lr_attend_prefill_rope and leaves the scratch untouched.  A scratch that is too small returns
 * PRECC_ERR_WORKSPACE and launches nothing. */
size_t precc_prefill_rope_scratch_bytes(const precc_layer_desc* desc, int32_t ctx_len, int32_t S);
int32_t precc_lr_attend_prefill_rope_scratch(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t S,
                                             int32_t agent, int32_t ctx_len, const int32_t* block_table,
                                             int32_t table_stride, int32_t first_block,
                                             const void* B_k, const void* B_v, const precc_rope* rope,
                                             const precc_cache* cache, void* out, void* key_scratch,
                                             size_t key_scratch_bytes, void* stream);

/* ------------------------------------------------------------- context-sharded decode (no paper counterpart)
 * When the tokens of a request are spread over several GPUs (each holds base and LR rows of a contiguous
 * token range in its own caches), softmax attention over the union is the split-KV merge taken once more
 * across GPUs.  Each shard calls precc_lr_attend_decode_partial over its LOCAL tokens; the records of all
 * shards are gathered (e.g. an NCCL all-gather) into [n_shards][B][n_kv_heads][R] floats, R =
 * precc_partial_record_floats(desc); precc_combine_partials merges them in shard order and applies the
 * value-side epilogue.  The result equals precc_lr_attend_decode over the concatenated context up to fp32
 * summation order.  Position-free path only.
 *   record = [ m[8] | l[8] | O'[group][head_dim + rank_v] ] fp32: running maximum (log2 domain), softmax
 *            denominator and un-normalised output (with the rank_v LR-V coordinates appended) per query head
 *   ctx_len [B] local token counts; 0 is allowed (the shard holds nothing of that request) and yields the
 *            neutral record; max_ctx >= 1 bounds them
 *   agent ids, q, B_k, block tables, workspace: as for precc_lr_attend_decode (B_v is not needed here) */
size_t precc_partial_record_floats(const precc_layer_desc* desc);
int32_t precc_lr_attend_decode_partial(precc_ctx* ctx, const precc_layer_desc* desc, const void* q, int32_t B,
                                       const int32_t* agent_id, const int32_t* ctx_len,
                                       const int32_t* block_table, int32_t table_stride,
                                       const int32_t* first_block, int32_t max_ctx, const void* B_k,
                                       const precc_cache* cache, float* records, void* workspace,
                                       size_t workspace_bytes, void* stream);
/*   records  device fp32 [n_shards][B][n_kv_heads][R], 1 <= n_shards <= 64;  out [B][n_q_heads][head_dim].
 * A request with no token on any shard gets zeros. */
int32_t precc_combine_partials(precc_ctx* ctx, const precc_layer_desc* desc, const float* records,
                               int32_t n_shards, int32_t B, const int32_t* agent_id, const void* B_v,
                               void* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PRECC_H_ */
