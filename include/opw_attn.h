/*
 * opw_attn.h -- C ABI of the decode-time core-attention stage (sm_100a).
 *
 * The stage is the operator that core-attention disaggregation (CAD) places on its own
 * device group: per decode step a (micro)batch of one-token queries arrives together
 * with the step's new key/value rows, the rows are appended to a paged KV cache that
 * stays resident on the stage, grouped-query attention (full or sliding-window) runs
 * over each sequence's pages, and the attention output goes back to the next stage
 * (paper: Section 3.4 "From Bounds to Plans: CAD and Its Limits"; Section 4, the CAD
 * template "isolates only the core attention kernels"; Section 6, first paragraph:
 * slots, shapes and buffers are static and bound once while token, position and
 * KV-cache metadata change between iterations).
 *
 * Conventions that hold for every entry point:
 *   - Plain C: no C++ types, no exceptions cross this boundary.  Every call returns an
 *     opw_status_t; nothing aborts, traps or waits without a bound.
 *   - "DEVICE" pointers are CUDA device addresses on the stage's device; "HOST"
 *     pointers are ordinary host addresses.  The library never allocates or frees
 *     device memory: pools, workspace, inputs and outputs are caller-owned and must
 *     stay valid until the work enqueued on the stream has finished.
 *   - Step calls only enqueue work on the given stream (a cudaStream_t passed as
 *     void*, NULL = default stream) and return; they never synchronise and never read
 *     device metadata on the host, so launch shapes depend only on create-time
 *     constants and on the `batch` argument.
 *   - One handle is used from one host thread at a time.
 *
 * KV pool layout (per layer, part of this ABI).  bf16 elements.  Element
 * (page p, kv head g, kv in {K = 0, V = 1}, slot t in [0, page_size), dim d) is at
 *     ((((p*Hkv + g)*2 + kv)*page_size + t)*D) + (((d/8) ^ (t & 7))*8) + (d % 8).
 * So each (page, head) owns one contiguous K tile followed by one V tile, each
 * page_size rows of D elements; inside a row the eight-element (16-byte) groups are
 * permuted by XOR with the low three bits of the slot (this makes a tile that is
 * copied linearly into shared memory conflict-free for matrix loads).
 * opw_kv_pool_index() evaluates the formula on the host.
 */
#ifndef OPW_ATTN_H_
#define OPW_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct opw_attn_stage opw_attn_stage_t; /* opaque handle (host memory only) */

typedef enum {
  OPW_OK = 0,
  OPW_ERR_INVALID_ARG = 1, /* NULL pointer, index out of range, misaligned pointer, bad struct_size */
  OPW_ERR_UNSUPPORTED = 2, /* head_dim / page_size / group size the kernels do not cover */
  OPW_ERR_CAPACITY = 3,    /* batch > max_batch, workspace too small */
  OPW_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed (no device, bad stream ...) */
  OPW_ERR_BAD_PAGE = 5,    /* device side: a page id outside [0, num_pages) or a position beyond the table */
  OPW_ERR_TIMEOUT = 6      /* device side: a bounded wait on a shared-memory copy ran out */
} opw_status_t;

#define OPW_FLAG_NONE 0u
#define OPW_FLAG_NO_PDL 1u /* launch the kernels without programmatic stream serialisation (see opw_decode_attention) */
#define OPW_FLAG_COPY_STREAMS 2u /* opw_decode_step_host copies on the stage's own streams (see there) */

typedef struct {
  uint32_t struct_size;           /* sizeof(opw_attn_stage_config_t); checked at create */
  int32_t device;                 /* CUDA ordinal the stage lives on */
  int32_t num_layers;             /* layers this stage owns (>= 1) */
  int32_t num_q_heads;            /* Hq */
  int32_t num_kv_heads;           /* Hkv; Hq % Hkv == 0 and Hq / Hkv <= 16 (<= 8 at head_dim 256) */
  int32_t head_dim;               /* D: 64, 128 or 256 */
  int32_t page_size;              /* 16 */
  int32_t max_batch;              /* static slot count; every call has batch <= max_batch */
  int32_t max_pages_per_seq;      /* row stride (entries) of every page table */
  const int32_t *layer_window;    /* HOST [num_layers]; 0 = full attention, W > 0 = the last W keys
                                     including the current token (Section 3.4: efficient layers
                                     "access a bounded window") */
  const int64_t *layer_num_pages; /* HOST [num_layers]; physical pages in each layer's pool */
  void *const *layer_kv_pool;     /* HOST [num_layers] of DEVICE pointers, 128-byte aligned, each at
                                     least opw_kv_pool_bytes() long; caller-owned */
  void *workspace;                /* DEVICE, 256-byte aligned, caller-owned scratch */
  size_t workspace_bytes;         /* >= opw_attn_stage_workspace_bytes(cfg) */
  float softmax_scale;            /* 0 -> 1/sqrt(head_dim) */
  uint32_t flags;                 /* OPW_FLAG_* */
  int32_t tune_warps;             /* 0 = default (8; 6 at head_dim 256, 12 at head_dim 64); warps per thread block
                                     (1..16; what does not fit the register file is refused with OPW_ERR_CAPACITY) */
  int32_t tune_stages;            /* 0 = default; shared-memory ring depth per warp (2..16) */
  int32_t tune_ctas_per_sm;       /* 0 = default; resident thread blocks per SM (1..4) */
  int32_t reserved;               /* must be 0 */
} opw_attn_stage_config_t;

/* Host helper: the pool layout formula above.  No device needed. */
int64_t opw_kv_pool_index(int64_t num_kv_heads, int64_t page_size, int64_t head_dim, int64_t page,
                          int64_t kv_head, int64_t kv, int64_t slot, int64_t dim);

/* Host helper: bytes of one layer's pool holding num_pages pages (0 on invalid arguments). */
size_t opw_kv_pool_bytes(int32_t num_kv_heads, int32_t page_size, int32_t head_dim, int64_t num_pages);

/*
 * Host helper: scratch bytes the stage needs (status word, split-KV bookkeeping and two sets
 * of partial-result slots, staging buffers of the host-buffer step): on a 148-SM device about
 * 70 MB for 32/8 heads of 128 and 140 MB for 64/8 heads, plus 4 bytes per page-table entry
 * per layer for the staged tables.  Depends only on the
 * shape fields and the tune_* fields; device pointers in cfg are ignored.  Returns 0
 * if cfg is NULL or its shape fields are invalid.  Needs a CUDA device only to read
 * the SM count; without one it assumes 148 SMs.
 */
size_t opw_attn_stage_workspace_bytes(const opw_attn_stage_config_t *cfg);

/*
 * Binds the static part of the stage (Section 6: shapes, slots and buffers are bound
 * once).  Validates cfg on the host first (returning INVALID_ARG / UNSUPPORTED /
 * CAPACITY without touching CUDA), then selects the device, reads its SM count, raises
 * the kernels' shared-memory limit and clears the status word in the workspace
 * (synchronously, on the default stream).  Copies layer_window, layer_num_pages and
 * the pool pointers; those host arrays need not outlive the call.  *out is written
 * only on OPW_OK.
 */
opw_status_t opw_attn_stage_create(const opw_attn_stage_config_t *cfg, opw_attn_stage_t **out);

/*
 * Reads back the static shape a stage was bound with (Section 6: the shapes are fixed at
 * bind time): device ordinal, layer count, Hq, Hkv, D and max_batch.  Any out pointer may be
 * NULL.  For code layered on a stage that has only the opaque handle.
 */
opw_status_t opw_attn_stage_shape(const opw_attn_stage_t *stage, int32_t *device, int32_t *num_layers,
                                  int32_t *num_q_heads, int32_t *num_kv_heads, int32_t *head_dim,
                                  int32_t *max_batch);

/*
 * KV append (Section 6: KV-cache contents and metadata change every iteration).  For
 * every b < batch with positions[b] >= 0, copies k_new[b] and v_new[b] bit for bit into
 * slot positions[b] % page_size of page page_table[b][positions[b] / page_size] of the
 * layer's pool.  positions[b] < 0 marks an inactive slot (nothing written).
 *   k_new, v_new : DEVICE bf16 [batch, Hkv, D], 16-byte aligned
 *   positions    : DEVICE int32 [batch]; the pre-append length of each sequence
 *   page_table   : DEVICE int32 [batch, max_pages_per_seq]
 * Two rows of one call must not target the same (page, slot).  A page id outside
 * [0, num_pages) or a position beyond the table is skipped and recorded as
 * OPW_ERR_BAD_PAGE in the status word (see opw_attn_stage_poll_error).
 */
opw_status_t opw_kv_append(opw_attn_stage_t *stage, int32_t layer, int32_t batch, const void *k_new,
                           const void *v_new, const int32_t *positions, const int32_t *page_table,
                           void *cuda_stream);

/*
 * Decode attention (Section 3.1 and Appendix A: memory-bound, latency = KV bytes over
 * bandwidth; Section 3.4: full layers read the whole context, window layers a bounded
 * window).  For every b < batch with n = kv_lens[b] > 0 and every query head h:
 *     out[b,h,:] = sum_j softmax_j(scale * <q[b,h,:], K_j[h/G,:]>) V_j[h/G,:],
 *     lse[b,h]   = log sum_j exp(scale * <q[b,h,:], K_j[h/G,:]>)
 * over the keys j in [lo, n), lo = 0 for a full layer and max(0, n - W) for a window
 * layer; G = Hq/Hkv; keys are read through page_table[b][j / page_size].  Rows with
 * kv_lens[b] <= 0 are inactive: out = 0, lse = -inf.  bf16 inputs, fp32 accumulation,
 * bf16 output rounded to nearest even.
 *   q       : DEVICE bf16 [batch, Hq, D], 16-byte aligned
 *   kv_lens : DEVICE int32 [batch]; keys visible after this step's append
 *   page_table : DEVICE int32 [batch, max_pages_per_seq]; entries outside the visible
 *             range (after the last page, or wholly before the window) are never read
 *   out     : DEVICE bf16 [batch, Hq, D], 16-byte aligned
 *   lse     : DEVICE float [batch, Hq] or NULL
 * Enqueues two kernels (split-KV partial attention, then the log-sum-exp combine).  The
 * library's kernels are launched with programmatic stream serialisation: each may begin
 * (reading kv_lens / positions and the page table only) while the previous kernel in the stream
 * is finishing, and waits on the device -- every block of every grid, also one with nothing to
 * do -- before touching anything else, so the order of the stream is kept transitively.  One
 * obligation follows: kv_lens, positions and page_table must not be written by a kernel that
 * itself releases its dependents early (griddepcontrol.launch_dependents) before it has written
 * them; ordinary kernels and copies placed in the stream before the call are always complete
 * when the prologue runs.  It takes 1 to 5 percent off a step (most on small batches);
 * OPW_FLAG_NO_PDL switches it off.
 * The split of each sequence depends only on kv_lens and the window, never on the
 * page ids, so permuting physical pages leaves the output bitwise unchanged.  Bad page
 * ids are masked out and recorded as OPW_ERR_BAD_PAGE.
 */
opw_status_t opw_decode_attention(opw_attn_stage_t *stage, int32_t layer, int32_t batch, const void *q,
                                  const int32_t *kv_lens, const int32_t *page_table, void *out, float *lse,
                                  void *cuda_stream);

/*
 * Append and attention in one call, and in one kernel fewer: exactly opw_kv_append(k_new,
 * v_new, positions) followed by opw_decode_attention with kv_lens[b] = positions[b] + 1
 * (0 for positions[b] < 0), but the new rows are stored by the attention kernel itself --
 * the warp that streams the last page of sequence b and kv head g writes k_new[b,g,:] and
 * v_new[b,g,:] into the pool and into its shared-memory copy of that page -- so no separate
 * append launch and no dependency on one.  Same argument rules, the same bit-exact pool
 * contents afterwards and the same status-word reporting as the two calls.
 */
opw_status_t opw_decode_step(opw_attn_stage_t *stage, int32_t layer, int32_t batch, const void *q,
                             const void *k_new, const void *v_new, const int32_t *positions,
                             const int32_t *page_table, void *out, float *lse, void *cuda_stream);

/*
 * One whole stage step from HOST buffers (Section 4: the stage's activation interface
 * is the per-request q/k/v in and attention output back): copies q, k_new, v_new,
 * positions and (if not NULL) page_table to staging areas in the workspace, runs
 * opw_decode_step on them, and copies out (and lse if
 * not NULL) back to the host, all enqueued on the stream.  Host buffers should be
 * pinned for the copies to be asynchronous; they must stay valid and unmodified until
 * the stream has passed the step.  page_table_host == NULL reuses the table staged by
 * the previous call for this layer's slot (tables rarely change between steps).
 *
 * With OPW_FLAG_COPY_STREAMS (Section 4: a stage keeps several microbatches resident so that
 * transfers hide behind compute; Section 6.2: overlapping communication) the stage owns two
 * streams and three events of its own (created at opw_attn_stage_create; no device memory): the
 * copies in run on the first, the kernels on the caller's stream once the copies have landed, the
 * copies out on the second once the kernels are done.  The caller's stream then carries kernels
 * only: when two stages (two microbatches) take turns on ONE compute stream, the kernels of one
 * follow the kernels of the other directly and every copy runs beside the other stage's kernels.
 * Synchronising the caller's stream no longer covers the copy out: call
 * opw_attn_stage_wait_host_output before reading out_host / lse_host and before the stage's next
 * opw_decode_step_host.  Not for use under stream capture.
 */
/*
 * Tensor packing for opw_decode_step_host (Section 6.2, low-overhead communication: many short
 * transfers per token cost more than the bytes they carry).  Returns byte offsets inside one
 * host buffer of total_bytes at which q, k_new, v_new and positions may be placed; when the
 * four host pointers given to opw_decode_step_host sit at exactly these offsets of one buffer,
 * they are sent with a single copy instead of four.  The offsets depend on the stage's
 * max_batch and head counts only.
 */
opw_status_t opw_attn_stage_host_layout(const opw_attn_stage_t *stage, size_t *q_off, size_t *k_off, size_t *v_off,
                                        size_t *pos_off, size_t *total_bytes);

opw_status_t opw_decode_step_host(opw_attn_stage_t *stage, int32_t layer, int32_t batch, const void *q_host,
                                  const void *k_new_host, const void *v_new_host, const int32_t *positions_host,
                                  const int32_t *page_table_host, void *out_host, float *lse_host,
                                  void *cuda_stream);

/* Blocks the host until the copy out of the stage's latest opw_decode_step_host has finished (a stage created
 * with OPW_FLAG_COPY_STREAMS; otherwise returns at once: the caller synchronises its own stream). */
opw_status_t opw_attn_stage_wait_host_output(opw_attn_stage_t *stage);

/*
 * Page-table delta from HOST memory (Section 6, first paragraph: only token, position and KV-cache
 * metadata change between iterations; Section 6.2, low-overhead communication: many short transfers
 * cost more than the bytes they carry).  A sequence gets a new page once every page_size steps, so
 * re-sending its whole table row each step moves thousands of entries to change one.  This call
 * updates the table that opw_decode_step_host keeps staged for `layer` (the one its
 * page_table_host == NULL reuses): triples_host is int32 [n][3] = (batch row, logical page, physical
 * page), copied with one transfer and scattered by one small kernel, both enqueued on the stream;
 * the host array must stay valid until the stream has passed the copy (pinned for an asynchronous
 * copy).  The staged table must have been sent in full once (opw_decode_step_host with a non-NULL
 * page_table_host).  n == 0 enqueues nothing.  n > 4 * max_batch: OPW_ERR_CAPACITY.  A row or a
 * logical page outside the table is skipped and recorded as OPW_ERR_BAD_PAGE in the status word; the
 * physical page id is checked when a step reads it, as for any table.
 */
opw_status_t opw_attn_stage_page_table_delta_host(opw_attn_stage_t *stage, int32_t layer, const int32_t *triples_host,
                                                  int32_t n, void *cuda_stream);

/*
 * Plans: the per-token action sequence of a stage, enqueued by ONE native call (Section 6.2,
 * "Single native submission": the complete per-rank sequence is compiled once and each token
 * enqueues all graph launches with no host dispatch between stages and microbatches; Section 6,
 * first paragraph: slots, shapes and buffers are static and bound once, only token, position
 * and KV-cache metadata change between iterations).
 *
 * An item is one (layer, microbatch) visit: append k_new/v_new at `positions`, then attend
 * with `kv_lens`, exactly as opw_kv_append followed by opw_decode_attention with the same
 * arguments (k_new == v_new == NULL skips the append; kv_lens == NULL with k_new set means
 * kv_lens = positions + 1 and runs the fused opw_decode_step).  All pointers are DEVICE addresses of
 * caller-owned static buffers: a plan binds them once, and each submission reads whatever
 * they hold at that time (the caller refreshes q, k_new, v_new and, when pages are added, the
 * page table between submissions, on the same stream or ordered by an event).
 * Items run in the order given, one after the other (they share the stage's workspace).
 *   OPW_PLAN_GRAPH   : capture the sequence into a CUDA graph at create; submit is one
 *                      cudaGraphLaunch.  (Instantiating a graph lets the CUDA runtime allocate
 *                      its own bookkeeping; the library's kernels still use caller memory only.)
 *   OPW_PLAN_ADVANCE : after the last item, add 1 to every distinct positions array (entries
 *                      >= 0) and kv_lens array (entries > 0), so that re-submitting the plan
 *                      is the next decode step with no host work on the metadata.
 *   OPW_PLAN_OVERLAP : run item i's combine kernel on a private side stream (a parallel branch
 *                      of the graph) beside item i+1's split-KV kernel, alternating between the
 *                      stage's two workspace sets; the submission still completes only when
 *                      every output is final.  Consecutive items must then have different out
 *                      (and lse) buffers (OPW_ERR_INVALID_ARG otherwise).  Takes the combine and
 *                      one launch gap off the critical path of all items but the last.
 * create validates every item on the host (same rules and codes as the step calls) and, with
 * OPW_PLAN_GRAPH, captures on a private stream: nothing executes until submit.  A plan must be
 * destroyed before its stage.
 */
typedef struct {
  int32_t layer;
  int32_t batch;
  const void *q;             /* DEVICE bf16 [batch, Hq, D] */
  const void *k_new;         /* DEVICE bf16 [batch, Hkv, D] or NULL (no append) */
  const void *v_new;
  int32_t *positions;        /* DEVICE int32 [batch]; required with k_new */
  int32_t *kv_lens;          /* DEVICE int32 [batch], or NULL with k_new: positions + 1 */
  const int32_t *page_table; /* DEVICE int32 [batch, max_pages_per_seq] */
  void *out;                 /* DEVICE bf16 [batch, Hq, D] */
  float *lse;                /* DEVICE float [batch, Hq] or NULL */
} opw_step_item_t;

typedef struct opw_attn_plan opw_attn_plan_t;
#define OPW_PLAN_GRAPH 1u
#define OPW_PLAN_ADVANCE 2u
#define OPW_PLAN_OVERLAP 4u

opw_status_t opw_attn_plan_create(opw_attn_stage_t *stage, const opw_step_item_t *items, int32_t n_items,
                                  uint32_t flags, opw_attn_plan_t **out);
/* Enqueue one token's whole sequence on the stream (a graph launch, or the plain launches). */
opw_status_t opw_attn_plan_submit(opw_attn_plan_t *plan, void *cuda_stream);
/* NULL is accepted. */
opw_status_t opw_attn_plan_destroy(opw_attn_plan_t *plan);

/*
 * Failure-detection self-test.  Enqueues a one-warp kernel that waits, with the same bounded
 * wait the attention kernel uses for its shared-memory copies, on a barrier nothing will ever
 * complete; after the bound (0.1 s) it records OPW_ERR_TIMEOUT in the status word and exits.
 * The next opw_attn_stage_poll_error must return OPW_ERR_TIMEOUT, and the stage must keep
 * working afterwards.  No fault, trap or endless loop is involved.
 */
opw_status_t opw_attn_stage_probe_timeout(opw_attn_stage_t *stage, void *cuda_stream);

/*
 * Synchronises the stream, then returns and clears the device status word: OPW_OK, or
 * the first of OPW_ERR_BAD_PAGE / OPW_ERR_TIMEOUT recorded by a kernel since the last
 * poll.  The only entry point that blocks.
 */
opw_status_t opw_attn_stage_poll_error(opw_attn_stage_t *stage, void *cuda_stream);

/*
 * Tracing hook (the stage's counterpart of the offline operator profiles that feed the
 * paper's planner, Section 4 "profiled execution latency").  With a non-NULL DEVICE buffer
 * of at least 32 * workers bytes (8-byte aligned; *num_workers, if not NULL, receives the
 * worker count), every later opw_decode_attention launch makes each of its workers (one
 * warp each) record four uint64: {SM id | units << 32, begin, first tile ready, end}, the
 * times in nanoseconds of the device's global timer.  Workers with no work leave their
 * record untouched.  trace == NULL switches tracing off.  The buffer is caller-owned.
 */
opw_status_t opw_attn_stage_set_trace(opw_attn_stage_t *stage, void *trace, size_t trace_bytes,
                                      int32_t *num_workers);

/* Kernels launched through this handle since create (the library's own count). */
int64_t opw_attn_stage_launch_count(const opw_attn_stage_t *stage);

/*
 * Decode attention without any allocation, for callers that cannot obtain device memory.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * Some callers of this library are not allowed to call cudaMalloc, and so cannot provide the
 * workspace a stage needs: a plug-in inside a serving process whose device memory is owned
 * and fully pre-sized by the host framework, code running after the memory budget has been
 * spent, a latency-critical path that must never take the allocator's lock.  This variant
 * needs no stage handle and no workspace.  It computes exactly what opw_decode_attention
 * computes (same arguments, same conventions, same layout of kv_pool), with the split-KV
 * scratch held in a fixed array inside the library: about 10.7 MB of device memory on every
 * GPU that loads the library, from load until the process exits, used or not.
 *
 * Limits (OPW_ERR_CAPACITY beyond them, nothing is launched): batch <= 4096;
 * (Hq/Hkv) * (head_dim + 2) <= 1040, i.e. a group of at most 8 query heads per KV head at
 * head_dim 128; a device with at most 160 SMs.  head_dim 64 or 128 and page_size 16, else
 * OPW_ERR_UNSUPPORTED.  It calls no cudaMalloc, cudaFree or allocating library routine.
 *
 * The device that holds the buffers must be the current device.  The first call on a device
 * also resolves the scratch array's device address and sets kernel attributes; make that
 * first call outside any stream capture.  All calls on a device share the one array, which
 * keeps the previous call's contents (each call clears the words that must start at zero and
 * overwrites what it later reads): two calls whose kernels may overlap on the GPU -- on
 * different streams, or from different host threads -- race on it and must be serialised by
 * the caller.  It runs the split-KV kernel with equal static shares only, so it is somewhat
 * slower than a stage on long contexts.  Bad page ids are masked out as in
 * opw_decode_attention, but there is no status word to poll.
 *   kv_pool : DEVICE, one layer's pool (layout at the top of this file), 128-byte aligned
 *   q, kv_lens, page_table, out, lse : as for opw_decode_attention (lse may be NULL)
 *   window : 0 = full attention, W > 0 = the last W keys; softmax_scale 0 -> 1/sqrt(head_dim)
 */
opw_status_t opw_decode_attention_noalloc(int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                                          int32_t page_size, int32_t window, float softmax_scale,
                                          const void *kv_pool, int64_t num_pages, int32_t batch,
                                          int32_t max_pages_per_seq, const void *q, const int32_t *kv_lens,
                                          const int32_t *page_table, void *out, float *lse, void *cuda_stream);

/*
 * Read-bandwidth probe: the ceiling the attention stage is measured against, next to the
 * nominal and the copy figures (Section 3.1 models attention time as memory traffic over
 * memory bandwidth; a decode step reads and writes almost nothing back, so the bandwidth that
 * counts is the read-only one).  Enqueues one kernel that reads `bytes` (a multiple of 16, the
 * buffer 16-byte aligned) of DEVICE memory once with 16-byte loads marked evict-first, sums
 * them and writes one float per thread block to `sink` (DEVICE, >= 4096 floats) so that the
 * loads cannot be dropped.  The caller times it (events) over a buffer larger than L2.
 */
opw_status_t opw_hbm_read_probe(const void *buffer, size_t bytes, float *sink, void *cuda_stream);

/* Frees the host-side handle.  Does not touch device memory.  NULL is accepted. */
opw_status_t opw_attn_stage_destroy(opw_attn_stage_t *stage);

/* Static string for a status code. */
const char *opw_status_string(opw_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* OPW_ATTN_H_ */
