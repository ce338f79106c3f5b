/*
 * opw_afd.h -- C ABI of the complete attention module as one stage (the AFD partition).
 *
 * Attention-FFN disaggregation, the fixed two-way baseline the paper compares with, "separates
 * complete attention modules from FFN or MoE operators" (Section 4), whereas CAD isolates only
 * the core attention kernels.  This module is that complete attention module built around the
 * core-attention stage of opw_attn.h, per decode step and layer:
 *     qkv = x W_qkv^T                      (bf16 in / fp32 accumulate / bf16 out)
 *     q, k <- rotary position encoding     (in the projection's epilogue, with the split into q / k_new / v_new)
 *     out = core attention                 (opw_decode_step: fused append + split-KV attention + combine)
 *     y = out W_o^T
 * The two projections run on a hand-written tcgen05 kernel made for decode shapes: the weight
 * rows fill the tensor core's M dimension and TMEM lanes, the few batch rows its N dimension,
 * TMA streams the weights once, K is split over CTAs so that every SM pulls weights (the K-splits of
 * a weight tile run as one thread-block cluster and add up their tiles through each other's shared
 * memory where the device can hold all clusters at once); batches of more than 256 rows are walked in
 * tiles of 256.  Only with OPW_AFD_LIBRARY_GEMM, kept as a
 * comparison arm, are they cuBLASLt calls followed by a separate rotary kernel instead.
 * It exists to measure the contrast the paper's analysis rests on (Section 3.1: memory-bound
 * attention against GEMM-dominated projections) on the same device, and to let a caller move
 * the stage boundary from CAD to AFD without touching the KV cache.
 *
 * The paper fixes no rotary convention; the reading taken here is the rotate-half form: for
 * i < D/2 the pair (x_i, x_{i+D/2}) turns by the angle position * theta^(-2i/D).
 *
 * Conventions as in opw_attn.h.  With OPW_AFD_LIBRARY_GEMM the module holds a cuBLASLt handle (the
 * library allocates its own host-side state for it); all device memory, including the GEMM
 * workspace, is the caller's.  The tensor-core kernels wait with a bound (0.2 s) on their
 * shared-memory barriers; a wait that runs out is recorded in a status word that
 * opw_afd_module_poll_error returns as OPW_ERR_TIMEOUT (the output of that step is undefined).
 */
#ifndef OPW_AFD_H_
#define OPW_AFD_H_

#include "opw_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct opw_afd_module opw_afd_module_t;

#define OPW_AFD_LIBRARY_GEMM 1u /* projections by cuBLASLt + separate rotary kernel */
#define OPW_AFD_NO_PDL 2u       /* launch the tensor-core projections without programmatic dependent launch (by
                                   default their set-up and first weight tiles overlap the tail of the previous
                                   kernel in the stream, as the stage's own kernels do) */
#define OPW_AFD_NO_CLUSTER 4u   /* never run the K-splits of a weight tile as a thread-block cluster: their partial tiles
                                   always meet in the workspace (the path taken anyway where the clusters of a launch do
                                   not all fit the device, and for heads that span two weight tiles) */

/* Scratch bytes of one module: qkv, q, k_new, v_new and attention-output buffers for
 * max_batch rows, split-K partial tiles, the table of rotation angles, 32 MiB of workspace for
 * the library arm.  0 on invalid
 * arguments. */
size_t opw_afd_module_workspace_bytes(int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t max_batch,
                                      int32_t hidden);

/*
 * Binds one layer's attention module to a stage.
 *   w_qkv : DEVICE bf16 [(Hq + 2*Hkv) * D, hidden] (output-feature major: rows q heads, then k, then v)
 *   w_o   : DEVICE bf16 [hidden, Hq * D]
 *   workspace : DEVICE, 256-byte aligned, >= opw_afd_module_workspace_bytes(...)
 * hidden must be a multiple of 8, the weights 16-byte aligned; rope_theta > 0 (e.g. 10000);
 * flags: OPW_AFD_* or 0.  Clears the module's counters in the workspace
 * (synchronously).  The stage and the weights must outlive the module.
 */
opw_status_t opw_afd_module_create(opw_attn_stage_t *stage, int32_t layer, int32_t hidden, const void *w_qkv,
                                   const void *w_o, float rope_theta, uint32_t flags, void *workspace,
                                   size_t workspace_bytes, opw_afd_module_t **out);

/*
 * One decode step of the module: x [batch, hidden] bf16 in, y [batch, hidden] bf16 out, the
 * layer's KV cache appended at positions[b] (< 0: inactive row, y row = 0).  x and y 16-byte
 * aligned.  Enqueues four kernels on the stream (QKV projection with the rotary epilogue,
 * attention, combine, output projection), five for batches above 96 rows, whose table of rotation
 * angles is written by a small kernel first instead of inside the QKV projection.
 */
opw_status_t opw_afd_module_step(opw_afd_module_t *module, int32_t batch, const void *x, const int32_t *positions,
                                 const int32_t *page_table, void *y, void *cuda_stream);

/* Device addresses of the step's intermediate q [batch,Hq,D], k_new and v_new [batch,Hkv,D]
 * (valid after a step has finished; for tests and tracing). */
opw_status_t opw_afd_module_intermediates(opw_afd_module_t *module, void **q, void **k_new, void **v_new, void **attn_out);

/* Synchronises the stream, returns and clears the module's status word: OPW_OK or OPW_ERR_TIMEOUT.
 * (The stage's own word is read with opw_attn_stage_poll_error.) */
opw_status_t opw_afd_module_poll_error(opw_afd_module_t *module, void *cuda_stream);

/*
 * Tracing of the tensor-core projections (off by default; NULL switches it off again).  trace:
 * DEVICE, 8-byte aligned, >= 2 * 1024 * 8 * 8 bytes = 131072: two regions of 1024 records of
 * 8 uint64 (region 0 the output projection, region 1 the QKV projection; record = CTA index
 * blockIdx.y * gridDim.x + blockIdx.x).  A record holds global-timer nanoseconds at: begin, ring
 * and TMEM ready, accumulator complete, accumulator copied to shared memory, partial tile
 * published, partial tiles reduced, end; word 7 is the SM id.
 */
opw_status_t opw_afd_module_set_trace(opw_afd_module_t *module, void *trace, size_t trace_bytes);

/* Kernels of this module launched so far (the stage counts its own). */
int64_t opw_afd_module_launch_count(const opw_afd_module_t *module);

opw_status_t opw_afd_module_destroy(opw_afd_module_t *module); /* NULL is accepted */

/*
 * One module step as an op of a mixed plan (opw_attn_plan_create_mixed in opw_linear_attn.h, kind
 * OPW_OP_AFD_MODULE): the single native submission of Section 6.2 for a stage that holds complete
 * attention modules.  Arguments as for opw_afd_module_step; `positions` is advanced by one per
 * submission under OPW_PLAN_ADVANCE.  The module must belong to the plan's stage and outlive the plan.
 */
typedef struct {
  opw_afd_module_t *module;
  int32_t batch;
  const void *x;             /* DEVICE bf16 [batch, hidden] */
  int32_t *positions;        /* DEVICE int32 [batch] */
  const int32_t *page_table; /* DEVICE int32 [batch, max_pages_per_seq] */
  void *y;                   /* DEVICE bf16 [batch, hidden] */
} opw_afd_item_t;

#ifdef __cplusplus
}
#endif
#endif /* OPW_AFD_H_ */
