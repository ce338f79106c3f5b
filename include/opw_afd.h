/*
 * opw_afd.h -- C ABI of the complete attention module as one stage (the AFD partition).
 *
 * Attention-FFN disaggregation, the fixed two-way baseline the paper compares with, "separates
 * complete attention modules from FFN or MoE operators" (Section 4), whereas CAD isolates only
 * the core attention kernels.  This module is that complete attention module built around the
 * core-attention stage of opw_attn.h, per decode step and layer:
 *     qkv = x W_qkv^T                      (library GEMM, cuBLASLt, bf16 in / fp32 accumulate / bf16 out)
 *     q, k <- rotary position encoding     (hand-written kernel, fused with the split into q / k_new / v_new)
 *     out = core attention                 (opw_decode_step: fused append + split-KV attention + combine)
 *     y = out W_o^T                        (library GEMM)
 * It exists to measure the contrast the paper's analysis rests on (Section 3.1: memory-bound
 * attention against GEMM-dominated projections) on the same device, and to let a caller move
 * the stage boundary from CAD to AFD without touching the KV cache.
 *
 * The paper fixes no rotary convention; the reading taken here is the rotate-half form: for
 * i < D/2 the pair (x_i, x_{i+D/2}) turns by the angle position * theta^(-2i/D).
 *
 * Conventions as in opw_attn.h.  The two projections are plain library GEMMs and the module
 * holds a cuBLASLt handle (the library allocates its own host-side state for it); all device
 * memory, including the GEMM workspace, is the caller's.
 */
#ifndef OPW_AFD_H_
#define OPW_AFD_H_

#include "opw_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct opw_afd_module opw_afd_module_t;

/* Scratch bytes of one module: qkv, q, k_new, v_new and attention-output buffers for
 * max_batch rows plus 32 MiB of GEMM workspace.  0 on invalid arguments. */
size_t opw_afd_module_workspace_bytes(int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t max_batch);

/*
 * Binds one layer's attention module to a stage.
 *   w_qkv : DEVICE bf16 [(Hq + 2*Hkv) * D, hidden] (output-feature major: rows q heads, then k, then v)
 *   w_o   : DEVICE bf16 [hidden, Hq * D]
 *   workspace : DEVICE, 256-byte aligned, >= opw_afd_module_workspace_bytes(...)
 * hidden must be a multiple of 8; rope_theta > 0 (e.g. 10000).  The stage must outlive the module.
 */
opw_status_t opw_afd_module_create(opw_attn_stage_t *stage, int32_t layer, int32_t hidden, const void *w_qkv,
                                   const void *w_o, float rope_theta, void *workspace, size_t workspace_bytes,
                                   opw_afd_module_t **out);

/*
 * One decode step of the module: x [batch, hidden] bf16 in, y [batch, hidden] bf16 out, the
 * layer's KV cache appended at positions[b] (< 0: inactive row, y row = 0).  Enqueues two
 * library GEMMs and three kernels on the stream.
 */
opw_status_t opw_afd_module_step(opw_afd_module_t *module, int32_t batch, const void *x, const int32_t *positions,
                                 const int32_t *page_table, void *y, void *cuda_stream);

/* Device addresses of the step's intermediate q [batch,Hq,D], k_new and v_new [batch,Hkv,D]
 * (valid after a step has finished; for tests and tracing). */
opw_status_t opw_afd_module_intermediates(opw_afd_module_t *module, void **q, void **k_new, void **v_new, void **attn_out);

opw_status_t opw_afd_module_destroy(opw_afd_module_t *module); /* NULL is accepted */

#ifdef __cplusplus
}
#endif
#endif /* OPW_AFD_H_ */
