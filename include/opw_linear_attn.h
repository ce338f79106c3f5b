/*
 * opw_linear_attn.h -- C ABI of the decode step of a recurrent-state ("linear attention") layer.
 *
 * Hybrid-attention models interleave full attention with layers that keep a compact recurrent
 * state instead of a KV cache (paper, Section 3.4: "efficient operators access a bounded
 * window or compact recurrent state"; Table 2 lists one evaluated model with linear layers
 * 3:1).  Core-attention disaggregation places those layers on the attention device group too,
 * so the attention stage needs their decode step as a second memory-bound operator: its
 * latency is the state traffic over the memory bandwidth, independent of the context length
 * (Section 7.2 contrasts 58 us for a linear layer with 700 us for full attention at 128K).
 *
 * The paper does not define the operator.  The reading taken here is the gated delta rule
 * (the published recurrence of gated delta networks), per sequence b and value head h, with
 * key head hk = h / (Hv / Hk):
 *     S1 = a[b,h] * S                       decay of the state S (dk x dv)
 *     u  = v[b,h,:] - S1^T k[b,hk,:]        prediction error of the stored value for key k
 *     S' = S1 + beta[b,h] * k[b,hk,:] u^T   rank-one correction
 *     o[b,h,:] = scale * S'^T q[b,hk,:]     read-out with the updated state
 * q and k arrive normalised and v, a, beta already computed (the projections and gates live in
 * the other stage).  State in fp32, q/k/v/out in bf16, a/beta in fp32.
 *
 * Conventions as in opw_attn.h: plain C, DEVICE pointers are caller-owned device memory, the
 * call only enqueues on the stream, no allocation, no synchronisation, status codes from
 * opw_status_t.
 */
#ifndef OPW_LINEAR_ATTN_H_
#define OPW_LINEAR_ATTN_H_

#include "opw_afd.h"
#include "opw_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * One decode step of a recurrent-state layer for `batch` sequences, in place on their states.
 *   state      : DEVICE float [num_slots, Hv, dk, dv] (dv contiguous), 16-byte aligned
 *   slot       : DEVICE int32 [batch]; state slot of each sequence, < 0 = inactive row (its
 *                state is untouched and its output is 0); two rows must not name the same slot
 *   q, k       : DEVICE bf16 [batch, Hk, dk]
 *   v          : DEVICE bf16 [batch, Hv, dv], 8-byte aligned
 *   a, beta    : DEVICE float [batch, Hv]
 *   out        : DEVICE bf16 [batch, Hv, dv], 8-byte aligned
 *   scale      : read-out scale; 0 -> 1/sqrt(dk)
 * dk in {64, 128}, dv in {64, 128, 256} (a multiple of 32), Hv % Hk == 0; otherwise
 * OPW_ERR_UNSUPPORTED.  A slot id >= num_slots is skipped (output 0); no status word here.
 */
opw_status_t opw_linear_attn_decode_step(int32_t batch, int32_t num_k_heads, int32_t num_v_heads, int32_t dk, int32_t dv,
                                         float *state, int64_t num_slots, const int32_t *slot, const void *q,
                                         const void *k, const void *v, const float *a, const float *beta, float scale,
                                         void *out, void *cuda_stream);

/*
 * Mixed plans: one native submission (Section 6.2) for a hybrid stack that interleaves
 * attention layers with recurrent-state layers, or for a stage that holds whole attention
 * modules.  An op is one attention item (see opw_step_item_t in opw_attn.h), one recurrent-state
 * step with the arguments of opw_linear_attn_decode_step, or one attention-module step
 * (opw_afd_item_t in opw_afd.h); ops run in the order given, one after the other.  Flags as for
 * opw_attn_plan_create, except that OPW_PLAN_OVERLAP is not available (OPW_ERR_UNSUPPORTED);
 * OPW_PLAN_ADVANCE touches the positions / kv_lens of attention items and module steps only.  Submit and destroy
 * with opw_attn_plan_submit / opw_attn_plan_destroy.
 */
typedef struct {
  int32_t batch, num_k_heads, num_v_heads, dk, dv;
  float *state;
  int64_t num_slots;
  const int32_t *slot;
  const void *q, *k, *v;
  const float *a, *beta;
  float scale;
  void *out;
} opw_linear_item_t;

#define OPW_OP_ATTENTION 0
#define OPW_OP_LINEAR 1
#define OPW_OP_AFD_MODULE 2
typedef struct {
  int32_t kind;                /* OPW_OP_ATTENTION, OPW_OP_LINEAR or OPW_OP_AFD_MODULE */
  opw_step_item_t attention;   /* used when kind == OPW_OP_ATTENTION */
  opw_linear_item_t linear;    /* used when kind == OPW_OP_LINEAR */
  opw_afd_item_t afd;          /* used when kind == OPW_OP_AFD_MODULE (see opw_afd.h) */
} opw_plan_op_t;

opw_status_t opw_attn_plan_create_mixed(opw_attn_stage_t *stage, const opw_plan_op_t *ops, int32_t n_ops,
                                        uint32_t flags, opw_attn_plan_t **out);

/* Host helper: bytes of the state of num_slots sequences. */
size_t opw_linear_attn_state_bytes(int32_t num_v_heads, int32_t dk, int32_t dv, int64_t num_slots);

#ifdef __cplusplus
}
#endif
#endif /* OPW_LINEAR_ATTN_H_ */
