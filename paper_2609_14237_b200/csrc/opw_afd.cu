// The complete attention module as one stage (AFD partition): QKV projection (cuBLASLt),
// rotary encoding fused with the split into q / k_new / v_new (own kernel), core attention
// (opw_decode_step), output projection (cuBLASLt).  See include/opw_afd.h.
#include "opw_afd.h"

#include <cmath>
#include <cstdint>
#include <new>

#include <cublasLt.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace {

constexpr size_t kGemmWorkspace = 32u << 20;
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// One block per sequence.  The first D/2 threads compute cos / sin of position * theta^(-2i/D)
// in double (a float angle loses 1e-7 * position radians, visible at long contexts), then every
// thread rotates pairs (i, i + D/2) of the q and k heads and copies v; results leave as bf16.
__global__ void rope_split_kernel(const __nv_bfloat16* __restrict__ qkv, const int32_t* __restrict__ positions,
                                  __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k,
                                  __nv_bfloat16* __restrict__ v, int Hq, int Hkv, int D, double log_theta) {
  extern __shared__ float cs[];                  // cos[D/2], sin[D/2]
  const int b = blockIdx.x, half = D / 2;
  int32_t pos = positions[b];
  if (pos < 0) pos = 0;                          // inactive row: anything finite will do, it is never appended
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const double ang = (double)pos * exp(-2.0 * i / D * log_theta);
    double s, c;
    sincos(ang, &s, &c);
    cs[i] = (float)c;
    cs[half + i] = (float)s;
  }
  __syncthreads();
  const int64_t row = (int64_t)b * (Hq + 2 * Hkv) * D;
  const int rot_pairs = (Hq + Hkv) * half;       // q heads, then k heads
  for (int t = threadIdx.x; t < rot_pairs; t += blockDim.x) {
    const int h = t / half, i = t - h * half;
    const float x0 = __bfloat162float(qkv[row + (int64_t)h * D + i]);
    const float x1 = __bfloat162float(qkv[row + (int64_t)h * D + i + half]);
    const float c = cs[i], s = cs[half + i];
    __nv_bfloat16* dst = h < Hq ? q + ((int64_t)b * Hq + h) * D : k + ((int64_t)b * Hkv + (h - Hq)) * D;
    dst[i] = __float2bfloat16_rn(x0 * c - x1 * s);
    dst[i + half] = __float2bfloat16_rn(x1 * c + x0 * s);
  }
  const int64_t voff = row + (int64_t)(Hq + Hkv) * D;
  for (int t = threadIdx.x; t < Hkv * D; t += blockDim.x) v[(int64_t)b * Hkv * D + t] = qkv[voff + t];
}

// One cached cuBLASLt plan: C[n_rows, n_out] = A[n_rows, k] * W[n_out, k]^T, all row-major bf16,
// fp32 accumulation.  In the library's column-major terms: C^T (n_out x n_rows) = op(W) * A^T with
// transa = T on W (stored k x n_out, ld k) and transb = N on A (stored k x n_rows, ld k).
struct GemmPlan {
  bool ready = false;
  cublasLtMatmulDesc_t op = nullptr;
  cublasLtMatrixLayout_t a = nullptr, b = nullptr, c = nullptr;
  cublasLtMatmulAlgo_t algo;
};

void destroy_plan(GemmPlan& p) {
  if (p.a) cublasLtMatrixLayoutDestroy(p.a);
  if (p.b) cublasLtMatrixLayoutDestroy(p.b);
  if (p.c) cublasLtMatrixLayoutDestroy(p.c);
  if (p.op) cublasLtMatmulDescDestroy(p.op);
  p = GemmPlan();
}

bool make_plan(cublasLtHandle_t lt, GemmPlan& p, int n_rows, int n_out, int k) {
  destroy_plan(p);
  const cublasOperation_t tr = CUBLAS_OP_T, no = CUBLAS_OP_N;
  bool ok = cublasLtMatmulDescCreate(&p.op, CUBLAS_COMPUTE_32F, CUDA_R_32F) == CUBLAS_STATUS_SUCCESS;
  ok = ok && cublasLtMatmulDescSetAttribute(p.op, CUBLASLT_MATMUL_DESC_TRANSA, &tr, sizeof(tr)) == CUBLAS_STATUS_SUCCESS;
  ok = ok && cublasLtMatmulDescSetAttribute(p.op, CUBLASLT_MATMUL_DESC_TRANSB, &no, sizeof(no)) == CUBLAS_STATUS_SUCCESS;
  ok = ok && cublasLtMatrixLayoutCreate(&p.a, CUDA_R_16BF, k, n_out, k) == CUBLAS_STATUS_SUCCESS;
  ok = ok && cublasLtMatrixLayoutCreate(&p.b, CUDA_R_16BF, k, n_rows, k) == CUBLAS_STATUS_SUCCESS;
  ok = ok && cublasLtMatrixLayoutCreate(&p.c, CUDA_R_16BF, n_out, n_rows, n_out) == CUBLAS_STATUS_SUCCESS;
  cublasLtMatmulPreference_t pref = nullptr;
  ok = ok && cublasLtMatmulPreferenceCreate(&pref) == CUBLAS_STATUS_SUCCESS;
  const size_t ws = kGemmWorkspace;
  ok = ok && cublasLtMatmulPreferenceSetAttribute(pref, CUBLASLT_MATMUL_PREF_MAX_WORKSPACE_BYTES, &ws, sizeof(ws)) ==
                 CUBLAS_STATUS_SUCCESS;
  cublasLtMatmulHeuristicResult_t res;
  int found = 0;
  ok = ok && cublasLtMatmulAlgoGetHeuristic(lt, p.op, p.a, p.b, p.c, p.c, pref, 1, &res, &found) == CUBLAS_STATUS_SUCCESS &&
       found > 0;
  if (pref) cublasLtMatmulPreferenceDestroy(pref);
  if (!ok) { destroy_plan(p); return false; }
  p.algo = res.algo;
  p.ready = true;
  return true;
}

bool run_plan(cublasLtHandle_t lt, const GemmPlan& p, const void* w, const void* a, void* c, void* ws, cudaStream_t s) {
  const float one = 1.f, zero = 0.f;
  return cublasLtMatmul(lt, p.op, &one, w, p.a, a, p.b, &zero, c, p.c, c, p.c, &p.algo, ws, kGemmWorkspace, s) ==
         CUBLAS_STATUS_SUCCESS;
}

}  // namespace

struct opw_afd_module {
  opw_attn_stage_t* stage;
  int32_t layer, hidden, Hq, Hkv, D, max_batch;
  const void* w_qkv;
  const void* w_o;
  double log_theta;
  unsigned char* ws;
  size_t off_qkv, off_q, off_k, off_v, off_out, off_gemm;
  cublasLtHandle_t lt;
  // Plans are keyed by the batch size; decode loops repeat a handful of sizes, so the last one
  // of each projection is kept and rebuilt when the batch changes.
  int32_t plan_batch;
  GemmPlan plan_qkv, plan_o;
};

namespace {

struct Carve { size_t qkv, q, k, v, out, gemm, total; };

Carve carve(int Hq, int Hkv, int D, int max_batch) {
  Carve c;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  c.qkv = take((size_t)max_batch * (Hq + 2 * Hkv) * D * 2);
  c.q = take((size_t)max_batch * Hq * D * 2);
  c.k = take((size_t)max_batch * Hkv * D * 2);
  c.v = take((size_t)max_batch * Hkv * D * 2);
  c.out = take((size_t)max_batch * Hq * D * 2);
  c.gemm = take(kGemmWorkspace);
  c.total = off;
  return c;
}

bool dims_ok(int Hq, int Hkv, int D, int max_batch) {
  return Hq >= 1 && Hkv >= 1 && Hq % Hkv == 0 && (D == 64 || D == 128 || D == 256) && max_batch >= 1;
}

}  // namespace

extern "C" {

size_t opw_afd_module_workspace_bytes(int32_t Hq, int32_t Hkv, int32_t D, int32_t max_batch) {
  if (!dims_ok(Hq, Hkv, D, max_batch)) return 0;
  return carve(Hq, Hkv, D, max_batch).total;
}

opw_status_t opw_afd_module_create(opw_attn_stage_t* stage, int32_t layer, int32_t hidden, const void* w_qkv,
                                   const void* w_o, float rope_theta, void* workspace, size_t workspace_bytes,
                                   opw_afd_module_t** out) {
  if (!stage || !w_qkv || !w_o || !workspace || !out) return OPW_ERR_INVALID_ARG;
  if (hidden < 8 || hidden % 8 != 0 || !(rope_theta > 0.f)) return OPW_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || (reinterpret_cast<uintptr_t>(w_qkv) & 15) ||
      (reinterpret_cast<uintptr_t>(w_o) & 15))
    return OPW_ERR_INVALID_ARG;
  int32_t device = 0, layers = 0, Hq = 0, Hkv = 0, D = 0, max_batch = 0;
  opw_status_t rc = opw_attn_stage_shape(stage, &device, &layers, &Hq, &Hkv, &D, &max_batch);
  if (rc != OPW_OK) return rc;
  if (layer < 0 || layer >= layers) return OPW_ERR_INVALID_ARG;
  const Carve c = carve(Hq, Hkv, D, max_batch);
  if (workspace_bytes < c.total) return OPW_ERR_CAPACITY;
  if (cudaSetDevice(device) != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  opw_afd_module* m = new (std::nothrow) opw_afd_module();
  if (!m) return OPW_ERR_CUDA;
  m->stage = stage;
  m->layer = layer; m->hidden = hidden; m->Hq = Hq; m->Hkv = Hkv; m->D = D; m->max_batch = max_batch;
  m->w_qkv = w_qkv; m->w_o = w_o;
  m->log_theta = std::log((double)rope_theta);
  m->ws = static_cast<unsigned char*>(workspace);
  m->off_qkv = c.qkv; m->off_q = c.q; m->off_k = c.k; m->off_v = c.v; m->off_out = c.out; m->off_gemm = c.gemm;
  m->plan_batch = 0;
  if (cublasLtCreate(&m->lt) != CUBLAS_STATUS_SUCCESS) { delete m; return OPW_ERR_CUDA; }
  *out = m;
  return OPW_OK;
}

opw_status_t opw_afd_module_step(opw_afd_module_t* m, int32_t batch, const void* x, const int32_t* positions,
                                 const int32_t* page_table, void* y, void* cuda_stream) {
  if (!m || !x || !positions || !page_table || !y) return OPW_ERR_INVALID_ARG;
  if (batch < 1) return OPW_ERR_INVALID_ARG;
  if (batch > m->max_batch) return OPW_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int n_qkv = (m->Hq + 2 * m->Hkv) * m->D, n_attn = m->Hq * m->D;
  if (m->plan_batch != batch) {
    m->plan_batch = 0;
    if (!make_plan(m->lt, m->plan_qkv, batch, n_qkv, m->hidden)) return OPW_ERR_CUDA;
    if (!make_plan(m->lt, m->plan_o, batch, m->hidden, n_attn)) return OPW_ERR_CUDA;
    m->plan_batch = batch;
  }
  __nv_bfloat16* qkv = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_qkv);
  __nv_bfloat16* q = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_q);
  __nv_bfloat16* k = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_k);
  __nv_bfloat16* v = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_v);
  __nv_bfloat16* attn = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_out);
  void* gemm_ws = m->ws + m->off_gemm;

  if (!run_plan(m->lt, m->plan_qkv, m->w_qkv, x, qkv, gemm_ws, stream)) return OPW_ERR_CUDA;
  rope_split_kernel<<<batch, 256, (size_t)m->D * sizeof(float), stream>>>(qkv, positions, q, k, v, m->Hq, m->Hkv, m->D,
                                                                         m->log_theta);
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
  opw_status_t rc = opw_decode_step(m->stage, m->layer, batch, q, k, v, positions, page_table, attn, nullptr, cuda_stream);
  if (rc != OPW_OK) return rc;
  if (!run_plan(m->lt, m->plan_o, m->w_o, attn, y, gemm_ws, stream)) return OPW_ERR_CUDA;
  return OPW_OK;
}

opw_status_t opw_afd_module_intermediates(opw_afd_module_t* m, void** q, void** k_new, void** v_new, void** attn_out) {
  if (!m) return OPW_ERR_INVALID_ARG;
  if (q) *q = m->ws + m->off_q;
  if (k_new) *k_new = m->ws + m->off_k;
  if (v_new) *v_new = m->ws + m->off_v;
  if (attn_out) *attn_out = m->ws + m->off_out;
  return OPW_OK;
}

opw_status_t opw_afd_module_destroy(opw_afd_module_t* m) {
  if (!m) return OPW_OK;
  destroy_plan(m->plan_qkv);
  destroy_plan(m->plan_o);
  cublasLtDestroy(m->lt);
  delete m;
  return OPW_OK;
}

}  // extern "C"
