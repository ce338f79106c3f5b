// The complete attention module as one stage (AFD partition): QKV projection with the rotary
// encoding and the split into q / k_new / v_new in its epilogue, core attention
// (opw_decode_step), output projection.  The projections run on the tcgen05 kernel of
// opw_afd_gemm.cuh at every batch size and head dimension; cuBLASLt plus a separate rotary
// kernel is a comparison arm that only OPW_AFD_LIBRARY_GEMM selects.  See include/opw_afd.h.
#include "opw_afd.h"
#include "opw_afd_gemm.cuh"

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

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct opw_afd_module {
  opw_attn_stage_t* stage;
  int32_t layer, hidden, Hq, Hkv, D, max_batch;
  const void* w_qkv;
  const void* w_o;
  double log_theta;
  unsigned char* ws;
  size_t off_qkv, off_q, off_k, off_v, off_out, off_gemm, off_partials, off_tickets, off_angles, off_status;
  // tensor-core path
  bool tc_qkv, tc_o, pdl, coop_ok, no_cluster;
  int max_clusters[2 * opw_afd::kMaxSplit + 1];   // [n]: thread-block clusters of n CTAs of the GEMM kernel the device holds at once
  int sms;
  TensorMapEncodeFn encode;
  CUtensorMap map_wqkv, map_wo;
  int64_t launches;
  unsigned long long* trace;
  // library path: plans are keyed by the batch size; decode loops repeat a handful of sizes, so the
  // last one of each projection is kept and rebuilt when the batch changes.
  cublasLtHandle_t lt;
  int32_t plan_batch;
  GemmPlan plan_qkv, plan_o;
};

namespace {

constexpr int kSmsBound = 160;             // split-K sizing assumes no more SMs than this
// Up to this batch the step's (cos, sin) table is computed inside the QKV kernel, in shared memory behind
// the ring; above it the table (batch * D/2 * 8 bytes) would crowd the ring out, so a small kernel
// writes it to global memory first.
constexpr int kSmemAngleBatch = 96;
constexpr int kCoopMinBatch = 128;         // above this batch the CTAs of a tile share the back end (cooperative launch)
constexpr size_t kGemmSmemBudget = 226 * 1024;

inline int round16(int x) { return (x + 15) / 16 * 16; }
inline int tiles_of(int n_out) { return (n_out + opw_afd::kTileM - 1) / opw_afd::kTileM; }
inline int batch_tiles_of(int batch) { return (batch + opw_afd::kMaxNb - 1) / opw_afd::kMaxNb; }
inline int nb_of(int batch) { return round16(batch < opw_afd::kMaxNb ? batch : opw_afd::kMaxNb); }
inline int ksplit_of(int n_out, int k, int batch, int sms) {
  int ks = sms / (tiles_of(n_out) * batch_tiles_of(batch));
  if (ks > opw_afd::kMaxSplit) ks = opw_afd::kMaxSplit;
  const int kblocks = (k + opw_afd::kBlockK - 1) / opw_afd::kBlockK;
  if (ks > kblocks) ks = kblocks;
  return ks < 1 ? 1 : ks;
}
inline size_t partial_bytes_at(int n_out, int k, int batch) {
  return (size_t)tiles_of(n_out) * batch_tiles_of(batch) * ksplit_of(n_out, k, batch, kSmsBound) * nb_of(batch) *
         opw_afd::kTileM * sizeof(float);
}
// Partial tiles of any batch up to max_batch on any device of at most kSmsBound SMs (more SMs split K further, never
// beyond kMaxSplit).  Up to 256 rows the need grows with the batch; beyond, the batch tiles multiply while the
// K-split falls to one, so the largest need is at 256 rows or at max_batch.
inline size_t partial_bytes(int n_out, int k, int max_batch) {
  const size_t a = partial_bytes_at(n_out, k, max_batch < opw_afd::kMaxNb ? max_batch : opw_afd::kMaxNb);
  const size_t b = partial_bytes_at(n_out, k, max_batch);
  return a > b ? a : b;
}

struct Carve { size_t qkv, q, k, v, out, gemm, partials, tickets, angles, status, total; };

Carve carve(int Hq, int Hkv, int D, int max_batch, int hidden) {
  Carve c;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const int n_qkv = (Hq + 2 * Hkv) * D, n_attn = Hq * D;
  c.qkv = take((size_t)max_batch * n_qkv * 2);
  c.q = take((size_t)max_batch * n_attn * 2);
  c.k = take((size_t)max_batch * Hkv * D * 2);
  c.v = take((size_t)max_batch * Hkv * D * 2);
  c.out = take((size_t)max_batch * n_attn * 2);
  c.gemm = take(kGemmWorkspace);
  // partial tiles: the largest over every batch <= max_batch (nb * batch tiles is monotone in the batch)
  const size_t p1 = partial_bytes(n_qkv, hidden, max_batch), p2 = partial_bytes(hidden, n_attn, max_batch);
  c.partials = take(p1 > p2 ? p1 : p2);
  c.angles = take((size_t)max_batch * (D / 2) * sizeof(float2));
  const int t1 = tiles_of(n_qkv), t2 = tiles_of(hidden);
  c.tickets = take((size_t)(t1 > t2 ? t1 : t2) * batch_tiles_of(max_batch) * 2 * sizeof(uint32_t));
  c.status = take(sizeof(uint32_t));
  c.total = off;
  return c;
}

bool dims_ok(int Hq, int Hkv, int D, int max_batch, int hidden) {
  return Hq >= 1 && Hkv >= 1 && Hq % Hkv == 0 && (D == 64 || D == 128 || D == 256) && max_batch >= 1 && hidden >= 8 &&
         hidden % 8 == 0;
}

// Row-major bf16 [rows, k] seen by TMA as a 2-D tensor, boxes of 64 x box_rows elements, 128-byte swizzle,
// zero fill outside the tensor (so ragged rows and a ragged K tail contribute nothing).
bool encode_map(TensorMapEncodeFn fn, CUtensorMap* map, const void* base, uint64_t rows, uint64_t k, uint32_t box_rows) {
  const cuuint64_t dims[2] = {k, rows};
  const cuuint64_t strides[1] = {k * 2};
  const cuuint32_t box[2] = {(cuuint32_t)opw_afd::kBlockK, box_rows};
  const cuuint32_t elem[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// `coop`: a cooperative launch -- the whole grid is resident at once or the launch is refused.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl, bool coop,
                       int cluster_x, int cluster_y, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[3];
  int n = 0;
  if (cluster_x * cluster_y > 1) {              // thread-block clusters of (cluster_x, cluster_y, 1)
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = (unsigned)cluster_y;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (coop) {
    attr[n].id = cudaLaunchAttributeCooperative;
    attr[n].val.cooperative = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// One projection on the tensor-core kernel.
opw_status_t run_tc_gemm(opw_afd_module* m, const CUtensorMap& map_w, const void* x, int batch, int n_out, int k, int mode,
                         const int32_t* positions, __nv_bfloat16* out, __nv_bfloat16* q, __nv_bfloat16* kn,
                         __nv_bfloat16* vn, cudaStream_t stream) {
  opw_afd::GemmParams p;
  p.n_out = n_out; p.k = k; p.batch = batch; p.nb = nb_of(batch);
  p.group = (mode == 1 && m->D > opw_afd::kTileM) ? 2 : 1;   // a head of 256 spans two weight tiles
  const size_t stage_bytes = opw_afd::kTileABytes + (size_t)p.nb * 128;
  // The step's (cos, sin) table: behind the ring for small batches, from global memory (written by a small
  // kernel launched just before) for large ones and wherever the table would leave the ring too small.
  // The epilogue reuses the ring: one tile of sums for all columns, or two tiles for a chunk of columns.
  p.ksplit = ksplit_of(n_out, k, batch, m->sms < kSmsBound ? m->sms : kSmsBound);
  // The K-split CTAs of a weight tile exchange their partial tiles inside a thread-block cluster when the device
  // can hold every cluster of the launch at once (a cluster needs its SMs in one GPC, so fewer CTAs fit than
  // there are SMs: 45 clusters of three on a B200 with 148 SMs, 33 of four, 74 of two); a narrower split that
  // fits is preferred to a wider one that does not.
  p.cluster = 0;
  if (p.ksplit * p.group > 1 && !m->no_cluster && tiles_of(n_out) % p.group == 0) {
    for (int ks = p.ksplit; ks * p.group >= 2; --ks)
      if (tiles_of(n_out) / p.group * batch_tiles_of(batch) <= m->max_clusters[ks * p.group]) {
        p.ksplit = ks;
        p.cluster = 1;
        break;
      }
  }
  const int ctas = tiles_of(n_out) * p.ksplit * batch_tiles_of(batch);
  // The shared back end pays at large batches, where publishing and reducing the partial tiles is bandwidth work
  // that a third of the CTAs would otherwise do alone (batch 256: 31 -> 27 us for the QKV projection); at small
  // batches the back end is a latency chain either way, and a cooperative launch cannot start under the previous
  // kernel's tail, which costs more than the sharing gives (batch 64: 149 -> 157 us per module step).
  p.coop = (!p.cluster && m->coop_ok && ctas <= m->sms && (p.ksplit > 1 || p.group > 1) && batch > kCoopMinBatch) ? 1 : 0;
  const int chunk_cols = batch < opw_afd::kChunkCols ? batch : opw_afd::kChunkCols;
  const int members = p.ksplit * p.group;
  // cooperative back end: the CTA's own tile, plus (two-tile heads) its slice of the other tile's sums
  const size_t epi_coop = ((size_t)p.nb + (p.group == 2 ? (size_t)((batch < opw_afd::kMaxNb ? batch : opw_afd::kMaxNb) + members - 1) / members + 1 : 0)) *
                          opw_afd::kTileM * sizeof(float);
  const size_t epi_last = p.group == 1 ? (size_t)p.nb * opw_afd::kTileM * sizeof(float)
                                       : ((size_t)opw_afd::kChunkCols + chunk_cols) * opw_afd::kTileM * sizeof(float);
  const size_t epi_bytes = (p.coop || (p.cluster && p.group == 2)) ? epi_coop : epi_last;
  bool angles_global = mode == 1 && batch > kSmemAngleBatch;
  size_t angle_bytes = 0;
  int stages = 0;
  for (;;) {
    angle_bytes = (mode == 1 && !angles_global) ? (size_t)batch * (m->D / 2) * sizeof(float2) + (size_t)(m->D / 2) * sizeof(double) : 0;
    stages = (int)((kGemmSmemBudget - 1024 - angle_bytes) / stage_bytes);
    if (stages > opw_afd::kMaxStages) stages = opw_afd::kMaxStages;
    if ((stages >= 4 && (size_t)stages * stage_bytes >= epi_bytes) || angles_global || mode != 1) break;
    angles_global = true;
  }
  if (stages < 2 || (size_t)stages * stage_bytes < epi_bytes) return OPW_ERR_UNSUPPORTED;
  p.stages = stages;
  p.mode = mode;
  p.out = out; p.q = q; p.kn = kn; p.vn = vn;
  p.positions = positions;
  p.log_theta = m->log_theta;
  p.Hq = m->Hq; p.Hkv = m->Hkv; p.D = m->D;
  p.partials = reinterpret_cast<float*>(m->ws + m->off_partials);
  p.tickets = reinterpret_cast<uint32_t*>(m->ws + m->off_tickets);
  p.status = reinterpret_cast<uint32_t*>(m->ws + m->off_status);
  p.angles_g = angles_global ? reinterpret_cast<const float2*>(m->ws + m->off_angles) : nullptr;
  // trace region 0: output projection, region 1: QKV projection
  p.trace = m->trace ? m->trace + (size_t)mode * opw_afd::kTraceMaxCtas * opw_afd::kTraceWords : nullptr;
  if (angles_global) {
    if (launch_pdl(opw_afd::rope_table_kernel, dim3(batch), dim3(128), 0, stream, m->pdl, false, 1, 1, positions,
                   reinterpret_cast<float2*>(m->ws + m->off_angles), (int)m->D, m->log_theta) != cudaSuccess) {
      (void)cudaGetLastError();
      return OPW_ERR_CUDA;
    }
    ++m->launches;
  }
  CUtensorMap map_x;       // the activation pointer and the batch change from call to call: encoded per launch, on the host
  if (!encode_map(m->encode, &map_x, x, (uint64_t)batch, (uint64_t)k, (uint32_t)p.nb)) return OPW_ERR_CUDA;
  const dim3 grid(tiles_of(n_out), p.ksplit, batch_tiles_of(batch));
  if (launch_pdl(opw_afd::skinny_gemm_kernel, grid, dim3(opw_afd::kGemmThreads), 1024 + (size_t)stages * stage_bytes + angle_bytes,
                 stream, m->pdl, p.coop != 0, p.cluster ? p.group : 1, p.cluster ? p.ksplit : 1, map_w, map_x, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  ++m->launches;
  return OPW_OK;
}

}  // namespace

extern "C" {

size_t opw_afd_module_workspace_bytes(int32_t Hq, int32_t Hkv, int32_t D, int32_t max_batch, int32_t hidden) {
  if (!dims_ok(Hq, Hkv, D, max_batch, hidden)) return 0;
  return carve(Hq, Hkv, D, max_batch, hidden).total;
}

opw_status_t opw_afd_module_create(opw_attn_stage_t* stage, int32_t layer, int32_t hidden, const void* w_qkv,
                                   const void* w_o, float rope_theta, uint32_t flags, void* workspace,
                                   size_t workspace_bytes, opw_afd_module_t** out) {
  if (!stage || !w_qkv || !w_o || !workspace || !out) return OPW_ERR_INVALID_ARG;
  if (hidden < 8 || hidden % 8 != 0 || !(rope_theta > 0.f) || (flags & ~(OPW_AFD_LIBRARY_GEMM | OPW_AFD_NO_PDL | OPW_AFD_NO_CLUSTER))) return OPW_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || (reinterpret_cast<uintptr_t>(w_qkv) & 15) ||
      (reinterpret_cast<uintptr_t>(w_o) & 15))
    return OPW_ERR_INVALID_ARG;
  int32_t device = 0, layers = 0, Hq = 0, Hkv = 0, D = 0, max_batch = 0;
  opw_status_t rc = opw_attn_stage_shape(stage, &device, &layers, &Hq, &Hkv, &D, &max_batch);
  if (rc != OPW_OK) return rc;
  if (layer < 0 || layer >= layers) return OPW_ERR_INVALID_ARG;
  const Carve c = carve(Hq, Hkv, D, max_batch, hidden);
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
  m->off_partials = c.partials; m->off_tickets = c.tickets; m->off_angles = c.angles; m->off_status = c.status;
  m->plan_batch = 0;
  m->launches = 0;
  m->trace = nullptr;
  m->lt = nullptr;
  m->encode = nullptr;
  const bool library = (flags & OPW_AFD_LIBRARY_GEMM) != 0;
  m->tc_qkv = !library;
  m->tc_o = !library;
  m->pdl = (flags & OPW_AFD_NO_PDL) == 0;
  m->no_cluster = (flags & OPW_AFD_NO_CLUSTER) != 0;
  bool ok = true;
  if (m->tc_qkv || m->tc_o) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
         qres == cudaDriverEntryPointSuccess && fn != nullptr;
    m->encode = reinterpret_cast<TensorMapEncodeFn>(fn);
    int sms = 0;
    ok = ok && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) == cudaSuccess && sms > 0;
    m->sms = sms;
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device) != cudaSuccess) { (void)cudaGetLastError(); coop = 0; }
    m->coop_ok = coop != 0;
    ok = ok && cudaFuncSetAttribute(opw_afd::skinny_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kGemmSmemBudget) == cudaSuccess;
    for (int ks = 0; ks <= 2 * opw_afd::kMaxSplit; ++ks) m->max_clusters[ks] = 0;
    for (int ks = 2; ok && ks <= 2 * opw_afd::kMaxSplit; ++ks) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(1, ks, 1);
      cfg.blockDim = dim3(opw_afd::kGemmThreads);
      cfg.dynamicSmemBytes = kGemmSmemBudget;      // the most a launch asks for
      cudaLaunchAttribute at;
      at.id = cudaLaunchAttributeClusterDimension;
      at.val.clusterDim.x = 1; at.val.clusterDim.y = (unsigned)ks; at.val.clusterDim.z = 1;
      cfg.attrs = &at;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, opw_afd::skinny_gemm_kernel, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
      m->max_clusters[ks] = n;
    }
    const int n_qkv = (Hq + 2 * Hkv) * D, n_attn = Hq * D;
    ok = ok && encode_map(m->encode, &m->map_wqkv, w_qkv, (uint64_t)n_qkv, (uint64_t)hidden, opw_afd::kTileM);
    ok = ok && encode_map(m->encode, &m->map_wo, w_o, (uint64_t)hidden, (uint64_t)n_attn, opw_afd::kTileM);
  }
  // tickets and the status word start at zero (synchronously, on the default stream, as the stage does)
  ok = ok && cudaMemset(m->ws + c.tickets, 0, c.total - c.tickets) == cudaSuccess;   // tickets, then the status word
  if (ok && library) ok = cublasLtCreate(&m->lt) == CUBLAS_STATUS_SUCCESS;   // only the comparison arm touches the library
  if (!ok) {
    (void)cudaGetLastError();
    if (m->lt) cublasLtDestroy(m->lt);
    delete m;
    return OPW_ERR_CUDA;
  }
  *out = m;
  return OPW_OK;
}

opw_status_t opw_afd_module_step(opw_afd_module_t* m, int32_t batch, const void* x, const int32_t* positions,
                                 const int32_t* page_table, void* y, void* cuda_stream) {
  if (!m || !x || !positions || !page_table || !y) return OPW_ERR_INVALID_ARG;
  if (batch < 1 || (reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(y) & 15)) return OPW_ERR_INVALID_ARG;
  if (batch > m->max_batch) return OPW_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int n_qkv = (m->Hq + 2 * m->Hkv) * m->D, n_attn = m->Hq * m->D;
  const bool tc_qkv = m->tc_qkv, tc_o = m->tc_o;
  if ((!tc_qkv || !tc_o) && m->plan_batch != batch) {
    m->plan_batch = 0;
    if (!tc_qkv && !make_plan(m->lt, m->plan_qkv, batch, n_qkv, m->hidden)) return OPW_ERR_CUDA;
    if (!tc_o && !make_plan(m->lt, m->plan_o, batch, m->hidden, n_attn)) return OPW_ERR_CUDA;
    m->plan_batch = batch;
  }
  __nv_bfloat16* qkv = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_qkv);
  __nv_bfloat16* q = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_q);
  __nv_bfloat16* k = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_k);
  __nv_bfloat16* v = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_v);
  __nv_bfloat16* attn = reinterpret_cast<__nv_bfloat16*>(m->ws + m->off_out);
  void* gemm_ws = m->ws + m->off_gemm;
  opw_status_t rc;

  if (tc_qkv) {
    rc = run_tc_gemm(m, m->map_wqkv, x, batch, n_qkv, m->hidden, 1, positions, nullptr, q, k, v, stream);
    if (rc != OPW_OK) return rc;
  } else {
    if (!run_plan(m->lt, m->plan_qkv, m->w_qkv, x, qkv, gemm_ws, stream)) return OPW_ERR_CUDA;
    rope_split_kernel<<<batch, 256, (size_t)m->D * sizeof(float), stream>>>(qkv, positions, q, k, v, m->Hq, m->Hkv, m->D,
                                                                           m->log_theta);
    if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
    ++m->launches;
  }
  rc = opw_decode_step(m->stage, m->layer, batch, q, k, v, positions, page_table, attn, nullptr, cuda_stream);
  if (rc != OPW_OK) return rc;
  if (tc_o) {
    rc = run_tc_gemm(m, m->map_wo, attn, batch, m->hidden, n_attn, 0, nullptr, static_cast<__nv_bfloat16*>(y), nullptr,
                     nullptr, nullptr, stream);
    if (rc != OPW_OK) return rc;
  } else if (!run_plan(m->lt, m->plan_o, m->w_o, attn, y, gemm_ws, stream)) {
    return OPW_ERR_CUDA;
  }
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

opw_status_t opw_afd_module_poll_error(opw_afd_module_t* m, void* cuda_stream) {
  if (!m) return OPW_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  uint32_t* d = reinterpret_cast<uint32_t*>(m->ws + m->off_status);
  if (cudaMemcpyAsync(&word, d, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemsetAsync(d, 0, 4, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  if (word & opw_afd::kGemmErrTimeout) {
    // a kernel that gave up may have left its group counters mid-count
    if (cudaMemsetAsync(m->ws + m->off_tickets, 0, m->off_status - m->off_tickets, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
      (void)cudaGetLastError();
      return OPW_ERR_CUDA;
    }
    return OPW_ERR_TIMEOUT;
  }
  return OPW_OK;
}

opw_status_t opw_afd_module_set_trace(opw_afd_module_t* m, void* trace, size_t trace_bytes) {
  if (!m) return OPW_ERR_INVALID_ARG;
  if (!trace) { m->trace = nullptr; return OPW_OK; }
  if (reinterpret_cast<uintptr_t>(trace) & 7) return OPW_ERR_INVALID_ARG;
  if (trace_bytes < (size_t)2 * opw_afd::kTraceMaxCtas * opw_afd::kTraceWords * 8) return OPW_ERR_CAPACITY;
  m->trace = static_cast<unsigned long long*>(trace);
  return OPW_OK;
}

int64_t opw_afd_module_launch_count(const opw_afd_module_t* m) { return m ? m->launches : 0; }

opw_status_t opw_afd_module_destroy(opw_afd_module_t* m) {
  if (!m) return OPW_OK;
  destroy_plan(m->plan_qkv);
  destroy_plan(m->plan_o);
  if (m->lt) cublasLtDestroy(m->lt);
  delete m;
  return OPW_OK;
}

}  // extern "C"
