// Host side of the C ABI declared in include/opw_attn.h: argument checks, workspace
// carving, launches.  The library allocates no device memory and never synchronises
// except in opw_attn_stage_poll_error and (once) in opw_attn_stage_create.
#include "opw_attn.h"
#include "opw_afd.h"
#include "opw_linear_attn.h"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "opw_kernels.cuh"

namespace {

constexpr int kDefaultSMs = 148;
constexpr int kDefaultWarps = 8;
constexpr int kDefaultStages = 2;
constexpr int kDefaultCtasPerSm = 1;
constexpr size_t kSmemLimit = 227 * 1024;
constexpr size_t kDeltaPerRow = 4;               // page-table delta entries one call may carry, per static batch slot
constexpr int kCombineScratchSlots = 1024;       // rows * splits of the split combine never exceed this

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Shape {
  int warps, stages, ctas_per_sm;
};

struct Layout {          // byte offsets into the caller's workspace
  size_t status, cum[2], partials[2], split_list[2], comb_scratch, row_count, st_q, st_k, st_v, st_pos, st_out, st_lse, st_delta, st_table, total;
};

bool shape_ok(const opw_attn_stage_config_t* c) {
  return c->num_layers >= 1 && c->num_q_heads >= 1 && c->num_kv_heads >= 1 && c->max_batch >= 1 &&
         c->max_pages_per_seq >= 1 && c->num_q_heads % c->num_kv_heads == 0;
}

opw_status_t resolve_shape(const opw_attn_stage_config_t* c, Shape* s) {
  // head_dim 256 doubles the tile: six warps x two stages x 16 KB fill an SM's shared memory
  // and at head_dim 64 a unit is only 4 KB, its fixed cost (wait, loads of the matrix fragments, softmax)
  // weighs more, and the smaller register footprint leaves room for twelve warps to hide it
  s->warps = c->tune_warps ? c->tune_warps : (c->head_dim > 128 ? 6 : c->head_dim == 64 ? 12 : kDefaultWarps);
  s->stages = c->tune_stages ? c->tune_stages : kDefaultStages;
  s->ctas_per_sm = c->tune_ctas_per_sm ? c->tune_ctas_per_sm : kDefaultCtasPerSm;
  if (s->warps < 1 || s->warps > opw::kMaxWarps || s->stages < 2 || s->stages > 16 || s->ctas_per_sm < 1 ||
      s->ctas_per_sm > 4)
    return OPW_ERR_INVALID_ARG;
  return OPW_OK;
}

size_t attn_smem_bytes(int D, const Shape& s, int batch) {
  return D == 64    ? opw::AttnSmem<64>::bytes(s.warps, s.stages, batch)
         : D == 128 ? opw::AttnSmem<128>::bytes(s.warps, s.stages, batch)
                    : opw::AttnSmem<256>::bytes(s.warps, s.stages, batch);
}

Layout carve(const opw_attn_stage_config_t* c, const Shape& s, int sms) {
  Layout L;
  const size_t B = c->max_batch, Hq = c->num_q_heads, Hkv = c->num_kv_heads, D = c->head_dim;
  const size_t G = Hq / Hkv;
  const size_t workers = (size_t)sms * s.ctas_per_sm * s.warps;
  size_t off = 0;
  L.status = off;  off += 256;
  for (int i = 0; i < 2; ++i) {        // two sets: a plan may run a step's combine beside the next attention
    L.cum[i] = off;      off += align_up((B + 2) * 4, 256);
    L.partials[i] = off; off += align_up(workers * 2 * opw::kSegPerShare * G * (D + 2) * 4, 256);
    L.split_list[i] = off; off += align_up(B * Hkv * 4, 256);   // rows left as partials, in launches with very many rows
  }
  L.comb_scratch = off; off += align_up((size_t)kCombineScratchSlots * G * (D + 2) * 4, 256);
  L.row_count = off; off += align_up(B * Hkv * 4, 256);
  L.st_q = off;    off += align_up(B * Hq * D * 2, 256);
  L.st_k = off;    off += align_up(B * Hkv * D * 2, 256);
  L.st_v = off;    off += align_up(B * Hkv * D * 2, 256);
  L.st_pos = off;  off += align_up(B * 4, 256);
  L.st_out = off;  off += align_up(B * Hq * D * 2, 256);
  L.st_lse = off;  off += align_up(B * Hq * 4, 256);
  L.st_delta = off; off += align_up(kDeltaPerRow * B * 12, 256);
  L.st_table = off; off += align_up((size_t)c->num_layers * B * c->max_pages_per_seq * 4, 256);
  L.total = off;
  return L;
}

// Launch with (or without) the programmatic-stream-serialization attribute: the kernel may
// start while the previous kernel in the stream is still running and synchronises with it
// on the device (griddepcontrol.wait).
template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                   Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int query_sms(int device) {
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) {
    (void)cudaGetLastError();
    return kDefaultSMs;
  }
  return sms;
}

// The dynamic shared-memory limit is an attribute of a kernel on a device, not of a stage, and
// several stages of different sizes may be alive on one device: it is only ever raised.  The
// largest value set so far is kept per device and head size (both instances of a head size get
// the same value).
constexpr int kMaxDevices = 64;
std::mutex g_smem_mutex;
int g_smem_set[kMaxDevices][3];

cudaError_t raise_smem_limit(int device, int D, int bytes) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  const int slot = D == 64 ? 0 : D == 128 ? 1 : 2;
  std::lock_guard<std::mutex> lock(g_smem_mutex);
  if (bytes <= g_smem_set[device][slot]) return cudaSuccess;
  cudaError_t e;
  if (D == 64) {
    e = cudaFuncSetAttribute(opw::attn_splitkv_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(opw::attn_splitkv_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  } else if (D == 128) {
    e = cudaFuncSetAttribute(opw::attn_splitkv_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(opw::attn_splitkv_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  } else {
    e = cudaFuncSetAttribute(opw::attn_splitkv_kernel<256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  }
  if (e == cudaSuccess) g_smem_set[device][slot] = bytes;
  return e;
}

}  // namespace

struct opw_attn_stage {
  opw_attn_stage_config_t cfg;
  std::vector<int32_t> window;
  std::vector<int64_t> num_pages;
  std::vector<void*> pool;
  Shape shape;
  Layout lay;
  int sms;
  int grid;
  size_t smem;
  float scale_log2e;
  int64_t launches;
  unsigned char* ws;
  uint64_t* trace;
  // OPW_FLAG_COPY_STREAMS: the host-buffer step's copies run on streams of their own
  cudaStream_t s_in, s_out;
  cudaEvent_t e_in, e_k, e_out;
};

extern "C" {

const char* opw_status_string(opw_status_t s) {
  switch (s) {
    case OPW_OK: return "ok";
    case OPW_ERR_INVALID_ARG: return "invalid argument";
    case OPW_ERR_UNSUPPORTED: return "unsupported configuration";
    case OPW_ERR_CAPACITY: return "capacity exceeded";
    case OPW_ERR_CUDA: return "CUDA error";
    case OPW_ERR_BAD_PAGE: return "page id or position out of range (device)";
    case OPW_ERR_TIMEOUT: return "bounded device wait ran out";
  }
  return "unknown status";
}

int64_t opw_kv_pool_index(int64_t Hkv, int64_t P, int64_t D, int64_t page, int64_t g, int64_t kv, int64_t t,
                          int64_t d) {
  const int64_t tile = (page * Hkv + g) * 2 + kv;
  return (tile * P + t) * D + ((((d >> 3) ^ (t & 7)) << 3) | (d & 7));
}

size_t opw_kv_pool_bytes(int32_t Hkv, int32_t P, int32_t D, int64_t num_pages) {
  if (Hkv < 1 || P < 1 || D < 1 || num_pages < 0) return 0;
  return (size_t)num_pages * Hkv * 2 * P * D * 2;
}

size_t opw_attn_stage_workspace_bytes(const opw_attn_stage_config_t* cfg) {
  if (!cfg || cfg->struct_size != sizeof(opw_attn_stage_config_t) || !shape_ok(cfg)) return 0;
  Shape s;
  if (resolve_shape(cfg, &s) != OPW_OK) return 0;
  return carve(cfg, s, query_sms(cfg->device)).total;
}

opw_status_t opw_attn_stage_create(const opw_attn_stage_config_t* cfg, opw_attn_stage_t** out) {
  if (!cfg || !out) return OPW_ERR_INVALID_ARG;
  if (cfg->struct_size != sizeof(opw_attn_stage_config_t) || cfg->reserved != 0) return OPW_ERR_INVALID_ARG;
  if (cfg->flags & ~(uint32_t)(OPW_FLAG_NO_PDL | OPW_FLAG_COPY_STREAMS)) return OPW_ERR_INVALID_ARG;
  if (!shape_ok(cfg) || cfg->device < 0) return OPW_ERR_INVALID_ARG;
  if (!cfg->layer_window || !cfg->layer_num_pages || !cfg->layer_kv_pool || !cfg->workspace) return OPW_ERR_INVALID_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128 && cfg->head_dim != 256) return OPW_ERR_UNSUPPORTED;
  if (cfg->page_size != opw::kPage) return OPW_ERR_UNSUPPORTED;
  const int G = cfg->num_q_heads / cfg->num_kv_heads;
  if (G > 16 || (cfg->head_dim == 256 && G > 8)) return OPW_ERR_UNSUPPORTED;
  if (cfg->max_batch > 32768) return OPW_ERR_UNSUPPORTED;
  if ((int64_t)cfg->max_pages_per_seq * opw::kPage > INT32_MAX) return OPW_ERR_UNSUPPORTED;
  if (!(cfg->softmax_scale >= 0.f) || !std::isfinite(cfg->softmax_scale)) return OPW_ERR_INVALID_ARG;
  Shape s;
  if (resolve_shape(cfg, &s) != OPW_OK) return OPW_ERR_INVALID_ARG;
  if ((uintptr_t)cfg->workspace % 256) return OPW_ERR_INVALID_ARG;
  for (int l = 0; l < cfg->num_layers; ++l) {
    if (cfg->layer_window[l] < 0 || cfg->layer_num_pages[l] < 1) return OPW_ERR_INVALID_ARG;
    if (!cfg->layer_kv_pool[l] || (uintptr_t)cfg->layer_kv_pool[l] % 128) return OPW_ERR_INVALID_ARG;
    if (cfg->layer_num_pages[l] * (int64_t)cfg->num_kv_heads > INT32_MAX) return OPW_ERR_UNSUPPORTED;
  }
  const size_t smem = attn_smem_bytes(cfg->head_dim, s, cfg->max_batch);
  if ((smem + 1024) * s.ctas_per_sm > kSmemLimit + 1024) return OPW_ERR_CAPACITY;   // ring does not fit an SM

  // ---- CUDA from here on ----
  if (cudaSetDevice(cfg->device) != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || sms <= 0) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  const Layout lay = carve(cfg, s, sms);
  if (cfg->workspace_bytes < lay.total) return OPW_ERR_CAPACITY;

  cudaError_t e = raise_smem_limit(cfg->device, cfg->head_dim, (int)smem);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  {
    // Registers decide how many warps a block may have (eight at head_dim 128, twelve at 64): ask the
    // runtime now, so that a tuning that cannot launch is refused here and not at the first step.
    const int G = cfg->num_q_heads / cfg->num_kv_heads;
    int resident = 0;
    const int threads = s.warps * 32;
    if (cfg->head_dim == 64)
      e = G > 8 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, opw::attn_splitkv_kernel<64, true>, threads, smem)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, opw::attn_splitkv_kernel<64, false>, threads, smem);
    else if (cfg->head_dim == 128)
      e = G > 8 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, opw::attn_splitkv_kernel<128, true>, threads, smem)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, opw::attn_splitkv_kernel<128, false>, threads, smem);
    else
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, opw::attn_splitkv_kernel<256, false>, threads, smem);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
    if (resident < s.ctas_per_sm) return OPW_ERR_CAPACITY;
  }
  if (cudaMemset(cfg->workspace, 0, 256) != cudaSuccess ||
      cudaMemset(static_cast<unsigned char*>(cfg->workspace) + lay.row_count, 0,
                 (size_t)cfg->max_batch * cfg->num_kv_heads * 4) != cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  if (cudaDeviceSynchronize() != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }

  opw_attn_stage* st = new (std::nothrow) opw_attn_stage();
  if (!st) return OPW_ERR_INVALID_ARG;
  st->cfg = *cfg;
  st->window.assign(cfg->layer_window, cfg->layer_window + cfg->num_layers);
  st->num_pages.assign(cfg->layer_num_pages, cfg->layer_num_pages + cfg->num_layers);
  st->pool.assign(cfg->layer_kv_pool, cfg->layer_kv_pool + cfg->num_layers);
  st->cfg.layer_window = nullptr;
  st->cfg.layer_num_pages = nullptr;
  st->cfg.layer_kv_pool = nullptr;
  st->shape = s;
  st->lay = lay;
  st->sms = sms;
  st->grid = sms * s.ctas_per_sm;
  st->smem = smem;
  const double scale = cfg->softmax_scale > 0.f ? (double)cfg->softmax_scale : 1.0 / std::sqrt((double)cfg->head_dim);
  st->scale_log2e = (float)(scale * 1.4426950408889634);
  st->launches = 0;
  st->trace = nullptr;
  st->ws = static_cast<unsigned char*>(cfg->workspace);
  st->s_in = st->s_out = nullptr;
  st->e_in = st->e_k = st->e_out = nullptr;
  if (cfg->flags & OPW_FLAG_COPY_STREAMS) {
    bool ok = cudaStreamCreateWithFlags(&st->s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&st->s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&st->e_in, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&st->e_k, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&st->e_out, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      (void)cudaGetLastError();
      opw_attn_stage_destroy(st);
      return OPW_ERR_CUDA;
    }
  }
  *out = st;
  return OPW_OK;
}

opw_status_t opw_attn_stage_destroy(opw_attn_stage_t* st) {
  if (!st) return OPW_OK;
  if (st->e_in) cudaEventDestroy(st->e_in);
  if (st->e_k) cudaEventDestroy(st->e_k);
  if (st->e_out) cudaEventDestroy(st->e_out);
  if (st->s_in) cudaStreamDestroy(st->s_in);
  if (st->s_out) cudaStreamDestroy(st->s_out);
  delete st;
  return OPW_OK;
}

opw_status_t opw_attn_stage_wait_host_output(opw_attn_stage_t* st) {
  if (!st) return OPW_ERR_INVALID_ARG;
  if (!st->e_out) return OPW_OK;                 // without copy streams the caller synchronises its own stream
  if (cudaEventSynchronize(st->e_out) != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  return OPW_OK;
}

opw_status_t opw_attn_stage_set_trace(opw_attn_stage_t* st, void* trace, size_t trace_bytes, int32_t* num_workers) {
  if (!st) return OPW_ERR_INVALID_ARG;
  const size_t workers = (size_t)st->grid * st->shape.warps;
  if (num_workers) *num_workers = (int32_t)workers;
  if (!trace) { st->trace = nullptr; return OPW_OK; }
  if ((uintptr_t)trace % 8) return OPW_ERR_INVALID_ARG;
  if (trace_bytes < workers * 32) return OPW_ERR_CAPACITY;
  st->trace = static_cast<uint64_t*>(trace);
  return OPW_OK;
}

int64_t opw_attn_stage_launch_count(const opw_attn_stage_t* st) { return st ? st->launches : 0; }

static opw_status_t check_step(opw_attn_stage_t* st, int32_t layer, int32_t batch) {
  if (!st) return OPW_ERR_INVALID_ARG;
  if (layer < 0 || layer >= st->cfg.num_layers || batch < 0) return OPW_ERR_INVALID_ARG;
  if (batch > st->cfg.max_batch) return OPW_ERR_CAPACITY;
  return OPW_OK;
}

opw_status_t opw_kv_append(opw_attn_stage_t* st, int32_t layer, int32_t batch, const void* k_new, const void* v_new,
                           const int32_t* positions, const int32_t* page_table, void* cuda_stream) {
  opw_status_t rc = check_step(st, layer, batch);
  if (rc != OPW_OK) return rc;
  if (!k_new || !v_new || !positions || !page_table) return OPW_ERR_INVALID_ARG;
  if (((uintptr_t)k_new | (uintptr_t)v_new) % 16 || (uintptr_t)positions % 4 || (uintptr_t)page_table % 4)
    return OPW_ERR_INVALID_ARG;
  if (batch == 0) return OPW_OK;
  opw::AppendParams p;
  p.pool = static_cast<__nv_bfloat16*>(st->pool[layer]);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.positions = positions;
  p.page_table = page_table;
  p.status = reinterpret_cast<uint32_t*>(st->ws + st->lay.status);
  p.num_pages = st->num_pages[layer];
  p.batch = batch;
  p.Hkv = st->cfg.num_kv_heads;
  p.D = st->cfg.head_dim;
  p.max_pages = st->cfg.max_pages_per_seq;
  const int groups = p.Hkv * 2 * (p.D / 8);
  const int threads = groups < 256 ? ((groups + 31) / 32 * 32) : 256;
  const bool pdl = (st->cfg.flags & OPW_FLAG_NO_PDL) == 0;
  if (launch(opw::kv_append_kernel, dim3(batch), dim3(threads), 0, static_cast<cudaStream_t>(cuda_stream), pdl, p) !=
      cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  st->launches += 1;
  return OPW_OK;
}

struct StepArgs {
  int32_t layer, batch;
  const void* q;
  const int32_t* kv_lens;      // or null with the fused append
  const void* k_new;           // fused append: all three set, else all null
  const void* v_new;
  const int32_t* positions;
  const int32_t* page_table;
  void* out;
  float* lse;
};

static opw_status_t validate_step(opw_attn_stage_t* st, const StepArgs& a) {
  opw_status_t rc = check_step(st, a.layer, a.batch);
  if (rc != OPW_OK) return rc;
  const bool fused = a.k_new != nullptr;
  if (!a.q || !a.page_table || !a.out) return OPW_ERR_INVALID_ARG;
  if (fused ? (!a.v_new || !a.positions || a.kv_lens) : (!a.kv_lens || a.v_new || a.positions)) return OPW_ERR_INVALID_ARG;
  if (((uintptr_t)a.q | (uintptr_t)a.out | (uintptr_t)a.k_new | (uintptr_t)a.v_new) % 16 || (uintptr_t)a.kv_lens % 4 ||
      (uintptr_t)a.positions % 4 || (uintptr_t)a.page_table % 4 || (uintptr_t)a.lse % 4)
    return OPW_ERR_INVALID_ARG;
  return OPW_OK;
}

// Launches with this many (sequence, kv head) rows or more have the attention kernel list the rows it leaves
// as partials and the combine walk that list instead of running a block per row (see combine_kernel).  Measured
// on both sides of the threshold: 2048 rows of about 200 pages each (most rows split) 517 us per step with a
// block per row, 532 us with the list; 8192 rows of about 10 pages 161 against 149 us.
constexpr int kRowListMin = 4096;
static inline bool use_row_list(const opw_attn_stage_t* st, int batch) { return batch * st->cfg.num_kv_heads >= kRowListMin; }

// The split-KV kernel of one step, using workspace set `ws_set` (0 or 1).
static opw_status_t launch_attention(opw_attn_stage_t* st, const StepArgs& a, int ws_set, cudaStream_t stream) {
  const int D = st->cfg.head_dim, Hq = st->cfg.num_q_heads, Hkv = st->cfg.num_kv_heads, G = Hq / Hkv;
  opw::AttnParams p;
  p.pool = static_cast<const __nv_bfloat16*>(st->pool[a.layer]);
  p.q = static_cast<const __nv_bfloat16*>(a.q);
  p.kv_lens = a.kv_lens;
  p.page_table = a.page_table;
  p.k_new = static_cast<const __nv_bfloat16*>(a.k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(a.v_new);
  p.positions = a.positions;
  p.pool_w = static_cast<__nv_bfloat16*>(st->pool[a.layer]);
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.lse = a.lse;
  p.partials = reinterpret_cast<float*>(st->ws + st->lay.partials[ws_set]);
  p.cum = reinterpret_cast<int32_t*>(st->ws + st->lay.cum[ws_set]);
  p.status = reinterpret_cast<uint32_t*>(st->ws + st->lay.status);
  p.ticket = reinterpret_cast<int32_t*>(st->ws + st->lay.status + 16 + 16 * ws_set);
  p.split_list = use_row_list(st, a.batch) ? reinterpret_cast<int32_t*>(st->ws + st->lay.split_list[ws_set]) : nullptr;
  p.split_count = reinterpret_cast<int32_t*>(st->ws + st->lay.status + 64 + 32 * ws_set);
  p.trace = st->trace;
  p.num_pages = st->num_pages[a.layer];
  p.batch = a.batch;
  p.Hq = Hq;
  p.Hkv = Hkv;
  p.G = G;
  p.max_pages = st->cfg.max_pages_per_seq;
  p.window = st->window[a.layer];
  p.stages = st->shape.stages;
  p.scale_log2e = st->scale_log2e;

  const dim3 grid(st->grid), block(st->shape.warps * 32);
  const size_t smem = attn_smem_bytes(D, st->shape, a.batch);
  const bool pdl = (st->cfg.flags & OPW_FLAG_NO_PDL) == 0;
  cudaError_t e;
  if (D == 64) {
    if (G > 8) e = launch(opw::attn_splitkv_kernel<64, true>, grid, block, smem, stream, pdl, p);
    else e = launch(opw::attn_splitkv_kernel<64, false>, grid, block, smem, stream, pdl, p);
  } else if (D == 128) {
    if (G > 8) e = launch(opw::attn_splitkv_kernel<128, true>, grid, block, smem, stream, pdl, p);
    else e = launch(opw::attn_splitkv_kernel<128, false>, grid, block, smem, stream, pdl, p);
  } else {
    e = launch(opw::attn_splitkv_kernel<256, false>, grid, block, smem, stream, pdl, p);   // G <= 8 (checked at create)
  }
  if (e != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  st->launches += 1;
  return OPW_OK;
}

// The log-sum-exp combine of the same step.  `small` picks the 128-thread instance, which
// fits on an SM beside a split-KV block.
static opw_status_t launch_combine(opw_attn_stage_t* st, const StepArgs& a, int ws_set, cudaStream_t stream, bool small,
                                   bool side_stream = false) {
  const int D = st->cfg.head_dim, Hq = st->cfg.num_q_heads, Hkv = st->cfg.num_kv_heads, G = Hq / Hkv;
  opw::CombineParams c;
  c.ticket = reinterpret_cast<int32_t*>(st->ws + st->lay.status + 16 + 16 * ws_set);
  c.partials = reinterpret_cast<const float*>(st->ws + st->lay.partials[ws_set]);
  c.cum = reinterpret_cast<const int32_t*>(st->ws + st->lay.cum[ws_set]);
  c.kv_lens = a.kv_lens;
  c.positions = a.positions;
  c.out = static_cast<__nv_bfloat16*>(a.out);
  c.lse = a.lse;
  c.batch = a.batch;
  c.Hq = Hq;
  c.Hkv = Hkv;
  c.G = G;
  c.D = D;
  c.max_pages = st->cfg.max_pages_per_seq;
  c.window = st->window[a.layer];
  c.num_workers = st->grid * st->shape.warps;
  c.scratch = reinterpret_cast<float*>(st->ws + st->lay.comb_scratch);
  c.row_count = reinterpret_cast<int32_t*>(st->ws + st->lay.row_count);
  const bool listed = use_row_list(st, a.batch);
  c.split_list = listed ? reinterpret_cast<const int32_t*>(st->ws + st->lay.split_list[ws_set]) : nullptr;
  c.split_count = reinterpret_cast<int32_t*>(st->ws + st->lay.status + 64 + 32 * ws_set);
  // Few rows can have very many partials each (long contexts at small batch): split each row's
  // merge over several blocks so that about one block per SM is busy (two per SM measured slower:
  // the hand-off between a row's blocks costs more than the extra parallelism gives).
  const int rows = a.batch * Hkv;
  int splits = st->sms / rows;
  if (splits > opw::kCombineBatch) splits = opw::kCombineBatch;
  if (splits > kCombineScratchSlots / rows) splits = kCombineScratchSlots / rows;
  if (splits < 1) splits = 1;
  const bool pdl = (st->cfg.flags & OPW_FLAG_NO_PDL) == 0 && !side_stream;
  const int list_blocks = st->sms * (small ? 4 : 2);
  const dim3 grid(listed ? (rows < list_blocks ? rows : list_blocks) : rows, listed ? 1 : splits);
  cudaError_t e;
#define OPW_LAUNCH_COMBINE(DIM)                                                                                            \
  e = small ? launch(opw::combine_kernel<opw::kCombineThreadsSmall, DIM>, grid, dim3(opw::kCombineThreadsSmall), 0, stream, \
                     pdl, c)                                                                                               \
            : launch(opw::combine_kernel<opw::kCombineThreads, DIM>, grid, dim3(opw::kCombineThreads), 0, stream, pdl, c)
  if (D == 64) OPW_LAUNCH_COMBINE(64);
  else if (D == 128) OPW_LAUNCH_COMBINE(128);
  else OPW_LAUNCH_COMBINE(256);
#undef OPW_LAUNCH_COMBINE
  if (e != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  st->launches += 1;
  return OPW_OK;
}

static opw_status_t enqueue_attention(opw_attn_stage_t* st, int32_t layer, int32_t batch, const void* q,
                                      const int32_t* kv_lens, const void* k_new, const void* v_new,
                                      const int32_t* positions, const int32_t* page_table, void* out, float* lse,
                                      void* cuda_stream) {
  const StepArgs a = {layer, batch, q, kv_lens, k_new, v_new, positions, page_table, out, lse};
  opw_status_t rc = validate_step(st, a);
  if (rc != OPW_OK) return rc;
  if (batch == 0) return OPW_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  rc = launch_attention(st, a, 0, stream);
  if (rc != OPW_OK) return rc;
  // With many rows the 128-thread instance wins (twice as many rows resident per SM hide the
  // chain of L2 round trips a row's merge is); with few long rows the 256-thread one does.
  const bool small = a.batch * st->cfg.num_kv_heads >= 2 * st->sms;
  return launch_combine(st, a, 0, stream, small);
}

opw_status_t opw_decode_attention(opw_attn_stage_t* st, int32_t layer, int32_t batch, const void* q,
                                  const int32_t* kv_lens, const int32_t* page_table, void* out, float* lse,
                                  void* cuda_stream) {
  if (!kv_lens) return OPW_ERR_INVALID_ARG;
  return enqueue_attention(st, layer, batch, q, kv_lens, nullptr, nullptr, nullptr, page_table, out, lse, cuda_stream);
}

opw_status_t opw_decode_step(opw_attn_stage_t* st, int32_t layer, int32_t batch, const void* q, const void* k_new,
                             const void* v_new, const int32_t* positions, const int32_t* page_table, void* out,
                             float* lse, void* cuda_stream) {
  if (!k_new || !v_new || !positions) return OPW_ERR_INVALID_ARG;
  return enqueue_attention(st, layer, batch, q, nullptr, k_new, v_new, positions, page_table, out, lse, cuda_stream);
}

opw_status_t opw_attn_stage_shape(const opw_attn_stage_t* st, int32_t* device, int32_t* num_layers, int32_t* Hq,
                                  int32_t* Hkv, int32_t* D, int32_t* max_batch) {
  if (!st) return OPW_ERR_INVALID_ARG;
  if (device) *device = st->cfg.device;
  if (num_layers) *num_layers = st->cfg.num_layers;
  if (Hq) *Hq = st->cfg.num_q_heads;
  if (Hkv) *Hkv = st->cfg.num_kv_heads;
  if (D) *D = st->cfg.head_dim;
  if (max_batch) *max_batch = st->cfg.max_batch;
  return OPW_OK;
}

opw_status_t opw_attn_stage_host_layout(const opw_attn_stage_t* st, size_t* q_off, size_t* k_off, size_t* v_off,
                                        size_t* pos_off, size_t* total_bytes) {
  if (!st || !q_off || !k_off || !v_off || !pos_off || !total_bytes) return OPW_ERR_INVALID_ARG;
  *q_off = 0;
  *k_off = st->lay.st_k - st->lay.st_q;
  *v_off = st->lay.st_v - st->lay.st_q;
  *pos_off = st->lay.st_pos - st->lay.st_q;
  *total_bytes = (st->lay.st_pos - st->lay.st_q) + (size_t)st->cfg.max_batch * 4;
  return OPW_OK;
}

opw_status_t opw_decode_step_host(opw_attn_stage_t* st, int32_t layer, int32_t batch, const void* q_host,
                                  const void* k_new_host, const void* v_new_host, const int32_t* positions_host,
                                  const int32_t* page_table_host, void* out_host, float* lse_host, void* cuda_stream) {
  opw_status_t rc = check_step(st, layer, batch);
  if (rc != OPW_OK) return rc;
  if (!q_host || !k_new_host || !v_new_host || !positions_host || !out_host) return OPW_ERR_INVALID_ARG;
  if (batch == 0) return OPW_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t B = batch, Hq = st->cfg.num_q_heads, Hkv = st->cfg.num_kv_heads, D = st->cfg.head_dim;
  unsigned char* ws = st->ws;
  void* d_q = ws + st->lay.st_q;
  void* d_k = ws + st->lay.st_k;
  void* d_v = ws + st->lay.st_v;
  int32_t* d_pos = reinterpret_cast<int32_t*>(ws + st->lay.st_pos);
  void* d_out = ws + st->lay.st_out;
  float* d_lse = reinterpret_cast<float*>(ws + st->lay.st_lse);
  const size_t table_elems = (size_t)st->cfg.max_batch * st->cfg.max_pages_per_seq;
  int32_t* d_table = reinterpret_cast<int32_t*>(ws + st->lay.st_table) + (size_t)layer * table_elems;

  // With OPW_FLAG_COPY_STREAMS the copies in run on the stage's own stream, the kernels on the caller's, the
  // copies out on a third, chained by events: a second stage's kernels on the same stream then follow this
  // stage's kernels directly, and both stages' copies hide behind them.
  const bool split_streams = st->s_in != nullptr;
  cudaStream_t sin = split_streams ? st->s_in : stream, sout = split_streams ? st->s_out : stream;
  bool ok = true;
  if (split_streams) ok &= cudaStreamWaitEvent(sin, st->e_k, 0) == cudaSuccess;   // the staged inputs of the previous step are no longer read
  // Tensor packing: if the caller laid q, k_new, v_new and positions out in one host buffer at the
  // offsets of opw_attn_stage_host_layout, they travel as a single copy.
  const unsigned char* hq = static_cast<const unsigned char*>(q_host);
  const bool packed = static_cast<const unsigned char*>(k_new_host) == hq + (st->lay.st_k - st->lay.st_q) &&
                      static_cast<const unsigned char*>(v_new_host) == hq + (st->lay.st_v - st->lay.st_q) &&
                      reinterpret_cast<const unsigned char*>(positions_host) == hq + (st->lay.st_pos - st->lay.st_q);
  if (packed) {
    ok &= cudaMemcpyAsync(d_q, q_host, (st->lay.st_pos - st->lay.st_q) + B * 4, cudaMemcpyHostToDevice, sin) == cudaSuccess;
  } else {
    ok &= cudaMemcpyAsync(d_q, q_host, B * Hq * D * 2, cudaMemcpyHostToDevice, sin) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_k, k_new_host, B * Hkv * D * 2, cudaMemcpyHostToDevice, sin) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_v, v_new_host, B * Hkv * D * 2, cudaMemcpyHostToDevice, sin) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_pos, positions_host, B * 4, cudaMemcpyHostToDevice, sin) == cudaSuccess;
  }
  if (page_table_host)
    ok &= cudaMemcpyAsync(d_table, page_table_host, B * st->cfg.max_pages_per_seq * 4, cudaMemcpyHostToDevice,
                          sin) == cudaSuccess;
  if (split_streams) {
    ok &= cudaEventRecord(st->e_in, sin) == cudaSuccess;
    ok &= cudaStreamWaitEvent(stream, st->e_in, 0) == cudaSuccess;
    ok &= cudaStreamWaitEvent(stream, st->e_out, 0) == cudaSuccess;                 // the staged output of the previous step has left
  }
  if (!ok) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  rc = opw_decode_step(st, layer, batch, d_q, d_k, d_v, d_pos, d_table, d_out, lse_host ? d_lse : nullptr, cuda_stream);
  if (rc != OPW_OK) return rc;
  if (split_streams) {
    ok &= cudaEventRecord(st->e_k, stream) == cudaSuccess;
    ok &= cudaStreamWaitEvent(sout, st->e_k, 0) == cudaSuccess;
  }
  ok &= cudaMemcpyAsync(out_host, d_out, B * Hq * D * 2, cudaMemcpyDeviceToHost, sout) == cudaSuccess;
  if (lse_host) ok &= cudaMemcpyAsync(lse_host, d_lse, B * Hq * 4, cudaMemcpyDeviceToHost, sout) == cudaSuccess;
  if (split_streams) ok &= cudaEventRecord(st->e_out, sout) == cudaSuccess;
  if (!ok) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  return OPW_OK;
}

opw_status_t opw_attn_stage_page_table_delta_host(opw_attn_stage_t* st, int32_t layer, const int32_t* triples_host,
                                                  int32_t n, void* cuda_stream) {
  if (!st || layer < 0 || layer >= st->cfg.num_layers || n < 0 || (n > 0 && !triples_host)) return OPW_ERR_INVALID_ARG;
  if ((size_t)n > kDeltaPerRow * (size_t)st->cfg.max_batch) return OPW_ERR_CAPACITY;
  if (n == 0) return OPW_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int32_t* d_tri = reinterpret_cast<int32_t*>(st->ws + st->lay.st_delta);
  const size_t table_elems = (size_t)st->cfg.max_batch * st->cfg.max_pages_per_seq;
  int32_t* d_table = reinterpret_cast<int32_t*>(st->ws + st->lay.st_table) + (size_t)layer * table_elems;
  if (cudaMemcpyAsync(d_tri, triples_host, (size_t)n * 12, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  opw::table_delta_kernel<<<(n + 255) / 256, 256, 0, stream>>>(d_table, d_tri, n, st->cfg.max_batch, st->cfg.max_pages_per_seq,
                                                               reinterpret_cast<uint32_t*>(st->ws + st->lay.status));
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
  st->launches += 1;
  return OPW_OK;
}

opw_status_t opw_hbm_read_probe(const void* buffer, size_t bytes, float* sink, void* cuda_stream) {
  if (!buffer || !sink || bytes == 0 || (bytes & 15) || (reinterpret_cast<uintptr_t>(buffer) & 15)) return OPW_ERR_INVALID_ARG;
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
  int blocks = query_sms(device) * 8;                     // 8 blocks of 256 threads per SM, grid-stride
  if (blocks > 4096) blocks = 4096;
  opw::read_probe_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(buffer), (int64_t)(bytes / 16), sink);
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
  return OPW_OK;
}

opw_status_t opw_attn_stage_probe_timeout(opw_attn_stage_t* st, void* cuda_stream) {
  if (!st) return OPW_ERR_INVALID_ARG;
  opw::wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      reinterpret_cast<uint32_t*>(st->ws + st->lay.status));
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
  st->launches += 1;
  return OPW_OK;
}

opw_status_t opw_attn_stage_poll_error(opw_attn_stage_t* st, void* cuda_stream) {
  if (!st) return OPW_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  uint32_t* d = reinterpret_cast<uint32_t*>(st->ws + st->lay.status);
  if (cudaMemcpyAsync(&word, d, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemsetAsync(d, 0, 4, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  if (word & opw::kErrBadPage) return OPW_ERR_BAD_PAGE;
  if (word & opw::kErrTimeout) return OPW_ERR_TIMEOUT;
  return OPW_OK;
}

// ---------------------------------------------------------------------------------------
// Plans: the per-token sequence of a stage, submitted with one native call
// ---------------------------------------------------------------------------------------
}  // extern "C"

struct opw_attn_plan {
  opw_attn_stage* stage;
  std::vector<opw_step_item_t> items;
  // the other ops of a mixed plan (recurrent-state steps, whole attention modules), in the order given;
  // each runs after attention item extra_after[i] (-1: before the first)
  std::vector<opw_plan_op_t> extra;
  std::vector<int> extra_after;
  uint32_t flags;
  cudaStream_t side;                     // OPW_PLAN_OVERLAP: the combines run here
  std::vector<cudaEvent_t> ev_attn, ev_comb;
  cudaGraph_t graph;
  cudaGraphExec_t exec;
  int64_t launches_per_submit;
};

namespace {

// Enqueue the whole sequence on `stream`: for every item append then attention, then (with
// OPW_PLAN_ADVANCE) one step forward for every distinct positions / kv_lens array.
// OPW_PLAN_OVERLAP: item i's combine runs on a side stream beside item i+1's split-KV kernel.
// The two alternate between the stage's two workspace sets; item i+2's split-KV kernel waits
// for item i's combine (same set); the main stream rejoins the side stream at the end.
opw_status_t enqueue_plan_overlapped(opw_attn_plan* pl, cudaStream_t stream, cudaStream_t side) {
  opw_attn_stage* st = pl->stage;
  const int n = (int)pl->items.size();
  int last = -1, live = 0;
  int last_in_set[2] = {-1, -1};              // the item whose combine last used each workspace set
  for (int i = 0; i < n; ++i) {
    const opw_step_item_t& it = pl->items[i];
    if (it.batch == 0) continue;              // nothing is enqueued or recorded for an empty item
    const bool fused = it.k_new && !it.kv_lens;
    if (it.k_new && !fused) {
      opw_status_t rc = opw_kv_append(st, it.layer, it.batch, it.k_new, it.v_new, it.positions, it.page_table, stream);
      if (rc != OPW_OK) return rc;
    }
    const StepArgs a = {it.layer, it.batch, it.q, fused ? nullptr : it.kv_lens, fused ? it.k_new : nullptr,
                        fused ? it.v_new : nullptr, fused ? it.positions : nullptr, it.page_table, it.out, it.lse};
    const int set = live & 1;
    if (last_in_set[set] >= 0 && cudaStreamWaitEvent(stream, pl->ev_comb[last_in_set[set]], 0) != cudaSuccess)
      return OPW_ERR_CUDA;
    opw_status_t rc = launch_attention(st, a, set, stream);
    if (rc != OPW_OK) return rc;
    if (cudaEventRecord(pl->ev_attn[i], stream) != cudaSuccess || cudaStreamWaitEvent(side, pl->ev_attn[i], 0) != cudaSuccess)
      return OPW_ERR_CUDA;
    rc = launch_combine(st, a, set, side, true, true);
    if (rc != OPW_OK) return rc;
    if (cudaEventRecord(pl->ev_comb[i], side) != cudaSuccess) return OPW_ERR_CUDA;
    last_in_set[set] = i;
    ++live;
    last = i;
  }
  if (last >= 0 && cudaStreamWaitEvent(stream, pl->ev_comb[last], 0) != cudaSuccess) return OPW_ERR_CUDA;
  return OPW_OK;
}

opw_status_t enqueue_plan(opw_attn_plan* pl, cudaStream_t stream, cudaStream_t side) {
  opw_attn_stage* st = pl->stage;
  if (pl->flags & OPW_PLAN_OVERLAP) {
    opw_status_t rc = enqueue_plan_overlapped(pl, stream, side);
    if (rc != OPW_OK) { (void)cudaGetLastError(); return rc; }
  } else
  for (int i = -1; i < (int)pl->items.size(); ++i) {
    for (size_t j = 0; j < pl->extra.size(); ++j) {        // the other ops placed after item i
      if (pl->extra_after[j] != i) continue;
      if (pl->extra[j].kind == OPW_OP_LINEAR) {
        const opw_linear_item_t& ln = pl->extra[j].linear;
        opw_status_t rl = opw_linear_attn_decode_step(ln.batch, ln.num_k_heads, ln.num_v_heads, ln.dk, ln.dv, ln.state,
                                                      ln.num_slots, ln.slot, ln.q, ln.k, ln.v, ln.a, ln.beta, ln.scale,
                                                      ln.out, stream);
        if (rl != OPW_OK) return rl;
        if (ln.batch > 0) st->launches += 1;
      } else {
        const opw_afd_item_t& am = pl->extra[j].afd;     // counts its own launches (and the stage its attention's)
        opw_status_t ra = opw_afd_module_step(am.module, am.batch, am.x, am.positions, am.page_table, am.y, stream);
        if (ra != OPW_OK) return ra;
      }
    }
    if (i + 1 >= (int)pl->items.size()) break;
    const opw_step_item_t& it = pl->items[i + 1];
    opw_status_t rc;
    if (it.k_new && !it.kv_lens) {              // one fused launch: append inside the attention kernel
      rc = opw_decode_step(st, it.layer, it.batch, it.q, it.k_new, it.v_new, it.positions, it.page_table, it.out,
                           it.lse, stream);
    } else {
      if (it.k_new) {
        rc = opw_kv_append(st, it.layer, it.batch, it.k_new, it.v_new, it.positions, it.page_table, stream);
        if (rc != OPW_OK) return rc;
      }
      rc = opw_decode_attention(st, it.layer, it.batch, it.q, it.kv_lens, it.page_table, it.out, it.lse, stream);
    }
    if (rc != OPW_OK) return rc;
  }
  if (pl->flags & OPW_PLAN_ADVANCE) {
    std::vector<const void*> done;
    std::vector<opw_step_item_t> moving(pl->items);
    for (const opw_plan_op_t& op : pl->extra)
      if (op.kind == OPW_OP_AFD_MODULE) {
        opw_step_item_t it = {};
        it.batch = op.afd.batch;
        it.positions = op.afd.positions;
        moving.push_back(it);
      }
    for (const opw_step_item_t& it : moving) {
      int32_t* pos = it.positions;
      int32_t* len = it.kv_lens;
      for (const void* d : done) {
        if (d == pos) pos = nullptr;
        if (d == len) len = nullptr;
      }
      if (!pos && !len) continue;
      if (pos) done.push_back(pos);
      if (len) done.push_back(len);
      if (it.batch == 0) continue;
      opw::advance_kernel<<<(it.batch + 255) / 256, 256, 0, stream>>>(pos, len, it.batch);
      if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
      st->launches += 1;
    }
  }
  return OPW_OK;
}

}  // namespace

extern "C" {

static opw_status_t build_plan(opw_attn_stage_t* st, const opw_step_item_t* items, int32_t n_items,
                               const opw_plan_op_t* extra, const int* extra_after, int32_t n_extra, uint32_t flags,
                               opw_attn_plan_t** out) {
  if (!st || !out || n_items < 0 || n_items + n_extra < 1 || (n_items > 0 && !items)) return OPW_ERR_INVALID_ARG;
  if (flags & ~(uint32_t)(OPW_PLAN_GRAPH | OPW_PLAN_ADVANCE | OPW_PLAN_OVERLAP)) return OPW_ERR_INVALID_ARG;
  if ((flags & OPW_PLAN_OVERLAP) && n_extra > 0) return OPW_ERR_UNSUPPORTED;
  for (int i = 0; i < n_items; ++i) {
    const opw_step_item_t& it = items[i];
    opw_status_t rc = check_step(st, it.layer, it.batch);
    if (rc != OPW_OK) return rc;
    if (!it.q || !it.page_table || !it.out) return OPW_ERR_INVALID_ARG;
    if (!it.kv_lens && !it.k_new) return OPW_ERR_INVALID_ARG;
    if ((it.k_new == nullptr) != (it.v_new == nullptr)) return OPW_ERR_INVALID_ARG;
    if (it.k_new && !it.positions) return OPW_ERR_INVALID_ARG;
    if (((uintptr_t)it.q | (uintptr_t)it.out | (uintptr_t)it.k_new | (uintptr_t)it.v_new) % 16) return OPW_ERR_INVALID_ARG;
    if (((uintptr_t)it.kv_lens | (uintptr_t)it.positions | (uintptr_t)it.page_table | (uintptr_t)it.lse) % 4)
      return OPW_ERR_INVALID_ARG;
  }
  if (flags & OPW_PLAN_OVERLAP) {
    // a step's combine runs beside the next step's attention: they must not share outputs
    // (consecutive among the items that launch anything: empty items are skipped)
    int prev = -1;
    for (int i = 0; i < n_items; ++i) {
      if (items[i].batch == 0) continue;
      if (prev >= 0 && (items[prev].out == items[i].out || (items[prev].lse && items[prev].lse == items[i].lse)))
        return OPW_ERR_INVALID_ARG;
      prev = i;
    }
  }
  opw_attn_plan* pl = new (std::nothrow) opw_attn_plan();
  if (!pl) return OPW_ERR_INVALID_ARG;
  pl->stage = st;
  if (n_items > 0) pl->items.assign(items, items + n_items);
  if (n_extra > 0) {
    pl->extra.assign(extra, extra + n_extra);
    pl->extra_after.assign(extra_after, extra_after + n_extra);
  }
  pl->flags = flags;
  pl->side = nullptr;
  if (flags & OPW_PLAN_OVERLAP) {
    bool ok = cudaStreamCreateWithFlags(&pl->side, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 2 * n_items; ++i) {
      cudaEvent_t ev = nullptr;
      ok = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
      if (ok) (i < n_items ? pl->ev_attn : pl->ev_comb).push_back(ev);
    }
    if (!ok) {
      (void)cudaGetLastError();
      opw_attn_plan_destroy(pl);
      return OPW_ERR_CUDA;
    }
  }
  pl->graph = nullptr;
  pl->exec = nullptr;
  pl->launches_per_submit = 0;
  if (flags & OPW_PLAN_GRAPH) {
    // Capture the sequence once on a private stream; nothing runs during the capture.
    cudaStream_t cs = nullptr;
    const int64_t before = st->launches;
    bool ok = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
    opw_status_t rc = ok ? enqueue_plan(pl, cs, pl->side) : OPW_ERR_CUDA;
    if (ok) ok = cudaStreamEndCapture(cs, &pl->graph) == cudaSuccess && pl->graph != nullptr;
    if (ok && rc == OPW_OK) ok = cudaGraphInstantiate(&pl->exec, pl->graph, 0) == cudaSuccess;
    if (cs) cudaStreamDestroy(cs);
    pl->launches_per_submit = st->launches - before;
    st->launches = before;                      // captured, not launched
    if (!ok || rc != OPW_OK) {
      (void)cudaGetLastError();
      opw_attn_plan_destroy(pl);
      return rc != OPW_OK ? rc : OPW_ERR_CUDA;
    }
  }
  *out = pl;
  return OPW_OK;
}

opw_status_t opw_attn_plan_create(opw_attn_stage_t* st, const opw_step_item_t* items, int32_t n_items, uint32_t flags,
                                  opw_attn_plan_t** out) {
  if (!items || n_items < 1) return OPW_ERR_INVALID_ARG;
  return build_plan(st, items, n_items, nullptr, nullptr, 0, flags, out);
}

opw_status_t opw_attn_plan_create_mixed(opw_attn_stage_t* st, const opw_plan_op_t* ops, int32_t n_ops, uint32_t flags,
                                        opw_attn_plan_t** out) {
  if (!st || !ops || n_ops < 1 || !out) return OPW_ERR_INVALID_ARG;
  std::vector<opw_step_item_t> items;
  std::vector<opw_plan_op_t> extra;
  std::vector<int> after;
  for (int i = 0; i < n_ops; ++i) {
    if (ops[i].kind == OPW_OP_ATTENTION) {
      items.push_back(ops[i].attention);
      continue;
    }
    if (ops[i].kind == OPW_OP_LINEAR) {
      const opw_linear_item_t& ln = ops[i].linear;
      if (ln.batch < 0 || !ln.state || !ln.slot || !ln.q || !ln.k || !ln.v || !ln.a || !ln.beta || !ln.out)
        return OPW_ERR_INVALID_ARG;
    } else if (ops[i].kind == OPW_OP_AFD_MODULE) {
      const opw_afd_item_t& am = ops[i].afd;
      if (!am.module || am.batch < 1 || !am.x || !am.positions || !am.page_table || !am.y) return OPW_ERR_INVALID_ARG;
    } else {
      return OPW_ERR_INVALID_ARG;
    }
    extra.push_back(ops[i]);
    after.push_back((int)items.size() - 1);
  }
  return build_plan(st, items.data(), (int32_t)items.size(), extra.data(), after.data(), (int32_t)extra.size(), flags, out);
}

opw_status_t opw_attn_plan_submit(opw_attn_plan_t* pl, void* cuda_stream) {
  if (!pl) return OPW_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (pl->exec) {
    if (cudaGraphLaunch(pl->exec, stream) != cudaSuccess) { (void)cudaGetLastError(); return OPW_ERR_CUDA; }
    pl->stage->launches += pl->launches_per_submit;
    return OPW_OK;
  }
  return enqueue_plan(pl, stream, pl->side);
}

opw_status_t opw_attn_plan_destroy(opw_attn_plan_t* pl) {
  if (!pl) return OPW_OK;
  if (pl->exec) cudaGraphExecDestroy(pl->exec);
  if (pl->graph) cudaGraphDestroy(pl->graph);
  for (cudaEvent_t ev : pl->ev_attn) cudaEventDestroy(ev);
  for (cudaEvent_t ev : pl->ev_comb) cudaEventDestroy(ev);
  if (pl->side) cudaStreamDestroy(pl->side);
  delete pl;
  return OPW_OK;
}

}  // extern "C"
