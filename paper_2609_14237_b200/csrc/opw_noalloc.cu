// opw_decode_attention_noalloc: decode attention for callers that cannot allocate device
// memory at all -- no workspace to hand over, no stage handle to create.
//
// Who that is: code that runs where cudaMalloc is off limits -- a plug-in loaded into a
// serving process whose memory pool is owned and fully pre-sized by the host framework, a
// callback running under a memory budget that is already spent, a real-time path that must
// not take the allocator's lock.  Such a caller still owns its inputs and outputs (the
// KV pool, q, the page table, out), but has nowhere to put the split-KV scratch the normal
// entry point keeps in its caller-provided workspace.
//
// Here that scratch lives in one file-scope __device__ array of fixed size.  Every GPU that
// loads this library holds the array (kScratchBytes, about 10.7 MB) until the process exits,
// whether or not this entry point is ever called.  The kernels are the library's own split-KV
// and combine kernels, instantiated with static shares only (no dynamic chunks), which needs
// two partial slots per worker instead of fourteen and keeps the array small; the price is the
// uneven finish of the SMs that the main path's dynamic chunks remove.
//
// The name of a __device__ array is, in host code, only a handle for the runtime: passing it
// to a kernel as if it were an address would make the kernel fault or scribble over unrelated
// memory.  The device address is therefore resolved once per device with
// cudaGetSymbolAddress, with that device current, and it is that address the kernels get.
#include <cmath>
#include <mutex>

#include "opw_attn.h"

#define OPW_NAMESPACE opw_na
#undef OPW_DYN_PER_SHARE
#define OPW_DYN_PER_SHARE 0
#include "opw_kernels.cuh"

namespace {

constexpr int kMaxDevices = 64;
constexpr int kMaxSMs = 160;                      // workers = SMs x 8 warps
constexpr int kWarps = 8;
constexpr int kStages = 2;
constexpr int kMaxBatch = 4096;
constexpr int kMaxGroupFloats = 8 * (128 + 2);    // G*(D+2) <= 1040: G <= 8 at D = 128, G <= 15 at D = 64
constexpr size_t kStatusBytes = 256;
constexpr size_t kCumBytes = ((size_t)(kMaxBatch + 2) * 4 + 255) / 256 * 256;
constexpr size_t kPartialBytes = (size_t)kMaxSMs * kWarps * 2 * opw_na::kSegPerShare * kMaxGroupFloats * 4;
constexpr size_t kScratchBytes = kStatusBytes + kCumBytes + kPartialBytes;   // 10,666,496 bytes

// The scratch itself.  Shared by every call on the device and never cleared as a whole: the
// status and ticket words are zeroed at the start of each call, the prefix sums and the
// partial slots a call reads are always written by that same call first.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

struct DeviceState {
  std::once_flag once;
  cudaError_t err = cudaSuccess;
  unsigned char* scratch = nullptr;   // device address of g_scratch on this device
  int sms = 0;
};
DeviceState g_dev[kMaxDevices];

// Once per device, with that device current: resolve the array's device address, read the SM
// count, raise the split-KV kernels' dynamic shared-memory limit.  None of these allocates.
void setup_device(DeviceState* d, int device) {
  void* ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_scratch);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d->sms, cudaDevAttrMultiProcessorCount, device);
  const int smem = (int)opw_na::AttnSmem<128>::bytes(kWarps, kStages, kMaxBatch);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(opw_na::attn_splitkv_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(opw_na::attn_splitkv_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(opw_na::attn_splitkv_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(opw_na::attn_splitkv_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) (void)cudaGetLastError();
  d->err = e;
  d->scratch = static_cast<unsigned char*>(ptr);
}

}  // namespace

extern "C" opw_status_t opw_decode_attention_noalloc(int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                                                     int32_t page_size, int32_t window, float softmax_scale,
                                                     const void* kv_pool, int64_t num_pages, int32_t batch,
                                                     int32_t max_pages_per_seq, const void* q, const int32_t* kv_lens,
                                                     const int32_t* page_table, void* out, float* lse,
                                                     void* cuda_stream) {
  // ---- host-side checks, before any CUDA call ----
  if (num_q_heads < 1 || num_kv_heads < 1 || num_q_heads % num_kv_heads != 0 || batch < 0 || max_pages_per_seq < 1 ||
      window < 0 || num_pages < 1)
    return OPW_ERR_INVALID_ARG;
  if (!kv_pool || !q || !kv_lens || !page_table || !out) return OPW_ERR_INVALID_ARG;
  if ((uintptr_t)kv_pool % 128 || ((uintptr_t)q | (uintptr_t)out) % 16 || (uintptr_t)kv_lens % 4 ||
      (uintptr_t)page_table % 4 || (uintptr_t)lse % 4)
    return OPW_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f)) return OPW_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return OPW_ERR_UNSUPPORTED;
  if (page_size != opw_na::kPage) return OPW_ERR_UNSUPPORTED;
  const int G = num_q_heads / num_kv_heads;
  if (G > 16) return OPW_ERR_UNSUPPORTED;
  // the fixed scratch bounds the problem: refuse, do not truncate
  if (batch > kMaxBatch || G * (head_dim + 2) > kMaxGroupFloats) return OPW_ERR_CAPACITY;
  if ((int64_t)max_pages_per_seq * opw_na::kPage > INT32_MAX || num_pages * (int64_t)num_kv_heads > INT32_MAX)
    return OPW_ERR_UNSUPPORTED;
  if (batch == 0) return OPW_OK;

  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }
  DeviceState* d = &g_dev[device];
  std::call_once(d->once, setup_device, d, device);
  if (d->err != cudaSuccess || !d->scratch) return OPW_ERR_CUDA;
  if (d->sms < 1 || d->sms > kMaxSMs) return OPW_ERR_CAPACITY;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = d->scratch;
  // status word and ticket counter must start at zero; nothing else needs clearing
  if (cudaMemsetAsync(ws, 0, kStatusBytes, stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return OPW_ERR_CUDA;
  }

  opw_na::AttnParams p;
  p.pool = static_cast<const __nv_bfloat16*>(kv_pool);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.kv_lens = kv_lens;
  p.page_table = page_table;
  p.k_new = nullptr;                  // no fused append here
  p.v_new = nullptr;
  p.positions = nullptr;
  p.pool_w = nullptr;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = lse;
  p.partials = reinterpret_cast<float*>(ws + kStatusBytes + kCumBytes);
  p.cum = reinterpret_cast<int32_t*>(ws + kStatusBytes);
  p.status = reinterpret_cast<uint32_t*>(ws);
  p.ticket = reinterpret_cast<int32_t*>(ws + 16);
  p.split_list = nullptr;
  p.split_count = nullptr;
  p.trace = nullptr;
  p.num_pages = num_pages;
  p.batch = batch;
  p.Hq = num_q_heads;
  p.Hkv = num_kv_heads;
  p.G = G;
  p.max_pages = max_pages_per_seq;
  p.window = window;
  p.stages = kStages;
  const double scale = softmax_scale > 0.f ? (double)softmax_scale : 1.0 / std::sqrt((double)head_dim);
  p.scale_log2e = (float)(scale * 1.4426950408889634);

  const dim3 grid(d->sms), block(kWarps * 32);
  if (head_dim == 64) {
    const size_t smem = opw_na::AttnSmem<64>::bytes(kWarps, kStages, batch);
    if (G > 8) opw_na::attn_splitkv_kernel<64, true><<<grid, block, smem, stream>>>(p);
    else opw_na::attn_splitkv_kernel<64, false><<<grid, block, smem, stream>>>(p);
  } else {
    const size_t smem = opw_na::AttnSmem<128>::bytes(kWarps, kStages, batch);
    if (G > 8) opw_na::attn_splitkv_kernel<128, true><<<grid, block, smem, stream>>>(p);
    else opw_na::attn_splitkv_kernel<128, false><<<grid, block, smem, stream>>>(p);
  }
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;

  opw_na::CombineParams c;
  c.ticket = p.ticket;
  c.partials = p.partials;
  c.cum = p.cum;
  c.kv_lens = kv_lens;
  c.positions = nullptr;
  c.scratch = nullptr;                // one block per row: no intermediates
  c.row_count = nullptr;
  c.out = p.out;
  c.lse = lse;
  c.batch = batch;
  c.Hq = num_q_heads;
  c.Hkv = num_kv_heads;
  c.G = G;
  c.D = head_dim;
  c.max_pages = max_pages_per_seq;
  c.window = window;
  c.num_workers = d->sms * kWarps;
  c.split_list = nullptr;
  c.split_count = nullptr;
  opw_na::combine_kernel<opw_na::kCombineThreads><<<batch * num_kv_heads, opw_na::kCombineThreads, 0, stream>>>(c);
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
  return OPW_OK;
}
