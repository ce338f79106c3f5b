// Device code of the decode attention stage: paged KV append, split-KV partial
// attention over TMA-staged pages, log-sum-exp combine.  sm_100a only.
//
// Work decomposition of the attention kernel.  A "unit" is one (sequence b, kv head g,
// logical page) triple inside the visible range of b; units are ordered by (b, g, page)
// and the U units of a launch are cut into equal contiguous shares, one per warp
// ("worker") of a persistent grid.  A share is cut again into kSegPerShare segments: the
// first 13/16 is the worker's own static segment, the last 3/16 is split into six ever
// smaller chunks that any worker may take through an atomic ticket once its static
// segment is done (SMs do not all stream at the same rate -- finish times of equal static
// shares spread by about 15 % -- and the chunks even them out).  The segment boundaries depend only on kv_lens, the window and the grid,
// never on which warp runs a segment or on page ids, so the result is deterministic.
// A worker streams one 2*P*D*2-byte tile (K rows then V rows of one page and head,
// contiguous in the pool) per unit.  A segment meets at most two rows (b, g) it does not
// cover completely, its first and its last: complete rows are normalised and stored
// directly; the incomplete ones go to the segment's two partial slots and are merged by
// the combine kernel.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

// A second translation unit may instantiate these kernels under another namespace with
// another OPW_DYN_PER_SHARE; the defaults below are the library's main path.
#ifndef OPW_NAMESPACE
#define OPW_NAMESPACE opw
#endif

namespace OPW_NAMESPACE {

constexpr int kPage = 16;               // tokens per page
constexpr uint32_t kErrBadPage = 1u;    // bits of the device status word
constexpr uint32_t kErrTimeout = 2u;
constexpr int kMaxWarps = 16;
constexpr uint64_t kWaitLimitNs = 100ull * 1000 * 1000;   // bound of a wait on a shared-memory copy: 0.1 s

struct AttnParams {
  const __nv_bfloat16* pool;
  const __nv_bfloat16* q;
  const int32_t* kv_lens;      // keys visible per sequence, or null: then positions[b] + 1
  const int32_t* page_table;
  // Fused append (all three null or all three set): the worker that streams the last page of
  // row (b, g) also stores k_new[b,g,:] / v_new[b,g,:] into slot positions[b] of that page,
  // in the pool and in its shared-memory copy of the tile.
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  const int32_t* positions;
  __nv_bfloat16* pool_w;
  __nv_bfloat16* out;
  float* lse;            // may be null
  float* partials;       // [num_workers*2][G*(D+2)]
  int32_t* cum;          // [batch+1] pages before sequence b (written by block 0)
  uint32_t* status;
  int32_t* ticket;       // dynamic-chunk counter, zero at launch (the combine kernel re-zeroes it)
  int32_t* split_list;   // or null.  Many-row launches: the rows left as partials, each listed once, by the worker
  int32_t* split_count;  // whose segment holds the row's first unit; [0] their number (zero at launch; the combine re-zeroes it)
  uint64_t* trace;       // optional [num_workers][4]: {smid | units<<32, t_begin, t_first_tile, t_end} in ns
  int64_t num_pages;
  int32_t batch, Hq, Hkv, G;
  int32_t max_pages;     // row stride of page_table
  int32_t window;        // 0 = full
  int32_t stages;        // ring depth per warp
  float scale_log2e;     // softmax scale * log2(e)
};

struct AppendParams {
  __nv_bfloat16* pool;
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  const int32_t* positions;
  const int32_t* page_table;
  uint32_t* status;
  int64_t num_pages;
  int32_t batch, Hkv, D, max_pages;
};

// ---------------------------------------------------------------------------------
// small PTX wrappers
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait: returns false if the phase did not complete within kWaitLimitNs of the
// device's global timer (checked every 64 polls).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  uint64_t t0;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    if (t - t0 > kWaitLimitNs) return false;
  }
}
// Linear bulk copy global -> shared of this CTA, completion counted on an mbarrier.  The KV
// stream is read once per step, so it is marked evict-first in L2 and leaves the small
// re-read data (partials, q, page tables) alone.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}
// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may
// start while its predecessor in the stream still runs; it must not touch anything the
// predecessor (or, transitively, earlier kernels) produces before pdl_wait() returns.
__device__ __forceinline__ void prefetch_l1(const void* p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ uint32_t sm_id() {
  uint32_t r;
  asm volatile("mov.u32 %0, %smid;" : "=r"(r));
  return r;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------------------------
// shared host/device arithmetic of the unit decomposition
// ---------------------------------------------------------------------------------
// keys visible to sequence b: given directly, or one more than its pre-append length
__device__ __forceinline__ int32_t visible_keys(const int32_t* kv_lens, const int32_t* positions, int b) {
  if (kv_lens) return kv_lens[b];
  const int32_t pos = positions[b];
  return pos >= 0 ? pos + 1 : 0;
}
// pages of sequence with n visible keys under `window` : first logical page and count
__host__ __device__ __forceinline__ void visible_pages(int32_t n, int32_t window, int32_t max_pages,
                                                       int32_t& first, int32_t& count, int32_t& lo) {
  if (n <= 0) { first = 0; count = 0; lo = 0; return; }
  lo = (window > 0 && n > window) ? n - window : 0;
  first = lo / kPage;
  int32_t last = (n - 1) / kPage;
  if (last >= max_pages) last = max_pages - 1;   // caller error; recorded separately
  count = last - first + 1;
  if (count < 0) count = 0;
}
__host__ __device__ __forceinline__ int64_t worker_begin(int64_t U, int64_t worker, int64_t num_workers) {
  return (U * worker) / num_workers;
}
// the worker whose share [begin(w), begin(w+1)) holds unit u
__host__ __device__ __forceinline__ int64_t worker_of(int64_t U, int64_t u, int64_t num_workers) {
  return ((u + 1) * num_workers - 1) / U;
}
// Segments of a share: k = 0 is the static first 13/16; k = 1..J cut the last 3/16 into ever
// smaller chunks (cut points in sixteenths of that part).  J depends on the share length
// only (the same for every share of a launch): a segment costs a couple of microseconds of
// fixed work (ticket, descriptors, Q reload, partial flush) and two more partials for the combine,
// so short shares get fewer chunks (measured per step, back to back: shares of 28 units 53.1 -> 50.3 us
// with none instead of two, shares of 69 units 107.9 -> 105.8 us with two instead of four; shares of
// 221 units run the same with four as with six).
#ifndef OPW_DYN_PER_SHARE
#define OPW_DYN_PER_SHARE 6      /* upper bound of J; 0 builds static shares only */
#endif
#ifndef OPW_DYN_32NDS
#define OPW_DYN_32NDS 6          /* the dynamic part of a share, in 32nds: 6/32 = 3/16 */
#endif
constexpr int kDynPerShare = OPW_DYN_PER_SHARE;
constexpr int kSegPerShare = kDynPerShare + 1;   // partial slots are indexed with this stride
#if OPW_DYN_PER_SHARE != 0 && OPW_DYN_PER_SHARE != 6
#error "unsupported OPW_DYN_PER_SHARE"
#endif
// number of dynamic chunks per share for a launch of U units on num_workers workers
__host__ __device__ __forceinline__ int dyn_chunks(int64_t U, int64_t num_workers) {
  if (kDynPerShare == 0) return 0;
  const int64_t per = U / num_workers;
  return per < 32 ? 0 : per < 96 ? 2 : per < 256 ? 4 : 6;
}
__host__ __device__ __forceinline__ int64_t dyn_cut(int J, int k) {   // five bits per cut point
  const uint64_t cuts6 = 0ull | (5ull << 5) | (9ull << 10) | (12ull << 15) | (14ull << 20) | (15ull << 25) |
                         (16ull << 30);                                  // 0,5,9,12,14,15,16
  const uint64_t cuts4 = 0ull | (6ull << 5) | (11ull << 10) | (14ull << 15) | (16ull << 20);   // 0,6,11,14,16
  const uint64_t cuts2 = 0ull | (9ull << 5) | (16ull << 10);            // 0,9,16
  const uint64_t cuts = J == 6 ? cuts6 : J == 4 ? cuts4 : cuts2;
  return (int64_t)((cuts >> (5 * k)) & 31);
}
__host__ __device__ __forceinline__ void segment_bounds(int64_t U, int64_t num_workers, int64_t w, int k,
                                                        int64_t& a, int64_t& b) {
  const int J = dyn_chunks(U, num_workers);
  const int64_t s0 = worker_begin(U, w, num_workers), s1 = worker_begin(U, w + 1, num_workers);
  const int64_t len = s1 - s0, dyn = J > 0 ? (len * OPW_DYN_32NDS) >> 5 : 0, stat = len - dyn;
  if (k == 0) { a = s0; b = s0 + stat; return; }
  if (k > J) { a = b = s1; return; }            // this launch has fewer chunks per share
  a = s0 + stat + ((dyn * dyn_cut(J, k - 1)) >> 4);
  b = s0 + stat + ((dyn * dyn_cut(J, k)) >> 4);
}

// The same boundaries with one 64-bit division per thread instead of two per segment (the combine
// kernel is bound by this integer arithmetic, not by memory):
// begin(w) = floor(U*w/nw) = per*w + floor(rem*w/nw) with per = U / nw, rem = U % nw, and
// rem*w < nw^2 fits 32 bits (nw <= 16 warps x 4 blocks x a few hundred SMs).
struct ShareMath {
  int64_t per;
  uint32_t rem, nw;
  int J;
  __device__ __forceinline__ void init(int64_t U, int64_t num_workers) {
    nw = (uint32_t)num_workers;
    per = U / num_workers;
    rem = (uint32_t)(U - per * num_workers);
    J = dyn_chunks(U, num_workers);
  }
  __device__ __forceinline__ int64_t begin(uint32_t w) const { return per * (int64_t)w + (int64_t)((rem * w) / nw); }
  __device__ __forceinline__ void bounds(uint32_t w, int k, int64_t& a, int64_t& b) const {   // == segment_bounds
    const int64_t s0 = begin(w), s1 = begin(w + 1);
    const int64_t len = s1 - s0, dyn = J > 0 ? (len * OPW_DYN_32NDS) >> 5 : 0, stat = len - dyn;
    if (k == 0) { a = s0; b = s0 + stat; return; }
    if (k > J) { a = b = s1; return; }
    a = s0 + stat + ((dyn * dyn_cut(J, k - 1)) >> 4);
    b = s0 + stat + ((dyn * dyn_cut(J, k)) >> 4);
  }
};

// ---------------------------------------------------------------------------------
// KV append: one thread block per sequence, one thread per 16-byte group
// ---------------------------------------------------------------------------------
__global__ void kv_append_kernel(AppendParams p) {
  pdl_launch_dependents();                    // the attention kernel may start its prologue now
  const int b = blockIdx.x;
  const int32_t pos = p.positions[b];         // inputs only before the wait
  pdl_wait();                                 // everything enqueued earlier has finished
  if (pos < 0) return;
  const int32_t lp = pos / kPage, t = pos % kPage;
  if (lp >= p.max_pages) {
    if (threadIdx.x == 0) atomicOr(p.status, kErrBadPage);
    return;
  }
  const int64_t pid = p.page_table[(int64_t)b * p.max_pages + lp];
  if (pid < 0 || pid >= p.num_pages) {
    if (threadIdx.x == 0) atomicOr(p.status, kErrBadPage);
    return;
  }
  const int groups = p.D / 8;                       // 16-byte groups per row
  const int total = p.Hkv * 2 * groups;
  for (int i = threadIdx.x; i < total; i += blockDim.x) {
    const int c = i % groups, kv = (i / groups) & 1, g = i / (2 * groups);
    const __nv_bfloat16* src = (kv ? p.v_new : p.k_new) + ((int64_t)b * p.Hkv + g) * p.D + c * 8;
    __nv_bfloat16* dst =
        p.pool + ((((pid * p.Hkv + g) * 2 + kv) * kPage + t) * (int64_t)p.D) + ((c ^ (t & 7)) * 8);
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }
}

// One decode step further: positions and kv_lens of active rows grow by one (plans that
// replay a captured step sequence keep their metadata on the device).
__global__ void advance_kernel(int32_t* positions, int32_t* kv_lens, int32_t n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    if (positions && positions[i] >= 0) positions[i] += 1;
    if (kv_lens && kv_lens[i] > 0) kv_lens[i] += 1;
  }
}

// Page-table delta: entry i of `triples` is (batch row, logical page, physical page); the staged table of a
// layer takes the new mapping.  Entries outside the table are skipped and recorded.
__global__ void table_delta_kernel(int32_t* table, const int32_t* triples, int32_t n, int32_t max_batch, int32_t max_pages,
                                   uint32_t* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int32_t row = triples[3 * i], lp = triples[3 * i + 1], pid = triples[3 * i + 2];
  if (row < 0 || row >= max_batch || lp < 0 || lp >= max_pages) {
    atomicOr(status, kErrBadPage);
    return;
  }
  table[(int64_t)row * max_pages + lp] = pid;
}

// Self-test of the bounded wait: one warp arms a shared-memory barrier for bytes that no copy
// will ever deliver, waits for it the way the attention kernel waits for a tile, and must come
// back after kWaitLimitNs with the time-out recorded in the status word.  Nothing is in
// flight, so the kernel exits cleanly and the context stays usable.
__global__ void wait_probe_kernel(uint32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect_tx(b, 16);
  }
  __syncwarp();
  if (!mbar_wait_bounded(b, 0) && threadIdx.x == 0) atomicOr(status, kErrTimeout);
}

// ---------------------------------------------------------------------------------
// read-bandwidth probe: every 16-byte word of a buffer once, evict-first, eight loads in flight
// per thread; the per-block sums keep the loads alive
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) read_probe_kernel(const uint4* __restrict__ buf, int64_t n16, float* __restrict__ sink) {
  const uint64_t pol = l2_evict_first_policy();
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  uint32_t acc = 0;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                   : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                   : "l"(buf + i + u * stride), "l"(pol));
#pragma unroll
    for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = __ldg(buf + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ uint32_t part[8];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int w = 0; w < 8; ++w) t ^= part[w];
    sink[blockIdx.x] = __uint_as_float(t & 0x3fffffffu);   // any value: it only has to depend on every load
  }
}

// ---------------------------------------------------------------------------------
// split-KV partial attention
// ---------------------------------------------------------------------------------
// Dynamic shared memory: [ring: warps*stages tiles][mbarriers: warps*stages x 8 B]
//                        [cum: batch+1 int32][lens: batch int32]
template <int D>
struct AttnSmem {
  static constexpr int kTileBytes = 2 * kPage * D * 2;   // K rows then V rows of one page and head
  __host__ __device__ static size_t bytes(int warps, int stages, int batch) {
    return (size_t)warps * stages * kTileBytes + (size_t)warps * stages * 8 + (size_t)(2 * batch + 2) * 4 + 16;
  }
};

struct UnitDesc {   // one per lane, describing unit (window base + lane)
  int32_t tile;     // pid*Hkv + g  (index of the K|V tile in the pool), 0 if masked out
  int32_t row;      // b*Hkv + g
  int32_t info;     // t0 | t1<<8 | first<<16 | last<<17   (valid slots [t0,t1) of the page)
};

template <int D, bool HI>   // HI: query rows 8..15 of the MMA tile are in use (8 < G <= 16)
__global__ void __maxnreg__(D > 128 ? 255 : 200) attn_splitkv_kernel(AttnParams p) {
  constexpr int KS = D / 16;                 // k-steps of Q*K^T
  constexpr int NT = D / 8;                  // n-tiles of P*V
  constexpr int ROWB = D * 2;                // bytes per token row
  constexpr int TILE = AttnSmem<D>::kTileBytes;
  extern __shared__ __align__(128) unsigned char smem[];

  const int warps = blockDim.x >> 5;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int stages = p.stages;
  unsigned char* ring = smem;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)warps * stages * TILE);
  int32_t* cum = reinterpret_cast<int32_t*>(bars + warps * stages);
  int32_t* lens = cum + p.batch + 1;

  // ---- pages per sequence and their exclusive prefix sum (whole block) ----
  {
    __shared__ int32_t wsum[kMaxWarps];
    __shared__ int32_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < p.batch; base += blockDim.x) {
      const int b = base + threadIdx.x;
      int32_t cnt = 0, n = 0;
      if (b < p.batch) {
        n = visible_keys(p.kv_lens, p.positions, b);
        int32_t first, lo;
        if (n > p.max_pages * kPage) {            // beyond the table: clamp and record
          n = p.max_pages * kPage;
          atomicOr(p.status, kErrBadPage);
        }
        visible_pages(n, p.window, p.max_pages, first, cnt, lo);
        lens[b] = n;
      }
      int32_t incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int32_t v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) wsum[warp] = incl;
      __syncthreads();
      int32_t before = carry;
      for (int w = 0; w < warp; ++w) before += wsum[w];
      if (b < p.batch) cum[b] = before + incl - cnt;
      __syncthreads();
      if (threadIdx.x == blockDim.x - 1) carry = before + incl;
      __syncthreads();
    }
    if (threadIdx.x == 0) cum[p.batch] = carry;
    __syncthreads();
  }

  const int64_t U = (int64_t)cum[p.batch] * p.Hkv;
  const int64_t num_workers = (int64_t)gridDim.x * warps;
  const int64_t worker = (int64_t)blockIdx.x * warps + warp;
  if (U == 0) {
    // Nothing to stream, but the grid must still pass the dependency wait before it completes: under
    // programmatic stream serialisation a grid that exits without waiting lets its successor's wait
    // return while the predecessor of this grid is still running (ordering would not be transitive).
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0) p.cum[p.batch] = 0;
    return;
  }
  uint64_t* tr = p.trace ? p.trace + worker * 4 : nullptr;
  if (tr && lane == 0) tr[1] = global_timer_ns();

  // ---- this warp's ring ----
  const uint32_t ring_base = smem_u32(ring + (size_t)warp * stages * TILE);
  const uint32_t bar_base = smem_u32(bars + warp * stages);
  if (lane == 0) {
    for (int s = 0; s < stages; ++s) mbar_init(bar_base + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncwarp();

  int64_t u0 = 0, u1 = 0;                     // the segment being processed: units [u0, u1)

  // ---- unit descriptors, 32 at a time, one per lane ----
  auto describe = [&](int64_t u, int64_t u_end) -> UnitDesc {
    UnitDesc d;
    d.tile = 0; d.row = 0; d.info = 0;
    if (u >= u_end) return d;
    // sequence: largest b with cum[b]*Hkv <= u
    int lo_b = 0, hi_b = p.batch;             // invariant: cum[lo_b]*Hkv <= u < cum[hi_b]*Hkv
    while (hi_b - lo_b > 1) {
      const int mid = (lo_b + hi_b) >> 1;
      if ((int64_t)cum[mid] * p.Hkv <= u) lo_b = mid; else hi_b = mid;
    }
    const int b = lo_b;
    const int32_t n = lens[b];
    int32_t first, cnt, lo;
    visible_pages(n, p.window, p.max_pages, first, cnt, lo);
    const int32_t rem = (int32_t)(u - (int64_t)cum[b] * p.Hkv);
    const int g = rem / cnt, pgi = rem - g * cnt;
    const int32_t lp = first + pgi;
    int64_t pid = p.page_table[(int64_t)b * p.max_pages + lp];
    int t0 = lo - lp * kPage; if (t0 < 0) t0 = 0;
    int t1 = n - lp * kPage; if (t1 > kPage) t1 = kPage;
    if (pid < 0 || pid >= p.num_pages) {      // never dereference a bad page: mask it out
      atomicOr(p.status, kErrBadPage);
      pid = 0; t0 = 0; t1 = 0;
    }
    d.tile = (int32_t)(pid * p.Hkv + g);
    d.row = b * p.Hkv + g;
    d.info = t0 | (t1 << 8) | ((pgi == 0) << 16) | ((pgi == cnt - 1) << 17);
    return d;
  };

  int64_t wbase = 0;                          // unit of lane 0 in window A
  UnitDesc wa = {0, 0, 0}, wb = {0, 0, 0};    // descriptors of units [wbase, wbase+32) and the next 32
  UnitDesc nx = {0, 0, 0};                    // descriptors of the first 32 units of the next segment

  const uint64_t kv_policy = l2_evict_first_policy();
  auto issue_tile = [&](int32_t tile, int slot) {   // lane 0 issues the copy of one K|V tile
    if (lane == 0) {
      const uint32_t bar = bar_base + 8 * slot;
      mbar_expect_tx(bar, TILE);
      bulk_load(ring_base + slot * TILE, reinterpret_cast<const unsigned char*>(p.pool) + (int64_t)tile * TILE,
                TILE, bar, kv_policy);
    }
  };
  auto tile_of = [&](int64_t u) -> int32_t {  // warp-uniform u in [wbase, wbase+64)
    const int rel = (int)(u - wbase);
    const int32_t a = __shfl_sync(0xffffffffu, wa.tile, rel & 31);
    const int32_t b = __shfl_sync(0xffffffffu, wb.tile, rel & 31);
    return rel < 32 ? a : b;
  };

  // per-lane constant offsets of the matrix loads
  const int mi = lane >> 3, rr = lane & 7;
  const int qrow = lane >> 2, qcol = (lane & 3) * 2;
  const uint32_t k_row_off = (uint32_t)((rr + 8 * (mi >> 1)) * ROWB);           // K: token row of this lane
  const uint32_t v_row_off = (uint32_t)(kPage * ROWB + (rr + 8 * (mi & 1)) * ROWB);

  // row state
  uint32_t qa[KS][4];
  float o[NT][4];
  float m_lo = -1e30f, l_lo = 0.f, m_hi = -1e30f, l_hi = 0.f;
  bool seg_from_first = false;
  bool failed = false;

  int slot = 0;
  uint32_t phase = 0;
  int inflight = 0;                           // copies issued and not yet consumed
  int64_t u = 0;
  int64_t units_done = 0;
  bool traced_first = false;
  const int32_t num_tickets = (int32_t)(num_workers * dyn_chunks(U, num_workers));

  // The segment being processed is [u0,u1) with partial slots slot_base, slot_base+1; first the
  // worker's own static segment, then whatever chunks the ticket counter hands out.  The next
  // segment [n0,n1) is resolved a few units before the current one ends, so that its first
  // tiles are already on their way when the current segment's last tile is consumed.
  int64_t slot_base = 2 * (worker * kSegPerShare);
  segment_bounds(U, num_workers, worker, 0, u0, u1);
  int64_t n0 = 0, n1 = 0, nslot_base = 0;
  int next_issued = 0;                        // units of the next segment already issued
  wbase = u0;
  wa = describe(wbase + lane, u1);
  wb = describe(wbase + 32 + lane, u1);
  // Up to here only this step's inputs (kv_lens, page table) were read.  The pool (appended to
  // by the previous kernel), the workspace and the outputs are touched after this point.
  pdl_wait();
  if (blockIdx.x == 0)
    for (int i = lane + 32 * warp; i <= p.batch; i += blockDim.x) p.cum[i] = cum[i];
  for (;;) {
  int32_t ticket = 0;                         // asked for now, looked at near the segment's end
  if (lane == 0 && num_tickets > 0) ticket = atomicAdd(p.ticket, 1);
  bool next_known = false;
  bool seg_on_first_row = true;               // partial slot 0 for the segment's first row, 1 for its last
  {
    const int64_t len = u1 - u0;
    const int want = (int)(len < stages ? len : stages);
    for (int s = next_issued; s < want; ++s) {  // (re)fill the ring: what the previous segment did not prefetch
      int sl = slot + s; if (sl >= stages) sl -= stages;
      issue_tile(tile_of(u0 + s), sl);
      ++inflight;
    }
    units_done += len;
  }
  // resolve the next segment: skip empty chunks, stop when the tickets run out
  auto resolve_next = [&]() {
    int32_t t = __shfl_sync(0xffffffffu, ticket, 0);
    n0 = n1 = 0;
    while (t < num_tickets) {
      const int64_t w = t % (int32_t)num_workers;           // large chunks of every share first, small ones last
      const int k = 1 + t / (int32_t)num_workers;
      segment_bounds(U, num_workers, w, k, n0, n1);
      nslot_base = 2 * (w * kSegPerShare + k);
      if (n0 < n1) break;
      if (lane == 0) t = atomicAdd(p.ticket, 1);
      t = __shfl_sync(0xffffffffu, t, 0);
    }
    if (t >= num_tickets) n0 = n1 = 0;
    nx = describe(n0 + lane, n1);
    next_known = true;
    next_issued = 0;
    if (n0 < n1) {                            // the next segment starts with a row switch: its queries, its new key and value
      const int64_t nrow = __shfl_sync(0xffffffffu, nx.row, 0);
      if (lane * 64 < p.G * D) prefetch_l1(p.q + nrow * p.G * D + lane * 64);
      if (p.k_new != nullptr && (lane & 15) * 64 < D) prefetch_l1((lane < 16 ? p.k_new : p.v_new) + nrow * D + (lane & 15) * 64);
    }
  };
  for (u = u0; u < u1; ++u) {
    if (u - wbase == 32) {                    // slide the descriptor windows
      wbase += 32;
      wa = wb;
      wb = describe(wbase + 32 + lane, u1);
    }
    if (!next_known && u + stages + 2 >= u1) resolve_next();
    const int rel = (int)(u - wbase);
    const int32_t row = __shfl_sync(0xffffffffu, wa.row, rel);
    const int32_t info = __shfl_sync(0xffffffffu, wa.info, rel);
    const int32_t this_tile = __shfl_sync(0xffffffffu, wa.tile, rel);
    const int t0 = info & 0xff, t1 = (info >> 8) & 0xff;
    const bool first = (info >> 16) & 1, last = (info >> 17) & 1;
    const int b = row / p.Hkv, g = row - b * p.Hkv;

    if (first || u == u0) {                   // a new row starts: load Q, reset the state
      seg_from_first = first;
      const __nv_bfloat16* qb = p.q + ((int64_t)b * p.Hq + (int64_t)g * p.G) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qa[ks][0] = qa[ks][1] = qa[ks][2] = qa[ks][3] = 0u;
        if (qrow < p.G) {
          qa[ks][0] = *reinterpret_cast<const uint32_t*>(qb + qrow * D + ks * 16 + qcol);
          qa[ks][2] = *reinterpret_cast<const uint32_t*>(qb + qrow * D + ks * 16 + 8 + qcol);
        }
        if (HI && qrow + 8 < p.G) {
          qa[ks][1] = *reinterpret_cast<const uint32_t*>(qb + (qrow + 8) * D + ks * 16 + qcol);
          qa[ks][3] = *reinterpret_cast<const uint32_t*>(qb + (qrow + 8) * D + ks * 16 + 8 + qcol);
        }
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
      m_lo = m_hi = -1e30f;
      l_lo = l_hi = 0.f;
      // Rows follow each other in memory (q: [row][G][D], k_new / v_new: [row][D]) and, mostly, in this
      // worker's units: ask L1 for the next row's queries and its new key and value now, so that the next row
      // switch and that row's last unit do not each wait for an L2 round trip.
      if (row + 1 < p.batch * p.Hkv) {
        if (lane * 64 < p.G * D) prefetch_l1(p.q + (int64_t)(row + 1) * p.G * D + lane * 64);
        if (p.k_new != nullptr && (lane & 15) * 64 < D)
          prefetch_l1((lane < 16 ? p.k_new : p.v_new) + (int64_t)(row + 1) * D + (lane & 15) * 64);
      }
    }

    // fused append: this unit is the page that receives the step's new key/value row
    // (not when kv_lens was clamped to the table: a position beyond the table appends nowhere)
    const bool patch = p.k_new != nullptr && last && t1 > 0 && p.positions[b] + 1 == lens[b];
    // lanes 0..15 carry the K row, 16..31 the V row; a lane holds the row's 16-byte groups
    // pc, pc + 16 (the second only for head_dim 256)
    constexpr int NG = D / 8;                  // 16-byte groups per row
    constexpr int GPL = (NG + 15) / 16;        // groups per lane
    uint4 new_row[GPL];
    const int pc = lane & 15;
#pragma unroll
    for (int i = 0; i < GPL; ++i) {
      new_row[i] = make_uint4(0u, 0u, 0u, 0u);
      if (patch && pc + 16 * i < NG) {
        const __nv_bfloat16* src =
            (lane < 16 ? p.k_new : p.v_new) + ((int64_t)b * p.Hkv + g) * D + (pc + 16 * i) * 8;
        new_row[i] = *reinterpret_cast<const uint4*>(src);
      }
    }

    // wait for this unit's tile
    if (!mbar_wait_bounded(bar_base + 8 * slot, phase)) { failed = true; break; }
    --inflight;
    if (tr && !traced_first && lane == 0) tr[2] = global_timer_ns();
    traced_first = true;

    const uint32_t tile = ring_base + slot * TILE;
    if (patch) {
      const int tn = t1 - 1;                   // slot of the newest key inside this page
#pragma unroll
      for (int i = 0; i < GPL; ++i) {
        const int c = pc + 16 * i;
        if (c < NG) {
          const uint32_t off = (uint32_t)((lane < 16 ? 0 : kPage * ROWB) + tn * ROWB + ((c ^ (tn & 7)) << 4));
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(tile + off), "r"(new_row[i].x),
                       "r"(new_row[i].y), "r"(new_row[i].z), "r"(new_row[i].w)
                       : "memory");
          *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(p.pool_w) + (int64_t)this_tile * TILE + off) =
              new_row[i];
        }
      }
      __syncwarp();
    }
    const bool ragged = (t0 > 0) || (t1 < kPage);
    if (ragged) {
      // Slots outside [t0,t1) may hold anything (never written, or stale): their scores are
      // masked below, and their V rows are zeroed here so that 0 * garbage cannot make a NaN.
      for (int t = 0; t < kPage; ++t) {
        if (t >= t0 && t < t1) continue;
        for (int off = lane * 16; off < ROWB; off += 512)
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(tile + kPage * ROWB + t * ROWB + off), "r"(0u) : "memory");
      }
      __syncwarp();
    }
    // ---- S = Q K^T for the 16 tokens of the page ----
    float s[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t r0, r1, r2, r3;
      ldsm_x4(tile + k_row_off + ((((2 * ks + (mi & 1)) ^ rr)) << 4), r0, r1, r2, r3);
      mma_bf16(s[0], qa[ks][0], HI ? qa[ks][1] : 0u, qa[ks][2], HI ? qa[ks][3] : 0u, r0, r1);
      mma_bf16(s[1], qa[ks][0], HI ? qa[ks][1] : 0u, qa[ks][2], HI ? qa[ks][3] : 0u, r2, r3);
    }
    // ---- online softmax (base 2) ----
    float x[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        x[nt][e] = s[nt][e] * p.scale_log2e;
        if (ragged) {
          const int t = nt * 8 + qcol + (e & 1);
          if (t < t0 || t >= t1) x[nt][e] = -INFINITY;
        }
      }
    float mx_lo = fmaxf(fmaxf(x[0][0], x[0][1]), fmaxf(x[1][0], x[1][1]));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo);
    float mn_hi = m_hi;
    if (HI) {
      float mx_hi = fmaxf(fmaxf(x[0][2], x[0][3]), fmaxf(x[1][2], x[1][3]));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      mn_hi = fmaxf(m_hi, mx_hi);
    }
    const bool grew = (mn_lo > m_lo) || (HI && mn_hi > m_hi);
    if (__any_sync(0xffffffffu, grew)) {
      const float a_lo = fast_exp2(m_lo - mn_lo);
      l_lo *= a_lo;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) { o[nt][0] *= a_lo; o[nt][1] *= a_lo; }
      m_lo = mn_lo;
      if (HI) {
        const float a_hi = fast_exp2(m_hi - mn_hi);
        l_hi *= a_hi;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { o[nt][2] *= a_hi; o[nt][3] *= a_hi; }
        m_hi = mn_hi;
      }
    }
    float pr[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      pr[nt][0] = fast_exp2(x[nt][0] - m_lo);
      pr[nt][1] = fast_exp2(x[nt][1] - m_lo);
      l_lo += pr[nt][0] + pr[nt][1];
      if (HI) {
        pr[nt][2] = fast_exp2(x[nt][2] - m_hi);
        pr[nt][3] = fast_exp2(x[nt][3] - m_hi);
        l_hi += pr[nt][2] + pr[nt][3];
      } else {
        pr[nt][2] = pr[nt][3] = 0.f;
      }
    }
    const uint32_t pa0 = pack_bf16(pr[0][0], pr[0][1]);
    const uint32_t pa2 = pack_bf16(pr[1][0], pr[1][1]);
    const uint32_t pa1 = HI ? pack_bf16(pr[0][2], pr[0][3]) : 0u;
    const uint32_t pa3 = HI ? pack_bf16(pr[1][2], pr[1][3]) : 0u;
    // ---- O += P V ----
#pragma unroll
    for (int j = 0; j < KS; ++j) {
      uint32_t r0, r1, r2, r3;
      ldsm_x4_t(tile + v_row_off + ((((2 * j + (mi >> 1)) ^ rr)) << 4), r0, r1, r2, r3);
      mma_bf16(o[2 * j], pa0, pa1, pa2, pa3, r0, r1);
      mma_bf16(o[2 * j + 1], pa0, pa1, pa2, pa3, r2, r3);
    }

    // ---- refill this slot with the unit `stages` ahead ----
    __syncwarp();
    {
      const int64_t target = u + stages;      // this worker's stream runs on into the next segment
      if (target < u1) {
        const int32_t tile = tile_of(target);
        if (lane == 0) fence_proxy_async();
        issue_tile(tile, slot);
        ++inflight;
      } else {
        // Next-segment units are prefetched strictly in order; a segment shorter than the
        // ring starts past unit 0 here and leaves the next segment's fill to the loop top.
        const int j = (int)(target - u1);
        if (j == next_issued && j < 32 && j < n1 - n0) {
          const int32_t tile = __shfl_sync(0xffffffffu, nx.tile, j);
          if (lane == 0) fence_proxy_async();
          issue_tile(tile, slot);
          ++inflight;
          next_issued = j + 1;
        }
      }
    }
    if (++slot == stages) { slot = 0; phase ^= 1u; }

    // ---- end of the row (or of this worker's share of it) ----
    if (last || u == u1 - 1) {
      float l0 = l_lo, l1 = l_hi;
      l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
      l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
      if (HI) {
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
      }
      const bool complete = seg_from_first && last;
      if (complete) {
        const float i0 = l0 > 0.f ? 1.f / l0 : 0.f;
        const float i1 = (HI && l1 > 0.f) ? 1.f / l1 : 0.f;
        __nv_bfloat16* ob = p.out + ((int64_t)b * p.Hq + (int64_t)g * p.G) * D;
        if (qrow < p.G) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            *reinterpret_cast<uint32_t*>(ob + qrow * D + nt * 8 + qcol) = pack_bf16(o[nt][0] * i0, o[nt][1] * i0);
          if (p.lse && (lane & 3) == 0)
            p.lse[(int64_t)b * p.Hq + g * p.G + qrow] = l0 > 0.f ? (m_lo + log2f(l0)) * 0.6931471805599453f : -INFINITY;
        }
        if (HI && qrow + 8 < p.G) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            *reinterpret_cast<uint32_t*>(ob + (qrow + 8) * D + nt * 8 + qcol) = pack_bf16(o[nt][2] * i1, o[nt][3] * i1);
          if (p.lse && (lane & 3) == 0)
            p.lse[(int64_t)b * p.Hq + g * p.G + qrow + 8] = l1 > 0.f ? (m_hi + log2f(l1)) * 0.6931471805599453f : -INFINITY;
        }
      } else {
        // partial: unnormalised o, running max and sum, into this worker's slot
        if (p.split_list != nullptr && seg_from_first && lane == 0) p.split_list[atomicAdd(p.split_count, 1)] = row;
        const int64_t pslot = slot_base + (seg_on_first_row ? 0 : 1);
        float* pb = p.partials + pslot * (int64_t)(p.G * (D + 2));
        if (qrow < p.G) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            *reinterpret_cast<float2*>(pb + qrow * D + nt * 8 + qcol) = make_float2(o[nt][0], o[nt][1]);
          if ((lane & 3) == 0) { pb[p.G * D + qrow] = m_lo; pb[p.G * D + p.G + qrow] = l0; }
        }
        if (HI && qrow + 8 < p.G) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
            *reinterpret_cast<float2*>(pb + (qrow + 8) * D + nt * 8 + qcol) = make_float2(o[nt][2], o[nt][3]);
          if ((lane & 3) == 0) { pb[p.G * D + qrow + 8] = m_hi; pb[p.G * D + p.G + qrow + 8] = l1; }
        }
      }
      seg_on_first_row = false;
    }
  }
  if (failed) break;
  if (!next_known) resolve_next();            // (an empty segment never enters the loop above)
  if (n0 >= n1) break;                        // no chunk left
  u0 = n0; u1 = n1; slot_base = nslot_base;
  wbase = u0;
  wa = nx;
  wb = describe(wbase + 32 + lane, u1);
  }

  // The first warp of a block to run out of work lets the combine kernel queue up behind this grid:
  // late enough that its blocks do not sit on the SMs while the stream is still running.
  pdl_launch_dependents();
  if (tr && lane == 0) {
    tr[0] = (uint64_t)sm_id() | ((uint64_t)units_done << 32);
    tr[3] = global_timer_ns();
  }
  if (failed) {
    // A copy did not arrive in time: record it, then give every copy still in flight a
    // bounded chance to land before this warp's shared memory is released.
    if (lane == 0) atomicOr(p.status, kErrTimeout);
    for (int i = 0; i < inflight; ++i) {
      (void)mbar_wait_bounded(bar_base + 8 * slot, phase);
      if (++slot == stages) { slot = 0; phase ^= 1u; }
    }
  }
}

// ---------------------------------------------------------------------------------
// log-sum-exp combine
// ---------------------------------------------------------------------------------
struct CombineParams {
  int32_t* ticket;       // the attention kernel's chunk counter: re-zeroed here for the next launch
  const float* partials;
  const int32_t* cum;
  const int32_t* kv_lens;     // or null: then positions[b] + 1
  const int32_t* positions;
  float* scratch;             // [rows * splits][G*(D+2)] intermediates (used when gridDim.y > 1)
  int32_t* row_count;         // [rows] arrival counters, zero between launches
  const int32_t* split_list;  // or null.  List mode (many rows, most of them complete): the rows to merge, as the attention
  int32_t* split_count;       // kernel listed them; [0] their number, [1] blocks that have read it (both zero between launches)
  __nv_bfloat16* out;
  float* lse;
  int32_t batch, Hq, Hkv, G, D;
  int32_t max_pages, window;
  int32_t num_workers;
};

// One block of kCT threads per (sequence, kv head) row (and split); thread t owns the output
// elements t, t + kCT, ... of the row's [G, D] block.  256 threads by default; the 128-thread
// instance is small enough (registers) to share an SM with a split-KV block, which lets a plan
// run a step's combine beside the next step's attention.
constexpr int kCombineThreads = 256;
constexpr int kCombineThreadsSmall = 128;
constexpr int kCombineMaxG = 16;
constexpr int kCombineBatch = 64;               // segments merged per pass
constexpr int kCombineScanBatch = 1024;         // up to this batch a combine block recomputes the page prefix sums itself
// acc[j] = acc[j] * scale[h] + sum over the listed partials of weight * o, for the thread's
// elements e = tid + j * kCT.  The loads of one pass are all independent.
template <int NEL, int kCT>
__device__ __forceinline__ void combine_accumulate(float* acc, const float* partials, const int32_t* seg_slot,
                                                   const float* w_s, const float* run_scale, int nseg, int64_t stride,
                                                   int G, int D, int GD) {
  constexpr int US = 32 / NEL;
  int hh[NEL];
  bool ok[NEL];
#pragma unroll
  for (int j = 0; j < NEL; ++j) {
    const int e = threadIdx.x + j * kCT;
    ok[j] = e < GD;
    hh[j] = ok[j] ? e / D : 0;
    acc[j] *= run_scale[hh[j]];
  }
  int sgm = 0;
  for (; sgm + US <= nseg; sgm += US) {
    float o[NEL][US];
#pragma unroll
    for (int u = 0; u < US; ++u) {
      const float* sp = partials + (int64_t)seg_slot[sgm + u] * stride + threadIdx.x;
#pragma unroll
      for (int j = 0; j < NEL; ++j) o[j][u] = ok[j] ? __ldcg(sp + j * kCT) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < US; ++u)
#pragma unroll
      for (int j = 0; j < NEL; ++j) acc[j] += w_s[(sgm + u) * G + hh[j]] * o[j][u];
  }
  for (; sgm < nseg; ++sgm) {
    const float* sp = partials + (int64_t)seg_slot[sgm] * stride + threadIdx.x;
#pragma unroll
    for (int j = 0; j < NEL; ++j)
      if (ok[j]) acc[j] += w_s[sgm * G + hh[j]] * __ldcg(sp + j * kCT);
  }
}

// grid = (rows, splits).  With splits == 1 a block merges all of its row's partials and writes
// the output.  With splits > 1 (few rows, many partials each: long contexts at small batch)
// block (row, y) merges every splits-th batch of the row's partials into one intermediate
// partial in `scratch`, and the block that finishes last for the row (an atomic counter,
// nothing waits) merges those `splits` intermediates and writes the output.
// kD: the head dimension as a compile-time constant (0: read it from the parameters); the kernel is
// bound by integer arithmetic more than by memory, and divisions by D are a good part of it.
// One row (and split).  `listed`: list mode -- the dependency wait is behind the caller, the row is known to be
// split, and the prefix sums are read from memory.
template <int kCT, int kD>
__device__ __forceinline__ void combine_row(const CombineParams& p, const int row, const int split, const int splits,
                                            const bool listed) {
  const int b = row / p.Hkv, g = row - b * p.Hkv;
  const int D = kD ? kD : p.D, G = p.G;
  const int GD = G * D;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ int32_t seg_slot[kCombineBatch];
  __shared__ int32_t warp_cnt[kCT / 32];
  __shared__ int32_t scan_s[2][kCT / 32];
  __shared__ float w_s[kCombineBatch * kCombineMaxG];   // per (segment, head): m, then the weight
  __shared__ float l_s[kCombineBatch * kCombineMaxG];
  __shared__ float run_M[kCombineMaxG], run_L[kCombineMaxG], run_scale[kCombineMaxG];
  __shared__ int32_t is_last;
  constexpr int kMaxElems = kCombineMaxG * 128 / kCT;   // 8 (256 threads) or 16 (128 threads)
  const int nel = (GD + kCT - 1) / kCT;
  const int64_t stride = (int64_t)G * (D + 2);
  float acc[kMaxElems];
#pragma unroll
  for (int j = 0; j < kMaxElems; ++j) acc[j] = 0.f;
  if (threadIdx.x < kCombineMaxG) { run_M[threadIdx.x] = -INFINITY; run_L[threadIdx.x] = 0.f; }

  // keys visible to sequence bb, as the attention kernel counts them (clamped to the table)
  auto keys_of = [&](int bb) -> int32_t {
    int32_t nn = visible_keys(p.kv_lens, p.positions, bb);
    if (nn > p.max_pages * kPage) nn = p.max_pages * kPage;
    return nn;
  };
  const int32_t n = keys_of(b);               // an input: may be read before the attention kernel is done

  // Which segments overlap this row follows from the step's metadata alone (kv_lens / positions, the
  // window, the grid).  For batches up to kCombineScanBatch the block therefore works it out BEFORE the
  // dependency wait -- the page prefix sums, the candidate test and the list of partial slots of the
  // first batch of candidates -- so that under programmatic dependent launch all of it runs beneath the
  // attention kernel's tail and only the loads of the partials are left for afterwards.  Larger batches
  // read the prefix sums the attention kernel stored, after the wait.
  const bool early = !listed && p.batch <= kCombineScanBatch;
  int32_t cum_b = 0, cum_all = 0, cnt = 0;
  int64_t U = 0, ustart = 0, uend = 0, wf = 0, wl = 0, ncand = 0;
  ShareMath sm;
  int segs = 1;
  bool by_unit = false, whole = false;
  int nseg_first = 0;

  // candidates [base, base + kCombineBatch): test, ordered compaction into seg_slot; returns how many were listed
  auto list_candidates = [&](int64_t base) -> int {
    const int64_t i = base + threadIdx.x;
    bool hit = false;
    int32_t slot = 0;
    if (threadIdx.x < kCombineBatch && i < ncand) {
      int64_t j;                                   // candidate i = (share or unit j, segment k); 32-bit division where it fits
      if (ncand < (int64_t)1 << 31) j = (int64_t)((uint32_t)i / (uint32_t)segs);
      else j = i / segs;
      const int k = (int)(i - j * segs);
      int64_t w;
      bool counted = true;
      if (by_unit) {
        w = worker_of(U, ustart + j, p.num_workers);
        counted = j == 0 || worker_of(U, ustart + j - 1, p.num_workers) != w;
      } else {
        w = wf + j;
      }
      int64_t a, bnd;
      sm.bounds((uint32_t)w, k, a, bnd);
      hit = counted && a < bnd && a < uend && bnd > ustart;
      slot = (int32_t)(2 * (w * kSegPerShare + k) + (a >= ustart ? 0 : 1));
    }
    const uint32_t bal = __ballot_sync(0xffffffffu, hit);
    if (lane == 0) warp_cnt[warp] = __popc(bal);
    __syncthreads();
    int pos = __popc(bal & ((1u << lane) - 1u));
    int nseg = 0;
    for (int j = 0; j < kCombineBatch / 32; ++j) {
      if (j < warp) pos += warp_cnt[j];
      nseg += warp_cnt[j];
    }
    if (hit) seg_slot[pos] = slot;
    __syncthreads();
    return nseg;
  };

  // everything between the prefix sums and the first list of partial slots
  auto prepare = [&]() {
    if (n <= 0) return;                         // (uniform over the block)
    int32_t first, lo;
    visible_pages(n, p.window, p.max_pages, first, cnt, lo);
    U = (int64_t)cum_all * p.Hkv;
    ustart = (int64_t)cum_b * p.Hkv + (int64_t)g * cnt;
    uend = ustart + cnt;
    wf = worker_of(U, ustart, p.num_workers);
    wl = worker_of(U, uend - 1, p.num_workers);
    // segments a share really has in this launch (1 + the number of ticketed chunks, which depends on the
    // share length only): small launches have fewer than kSegPerShare, and fewer candidates to test
    sm.init(U, p.num_workers);
    segs = sm.J + 1;
    // If the segment that holds the row's first unit also holds its last, that segment's worker
    // stores the final result itself: nothing to merge (every block of the row sees this).
    bool w0 = false;
    if (threadIdx.x < segs) {
      int64_t a, bnd;
      sm.bounds((uint32_t)wf, (int)threadIdx.x, a, bnd);
      w0 = a <= ustart && ustart < bnd && bnd >= uend;
    }
    whole = __syncthreads_or(w0);
    if (whole) return;
    // Candidate shares are listed by share index (wf..wl), or, when the row has fewer units than
    // that (tiny launches: most shares are empty), by unit: the share holding unit ustart + j,
    // counted once, at its first unit inside the row.
    by_unit = (wl - wf + 1) > (int64_t)cnt;
    ncand = (by_unit ? (int64_t)cnt : (wl - wf + 1)) * segs;
    if ((int64_t)split * kCombineBatch < ncand) nseg_first = list_candidates((int64_t)split * kCombineBatch);
  };

  if (early) {
    // pages before sequence b and of the whole batch, from the metadata
    int32_t before = 0, total = 0;
    for (int bb = threadIdx.x; bb < p.batch; bb += kCT) {
      int32_t f, c, l;
      visible_pages(keys_of(bb), p.window, p.max_pages, f, c, l);
      total += c;
      if (bb < b) before += c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      before += __shfl_xor_sync(0xffffffffu, before, o);
      total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if (lane == 0) { scan_s[0][warp] = before; scan_s[1][warp] = total; }
    __syncthreads();
    for (int wq = 0; wq < kCT / 32; ++wq) { cum_b += scan_s[0][wq]; cum_all += scan_s[1][wq]; }
    prepare();
  }

  if (!listed) {
    pdl_wait();                                // partials and complete rows are final now
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *p.ticket = 0;
  }
  __nv_bfloat16* ob = p.out + ((int64_t)b * p.Hq + (int64_t)g * G) * D;
  float* lse_row = p.lse ? p.lse + (int64_t)b * p.Hq + g * G : nullptr;
  if (n <= 0) {   // inactive slot: zeros, lse = -inf
    if (split == 0) {
      for (int e = threadIdx.x; e < GD; e += kCT) ob[e] = __float2bfloat16(0.f);
      if (lse_row && threadIdx.x < G) lse_row[threadIdx.x] = -INFINITY;
    }
    return;
  }
  if (!early) {
    cum_b = p.cum[b];
    cum_all = p.cum[p.batch];
    prepare();
  }
  if (whole) return;
  // The row's partials come from the segments (share w in wf..wl, k in 0..kSegPerShare) that
  // overlap it.  A batch of candidate segments at a time: each thread tests one, an ordered
  // compaction lists the partial slots in shared memory, one warp per head turns the partials'
  // running maxima into weights 2^(m - M), and every thread sums its elements over the list.
  // A segment's partial for this row is in the segment's slot 0 if the segment starts inside
  // the row, else in slot 1.

  // One merge pass over `nseg` listed partials at `base_ptr` (slot stride `stride`): stage
  // (m, l), weights per head, then the weighted sums.
  auto merge_listed = [&](const float* base_ptr, int nseg) {
    for (int idx = threadIdx.x; idx < nseg * G; idx += kCT) {   // stage (m, l): independent loads
      const int sgm = idx / G, h = idx - sgm * G;
      const float* sp = base_ptr + (int64_t)seg_slot[sgm] * stride + GD;
      w_s[idx] = __ldcg(sp + h);
      l_s[idx] = __ldcg(sp + G + h);
    }
    __syncthreads();
    for (int h = warp; h < G; h += kCT / 32) {   // a warp per head: max, weights, sum of l
      float Mc = run_M[h];
      for (int sgm = lane; sgm < nseg; sgm += 32) Mc = fmaxf(Mc, w_s[sgm * G + h]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) Mc = fmaxf(Mc, __shfl_xor_sync(0xffffffffu, Mc, o));
      float Lc = 0.f;
      for (int sgm = lane; sgm < nseg; sgm += 32) {
        const float wgt = Mc == -INFINITY ? 0.f : exp2f(w_s[sgm * G + h] - Mc);
        w_s[sgm * G + h] = wgt;
        Lc += wgt * l_s[sgm * G + h];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) Lc += __shfl_xor_sync(0xffffffffu, Lc, o);
      if (lane == 0) {
        const float sc = Mc == -INFINITY ? 0.f : exp2f(run_M[h] - Mc);   // 0 on the first batch (run_M = -inf)
        run_L[h] = run_L[h] * sc + Lc;
        run_M[h] = Mc;
        run_scale[h] = sc;
      }
    }
    __syncthreads();
    // about 32 independent loads in flight per thread: NEL elements x (32 / NEL) segments
    if (nel <= 1) combine_accumulate<1, kCT>(acc, base_ptr, seg_slot, w_s, run_scale, nseg, stride, G, D, GD);
    else if (nel <= 2) combine_accumulate<2, kCT>(acc, base_ptr, seg_slot, w_s, run_scale, nseg, stride, G, D, GD);
    else if (nel <= 4) combine_accumulate<4, kCT>(acc, base_ptr, seg_slot, w_s, run_scale, nseg, stride, G, D, GD);
    else if (nel <= 8 || kMaxElems <= 8) combine_accumulate<(kMaxElems < 8 ? kMaxElems : 8), kCT>(acc, base_ptr, seg_slot, w_s, run_scale, nseg, stride, G, D, GD);
    else combine_accumulate<kMaxElems, kCT>(acc, base_ptr, seg_slot, w_s, run_scale, nseg, stride, G, D, GD);
    __syncthreads();
  };

  for (int64_t base = (int64_t)split * kCombineBatch; base < ncand; base += (int64_t)splits * kCombineBatch) {
    // the first batch was listed by prepare()
    const int nseg = base == (int64_t)split * kCombineBatch ? nseg_first : list_candidates(base);
    merge_listed(p.partials, nseg);
  }

  if (splits > 1) {
    // hand this block's intermediate (un-normalised sums relative to run_M) to the row's last block
    float* mine = p.scratch + ((int64_t)row * splits + split) * stride;
#pragma unroll
    for (int j = 0; j < kMaxElems; ++j) {
      const int e = threadIdx.x + j * kCT;
      if (e < GD) __stcg(mine + e, acc[j]);
    }
    if (threadIdx.x < G) {
      __stcg(mine + GD + threadIdx.x, run_M[threadIdx.x]);
      __stcg(mine + GD + G + threadIdx.x, run_L[threadIdx.x]);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const int32_t arrived = atomicAdd(p.row_count + row, 1);
      is_last = arrived == splits - 1;
      if (is_last) p.row_count[row] = 0;        // ready for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // merge the row's `splits` intermediates (splits <= kCombineBatch), in split order
#pragma unroll
    for (int j = 0; j < kMaxElems; ++j) acc[j] = 0.f;
    if (threadIdx.x < kCombineMaxG) { run_M[threadIdx.x] = -INFINITY; run_L[threadIdx.x] = 0.f; }
    if (threadIdx.x < splits) seg_slot[threadIdx.x] = row * splits + threadIdx.x;
    __syncthreads();
    merge_listed(p.scratch, splits);
  }
#pragma unroll
  for (int j = 0; j < kMaxElems; ++j) {
    const int e = threadIdx.x + j * kCT;
    if (e < GD) {
      const int h = e / D;
      const float Lh = run_L[h];
      ob[e] = __float2bfloat16_rn(Lh > 0.f ? acc[j] / Lh : 0.f);
      if (lse_row && e == h * D) lse_row[h] = Lh > 0.f ? (run_M[h] + log2f(Lh)) * 0.6931471805599453f : -INFINITY;
    }
  }
}


// grid = (rows, splits), or in list mode (p.split_list set; splits == 1) any number of blocks: a launch with very
// many rows has most of them complete (a row can only be split at one of the launch's segment boundaries, a few
// thousand), and a block per row just to find that out costs more than the merges.  There the attention kernel
// lists the rows it left as partials, and the blocks of this kernel walk that list; inactive rows, which no
// worker sees, are found and zeroed here.
template <int kCT, int kD = 0>
__global__ void __launch_bounds__(kCT, kCT == 128 ? 5 : 2) combine_kernel(CombineParams p) {
  pdl_launch_dependents();
  if (p.split_list == nullptr) {
    combine_row<kCT, kD>(p, blockIdx.x, blockIdx.y, gridDim.y, false);
    return;
  }
  __shared__ int32_t n_listed;
  pdl_wait();                                  // the list, the partials and the complete rows are final now
  if (threadIdx.x == 0) {
    n_listed = __ldcg(p.split_count);
    if (blockIdx.x == 0) *p.ticket = 0;
    // the last block to have read the count puts both counters back to zero for the next launch
    if (atomicAdd(p.split_count + 1, 1) == (int32_t)gridDim.x - 1) { p.split_count[0] = 0; p.split_count[1] = 0; }
  }
  __syncthreads();
  const int D = kD ? kD : p.D;
  for (int b = blockIdx.x; b < p.batch; b += gridDim.x) {     // inactive slots: zeros, lse = -inf
    if (visible_keys(p.kv_lens, p.positions, b) > 0) continue;
    __nv_bfloat16* ob = p.out + (int64_t)b * p.Hq * D;
    for (int e = threadIdx.x; e < p.Hq * D; e += kCT) ob[e] = __float2bfloat16(0.f);
    if (p.lse) for (int h = threadIdx.x; h < p.Hq; h += kCT) p.lse[(int64_t)b * p.Hq + h] = -INFINITY;
  }
  const int n = n_listed;
  for (int i = blockIdx.x; i < n; i += gridDim.x) {
    combine_row<kCT, kD>(p, __ldcg(p.split_list + i), 0, 1, true);
    __syncthreads();                           // the next row reuses the shared-memory state
  }
}

}  // namespace OPW_NAMESPACE
