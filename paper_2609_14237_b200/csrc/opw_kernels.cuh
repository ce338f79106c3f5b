// Device code of the decode attention stage: paged KV append, split-KV partial
// attention over TMA-staged pages, log-sum-exp combine.  sm_100a only.
//
// Work decomposition of the attention kernel.  A "unit" is one (sequence b, kv head g,
// logical page) triple inside the visible range of b; units are ordered by (b, g, page)
// and the U units of a launch are cut into equal contiguous ranges, one per warp
// ("worker") of a persistent grid.  A worker therefore streams one 2*P*D*2-byte tile
// (K rows then V rows of one page and head, contiguous in the pool) per unit, and meets
// at most two rows (b, g) it does not own completely: the first and the last of its
// range.  Complete rows are normalised and stored directly; the (at most two) incomplete
// ones go to fixed partial slots 2*worker and 2*worker+1 and are merged by the combine
// kernel.  Nothing in this scheme depends on page ids, only on kv_lens and the window.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace opw {

constexpr int kPage = 16;               // tokens per page
constexpr uint32_t kErrBadPage = 1u;    // bits of the device status word
constexpr uint32_t kErrTimeout = 2u;
constexpr int kMaxWarps = 8;
constexpr uint32_t kSpinLimit = 1u << 22;   // bounded wait on a shared-memory copy

struct AttnParams {
  const __nv_bfloat16* pool;
  const __nv_bfloat16* q;
  const int32_t* kv_lens;
  const int32_t* page_table;
  __nv_bfloat16* out;
  float* lse;            // may be null
  float* partials;       // [num_workers*2][G*(D+2)]
  int32_t* cum;          // [batch+1] pages before sequence b (written by block 0)
  uint32_t* status;
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
// Bounded wait: returns false if the phase did not complete within kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// Linear bulk copy global -> shared of this CTA, completion counted on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
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
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------------------------
// shared host/device arithmetic of the unit decomposition
// ---------------------------------------------------------------------------------
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
// the worker whose range [begin(w), begin(w+1)) holds unit u
__host__ __device__ __forceinline__ int64_t worker_of(int64_t U, int64_t u, int64_t num_workers) {
  return ((u + 1) * num_workers - 1) / U;
}

// ---------------------------------------------------------------------------------
// KV append: one thread block per sequence, one thread per 16-byte group
// ---------------------------------------------------------------------------------
__global__ void kv_append_kernel(AppendParams p) {
  const int b = blockIdx.x;
  const int32_t pos = p.positions[b];
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

// kv_lens = positions + 1 for the host-buffer step (inactive rows become 0)
__global__ void lens_from_positions_kernel(const int32_t* pos, int32_t* lens, int32_t n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) lens[i] = pos[i] >= 0 ? pos[i] + 1 : 0;
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
__global__ void __launch_bounds__(kMaxWarps * 32, 1) attn_splitkv_kernel(AttnParams p) {
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
        n = p.kv_lens[b];
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
    if (blockIdx.x == 0)
      for (int i = threadIdx.x; i <= p.batch; i += blockDim.x) p.cum[i] = cum[i];
  }

  const int64_t U = (int64_t)cum[p.batch] * p.Hkv;
  const int64_t num_workers = (int64_t)gridDim.x * warps;
  const int64_t worker = (int64_t)blockIdx.x * warps + warp;
  const int64_t u0 = worker_begin(U, worker, num_workers);
  const int64_t u1 = worker_begin(U, worker + 1, num_workers);
  if (u0 >= u1) return;

  // ---- this warp's ring ----
  const uint32_t ring_base = smem_u32(ring + (size_t)warp * stages * TILE);
  const uint32_t bar_base = smem_u32(bars + warp * stages);
  if (lane == 0) {
    for (int s = 0; s < stages; ++s) mbar_init(bar_base + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncwarp();

  // ---- unit descriptors, 32 at a time, one per lane ----
  auto describe = [&](int64_t u) -> UnitDesc {
    UnitDesc d;
    d.tile = 0; d.row = 0; d.info = 0;
    if (u >= u1) return d;
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

  int64_t wbase = u0;                         // unit of lane 0 in window A
  UnitDesc wa = describe(wbase + lane);
  UnitDesc wb = describe(wbase + 32 + lane);

  auto tile_of = [&](int64_t u) -> int32_t {  // warp-uniform u in [wbase, wbase+64)
    const int rel = (int)(u - wbase);
    const int32_t a = __shfl_sync(0xffffffffu, wa.tile, rel & 31);
    const int32_t b = __shfl_sync(0xffffffffu, wb.tile, rel & 31);
    return rel < 32 ? a : b;
  };
  auto issue = [&](int64_t u, int slot) {     // all lanes call; lane 0 issues
    const int32_t tile = tile_of(u);
    if (lane == 0) {
      const uint32_t bar = bar_base + 8 * slot;
      mbar_expect_tx(bar, TILE);
      bulk_load(ring_base + slot * TILE, reinterpret_cast<const unsigned char*>(p.pool) + (int64_t)tile * TILE,
                TILE, bar);
    }
  };

  // prologue: fill the ring
  const int prolog = (int)((u1 - u0) < stages ? (u1 - u0) : stages);
  for (int s = 0; s < prolog; ++s) issue(u0 + s, s);

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
  bool seg_is_workers_first = true;
  bool failed = false;

  int slot = 0;
  uint32_t phase = 0;
  int64_t u = u0;
  for (; u < u1; ++u) {
    if (u - wbase == 32) {                    // slide the descriptor windows
      wbase += 32;
      wa = wb;
      wb = describe(wbase + 32 + lane);
    }
    const int rel = (int)(u - wbase);
    const int32_t row = __shfl_sync(0xffffffffu, wa.row, rel);
    const int32_t info = __shfl_sync(0xffffffffu, wa.info, rel);
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
    }

    // wait for this unit's tile
    if (!mbar_wait_bounded(bar_base + 8 * slot, phase)) { failed = true; break; }

    const uint32_t tile = ring_base + slot * TILE;
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
    if (u + stages < u1) {
      if (lane == 0) fence_proxy_async();
      issue(u + stages, slot);
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
        const int64_t pslot = worker * 2 + (seg_is_workers_first ? 0 : 1);
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
      seg_is_workers_first = false;
    }
  }

  if (failed) {
    // A copy did not arrive in time: record it, then give every copy still in flight a
    // bounded chance to land before this warp's shared memory is released.
    if (lane == 0) atomicOr(p.status, kErrTimeout);
    int64_t issued_end = u + stages < u1 ? u + stages : u1;   // units [u, issued_end) are in flight
    for (int64_t v = u; v < issued_end; ++v) {
      (void)mbar_wait_bounded(bar_base + 8 * slot, phase);
      if (++slot == stages) { slot = 0; phase ^= 1u; }
    }
  }
}

// ---------------------------------------------------------------------------------
// log-sum-exp combine: one block per (sequence, kv head) row
// ---------------------------------------------------------------------------------
struct CombineParams {
  const float* partials;
  const int32_t* cum;
  const int32_t* kv_lens;
  __nv_bfloat16* out;
  float* lse;
  int32_t batch, Hq, Hkv, G, D;
  int32_t max_pages, window;
  int32_t num_workers;
};

__global__ void combine_kernel(CombineParams p) {
  const int row = blockIdx.x;
  const int b = row / p.Hkv, g = row - b * p.Hkv;
  const int D = p.D;
  int32_t n = p.kv_lens[b];
  if (n > p.max_pages * kPage) n = p.max_pages * kPage;
  __nv_bfloat16* ob = p.out + ((int64_t)b * p.Hq + (int64_t)g * p.G) * D;
  if (n <= 0) {   // inactive slot: zeros, lse = -inf
    for (int i = threadIdx.x; i < p.G * D; i += blockDim.x) ob[i] = __float2bfloat16(0.f);
    if (p.lse)
      for (int i = threadIdx.x; i < p.G; i += blockDim.x) p.lse[(int64_t)b * p.Hq + g * p.G + i] = -INFINITY;
    return;
  }
  int32_t first, cnt, lo;
  visible_pages(n, p.window, p.max_pages, first, cnt, lo);
  const int64_t U = (int64_t)p.cum[p.batch] * p.Hkv;
  const int64_t ustart = (int64_t)p.cum[b] * p.Hkv + (int64_t)g * cnt;
  const int64_t uend = ustart + cnt;
  const int64_t wf = worker_of(U, ustart, p.num_workers), wl = worker_of(U, uend - 1, p.num_workers);
  if (wf == wl) return;                       // the row was finished by a single worker
  const int64_t stride = (int64_t)p.G * (D + 2);
  // Walk the row's segments: the worker holding unit u owns [u, min(end of its range, uend)).
  // (Workers with an empty range hold no unit and are never visited.)  A worker's partial is
  // in its slot 0 if the row is the first one it touches, else in slot 1.
  auto slot_at = [&](int64_t u, int64_t& next_u) -> const float* {
    const int64_t w = worker_of(U, u, p.num_workers);
    const int64_t wb = worker_begin(U, w, p.num_workers);
    next_u = worker_begin(U, w + 1, p.num_workers);
    const bool is_first_row = wb >= ustart;
    return p.partials + (w * 2 + (is_first_row ? 0 : 1)) * stride;
  };
  for (int h = 0; h < p.G; ++h) {
    float M = -INFINITY;
    for (int64_t u = ustart, nu; u < uend; u = nu) M = fmaxf(M, slot_at(u, nu)[p.G * D + h]);
    float L = 0.f;
    for (int64_t u = ustart, nu; u < uend; u = nu) {
      const float* s = slot_at(u, nu);
      L += exp2f(s[p.G * D + h] - M) * s[p.G * D + p.G + h];
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
      float acc = 0.f;
      for (int64_t u = ustart, nu; u < uend; u = nu) {
        const float* s = slot_at(u, nu);
        acc += exp2f(s[p.G * D + h] - M) * s[h * D + d];
      }
      ob[h * D + d] = __float2bfloat16_rn(acc * inv);
    }
    if (p.lse && threadIdx.x == 0)
      p.lse[(int64_t)b * p.Hq + g * p.G + h] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
  }
}

}  // namespace opw
