// Skinny projection GEMM of the decode step on the 5th-generation tensor cores (sm_100a).
//
//   C[b, n] = sum_k x[b, k] * W[n, k]          x: [batch, K] bf16, W: [N, K] bf16, fp32 accumulate
//                                               (any batch: blockIdx.z walks over tiles of 256 rows)
//
// A decode step has few rows (the batch) and a large weight matrix that is read once, so the
// kernel is built around streaming W: the WEIGHT rows take the tensor core's M dimension (one
// CTA = 128 weight rows = 128 TMEM lanes), the batch takes its N dimension (16..256 columns of
// fp32 accumulators in TMEM), and K is cut into 64-element blocks (128 bytes = one swizzle row)
// that TMA brings into a shared-memory ring.  One thread issues the copies, one thread issues
// tcgen05.mma (4 per block, K = 16 each) and releases ring slots with tcgen05.commit, and after
// the last block sixteen warps read the accumulators back with tcgen05.ld (four lane quadrants x
// four column groups) -- the epilogue is a chain of L2 round trips, so it wants many threads.
//
// With N/128 tiles alone a 6144 x 4096 projection would occupy 48 of 148 SMs, too few to pull
// the weights at HBM speed, so K is also split over `ksplit` CTAs per tile, and the partial tiles
// have to meet.  Three back ends, chosen by the host:
//   * cluster: the ksplit CTAs of a tile -- or, where a head spans two weight tiles (D = 256), the 2 * ksplit
//     CTAs of both -- are one thread-block cluster (1 or 2, ksplit, 1).  They are resident together by
//     construction, meet at the cluster's hardware barrier, and each adds up and finishes its own slice of the
//     batch columns, reading the other members' tiles from their shared memory.  Used whenever the device
//     holds all clusters of the launch at once (a cluster needs its SMs in one GPC).
//   * cooperative: the whole grid is resident (cooperative launch); the CTAs of a tile meet at a counter in
//     global memory and share the back end the same way, the partial tiles passing through the workspace.
//     Used at large batches where the clusters do not fit.
//   * last CTA: with no residency guarantee nobody may wait; every CTA writes its partial tile to the
//     workspace and the last one of a tile to arrive (an atomic ticket) reduces and finishes all of it.
// In all three the partial tiles are added in split order: deterministic.
//
// Epilogues: plain (bf16 C[b, n]) and rotary (the QKV projection of the attention module: pairs
// (d, d + D/2) of the q and k heads are rotated, still as fp32 accumulators, by angles that the
// warps idle in the main loop compute meanwhile, v is passed through, everything is rounded to
// bf16 once, and the three outputs go to separate [batch, heads, D] buffers).  The rotary form needs both elements of a pair in one
// 128-row tile: D in {64, 128}.
//
// Every wait is bounded by the global timer (kGemmWaitNs); a wait that runs out records
// kGemmErrTimeout in the status word, the CTA skips its epilogue, frees its TMEM and exits.
#pragma once

#include <cstdint>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace opw_afd {

constexpr int kTileM = 128;               // weight rows per CTA
constexpr int kBlockK = 64;               // bf16 elements per k-block (128 bytes)
constexpr int kGemmThreads = 512;        // 16 warps: 2 single-thread roles in the main loop, all of them in the epilogue
constexpr int kColPhases = kGemmThreads / 64;   // epilogue: thread = 2 adjacent rows x every kColPhases-th batch column
constexpr int kMaxStages = 12;
constexpr int kMaxSplit = 4;
constexpr uint32_t kTileABytes = kTileM * kBlockK * 2;
constexpr uint64_t kGemmWaitNs = 200ull * 1000 * 1000;
constexpr uint32_t kGemmErrTimeout = 2u;  // same bit as the attention kernels' timeout

constexpr int kMaxNb = 256;               // batch rows per CTA (the MMA's N); more rows: blockIdx.z
constexpr int kChunkCols = 128;           // batch columns the epilogue of a two-tile group handles at a time

struct GemmParams {
  int n_out, k, batch;
  int nb;                 // MMA N of a full batch tile: min(batch, 256) rounded up to a multiple of 16
  int group;              // weight tiles that share a ticket and an epilogue: 1, or 2 (rotary at D = 256)
  int coop;               // the launch is cooperative (every CTA resident): the CTAs of a ticket group share the back end
  int cluster;            // the ksplit * group CTAs of a ticket group form a thread-block cluster (group, ksplit, 1): they
                          // exchange their partial tiles through distributed shared memory
  const float2* angles_g; // mode 1: [batch, D/2] (cos, sin) in global memory, or null: computed here in shared memory
  int stages;
  int ksplit;
  int mode;               // 0: plain, 1: rotary + split into q / k / v
  __nv_bfloat16* out;     // mode 0: [batch, n_out]
  __nv_bfloat16* q;       // mode 1: [batch, Hq, D]
  __nv_bfloat16* kn;      //         [batch, Hkv, D]
  __nv_bfloat16* vn;      //         [batch, Hkv, D]
  const int32_t* positions;  // mode 1: [batch]; the rotation angle of pair i is position * theta^(-2i/D)
  double log_theta;
  int Hq, Hkv, D;
  float* partials;        // [tiles, ksplit, nb, 128] fp32, used when ksplit > 1
  uint32_t* tickets;      // [ticket groups][2] {arrived, departed}, zero between launches
  uint32_t* status;
  unsigned long long* trace;   // optional: [grid][8] global-timer stamps of each CTA's phases (see kTrace*)
};

// Trace record of one CTA: begin, ring and TMEM ready, accumulator complete, accumulator in shared
// memory, partial tile published (ticket taken), partial tiles reduced, end; then the SM id.
constexpr int kTraceWords = 8;
constexpr int kTraceMaxCtas = 1024;
__device__ __forceinline__ void g_stamp(const GemmParams& p, int cta, int slot) {
  if (p.trace && cta < kTraceMaxCtas && threadIdx.x == 0) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    p.trace[(size_t)cta * kTraceWords + slot] = t;
  }
}

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t g_smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void g_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void g_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t g_mbar_try_wait(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool g_mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (g_mbar_try_wait(bar, parity)) return true;
  uint64_t t0, t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (g_mbar_try_wait(bar, parity)) return true;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    if (t - t0 > kGemmWaitNs) return false;
  }
}
// 2-D tiled TMA load (no multicast): box of the tensor map at element coordinates (c0 = k, c1 = row).
__device__ __forceinline__ void g_tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void g_tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void g_tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void g_tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void g_tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 in, fp32 out, M = 128, N from the instruction descriptor, K = 16.
__device__ __forceinline__ void g_umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void g_umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void g_tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Thread-block cluster: the shared-memory address of the same variable in the CTA of rank `rank`, loads from
// it, and the cluster's hardware barrier (split in two halves; it does not spin, every CTA of a cluster is
// resident with the others).
__device__ __forceinline__ uint32_t g_mapa(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 g_ld_cluster_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t g_ld_cluster_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void g_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void g_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, stored as TMA's
// 128-byte swizzle leaves them: 8-row groups 1024 bytes apart (stride byte offset), leading
// byte offset unused (1), descriptor version 1, layout type 2 = 128-byte swizzle.  Addresses and
// offsets are in 16-byte units.
__device__ __forceinline__ uint64_t g_smem_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9
// and 10-12 = 1), both K-major (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28.
__device__ __forceinline__ uint32_t g_instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

// dst[i] = sum over the ksplit partial tiles of part[s * split_stride + i], in split order (so the result does
// not depend on which CTA came last); if own >= 0 the partial of that split is read from dst itself (it is
// still in shared memory there).  Every other split's values are requested at once: the reduction would
// otherwise be a chain of L2 round trips.  A function of its own so that it is compiled once.
__device__ __noinline__ void gemm_reduce_partials(const float4* part, float4* dst, int n4, int ksplit, int own, size_t split_stride) {
  constexpr int R = 2;
  const int step = R * kGemmThreads;
  auto fetch = [&](float4 (&v)[R][kMaxSplit], int ib) {
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int sp = 0; sp < kMaxSplit; ++sp) {
        const int i = ib + r * kGemmThreads;
        if (i < n4 && sp < ksplit && sp != own) v[r][sp] = __ldcg(part + sp * split_stride + i);
      }
  };
  auto sum = [&](const float4 (&v)[R][kMaxSplit], int ib) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int i = ib + r * kGemmThreads;
      if (i >= n4) break;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int sp = 0; sp < kMaxSplit; ++sp)
        if (sp < ksplit) {
          const float4 t = sp == own ? dst[i] : v[r][sp];
          acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
      dst[i] = acc;
    }
  };
  // two buffers: the loads of the next pair of rows are in flight while this pair is summed
  float4 va[R][kMaxSplit], vb[R][kMaxSplit];
  int ib = threadIdx.x;
  if (ib < n4) fetch(va, ib);
  for (; ib < n4; ib += 2 * step) {
    if (ib + step < n4) fetch(vb, ib + step);
    sum(va, ib);
    if (ib + 2 * step < n4) fetch(va, ib + 2 * step);
    if (ib + step < n4) sum(vb, ib + step);
  }
}

// (cos, sin) of position * theta^(-2i/D) for every sequence b and pair i < D/2, in double (a float angle is
// off by 1e-7 * position radians), stored as float2 [batch, D/2].  One block per sequence.
__global__ void rope_table_kernel(const int32_t* __restrict__ positions, float2* __restrict__ table, int D, double log_theta) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int b = blockIdx.x, half = D >> 1;
  int32_t pos = positions[b];
  if (pos < 0) pos = 0;                              // inactive row: any finite value, the row is never appended
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the table may still be read by an earlier kernel of the stream
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    double sn, cn;
    sincos((double)pos * exp(-2.0 * i / D * log_theta), &sn, &cn);
    table[(size_t)b * half + i] = make_float2((float)cn, (float)sn);
  }
}

// grid = (ceil(n_out / 128), ksplit, ceil(batch / 256)), 512 threads, 1 CTA per SM.
// Dynamic shared memory: 1024 (alignment slack) + stages * (16384 + nb * 128) bytes, then in mode 1 without a
// global angle table the table itself, batch * D/2 (cos, sin) pairs of 8 bytes and D/2 doubles.
__global__ void __launch_bounds__(kGemmThreads, 1)
skinny_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const GemmParams p) {
  extern __shared__ unsigned char g_smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int s_fail;
  __shared__ int s_last;
  __shared__ volatile uint32_t s_flags[kMaxSplit];           // written by the other CTAs of a cluster: their accumulators are good

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, split = blockIdx.y;
  const int b_off = blockIdx.z * kMaxNb;                     // first batch row of this CTA's batch tile
  const int batch_here = p.batch - b_off < kMaxNb ? p.batch - b_off : kMaxNb;
  const int nb = p.nb;                                       // MMA N (rows beyond the batch arrive as zeros)
  const uint32_t raw = g_smem_u32(g_smem_raw);
  const uint32_t ring = (raw + 1023u) & ~1023u;             // swizzled tiles need 1024-byte alignment
  float* stage_f = reinterpret_cast<float*>(g_smem_raw + (ring - raw));   // the ring again, after the last MMA: [col][128] fp32
  const uint32_t stage_bytes = kTileABytes + (uint32_t)nb * 128u;
  const int half = p.D >> 1;
  float2* angles_s = reinterpret_cast<float2*>(g_smem_raw + (ring - raw) + (size_t)p.stages * stage_bytes);   // [batch_here][D/2]
  const float2* angles = p.angles_g ? p.angles_g + (size_t)b_off * half : angles_s;   // indexed by the local row
  const int kblocks = (p.k + kBlockK - 1) / kBlockK;
  const int kb0 = (int)((int64_t)kblocks * split / p.ksplit);
  const int kb1 = (int)((int64_t)kblocks * (split + 1) / p.ksplit);
  const int nkb = kb1 - kb0;
  uint32_t ncols = 32;
  while (ncols < (uint32_t)nb) ncols <<= 1;
  const int cta = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
  g_stamp(p, cta, 0);
  if (p.trace && cta < kTraceMaxCtas && tid == 0) {
    uint32_t sm;
    asm volatile("mov.u32 %0, %smid;" : "=r"(sm));
    p.trace[(size_t)cta * kTraceWords + 7] = sm;
  }

  // Slot i % stages takes the weight tile and the activation tile of k-block i; both count on one barrier.
  auto issue_w = [&](int i) {
    const int s = i % p.stages;
    const uint32_t fb = g_smem_u32(&full_bar[s]);
    g_mbar_expect_tx(fb, stage_bytes);
    g_tma_load_2d(ring + (uint32_t)s * stage_bytes, &map_w, (kb0 + i) * kBlockK, tile * kTileM, fb);
  };
  auto issue_x = [&](int i) {
    const int s = i % p.stages;
    g_tma_load_2d(ring + (uint32_t)s * stage_bytes + kTileABytes, &map_x, (kb0 + i) * kBlockK, b_off, g_smem_u32(&full_bar[s]));
  };

  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    for (int s = 0; s < p.stages; ++s) {
      g_mbar_init(g_smem_u32(&full_bar[s]), 1);
      g_mbar_init(g_smem_u32(&empty_bar[s]), 1);
    }
    g_mbar_init(g_smem_u32(&acc_bar), 1);
    s_fail = 0;
    s_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // The weights depend on nothing earlier in the stream and the first round of the ring needs no
    // free-slot wait: their stream starts before the TMEM allocation and, under programmatic
    // dependent launch, while the previous kernel is still draining.
    for (int i = 0; i < nkb && i < p.stages; ++i) issue_w(i);
  }
  if (warp == 1) g_tmem_alloc(g_smem_u32(&tmem_slot), ncols);
  g_tc_fence_before();
  __syncthreads();
  g_tc_fence_after();
  const uint32_t tmem_d = tmem_slot;
  // Programmatic dependent launch (no-ops without the launch attribute): the next kernel may queue
  // up now; from here on this one touches what earlier kernels wrote (activations, positions, the
  // angle table, partial tiles, tickets), so it waits for them to be complete.  Every thread of
  // every CTA passes this wait.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  g_stamp(p, cta, 1);

  if (tid == 0) {
    // ---- producer: one TMA load of the weight tile and one of the activation tile per k-block ----
    for (int i = 0; i < nkb && i < p.stages; ++i) issue_x(i);
    for (int i = p.stages; i < nkb; ++i) {
      if (!g_mbar_wait_bounded(g_smem_u32(&empty_bar[i % p.stages]), (uint32_t)((i / p.stages) - 1) & 1u)) {
        s_fail = 1;
        atomicOr(p.status, kGemmErrTimeout);
        break;
      }
      issue_w(i);
      issue_x(i);
    }
  } else if (tid == 32) {
    // ---- MMA issuer ----
    const uint32_t idesc = g_instr_desc(nb);
    bool ok = true;
    for (int i = 0; i < nkb; ++i) {
      const int s = i % p.stages;
      if (!g_mbar_wait_bounded(g_smem_u32(&full_bar[s]), (uint32_t)(i / p.stages) & 1u)) {
        s_fail = 1;
        atomicOr(p.status, kGemmErrTimeout);
        ok = false;
        break;
      }
      g_tc_fence_after();
      const uint32_t a = ring + (uint32_t)s * stage_bytes;
      const uint64_t adesc = g_smem_desc(a), bdesc = g_smem_desc(a + kTileABytes);
#pragma unroll
      for (int k4 = 0; k4 < kBlockK / 16; ++k4)         // 32 bytes along K per MMA: +2 in 16-byte units
        g_umma_bf16(tmem_d, adesc + 2u * k4, bdesc + 2u * k4, idesc, (uint32_t)((i | k4) != 0));
      g_umma_commit(g_smem_u32(&empty_bar[s]));         // the slot is free once these MMAs have read it
    }
    if (ok) g_umma_commit(g_smem_u32(&acc_bar));        // the accumulator is complete
  } else if (tid >= 64 && p.mode == 1 && p.angles_g == nullptr && (tile * kTileM) / p.D < p.Hq + p.Hkv) {
    // ---- warps 2..15, idle in the main loop: the (cos, sin) table of this batch tile, in double ----
    const int t = tid - 64;
    double* inv_freq = reinterpret_cast<double*>(angles_s + (size_t)batch_here * half);
    for (int i = t; i < half; i += kGemmThreads - 64) inv_freq[i] = exp(-2.0 * i / p.D * p.log_theta);
    asm volatile("bar.sync 1, %0;" ::"n"(kGemmThreads - 64) : "memory");
    for (int idx = t; idx < batch_here * half; idx += kGemmThreads - 64) {
      const int b = idx / half, i = idx - b * half;
      int32_t pos = __ldg(p.positions + b_off + b);
      if (pos < 0) pos = 0;                             // inactive row: any finite value, the row is never appended
      double sn, cn;
      sincos((double)pos * inv_freq[i], &sn, &cn);
      angles_s[idx] = make_float2((float)cn, (float)sn);
    }
  }
  __syncwarp();

  // ---- accumulators: TMEM -> registers -> shared memory, transposed to [column b][row] ----
  // warp = (lane quadrant it may read, column group): quadrant = warp % 4, columns 16 * (warp / 4) + 64 j
  const bool arrived = g_mbar_wait_bounded(g_smem_u32(&acc_bar), 0);
  if (!arrived && tid == 0) atomicOr(p.status, kGemmErrTimeout);
  const bool good = __syncthreads_and(arrived ? 1 : 0) && s_fail == 0;
  g_stamp(p, cta, 2);
  if (good) {
    g_tc_fence_after();
    const int quad = warp & 3, row = quad * 32 + lane;
    for (int c0 = 16 * (warp >> 2); c0 < nb; c0 += 64) {
      uint32_t r[16];
      g_tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, r);
#pragma unroll
      for (int j = 0; j < 16; ++j) stage_f[(c0 + j) * kTileM + row] = __uint_as_float(r[j]);
    }
    g_tc_fence_before();
  }
  __syncthreads();
  if (warp == 1) g_tmem_dealloc(tmem_d, ncols);
  g_stamp(p, cta, 3);

  const bool shared_epilogue = p.ksplit > 1 || p.group > 1;
  const int ptile = blockIdx.z * gridDim.x + tile;                       // tile index over all batch tiles
  const size_t split_floats = (size_t)nb * kTileM;                        // one CTA's partial tile

  // Epilogue of weight tile T over the local batch columns [cb, ce): `val` holds the tile's sums as
  // [column - cb][128 rows], `par` the sums of the tile that holds the rotation partners (val itself
  // when a head fits one tile).  Thread = two adjacent weight rows, every kColPhases-th column.
  auto epilogue = [&](int T, const float* val, const float* par, int cb, int ce) {
    const int r0 = 2 * (tid & 63), n0 = T * kTileM + r0;
    if (n0 >= p.n_out) return;
    if (p.mode == 0) {
      for (int b = cb + (tid >> 6); b < ce; b += kColPhases) {
        const float2 v = *reinterpret_cast<const float2*>(&val[(b - cb) * kTileM + r0]);
        *reinterpret_cast<__nv_bfloat162*>(&p.out[(size_t)(b_off + b) * p.n_out + n0]) = __floats2bfloat162_rn(v.x, v.y);
      }
      return;
    }
    const int head = n0 / p.D, d = n0 - head * p.D;
    int hh, H;
    __nv_bfloat16* base;
    if (head < p.Hq) { base = p.q; hh = head; H = p.Hq; }
    else if (head < p.Hq + p.Hkv) { base = p.kn; hh = head - p.Hq; H = p.Hkv; }
    else { base = p.vn; hh = head - p.Hq - p.Hkv; H = p.Hkv; }
    const bool rotate = head < p.Hq + p.Hkv;
    const int pr = half < kTileM ? (r0 ^ half) : r0;          // the partner's row in `par`
    const int i0 = d & (half - 1);
    const float sgn = d < half ? -1.f : 1.f;      // out_i = x_i c - x_{i+half} s ; out_{i+half} = x_{i+half} c + x_i s
    const float4* angles4 = reinterpret_cast<const float4*>(angles);   // (cos, sin) of pairs i0 and i0 + 1: 16 bytes
    // four columns at a time: the angle table may sit in global memory, and four independent loads in
    // flight per thread keep the loop from being a chain of L2 round trips
    constexpr int UN = 4;
    for (int b = cb + (tid >> 6); b < ce; b += UN * kColPhases) {
      float4 cs[UN];
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int bu = b + u * kColPhases;
        cs[u] = (rotate && bu < ce) ? angles4[(bu * half + i0) >> 1] : make_float4(1.f, 0.f, 1.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int bu = b + u * kColPhases;
        if (bu >= ce) break;
        float2 v = *reinterpret_cast<const float2*>(&val[(bu - cb) * kTileM + r0]);
        if (rotate) {                            // on the fp32 accumulators: one rounding, at the bf16 output
          const float2 w = *reinterpret_cast<const float2*>(&par[(bu - cb) * kTileM + pr]);
          v = make_float2(v.x * cs[u].x + sgn * (w.x * cs[u].y), v.y * cs[u].z + sgn * (w.y * cs[u].w));
        }
        *reinterpret_cast<__nv_bfloat162*>(&base[((size_t)(b_off + bu) * H + hh) * p.D + d]) = __floats2bfloat162_rn(v.x, v.y);
      }
    }
  };

  // Sum of the ksplit partial tiles of weight tile index `pt` (over all batch tiles) for the local columns
  // [cb, ce), in split order, into dst[column - cb][128].  `own`: this CTA's own partial of that tile is still
  // in shared memory at `dst` and is taken from there.
  auto reduce_tile = [&](int pt, float* dst, int cb, int ce, bool own) {
    const float4* part = reinterpret_cast<const float4*>(p.partials + (size_t)pt * p.ksplit * split_floats) + (size_t)cb * kTileM / 4;
    gemm_reduce_partials(part, reinterpret_cast<float4*>(dst), (ce - cb) * kTileM / 4, p.ksplit, own ? split : -1, split_floats / 4);
  };

  if (p.cluster) {
    // ---- hand-off inside a thread-block cluster: the ksplit CTAs of this weight tile run at the same time on
    // SMs of one GPC (a cluster is resident as a whole), meet at the cluster's hardware barrier instead of
    // counting arrivals in global memory, and read each other's shared memory.  Member r takes a slice of the
    // batch columns, adds that slice of all members' tiles in split order and finishes it.  Every CTA passes
    // both barriers whatever happened to it (its waits are bounded), so no member is left waiting; a member that
    // failed makes all skip the epilogue.
    // Measured alternatives: members sending their accumulators into the owner's shared memory with remote
    // stores, and members exchanging the slices through the workspace in L2 with only the barrier taken from the
    // cluster, were both slower (the cluster's network moves some 20 GB/s per SM either way; a write to L2 and a
    // read back are two round trips where this is one). ----
    // A head that spans two weight tiles (group = 2) makes the cluster (2, ksplit, 1): the 2 * ksplit CTAs of both
    // tiles, each owning a slice of the columns for which it sums both tiles (its own in place, the other into a
    // second buffer) and rotates each against the other.
    const int ks = p.ksplit, members = ks * p.group;
    const int tl = p.group == 2 ? (tile & 1) : 0;                         // this CTA's tile inside the group
    const int rank = tl * ks + split;                                     // which slice it owns
    auto cta_of = [&](int tl_, int sp_) -> uint32_t { return p.group == 2 ? (uint32_t)(tl_ + 2 * sp_) : (uint32_t)sp_; };
    uint32_t my_cta;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(my_cta));
    if (tid == 0) s_flags[0] = (good && my_cta == cta_of(tl, split)) ? 1u : 0u;   // (a rank order other than x-major: treated as a failure)
    g_cluster_arrive();
    g_cluster_wait();
    g_stamp(p, cta, 4);
    const int cb = (int)((int64_t)batch_here * rank / members), ce = (int)((int64_t)batch_here * (rank + 1) / members);
    float* mine = stage_f + (size_t)cb * kTileM;
    float* other = stage_f + split_floats;                                // the head's other tile, this slice (group = 2)
    // The members' flags and the values are requested together: one round trip through the cluster's network,
    // not one per member.  The sums are formed whatever the flags say (a failed member's tile is just numbers);
    // only the epilogue depends on them.
    uint32_t flags_and = 1u;
    const uint32_t flag_local = g_smem_u32(const_cast<uint32_t*>(&s_flags[0]));
    {
      uint32_t flag[2 * kMaxSplit];
#pragma unroll
      for (int m = 0; m < 2 * kMaxSplit; ++m) flag[m] = m < members ? g_ld_cluster_u32(g_mapa(flag_local, (uint32_t)m)) : 1u;
      // dst[i] = sum over the splits of tile `tls` of their values at the slice, in split order; `own`: this CTA's
      // own partial is one of them and is read from `src_local` (which may be dst itself)
      const int n4 = (ce - cb) * kTileM / 4;
      const uint32_t slice_local = g_smem_u32(mine);
      auto pull_sum = [&](float4* dst, int tls, bool own) {
        uint32_t remote[kMaxSplit];
#pragma unroll
        for (int sp = 0; sp < kMaxSplit; ++sp) remote[sp] = sp < ks ? g_mapa(slice_local, cta_of(tls, sp)) : 0u;
        constexpr int R = 2;
        for (int ib = tid; ib < n4; ib += R * kGemmThreads) {
          float4 v[R][kMaxSplit];
#pragma unroll
          for (int r = 0; r < R; ++r)
#pragma unroll
            for (int sp = 0; sp < kMaxSplit; ++sp) {
              const int i = ib + r * kGemmThreads;
              if (i < n4 && sp < ks && !(own && sp == split)) v[r][sp] = g_ld_cluster_f4(remote[sp] + 16u * (uint32_t)i);
            }
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const int i = ib + r * kGemmThreads;
            if (i >= n4) break;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int sp = 0; sp < kMaxSplit; ++sp)
              if (sp < ks) {
                const float4 t = (own && sp == split) ? reinterpret_cast<const float4*>(mine)[i] : v[r][sp];
                acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
              }
            dst[i] = acc;
          }
        }
      };
      pull_sum(reinterpret_cast<float4*>(mine), tl, true);
      if (p.group == 2) pull_sum(reinterpret_cast<float4*>(other), tl ^ 1, false);
#pragma unroll
      for (int m = 0; m < 2 * kMaxSplit; ++m) flags_and &= flag[m];
    }
    const bool all_good = flags_and != 0;
    __syncthreads();
    g_cluster_arrive();                         // this CTA no longer reads the others' shared memory
    g_stamp(p, cta, 5);
    if (all_good && ce > cb) {
      if (p.group == 1) {
        epilogue(tile, mine, mine, cb, ce);
      } else {
        epilogue(tile, mine, other, cb, ce);
        epilogue(tile ^ 1, other, mine, cb, ce);
      }
    }
    g_cluster_wait();                           // and leaves only when nobody reads its own any more
    g_stamp(p, cta, 6);
    return;
  }

  if (!shared_epilogue) {                     // one CTA holds the whole sum of its tile
    if (good) epilogue(tile, stage_f, stage_f, 0, batch_here);
    g_stamp(p, cta, 6);
    return;
  }

  // ---- hand-off through global memory: every CTA publishes its partial tile ----
  // A ticket group is the ksplit CTAs of one weight tile, or of the two tiles of a head (group = 2).
  // Ordering: every thread's partial stores happen before the CTA barrier, thread 0's arrival is an
  // acq_rel atomic at gpu scope after it (release is cumulative over the barrier), and readers read
  // only after a barrier behind their own acquire of the full count.
  {
    const int n4 = batch_here * kTileM / 4;
    float4* part = reinterpret_cast<float4*>(p.partials + ((size_t)ptile * p.ksplit + split) * split_floats);
    if (good)
      for (int i = tid; i < n4; i += kGemmThreads) part[i] = reinterpret_cast<const float4*>(stage_f)[i];
  }
  __syncthreads();
  const int members = p.ksplit * p.group;                                 // CTAs of this ticket group
  uint32_t* tk = p.tickets + 2 * (ptile / p.group);                       // {arrived, departed}, zero between launches
  const int t0 = tile - tile % p.group;                                   // first tile of the group

  if (p.coop) {
    // ---- every CTA of the group takes a slice of the batch columns (the launch is cooperative: all CTAs are
    // resident, so the wait below ends when the slowest member has published; it is bounded all the same) ----
    if (tid == 0) {
      uint32_t seen;
      asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(seen) : "l"(tk) : "memory");
      ++seen;
      uint64_t t_start, t_now;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_start));
      while (seen < (uint32_t)members) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(tk) : "memory");
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_now));
        if (t_now - t_start > kGemmWaitNs) break;
      }
      if (seen < (uint32_t)members) {
        s_fail = 1;
        atomicOr(p.status, kGemmErrTimeout);
      }
    }
    __syncthreads();
    g_stamp(p, cta, 4);
    if (s_fail != 0 || !good) {                 // recorded; the host clears the counters when it polls the error
      g_stamp(p, cta, 6);
      return;
    }
    const int rank = (tile - t0) * p.ksplit + split;
    const int cb = (int)((int64_t)batch_here * rank / members), ce = (int)((int64_t)batch_here * (rank + 1) / members);
    if (ce > cb) {
      float* mine = stage_f + (size_t)cb * kTileM;                        // this tile's sums, in place over the own partial
      reduce_tile(ptile, mine, cb, ce, true);
      float* other = stage_f + split_floats;                              // the head's other tile (group = 2)
      if (p.group == 2) reduce_tile(blockIdx.z * gridDim.x + (tile ^ 1), other, cb, ce, false);
      __syncthreads();
      g_stamp(p, cta, 5);
      if (p.group == 1) {
        epilogue(tile, mine, mine, cb, ce);
      } else {
        epilogue(tile, mine, other, cb, ce);
        epilogue(tile ^ 1, other, mine, cb, ce);
      }
    }
    __syncthreads();
    if (tid == 0) {                             // the last member to leave puts both counters back to zero
      uint32_t left;
      asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(left) : "l"(tk + 1) : "memory");
      if (left == (uint32_t)members - 1u) { tk[0] = 0; tk[1] = 0; }
    }
    g_stamp(p, cta, 6);
    return;
  }

  // ---- no residency guarantee (more CTAs than SMs): the last CTA of the group to arrive does it all, nobody waits ----
  if (tid == 0) {
    uint32_t prev;                                             // taken on failure too, so the count always completes
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(tk) : "memory");
    s_last = prev == (uint32_t)members - 1u;
    if (s_last) *tk = 0;                                       // ready for the next launch
  }
  __syncthreads();
  g_stamp(p, cta, 4);
  if (!(good && s_last != 0)) {
    g_stamp(p, cta, 6);
    return;
  }
  if (p.group == 1) {
    // Every other split's values are fetched at once (the reduction would otherwise be a chain of
    // L2 round trips); this CTA's own are already in shared memory.  Summed in split order, so the
    // result does not depend on which CTA came last.
    reduce_tile(ptile, stage_f, 0, batch_here, true);
    __syncthreads();
    g_stamp(p, cta, 5);
    epilogue(tile, stage_f, stage_f, 0, batch_here);
  } else {
    // Two tiles of one head: both are reduced from the partial tiles in global memory (this CTA's own
    // included), kChunkCols batch columns at a time so that both fit the ring's shared memory.
    float* buf0 = stage_f;
    float* buf1 = stage_f + (size_t)kChunkCols * kTileM;
    for (int cb = 0; cb < batch_here; cb += kChunkCols) {
      const int ce = cb + kChunkCols < batch_here ? cb + kChunkCols : batch_here;
      __syncthreads();                                         // the previous chunk's epilogue is done with the buffers
      reduce_tile(blockIdx.z * gridDim.x + t0, buf0, cb, ce, false);
      reduce_tile(blockIdx.z * gridDim.x + t0 + 1, buf1, cb, ce, false);
      __syncthreads();
      epilogue(t0, buf0, buf1, cb, ce);
      epilogue(t0 + 1, buf1, buf0, cb, ce);
    }
    g_stamp(p, cta, 5);
  }
  g_stamp(p, cta, 6);
}

}  // namespace opw_afd
