// Decode step of a recurrent-state ("linear attention") layer: the gated delta rule, in place on
// fp32 states.  One thread block per (sequence, value head, 128-column block); thread (cx, r)
// owns eight rows of four adjacent columns of the dk x dv state and keeps them in registers,
// so the state is read once and written once with 16-byte accesses, a warp covering 512
// contiguous bytes of a row; the two dot products per column are finished through shared
// memory in a fixed order.  The
// operator is a read-modify-write stream of the states: 2 * dk * dv * 4 bytes per (b, h), the
// copy-bandwidth roofline applies.
#include <cmath>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "opw_linear_attn.h"

namespace opw_lin {

struct Params {
  float* state;
  const int32_t* slot;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  const float* a;
  const float* beta;
  __nv_bfloat16* out;
  int64_t num_slots;
  int32_t Hk, Hv, dv;
  float scale;
};

constexpr int kRowsPerThread = 8;  // thread (cx, r) owns rows [8r, 8r+8) of columns [4cx, 4cx+4)

template <int DK>
__global__ void __launch_bounds__(32 * (DK / kRowsPerThread), 2) decode_step_kernel(Params p) {
  constexpr int RS = DK / kRowsPerThread;                          // row groups = blockDim.y
  __shared__ float ks[DK], qs[DK];
  __shared__ float4 red[2][RS][32];                                // partial dot products per column group
  // a block covers up to 128 columns of one state; blockIdx.z picks the column block
  const int h = blockIdx.x, b = blockIdx.y, cx = threadIdx.x, r = threadIdx.y;
  const int j = (blockIdx.z * blockDim.x + cx) * 4;                // first of this thread's four columns, < dv
  const int hk = h / (p.Hv / p.Hk);
  const int64_t s = p.slot[b];
  __nv_bfloat16* o = p.out + ((int64_t)b * p.Hv + h) * p.dv;
  if (s < 0 || s >= p.num_slots) {                                // inactive row: output 0, state untouched
    if (r == 0) *reinterpret_cast<uint2*>(o + j) = make_uint2(0u, 0u);
    return;
  }
  const int tid = r * blockDim.x + cx;
  for (int i = tid; i < DK; i += blockDim.x * RS) {
    ks[i] = __bfloat162float(p.k[((int64_t)b * p.Hk + hk) * DK + i]);
    qs[i] = __bfloat162float(p.q[((int64_t)b * p.Hk + hk) * DK + i]);
  }
  const float a = p.a[(int64_t)b * p.Hv + h], beta = p.beta[(int64_t)b * p.Hv + h];
  const uint2 vraw = *reinterpret_cast<const uint2*>(p.v + ((int64_t)b * p.Hv + h) * p.dv + j);
  const float2 v01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vraw.x));
  const float2 v23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vraw.y));
  float* S = p.state + (((int64_t)s * p.Hv + h) * DK + (int64_t)r * kRowsPerThread) * p.dv + j;
  const int64_t dv = p.dv;
  float4 col[kRowsPerThread];
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) col[i] = __ldcs(reinterpret_cast<const float4*>(S + i * dv));   // streamed once
  __syncthreads();
  float4 pred = make_float4(0.f, 0.f, 0.f, 0.f);                  // this thread's share of (S1^T k) for its columns
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    const float kk = ks[r * kRowsPerThread + i];
    col[i].x *= a; col[i].y *= a; col[i].z *= a; col[i].w *= a;
    pred.x = fmaf(col[i].x, kk, pred.x); pred.y = fmaf(col[i].y, kk, pred.y);
    pred.z = fmaf(col[i].z, kk, pred.z); pred.w = fmaf(col[i].w, kk, pred.w);
  }
  red[0][r][cx] = pred;
  __syncthreads();
  pred = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int rr = 0; rr < RS; ++rr) {                                // fixed order: every thread gets the same sum
    const float4 t = red[0][rr][cx];
    pred.x += t.x; pred.y += t.y; pred.z += t.z; pred.w += t.w;
  }
  const float4 bu = make_float4(beta * (v01.x - pred.x), beta * (v01.y - pred.y), beta * (v23.x - pred.z),
                                beta * (v23.y - pred.w));
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);                   // this thread's share of (S'^T q)
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    const float kk = ks[r * kRowsPerThread + i], qq = qs[r * kRowsPerThread + i];
    col[i].x = fmaf(kk, bu.x, col[i].x); col[i].y = fmaf(kk, bu.y, col[i].y);
    col[i].z = fmaf(kk, bu.z, col[i].z); col[i].w = fmaf(kk, bu.w, col[i].w);
    acc.x = fmaf(col[i].x, qq, acc.x); acc.y = fmaf(col[i].y, qq, acc.y);
    acc.z = fmaf(col[i].z, qq, acc.z); acc.w = fmaf(col[i].w, qq, acc.w);
    __stcs(reinterpret_cast<float4*>(S + i * dv), col[i]);
  }
  red[1][r][cx] = acc;
  __syncthreads();
  if (r == 0) {
    acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int rr = 0; rr < RS; ++rr) {
      const float4 t = red[1][rr][cx];
      acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
    }
    __nv_bfloat162 o01 = __floats2bfloat162_rn(acc.x * p.scale, acc.y * p.scale);
    __nv_bfloat162 o23 = __floats2bfloat162_rn(acc.z * p.scale, acc.w * p.scale);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&o01);
    packed.y = *reinterpret_cast<uint32_t*>(&o23);
    *reinterpret_cast<uint2*>(o + j) = packed;
  }
}

}  // namespace opw_lin

extern "C" size_t opw_linear_attn_state_bytes(int32_t Hv, int32_t dk, int32_t dv, int64_t num_slots) {
  if (Hv < 1 || dk < 1 || dv < 1 || num_slots < 0) return 0;
  return (size_t)num_slots * Hv * dk * dv * 4;
}

extern "C" opw_status_t opw_linear_attn_decode_step(int32_t batch, int32_t Hk, int32_t Hv, int32_t dk, int32_t dv,
                                                    float* state, int64_t num_slots, const int32_t* slot, const void* q,
                                                    const void* k, const void* v, const float* a, const float* beta,
                                                    float scale, void* out, void* cuda_stream) {
  if (batch < 0 || Hk < 1 || Hv < 1 || Hv % Hk != 0 || num_slots < 1) return OPW_ERR_INVALID_ARG;
  if (!state || !slot || !q || !k || !v || !a || !beta || !out) return OPW_ERR_INVALID_ARG;
  if ((uintptr_t)state % 16 || ((uintptr_t)q | (uintptr_t)k) % 2 || ((uintptr_t)v | (uintptr_t)out) % 8 ||
      ((uintptr_t)a | (uintptr_t)beta | (uintptr_t)slot) % 4)
    return OPW_ERR_INVALID_ARG;
  if (!(scale >= 0.f) || !std::isfinite(scale)) return OPW_ERR_INVALID_ARG;
  if ((dk != 64 && dk != 128) || (dv != 64 && dv != 128 && dv != 256)) return OPW_ERR_UNSUPPORTED;
  if (batch > 65535) return OPW_ERR_CAPACITY;
  if (batch == 0) return OPW_OK;
  opw_lin::Params p;
  p.state = state;
  p.slot = slot;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.v = static_cast<const __nv_bfloat16*>(v);
  p.a = a;
  p.beta = beta;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.num_slots = num_slots;
  p.Hk = Hk;
  p.Hv = Hv;
  p.dv = dv;
  p.scale = scale > 0.f ? scale : (float)(1.0 / std::sqrt((double)dk));
  const int cols = dv < 128 ? dv : 128;                            // columns per block, four per thread
  const dim3 grid(Hv, batch, dv / cols), block(cols / 4, dk / opw_lin::kRowsPerThread);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (dk == 64) opw_lin::decode_step_kernel<64><<<grid, block, 0, stream>>>(p);
  else opw_lin::decode_step_kernel<128><<<grid, block, 0, stream>>>(p);
  if (cudaGetLastError() != cudaSuccess) return OPW_ERR_CUDA;
  return OPW_OK;
}
