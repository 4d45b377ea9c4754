// Warp-level building blocks of the binary32 SIMT attention kernels.
// A warp owns QW = 4 query rows; inside a chunk of 32 staged key columns, lane j owns column j for the
// logits, and output elements {lane + 32 t} for the value aggregation.
#pragma once
#include "fl_internal.cuh"

constexpr int kQW = 4;        // queries per warp
constexpr int kChunk = 32;    // key columns per staged chunk
constexpr int kAttnWarps = 8;
constexpr int kAttnThreads = kAttnWarps * 32;
constexpr int kQTile = kAttnWarps * kQW;  // 32 queries per CTA

// logits of the warp's 4 queries against the 32 staged keys; q4[x] = (q0[x], q1[x], q2[x], q3[x])
template <int DH>
__device__ __forceinline__ void warp_qk(const float4* __restrict__ q4, const float* __restrict__ k_tile, int lane,
                                        float (&s)[kQW]) {
  const float* kr = k_tile + lane * (DH + 1);
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 16
  for (int x = 0; x < DH; ++x) {
    const float4 q = q4[x];
    const float kv = kr[x];
    a0 = fmaf(q.x, kv, a0);
    a1 = fmaf(q.y, kv, a1);
    a2 = fmaf(q.z, kv, a2);
    a3 = fmaf(q.w, kv, a3);
  }
  s[0] = a0; s[1] = a1; s[2] = a2; s[3] = a3;
}

// acc[qi][t] += sum_j p[j][qi] * V[j][lane + 32 t];  p4[j] = (p of the 4 queries for column j)
template <int DH>
__device__ __forceinline__ void warp_pv(const float4* __restrict__ p4, const float* __restrict__ v_tile, int lane,
                                        float (&acc)[kQW][DH / 32]) {
#pragma unroll 4
  for (int j = 0; j < kChunk; ++j) {
    const float4 p = p4[j];
    const float* vr = v_tile + j * DH + lane;
#pragma unroll
    for (int t = 0; t < DH / 32; ++t) {
      const float v = vr[32 * t];
      acc[0][t] = fmaf(p.x, v, acc[0][t]);
      acc[1][t] = fmaf(p.y, v, acc[1][t]);
      acc[2][t] = fmaf(p.z, v, acc[2][t]);
      acc[3][t] = fmaf(p.w, v, acc[3][t]);
    }
  }
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T>
__device__ __forceinline__ float to_float(T v);
template <>
__device__ __forceinline__ float to_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_float(float v);
template <>
__device__ __forceinline__ float from_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
