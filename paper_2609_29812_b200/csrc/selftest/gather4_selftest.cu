// Self-test of the TMA row gather (tile::gather4) into a 128B-swizzled K-major operand tile, consumed by
// tcgen05.mma: S = Q Kg^T where Kg = 64 gathered rows of a [rows, 128] bf16 matrix (out-of-range rows -> 0).
#include <cuda.h>
#include <cuda_bf16.h>

#include "../tc_ptx.cuh"

namespace {

constexpr int M = 128, DH = 128, NC = 64;

__global__ void __launch_bounds__(128) gather4_selftest_kernel(const __grid_constant__ CUtensorMap tmap,
                                                               const __nv_bfloat16* q, const int* idx, float* s_out,
                                                               int* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_tile = smem;            // 32 KB
  uint8_t* k_tile = q_tile + 32768;  // 16 KB: 2 slabs x 64 rows x 128 B
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ int idx_s[NC];
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    tc::mbar_init(&bar[0], 1);
    tc::mbar_init(&bar[1], 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (tid < NC) idx_s[tid] = idx[tid];
  if (warp == 0) { tc::tmem_alloc(&tmem_base_s, 64); tc::tmem_relinquish(); }
  for (int it = tid; it < M * 16; it += 128) {
    const int r = it >> 4, ch = it & 15;
    *reinterpret_cast<uint4*>(q_tile + (ch >> 3) * (M * 128) + tc::sw128_offset(r, ch & 7)) =
        *reinterpret_cast<const uint4*>(q + (size_t)r * DH + ch * 8);
  }
  tc::fence_proxy_async_smem();
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  if (tid == 0) {
    tc::mbar_arrive_expect_tx(&bar[0], NC * DH * 2);
    for (int slab = 0; slab < 2; ++slab)
      for (int g = 0; g < NC / 4; ++g)
        tc::tma_gather4(k_tile + slab * (NC * 128) + g * 512, &tmap, &bar[0], slab * 64, idx_s[4 * g], idx_s[4 * g + 1],
                        idx_s[4 * g + 2], idx_s[4 * g + 3]);
    bool ok = tc::mbar_wait(&bar[0], 0, &abort_flag);
    tc::tc_fence_after();
    const uint32_t idesc = tc::make_idesc_bf16(M, NC, false);
    const uint64_t a0 = tc::make_desc_sw128(tc::smem_u32(q_tile), 16, 1024);
    const uint64_t b0 = tc::make_desc_sw128(tc::smem_u32(k_tile), 16, 1024);
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk)
      tc::mma_ss(tmem, a0 + (uint64_t)(((kk >> 2) * (M * 128) + (kk & 3) * 32) >> 4),
                 b0 + (uint64_t)(((kk >> 2) * (NC * 128) + (kk & 3) * 32) >> 4), idesc, kk > 0);
    tc::mma_commit(&bar[1]);
    if (!ok) *status = -5;
  }
  const bool ok2 = tc::mbar_wait(&bar[1], 0, &abort_flag);
  tc::tc_fence_after();
  uint32_t r[32];
  for (int hf = 0; hf < 2; ++hf) {
    tc::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + hf * 32, r);
    tc::tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) s_out[(size_t)tid * NC + hf * 32 + i] = __uint_as_float(r[i]);
  }
  if (!ok2 && tid == 0) *status = -5;
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 64);
}

typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

extern "C" __attribute__((visibility("default"))) int fl_selftest_gather4(const void* base, int rows, const void* q,
                                                                           const int* idx, float* s_out, int* status,
                                                                           void* stream) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return -2;
  CUtensorMap tmap;
  const cuuint64_t gdim[2] = {(cuuint64_t)DH, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)DH * 2};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  if (reinterpret_cast<encode_fn>(fn)(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride,
                                      box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return -1;
  const int smem = 49152 + 1024;
  if (cudaFuncSetAttribute(gather4_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return -4;
  gather4_selftest_kernel<<<1, 128, smem, static_cast<cudaStream_t>(stream)>>>(
      tmap, static_cast<const __nv_bfloat16*>(q), idx, s_out, status);
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}
