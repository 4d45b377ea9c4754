// Self-test of the tensor-path building blocks (separate library, loaded only by a GPU test):
// S = Q K^T with both operands K-major in 128B-swizzled shared memory (tcgen05.mma SS form), then
// O = bf16(S) V with A read from tensor memory and B = V as an MN-major operand (TS form).
#include <cuda_bf16.h>

#include "../tc_ptx.cuh"

namespace {

constexpr int M = 128, DH = 128, NC = 64;

// stage `rows` rows of 128 bf16 (256 B) from global into two 128B-swizzled slabs [rows x 64 elements]
__device__ void stage_rows(const __nv_bfloat16* g, int rows, uint8_t* tile, int tid, int nthreads) {
  const int slab_bytes = rows * 128;
  for (int it = tid; it < rows * 16; it += nthreads) {
    const int r = it >> 4, ch = it & 15;
    const uint4 v = *reinterpret_cast<const uint4*>(g + (size_t)r * DH + ch * 8);
    *reinterpret_cast<uint4*>(tile + (ch >> 3) * slab_bytes + tc::sw128_offset(r, ch & 7)) = v;
  }
}

__global__ void __launch_bounds__(128) umma_selftest_kernel(const __nv_bfloat16* q, const __nv_bfloat16* k,
                                                            const __nv_bfloat16* v, float* s_out, float* o_out,
                                                            int* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_tile = smem;                  // 2 slabs x 128 rows x 128 B = 32 KB
  uint8_t* k_tile = q_tile + 32768;        // 2 slabs x 64 rows x 128 B  = 16 KB
  uint8_t* v_tile = k_tile + 16384;        // 16 KB
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    tc::mbar_init(&bar[0], 1);
    tc::mbar_init(&bar[1], 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 0) {
    tc::tmem_alloc(&tmem_base_s, 256);
    tc::tmem_relinquish();
  }
  stage_rows(q, M, q_tile, tid, 128);
  stage_rows(k, NC, k_tile, tid, 128);
  stage_rows(v, NC, v_tile, tid, 128);
  tc::fence_proxy_async_smem();
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const uint32_t s_col = 0, o_col = 128;   // S: 64 columns, O: 128 columns
  if (tid == 0) {
    const uint32_t idesc = tc::make_idesc_bf16(M, NC, false);
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
      const uint64_t a = tc::make_desc_sw128(tc::smem_u32(q_tile) + (kk >> 2) * (M * 128) + (kk & 3) * 32, 16, 1024);
      const uint64_t b = tc::make_desc_sw128(tc::smem_u32(k_tile) + (kk >> 2) * (NC * 128) + (kk & 3) * 32, 16, 1024);
      tc::mma_ss(tmem + s_col, a, b, idesc, kk > 0);
    }
    tc::mma_commit(&bar[0]);
  }
  bool ok = tc::mbar_wait(&bar[0], 0, &abort_flag);
  tc::tc_fence_after();
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  uint32_t r[32];
  uint32_t p[32];
  for (int half = 0; half < 2; ++half) {
    tc::tmem_ld32(tmem + lane_base + s_col + half * 32, r);
    tc::tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) s_out[(size_t)tid * NC + half * 32 + i] = __uint_as_float(r[i]);
#pragma unroll
    for (int i = 0; i < 16; ++i) p[half * 16 + i] = tc::pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
  }
  // P (bf16, 32 columns) overwrites the start of the S region
  tc::tmem_st32(tmem + lane_base + s_col, p);
  tc::tmem_wait_st();
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  if (tid == 0) {
    const uint32_t idesc = tc::make_idesc_bf16(M, DH, true);
#pragma unroll
    for (int kk = 0; kk < NC / 16; ++kk) {
      // V tile: rows = key index (K dimension), 2 slabs of 64 head-dim elements (N dimension)
      const uint64_t b = tc::make_desc_sw128(tc::smem_u32(v_tile) + kk * 2048, NC * 128, 1024);
      tc::mma_ts(tmem + o_col, tmem + s_col + kk * 8, b, idesc, kk > 0);
    }
    tc::mma_commit(&bar[1]);
  }
  ok = tc::mbar_wait(&bar[1], 0, &abort_flag) && ok;
  tc::tc_fence_after();
  for (int q4 = 0; q4 < 4; ++q4) {
    tc::tmem_ld32(tmem + lane_base + o_col + q4 * 32, r);
    tc::tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) o_out[(size_t)tid * DH + q4 * 32 + i] = __uint_as_float(r[i]);
  }
  if (!ok && tid == 0) *status = -5;
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 256);
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int fl_selftest_umma(const void* q, const void* k, const void* v,
                                                                        float* s_out, float* o_out, int* status,
                                                                        void* stream) {
  const int smem = 65536 + 1024;
  if (cudaFuncSetAttribute(umma_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return -4;
  umma_selftest_kernel<<<1, 128, smem, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
      s_out, o_out, status);
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}
