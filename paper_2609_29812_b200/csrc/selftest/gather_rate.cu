// Micro-benchmark (self-test library): how fast can one SM gather 256-byte rows (one head of one token)
// from an [rows, 2048] bf16 matrix into shared memory?
//   mode 0: TMA tile::gather4, 4 rows x 128 B per copy, issued by `n_warps` warps (32 lanes each)
//   mode 1: cp.async.cg 16 B per lane
//   mode 2: ld.global.nc 16 B per lane + st.shared
// Row indices are pseudo-random. Reports cycles per CTA; bytes moved per CTA = iters * 32 KB.
#include <cuda.h>
#include <cuda_bf16.h>

#include "../tc_ptx.cuh"

namespace {

__device__ __forceinline__ uint32_t hash32(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
  return x;
}

__global__ void __launch_bounds__(512) gather_rate_kernel(const __grid_constant__ CUtensorMap tmap,
                                                          const __nv_bfloat16* base, int rows, int mode, int n_warps,
                                                          int iters, long long* cycles_out) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar[4];
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < 4; ++i) tc::mbar_init(&bar[i], n_warps);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  const long long t0 = clock64();
  if (warp < n_warps) {
    // each iteration fills one 32 KB slot (64 rows x 512 B: K and V pieces); 4 slots in flight
    for (int it = 0; it < iters; ++it) {
      const int slot = it & 3;
      uint8_t* dst = smem + slot * 32768;
      if (mode == 0) {
        if (it >= 4) tc::mbar_wait(&bar[slot], ((it >> 2) - 1) & 1, &abort_flag, 1u << 22);
        const int per_warp = 64 / n_warps;   // gathers per warp (n_warps divides 64)
        if (lane == 0) tc::mbar_arrive_expect_tx(&bar[slot], per_warp * 512);
        __syncwarp();
        for (int g = lane; g < per_warp; g += 32) {
          const int gi = warp * per_warp + g;
          const uint32_t r0 = hash32(blockIdx.x * 7919u + it * 64u + gi * 4u);
          tc::tma_gather4(dst + gi * 512, &tmap, &bar[slot], ((r0 >> 20) & 15) * 128 + (gi & 1) * 64, r0 % rows,
                          hash32(r0) % rows, hash32(r0 + 1) % rows, hash32(r0 + 2) % rows);
        }
      } else {
        // 64 rows x 512 B = 2048 16-byte pieces per slot, spread over n_warps * 32 lanes
        const int nthreads = n_warps * 32;
        if (mode == 1 && it >= 4) tc::cp_async_wait<3>();
        for (int p = tid; p < 2048; p += nthreads) {
          const int row_i = p >> 5, piece = p & 31;
          const uint32_t r0 = hash32(blockIdx.x * 7919u + it * 64u + row_i);
          const __nv_bfloat16* src = base + (size_t)(r0 % rows) * 2048 + ((r0 >> 20) & 3) * 512 + piece * 8;
          if (mode == 1) tc::cp_async16(dst + p * 16, src);
          else *reinterpret_cast<uint4*>(dst + p * 16) = __ldg(reinterpret_cast<const uint4*>(src));
        }
        if (mode == 1) tc::cp_async_commit();
      }
    }
    if (mode == 0) {
      for (int s = 0; s < 4; ++s) {
        const int last = ((iters - 1 - s) >> 2);   // phase index of the slot's last fill
        if (iters - 1 - s >= 0) tc::mbar_wait(&bar[(iters - 1 - s) & 3], last & 1, &abort_flag, 1u << 22);
      }
    } else if (mode == 1) {
      tc::cp_async_wait<0>();
    }
  }
  __syncthreads();
  if (tid == 0) cycles_out[blockIdx.x] = clock64() - t0;
}

typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
}  // namespace

extern "C" __attribute__((visibility("default"))) int fl_selftest_gather_rate(const void* base, int rows, int mode,
                                                                               int n_warps, int iters, int n_ctas,
                                                                               long long* cycles_out, void* stream) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess) return -2;
  CUtensorMap tmap;
  const cuuint64_t gdim[2] = {2048, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {4096};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  if (reinterpret_cast<encode_fn>(fn)(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride,
                                      box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return -1;
  const int smem = 4 * 32768 + 1024;
  if (cudaFuncSetAttribute(gather_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return -4;
  gather_rate_kernel<<<n_ctas, 512, smem, static_cast<cudaStream_t>(stream)>>>(
      tmap, static_cast<const __nv_bfloat16*>(base), rows, mode, n_warps, iters, cycles_out);
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}
