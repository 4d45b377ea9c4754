// Micro-benchmark of the tensor pipe as this library drives it (separate self-test library): cycles per
// tcgen05.mma for the operand forms the attention kernels use. One CTA per SM, one issuing thread.
//   mode 0: SS, M128 x N64  x K16  (S = Q Khat^T chunk of 64 columns)
//   mode 1: SS, M128 x N128 x K16
//   mode 2: SS, M128 x N256 x K16
//   mode 3: TS, M128 x N128 x K16, B MN-major (acc += P Vhat)
//   mode 4: one thread, per iteration 16 of mode 0 followed by 8 of mode 3 (one attention chunk, grouped)
//   mode 5: one thread, the same 24 interleaved (SS, SS, TS)
//   mode 6: two threads of different warps: one issues the 16 SS, the other the 8 TS of every iteration
// Modes 4-6 report cycles per iteration (24 MMAs) / 8 so that the driver's "per MMA" column is cycles per 3 MMAs.
#include <cuda_bf16.h>

#include "../tc_ptx.cuh"

namespace {


// `noise` adds work by the CTA's other warps while the MMAs run:
//   1: tensor-memory loads (64 columns per step), 2: 16-byte shared-memory stores, 4: exp2 + pack arithmetic,
//   8: tensor-memory stores (32 columns per step)
__device__ __noinline__ void noise_loop(int noise, uint32_t tmem, uint8_t* smem, volatile int* stop_flag,
                                        long long* cycles_out) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
  float accf = 0.f;
  uint32_t accu = 0;
  for (int it = 0; it < (1 << 22) && !*stop_flag; ++it) {
    if (noise & 1) {
      uint32_t r[32];
      tc::tmem_ld32(tmem + lane_base + 320, r);
      tc::tmem_ld32(tmem + lane_base + 352, r);
      tc::tmem_wait_ld();
      accu ^= r[0] ^ r[31];
    }
    if (noise & 8) {
      uint32_t r[32];
#pragma unroll
      for (int k = 0; k < 32; ++k) r[k] = accu + k;
      tc::tmem_st32(tmem + lane_base + 352, r);
      tc::tmem_wait_st();
    }
    if (noise & 2) {
#pragma unroll
      for (int k = 0; k < 8; ++k)
        *reinterpret_cast<uint4*>(smem + 81920 + ((tid * 16 + k * 2048 + it * 64) & 16383)) = make_uint4(accu, it, k, tid);
    }
    if (noise & 4) {
#pragma unroll
      for (int k = 0; k < 64; ++k) accf += tc::ex2(accf * 1e-3f + (float)k);
      accu ^= tc::pack_bf16(accf, accf * 0.5f);
    }
  }
  if (accu == 0x12345u && accf == 1.f) cycles_out[blockIdx.x] = 1;
}

__global__ void __launch_bounds__(320) mma_rate_kernel(int mode, int noise, int iters, long long* cycles_out) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar;
  __shared__ uint64_t bar2;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ volatile int stop_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) stop_flag = 0;
  for (int i = tid; i < 96 * 1024 / 16; i += blockDim.x) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u);
  if (tid == 0) { tc::mbar_init(&bar, 1); tc::mbar_init(&bar2, 1); abort_flag = 0; tc::fence_barrier_init(); }
  if (warp == 0) { tc::tmem_alloc(&tmem_base_s, 512); tc::tmem_relinquish(); }
  tc::fence_proxy_async_smem();
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  if (mode >= 7) {
    // issue-path experiments: SS N64 MMAs whose B descriptor moves between four ring slots every iteration
    //   7: one thread inside a divergent branch, slot read from shared memory
    //   8: the whole warp runs the loop, the MMA is predicated on lane 0, slot read from shared memory
    //   9: as 8, slot derived from the loop counter
    //  10: as 7, slot derived from the loop counter
    __shared__ volatile int slot_tab[4];
    if (tid < 4) slot_tab[tid] = tid;
    __syncthreads();
    if (warp == 0) {
      const uint32_t idesc = tc::make_idesc_bf16(128, 64, false);
      const uint64_t a_desc = tc::make_desc_sw128(tc::smem_u32(smem), 16, 1024);
      const uint64_t b_desc = tc::make_desc_sw128(tc::smem_u32(smem) + 32768, 16, 1024);
      const uint32_t hi = (uint32_t)(a_desc >> 32), a_lo = (uint32_t)a_desc, b_lo0 = (uint32_t)b_desc;
      const long long t0 = clock64();
      if (mode == 7 || mode == 10) {
        if (tid == 0) {
          for (int it = 0; it < iters; ++it) {
            const int slot = mode == 7 ? slot_tab[it & 3] : (it & 3);
            const uint32_t b_lo = b_lo0 + slot * (16384 >> 4);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              tc::mma_ss_lo<true>(tmem + 256, a_lo + ((((kk >> 2) * (128 * 128) + (kk & 3) * 32)) >> 4), hi,
                                  b_lo + ((((kk >> 2) * (64 * 128) + (kk & 3) * 32)) >> 4), hi, idesc);
          }
          tc::mma_commit(&bar);
        }
      } else {
        const uint32_t issue = tid == 0 ? 1u : 0u;
        for (int it = 0; it < iters; ++it) {
          const int slot = mode == 8 ? slot_tab[it & 3] : (it & 3);
          const uint32_t b_lo = b_lo0 + slot * (16384 >> 4);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            tc::mma_ss_lo_p<true>(tmem + 256, a_lo + ((((kk >> 2) * (128 * 128) + (kk & 3) * 32)) >> 4), hi,
                                  b_lo + ((((kk >> 2) * (64 * 128) + (kk & 3) * 32)) >> 4), hi, idesc, issue);
        }
        tc::mma_commit_p(&bar, issue);
      }
      if (tid == 0) {
        tc::mbar_wait(&bar, 0, &abort_flag, 1u << 24);
        cycles_out[blockIdx.x] = clock64() - t0;
        stop_flag = 1;
      }
    } else if (noise != 0) {
      noise_loop(noise, tmem, smem, &stop_flag, cycles_out);   // the issuing thread's neighbours on the schedulers
    }
  } else if (mode >= 4) {
    if (tid == 0 || (mode == 6 && tid == 32)) {
      const uint32_t idesc_ss = tc::make_idesc_bf16(128, 64, false), idesc_ts = tc::make_idesc_bf16(128, 128, true);
      const uint64_t a_desc = tc::make_desc_sw128(tc::smem_u32(smem), 16, 1024);
      const uint64_t b_desc = tc::make_desc_sw128(tc::smem_u32(smem) + 32768, 16, 1024);
      const uint64_t v_desc = tc::make_desc_sw128(tc::smem_u32(smem) + 65536, 64 * 128, 1024);
      uint64_t ad[8], bd[8], vd[4];
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        ad[kk] = a_desc + (uint64_t)(((kk >> 2) * (128 * 128) + (kk & 3) * 32) >> 4);
        bd[kk] = b_desc + (uint64_t)(((kk >> 2) * (64 * 128) + (kk & 3) * 32) >> 4);
      }
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) vd[kk] = v_desc + (uint64_t)(kk * (2048 >> 4));
      const uint32_t s_old = tmem + 256, s_new = tmem + 320, p_old = tmem + 384, p_new = tmem + 448;
      const long long t0 = clock64();
      for (int it = 0; it < iters; ++it) {
        if (mode == 4 || (mode == 6 && tid == 0)) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) tc::mma_ss(s_old, ad[kk], bd[kk], idesc_ss, kk > 0);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) tc::mma_ss(s_new, ad[kk], bd[kk], idesc_ss, kk > 0);
        }
        if (mode == 4 || (mode == 6 && tid == 32)) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) tc::mma_ts(tmem, p_old + kk * 8, vd[kk], idesc_ts, true);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) tc::mma_ts(tmem + 128, p_new + kk * 8, vd[kk], idesc_ts, true);
        }
        if (mode == 5) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            tc::mma_ss(s_old, ad[2 * kk], bd[2 * kk], idesc_ss, kk > 0);
            tc::mma_ss(s_old, ad[2 * kk + 1], bd[2 * kk + 1], idesc_ss, true);
            tc::mma_ts(tmem, p_old + kk * 8, vd[kk], idesc_ts, true);
          }
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            tc::mma_ss(s_new, ad[2 * kk], bd[2 * kk], idesc_ss, kk > 0);
            tc::mma_ss(s_new, ad[2 * kk + 1], bd[2 * kk + 1], idesc_ss, true);
            tc::mma_ts(tmem + 128, p_new + kk * 8, vd[kk], idesc_ts, true);
          }
        }
      }
      uint64_t* mybar = tid == 0 ? &bar : &bar2;
      tc::mma_commit(mybar);
      tc::mbar_wait(mybar, 0, &abort_flag, 1u << 24);
      const long long t1 = clock64();
      if (tid == 0) { cycles_out[blockIdx.x] = t1 - t0; stop_flag = 1; }
    } else if (warp >= 2 && noise != 0) {
      noise_loop(noise, tmem, smem, &stop_flag, cycles_out);
    }
  } else if (tid == 0) {
    const int n = mode == 0 ? 64 : (mode == 2 ? 256 : 128);
    const uint32_t idesc = tc::make_idesc_bf16(128, n, mode == 3);
    const uint64_t a_desc = tc::make_desc_sw128(tc::smem_u32(smem), 16, 1024);                 // 32 KB A tile
    const uint64_t b_desc = mode == 3 ? tc::make_desc_sw128(tc::smem_u32(smem) + 32768, 64 * 128, 1024)
                                      : tc::make_desc_sw128(tc::smem_u32(smem) + 32768, 16, 1024);
    // descriptors of the 8 K steps are loop invariants: the timed loop holds nothing but the MMAs
    uint64_t ad[8], bd[8];
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      ad[kk] = a_desc + (uint64_t)(((kk >> 2) * (128 * 128) + (kk & 3) * 32) >> 4);
      bd[kk] = mode == 3 ? b_desc + (uint64_t)(kk * (2048 >> 4))
                         : b_desc + (uint64_t)(((kk >> 2) * (n * 128) + (kk & 3) * 32) >> 4);
    }
    const long long t0 = clock64();
    if (mode == 3) {
      for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) tc::mma_ts(tmem + 256, tmem + kk * 8, bd[kk], idesc, true);
      }
    } else {
      for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) tc::mma_ss(tmem + 256, ad[kk], bd[kk], idesc, true);
      }
    }
    tc::mma_commit(&bar);
    tc::mbar_wait(&bar, 0, &abort_flag, 1u << 24);
    const long long t1 = clock64();
    cycles_out[blockIdx.x] = t1 - t0;
    stop_flag = 1;
  } else if (warp > 0 && noise != 0) {
    noise_loop(noise, tmem, smem, &stop_flag, cycles_out);
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int fl_selftest_mma_rate(int mode, int noise, int iters, int n_ctas,
                                                                            long long* cycles_out, void* stream) {
  const int smem = 100 * 1024;
  if (cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return -4;
  mma_rate_kernel<<<n_ctas, mode >= 4 ? 320 : 128, smem, static_cast<cudaStream_t>(stream)>>>(mode, noise, iters, cycles_out);
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}
