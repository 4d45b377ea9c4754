// Projection of the active rows (Section 4.4 and Appendix G: the selected token rows are gathered so that the
// projections stay regular GEMMs, and only those rows pass through the block): Y[dst(t), :] (+)= X[src(t), :] W^T for
// the n listed rows, as ONE tensor-core GEMM whose A operand is gathered row by row by TMA (no compact copy of the rows
// is made first) and whose epilogue writes, or adds into, rows of a position-indexed matrix (the output projection with
// its residual add scattered back).
//
// Persistent kernel, one CTA per SM, 128 x 256 (or 128 x 128) output tiles in a static round-robin order (tiles that share their
// rows of X run side by side on neighbouring SMs). K advances in slabs of 64 elements through a ring of four
// (16 KB of A + 32 KB of W) stages; tcgen05.mma M128 x N256 x K16 accumulates in one of two accumulators
// in tensor memory, so that the epilogue of a tile (tensor memory -> registers -> bf16 -> global) runs under the
// main loop of the next.
//
//   warps 0-3  epilogue: thread = output row (TMEM lane), 32 columns at a time
//   warp  4    MMA issuer (one thread), owner of the tensor-memory allocation
//   warp  5    W slabs (one tile copy per stage); the A slabs too when the rows are not gathered
//   warps 6-13 A row gathers: four lanes per warp, one four-row copy each per stage
#include "tc_attn_common.cuh"

namespace {

using fl_tc::warp_wait;

constexpr int kBM = 128, kBK = 64;   // the tile's width BN (256 or 128) is a template parameter
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK * 2;              // 16 KB
constexpr int kStageBytes = kABytes + 256 * kBK * 2;   // 16 KB of A + up to 32 KB of W
constexpr int kGatherWarps = 8;
constexpr int kIssueWarp = 4, kLoadWarp = 5, kFirstGatherWarp = 6;
constexpr int kThreads = (kFirstGatherWarp + kGatherWarps) * 32;
constexpr uint32_t kTmemCols = 512;                 // two accumulators of up to 256 columns

struct __align__(16) ProjCtl {
  uint64_t full[kStages], empty[kStages];
  uint64_t acc_full[2], acc_free[2];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr size_t kProjSmem = 1024 + (size_t)kStages * kStageBytes + sizeof(ProjCtl);

struct ProjArgs {
  CUtensorMap x_map;   // X [x_rows, d_in] bf16: box 64 x 1 (row gathers) or 64 x 128 (rows taken in order)
  CUtensorMap w_map;   // W [d_out, d_in] bf16: box 64 x BN
  const int32_t* src_idx;   // [n] rows of X, or null
  const int32_t* dst_idx;   // [n] rows of Y, or null
  __nv_bfloat16* y;
  int n, d_in, d_out;
  int m_tiles, n_tiles;
  int accumulate;
  int* status;
};

__device__ __forceinline__ void mma_ss_acc(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                           uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accum)
      : "memory");
}

template <bool GATHER, int kBN>
__global__ void __launch_bounds__(kThreads, 1) proj_rows_kernel(const __grid_constant__ ProjArgs a) {
  constexpr int kBBytes = kBN * kBK * 2;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  ProjCtl& ctl = *reinterpret_cast<ProjCtl*>(smem + (size_t)kStages * kStageBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_slabs = a.d_in / kBK;
  const int n_work = a.m_tiles * a.n_tiles;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      tc::mbar_init(&ctl.full[s], GATHER ? 1 + kGatherWarps : 1);
      tc::mbar_init(&ctl.empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(&ctl.acc_full[b], 1);
      tc::mbar_init(&ctl.acc_free[b], 4);
    }
    ctl.abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == kIssueWarp) {
    tc::tmem_alloc(&ctl.tmem_base, kTmemCols);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = ctl.tmem_base;
  volatile int* abort_flag = &ctl.abort_flag;
  fl_grid_wait();
  fl_grid_release();

  if (warp >= kFirstGatherWarp) {
    if (GATHER) {
      const int gw = warp - kFirstGatherWarp;
      const int g4 = gw * 4 + (lane & 3);            // the lane's group of four rows inside the tile
      bool ok = true;
      int g = 0;
      for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
        const int m0 = (w / a.n_tiles) * kBM + g4 * 4;
        int r[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) r[q] = __ldg(a.src_idx + min(m0 + q, a.n - 1));   // rows past n repeat the last row
        for (int ks = 0; ks < n_slabs; ++ks, ++g) {
          const int st = g % kStages;
          if (g >= kStages) ok = warp_wait(&ctl.empty[st], ((g / kStages) - 1) & 1, abort_flag);
          if (!ok) break;
          if (lane == 0) tc::mbar_arrive_expect_tx(&ctl.full[st], 4 * 512);
          __syncwarp();
          if (lane < 4)
            tc::tma_gather4(smem + (size_t)st * kStageBytes + g4 * 512, &a.x_map, &ctl.full[st], ks * kBK, r[0], r[1],
                            r[2], r[3]);
        }
      }
    }
  } else if (warp == kLoadWarp) {
    bool ok = true;
    int g = 0;
    for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
      const int m0 = (w / a.n_tiles) * kBM, n0 = (w % a.n_tiles) * kBN;
      for (int ks = 0; ks < n_slabs; ++ks, ++g) {
        const int st = g % kStages;
        if (g >= kStages) ok = warp_wait(&ctl.empty[st], ((g / kStages) - 1) & 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          uint8_t* stage = smem + (size_t)st * kStageBytes;
          tc::mbar_arrive_expect_tx(&ctl.full[st], GATHER ? kBBytes : kABytes + kBBytes);
          tc::tma_tile2d(stage + kABytes, &a.w_map, &ctl.full[st], ks * kBK, n0);
          if (!GATHER) tc::tma_tile2d(stage, &a.x_map, &ctl.full[st], ks * kBK, m0);
        }
        __syncwarp();
      }
    }
  } else if (warp == kIssueWarp) {
    if (lane == 0) {
      const uint32_t idesc = tc::make_idesc_bf16(kBM, kBN, false);
      const uint64_t desc0 = tc::make_desc_sw128(tc::smem_u32(smem), 16, 1024);
      const uint32_t hi = (uint32_t)(desc0 >> 32), lo0 = (uint32_t)desc0;
      int g = 0, i = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x, ++i) {
        const int buf = i & 1;
        if (i >= 2) ok = tc::mbar_wait(&ctl.acc_free[buf], ((i >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        tc::tc_fence_after();
        const uint32_t d_dst = tmem + buf * kBN;
        for (int ks = 0; ks < n_slabs; ++ks, ++g) {
          const int st = g % kStages;
          if (!tc::mbar_wait(&ctl.full[st], (g / kStages) & 1, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          const uint32_t a_lo = lo0 + ((st * kStageBytes) >> 4), b_lo = a_lo + (kABytes >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ss_acc(d_dst, a_lo + kk * 2, b_lo + kk * 2, hi, idesc, (ks | kk) != 0 ? 1u : 0u);
          tc::mma_commit(&ctl.empty[st]);
        }
        if (ok) tc::mma_commit(&ctl.acc_full[buf]);
      }
    }
    __syncwarp();
  } else {
    // epilogue: the thread's row of the tile is its lane of tensor memory
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    int i = 0;
    for (int w = blockIdx.x; w < n_work; w += gridDim.x, ++i) {
      const int buf = i & 1;
      const int m = (w / a.n_tiles) * kBM + warp * 32 + lane, n0 = (w % a.n_tiles) * kBN;
      const bool row_ok = m < a.n;
      const int64_t dst_row = row_ok ? (a.dst_idx != nullptr ? (int64_t)__ldg(a.dst_idx + m) : (int64_t)m) : 0;
      __nv_bfloat16* y_row = a.y + dst_row * a.d_out + n0;
      // the rows this tile adds into are read one piece ahead of the accumulator (the first piece before the
      // accumulator is even complete): nothing else writes them during the launch
      const bool rmw = a.accumulate != 0 && row_ok;
      uint4 old_cur[4], old_nxt[4];
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        old_cur[v] = make_uint4(0u, 0u, 0u, 0u);
        if (rmw && n0 + v * 8 < a.d_out) old_cur[v] = *reinterpret_cast<const uint4*>(y_row + v * 8);
      }
      if (!warp_wait(&ctl.acc_full[buf], (i >> 1) & 1, abort_flag)) break;
      tc::tc_fence_after();
#pragma unroll 1
      for (int p = 0; p < kBN / 32; ++p) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          old_nxt[v] = make_uint4(0u, 0u, 0u, 0u);
          if (rmw && p + 1 < kBN / 32 && n0 + (p + 1) * 32 + v * 8 < a.d_out)
            old_nxt[v] = *reinterpret_cast<const uint4*>(y_row + (p + 1) * 32 + v * 8);
        }
        uint32_t r[32];
        tc::tmem_ld32(tmem + lane_base + buf * kBN + p * 32, r);
        tc::tmem_wait_ld();
        if (p == kBN / 32 - 1) {
          // the accumulator is in registers: the issuer may start the tile after next
          tc::tc_fence_before();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&ctl.acc_free[buf]);
        }
        if (row_ok) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            if (n0 + p * 32 + v * 8 < a.d_out) {
              float x[8], old[8];
              fl_tc::unpack8(old_cur[v], old);      // zeros unless the call accumulates
#pragma unroll
              for (int u = 0; u < 8; ++u) x[u] = __uint_as_float(r[v * 8 + u]) + old[u];
              *reinterpret_cast<uint4*>(y_row + p * 32 + v * 8) = fl_tc::pack8(x);
            }
          }
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) old_cur[v] = old_nxt[v];
      }
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kIssueWarp) {
    if (ctl.abort_flag) {
      // give copies and MMAs still in flight time to land before the tensor memory is returned
      if (lane == 0) tc::mma_commit(&ctl.acc_full[0]);
      __syncwarp();
      for (int it = 0; it < (1 << 16); ++it) __nanosleep(256);
    }
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

}  // namespace

extern "C" int fl_project_rows(fl_ctx* ctx, const void* x, int64_t x_rows, const int32_t* src_idx, int32_t n,
                               int32_t d_in, const void* w, int32_t d_out, void* y, int64_t y_rows,
                               const int32_t* dst_idx, int32_t accumulate, int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  FL_REQUIRE(n >= 0 && d_in > 0 && d_out > 0 && x_rows > 0 && y_rows > 0);
  FL_REQUIRE(accumulate == 0 || accumulate == 1);
  FL_REQUIRE(x_rows <= INT32_MAX && y_rows <= INT32_MAX);
  FL_REQUIRE(src_idx != nullptr || n <= x_rows);
  FL_REQUIRE(dst_idx != nullptr || n <= y_rows);
  if (d_in % kBK != 0 || d_out % 8 != 0) return FL_ERR_UNSUPPORTED;
  if (n == 0) return FL_OK;
  FL_REQUIRE(x != nullptr && w != nullptr && y != nullptr);
  FL_REQUIRE(fl_aligned16(x) && fl_aligned16(w) && fl_aligned16(y));
  FL_REQUIRE(x != y && w != y);
  if ((size_t)ctx->max_smem_optin < kProjSmem || ctx->encode_tiled == nullptr || ctx->tmaps == nullptr)
    return FL_ERR_UNSUPPORTED;
  {
    const fl_idx_check ck[2] = {{src_idx, n, 0, nullptr, 0, (int32_t)x_rows - 1, 0},
                                {dst_idx, n, 0, nullptr, 0, (int32_t)y_rows - 1, 1}};
    const int rc = fl_debug_check(ctx, ck, 2, status, stream);
    if (rc != FL_OK) return rc;
  }
  ProjArgs a;
  const bool gather = src_idx != nullptr;
  a.m_tiles = (n + kBM - 1) / kBM;
  // Tile width: 256 columns keep the tensor pipe busiest per byte loaded; 128 columns when that leaves the last of the
  // rounds over the SMs mostly empty (a narrow tile costs about 0.58 of a wide one, 0.8 when its rows are gathered).
  const auto rounds = [&](int bn) {
    const int64_t tiles = (int64_t)a.m_tiles * ((d_out + bn - 1) / bn);
    return (double)((tiles + ctx->sm_count - 1) / ctx->sm_count);
  };
  const int bn = rounds(128) * (gather ? 0.8 : 0.58) < rounds(256) ? 128 : 256;
  if (!fl_tile_tmap(ctx, x, x_rows, d_in, gather ? 1 : kBM, &a.x_map) || !fl_tile_tmap(ctx, w, d_out, d_in, bn, &a.w_map))
    return FL_ERR_CUDA;
  a.src_idx = src_idx;
  a.dst_idx = dst_idx;
  a.y = static_cast<__nv_bfloat16*>(y);
  a.n = n;
  a.d_in = d_in;
  a.d_out = d_out;
  a.n_tiles = (d_out + bn - 1) / bn;
  a.accumulate = accumulate;
  a.status = status;
  const int64_t n_work = (int64_t)a.m_tiles * a.n_tiles;
  const int grid = (int)(n_work < ctx->sm_count ? n_work : ctx->sm_count);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define FL_PROJ(G, BN)                                                                                              \
  do {                                                                                                              \
    auto kern = proj_rows_kernel<G, BN>;                                                                            \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProjSmem));         \
    FL_CHECK_CUDA(fl_launch(ctx, kern, dim3(grid), dim3(kThreads), kProjSmem, st, a));                              \
  } while (0)
  if (gather) {
    if (bn == 256) FL_PROJ(true, 256); else FL_PROJ(true, 128);
  } else {
    if (bn == 256) FL_PROJ(false, 256); else FL_PROJ(false, 128);
  }
#undef FL_PROJ
  return fl_launch_status();
}
