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
  int y_stride, y_cols;     // row stride of y and the number of output columns that go to it
  int m_tiles, n_tiles;
  int accumulate;
  int* status;
  // Fused residual codec (Eq. 8) of the K and V columns of a stacked Q/K/V projection: output columns
  // [d_model, 2 d_model) are the new K rows, [2 d_model, 3 d_model) the new V rows of the active positions src_idx.
  DevSide k, v;             // base + earlier streams (read), in loop order
  uint8_t* k_codes; __half* k_scale; __half* k_zero;   // the stream being written
  uint8_t* v_codes; __half* v_scale; __half* v_zero;
  __nv_bfloat16* k_rows_prev; __nv_bfloat16* k_rows_cur;   // optional [n, d_model]: Xhat^(r-1) / Xhat^(r) of the active rows
  __nv_bfloat16* v_rows_prev; __nv_bfloat16* v_rows_cur;
  __nv_bfloat16* kv_out;    // optional [n, 2 d_model]: the new K | V rows themselves (bf16), as the codec saw them
  int d_model, n_prev, group;
};

// Xhat^(r-1) of 8 consecutive elements of position pos: base plus the earlier streams in loop order (binary32)
template <int BITS>
__device__ __forceinline__ void chain8(const DevSide& side, int n_prev, int pos, int elem, int d, int group,
                                       float (&xh)[8]) {
  load8<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(side.base) + (size_t)pos * d + elem, xh);
  for (int s = 0; s < n_prev; ++s) apply_stream8<__nv_bfloat16, BITS>(side.s[s], pos, elem, d, group, xh);
}

// The codec on one row of a 256-column K or V tile, by the thread that owns the row's lane of tensor memory: every
// group of `group` columns lies inside the thread's own 256 accumulator values, so minimum and maximum need no
// exchange. Two passes over a group (range, then codes); the accumulator is read from tensor memory twice and the
// previous reconstruction rebuilt twice (the second time from L1/L2). Arithmetic as in the stand-alone quantizer:
// binary32, offset rounded down and scale rounded up to fp16, codes by round-half-even of the true quotient.
template <int BITS>
__device__ __forceinline__ void codec_row(const ProjArgs& a, uint32_t tmem_row, bool row_ok, int t, int pos, bool is_v,
                                          int elem0, uint64_t* acc_free, int lane) {
  const DevSide& side = is_v ? a.v : a.k;
  uint8_t* codes = is_v ? a.v_codes : a.k_codes;
  __half* scale = is_v ? a.v_scale : a.k_scale;
  __half* zero = is_v ? a.v_zero : a.k_zero;
  __nv_bfloat16* rows_prev = is_v ? a.v_rows_prev : a.k_rows_prev;
  __nv_bfloat16* rows_cur = is_v ? a.v_rows_cur : a.k_rows_cur;
  const int d = a.d_model, g = a.group, pieces = g >> 5, n_groups = 256 / g;
  const float qmax = (float)((1 << BITS) - 1);
  for (int gi = 0; gi < n_groups; ++gi) {
    const int e_g = elem0 + gi * g;
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll 1
    for (int pc = 0; pc < pieces; ++pc) {
      uint32_t r[32];
      tc::tmem_ld32(tmem_row + gi * g + pc * 32, r);
      tc::tmem_wait_ld();
      if (row_ok) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float xh[8];
          chain8<BITS>(side, a.n_prev, pos, e_g + pc * 32 + v * 8, d, g, xh);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const float xn = __bfloat162float(__float2bfloat16_rn(__uint_as_float(r[v * 8 + u])));
            const float dl = __fsub_rn(xn, xh[u]);
            mn = fminf(mn, dl);
            mx = fmaxf(mx, dl);
          }
        }
      }
    }
    const __half zh = __float2half_rd(mn);
    const float zf = __half2float(zh);
    const float range = __fsub_rn(mx, zf);
    const __half sh = range == 0.f ? __float2half_rn(0.f) : __float2half_ru(__fdiv_rn(range, qmax));
    const float sf = __half2float(sh);
#pragma unroll 1
    for (int pc = 0; pc < pieces; ++pc) {
      uint32_t r[32];
      tc::tmem_ld32(tmem_row + gi * g + pc * 32, r);
      tc::tmem_wait_ld();
      if (gi == n_groups - 1 && pc == pieces - 1) {
        // last read of the accumulator: the issuer may start the tile after next
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(acc_free);
      }
      if (!row_ok) continue;
      const int e_p = e_g + pc * 32;
      uint32_t packed[8];     // 32 codes: BITS / 8 words of 32 bits each hold 32 / BITS ... filled below
#pragma unroll
      for (int wd = 0; wd < 8; ++wd) packed[wd] = 0u;
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        float xh[8], xn[8], xc[8];
        chain8<BITS>(side, a.n_prev, pos, e_p + v * 8, d, g, xh);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          xn[u] = __bfloat162float(__float2bfloat16_rn(__uint_as_float(r[v * 8 + u])));
          const float dl = __fsub_rn(xn[u], xh[u]);
          const float q = sf == 0.f ? 0.f : rintf(__fdiv_rn(__fsub_rn(dl, zf), sf));
          xc[u] = __fadd_rn(xh[u], __fmaf_rn(q, sf, zf));
          const int idx = v * 8 + u;                       // code index inside the piece
          packed[(idx * BITS) >> 5] |= (uint32_t)q << ((idx * BITS) & 31);
        }
        if (rows_prev != nullptr) store8<__nv_bfloat16>(rows_prev + (size_t)t * d + e_p + v * 8, xh);
        if (rows_cur != nullptr) store8<__nv_bfloat16>(rows_cur + (size_t)t * d + e_p + v * 8, xc);
        if (a.kv_out != nullptr)
          store8<__nv_bfloat16>(a.kv_out + (size_t)t * (2 * d) + (is_v ? d : 0) + e_p + v * 8, xn);
      }
      uint8_t* crow = codes + (size_t)t * (d * BITS / 8) + e_p * BITS / 8;
      if (BITS == 8) {
        *reinterpret_cast<uint4*>(crow) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        *reinterpret_cast<uint4*>(crow + 16) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
      } else if (BITS == 4) {
        *reinterpret_cast<uint4*>(crow) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
      } else {
        *reinterpret_cast<uint2*>(crow) = make_uint2(packed[0], packed[1]);
      }
    }
    if (row_ok) {
      const int gs = 31 - __clz(g);
      const size_t mi = (size_t)t * (d >> gs) + (e_g >> gs);
      scale[mi] = sh;
      zero[mi] = zh;
    }
  }
}

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

template <bool GATHER, int kBN, int CODEC>   // CODEC: 0, or the bit width of the fused residual codec (wide tiles only)
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
      if (CODEC != 0 && n0 >= a.d_model) {
        // a K or V tile of the stacked projection: the residual codec instead of a plain store
        const bool is_v = n0 >= 2 * a.d_model;
        const int pos = row_ok ? __ldg(a.src_idx + m) : 0;
        if (!warp_wait(&ctl.acc_full[buf], (i >> 1) & 1, abort_flag)) break;
        tc::tc_fence_after();
        codec_row<CODEC == 0 ? 4 : CODEC>(a, tmem + lane_base + buf * kBN, row_ok, m, pos, is_v,
                                          n0 - (is_v ? 2 : 1) * a.d_model, &ctl.acc_free[buf], lane);
        continue;
      }
      const int64_t dst_row = row_ok ? (a.dst_idx != nullptr ? (int64_t)__ldg(a.dst_idx + m) : (int64_t)m) : 0;
      __nv_bfloat16* y_row = a.y + dst_row * a.y_stride + n0;
      // the rows this tile adds into are read one piece ahead of the accumulator (the first piece before the
      // accumulator is even complete): nothing else writes them during the launch
      const bool rmw = a.accumulate != 0 && row_ok;
      uint4 old_cur[4], old_nxt[4];
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        old_cur[v] = make_uint4(0u, 0u, 0u, 0u);
        if (rmw && n0 + v * 8 < a.y_cols) old_cur[v] = *reinterpret_cast<const uint4*>(y_row + v * 8);
      }
      if (!warp_wait(&ctl.acc_full[buf], (i >> 1) & 1, abort_flag)) break;
      tc::tc_fence_after();
#pragma unroll 1
      for (int p = 0; p < kBN / 32; ++p) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          old_nxt[v] = make_uint4(0u, 0u, 0u, 0u);
          if (rmw && p + 1 < kBN / 32 && n0 + (p + 1) * 32 + v * 8 < a.y_cols)
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
            if (n0 + p * 32 + v * 8 < a.y_cols) {
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
  ProjArgs a = {};
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
  a.y_stride = d_out;
  a.y_cols = d_out;
  a.d_model = 0;
  a.n_tiles = (d_out + bn - 1) / bn;
  a.accumulate = accumulate;
  a.status = status;
  const int64_t n_work = (int64_t)a.m_tiles * a.n_tiles;
  const int grid = (int)(n_work < ctx->sm_count ? n_work : ctx->sm_count);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define FL_PROJ(G, BN)                                                                                              \
  do {                                                                                                              \
    auto kern = proj_rows_kernel<G, BN, 0>;                                                                          \
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

extern "C" int fl_project_qkv_quant(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* x, int64_t x_rows,
                                    const int32_t* active_idx, int32_t n_active, const void* w_qkv, void* q_out,
                                    void* kv_out, const fl_kv_store* store, int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(loop_r >= 2 && loop_r <= FL_MAX_LOOPS + 1);
  FL_REQUIRE(n_active >= 0 && n_active <= shape->L && x_rows > 0 && x_rows <= INT32_MAX);
  rc = fl_check_store(shape, store, loop_r - 1);
  if (rc != FL_OK) return rc;
  const fl_kv_stream& ks = store->k_res[loop_r - 2];
  const fl_kv_stream& vs = store->v_res[loop_r - 2];
  FL_REQUIRE(ks.n_rows == n_active && vs.n_rows == n_active);
  const int d = shape->n_heads * shape->head_dim;
  // bf16 storage, a real codec, groups that tile a 256-column output tile, Q / K / V boundaries on tile boundaries
  if (shape->dtype != FL_BF16 || shape->bits == 16 || shape->group < 32 || d % 256 != 0) return FL_ERR_UNSUPPORTED;
  if (n_active == 0) return FL_OK;
  FL_REQUIRE(x != nullptr && w_qkv != nullptr && q_out != nullptr && active_idx != nullptr);
  FL_REQUIRE(fl_aligned16(x) && fl_aligned16(w_qkv) && fl_aligned16(q_out) && fl_aligned16(kv_out));
  FL_REQUIRE(x != q_out && w_qkv != q_out && kv_out != q_out);
  if ((size_t)ctx->max_smem_optin < kProjSmem || ctx->encode_tiled == nullptr || ctx->tmaps == nullptr)
    return FL_ERR_UNSUPPORTED;
  {
    fl_idx_check ck[1 + 2 * FL_MAX_LOOPS];
    int nck = 0;
    ck[nck++] = {active_idx, n_active, 0, nullptr, 0, (int32_t)(x_rows < shape->L ? x_rows : shape->L) - 1, 1};
    for (int i = 0; i < loop_r - 2; ++i) {
      ck[nck++] = {store->k_res[i].slot_of_pos, shape->L, 0, nullptr, -1, store->k_res[i].n_rows - 1, 0};
      ck[nck++] = {store->v_res[i].slot_of_pos, shape->L, 0, nullptr, -1, store->v_res[i].n_rows - 1, 0};
    }
    rc = fl_debug_check(ctx, ck, nck, status, stream);
    if (rc != FL_OK) return rc;
  }
  ProjArgs a = {};
  if (!fl_tile_tmap(ctx, x, x_rows, d, 1, &a.x_map) || !fl_tile_tmap(ctx, w_qkv, 3 * (int64_t)d, d, 256, &a.w_map))
    return FL_ERR_CUDA;
  a.src_idx = active_idx;
  a.dst_idx = nullptr;
  a.y = static_cast<__nv_bfloat16*>(q_out);
  a.n = n_active;
  a.d_in = d;
  a.d_out = 3 * d;
  a.y_stride = d;
  a.y_cols = d;
  a.m_tiles = (n_active + kBM - 1) / kBM;
  a.n_tiles = 3 * d / 256;
  a.accumulate = 0;
  a.status = status;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.k_codes = static_cast<uint8_t*>(ks.codes); a.k_scale = reinterpret_cast<__half*>(ks.scale);
  a.k_zero = reinterpret_cast<__half*>(ks.zero);
  a.v_codes = static_cast<uint8_t*>(vs.codes); a.v_scale = reinterpret_cast<__half*>(vs.scale);
  a.v_zero = reinterpret_cast<__half*>(vs.zero);
  a.k_rows_prev = static_cast<__nv_bfloat16*>(ks.rows_prev);   // each written when it is there
  a.k_rows_cur = static_cast<__nv_bfloat16*>(ks.rows_cur);
  a.v_rows_prev = static_cast<__nv_bfloat16*>(vs.rows_prev);
  a.v_rows_cur = static_cast<__nv_bfloat16*>(vs.rows_cur);
  a.kv_out = static_cast<__nv_bfloat16*>(kv_out);
  a.d_model = d;
  a.n_prev = loop_r - 2;
  a.group = shape->group;
  const int64_t n_work = (int64_t)a.m_tiles * a.n_tiles;
  const int grid = (int)(n_work < ctx->sm_count ? n_work : ctx->sm_count);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define FL_PROJQ(BITS)                                                                                              \
  do {                                                                                                              \
    auto kern = proj_rows_kernel<true, 256, BITS>;                                                                  \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kProjSmem));         \
    FL_CHECK_CUDA(fl_launch(ctx, kern, dim3(grid), dim3(kThreads), kProjSmem, st, a));                              \
  } while (0)
  if (shape->bits == 8) FL_PROJQ(8); else if (shape->bits == 4) FL_PROJQ(4); else FL_PROJQ(2);
#undef FL_PROJQ
  return fl_launch_status();
}
