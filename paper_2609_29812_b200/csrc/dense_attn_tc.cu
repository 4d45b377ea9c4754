// Dense source loop on the Blackwell tensor path (bf16 storage, head dimension 128): causal attention of all L rows
// (Eq. 2) and the block column statistics loop 2 starts from (Eq. 6 with every causal key a candidate and m_C = 1).
//
// Two kernels, because the statistics need each row's final normaliser:
//   dense_flash_kernel     one CTA per (128-row query tile, head): S = Q K^T per chunk of 64 keys, online softmax with a
//                          lazily moved reference, acc += P V; writes O = acc / l and lse = ref + log l.
//   dense_colsum_kernel    one CTA per (chunk of 128 keys, query block, head): S^T = K Q^T with the KEYS as the
//                          accumulator's rows, so that the thread that owns a key sums exp(s - lse_i) over the block's
//                          queries in registers, in a fixed order (no atomics, no cross-thread reduction):
//                          col_scores[h, b, j] = sum_{i in block b, i >= j} p_ij.
// Both keep two CTAs per SM (half the shared memory and 256 tensor-memory columns each) so that one CTA's dependent
// chain MMA -> exponentials -> MMA runs under the other's. Operand tiles come by plain TMA tile loads (the rows are
// consecutive), 128B-swizzled; rows beyond L read as zero and are masked. Every mbarrier wait is bounded.
#include "tc_attn_common.cuh"

namespace {

using namespace fl_tc;

constexpr int kIssueWarp = 4;
constexpr int kTmaWarp = 5;
constexpr int kThreads = 6 * 32;
constexpr uint32_t kAcc = 0, kS = 128;
constexpr uint32_t kTmemCols = 256;

struct alignas(64) DnArgs {
  CUtensorMap q_map;      // [L, d] bf16, box 64 elements x 128 rows
  CUtensorMap k_map;      // box 64 x 64 rows (flash: a chunk of keys) or 64 x 128 rows (column sums: K is the M operand)
  CUtensorMap v_map;      // box 64 x 64 rows
  __nv_bfloat16* o;       // [L, d]
  float* lse;             // [H, L] (flash: written, may be null; column sums: read)
  float* col_scores;      // [H, nb, L]
  int32_t* status;
  int L, H, d, q_block, nb;
  float scale;
};

struct __align__(16) FlashCtl {
  uint64_t q_full, k_landed[2], v_landed[2], s_full[2], p_full[2], p_free[2], acc_done;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr size_t kFlashSmem = 1024 + kQTileBytes + 4 * kTileBytes + sizeof(FlashCtl);

__global__ void __launch_bounds__(kThreads, 2) dense_flash_kernel(const __grid_constant__ DnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_tile = smem;
  uint8_t* k_ring = smem + kQTileBytes;
  uint8_t* v_ring = k_ring + 2 * kTileBytes;
  FlashCtl& ctl = *reinterpret_cast<FlashCtl*>(v_ring + 2 * kTileBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // later tiles see more keys: they are dispatched first
  const int n_tiles = (a.L + kM - 1) / kM;
  const int tile = n_tiles - 1 - (int)(blockIdx.x / a.H), h = blockIdx.x % a.H;
  const int s0 = tile * kM, n_rows = min(kM, a.L - s0);
  const int n_chunks = (s0 + n_rows + kNC - 1) / kNC;
  if (tid == 0) {
    tc::mbar_init(&ctl.q_full, 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&ctl.k_landed[s], 1);
      tc::mbar_init(&ctl.v_landed[s], 1);
      tc::mbar_init(&ctl.s_full[s], 1);
      tc::mbar_init(&ctl.p_full[s], 4);
      tc::mbar_init(&ctl.p_free[s], 1);
    }
    tc::mbar_init(&ctl.acc_done, 1);
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

  if (warp == kTmaWarp) {
    if (lane == 0) {
      tc::mbar_arrive_expect_tx(&ctl.q_full, kQTileBytes);
      tc::tma_tile2d(q_tile, &a.q_map, &ctl.q_full, h * kDH, s0);
      tc::tma_tile2d(q_tile + kM * 128, &a.q_map, &ctl.q_full, h * kDH + 64, s0);
      auto fill = [&](int ci, bool is_v) {
        uint64_t* bar = is_v ? &ctl.v_landed[ci & 1] : &ctl.k_landed[ci & 1];
        uint8_t* dst = (is_v ? v_ring : k_ring) + (ci & 1) * kTileBytes;
        const void* map = is_v ? static_cast<const void*>(&a.v_map) : static_cast<const void*>(&a.k_map);
        tc::mbar_arrive_expect_tx(bar, kTileBytes);
        tc::tma_tile2d(dst, map, bar, h * kDH, ci * kNC);
        tc::tma_tile2d(dst + kNC * 128, map, bar, h * kDH + 64, ci * kNC);
      };
      bool ok = true;
      fill(0, false);
      // K of chunk n + 1 (free once QK^T of chunk n - 1 has completed), then V of chunk n (free once PV of n - 2 has)
      for (int ci = 0; ci < n_chunks && ok; ++ci) {
        if (ci + 1 < n_chunks) {
          if (ci + 1 >= 2) ok = tc::mbar_wait(&ctl.s_full[(ci + 1) & 1], (((ci + 1) >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
          fill(ci + 1, false);
        }
        if (ci >= 2) ok = tc::mbar_wait(&ctl.p_free[ci & 1], ((ci >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        fill(ci, true);
      }
    }
    __syncwarp();
  } else if (warp == kIssueWarp) {
    if (lane == 0) {
      const uint32_t idesc_qk = tc::make_idesc_bf16(kM, kNC, false);
      const uint32_t idesc_pv = tc::make_idesc_bf16(kM, kDH, true);
      const uint64_t q_desc = tc::make_desc_sw128(tc::smem_u32(q_tile), 16, 1024);
      const uint64_t k_desc0 = tc::make_desc_sw128(tc::smem_u32(k_ring), 16, 1024);
      const uint32_t kq_hi = (uint32_t)(k_desc0 >> 32);
      const uint32_t q_lo_w = (uint32_t)q_desc, k_lo0 = (uint32_t)k_desc0;
      const uint64_t v_desc0 = tc::make_desc_sw128(tc::smem_u32(v_ring), kNC * 128, 1024);
      const uint32_t v_hi = (uint32_t)(v_desc0 >> 32), v_lo0 = (uint32_t)v_desc0;
      const uint32_t s_base = tmem + kS, acc = tmem + kAcc;
#pragma unroll 1
      for (int n = 0; n <= n_chunks; ++n) {
        if (n < n_chunks) {
          const int sl = n & 1;
          if (n == 0 && !tc::mbar_wait(&ctl.q_full, 0, abort_flag)) break;
          if (!tc::mbar_wait(&ctl.k_landed[sl], (n >> 1) & 1, abort_flag)) break;
          if (n >= 2 && !tc::mbar_wait(&ctl.p_free[sl], ((n >> 1) - 1) & 1, abort_flag)) break;
          const uint32_t s_dst = s_base + sl * kNC;
          tc::tc_fence_after();
          const uint32_t k_lo = k_lo0 + sl * (kTileBytes >> 4);
#define FL_QK(KK, ACC)                                                                                       \
  tc::mma_ss_lo<ACC>(s_dst, q_lo_w + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), kq_hi,               \
                     k_lo + ((((KK) >> 2) * (kNC * 128) + ((KK)&3) * 32) >> 4), kq_hi, idesc_qk)
          FL_QK(0, false); FL_QK(1, true); FL_QK(2, true); FL_QK(3, true);
          FL_QK(4, true);  FL_QK(5, true); FL_QK(6, true); FL_QK(7, true);
#undef FL_QK
          tc::mma_commit(&ctl.s_full[sl]);
        }
        if (n > 0) {
          const int gp = n - 1, pb = gp & 1;
          if (!tc::mbar_wait(&ctl.v_landed[pb], (gp >> 1) & 1, abort_flag)) break;
          if (!tc::mbar_wait(&ctl.p_full[pb], (gp >> 1) & 1, abort_flag)) break;
          tc::tc_fence_after();
          const uint32_t v_lo = v_lo0 + pb * (kTileBytes >> 4);
          const uint32_t p_src = s_base + pb * kNC;
          const uint32_t acc0 = n > 1 ? 1u : 0u;
#pragma unroll
          for (int kk = 0; kk < kNC / 16; ++kk)
            tc::mma_ts_lo(acc, p_src + kk * 8, v_lo + kk * (2048 >> 4), v_hi, idesc_pv, kk > 0 ? 1u : acc0);
          tc::mma_commit(&ctl.p_free[pb]);
        }
      }
      tc::mma_commit(&ctl.acc_done);
    }
    __syncwarp();
  } else {
    // ============================================ softmax ============================================
    const int row = warp * 32 + lane;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const bool row_ok = row < n_rows;
    const int pos = s0 + row;
    const float c2 = a.scale * kLog2e;
    const uint32_t s_addr = tmem + lane_base + kS;
    float ell = 0.f, ref = -INFINITY;
    bool ok = true;
    for (int ci = 0; ci < n_chunks; ++ci) {
      const int pb = ci & 1;
      if (!warp_wait(&ctl.s_full[pb], (ci >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      // causal mask: the chunk's columns are 64 ci .. 64 ci + 63; the visible ones of a row are a prefix
      const bool unmasked = __all_sync(0xffffffffu, !row_ok || ci * kNC + kNC - 1 <= pos);
      const int vis = row_ok ? min(kNC, max(0, pos - ci * kNC + 1)) : 0;
      const uint32_t sp_addr = s_addr + pb * kNC;
#pragma unroll 1
      for (int hf = 0; hf < 2 && ok; ++hf) {
        uint32_t r[32];
        tc::tmem_ld32(sp_addr + hf * 32, r);
        tc::tmem_wait_ld();
        if (!unmasked) {
          const int lim = vis - hf * 32;
#pragma unroll
          for (int u = 0; u < 32; ++u) r[u] = u < lim ? r[u] : 0xff800000u;
        }
        float cm = -INFINITY;
#pragma unroll
        for (int u = 0; u < 32; u += 2) cm = fmaxf(cm, fmaxf(__uint_as_float(r[u]), __uint_as_float(r[u + 1])));
        cm *= c2;
        const bool first = ref == -INFINITY && cm > -INFINITY;
        const bool over = ref > -INFINITY && cm - ref > kRescaleThreshold;
        if (first) ref = cm;
        if (__any_sync(0xffffffffu, over)) {
          float factor = 1.f;
          if (over) { factor = tc::ex2(ref - cm); ref = cm; }
          if (ci > 0) {
            if (!warp_wait(&ctl.p_free[(ci - 1) & 1], ((ci - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
#pragma unroll 1
            for (int q4 = 0; q4 < 8; ++q4) {
              uint32_t acc[16];
              tc::tmem_ld16(tmem + lane_base + kAcc + q4 * 16, acc);
              tc::tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * factor);
              tc::tmem_st16(tmem + lane_base + kAcc + q4 * 16, acc);
            }
            tc::tmem_wait_st();
          }
          ell *= factor;
          if (hf == 1) {
            uint32_t ph[16];
            tc::tmem_wait_st();
            tc::tmem_ld16(sp_addr, ph);
            tc::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(&ph[i]);
              const float2 f = __bfloat1622float2(v);
              ph[i] = tc::pack_bf16(f.x * factor, f.y * factor);
            }
            tc::tmem_st16(sp_addr, ph);
          }
        }
        const float sub = ref == -INFINITY ? 0.f : ref;
        float sum = 0.f;
#pragma unroll
        for (int u = 0; u < 32; u += 2) {
          const float p0 = tc::ex2(fmaf(__uint_as_float(r[u]), c2, -sub));
          const float p1 = tc::ex2(fmaf(__uint_as_float(r[u + 1]), c2, -sub));
          sum += p0 + p1;
          r[u >> 1] = tc::pack_bf16(p0, p1);
        }
        ell += sum;
        tc::tmem_st16(sp_addr + hf * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[0]));
      }
      if (!ok) break;
      tc::tmem_wait_st();
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl.p_full[pb]);
    }
    // ---- epilogue: O = acc / l, staged in the Q tile (every QK^T has retired) and written out coalesced ---------
    if (ok) ok = warp_wait(&ctl.acc_done, 0, abort_flag);
    tc::tc_fence_after();
    asm volatile("bar.sync 1, 128;" ::: "memory");
    const float w = (ok && ell > 0.f) ? 1.f / ell : 0.f;
    uint8_t* stage = q_tile;
#pragma unroll 1
    for (int c16 = 0; c16 < 16; ++c16) {
      uint32_t av[8];
      tc::tmem_ld8(tmem + lane_base + kAcc + c16 * 8, av);
      tc::tmem_wait_ld();
      float pv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) pv[i] = w * __uint_as_float(av[i]);
      *reinterpret_cast<uint4*>(stage + row * 256 + ((c16 ^ (row & 7)) << 4)) = pack8(pv);
    }
    if (row_ok && a.lse != nullptr && ok) a.lse[(size_t)h * a.L + pos] = (ref + log2f(ell)) * kLn2;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ok) {
#pragma unroll 1
      for (int k = 0; k < 16; ++k) {
        const int idx = k * 128 + tid, rr = idx >> 4, cc = idx & 15;
        if (rr < n_rows)
          *reinterpret_cast<uint4*>(a.o + (size_t)(s0 + rr) * a.d + (size_t)h * kDH + cc * 8) =
              *reinterpret_cast<const uint4*>(stage + rr * 256 + ((cc ^ (rr & 7)) << 4));
      }
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kIssueWarp) {
    if (ctl.abort_flag) {
      if (lane == 0) tc::mma_commit(&ctl.acc_done);
      __syncwarp();
      for (int it = 0; it < (1 << 16); ++it) __nanosleep(256);
    }
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------------------
// Column sums. Accumulator tile D[key j (128 lanes)][query i (128 columns)] = K_chunk Q_tile^T; the thread of lane j
// adds exp(scale s_ji - lse_i) over the queries i >= j of the block, tile after tile.
// ------------------------------------------------------------------------------------------------------------
struct __align__(16) ColsumCtl {
  uint64_t k_full, q_full[2], d_full[2], d_free[2];
  uint32_t tmem_base;
  int abort_flag;
  float lse2[2][kM];      // log-normalisers of the tile's queries, in log2 units
};
constexpr size_t kColsumSmem = 1024 + 3 * kQTileBytes + sizeof(ColsumCtl);

__global__ void __launch_bounds__(kThreads, 2) dense_colsum_kernel(const __grid_constant__ DnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* k_tile = smem;                       // [128 keys][128] as the M operand
  uint8_t* q_ring = smem + kQTileBytes;         // two query tiles [128 queries][128] as the N operand
  ColsumCtl& ctl = *reinterpret_cast<ColsumCtl*>(q_ring + 2 * kQTileBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int kc = blockIdx.x, b = a.nb - 1 - (int)blockIdx.y, h = blockIdx.z;
  const int blk_lo = b * a.q_block, blk_hi = min(a.L, (b + 1) * a.q_block);
  const int j0 = kc * kM;
  if (j0 >= blk_hi) return;                      // the chunk lies beyond the block's last row: no candidates
  const int n_tiles = (blk_hi - blk_lo + kM - 1) / kM;
  const int t_first = j0 > blk_lo ? (j0 - blk_lo) / kM : 0;    // earlier tiles hold no query at or after the first key
  if (tid == 0) {
    tc::mbar_init(&ctl.k_full, 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&ctl.q_full[s], 2);          // the tile's bytes (one arrival with the byte count) + its normalisers
      tc::mbar_init(&ctl.d_full[s], 1);
      tc::mbar_init(&ctl.d_free[s], 4);
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

  if (warp == kTmaWarp) {
    if (lane == 0) {
      tc::mbar_arrive_expect_tx(&ctl.k_full, kQTileBytes);
      tc::tma_tile2d(k_tile, &a.k_map, &ctl.k_full, h * kDH, j0);
      tc::tma_tile2d(k_tile + kM * 128, &a.k_map, &ctl.k_full, h * kDH + 64, j0);
    }
    bool ok = true;
    for (int t = t_first, n = 0; t < n_tiles && ok; ++t, ++n) {
      const int sl = n & 1, i0 = blk_lo + t * kM;
      // the slot is free once the MMAs of the tile two back have completed (they also read its normalisers' slot,
      // which the epilogue has released by then: it runs behind the MMAs)
      if (n >= 2) ok = warp_wait(&ctl.d_full[sl], ((n >> 1) - 1) & 1, abort_flag) &&
                       warp_wait(&ctl.d_free[sl], ((n >> 1) - 1) & 1, abort_flag);
      if (!ok) break;
      if (lane == 0) {
        tc::mbar_arrive_expect_tx(&ctl.q_full[sl], kQTileBytes);
        tc::tma_tile2d(q_ring + sl * kQTileBytes, &a.q_map, &ctl.q_full[sl], h * kDH, i0);
        tc::tma_tile2d(q_ring + sl * kQTileBytes + kM * 128, &a.q_map, &ctl.q_full[sl], h * kDH + 64, i0);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = i0 + q * 32 + lane;
        ctl.lse2[sl][q * 32 + lane] = i < blk_hi ? __ldg(a.lse + (size_t)h * a.L + i) * kLog2e : INFINITY;
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl.q_full[sl]);
    }
  } else if (warp == kIssueWarp) {
    if (lane == 0) {
      const uint32_t idesc = tc::make_idesc_bf16(kM, kM, false);
      const uint64_t k_desc = tc::make_desc_sw128(tc::smem_u32(k_tile), 16, 1024);
      const uint64_t q_desc0 = tc::make_desc_sw128(tc::smem_u32(q_ring), 16, 1024);
      const uint32_t hi = (uint32_t)(k_desc >> 32);
      const uint32_t k_lo_w = (uint32_t)k_desc, q_lo0 = (uint32_t)q_desc0;
      for (int t = t_first, n = 0; t < n_tiles; ++t, ++n) {
        const int sl = n & 1;
        if (n == 0 && !tc::mbar_wait(&ctl.k_full, 0, abort_flag)) break;
        if (!tc::mbar_wait(&ctl.q_full[sl], (n >> 1) & 1, abort_flag)) break;
        if (n >= 2 && !tc::mbar_wait(&ctl.d_free[sl], ((n >> 1) - 1) & 1, abort_flag)) break;
        tc::tc_fence_after();
        const uint32_t d_dst = tmem + sl * kM;
        const uint32_t q_lo = q_lo0 + sl * (kQTileBytes >> 4);
#define FL_KQ(KK, ACC)                                                                                       \
  tc::mma_ss_lo<ACC>(d_dst, k_lo_w + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), hi,                  \
                     q_lo + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), hi, idesc)
        FL_KQ(0, false); FL_KQ(1, true); FL_KQ(2, true); FL_KQ(3, true);
        FL_KQ(4, true);  FL_KQ(5, true); FL_KQ(6, true); FL_KQ(7, true);
#undef FL_KQ
        tc::mma_commit(&ctl.d_full[sl]);
      }
    }
    __syncwarp();
  } else {
    // the thread's key: lane of tensor memory = row of the accumulator
    const int jr = warp * 32 + lane, j = j0 + jr;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const float c2 = a.scale * kLog2e;
    float sum = 0.f;
    bool ok = true;
    for (int t = t_first, n = 0; t < n_tiles; ++t, ++n) {
      const int sl = n & 1, i0 = blk_lo + t * kM;
      if (!warp_wait(&ctl.q_full[sl], (n >> 1) & 1, abort_flag)) { ok = false; break; }   // the normalisers
      if (!warp_wait(&ctl.d_full[sl], (n >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      // queries before the key see nothing of it; queries beyond the block carry lse = +inf (probability 0)
      const bool all_visible = __all_sync(0xffffffffu, j <= i0);
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        uint32_t r[32];
        tc::tmem_ld32(tmem + lane_base + sl * kM + q * 32, r);
        tc::tmem_wait_ld();
        const float* l2 = ctl.lse2[sl] + q * 32;
        float part = 0.f;
        if (all_visible) {
#pragma unroll
          for (int u = 0; u < 32; ++u) part += tc::ex2(fmaf(__uint_as_float(r[u]), c2, -l2[u]));
        } else {
          const int first = j - (i0 + q * 32);        // queries u >= first are at or after the key
#pragma unroll
          for (int u = 0; u < 32; ++u) {
            const float p = tc::ex2(fmaf(__uint_as_float(r[u]), c2, -l2[u]));
            part += u >= first ? p : 0.f;
          }
        }
        sum += part;
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl.d_free[sl]);
    }
    if (ok && j < blk_hi) a.col_scores[((size_t)h * a.nb + b) * a.L + j] = sum;
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kIssueWarp) {
    if (ctl.abort_flag) {
      if (lane == 0) tc::mma_commit(&ctl.d_full[0]);
      __syncwarp();
      for (int it = 0; it < (1 << 16); ++it) __nanosleep(256);
    }
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------------------
// Next-loop column scores of a SPARSE loop (Appendix D.2: a sparse source loop offers its own selected columns as
// candidates, scored by the block sums of its new probabilities): the same K Q^T tiles, with the 128 keys of a tile
// gathered by position from the base (four rows per TMA copy) and the columns that carry residual payloads rebuilt
// in place (Eq. 8 chain up to the loop itself), and the queries taken from the compact rows of the block's active
// tokens. col_scores_next[h, b, u] = sum over the block's active rows i >= S[u] of exp(s_iu - lse_i), lse the loop's
// new log-normaliser.
// ------------------------------------------------------------------------------------------------------------
struct alignas(64) SpArgs {
  CUtensorMap k_map;      // K base [L, d], box 64 x 1 (row gathers)
  CUtensorMap q_map;      // compact new Q rows [n_active, d], box 64 x 128
  DevSide k;
  int n_use;              // residual streams contained in Khat^(r): loop_r - 1
  const int32_t* active_idx;
  int n_active;
  const int32_t* col_idx;
  const int32_t* col_cnt;
  int c;
  const float* lse;       // [H, L]: the loop's new log-normalisers
  float* out;             // [H, nb, c]
  int32_t* status;
  int L, H, d, q_block, nb, group;
  float scale;
};

struct __align__(16) SpColsumCtl {
  uint64_t k_full, k_ready, q_full[2], d_full[2], d_free[2];
  uint32_t tmem_base;
  int abort_flag;
  int q_lo, q_hi;
  float lse2[2][kM];
  int pos[2][kM];
};
constexpr size_t kSpColsumSmem = 1024 + 3 * kQTileBytes + sizeof(SpColsumCtl);

template <int BITS>
__global__ void __launch_bounds__(kThreads, 2) sparse_colsum_kernel(const __grid_constant__ SpArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* k_tile = smem;
  uint8_t* q_ring = smem + kQTileBytes;
  SpColsumCtl& ctl = *reinterpret_cast<SpColsumCtl*>(q_ring + 2 * kQTileBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int kc = blockIdx.x, b = blockIdx.y, h = blockIdx.z;
  const size_t prob = (size_t)h * a.nb + b;
  const int cnt = min(__ldg(a.col_cnt + prob), a.c);
  const int u0 = kc * kM;
  if (u0 >= cnt) return;
  const int32_t* cols = a.col_idx + prob * a.c;
  if (warp < 2) {
    const int target = warp == 0 ? b * a.q_block : min(a.L, (b + 1) * a.q_block);
    int below;
    const int r = lower_bound_warp(a.active_idx, a.n_active, target, lane, &below);
    if (lane == 0) { if (warp == 0) ctl.q_lo = r; else ctl.q_hi = r; }
  }
  if (tid == 0) {
    tc::mbar_init(&ctl.k_full, 1);
    tc::mbar_init(&ctl.k_ready, 4);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&ctl.q_full[s], 2);
      tc::mbar_init(&ctl.d_full[s], 1);
      tc::mbar_init(&ctl.d_free[s], 4);
    }
    ctl.abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  const int q_lo = ctl.q_lo, q_hi = ctl.q_hi;
  if (q_hi <= q_lo) {   // no active row in the block: every score is zero
    for (int u = u0 + tid; u < min(cnt, u0 + kM); u += kThreads) a.out[prob * a.c + u] = 0.f;
    return;
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
  const int n_tiles = (q_hi - q_lo + kM - 1) / kM;

  if (warp == kTmaWarp) {
    // the tile's 128 selected columns: base rows by position, four per copy; positions past the count read as zero
    if (lane == 0) tc::mbar_arrive_expect_tx(&ctl.k_full, kQTileBytes);
    __syncwarp();
    {
      int y[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int u = u0 + lane * 4 + i;
        y[i] = u < cnt ? __ldg(cols + u) : a.L;
      }
      tc::tma_gather4(k_tile + lane * 512, &a.k_map, &ctl.k_full, h * kDH, y[0], y[1], y[2], y[3]);
      tc::tma_gather4(k_tile + kM * 128 + lane * 512, &a.k_map, &ctl.k_full, h * kDH + 64, y[0], y[1], y[2], y[3]);
    }
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int sl = t & 1, s0 = q_lo + t * kM;
      if (t >= 2) ok = warp_wait(&ctl.d_full[sl], ((t >> 1) - 1) & 1, abort_flag) &&
                       warp_wait(&ctl.d_free[sl], ((t >> 1) - 1) & 1, abort_flag);
      if (!ok) break;
      if (lane == 0) {
        tc::mbar_arrive_expect_tx(&ctl.q_full[sl], kQTileBytes);
        tc::tma_tile2d(q_ring + sl * kQTileBytes, &a.q_map, &ctl.q_full[sl], h * kDH, s0);
        tc::tma_tile2d(q_ring + sl * kQTileBytes + kM * 128, &a.q_map, &ctl.q_full[sl], h * kDH + 64, s0);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = s0 + q * 32 + lane;
        const int pos = i < q_hi ? __ldg(a.active_idx + i) : -1;
        ctl.pos[sl][q * 32 + lane] = pos;
        ctl.lse2[sl][q * 32 + lane] = pos >= 0 ? __ldg(a.lse + (size_t)h * a.L + pos) * kLog2e : INFINITY;
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl.q_full[sl]);
    }
  } else if (warp == kIssueWarp) {
    if (lane == 0) {
      const uint32_t idesc = tc::make_idesc_bf16(kM, kM, false);
      const uint64_t k_desc = tc::make_desc_sw128(tc::smem_u32(k_tile), 16, 1024);
      const uint64_t q_desc0 = tc::make_desc_sw128(tc::smem_u32(q_ring), 16, 1024);
      const uint32_t hi = (uint32_t)(k_desc >> 32);
      const uint32_t k_lo_w = (uint32_t)k_desc, q_lo0 = (uint32_t)q_desc0;
      for (int t = 0; t < n_tiles; ++t) {
        const int sl = t & 1;
        if (t == 0 && !tc::mbar_wait(&ctl.k_ready, 0, abort_flag)) break;
        if (!tc::mbar_wait(&ctl.q_full[sl], (t >> 1) & 1, abort_flag)) break;
        if (t >= 2 && !tc::mbar_wait(&ctl.d_free[sl], ((t >> 1) - 1) & 1, abort_flag)) break;
        tc::tc_fence_after();
        const uint32_t d_dst = tmem + sl * kM;
        const uint32_t q_lo_w = q_lo0 + sl * (kQTileBytes >> 4);
#define FL_KQ(KK, ACC)                                                                                       \
  tc::mma_ss_lo<ACC>(d_dst, k_lo_w + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), hi,                  \
                     q_lo_w + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), hi, idesc)
        FL_KQ(0, false); FL_KQ(1, true); FL_KQ(2, true); FL_KQ(3, true);
        FL_KQ(4, true);  FL_KQ(5, true); FL_KQ(6, true); FL_KQ(7, true);
#undef FL_KQ
        tc::mma_commit(&ctl.d_full[sl]);
      }
    }
    __syncwarp();
  } else {
    // ---- the four epilogue warps first rebuild the columns that carry residual payloads (Eq. 8 chain) ----------
    bool ok = warp_wait(&ctl.k_full, 0, abort_flag);
    if (ok) {
      const int ch = tid & 15;                        // 16-byte piece of the row
      const int elem = h * kDH + ch * 8;
      const __nv_bfloat16* base_rows = static_cast<const __nv_bfloat16*>(a.k.base) + elem;
#pragma unroll 1
      for (int u = tid >> 4; u < kM; u += 8) {
        if (u0 + u >= cnt) break;
        const int j = __ldg(cols + u0 + u);
        float x[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(base_rows + (size_t)j * a.d)), x);
        bool any = false;
#pragma unroll 1
        for (int s = 0; s < a.n_use; ++s) any |= apply_stream8<__nv_bfloat16, BITS>(a.k.s[s], j, elem, a.d, a.group, x);
        if (any) *reinterpret_cast<uint4*>(k_tile + (ch >> 3) * (kM * 128) + tc::sw128_offset(u, ch & 7)) = pack8(x);
      }
      tc::fence_proxy_async_smem();
    }
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(&ctl.k_ready);
    // ---- then sum the tiles: the thread of lane u owns selected column u0 + u -----------------------------------
    const int ur = warp * 32 + lane;
    const int jpos = u0 + ur < cnt ? __ldg(cols + u0 + ur) : INT32_MAX;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const float c2 = a.scale * kLog2e;
    float sum = 0.f;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int sl = t & 1;
      if (!warp_wait(&ctl.q_full[sl], (t >> 1) & 1, abort_flag)) { ok = false; break; }
      if (!warp_wait(&ctl.d_full[sl], (t >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      // the active rows ascend: when the tile's first row lies at or after every column of the warp nothing is masked
      const int pos_first = ctl.pos[sl][0];
      const bool all_visible = __all_sync(0xffffffffu, jpos == INT32_MAX || jpos <= pos_first);
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        uint32_t r[32];
        tc::tmem_ld32(tmem + lane_base + sl * kM + q * 32, r);
        tc::tmem_wait_ld();
        const float* l2 = ctl.lse2[sl] + q * 32;
        float part = 0.f;
        if (all_visible) {
#pragma unroll
          for (int u = 0; u < 32; ++u) part += tc::ex2(fmaf(__uint_as_float(r[u]), c2, -l2[u]));
        } else {
          const int* ps = ctl.pos[sl] + q * 32;
#pragma unroll
          for (int u = 0; u < 32; ++u) {
            const float p = tc::ex2(fmaf(__uint_as_float(r[u]), c2, -l2[u]));
            part += ps[u] >= jpos ? p : 0.f;
          }
        }
        sum += part;
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl.d_free[sl]);
    }
    if (ok && u0 + ur < cnt) a.out[prob * a.c + u0 + ur] = sum;
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kIssueWarp) {
    if (ctl.abort_flag) {
      if (lane == 0) tc::mma_commit(&ctl.d_full[0]);
      __syncwarp();
      for (int it = 0; it < (1 << 16); ++it) __nanosleep(256);
    }
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

}  // namespace

// Returns FL_ERR_UNSUPPORTED when the tensor path does not cover the request (the caller then runs the binary32
// kernels).
int fl_launch_dense_tc(fl_ctx* ctx, const fl_shape* s, const void* q, const void* k, const void* v, void* o, float* lse,
                       float* col_scores, int32_t* status, cudaStream_t st) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH || ctx->force_simt) return FL_ERR_UNSUPPORTED;
  if ((size_t)ctx->max_smem_optin < kColsumSmem || ctx->encode_tiled == nullptr || ctx->tmaps == nullptr)
    return FL_ERR_UNSUPPORTED;
  DnArgs a{};
  const int64_t d_row = (int64_t)s->n_heads * s->head_dim;
  if (!fl_tile_tmap(ctx, q, s->L, d_row, kM, &a.q_map) || !fl_tile_tmap(ctx, k, s->L, d_row, kNC, &a.k_map) ||
      !fl_tile_tmap(ctx, v, s->L, d_row, kNC, &a.v_map))
    return FL_ERR_UNSUPPORTED;
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.col_scores = col_scores;
  a.status = status;
  a.L = s->L; a.H = s->n_heads; a.d = (int)d_row; a.q_block = s->q_block; a.nb = fl_n_blocks(s);
  a.scale = s->sm_scale;
  const int n_tiles = (s->L + kM - 1) / kM;
  FL_CHECK_CUDA(cudaFuncSetAttribute(dense_flash_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFlashSmem));
  FL_CHECK_CUDA(cudaFuncSetAttribute(dense_flash_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     (int)cudaSharedmemCarveoutMaxShared));
  dense_flash_kernel<<<dim3(n_tiles * s->n_heads), kThreads, kFlashSmem, st>>>(a);
  int rc = fl_launch_status();
  if (rc != FL_OK || col_scores == nullptr) return rc;
  if (!fl_tile_tmap(ctx, k, s->L, d_row, kM, &a.k_map)) return FL_ERR_CUDA;
  FL_CHECK_CUDA(cudaFuncSetAttribute(dense_colsum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kColsumSmem));
  FL_CHECK_CUDA(cudaFuncSetAttribute(dense_colsum_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     (int)cudaSharedmemCarveoutMaxShared));
  dense_colsum_kernel<<<dim3(n_tiles, a.nb, s->n_heads), kThreads, kColsumSmem, st>>>(a);
  return fl_launch_status();
}

// Next-loop column scores of a sparse loop on the tensor path; FL_ERR_UNSUPPORTED when it does not cover the request.
int fl_launch_sparse_colsum_tc(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const int32_t* active_idx,
                               int n_active, const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt,
                               int c, const float* lse, float* out, int32_t* status, cudaStream_t st) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH || ctx->force_simt || n_active < 1) return FL_ERR_UNSUPPORTED;
  if ((size_t)ctx->max_smem_optin < kSpColsumSmem || ctx->encode_tiled == nullptr || ctx->tmaps == nullptr)
    return FL_ERR_UNSUPPORTED;
  SpArgs a{};
  const int64_t d_row = (int64_t)s->n_heads * s->head_dim;
  if (!fl_tile_tmap(ctx, store->k_base, s->L, d_row, 1, &a.k_map) ||
      !fl_tile_tmap(ctx, q_new, n_active, d_row, kM, &a.q_map))
    return FL_ERR_UNSUPPORTED;
  fl_dev_side(store, true, &a.k);
  a.n_use = loop_r - 1;
  a.active_idx = active_idx; a.n_active = n_active;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.lse = lse; a.out = out; a.status = status;
  a.L = s->L; a.H = s->n_heads; a.d = (int)d_row; a.q_block = s->q_block; a.nb = fl_n_blocks(s); a.group = s->group;
  a.scale = s->sm_scale;
  const dim3 grid((c + kM - 1) / kM, a.nb, s->n_heads);
#define FL_SC(BITS)                                                                                               \
  do {                                                                                                            \
    auto kern = sparse_colsum_kernel<BITS>;                                                                       \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSpColsumSmem));  \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,                     \
                                       (int)cudaSharedmemCarveoutMaxShared));                                    \
    kern<<<grid, kThreads, kSpColsumSmem, st>>>(a);                                                               \
  } while (0)
  switch (s->bits) {
    case 2: FL_SC(2); break;
    case 4: FL_SC(4); break;
    case 8: FL_SC(8); break;
    default: FL_SC(16); break;
  }
#undef FL_SC
  return fl_launch_status();
}
