// Stages 2 + 4 on the Blackwell tensor path: the attention replacement of Eq. 7 for one (head, query
// block, tile of up to 128 active queries) per CTA, with K/V of the selected columns gathered from the
// bf16 base and patched with the dequantized residual streams (Eq. 8) on their way into shared memory.
//
// Warp roles (17 warps):
//   warps 0-3   softmax of the OLD term  (fixed normaliser lse_prev: p_old = exp(s_old - lse_prev), mass m_i)
//   warps 4-7   softmax of the NEW term  (running reference with lazy rescale of the accumulator)
//   warp  8     one elected thread issues every tcgen05.mma; the warp owns the tensor-memory allocation
//   warps 9-16  producers: gather selected columns, dequantize-and-add, write 128B-swizzled operand tiles
// Per chunk of 64 selected columns:  S_old = Q_old Khat_old^T, S_new = Q_new Khat_new^T  (SS MMAs, f32 in TMEM),
// P = softmax pieces written back to TMEM as bf16, then acc_old += P_old Vhat_old, acc_new += P_new Vhat_new
// (TS MMAs, V as MN-major operand). Epilogue: O = O_prev - acc_old + (m / l) acc_new.
// Tensor memory (512 columns): acc_old 0-127, acc_new 128-255, two S/P buffers of 128 columns.
// Every mbarrier wait is bounded; on a timeout the CTA raises a flag, drains and reports FL_ERR_TIMEOUT.
#include "fl_internal.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int kM = 128;
constexpr int kDH = 128;
constexpr int kNC = 64;
constexpr int kStages = 2;
constexpr int kTileBytes = kNC * kDH * 2;   // 16 KB
constexpr int kQTileBytes = kM * kDH * 2;   // 32 KB
constexpr int kSoftmaxWarps = 8;
constexpr int kMmaWarp = 8;
constexpr int kProducerWarps = 8;
constexpr int kThreads = (kSoftmaxWarps + 1 + kProducerWarps) * 32;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr uint32_t kAccOld = 0, kAccNew = 128, kSBase = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 60.f;   // in log2 units: rescale only when the reference falls this far behind

struct TcArgs {
  const __nv_bfloat16* q_new;
  const __nv_bfloat16* q_old;
  const __nv_bfloat16* o_prev;
  __nv_bfloat16* o_out;
  const int32_t* active_idx;
  int n_active;
  DevSide k, v;
  int n_old;
  const int32_t* col_idx;
  const int32_t* col_cnt;
  int c;
  const float* lse_prev;
  float* lse_out;
  int32_t* status;
  int L, H, q_block, nb, d, group;
  float scale;
};

struct __align__(16) TcSmemCtl {
  uint64_t full[kStages];     // producers -> MMA: operand tiles of the stage are written
  uint64_t done[kStages];     // MMA -> producers / softmax: PV of the chunk finished (stage and S buffer free)
  uint64_t s_full[kStages];   // MMA -> softmax: S of the chunk is in tensor memory
  uint64_t p_full[kStages];   // softmax -> MMA: P of the chunk is in tensor memory
  uint64_t acc_done;          // MMA -> softmax: all accumulation finished
  uint32_t tmem_base;
  int abort_flag;
  int col_pos[kStages][kNC];
  float mass[kM];
  float ell[kM];
  float ref[kM];
};

constexpr size_t kTcSmemBytes = 1024 /* alignment slack */ + 2 * kQTileBytes + kStages * 4 * kTileBytes + sizeof(TcSmemCtl);

// bounded wait whose verdict is the same for every lane of the (fully converged) warp
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const bool ok = tc::mbar_wait(bar, parity, abort_flag);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ uint4 pack8(const float (&x)[8]) {
  uint4 r;
  r.x = tc::pack_bf16(x[0], x[1]);
  r.y = tc::pack_bf16(x[2], x[3]);
  r.z = tc::pack_bf16(x[4], x[5]);
  r.w = tc::pack_bf16(x[6], x[7]);
  return r;
}

__device__ __forceinline__ void unpack8(const uint4& raw, float (&x)[8]) {
  const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(hp[i]);
    x[2 * i] = f.x;
    x[2 * i + 1] = f.y;
  }
}

template <int BITS>
__global__ void __launch_bounds__(kThreads, 1) loop_attn_tc_kernel(const __grid_constant__ TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_old_tile = smem;
  uint8_t* q_new_tile = smem + kQTileBytes;
  uint8_t* stage_base = smem + 2 * kQTileBytes;  // per stage: k_old, k_new, v_old, v_new
  TcSmemCtl& ctl = *reinterpret_cast<TcSmemCtl*>(stage_base + kStages * 4 * kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.y, h = blockIdx.z;
  const size_t prob = (size_t)h * a.nb + b;
  // ---- rows of this tile -----------------------------------------------------------------------
  const int blk_lo = b * a.q_block, blk_hi = min(a.L, (b + 1) * a.q_block);
  int lo = 0, hi = a.n_active;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(a.active_idx + mid) < blk_lo) lo = mid + 1; else hi = mid; }
  const int q_lo = lo; hi = a.n_active;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(a.active_idx + mid) < blk_hi) lo = mid + 1; else hi = mid; }
  const int q_hi = lo;
  const int s0 = q_lo + blockIdx.x * kM;
  if (s0 >= q_hi) return;
  const int n_rows = min(kM, q_hi - s0);
  const int i_max = __ldg(a.active_idx + s0 + n_rows - 1);
  // ---- causal prefix of the block's ascending column set -------------------------------------------
  const int32_t* cols = a.col_idx + prob * a.c;
  const int cnt = __ldg(a.col_cnt + prob);
  lo = 0; hi = cnt;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(cols + mid) <= i_max) lo = mid + 1; else hi = mid; }
  const int cnt_eff = lo;
  const int n_chunks = (cnt_eff + kNC - 1) / kNC;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      tc::mbar_init(&ctl.full[s], kProducerThreads);
      tc::mbar_init(&ctl.done[s], 1);
      tc::mbar_init(&ctl.s_full[s], 1);
      tc::mbar_init(&ctl.p_full[s], kSoftmaxWarps * 32);
    }
    tc::mbar_init(&ctl.acc_done, 1);
    ctl.abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == kMmaWarp) {
    tc::tmem_alloc(&ctl.tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem = ctl.tmem_base;
  volatile int* abort_flag = &ctl.abort_flag;

  if (warp > kMmaWarp) {
    // =========================================== producers ===========================================
    const int pt = tid - (kMmaWarp + 1) * 32;  // 0..255
    const int pw = pt >> 5;
    // Q tiles (once)
    for (int it = pt; it < 2 * kM * 16; it += kProducerThreads) {
      const int which = it / (kM * 16);
      const int rem = it % (kM * 16);
      const int r = rem >> 4, ch = rem & 15;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < n_rows) {
        const __nv_bfloat16* src = (which ? a.q_new : a.q_old) + (size_t)(s0 + r) * a.d + h * kDH + ch * 8;
        v = __ldg(reinterpret_cast<const uint4*>(src));
      }
      uint8_t* tile = which ? q_new_tile : q_old_tile;
      *reinterpret_cast<uint4*>(tile + (ch >> 3) * (kM * 128) + tc::sw128_offset(r, ch & 7)) = v;
    }
    const int half = lane >> 4;          // 0: K row, 1: V row
    const int ch = lane & 15;            // 16-byte chunk inside the 256-byte row
    const DevSide& side = half ? a.v : a.k;
    const int elem = h * kDH + ch * 8;
    for (int ci = 0; ci < n_chunks; ++ci) {
      const int st = ci % kStages;
      if (ci >= kStages) {
        if (!warp_wait(&ctl.done[st], ((ci / kStages) - 1) & 1, abort_flag)) break;
      }
      uint8_t* sb = stage_base + st * 4 * kTileBytes;
      uint8_t* t_old = sb + (half ? 2 : 0) * kTileBytes;
      uint8_t* t_new = t_old + kTileBytes;
      const int u0 = ci * kNC + pw * 8;
      int jj[8], sl_new[8];
#pragma unroll
      for (int it = 0; it < 8; ++it) jj[it] = (u0 + it < cnt_eff) ? __ldg(cols + u0 + it) : -1;
      if (lane < 8) ctl.col_pos[st][pw * 8 + lane] = (u0 + lane < cnt_eff) ? __ldg(cols + u0 + lane) : INT32_MAX;
      // base rows of 8 columns in flight; most columns carry no residual and go to shared memory untouched
      uint4 raw[8];
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        raw[it] = make_uint4(0, 0, 0, 0);
        sl_new[it] = -1;
        if (jj[it] >= 0) {
          raw[it] = __ldg(reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(side.base) +
                                                          (size_t)jj[it] * a.d + elem));
          sl_new[it] = __ldg(side.s[a.n_old].slot + jj[it]);
        }
      }
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int u = pw * 8 + it;
        const uint32_t off = (ch >> 3) * (kNC * 128) + tc::sw128_offset(u, ch & 7);
        uint4 v_old = raw[it];
        float x[8];
        bool unpacked = false;
        if (jj[it] >= 0) {
          for (int s = 0; s < a.n_old; ++s) {           // residuals of earlier loops (Eq. 8 chain, loop order)
            if (__ldg(side.s[s].slot + jj[it]) < 0) continue;
            if (!unpacked) { unpack8(raw[it], x); unpacked = true; }
            apply_stream8<__nv_bfloat16, BITS>(side.s[s], jj[it], elem, a.d, a.group, x);
          }
          if (unpacked) v_old = pack8(x);
        }
        *reinterpret_cast<uint4*>(t_old + off) = v_old;
        uint4 v_new = v_old;
        if (sl_new[it] >= 0) {                          // this loop's residual
          if (!unpacked) unpack8(raw[it], x);
          apply_stream8<__nv_bfloat16, BITS>(side.s[a.n_old], jj[it], elem, a.d, a.group, x);
          v_new = pack8(x);
        }
        *reinterpret_cast<uint4*>(t_new + off) = v_new;
      }
      tc::fence_proxy_async_smem();
      tc::mbar_arrive(&ctl.full[st]);
    }
  } else if (warp == kMmaWarp) {
    // =========================================== MMA issuer ==========================================
    if (lane == 0) {
      const uint32_t idesc_qk = tc::make_idesc_bf16(kM, kNC, false);
      const uint32_t idesc_pv = tc::make_idesc_bf16(kM, kDH, true);
      const uint32_t q_old_addr = tc::smem_u32(q_old_tile), q_new_addr = tc::smem_u32(q_new_tile);
      bool ok = true;
      auto issue_pv = [&](int cj) -> bool {
        const int sbuf = cj % kStages;
        if (!tc::mbar_wait(&ctl.p_full[sbuf], (cj / kStages) & 1, abort_flag)) return false;
        tc::tc_fence_after();
        const uint32_t stg = tc::smem_u32(stage_base + sbuf * 4 * kTileBytes);
        const uint32_t p_old = tmem + kSBase + sbuf * 128, p_new = p_old + 64;
#pragma unroll
        for (int kk = 0; kk < kNC / 16; ++kk) {
          const uint64_t bd = tc::make_desc_sw128(stg + 2 * kTileBytes + kk * 2048, kNC * 128, 1024);
          tc::mma_ts(tmem + kAccOld, p_old + kk * 8, bd, idesc_pv, cj > 0 || kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < kNC / 16; ++kk) {
          const uint64_t bd = tc::make_desc_sw128(stg + 3 * kTileBytes + kk * 2048, kNC * 128, 1024);
          tc::mma_ts(tmem + kAccNew, p_new + kk * 8, bd, idesc_pv, cj > 0 || kk > 0);
        }
        tc::mma_commit(&ctl.done[sbuf]);
        return true;
      };
      for (int ci = 0; ci < n_chunks && ok; ++ci) {
        const int st = ci % kStages;
        if (!tc::mbar_wait(&ctl.full[st], (ci / kStages) & 1, abort_flag)) { ok = false; break; }
        tc::tc_fence_after();
        const uint32_t stg = tc::smem_u32(stage_base + st * 4 * kTileBytes);
        const uint32_t s_old = tmem + kSBase + st * 128, s_new = s_old + 64;
#pragma unroll
        for (int kk = 0; kk < kDH / 16; ++kk) {
          const uint64_t ad = tc::make_desc_sw128(q_old_addr + (kk >> 2) * (kM * 128) + (kk & 3) * 32, 16, 1024);
          const uint64_t bd = tc::make_desc_sw128(stg + (kk >> 2) * (kNC * 128) + (kk & 3) * 32, 16, 1024);
          tc::mma_ss(s_old, ad, bd, idesc_qk, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < kDH / 16; ++kk) {
          const uint64_t ad = tc::make_desc_sw128(q_new_addr + (kk >> 2) * (kM * 128) + (kk & 3) * 32, 16, 1024);
          const uint64_t bd = tc::make_desc_sw128(stg + kTileBytes + (kk >> 2) * (kNC * 128) + (kk & 3) * 32, 16, 1024);
          tc::mma_ss(s_new, ad, bd, idesc_qk, kk > 0);
        }
        tc::mma_commit(&ctl.s_full[st]);
        if (ci >= 1) ok = issue_pv(ci - 1);
      }
      if (ok && n_chunks > 0) ok = issue_pv(n_chunks - 1);
      tc::mma_commit(&ctl.acc_done);
    }
    __syncwarp();
  } else {
    // ============================================ softmax ============================================
    const int grp = warp >> 2;                    // 0: old term, 1: new term
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const bool row_ok = row < n_rows;
    const int pos = row_ok ? __ldg(a.active_idx + s0 + row) : -1;
    const float c2 = a.scale * kLog2e;
    const float lse_prev = row_ok ? a.lse_prev[(size_t)h * a.L + pos] : 0.f;
    const float lse2 = lse_prev * kLog2e;
    float mass = 0.f, ell = 0.f, ref = -INFINITY;
    bool ok = true;
    for (int ci = 0; ci < n_chunks; ++ci) {
      const int sbuf = ci % kStages;
      // full[] first: orders the producers' column-position writes before the reads below
      if (!warp_wait(&ctl.full[sbuf], (ci / kStages) & 1, abort_flag) ||
          !warp_wait(&ctl.s_full[sbuf], (ci / kStages) & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t s_addr = tmem + lane_base + kSBase + sbuf * 128 + grp * 64;
      const int* cp = ctl.col_pos[sbuf];
      // P (bf16, 32 columns) overwrites the first half of the 64-column S region: S[0:32) is consumed before
      // P[0:16) is stored, S[32:64) before P[16:32).
      if (grp == 0) {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t r[32], p[16];
          tc::tmem_ld32(s_addr + hf * 32, r);
          tc::tmem_wait_ld();
#pragma unroll
          for (int u = 0; u < 32; u += 2) {
            const float p0 = cp[hf * 32 + u] <= pos ? tc::ex2(fmaf(__uint_as_float(r[u]), c2, -lse2)) : 0.f;
            const float p1 = cp[hf * 32 + u + 1] <= pos ? tc::ex2(fmaf(__uint_as_float(r[u + 1]), c2, -lse2)) : 0.f;
            mass += p0 + p1;
            p[u >> 1] = tc::pack_bf16(p0, p1);
          }
          tc::tmem_st16(s_addr + hf * 16, p);
        }
      } else {
        float cm = -INFINITY;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t r[32];
          tc::tmem_ld32(s_addr + hf * 32, r);
          tc::tmem_wait_ld();
#pragma unroll
          for (int u = 0; u < 32; ++u)
            if (cp[hf * 32 + u] <= pos) cm = fmaxf(cm, __uint_as_float(r[u]));
        }
        cm *= c2;                                    // c2 > 0: scaling commutes with the maximum
        float factor = 1.f;
        bool need = false;
        if (ref == -INFINITY) {
          ref = cm;                                  // first causal column(s) of this row: accumulator row is still zero
        } else if (cm - ref > kRescaleThreshold) {
          factor = tc::ex2(ref - cm);
          ref = cm;
          need = true;
        }
        if (__any_sync(0xffffffffu, need)) {
          // lazy rescale of acc_new (rare): every earlier PV must have completed before the rows are rewritten
          if (ci >= 1) {
            if (!warp_wait(&ctl.done[(ci - 1) % kStages], ((ci - 1) / kStages) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
          }
          ell *= factor;
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t acc[32];
            tc::tmem_ld32(tmem + lane_base + kAccNew + q4 * 32, acc);
            tc::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * factor);
            tc::tmem_st32(tmem + lane_base + kAccNew + q4 * 32, acc);
          }
          tc::tmem_wait_st();
        }
        const float rr = ref == -INFINITY ? 0.f : ref;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t r[32], p[16];
          tc::tmem_ld32(s_addr + hf * 32, r);
          tc::tmem_wait_ld();
#pragma unroll
          for (int u = 0; u < 32; u += 2) {
            const float p0 = cp[hf * 32 + u] <= pos ? tc::ex2(fmaf(__uint_as_float(r[u]), c2, -rr)) : 0.f;
            const float p1 = cp[hf * 32 + u + 1] <= pos ? tc::ex2(fmaf(__uint_as_float(r[u + 1]), c2, -rr)) : 0.f;
            ell += p0 + p1;
            p[u >> 1] = tc::pack_bf16(p0, p1);
          }
          tc::tmem_st16(s_addr + hf * 16, p);
        }
      }
      tc::tmem_wait_st();
      tc::tc_fence_before();
      tc::mbar_arrive(&ctl.p_full[sbuf]);
    }
    // ---- epilogue ------------------------------------------------------------------------------------
    if (ok) ok = warp_wait(&ctl.acc_done, 0, abort_flag);
    tc::tc_fence_after();
    if (grp == 0) ctl.mass[row] = mass;
    else { ctl.ell[row] = ell; ctl.ref[row] = ref; }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const float m_i = ctl.mass[row], l_i = ctl.ell[row], ref_i = ctl.ref[row];
    const bool acc_valid = ok && n_chunks > 0;            // warp-uniform: the tensor-memory reads below are collective
    const bool has = acc_valid && ref_i > -INFINITY;      // per row: T_i is not empty
    const float w = has ? m_i / l_i : 0.f;
    for (int hh = 0; hh < 2; ++hh) {
      // each group finishes 64 of the 128 head-dim columns
      const int col0 = grp * 64 + hh * 32;
      uint32_t ao[32], an[32];
      if (acc_valid) {
        tc::tmem_ld32(tmem + lane_base + kAccOld + col0, ao);
        tc::tmem_ld32(tmem + lane_base + kAccNew + col0, an);
        tc::tmem_wait_ld();
      }
      if (!row_ok) continue;
      const size_t off = (size_t)(s0 + row) * a.d + h * kDH + col0;
      if (has) {
#pragma unroll
        for (int v8 = 0; v8 < 4; ++v8) {
          float prev[8], out[8];
          load8<__nv_bfloat16>(a.o_prev + off + v8 * 8, prev);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            out[i] = prev[i] - __uint_as_float(ao[v8 * 8 + i]) + w * __uint_as_float(an[v8 * 8 + i]);
          store8<__nv_bfloat16>(a.o_out + off + v8 * 8, out);
        }
      } else if (a.o_out != a.o_prev) {
#pragma unroll
        for (int v8 = 0; v8 < 4; ++v8)
          *reinterpret_cast<uint4*>(a.o_out + off + v8 * 8) = *reinterpret_cast<const uint4*>(a.o_prev + off + v8 * 8);
      }
    }
    if (grp == 1 && row_ok)
      a.lse_out[(size_t)h * a.L + pos] = has ? (ref_i + log2f(l_i)) * kLn2 - logf(m_i) : lse_prev;
  }
  // ---- teardown ------------------------------------------------------------------------------------------
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    if (ctl.abort_flag) {
      // let outstanding tensor work drain (bounded) before the columns are released
      if (lane == 0) tc::mma_commit(&ctl.acc_done);
      __syncwarp();
      for (int it = 0; it < (1 << 16); ++it) __nanosleep(256);
    }
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

}  // namespace

// Returns FL_ERR_UNSUPPORTED when the tensor path does not cover the request (caller falls back to the
// SIMT kernel, which is also CUDA).
int fl_launch_loop_attn_tc(const fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_old,
                           const int32_t* active_idx, int n_active, const fl_kv_store* store, const int32_t* col_idx,
                           const int32_t* col_cnt, int c, const float* lse_prev, float* lse_out, const void* o_prev,
                           void* o_out, int32_t* status, cudaStream_t st) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH) return FL_ERR_UNSUPPORTED;
  if ((size_t)ctx->max_smem_optin < kTcSmemBytes) return FL_ERR_UNSUPPORTED;
  TcArgs a{};
  a.q_new = static_cast<const __nv_bfloat16*>(q_new);
  a.q_old = static_cast<const __nv_bfloat16*>(q_old);
  a.o_prev = static_cast<const __nv_bfloat16*>(o_prev);
  a.o_out = static_cast<__nv_bfloat16*>(o_out);
  a.active_idx = active_idx; a.n_active = n_active;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.n_old = loop_r - 2;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.lse_prev = lse_prev; a.lse_out = lse_out; a.status = status;
  a.L = s->L; a.H = s->n_heads; a.q_block = s->q_block; a.nb = fl_n_blocks(s);
  a.d = s->n_heads * s->head_dim; a.group = s->group; a.scale = s->sm_scale;
  const int per_block = s->q_block < n_active ? s->q_block : n_active;
  const dim3 grid((per_block + kM - 1) / kM, a.nb, s->n_heads);
#define FL_TC(BITS)                                                                                              \
  do {                                                                                                           \
    auto kern = loop_attn_tc_kernel<BITS>;                                                                       \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes));  \
    kern<<<grid, kThreads, kTcSmemBytes, st>>>(a);                                                               \
  } while (0)
  switch (s->bits) {
    case 2: FL_TC(2); break;
    case 4: FL_TC(4); break;
    case 8: FL_TC(8); break;
    default: FL_TC(16); break;
  }
#undef FL_TC
  return fl_launch_status();
}
