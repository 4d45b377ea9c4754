// Stages 2 + 4 on the Blackwell tensor path: the attention replacement of Eq. 7 for one (query block,
// head) per CTA, with K/V of the selected columns gathered from the bf16 base and patched with the
// dequantized residual streams (Eq. 8) on their way into shared memory.
//
// Warp roles (16 warps, 512 threads):
//   warps 0-3   softmax of the OLD term  (fixed normaliser lse_prev: p_old = exp(s_old - lse_prev), mass m_i)
//   warps 4-7   softmax of the NEW term  (running reference with lazy rescale of the accumulator)
//   warp  8     one elected thread issues every tcgen05.mma; the warp owns the tensor-memory allocation
//   warps 9-15  producers: gather selected columns, dequantize-and-add, write 128B-swizzled operand tiles
//
// Prologue (whole CTA): the block's causal column list is copied to shared memory together with a bit mask
// of the residual streams that carry each column, and stably partitioned into columns WITHOUT a payload in
// the current loop (Khat_old == Khat_new, one K tile and one V tile serve both terms) followed by columns
// WITH one (separate old / new tiles). Most columns are of the first kind and are a plain gather.
//
// Per chunk of 64 columns:  S_old = Q_old Khat_old^T, S_new = Q_new Khat_new^T  (SS MMAs, f32 in TMEM),
// P = softmax pieces written back to TMEM as bf16, then acc_old += P_old Vhat_old, acc_new += P_new Vhat_new
// (TS MMAs, V as MN-major operand). Epilogue: O = O_prev - acc_old + (m / l) acc_new.
// Shared memory: Q_old, Q_new tiles (64 KB) + a ring of four 32 KB operand slots (K tile | V tile); a chunk of
// the first kind takes one slot, of the second kind two. Tensor memory (512 columns): acc_old 0-127,
// acc_new 128-255, two S/P buffers of 128 columns.
// Every mbarrier wait is bounded; on a timeout the CTA raises a flag, drains and reports FL_ERR_TIMEOUT.
#include "fl_internal.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int kM = 128;
constexpr int kDH = 128;
constexpr int kNC = 64;
constexpr int kSlots = 4;
constexpr int kTileBytes = kNC * kDH * 2;   // 16 KB
constexpr int kSlotBytes = 2 * kTileBytes;  // K tile | V tile
constexpr int kQTileBytes = kM * kDH * 2;   // 32 KB
constexpr int kSoftmaxWarps = 8;
constexpr int kMmaWarp = 8;
constexpr int kProducerWarps = 7;
constexpr int kWarps = kSoftmaxWarps + 1 + kProducerWarps;  // 16
constexpr int kThreads = kWarps * 32;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kMaxCols = 3072;              // column budget the shared-memory column list can hold
constexpr uint32_t kAccOld = 0, kAccNew = 128, kSBase = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 60.f;   // in log2 units: rescale only when the reference falls this far behind

// Optional device-side timeline for tuning (compile with -DFL_TC_TRACE): the CTA (block 1, head 0) writes
// clock64() stamps into the buffer passed as `status`: trace[(role * 64 + chunk) * 4 + event].
#ifdef FL_TC_TRACE
#define TC_TRACE(role, chunk, ev)                                                                      \
  do {                                                                                                 \
    if (blockIdx.x == 1 && blockIdx.y == 0 && (chunk) < 64 && a.status != nullptr)                     \
      reinterpret_cast<long long*>(a.status)[((role) * 64 + (chunk)) * 4 + (ev)] = clock64();          \
  } while (0)
#else
#define TC_TRACE(role, chunk, ev) do { } while (0)
#endif

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
  uint64_t full[kSlots];   // producers -> MMA: the slot's operand tiles are written
  uint64_t done[kSlots];   // MMA -> producers / softmax: the MMAs that read the slot have finished
  uint64_t s_full[2];      // MMA -> softmax: S of the chunk is in tensor memory
  uint64_t p_full[2];      // softmax -> MMA: P of the chunk is in tensor memory
  uint64_t acc_done;       // MMA -> softmax: all accumulation of the tile finished
  uint32_t tmem_base;
  int abort_flag;
  int q_lo, q_hi;          // block's slot range in active_idx
  int n_plain, n_patch;    // columns without / with a payload in the current loop
  int warp_cnt[kWarps][2];
  int col_pos[kSlots][kNC];
  int col_last[kSlots];    // largest column position of the chunk, INT32_MAX if the chunk is padded
  float mass[kM];
  float ell[kM];
  float ref[kM];
};

constexpr size_t kTcSmemBytes = 1024 /* alignment slack */ + 2 * kQTileBytes + kSlots * kSlotBytes + sizeof(TcSmemCtl) +
                                2 * kMaxCols * sizeof(int32_t);

// Bounded wait of a fully converged warp: lane 0 polls, the verdict is shared, and every lane then observes
// the completed phase itself (one immediate poll) so that it acquires what the arriving threads released.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) ok = tc::mbar_wait(bar, parity, abort_flag);
  ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  if (ok) {
    bool seen = false;
    for (int it = 0; it < 1024 && !seen; ++it) seen = tc::mbar_try_wait(bar, parity);
    ok = __all_sync(0xffffffffu, seen);
  }
  return ok;
}

// first index in the ascending array with value >= target; all 32 lanes cooperate (32-ary search)
__device__ __forceinline__ int lower_bound32(const int32_t* __restrict__ arr, int n, int target, int lane) {
  int lo = 0, hi = n;
  while (hi > lo) {
    const int step = (hi - lo + 31) >> 5;
    const int idx = lo + lane * step + step - 1;
    const bool less = idx < hi && __ldg(arr + idx) < target;
    const int k = __popc(__ballot_sync(0xffffffffu, less));
    const int new_lo = lo + k * step;
    hi = min(hi, new_lo + step - 1);
    lo = min(new_lo, hi);
  }
  return lo;
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

// Dequantize-and-add for one 16-byte piece of a column that carries residual payloads (Eq. 8 chain in
// binary32, loop order): the rare path of the gather.
template <int BITS>
__device__ __forceinline__ void patch_piece(const DevSide& side, int n_old, uint32_t mask, int j, int elem, int d,
                                         int group, const uint4& raw, uint4& v_old, uint4& v_new) {
  float x[8];
  unpack8(raw, x);
  for (int s = 0; s < n_old; ++s)
    if ((mask >> s) & 1u) apply_stream8<__nv_bfloat16, BITS>(side.s[s], j, elem, d, group, x);
  v_old = (mask & ((1u << n_old) - 1u)) ? pack8(x) : raw;
  v_new = v_old;
  if ((mask >> n_old) & 1u) {
    apply_stream8<__nv_bfloat16, BITS>(side.s[n_old], j, elem, d, group, x);
    v_new = pack8(x);
  }
}

// chunk ci of the partitioned column list: plain chunks first, then patched chunks
struct ChunkInfo {
  int off;      // offset into the ordered column list
  int n_valid;  // valid columns (<= kNC)
  bool patch;   // columns carry a payload in the current loop: separate old / new operand tiles (two slots)
};
__device__ __forceinline__ ChunkInfo chunk_info(int ci, int n_plain, int n_patch) {
  const int n_plain_chunks = (n_plain + kNC - 1) / kNC;
  ChunkInfo c;
  if (ci < n_plain_chunks) {
    c.off = ci * kNC;
    c.n_valid = min(kNC, n_plain - c.off);
    c.patch = false;
  } else {
    const int k = ci - n_plain_chunks;
    c.off = n_plain + k * kNC;
    c.n_valid = min(kNC, n_patch - k * kNC);
    c.patch = true;
  }
  return c;
}

template <int BITS>
__global__ void __launch_bounds__(kThreads, 1) loop_attn_tc_kernel(const __grid_constant__ TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_old_tile = smem;
  uint8_t* q_new_tile = smem + kQTileBytes;
  uint8_t* ring = smem + 2 * kQTileBytes;
  TcSmemCtl& ctl = *reinterpret_cast<TcSmemCtl*>(ring + kSlots * kSlotBytes);
  int32_t* ord_col = reinterpret_cast<int32_t*>(&ctl + 1);               // [kMaxCols] column positions, partitioned
  uint32_t* ord_mask = reinterpret_cast<uint32_t*>(ord_col + kMaxCols);  // bit s: payload in stream s

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.x, h = blockIdx.y;
  const size_t prob = (size_t)h * a.nb + b;
  const int32_t* cols = a.col_idx + prob * a.c;
  const int cnt = min(__ldg(a.col_cnt + prob), kMaxCols);

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) {
      tc::mbar_init(&ctl.full[s], kProducerThreads);
      tc::mbar_init(&ctl.done[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&ctl.s_full[s], 1);
      tc::mbar_init(&ctl.p_full[s], kSoftmaxWarps * 32);
    }
    tc::mbar_init(&ctl.acc_done, 1);
    ctl.abort_flag = 0;
    tc::fence_barrier_init();
  }
  // ---- rows of this block: 32-ary searches in the ascending active list (warps 0 and 1) ----------------
  if (warp < 2) {
    const int target = warp == 0 ? b * a.q_block : min(a.L, (b + 1) * a.q_block);
    const int r = lower_bound32(a.active_idx, a.n_active, target, lane);
    if (lane == 0) { if (warp == 0) ctl.q_lo = r; else ctl.q_hi = r; }
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
  const int q_lo = ctl.q_lo, q_hi = ctl.q_hi;
  if (q_hi > q_lo) {   // CTA-uniform: blocks without active rows only release the tensor memory
  // ---- column list of the block: causal prefix, stream masks, stable partition -------------------------
  {
    const int i_last = __ldg(a.active_idx + q_hi - 1);            // last active row of the block
    const int span = ((cnt + kWarps - 1) / kWarps + 31) & ~31;     // contiguous span per warp, multiple of 32
    const int beg = warp * span, end = min(cnt, beg + span);
    int n0 = 0, n1 = 0;                                            // plain / patched columns in this warp's span
    for (int base = beg; base < end; base += 32) {
      const int u = base + lane;
      const int j = u < end ? __ldg(cols + u) : INT32_MAX;
      const bool live = j <= i_last;
      const bool patched = live && __ldg(a.k.s[a.n_old].slot + j) >= 0;
      n0 += __popc(__ballot_sync(0xffffffffu, live && !patched));
      n1 += __popc(__ballot_sync(0xffffffffu, patched));
    }
    if (lane == 0) { ctl.warp_cnt[warp][0] = n0; ctl.warp_cnt[warp][1] = n1; }
    __syncthreads();
    int before0 = 0, before1 = 0, tot0 = 0, tot1 = 0;
    for (int wv = 0; wv < kWarps; ++wv) {
      const int c0 = ctl.warp_cnt[wv][0], c1 = ctl.warp_cnt[wv][1];
      if (wv < warp) { before0 += c0; before1 += c1; }
      tot0 += c0; tot1 += c1;
    }
    if (tid == 0) { ctl.n_plain = tot0; ctl.n_patch = tot1; }
    for (int base = beg; base < end; base += 32) {
      const int u = base + lane;
      const int j = u < end ? __ldg(cols + u) : INT32_MAX;
      const bool live = j <= i_last;
      uint32_t mask = 0;
      if (live)
        for (int s = 0; s <= a.n_old; ++s) mask |= (__ldg(a.k.s[s].slot + j) >= 0 ? 1u : 0u) << s;
      const bool patched = live && ((mask >> a.n_old) & 1u);
      const uint32_t m0 = __ballot_sync(0xffffffffu, live && !patched);
      const uint32_t m1 = __ballot_sync(0xffffffffu, patched);
      const uint32_t lt = (1u << lane) - 1;
      if (live) {
        const int dst = patched ? tot0 + before1 + __popc(m1 & lt) : before0 + __popc(m0 & lt);
        ord_col[dst] = j;
        ord_mask[dst] = mask;
      }
      before0 += __popc(m0);
      before1 += __popc(m1);
    }
    __syncthreads();
  }
  const int n_plain = ctl.n_plain, n_patch = ctl.n_patch;
  const int n_chunks = (n_plain + kNC - 1) / kNC + (n_patch + kNC - 1) / kNC;
  int g = 0;    // chunks issued so far (all tiles): S/P buffer = g & 1, phase = (g >> 1) & 1
  int fill = 0; // ring slots filled so far: slot = fill % kSlots, phase = (fill / kSlots) & 1

  for (int s0 = q_lo, tile = 0; s0 < q_hi; s0 += kM, ++tile) {
  const int n_rows = min(kM, q_hi - s0);
  const int g0 = g, fill0 = fill;

  if (warp > kMmaWarp) {
    // =========================================== producers ===========================================
    const int pt = tid - (kMmaWarp + 1) * 32;
    const int pw = pt >> 5;
    // Q tiles (once per tile): asynchronous copies, part of the first commit group
    for (int it = pt; it < 2 * kM * 16; it += kProducerThreads) {
      const int which = it / (kM * 16);
      const int rem = it % (kM * 16);
      const int r = rem >> 4, ch = rem & 15;
      uint8_t* dst = (which ? q_new_tile : q_old_tile) + (ch >> 3) * (kM * 128) + tc::sw128_offset(r, ch & 7);
      if (r < n_rows)
        tc::cp_async16(dst, (which ? a.q_new : a.q_old) + (size_t)(s0 + r) * a.d + h * kDH + ch * 8);
      else
        *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
    }
    const int half = lane >> 4;          // 0: K row, 1: V row
    const int ch = lane & 15;            // 16-byte chunk inside the 256-byte row
    const DevSide& side = half ? a.v : a.k;
    const int elem = h * kDH + ch * 8;
    const __nv_bfloat16* base_rows = static_cast<const __nv_bfloat16*>(side.base) + elem;
    const uint32_t ch_off = (ch >> 3) * (kNC * 128);
    // Software pipeline over chunks, kAhead chunks of asynchronous gathers in flight per thread:
    //   issue(ci)   : wait until the chunk's ring slot(s) are free, start the 16-byte copies of the base rows
    //                 (warp pw owns columns pw, pw + 7, ...; lanes 0-15 the K row, lanes 16-31 the V row)
    //   finish(ci)  : wait for those copies, overwrite the columns that carry residual payloads with their
    //                 dequantize-and-add result, publish the column positions, hand the slot(s) to the MMA warp
    // At most kAhead chunks are in flight, and never more slots than the ring has (a chunk that still waits to
    // be finished must not hold a slot the next issue needs).
    constexpr int kAhead = 2;
    int f_issue = fill0, f_fin = fill0;
    int ci_issue = 0, ci_fin = 0;
    bool ok = true;
#pragma unroll 1
    while (ci_fin < n_chunks && ok) {
      bool can_issue = ci_issue < n_chunks && ci_issue - ci_fin < kAhead;
      if (can_issue) {
        // A slot is released by PV(y) of the chunk y that held it, and the MMA warp issues PV(y) only after
        // QK(y+1), i.e. after chunk y+1 has been handed over: chunk y+1 must be finished before we wait.
        const ChunkInfo nk = chunk_info(ci_issue, n_plain, n_patch);
        const int n_plain_chunks = (n_plain + kNC - 1) / kNC;
        auto holder = [&](int fill_no) {   // chunk (of this tile) that filled the same slot one lap earlier
          const int rel = fill_no - kSlots - fill0;
          if (rel < 0) return -1;
          return rel < n_plain_chunks ? rel : n_plain_chunks + (rel - n_plain_chunks) / 2;
        };
        int hmax = holder(f_issue);
        if (nk.patch) hmax = max(hmax, holder(f_issue + 1));
        can_issue = f_issue + (nk.patch ? 2 : 1) - f_fin <= kSlots && (hmax < 0 || ci_fin >= hmax + 2);
      }
      if (can_issue) {
        const int ci = ci_issue;
        const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
        const int slot0 = f_issue % kSlots, slot1 = (f_issue + 1) % kSlots;
        if (pt == 0) TC_TRACE(0, ci, 0);
        if (f_issue >= kSlots) ok = warp_wait(&ctl.done[slot0], ((f_issue / kSlots) - 1) & 1, abort_flag);
        if (ok && ck.patch && f_issue + 1 >= kSlots)
          ok = warp_wait(&ctl.done[slot1], (((f_issue + 1) / kSlots) - 1) & 1, abort_flag);
        if (!ok) break;
        if (pt == 0) TC_TRACE(0, ci, 1);
        uint8_t* t_old = ring + slot0 * kSlotBytes + half * kTileBytes + ch_off;
        uint8_t* t_new = ring + slot1 * kSlotBytes + half * kTileBytes + ch_off;
#pragma unroll 2
        for (int u = pw; u < kNC; u += kProducerWarps) {
          const uint32_t off = tc::sw128_offset(u, ch & 7);
          if (u < ck.n_valid) {
            const __nv_bfloat16* src = base_rows + (size_t)ord_col[ck.off + u] * a.d;
            tc::cp_async16(t_old + off, src);
            if (ck.patch) tc::cp_async16(t_new + off, src);
          } else {
            *reinterpret_cast<uint4*>(t_old + off) = make_uint4(0, 0, 0, 0);
            if (ck.patch) *reinterpret_cast<uint4*>(t_new + off) = make_uint4(0, 0, 0, 0);
          }
        }
        tc::cp_async_commit();
        f_issue += ck.patch ? 2 : 1;
        ++ci_issue;
      } else {
        const int cf = ci_fin;
        // groups complete in order: all but the (ci_issue - cf - 1) newer ones must have landed
        if (ci_issue - cf - 1 >= 1) tc::cp_async_wait<1>(); else tc::cp_async_wait<0>();
        const ChunkInfo ck = chunk_info(cf, n_plain, n_patch);
        const int slot0 = f_fin % kSlots, slot1 = (f_fin + 1) % kSlots;
        uint8_t* t_old = ring + slot0 * kSlotBytes + half * kTileBytes + ch_off;
        uint8_t* t_new = ring + slot1 * kSlotBytes + half * kTileBytes + ch_off;
        for (int u = pt; u < kNC; u += kProducerThreads)
          ctl.col_pos[slot0][u] = u < ck.n_valid ? ord_col[ck.off + u] : INT32_MAX;
        if (pt == 0) ctl.col_last[slot0] = ck.n_valid == kNC ? ord_col[ck.off + kNC - 1] : INT32_MAX;
#pragma unroll 1
        for (int u = pw; u < ck.n_valid; u += kProducerWarps) {
          const uint32_t mask = ord_mask[ck.off + u];
          if (mask == 0) continue;
          const int j = ord_col[ck.off + u];
          const uint4 base16 = __ldg(reinterpret_cast<const uint4*>(base_rows + (size_t)j * a.d));
          uint4 v_old, v_new;
          patch_piece<BITS>(side, a.n_old, mask, j, elem, a.d, a.group, base16, v_old, v_new);
          const uint32_t off = tc::sw128_offset(u, ch & 7);
          *reinterpret_cast<uint4*>(t_old + off) = v_old;
          if (ck.patch) *reinterpret_cast<uint4*>(t_new + off) = v_new;
        }
        if (pt == 0) TC_TRACE(0, cf, 2);
        tc::fence_proxy_async_smem();
        tc::mbar_arrive(&ctl.full[slot0]);
        if (ck.patch) tc::mbar_arrive(&ctl.full[slot1]);
        f_fin += ck.patch ? 2 : 1;
        ++ci_fin;
        if (pt == 0) TC_TRACE(0, cf, 3);
      }
    }
    tc::cp_async_wait<0>();
  } else if (warp == kMmaWarp) {
    // =========================================== MMA issuer ==========================================
    if (lane == 0) {
      const uint32_t idesc_qk = tc::make_idesc_bf16(kM, kNC, false);
      const uint32_t idesc_pv = tc::make_idesc_bf16(kM, kDH, true);
      // Descriptors differ only in their start-address field (bits 0-13, units of 16 bytes), so a step along
      // K is one 64-bit add. K-major operands (Q, Khat): 32 bytes per 16-element K step inside a 64-element
      // slab, then the next slab. MN-major Vhat: 16 key rows = two 1024-byte row groups per K step.
      const uint64_t q_old_desc = tc::make_desc_sw128(tc::smem_u32(q_old_tile), 16, 1024);
      const uint64_t q_new_desc = tc::make_desc_sw128(tc::smem_u32(q_new_tile), 16, 1024);
      const uint64_t k_desc0 = tc::make_desc_sw128(tc::smem_u32(ring), 16, 1024);
      const uint64_t v_desc0 = tc::make_desc_sw128(tc::smem_u32(ring) + kTileBytes, kNC * 128, 1024);
      bool ok = true;
      int f = fill0;        // slot counter of the chunk whose QK is issued next
      int f_pv = fill0;     // slot counter of the chunk whose PV is issued next
      // iteration ci issues QK(ci) and then PV(ci-1): the softmax of chunk ci-1 overlaps QK(ci)
#pragma unroll 1
      for (int ci = 0; ci <= n_chunks && ok; ++ci) {
        if (ci < n_chunks) {
          const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
          const int slot0 = f % kSlots, slot1 = (f + 1) % kSlots;
          TC_TRACE(1, ci, 0);
          if (!tc::mbar_wait(&ctl.full[slot0], (f / kSlots) & 1, abort_flag)) { ok = false; break; }
          if (ck.patch && !tc::mbar_wait(&ctl.full[slot1], ((f + 1) / kSlots) & 1, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          TC_TRACE(1, ci, 1);
          const uint64_t k_old = k_desc0 + (uint64_t)(slot0 * (kSlotBytes >> 4));
          const uint64_t k_new = ck.patch ? k_desc0 + (uint64_t)(slot1 * (kSlotBytes >> 4)) : k_old;
          const int sbuf = (g0 + ci) & 1;
          const uint32_t s_old = tmem + kSBase + sbuf * 128, s_new = s_old + 64;
#pragma unroll
          for (int kk = 0; kk < kDH / 16; ++kk)
            tc::mma_ss(s_old, q_old_desc + (uint64_t)(((kk >> 2) * (kM * 128) + (kk & 3) * 32) >> 4),
                       k_old + (uint64_t)(((kk >> 2) * (kNC * 128) + (kk & 3) * 32) >> 4), idesc_qk, kk > 0);
#pragma unroll
          for (int kk = 0; kk < kDH / 16; ++kk)
            tc::mma_ss(s_new, q_new_desc + (uint64_t)(((kk >> 2) * (kM * 128) + (kk & 3) * 32) >> 4),
                       k_new + (uint64_t)(((kk >> 2) * (kNC * 128) + (kk & 3) * 32) >> 4), idesc_qk, kk > 0);
          tc::mma_commit(&ctl.s_full[sbuf]);
          f += ck.patch ? 2 : 1;
          TC_TRACE(1, ci, 2);
        }
        if (ci >= 1) {
          const int cj = ci - 1;
          const ChunkInfo ck = chunk_info(cj, n_plain, n_patch);
          const int sbuf = (g0 + cj) & 1;
          if (!tc::mbar_wait(&ctl.p_full[sbuf], ((g0 + cj) >> 1) & 1, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          const int slot0 = f_pv % kSlots, slot1 = (f_pv + 1) % kSlots;
          const uint64_t v_old = v_desc0 + (uint64_t)(slot0 * (kSlotBytes >> 4));
          const uint64_t v_new = ck.patch ? v_desc0 + (uint64_t)(slot1 * (kSlotBytes >> 4)) : v_old;
          const uint32_t p_old = tmem + kSBase + sbuf * 128, p_new = p_old + 64;
#pragma unroll
          for (int kk = 0; kk < kNC / 16; ++kk)
            tc::mma_ts(tmem + kAccOld, p_old + kk * 8, v_old + (uint64_t)(kk * (2048 >> 4)), idesc_pv, cj > 0 || kk > 0);
#pragma unroll
          for (int kk = 0; kk < kNC / 16; ++kk)
            tc::mma_ts(tmem + kAccNew, p_new + kk * 8, v_new + (uint64_t)(kk * (2048 >> 4)), idesc_pv, cj > 0 || kk > 0);
          tc::mma_commit(&ctl.done[slot0]);
          if (ck.patch) tc::mma_commit(&ctl.done[slot1]);
          f_pv += ck.patch ? 2 : 1;
          TC_TRACE(1, cj, 3);
        }
      }
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
    int f = fill0, f_prev = fill0;
    for (int ci = 0; ci < n_chunks; ++ci) {
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      const int gc = g0 + ci;
      const int sbuf = gc & 1;
      const int slot0 = f % kSlots;
      if ((tid & 127) == 0) TC_TRACE(2 + grp, ci, 0);
      // full[] first: orders the producers' column-position writes before the reads below
      if (!warp_wait(&ctl.full[slot0], (f / kSlots) & 1, abort_flag) ||
          !warp_wait(&ctl.s_full[sbuf], (gc >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      if ((tid & 127) == 0) TC_TRACE(2 + grp, ci, 1);
      const uint32_t s_addr = tmem + lane_base + kSBase + sbuf * 128 + grp * 64;
      const int* cp = ctl.col_pos[slot0];
      // rows of a warp that lie at or after every column of the chunk need no causal mask
      const bool unmasked = __all_sync(0xffffffffu, row_ok && ctl.col_last[slot0] <= pos);
      // The loops over the 64 logits are rolled (16 columns per step) to keep the instruction footprint of the
      // three concurrently running roles small.
      float sub;                                         // exponent offset of this chunk: p = 2^(s * c2 - sub)
      if (grp == 0) {
        sub = lse2;
      } else {
        float cm = -INFINITY;                            // row maximum (first of two passes over the S region)
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
          uint32_t r[16];
          tc::tmem_ld16(s_addr + q * 16, r);
          tc::tmem_wait_ld();
          if (unmasked) {
#pragma unroll
            for (int u = 0; u < 16; ++u) cm = fmaxf(cm, __uint_as_float(r[u]));
          } else {
#pragma unroll
            for (int u = 0; u < 16; ++u)
              if (cp[q * 16 + u] <= pos) cm = fmaxf(cm, __uint_as_float(r[u]));
          }
        }
        cm *= c2;                                        // c2 > 0: scaling commutes with the maximum
        float factor = 1.f;
        bool need = false;
        if (ref == -INFINITY) {
          ref = cm;                                      // first causal column(s) of this row: accumulator row is still zero
        } else if (cm - ref > kRescaleThreshold) {
          factor = tc::ex2(ref - cm);
          ref = cm;
          need = true;
        }
        if (__any_sync(0xffffffffu, need)) {
          // lazy rescale of acc_new (rare): every earlier PV must have completed before the rows are rewritten
          if (ci >= 1) {
            if (!warp_wait(&ctl.done[f_prev % kSlots], (f_prev / kSlots) & 1, abort_flag)) { ok = false; break; }
            tc::tc_fence_after();
          }
          ell *= factor;
#pragma unroll 1
          for (int q4 = 0; q4 < 8; ++q4) {
            uint32_t acc[16];
            tc::tmem_ld16(tmem + lane_base + kAccNew + q4 * 16, acc);
            tc::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * factor);
            tc::tmem_st16(tmem + lane_base + kAccNew + q4 * 16, acc);
          }
          tc::tmem_wait_st();
        }
        sub = ref == -INFINITY ? 0.f : ref;
      }
      // exponentials, row sum, bf16 packing. P (bf16, 32 columns) overwrites the first half of the 64-column
      // S region: step q consumes S[16q, 16q+16) and then stores P[8q, 8q+8), which never reaches unread S.
      float sum = 0.f;
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        uint32_t r[16], p[8];
        tc::tmem_ld16(s_addr + q * 16, r);
        tc::tmem_wait_ld();
        if (unmasked) {
#pragma unroll
          for (int u = 0; u < 16; u += 2) {
            const float p0 = tc::ex2(fmaf(__uint_as_float(r[u]), c2, -sub));
            const float p1 = tc::ex2(fmaf(__uint_as_float(r[u + 1]), c2, -sub));
            sum += p0 + p1;
            p[u >> 1] = tc::pack_bf16(p0, p1);
          }
        } else {
#pragma unroll
          for (int u = 0; u < 16; u += 2) {
            const float p0 = cp[q * 16 + u] <= pos ? tc::ex2(fmaf(__uint_as_float(r[u]), c2, -sub)) : 0.f;
            const float p1 = cp[q * 16 + u + 1] <= pos ? tc::ex2(fmaf(__uint_as_float(r[u + 1]), c2, -sub)) : 0.f;
            sum += p0 + p1;
            p[u >> 1] = tc::pack_bf16(p0, p1);
          }
        }
        tc::tmem_st8(s_addr + q * 8, p);
      }
      if (grp == 0) mass += sum; else ell += sum;
      tc::tmem_wait_st();
      if ((tid & 127) == 0) TC_TRACE(2 + grp, ci, 2);
      tc::tc_fence_before();
      tc::mbar_arrive(&ctl.p_full[sbuf]);
      f_prev = f + (ck.patch ? 1 : 0);     // last slot of this chunk: its done[] marks the completion of PV(ci)
      f += ck.patch ? 2 : 1;
      if ((tid & 127) == 0) TC_TRACE(2 + grp, ci, 3);
    }
    // ---- epilogue ------------------------------------------------------------------------------------
    if (ok) ok = warp_wait(&ctl.acc_done, tile & 1, abort_flag);
    tc::tc_fence_after();
    if (grp == 0) ctl.mass[row] = mass;
    else { ctl.ell[row] = ell; ctl.ref[row] = ref; }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const float m_i = ctl.mass[row], l_i = ctl.ell[row], ref_i = ctl.ref[row];
    const bool acc_valid = ok && n_chunks > 0;            // warp-uniform: the tensor-memory reads below are collective
    const bool has = acc_valid && ref_i > -INFINITY;      // per row: T_i is not empty
    const float w = has ? m_i / l_i : 0.f;
#pragma unroll 1
    for (int hh = 0; hh < 4; ++hh) {
      // each group finishes 64 of the 128 head-dim columns, 16 at a time
      const int col0 = grp * 64 + hh * 16;
      uint32_t ao[16], an[16];
      if (acc_valid) {
        tc::tmem_ld16(tmem + lane_base + kAccOld + col0, ao);
        tc::tmem_ld16(tmem + lane_base + kAccNew + col0, an);
        tc::tmem_wait_ld();
      }
      if (!row_ok) continue;
      const size_t off = (size_t)(s0 + row) * a.d + h * kDH + col0;
      if (has) {
#pragma unroll
        for (int v8 = 0; v8 < 2; ++v8) {
          float prev[8], out[8];
          load8<__nv_bfloat16>(a.o_prev + off + v8 * 8, prev);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            out[i] = prev[i] - __uint_as_float(ao[v8 * 8 + i]) + w * __uint_as_float(an[v8 * 8 + i]);
          store8<__nv_bfloat16>(a.o_out + off + v8 * 8, out);
        }
      } else if (a.o_out != a.o_prev) {
#pragma unroll
        for (int v8 = 0; v8 < 2; ++v8)
          *reinterpret_cast<uint4*>(a.o_out + off + v8 * 8) = *reinterpret_cast<const uint4*>(a.o_prev + off + v8 * 8);
      }
    }
    if (grp == 1 && row_ok)
      a.lse_out[(size_t)h * a.L + pos] = has ? (ref_i + log2f(l_i)) * kLn2 - logf(m_i) : lse_prev;
  }
  // every role is done with this tile: accumulators, Q tiles and the ring bookkeeping move on together
  g += n_chunks;
  fill += (n_plain + kNC - 1) / kNC + 2 * ((n_patch + kNC - 1) / kNC);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  if (ctl.abort_flag) break;
  }  // tiles of the block
  }  // block has active rows
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
#ifndef FL_TC_TRACE
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
#endif
}

}  // namespace

// Returns FL_ERR_UNSUPPORTED when the tensor path does not cover the request (caller falls back to the
// SIMT kernel, which is also CUDA).
int fl_launch_loop_attn_tc(const fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_old,
                           const int32_t* active_idx, int n_active, const fl_kv_store* store, const int32_t* col_idx,
                           const int32_t* col_cnt, int c, const float* lse_prev, float* lse_out, const void* o_prev,
                           void* o_out, int32_t* status, cudaStream_t st) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH || c > kMaxCols) return FL_ERR_UNSUPPORTED;
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
  const dim3 grid(a.nb, s->n_heads);   // one CTA per (query block, head); it walks the block's 128-row tiles
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
