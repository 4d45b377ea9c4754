// Stages 2 + 4 on the Blackwell tensor path: the attention replacement of Eq. 7 for one (query block,
// head) per CTA, with K/V of the selected columns gathered from the bf16 base and patched with the
// dequantized residual streams (Eq. 8) on their way into shared memory.
//
// Warp roles (16 warps, 512 threads):
//   warps 0-3   softmax of the OLD term  (fixed normaliser lse_prev: p_old = exp(s_old - lse_prev), mass m_i)
//   warps 4-7   softmax of the NEW term  (running reference with lazy rescale of the accumulator)
//   warp  8     one thread issues the S = Q Khat^T MMAs; the warp owns the tensor-memory allocation
//   warp  9     one thread issues the acc += P Vhat MMAs (a single thread cannot issue 64-column MMAs as fast
//               as the tensor pipe retires them; two issuers keep it fed)
//   warps 10-13 TMA: row gathers (cp.async.bulk.tensor tile::gather4, 4 selected columns per copy) of the bf16
//               base K/V rows straight into 128B-swizzled operand tiles; completion on mbarriers
//   warps 14-15 patch: stage the Q tiles; for the columns that carry residual payloads, overwrite the gathered
//               base rows with the dequantize-and-add result (Eq. 8)
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
constexpr int kPvWarp = 9;         // second MMA issuer (the first, kMmaWarp, issues QK^T)
constexpr int kTmaWarp = 10;       // first of the TMA warps
constexpr int kTmaWarps = 4;       // a single warp cannot issue four-row gathers fast enough; four come close
constexpr int kPatchWarps = 2;
constexpr int kWarps = kSoftmaxWarps + 2 + kTmaWarps + kPatchWarps;  // 16
constexpr int kThreads = kWarps * 32;
constexpr int kPatchThreads = kPatchWarps * 32;
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

struct alignas(64) TcArgs {
  CUtensorMap k_map, v_map;   // row-gather maps of the K / V base ([L, d] bf16, box 64 x 1, 128B swizzle)
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
  uint64_t landed[kSlots];   // TMA -> everyone: the slot's gathered tiles (32 KB) have arrived
  uint64_t patched[kSlots];  // patch warps -> MMA: residual-carrying columns of the slot are rewritten (dirty chunks only)
  uint64_t done[kSlots];     // MMA -> TMA / softmax: the MMAs that read the slot have finished
  uint64_t q_full;           // patch warps -> MMA: the Q tiles of the current row tile are staged
  uint64_t s_full[2];      // MMA -> softmax: S of the chunk is in tensor memory
  uint64_t p_full[2];      // softmax -> MMA: P of the chunk is in tensor memory
  uint64_t s_free[2];      // PV issuer -> QK issuer: the PV MMAs that read P from the buffer have finished
  uint64_t acc_done;       // MMA -> softmax: all accumulation of the tile finished
  uint32_t tmem_base;
  int abort_flag;
  int q_lo, q_hi;          // block's slot range in active_idx
  int n_plain, n_patch;    // columns without / with a payload in the current loop
  int warp_cnt[kWarps][2];
  int col_pos[kSlots][kNC];
  int col_last[kSlots];    // largest column position of the chunk, INT32_MAX if the chunk is padded
  uint32_t chunk_mask[kMaxCols / kNC + 2];  // OR of the stream masks of the chunk's columns (0: plain gather only)
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

// chunk ci of the partitioned column list: patched chunks first (the first two are built by the whole CTA
// before the pipeline starts), then plain chunks. In the ordered list the plain columns come first.
struct ChunkInfo {
  int off;      // offset into the ordered column list
  int n_valid;  // valid columns (<= kNC)
  bool patch;   // columns carry a payload in the current loop: separate old / new operand tiles (two slots)
};
__device__ __forceinline__ ChunkInfo chunk_info(int ci, int n_plain, int n_patch) {
  const int n_patch_chunks = (n_patch + kNC - 1) / kNC;
  ChunkInfo c;
  if (ci < n_patch_chunks) {
    c.off = n_plain + ci * kNC;
    c.n_valid = min(kNC, n_patch - ci * kNC);
    c.patch = true;
  } else {
    const int k = ci - n_patch_chunks;
    c.off = k * kNC;
    c.n_valid = min(kNC, n_plain - c.off);
    c.patch = false;
  }
  return c;
}
constexpr int kPrefillChunks = 2;   // patched chunks the whole CTA builds at the start of a row tile (4 ring slots)

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
      tc::mbar_init(&ctl.landed[s], kTmaWarps);
      tc::mbar_init(&ctl.patched[s], kPatchWarps);
      tc::mbar_init(&ctl.done[s], 1);
    }
    tc::mbar_init(&ctl.q_full, kPatchThreads);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&ctl.s_full[s], 1);
      tc::mbar_init(&ctl.p_full[s], kSoftmaxWarps * 32);
      tc::mbar_init(&ctl.s_free[s], 1);
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
    for (int i = tid; i < kMaxCols / kNC + 2; i += kThreads) ctl.chunk_mask[i] = 0;
    __syncthreads();
    const int patch_chunks = (tot1 + kNC - 1) / kNC;
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
        if (mask != 0) atomicOr(&ctl.chunk_mask[patched ? (dst - tot0) / kNC : patch_chunks + dst / kNC], mask);
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
  uint32_t dirty_par_cta = 0;  // per-slot phase parity of the patched[] barriers (they only see dirty chunks)

  for (int s0 = q_lo, tile = 0; s0 < q_hi; s0 += kM, ++tile) {
  const int n_rows = min(kM, q_hi - s0);
  const int g0 = g, fill0 = fill;
  const uint32_t dirty_par0 = dirty_par_cta;
  const int n_pre = min((n_patch + kNC - 1) / kNC, kPrefillChunks);
  // ---- the first patched chunks are built by all 512 threads straight into the (idle) ring: base row plus
  // dequantized residuals (Eq. 8), old and new operand tiles. Left to the two patch warps this would take an
  // order of magnitude longer than a plain chunk; done here it costs a few dependent loads per thread.
  {
#pragma unroll 2
    for (int p = tid; p < n_pre * kNC * 32; p += kThreads) {
      const int pc = p / (kNC * 32), q = p % (kNC * 32);
      const int u = q >> 5, half = (q >> 4) & 1, ch = q & 15;
      const ChunkInfo ck = chunk_info(pc, n_plain, n_patch);
      const int slot0 = (fill0 + 2 * pc) % kSlots, slot1 = (fill0 + 2 * pc + 1) % kSlots;
      const uint32_t off = half * kTileBytes + (ch >> 3) * (kNC * 128) + tc::sw128_offset(u, ch & 7);
      uint4 v_old = make_uint4(0, 0, 0, 0), v_new = make_uint4(0, 0, 0, 0);
      if (u < ck.n_valid) {
        const DevSide& side = half ? a.v : a.k;
        const int j = ord_col[ck.off + u];
        const int elem = h * kDH + ch * 8;
        const uint4 base16 =
            __ldg(reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(side.base) + (size_t)j * a.d + elem));
        patch_piece<BITS>(side, a.n_old, ord_mask[ck.off + u], j, elem, a.d, a.group, base16, v_old, v_new);
      }
      *reinterpret_cast<uint4*>(ring + slot0 * kSlotBytes + off) = v_old;
      *reinterpret_cast<uint4*>(ring + slot1 * kSlotBytes + off) = v_new;
    }
    for (int p = tid; p < n_pre * kNC; p += kThreads) {
      const int pc = p / kNC, u = p % kNC;
      const ChunkInfo ck = chunk_info(pc, n_plain, n_patch);
      const int slot0 = (fill0 + 2 * pc) % kSlots;
      ctl.col_pos[slot0][u] = u < ck.n_valid ? ord_col[ck.off + u] : INT32_MAX;
      if (u == 0) ctl.col_last[slot0] = ck.n_valid == kNC ? ord_col[ck.off + kNC - 1] : INT32_MAX;
    }
    tc::fence_proxy_async_smem();
    __syncthreads();
  }

  if (warp >= kTmaWarp && warp < kTmaWarp + kTmaWarps) {
    // ============================================== TMA ==============================================
    // In-order fills of the ring; the lookahead is whatever the four slots allow. The 64 four-row gathers
    // of a slot (K: 2 slabs x 16 groups, V: the same) are split over the TMA warps, 16 each, one per lane;
    // every warp announces its own share of the bytes on the slot's barrier.
    const int tw = warp - kTmaWarp;
    const int is_v = tw >> 1, slab = tw & 1, grp = lane & 15;
    const void* map = is_v ? static_cast<const void*>(&a.v_map) : static_cast<const void*>(&a.k_map);
    int f = fill0;
    bool ok = true;
#pragma unroll 1
    for (int ci = 0; ci < n_chunks && ok; ++ci) {
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      const int n_slots = ck.patch ? 2 : 1;
      if (ci < n_pre) {   // built by the whole CTA above: only the barrier phase is left to complete
        if (lane == 0)
          for (int k = 0; k < n_slots; ++k) tc::mbar_arrive(&ctl.landed[(f + k) % kSlots]);
        f += n_slots;
        continue;
      }
      for (int k = 0; k < n_slots && ok; ++k)
        if (f + k >= kSlots) ok = warp_wait(&ctl.done[(f + k) % kSlots], (((f + k) / kSlots) - 1) & 1, abort_flag);
      if (!ok) break;
      const int slot0 = f % kSlots;
      if (tid == kTmaWarp * 32) TC_TRACE(0, ci, 0);
      if (tw == 0) {
        for (int u = lane; u < kNC; u += 32) ctl.col_pos[slot0][u] = u < ck.n_valid ? ord_col[ck.off + u] : INT32_MAX;
        if (lane == 0) ctl.col_last[slot0] = ck.n_valid == kNC ? ord_col[ck.off + kNC - 1] : INT32_MAX;
      }
      __syncwarp();
      if (lane == 0)
        for (int k = 0; k < n_slots; ++k) tc::mbar_arrive_expect_tx(&ctl.landed[(f + k) % kSlots], kSlotBytes / kTmaWarps);
      __syncwarp();
      if (lane < 16) {
        int y[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int u = grp * 4 + i;
          y[i] = u < ck.n_valid ? ord_col[ck.off + u] : a.L;   // row L is outside the tensor: reads as zero
        }
        for (int k = 0; k < n_slots; ++k) {
          const int slot = (f + k) % kSlots;
          tc::tma_gather4(ring + slot * kSlotBytes + is_v * kTileBytes + slab * (kNC * 128) + grp * 512, map,
                          &ctl.landed[slot], h * kDH + slab * 64, y[0], y[1], y[2], y[3]);
        }
      }
      f += n_slots;
      if (tid == kTmaWarp * 32) TC_TRACE(0, ci, 1);
    }
  } else if (warp >= kTmaWarp + kTmaWarps) {
    // ============================================= patch =============================================
    const int pt = tid - (kTmaWarp + kTmaWarps) * 32;   // 0..95
    const int pw = pt >> 5;
    // Q tiles (once per row tile): asynchronous 16-byte copies
    for (int it = pt; it < 2 * kM * 16; it += kPatchThreads) {
      const int which = it / (kM * 16);
      const int rem = it % (kM * 16);
      const int r = rem >> 4, ch = rem & 15;
      uint8_t* dst = (which ? q_new_tile : q_old_tile) + (ch >> 3) * (kM * 128) + tc::sw128_offset(r, ch & 7);
      if (r < n_rows)
        tc::cp_async16(dst, (which ? a.q_new : a.q_old) + (size_t)(s0 + r) * a.d + h * kDH + ch * 8);
      else
        *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
    }
    tc::cp_async_commit();
    tc::cp_async_wait<0>();
    tc::fence_proxy_async_smem();
    tc::mbar_arrive(&ctl.q_full);
    // dirty chunks: lanes 0-15 own the K row, lanes 16-31 the V row of one column at a time
    const int half = lane >> 4, ch = lane & 15;
    const DevSide& side = half ? a.v : a.k;
    const int elem = h * kDH + ch * 8;
    const __nv_bfloat16* base_rows = static_cast<const __nv_bfloat16*>(side.base) + elem;
    const uint32_t ch_off = (ch >> 3) * (kNC * 128);
    int f = fill0;
    uint32_t dirty_par = dirty_par0;     // bit s: parity of the dirty fills slot s has seen
    bool ok = true;
#pragma unroll 1
    for (int ci = 0; ci < n_chunks && ok; ++ci) {
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      const int n_slots = ck.patch ? 2 : 1;
      // Every fill is waited for, clean chunks included: a parity wait is only meaningful for the phase in
      // progress, so a waiter must never skip a phase of a barrier it will wait on again.
      for (int k = 0; k < n_slots && ok; ++k)
        ok = warp_wait(&ctl.landed[(f + k) % kSlots], ((f + k) / kSlots) & 1, abort_flag);
      if (!ok) break;
      if (ctl.chunk_mask[ci] != 0) {
        uint8_t* t_old = ring + (f % kSlots) * kSlotBytes + half * kTileBytes + ch_off;
        uint8_t* t_new = ring + ((f + 1) % kSlots) * kSlotBytes + half * kTileBytes + ch_off;
        if (ci >= n_pre)
#pragma unroll 1
        for (int u = pw; u < ck.n_valid; u += kPatchWarps) {
          const uint32_t mask = ord_mask[ck.off + u];
          if (mask == 0) continue;
          const int j = ord_col[ck.off + u];
          const uint4 base16 = __ldg(reinterpret_cast<const uint4*>(base_rows + (size_t)j * a.d));
          uint4 v_old, v_new;
          patch_piece<BITS>(side, a.n_old, mask, j, elem, a.d, a.group, base16, v_old, v_new);
          const uint32_t off = tc::sw128_offset(u, ch & 7);
          if (mask & ((1u << a.n_old) - 1u)) *reinterpret_cast<uint4*>(t_old + off) = v_old;
          if (ck.patch) *reinterpret_cast<uint4*>(t_new + off) = v_new;
        }
        tc::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0)
          for (int k = 0; k < n_slots; ++k) tc::mbar_arrive(&ctl.patched[(f + k) % kSlots]);
        for (int k = 0; k < n_slots; ++k) dirty_par ^= 1u << ((f + k) % kSlots);
      }
      f += n_slots;
    }
  } else if (warp == kMmaWarp) {
    // ========================================= QK^T issuer ==========================================
    if (lane == 0) {
      const uint32_t idesc_qk = tc::make_idesc_bf16(kM, kNC, false);
      // Descriptors differ only in their start-address field (bits 0-13, units of 16 bytes): the low word
      // moves (no carry into the other fields: shared memory is < 256 KB), the high word stays.
      // K-major operands (Q, Khat): 32 bytes per 16-element K step inside a 64-element slab, then the next slab.
      const uint64_t q_old_desc = tc::make_desc_sw128(tc::smem_u32(q_old_tile), 16, 1024);
      const uint64_t q_new_desc = tc::make_desc_sw128(tc::smem_u32(q_new_tile), 16, 1024);
      const uint64_t k_desc0 = tc::make_desc_sw128(tc::smem_u32(ring), 16, 1024);
      const uint32_t kq_hi = (uint32_t)(k_desc0 >> 32);
      const uint32_t q_old_lo = (uint32_t)q_old_desc, q_new_lo = (uint32_t)q_new_desc, k_lo0 = (uint32_t)k_desc0;
      int f = fill0;
      uint32_t dirty_par = dirty_par0;
#pragma unroll 1
      for (int ci = 0; ci < n_chunks; ++ci) {
        const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
        const int slot0 = f % kSlots, slot1 = (f + 1) % kSlots;
        const int gc = g0 + ci, sbuf = gc & 1;
        TC_TRACE(1, ci, 0);
        if (ci == 0 && !tc::mbar_wait(&ctl.q_full, tile & 1, abort_flag)) break;
        if (!tc::mbar_wait(&ctl.landed[slot0], (f / kSlots) & 1, abort_flag)) break;
        if (ck.patch && !tc::mbar_wait(&ctl.landed[slot1], ((f + 1) / kSlots) & 1, abort_flag)) break;
        if (ctl.chunk_mask[ci] != 0) {       // residual-carrying columns are rewritten by the patch warps
          if (!tc::mbar_wait(&ctl.patched[slot0], (dirty_par >> slot0) & 1, abort_flag)) break;
          dirty_par ^= 1u << slot0;
          if (ck.patch) {
            if (!tc::mbar_wait(&ctl.patched[slot1], (dirty_par >> slot1) & 1, abort_flag)) break;
            dirty_par ^= 1u << slot1;
          }
        }
        // the S buffer still holds P of chunk gc-2 until the PV MMAs that read it have retired
        if (gc >= 2 && !tc::mbar_wait(&ctl.s_free[sbuf], ((gc >> 1) - 1) & 1, abort_flag)) break;
        TC_TRACE(1, ci, 1);
        const uint32_t k_old = k_lo0 + slot0 * (kSlotBytes >> 4);
        const uint32_t k_new = ck.patch ? k_lo0 + slot1 * (kSlotBytes >> 4) : k_old;
        const uint32_t s_old = tmem + kSBase + sbuf * 128, s_new = s_old + 64;
#define FL_QK(D, QLO, KLO, KK, ACC)                                                                          \
  tc::mma_ss_lo<ACC>(D, (QLO) + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), kq_hi,                    \
                     (KLO) + ((((KK) >> 2) * (kNC * 128) + ((KK)&3) * 32) >> 4), kq_hi, idesc_qk)
        FL_QK(s_old, q_old_lo, k_old, 0, false); FL_QK(s_old, q_old_lo, k_old, 1, true);
        FL_QK(s_old, q_old_lo, k_old, 2, true);  FL_QK(s_old, q_old_lo, k_old, 3, true);
        FL_QK(s_old, q_old_lo, k_old, 4, true);  FL_QK(s_old, q_old_lo, k_old, 5, true);
        FL_QK(s_old, q_old_lo, k_old, 6, true);  FL_QK(s_old, q_old_lo, k_old, 7, true);
        FL_QK(s_new, q_new_lo, k_new, 0, false); FL_QK(s_new, q_new_lo, k_new, 1, true);
        FL_QK(s_new, q_new_lo, k_new, 2, true);  FL_QK(s_new, q_new_lo, k_new, 3, true);
        FL_QK(s_new, q_new_lo, k_new, 4, true);  FL_QK(s_new, q_new_lo, k_new, 5, true);
        FL_QK(s_new, q_new_lo, k_new, 6, true);  FL_QK(s_new, q_new_lo, k_new, 7, true);
#undef FL_QK
        tc::mma_commit(&ctl.s_full[sbuf]);
        f += ck.patch ? 2 : 1;
        TC_TRACE(1, ci, 2);
      }
    }
    __syncwarp();
  } else if (warp == kPvWarp) {
    // ========================================== P V issuer ==========================================
    if (lane == 0) {
      const uint32_t idesc_pv = tc::make_idesc_bf16(kM, kDH, true);
      // MN-major Vhat: 16 key rows = two 1024-byte row groups per K step
      const uint64_t v_desc0 = tc::make_desc_sw128(tc::smem_u32(ring) + kTileBytes, kNC * 128, 1024);
      const uint32_t v_hi = (uint32_t)(v_desc0 >> 32), v_lo0 = (uint32_t)v_desc0;
      int f = fill0;
#pragma unroll 1
      for (int cj = 0; cj < n_chunks; ++cj) {
        const ChunkInfo ck = chunk_info(cj, n_plain, n_patch);
        const int gc = g0 + cj, sbuf = gc & 1;
        if (!tc::mbar_wait(&ctl.p_full[sbuf], (gc >> 1) & 1, abort_flag)) break;
        tc::tc_fence_after();
        const int slot0 = f % kSlots, slot1 = (f + 1) % kSlots;
        const uint32_t v_old = v_lo0 + slot0 * (kSlotBytes >> 4);
        const uint32_t v_new = ck.patch ? v_lo0 + slot1 * (kSlotBytes >> 4) : v_old;
        const uint32_t p_old = tmem + kSBase + sbuf * 128, p_new = p_old + 64;
        const uint32_t acc0 = cj > 0 ? 1u : 0u;          // first chunk of the tile overwrites the accumulators
#pragma unroll
        for (int kk = 0; kk < kNC / 16; ++kk)
          tc::mma_ts_lo(tmem + kAccOld, p_old + kk * 8, v_old + kk * (2048 >> 4), v_hi, idesc_pv, kk > 0 ? 1u : acc0);
#pragma unroll
        for (int kk = 0; kk < kNC / 16; ++kk)
          tc::mma_ts_lo(tmem + kAccNew, p_new + kk * 8, v_new + kk * (2048 >> 4), v_hi, idesc_pv, kk > 0 ? 1u : acc0);
        tc::mma_commit(&ctl.done[slot0]);
        if (ck.patch) tc::mma_commit(&ctl.done[slot1]);
        tc::mma_commit(&ctl.s_free[sbuf]);
        f += ck.patch ? 2 : 1;
        TC_TRACE(1, cj, 3);
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
      // landed[] first: orders the TMA warp's column-position writes before the reads below
      if (!warp_wait(&ctl.landed[slot0], (f / kSlots) & 1, abort_flag) ||
          !warp_wait(&ctl.s_full[sbuf], (gc >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      if ((tid & 127) == 0) TC_TRACE(2 + grp, ci, 1);
      const uint32_t s_addr = tmem + lane_base + kSBase + sbuf * 128 + grp * 64;
      const int* cp = ctl.col_pos[slot0];
      // rows of a warp that lie at or after every column of the chunk need no causal mask
      const bool unmasked = __all_sync(0xffffffffu, row_ok && ctl.col_last[slot0] <= pos);
      // One pass over the 64 logits of the row: load them, form p = 2^(s * c2 - sub) in place and pack to bf16.
      // For the new term `sub` is the running reference; the chunk maximum is tracked on the side, and only if
      // some row of the warp has no reference yet or would overflow (its maximum beats the reference by more
      // than the threshold) does the warp take the slow path: fix the reference, rescale, recompute. The S
      // region is still intact at that point because P is stored last.
      uint32_t r[64];
      tc::tmem_ld32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
      tc::tmem_ld32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
      tc::tmem_wait_ld();
      float sub = grp == 0 ? lse2 : (ref == -INFINITY ? 0.f : ref);
      float cm = -INFINITY, sum = 0.f;
      bool stored = false;                               // warp-uniform: the slow path stores P itself
      if (unmasked) {
#pragma unroll
        for (int u = 0; u < 64; u += 2) {
          const float t0 = __uint_as_float(r[u]), t1 = __uint_as_float(r[u + 1]);
          cm = fmaxf(cm, fmaxf(t0, t1));
          const float p0 = tc::ex2(fmaf(t0, c2, -sub)), p1 = tc::ex2(fmaf(t1, c2, -sub));
          sum += p0 + p1;
          r[u >> 1] = tc::pack_bf16(p0, p1);
        }
      } else {
#pragma unroll
        for (int u = 0; u < 64; u += 2) {
          const float t0 = cp[u] <= pos ? __uint_as_float(r[u]) : -INFINITY;
          const float t1 = cp[u + 1] <= pos ? __uint_as_float(r[u + 1]) : -INFINITY;
          cm = fmaxf(cm, fmaxf(t0, t1));
          const float p0 = tc::ex2(fmaf(t0, c2, -sub)), p1 = tc::ex2(fmaf(t1, c2, -sub));
          sum += p0 + p1;
          r[u >> 1] = tc::pack_bf16(p0, p1);
        }
      }
      if (grp == 1) {
        cm *= c2;                                        // c2 > 0: scaling commutes with the maximum
        const bool first = ref == -INFINITY && cm > -INFINITY;
        const bool over = ref > -INFINITY && cm - ref > kRescaleThreshold;
        if (__any_sync(0xffffffffu, first || over)) {
          // ---- slow path (first chunk of a row, or a reference that fell too far behind) -----------------
          float factor = 1.f;
          if (first) ref = cm;                           // accumulator row is still zero: nothing to rescale
          if (over) { factor = tc::ex2(ref - cm); ref = cm; }
          if (__any_sync(0xffffffffu, over)) {
            // every earlier PV must have completed before the accumulator rows are rewritten
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
          sum = 0.f;
#pragma unroll 1
          for (int q = 0; q < 4; ++q) {                  // recompute P from the untouched S region
            uint32_t t[16];
            tc::tmem_ld16(s_addr + q * 16, t);
            tc::tmem_wait_ld();
#pragma unroll
            for (int u = 0; u < 16; u += 2) {
              const bool m0 = unmasked || cp[q * 16 + u] <= pos, m1 = unmasked || cp[q * 16 + u + 1] <= pos;
              const float p0 = m0 ? tc::ex2(fmaf(__uint_as_float(t[u]), c2, -sub)) : 0.f;
              const float p1 = m1 ? tc::ex2(fmaf(__uint_as_float(t[u + 1]), c2, -sub)) : 0.f;
              sum += p0 + p1;
              t[u >> 1] = tc::pack_bf16(p0, p1);
            }
            // S[16q, 16q+16) is consumed; P[8q, 8q+8) never reaches unread S
            tc::tmem_st8(s_addr + q * 8, *reinterpret_cast<uint32_t(*)[8]>(&t[0]));
          }
          stored = true;
        }
      }
      if (grp == 0) mass += sum; else ell += sum;
      // P (bf16, 32 columns) overwrites the first half of the 64-column S region, all of which was consumed
      if (!stored) tc::tmem_st32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
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
  {
    int f = fill;
    for (int ci = 0; ci < n_chunks; ++ci) {   // replay the tile's fills (same for every role)
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      const int n_slots = ck.patch ? 2 : 1;
      if (ctl.chunk_mask[ci] != 0)
        for (int k = 0; k < n_slots; ++k) dirty_par_cta ^= 1u << ((f + k) % kSlots);
      f += n_slots;
    }
    fill = f;
  }
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
int fl_launch_loop_attn_tc(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_old,
                           const int32_t* active_idx, int n_active, const fl_kv_store* store, const int32_t* col_idx,
                           const int32_t* col_cnt, int c, const float* lse_prev, float* lse_out, const void* o_prev,
                           void* o_out, int32_t* status, cudaStream_t st) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH || c > kMaxCols) return FL_ERR_UNSUPPORTED;
  if ((size_t)ctx->max_smem_optin < kTcSmemBytes) return FL_ERR_UNSUPPORTED;
  TcArgs a{};
  if (!fl_row_gather_tmap(ctx, store->k_base, s->L, (int64_t)s->n_heads * s->head_dim, &a.k_map) ||
      !fl_row_gather_tmap(ctx, store->v_base, s->L, (int64_t)s->n_heads * s->head_dim, &a.v_map))
    return FL_ERR_UNSUPPORTED;
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
