// Stages 2 + 4 on the Blackwell tensor path, one TERM of the attention replacement (Eq. 7) per launch.
//
// Eq. 7 adds two sums over the selected columns T_i of a row: minus the old term (the previous loop's probabilities
// times the previous loop's values) plus the new term (the cached mass times a local softmax of the new logits, times
// the new values). They share nothing but the row's previous output, so they can be computed by two launches that
// hand over one row of storage-type numbers and one binary32 number per (head, row):
//   OLD pass:  p_j = exp(sm_scale q_old . Khat^(r-1)_j - lse_prev);  m_i = sum p_j;  B_i = o_prev_i - sum p_j Vhat^(r-1)_j
//              -> writes B_i (the row's background) and m_i
//   NEW pass:  p_j = m_i softmax_{T_i}(sm_scale q_new . Khat^(r)_j);  o_i = B_i + sum p_j Vhat^(r)_j;
//              lse_i = logsumexp_{T_i} - log m_i     -> writes o_i, lse_i and the new Q rows
// While the column sets stay what they were, later loops need the NEW pass only (the old term of loop r is the new
// term of loop r-1, so B_i and m_i carry over).
//
// A CTA computes one (query block, head) problem with ONE pipeline, which leaves room for two CTAs per SM (half the
// shared memory, half the tensor memory, 256 threads each): the second CTA's gathers, MMAs and exponentials fill the
// gaps that the dependent chain  QK^T -> exponentials -> PV  leaves in the first one's, and one CTA's prologue and
// epilogue run under the other's main loop. (cudaOccupancyMaxActiveBlocksPerMultiprocessor answers 1 for any kernel
// that allocates tensor memory; two CTAs of 256 columns each do run side by side.) What bounds the pair is the rate
// at which an SM's TMA unit takes four-row gathers: a 32 KB chunk per ~1.3 k cycles with eight issuing warps.
//
// Warp roles (9 warps): 0-3 softmax (one row of the 128-row tile per thread), 4 the MMA issuer (one thread), 5-8 TMA:
// the Q tile, then per chunk of 64 columns the K tile and the V tile, each gathered four rows per copy
// (cp.async.bulk.tensor tile::gather4) into 128B-swizzled operand tiles. K and V have rings of their own (two tiles
// each): a K tile is free again as soon as its QK^T has completed, long before the chunk's PV.
// Columns that are active in this loop are gathered from the rows fl_quant_kv_residual materialized (before the
// loop's residual for the OLD pass, after it for the NEW pass); this kernel requires them. Columns that carry a
// payload from an earlier loop only (token sets that shrink) are rebuilt in place by the TMA warps (Eq. 8 chain).
// Tensor memory (256 columns): accumulator 0-127, two S / P buffers of 64 columns (P, bf16, is written over the first
// half of the S buffer it was computed from).
// Every mbarrier wait is bounded; on a timeout the CTA raises a flag, drains and reports FL_ERR_TIMEOUT.
#include "tc_attn_common.cuh"

namespace {

using namespace fl_tc;

constexpr int kSmWarps = 4;
constexpr int kIssueWarp = 4;
constexpr int kTmaWarp = 5;
constexpr int kTmaWarps = 4;
constexpr int kWarps = 9;
constexpr int kThreads = kWarps * 32;
constexpr int kColWarps = 7;                   // warps that read the column list in the prologue (the other two search rows)
constexpr int kMaxCols = 3072;
constexpr int kMaxChunks = kMaxCols / kNC + 2;
constexpr int kTileGathers = kTileBytes / 512; // 32 four-row gathers of 128-byte rows fill a K or V tile
constexpr uint32_t kAcc = 0, kS = 128;         // tensor-memory columns
constexpr uint32_t kTmemCols = 256;
static_assert(3 * kMaxCols * 4 <= 4 * kTileBytes, "prologue staging must fit in the K and V rings");

enum { kOldPass = 0, kNewPass = 1 };

struct alignas(64) StArgs {
  CUtensorMap k_map, v_map;            // row-gather maps of the K / V base ([L, d] bf16, box 64 x 1, 128B swizzle)
  CUtensorMap k_rows_map, v_rows_map;  // row-gather maps of the loop's materialized rows ([n_active, d])
  CUtensorMap q_map;                   // NEW: tile map of the compact new Q rows (box 64 x 128); OLD: row-gather map of the Q store
  const __nv_bfloat16* rows_in;        // [L, d] by position. OLD: previous outputs; NEW: backgrounds
  __nv_bfloat16* rows_out;             // [L, d] by position. OLD: backgrounds; NEW: outputs
  float* mass;                         // [H, L]: written by the OLD pass, read by the NEW pass
  const float* lse_prev;               // [H, L]: OLD pass (required); NEW pass: copied to lse_out for rows with empty T_i, or null
  float* lse_out;                      // NEW pass
  const __nv_bfloat16* q_new;          // NEW pass: compact new Q rows, copied into q_store at the end
  __nv_bfloat16* q_store;              // NEW pass: Q store [L, d] that receives them, or null
  const int32_t* active_idx;
  int n_active;
  DevSide k, v;
  int n_old;                           // streams contained in Xhat^(r-1); stream index n_old is loop r's own
  const int32_t* col_idx;
  const int32_t* col_cnt;
  int c;
  int32_t* status;
  int L, H, q_block, nb, d, group;
  float scale;
};

struct __align__(16) StSmemCtl {
  uint64_t q_full;          // TMA -> issuer: the Q tile of the current row tile has arrived
  uint64_t k_landed[2];     // TMA -> issuer: the K tile of the chunk has arrived
  uint64_t v_landed[2];     // TMA -> issuer: the V tile
  uint64_t patched[2];      // TMA warps -> issuer: stale columns of the chunk's tiles are rebuilt (dirty chunks only)
  uint64_t s_full[2];       // issuer -> softmax, TMA: S of the chunk is in tensor memory (and its K tile is free)
  uint64_t p_full[2];       // softmax -> issuer: P of the chunk is in tensor memory
  uint64_t p_free[2];       // issuer -> issuer, TMA: the PV MMAs of the chunk have finished (S buffer and V tile free)
  uint64_t acc_done;        // issuer -> softmax: all accumulation of the tile finished
  uint32_t tmem_base;
  int abort_flag;
  int q_lo, q_hi, i_last;
  int n_plain, n_patch;
  int warp_cnt[kWarps][2];
  int chunk_last[kMaxChunks];        // largest column position of the chunk, INT32_MAX if the chunk is padded
  uint32_t stale[kMaxCols / 32];     // bit u: ordered column u carries a payload from an earlier loop only
};

constexpr size_t kStSmemBytes = 1024 /* alignment slack */ + kQTileBytes + 4 * kTileBytes + sizeof(StSmemCtl) +
                                kMaxCols * sizeof(int32_t);
static_assert(2 * (kStSmemBytes + 1024) <= 233472, "two CTAs share an SM's 228 KB of shared memory");

template <int BITS, int MODE>
__global__ void __launch_bounds__(kThreads, 2) loop_attn_stream_kernel(const __grid_constant__ StArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_tile = smem;
  uint8_t* k_ring = smem + kQTileBytes;                 // two K tiles
  uint8_t* v_ring = k_ring + 2 * kTileBytes;            // two V tiles
  StSmemCtl& ctl = *reinterpret_cast<StSmemCtl*>(v_ring + 2 * kTileBytes);
  int32_t* ord_col = reinterpret_cast<int32_t*>(&ctl + 1);   // [kMaxCols] column positions: plain ones, then patched ones

  fl_grid_wait();      // nothing below runs ahead of the previous kernel of the stream
  fl_grid_release();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // problem (query block b, head h): every chunk of a first-block problem needs the causal mask, which makes them the
  // longest jobs: they come first
  const int item = blockIdx.x;
  int b, h;
  if (a.nb == 1) { b = 0; h = item; }
  else if (item < a.H) { b = 0; h = item; }
  else { h = (item - a.H) / (a.nb - 1); b = 1 + (item - a.H) % (a.nb - 1); }
  const size_t prob = (size_t)h * a.nb + b;
  const int32_t* cols = a.col_idx + prob * a.c;
  const int cnt = min(__ldg(a.col_cnt + prob), kMaxCols);

  if (tid == 0) {
    tc::mbar_init(&ctl.q_full, 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&ctl.k_landed[s], kTmaWarps);
      tc::mbar_init(&ctl.v_landed[s], kTmaWarps);
      tc::mbar_init(&ctl.patched[s], kTmaWarps);
      tc::mbar_init(&ctl.s_full[s], 1);
      tc::mbar_init(&ctl.p_full[s], kSmWarps);
      tc::mbar_init(&ctl.p_free[s], 1);
    }
    tc::mbar_init(&ctl.acc_done, 1);
    ctl.abort_flag = 0;
    tc::fence_barrier_init();
  }
  for (int i = tid; i < kMaxCols / 32; i += kThreads) ctl.stale[i] = 0u;
  // ---- prologue: the raw column list, a flag per column and the rows of the block ------------------------------
  int32_t* raw_col = reinterpret_cast<int32_t*>(k_ring);                   // [kMaxCols], staged in the idle rings
  uint32_t* raw_flag = reinterpret_cast<uint32_t*>(raw_col + kMaxCols);    // bit 0: payload in this loop, bit 1: in an earlier one
  const int c_cap = min(a.c, kMaxCols);
  if (warp >= kColWarps) {
    const int target = warp == kColWarps ? b * a.q_block : min(a.L, (b + 1) * a.q_block);
    int below;
    const int r = lower_bound_warp(a.active_idx, a.n_active, target, lane, &below);
    if (lane == 0) {
      if (warp == kColWarps) ctl.q_lo = r;
      else { ctl.q_hi = r; ctl.i_last = r > 0 ? below : -1; }
    }
  } else {
    // the whole row of the column table is read without waiting for its count (entries past the count are -1); the
    // thread that read a column looks it up in the slot map of every residual stream
    constexpr int kBatch = 3, kStride = kColWarps * 32;
#pragma unroll 1
    for (int u0 = tid; u0 < c_cap; u0 += kBatch * kStride) {
      int j[kBatch];
      uint32_t flag[kBatch];
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        j[k] = u0 + k * kStride < c_cap ? __ldg(cols + u0 + k * kStride) : -1;
        flag[k] = 0;
      }
#pragma unroll 1
      for (int sg = 0; sg <= a.n_old; sg += 4) {
        int sl[kBatch][4];
#pragma unroll
        for (int k = 0; k < kBatch; ++k)
#pragma unroll
          for (int q = 0; q < 4; ++q)
            sl[k][q] = (j[k] >= 0 && sg + q <= a.n_old) ? __ldg(a.k.s[sg + q].slot + j[k]) : -1;
#pragma unroll
        for (int k = 0; k < kBatch; ++k)
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (sl[k][q] >= 0) flag[k] |= (sg + q == a.n_old) ? 1u : 2u;
      }
#pragma unroll
      for (int k = 0; k < kBatch; ++k)
        if (u0 + k * kStride < c_cap) {
          raw_col[u0 + k * kStride] = j[k];
          raw_flag[u0 + k * kStride] = flag[k];
        }
    }
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
  const int q_lo = ctl.q_lo, q_hi = ctl.q_hi;
  if (q_hi > q_lo) {   // CTA-uniform: blocks without active rows only release the tensor memory
  {
    // causal prefix, stable partition into plain / patched columns: every warp owns a contiguous span
    const int i_last = ctl.i_last;
    const int span = ((cnt + kWarps - 1) / kWarps + 31) & ~31;
    const int beg = warp * span, end = min(cnt, beg + span);
    int n0 = 0, n1 = 0;
#pragma unroll 1
    for (int base = beg; base < end; base += 32) {
      const int u = base + lane;
      const bool live = u < end && raw_col[u] <= i_last;
      const bool patched = live && (raw_flag[u] & 1u);
      n0 += __popc(__ballot_sync(0xffffffffu, live && !patched));
      n1 += __popc(__ballot_sync(0xffffffffu, patched));
    }
    if (lane == 0) { ctl.warp_cnt[warp][0] = n0; ctl.warp_cnt[warp][1] = n1; }
    __syncthreads();
    int inc0 = lane < kWarps ? ctl.warp_cnt[lane][0] : 0, inc1 = lane < kWarps ? ctl.warp_cnt[lane][1] : 0;
#pragma unroll
    for (int off = 1; off < kWarps; off <<= 1) {
      const int t0 = __shfl_up_sync(0xffffffffu, inc0, off), t1 = __shfl_up_sync(0xffffffffu, inc1, off);
      if (lane >= off) { inc0 += t0; inc1 += t1; }
    }
    const int tot0 = __shfl_sync(0xffffffffu, inc0, kWarps - 1), tot1 = __shfl_sync(0xffffffffu, inc1, kWarps - 1);
    const int up0 = __shfl_sync(0xffffffffu, inc0, (warp + 31) & 31), up1 = __shfl_sync(0xffffffffu, inc1, (warp + 31) & 31);
    int before0 = warp > 0 ? up0 : 0, before1 = warp > 0 ? up1 : 0;
    if (tid == 0) { ctl.n_plain = tot0; ctl.n_patch = tot1; }
    const uint32_t lt = (1u << lane) - 1;
#pragma unroll 1
    for (int base = beg; base < end; base += 32) {
      const int u = base + lane;
      const int j = u < end ? raw_col[u] : INT32_MAX;
      const uint32_t flag = u < end ? raw_flag[u] : 0u;
      const bool live = j <= i_last;
      const bool patched = live && (flag & 1u);
      const uint32_t m0 = __ballot_sync(0xffffffffu, live && !patched);
      const uint32_t m1 = __ballot_sync(0xffffffffu, patched);
      if (live) {
        const int dst = patched ? tot0 + before1 + __popc(m1 & lt) : before0 + __popc(m0 & lt);
        ord_col[dst] = j;
        if (!patched && (flag & 2u)) atomicOr(&ctl.stale[dst >> 5], 1u << (dst & 31));
      }
      before0 += __popc(m0);
      before1 += __popc(m1);
    }
    __syncthreads();
  }
  const int n_plain = ctl.n_plain, n_patch = ctl.n_patch;
  const int n_chunks = (n_plain + kNC - 1) / kNC + (n_patch + kNC - 1) / kNC;
  for (int ci = tid; ci < n_chunks; ci += kThreads) {
    const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
    ctl.chunk_last[ci] = ck.n_valid == kNC ? ord_col[ck.off + kNC - 1] : INT32_MAX;
  }
  __syncthreads();
  // plain chunks start at multiples of 64 in the ordered list: two words of the stale bit map per chunk
  auto chunk_dirty = [&](const ChunkInfo& ck) -> bool {
    return !ck.patch && (ctl.stale[ck.off >> 5] | ctl.stale[(ck.off >> 5) + 1]) != 0u;
  };
  int g = 0;                    // chunks issued so far (all tiles): buffers = g & 1, one phase of their barriers per use
  uint32_t dirty_par_cta = 0;   // per-slot phase parity of the patched[] barriers (they only see dirty chunks)

  for (int s0 = q_lo, tile = 0; s0 < q_hi; s0 += kM, ++tile) {
  const int n_rows = min(kM, q_hi - s0);
  const int g0 = g;
  const uint32_t dirty_par0 = dirty_par_cta;
  if (warp == kTmaWarp) {
    if (MODE == kNewPass) {
      // Q tile of this row tile: two 64-element slabs; rows past the compact list read as zero, rows of the next
      // block (past n_rows) are computed and dropped
      if (lane == 0) {
        tc::mbar_arrive_expect_tx(&ctl.q_full, kQTileBytes);
        tc::tma_tile2d(q_tile, &a.q_map, &ctl.q_full, h * kDH, s0);
        tc::tma_tile2d(q_tile + kM * 128, &a.q_map, &ctl.q_full, h * kDH + 64, s0);
      }
    } else {
      // the previous loop's Q rows come from the store: four-row gathers by position, one group of rows per lane
      if (lane == 0) tc::mbar_arrive_expect_tx(&ctl.q_full, kQTileBytes);
      __syncwarp();
      int y[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = lane * 4 + i;
        y[i] = r < n_rows ? __ldg(a.active_idx + s0 + r) : a.L;   // row L is outside the tensor: reads as zero
      }
      tc::tma_gather4(q_tile + lane * 512, &a.q_map, &ctl.q_full, h * kDH, y[0], y[1], y[2], y[3]);
      tc::tma_gather4(q_tile + kM * 128 + lane * 512, &a.q_map, &ctl.q_full, h * kDH + 64, y[0], y[1], y[2], y[3]);
    }
  }

  if (warp >= kTmaWarp) {
    // ========================================== TMA + patch ==========================================
    // Per chunk n, in this order: the K tile of chunk n + 1 (its ring slot is free once QK^T of chunk n - 1 has
    // completed), then the V tile of chunk n (free once PV of chunk n - 2 has completed: V is needed a whole softmax
    // later than K). The 32 four-row gathers of a tile (2 slabs x 16 groups) are dealt round robin to the warps, one
    // per lane; every warp announces its own share of the bytes on the tile's barrier.
    const int tw = warp - kTmaWarp;
    const int req = lane * kTmaWarps + tw;
    const int my_reqs = (kTileGathers - 1 - tw) / kTmaWarps + 1;     // requests of this warp per tile (lanes 0 .. my_reqs - 1)
    const int slab = (req >> 4) & 1, grp = req & 15;
    const int half = lane >> 4, ch = lane & 15;
    const DevSide& side = half ? a.v : a.k;
    const int elem = h * kDH + ch * 8;
    const __nv_bfloat16* base_rows = static_cast<const __nv_bfloat16*>(side.base) + elem;
    const uint32_t ch_off = (ch >> 3) * (kNC * 128);
    bool ok = true;
    // gather one tile (is_v: V, else K) of chunk ci into ring slot (gc & 1)
    auto fill = [&](int ci, int gc, bool is_v) {
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      uint64_t* bar = is_v ? &ctl.v_landed[gc & 1] : &ctl.k_landed[gc & 1];
      if (lane == 0) tc::mbar_arrive_expect_tx(bar, my_reqs * 512);
      __syncwarp();
      if (req < kTileGathers) {
        int y[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int u = grp * 4 + i;
          // a row past the end of the tensor reads as zero. Columns that are active in this loop come from the
          // materialized rows, indexed by their row in the loop's stream
          if (ck.patch) y[i] = u < ck.n_valid ? __ldg(a.k.s[a.n_old].slot + ord_col[ck.off + u]) : a.n_active;
          else y[i] = u < ck.n_valid ? ord_col[ck.off + u] : a.L;
        }
        const void* src = ck.patch ? (is_v ? static_cast<const void*>(&a.v_rows_map) : static_cast<const void*>(&a.k_rows_map))
                                   : (is_v ? static_cast<const void*>(&a.v_map) : static_cast<const void*>(&a.k_map));
        uint8_t* dst = (is_v ? v_ring : k_ring) + (gc & 1) * kTileBytes + slab * (kNC * 128) + grp * 512;
        tc::tma_gather4(dst, src, bar, h * kDH + slab * 64, y[0], y[1], y[2], y[3]);
      }
    };
    const int n_mine = n_chunks;
    if (n_mine > 0) {
      if (g0 >= 2) ok = warp_wait(&ctl.s_full[g0 & 1], ((g0 >> 1) - 1) & 1, abort_flag);
      if (ok) fill(0, g0, false);
    }
#pragma unroll 1
    for (int ci = 0; ci < n_mine && ok; ++ci) {
      const int gc = g0 + ci;
      if (ci + 1 < n_mine) {
        if (gc + 1 >= 2) ok = warp_wait(&ctl.s_full[(gc + 1) & 1], (((gc + 1) >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        fill(ci + 1, gc + 1, false);
      }
      if (gc >= 2) ok = warp_wait(&ctl.p_free[gc & 1], ((gc >> 1) - 1) & 1, abort_flag);
      if (!ok) break;
      fill(ci, gc, true);
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      if (chunk_dirty(ck)) {
        // stale columns: their tiles hold base rows; the rows after the earlier loops' residuals take their place
        // (lanes 0-15 the K row, lanes 16-31 the V row, one column per warp at a time)
        ok = warp_wait(&ctl.k_landed[gc & 1], (gc >> 1) & 1, abort_flag) &&
             warp_wait(&ctl.v_landed[gc & 1], (gc >> 1) & 1, abort_flag);
        if (!ok) break;
        uint8_t* tile = (half ? v_ring : k_ring) + (gc & 1) * kTileBytes + ch_off;
#pragma unroll 1
        for (int u = tw; u < ck.n_valid; u += kTmaWarps) {
          const int ou = ck.off + u;
          if (!((ctl.stale[ou >> 5] >> (ou & 31)) & 1u)) continue;
          const int j = ord_col[ou];
          float x[8];
          unpack8(__ldg(reinterpret_cast<const uint4*>(base_rows + (size_t)j * a.d)), x);
#pragma unroll 1
          for (int s = 0; s < a.n_old; ++s) apply_stream8<__nv_bfloat16, BITS>(side.s[s], j, elem, a.d, a.group, x);
          *reinterpret_cast<uint4*>(tile + tc::sw128_offset(u, ch & 7)) = pack8(x);
        }
        tc::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&ctl.patched[gc & 1]);
      }
    }
    if (MODE == kNewPass && a.q_store != nullptr && ok) {
      // the new Q rows take their place in the Q store for the next loop (this pass reads no Q row from it)
      const int pt = tid - kTmaWarp * 32;
#pragma unroll 1
      for (int it = pt; it < n_rows * 16; it += kTmaWarps * 32) {
        const int r = it >> 4, c16 = it & 15;
        const int pos_r = __ldg(a.active_idx + s0 + r);
        *reinterpret_cast<uint4*>(a.q_store + (size_t)pos_r * a.d + h * kDH + c16 * 8) =
            __ldg(reinterpret_cast<const uint4*>(a.q_new + (size_t)(s0 + r) * a.d + h * kDH + c16 * 8));
      }
    }
  } else if (warp == kIssueWarp) {
    // ========================================== MMA issuer ===========================================
    // QK^T of chunk n (its S buffer is free once PV of chunk n - 2 has retired), then PV of chunk n - 1 (its P is
    // written while QK^T of chunk n executes).
    if (lane == 0) {
      const uint32_t idesc_qk = tc::make_idesc_bf16(kM, kNC, false);
      const uint32_t idesc_pv = tc::make_idesc_bf16(kM, kDH, true);
      const uint64_t q_desc = tc::make_desc_sw128(tc::smem_u32(q_tile), 16, 1024);
      const uint64_t k_desc0 = tc::make_desc_sw128(tc::smem_u32(k_ring), 16, 1024);
      const uint32_t kq_hi = (uint32_t)(k_desc0 >> 32);
      const uint32_t q_lo_w = (uint32_t)q_desc, k_lo0 = (uint32_t)k_desc0;
      // MN-major Vhat: 16 key rows = two 1024-byte row groups per K step
      const uint64_t v_desc0 = tc::make_desc_sw128(tc::smem_u32(v_ring), kNC * 128, 1024);
      const uint32_t v_hi = (uint32_t)(v_desc0 >> 32), v_lo0 = (uint32_t)v_desc0;
      const uint32_t s_base = tmem + kS, acc = tmem + kAcc;
      uint32_t dirty_par = dirty_par0;
#pragma unroll 1
      for (int n = 0; n <= n_chunks; ++n) {
        const int gc = g0 + n;
        if (n < n_chunks) {
          const int sl = gc & 1;
          if (n == 0 && !tc::mbar_wait(&ctl.q_full, tile & 1, abort_flag)) break;
          if (!tc::mbar_wait(&ctl.k_landed[sl], (gc >> 1) & 1, abort_flag)) break;
          if (chunk_dirty(chunk_info(n, n_plain, n_patch))) {
            if (!tc::mbar_wait(&ctl.patched[sl], (dirty_par >> sl) & 1, abort_flag)) break;
            dirty_par ^= 1u << sl;
          }
          // the S buffer holds P of the chunk before the previous one until its PV MMAs have read it
          if (gc >= 2 && !tc::mbar_wait(&ctl.p_free[sl], ((gc >> 1) - 1) & 1, abort_flag)) break;
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
          const int gp = gc - 1, pb = gp & 1;
          if (!tc::mbar_wait(&ctl.v_landed[pb], (gp >> 1) & 1, abort_flag)) break;
          if (!tc::mbar_wait(&ctl.p_full[pb], (gp >> 1) & 1, abort_flag)) break;
          tc::tc_fence_after();
          const uint32_t v_lo = v_lo0 + pb * (kTileBytes >> 4);
          const uint32_t p_src = s_base + pb * kNC;
          const uint32_t acc0 = n > 1 ? 1u : 0u;           // the tile's first chunk overwrites the accumulator
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
    const int pos = row_ok ? __ldg(a.active_idx + s0 + row) : -1;
    const float c2 = a.scale * kLog2e;
    const float lse2 = ((row_ok && MODE == kOldPass) ? a.lse_prev[(size_t)h * a.L + pos] : 0.f) * kLog2e;
    // the epilogue reads the row's previous output (NEW pass: its background): have it in L2 by then
    if (row_ok) {
      tc::prefetch_l2(a.rows_in + (size_t)pos * a.d + h * kDH);
      tc::prefetch_l2(a.rows_in + (size_t)pos * a.d + h * kDH + 64);
    }
    const uint32_t s_addr = tmem + lane_base + kS;
    float ell = 0.f, ref = -INFINITY;    // OLD pass: ell is the mass, ref stays unused
    bool ok = true;
    for (int ci = 0; ci < n_chunks; ++ci) {
      const int gc = g0 + ci, pb = gc & 1, n_use = gc >> 1;
      if (!warp_wait(&ctl.s_full[pb], n_use & 1, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      // rows of a warp that lie at or after every column of the chunk need no causal mask; rows beyond the
      // tile's last (their results are never stored) must not force the masked path
      const bool unmasked = __all_sync(0xffffffffu, !row_ok || ctl.chunk_last[ci] <= pos);
      int vis = kNC;
      if (!unmasked) {
        // the chunk's columns ascend: the visible ones are a prefix, found by bisection; the rest read as -inf
        const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
        const int32_t* cp = ord_col + ck.off;
        int lo = 0, hi = row_ok ? ck.n_valid : 0;
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (cp[mid] <= pos) lo = mid + 1; else hi = mid;
        }
        vis = lo;
      }
      // P goes over the first half of this S buffer: the first 32 logits are in registers before columns 0-15 are
      // stored, the second 32 (columns 32-63) before columns 16-31 are
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
        float sub = lse2;
        if (MODE == kNewPass) {
          // running reference: taken from the first columns that show a finite logit and moved (with a rescale of
          // the accumulator row) only when a maximum beats it by more than the threshold
          float cm = -INFINITY;
#pragma unroll
          for (int u = 0; u < 32; u += 2) cm = fmaxf(cm, fmaxf(__uint_as_float(r[u]), __uint_as_float(r[u + 1])));
          cm *= c2;                                        // c2 > 0: scaling commutes with the maximum
          const bool first = ref == -INFINITY && cm > -INFINITY;
          const bool over = ref > -INFINITY && cm - ref > kRescaleThreshold;
          if (first) ref = cm;                             // accumulator row is still zero: nothing to rescale
          if (__any_sync(0xffffffffu, over)) {
            float factor = 1.f;
            if (over) { factor = tc::ex2(ref - cm); ref = cm; }
            // every earlier PV must have completed before the accumulator rows are rewritten
            if (ci > 0) {
              if (!warp_wait(&ctl.p_free[(gc - 1) & 1], ((gc - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
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
              // the first half of this chunk's P was formed against the old reference: bring it along
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
          sub = ref == -INFINITY ? 0.f : ref;
        }
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
    // ---- epilogue ------------------------------------------------------------------------------------
    // The rows that come in (previous outputs / backgrounds) are staged in the Q tile (every QK^T has retired once
    // the last S arrived) with coalesced asynchronous copies, combined in place by the row-owning threads, and
    // written out coalesced again.
    uint8_t* stage = q_tile;                     // [128 rows][16 x 16 B], 16-byte cells XOR-swizzled by row
    const size_t col0 = (size_t)h * kDH;
    // a tile without a single chunk: nobody has waited for the Q tile, which is still on its way into this memory
    if (ok && n_chunks == 0) ok = warp_wait(&ctl.q_full, tile & 1, abort_flag);
    asm volatile("bar.sync 1, 128;" ::: "memory");    // every softmax warp is past its last S: no QK^T reads Q any more
#pragma unroll 1
    for (int k = 0; k < 16; ++k) {
      const int idx = k * 128 + tid, rr = idx >> 4, cc = idx & 15;
      if (rr < n_rows) {
        const size_t src_row = (size_t)__ldg(a.active_idx + s0 + rr);
        tc::cp_async16(stage + rr * 256 + ((cc ^ (rr & 7)) << 4), a.rows_in + src_row * a.d + col0 + cc * 8);
      }
    }
    tc::cp_async_commit();
    float m_i = MODE == kNewPass ? (row_ok ? a.mass[(size_t)h * a.L + pos] : 0.f) : ell;
    if (ok) ok = warp_wait(&ctl.acc_done, tile & 1, abort_flag);
    tc::tc_fence_after();
    tc::cp_async_wait<0>();
    asm volatile("bar.sync 1, 128;" ::: "memory");
    const bool valid = ok && n_chunks > 0;                 // warp-uniform: the tensor-memory reads below are collective
    bool has;                                              // per row: T_i is not empty
    float w;
    if (MODE == kNewPass) {
      has = valid && ref > -INFINITY && m_i > 0.f;
      w = has ? m_i / ell : 0.f;
    } else {
      has = valid && m_i > 0.f;
      w = -1.f;
    }
#pragma unroll 1
    for (int c16 = 0; c16 < 16; ++c16) {   // 8 head-dim columns = one 16-byte cell of the staged row at a time
      uint32_t av[8];
      if (valid) {
        tc::tmem_ld8(tmem + lane_base + kAcc + c16 * 8, av);
        tc::tmem_wait_ld();
      }
      if (has) {
        uint4* cell = reinterpret_cast<uint4*>(stage + row * 256 + ((c16 ^ (row & 7)) << 4));
        float pv[8];
        unpack8(*cell, pv);
#pragma unroll
        for (int i = 0; i < 8; ++i) pv[i] = pv[i] + w * __uint_as_float(av[i]);
        *cell = pack8(pv);
      }
    }
    if (row_ok) {
      if (MODE == kNewPass) {
        if (has) a.lse_out[(size_t)h * a.L + pos] = (ref + log2f(ell)) * kLn2 - logf(m_i);
        else if (a.lse_prev != nullptr) a.lse_out[(size_t)h * a.L + pos] = a.lse_prev[(size_t)h * a.L + pos];
      } else {
        a.mass[(size_t)h * a.L + pos] = has ? m_i : 0.f;
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll 1
    for (int k = 0; k < 16; ++k) {
      const int idx = k * 128 + tid, rr = idx >> 4, cc = idx & 15;
      if (rr < n_rows) {
        const size_t dst_row = (size_t)__ldg(a.active_idx + s0 + rr);
        *reinterpret_cast<uint4*>(a.rows_out + dst_row * a.d + col0 + cc * 8) =
            *reinterpret_cast<const uint4*>(stage + rr * 256 + ((cc ^ (rr & 7)) << 4));
      }
    }
  }
  // every role is done with this tile: accumulator, Q tile and the ring bookkeeping move on together
  if (s0 + kM < q_hi) {   // CTA-uniform: another row tile of the block follows
    for (int ci = 0; ci < n_chunks; ++ci)
      if (chunk_dirty(chunk_info(ci, n_plain, n_patch))) dirty_par_cta ^= 1u << ((g + ci) & 1);
    g += n_chunks;
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (ctl.abort_flag) break;
  }
  }  // tiles of the block
  }  // block has active rows
  // ---- teardown ------------------------------------------------------------------------------------------
  tc::tc_fence_before();
  __syncthreads();
  if (warp == kIssueWarp) {
    if (ctl.abort_flag) {
      // let outstanding tensor work drain (bounded) before the columns are released
      if (lane == 0) tc::mma_commit(&ctl.acc_done);
      __syncwarp();
      for (int it = 0; it < (1 << 16); ++it) __nanosleep(256);
    }
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

template <int MODE>
int launch_mode(fl_ctx* ctx, int bits, dim3 grid, const StArgs& a, cudaStream_t st) {
#define FL_ST(BITS)                                                                                              \
  do {                                                                                                           \
    auto kern = loop_attn_stream_kernel<BITS, MODE>;                                                             \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStSmemBytes));  \
    /* two CTAs per SM need the SM's whole shared memory: ask for the largest carve-out */                      \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,                    \
                                       (int)cudaSharedmemCarveoutMaxShared));                                   \
    FL_CHECK_CUDA(fl_launch(ctx, kern, grid, dim3(kThreads), kStSmemBytes, st, a));                             \
  } while (0)
  switch (bits) {
    case 2: FL_ST(2); break;
    case 4: FL_ST(4); break;
    case 8: FL_ST(8); break;
    default: FL_ST(16); break;
  }
#undef FL_ST
  return fl_launch_status();
}

}  // namespace

// Whether the single-term kernels can take the call: the loop's materialized rows must be there (the rows after the
// loop's residual for the new-term pass; those before it as well when the old-term pass runs).
bool fl_loop_attn_stream_covers(const fl_ctx* ctx, const fl_shape* s, int loop_r, int n_active,
                                const fl_kv_store* store, int c, bool old_pass) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH || c > kMaxCols) return false;
  if ((size_t)ctx->max_smem_optin < kStSmemBytes || ctx->encode_tiled == nullptr || ctx->tmaps == nullptr) return false;
  const fl_kv_stream& ks = store->k_res[loop_r - 2];
  const fl_kv_stream& vs = store->v_res[loop_r - 2];
  if (old_pass && (ks.rows_prev == nullptr || vs.rows_prev == nullptr)) return false;
  return ks.rows_cur != nullptr && vs.rows_cur != nullptr && ks.n_rows == n_active && n_active > 0;
}

// Position-indexed loop attention with the carried old term, as one or two single-term launches:
// carry->reuse == 0: OLD pass (writes carry->bg_store, carry->mass), then NEW pass; else the NEW pass alone.
int fl_launch_loop_attn_stream(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_store_in,
                               void* q_store_out, const int32_t* active_idx, int n_active, const fl_kv_store* store,
                               const int32_t* col_idx, const int32_t* col_cnt, int c, const float* lse_in,
                               float* lse_out, const void* o_store_in, void* o_store_out, const fl_attn_carry* carry,
                               int32_t* status, cudaStream_t st) {
  if (!fl_loop_attn_stream_covers(ctx, s, loop_r, n_active, store, c, carry->reuse == 0)) return FL_ERR_UNSUPPORTED;
  StArgs a{};
  const int64_t d_row = (int64_t)s->n_heads * s->head_dim;
  const fl_kv_stream& ks = store->k_res[loop_r - 2];
  const fl_kv_stream& vs = store->v_res[loop_r - 2];
  if (!fl_tile_tmap(ctx, store->k_base, s->L, d_row, 1, &a.k_map) ||
      !fl_tile_tmap(ctx, store->v_base, s->L, d_row, 1, &a.v_map))
    return FL_ERR_UNSUPPORTED;
  a.active_idx = active_idx; a.n_active = n_active;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.n_old = loop_r - 2;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.status = status;
  a.L = s->L; a.H = s->n_heads; a.q_block = s->q_block; a.nb = fl_n_blocks(s);
  a.d = s->n_heads * s->head_dim; a.group = s->group; a.scale = s->sm_scale;
  a.mass = carry->mass;
  const dim3 grid(a.nb * s->n_heads);
  if (!carry->reuse) {
    if (!fl_tile_tmap(ctx, ks.rows_prev, n_active, d_row, 1, &a.k_rows_map) ||
        !fl_tile_tmap(ctx, vs.rows_prev, n_active, d_row, 1, &a.v_rows_map) ||
        !fl_tile_tmap(ctx, q_store_in, s->L, d_row, 1, &a.q_map))
      return FL_ERR_UNSUPPORTED;
    a.rows_in = static_cast<const __nv_bfloat16*>(o_store_in);
    a.rows_out = static_cast<__nv_bfloat16*>(carry->bg_store);
    a.lse_prev = lse_in;
    const int rc = launch_mode<kOldPass>(ctx, s->bits, grid, a, st);
    if (rc != FL_OK) return rc;
  }
  if (!fl_tile_tmap(ctx, ks.rows_cur, n_active, d_row, 1, &a.k_rows_map) ||
      !fl_tile_tmap(ctx, vs.rows_cur, n_active, d_row, 1, &a.v_rows_map) ||
      !fl_tile_tmap(ctx, q_new, n_active, d_row, kM, &a.q_map))
    return FL_ERR_UNSUPPORTED;
  a.rows_in = static_cast<const __nv_bfloat16*>(carry->bg_store);
  a.rows_out = static_cast<__nv_bfloat16*>(o_store_out);
  a.lse_prev = lse_in;
  a.lse_out = lse_out;
  a.q_new = static_cast<const __nv_bfloat16*>(q_new);
  a.q_store = static_cast<__nv_bfloat16*>(q_store_out);
  return launch_mode<kNewPass>(ctx, s->bits, grid, a, st);
}
