// Stages 2 + 4 on the Blackwell tensor path: the attention replacement of Eq. 7 for one (query block,
// head) per CTA, with K/V of the selected columns gathered from the bf16 base and patched with the
// dequantized residual streams (Eq. 8) on their way into shared memory.
//
// Warp roles (16 warps, 512 threads):
//   warps 0-3   softmax of the OLD term  (fixed normaliser lse_prev: p_old = exp(s_old - lse_prev), mass m_i)
//   warps 4-7   softmax of the NEW term  (running reference, lazy rescale of the accumulator)
//   warps 8-9   MMA issuers, one thread per term: S = Q Khat^T of chunk n, then acc += P Vhat of chunk n - 1. A single
//               thread issues a 128x64x16 MMA every ~60-90 cycles while the tensor pipe retires one in 48; two threads
//               on two schedulers keep up with a chunk period that the exponentials set
//   warps 10-15 TMA + patch: the Q tiles (two 2-D tile loads each), row gathers (cp.async.bulk.tensor
//               tile::gather4, 4 selected columns per copy) of bf16 K/V rows straight into 128B-swizzled
//               operand tiles, and for columns that carry residual payloads which nobody has materialized the
//               overwrite of the gathered base rows with the dequantize-and-add result (Eq. 8)
//
// Prologue (whole CTA): the block's causal column list is copied to shared memory together with a bit mask
// of the residual streams that carry each column, and stably partitioned into columns WITHOUT a payload in
// the current loop (Khat_old == Khat_new, one K tile and one V tile serve both terms) followed by columns
// WITH one (separate old / new tiles). Most columns are of the first kind and are a plain gather of base rows.
// The second kind are the loop's active tokens: the quantization kernel of the same loop, which holds both
// Xhat^(r-1) and Xhat^(r) of those rows in registers, leaves them as bf16 rows in a transient workspace, and the
// old / new tiles are plain gathers from there (indexed by the token's row in the loop's stream). Without that
// workspace, and for columns whose only payloads are from earlier loops, the patch warps rebuild the rows here.
//
// Per chunk of 64 columns and per term: S (f32, 64 tensor-memory columns, two buffers: the next chunk's QK^T runs
// under the current chunk's exponentials); P (bf16, 32 columns) is written over the first half of the S buffer it
// was computed from, once those logits are in registers, so PV of a chunk runs under the next chunk's exponentials
// and the QK^T of the chunk after that waits for it before it overwrites the buffer.
// The two terms are independent pipelines. Epilogue: O = O_prev - acc_old + (m / l) acc_new.
// Shared memory: Q_old, Q_new tiles (64 KB) + a ring of four 32 KB operand slots (K tile | V tile); a chunk of
// the first kind takes one slot, of the second kind two. Tensor memory (512 columns): acc_old 0-127,
// acc_new 128-255, S_old / P_old 256-383 (two buffers), S_new / P_new 384-511.
// One CTA per problem, except that the problems of a partly empty last wave are given to pairs of CTAs when the
// caller has lent a workspace: each CTA of a pair takes half of the chunks, the one that completes first leaves its
// accumulators and row statistics in the workspace and the other merges them into its own before the epilogue.
// Every wait (mbarriers, the pair's counter) is bounded; on a timeout the CTA raises a flag, drains and reports
// FL_ERR_TIMEOUT.
//
// Old-term economy (template parameter ECON). When the column sets of a (head, block) are the ones of the loop
// before and the row was active in it, the old term of Eq. 7 is that loop's new term, so
//   O^(r) = B + new^(r),   B = O^(w-1) - old^(w)   of the last loop w that recomputed the old term,
// and the cached mass m_i is the one of loop w (Eq. 6: it does not change while the set does not). A recomputing
// launch can leave B (storage type, by position) and m_i (binary32, [H, L]) in buffers of the caller; an ECON launch
// reads them and computes the new term only. Its two pipelines then are two STREAMS of the new term (even and odd
// chunks of the column list, an accumulator, a running reference and a row sum each), merged in the epilogue like the
// two halves of a split problem; the previous loop's Q rows, O rows and log-normalisers are not read.
#include "tc_attn_common.cuh"

namespace {

using namespace fl_tc;

constexpr int kSlots = 4;
constexpr int kSlotBytes = 2 * kTileBytes;  // K tile | V tile
constexpr int kSoftmaxWarps = 8;
constexpr int kIssueWarp = 8;      // warps 8, 9: the MMA issuers of the old and of the new term (QK^T and PV each)
constexpr int kIssueWarps = 2;
constexpr int kTmaWarp = 10;       // first of the TMA / patch warps
constexpr int kTmaWarps = 6;       // a warp's four-row gathers are taken one lane after the other (~100 cycles each):
                                   // the 64 gathers of a ring slot need as many warps as can be had
constexpr int kWarps = kSoftmaxWarps + kIssueWarps + kTmaWarps;  // 16
constexpr int kSlotGathers = kSlotBytes / 512;   // 64 four-row gathers of 128-byte rows fill a slot
constexpr int kThreads = kWarps * 32;
constexpr int kColWarps = 14;               // warps that read the column list in the prologue (the other two search rows)
constexpr int kMaxCols = 3072;              // column budget the shared-memory column list can hold
constexpr int kMaxChunks = kMaxCols / kNC + 2;
constexpr uint32_t kAccOld = 0, kAccNew = 128, kSOld = 256, kSNew = 384;   // two S buffers of kNC columns each
// A problem can be split over two CTAs, each taking half of the chunks: a CTA's partial result is both accumulators
// (column-major, so that the row-owning threads write and read coalesced) and the three per-row statistics.
constexpr int kPartFloats = kFlPartFloats;
constexpr int kMaxSplit = kFlMaxSplit;      // counters at the head of the workspace
static_assert(kPartFloats == 2 * kM * kDH + 4 * kM, "partial result: two accumulators and four statistics per row");
static_assert(3 * kMaxCols * 4 <= kSlots * kSlotBytes, "prologue staging must fit in the ring");
static_assert(kAccNew == kAccOld + kDH, "the two accumulators are adjacent in tensor memory");

struct alignas(64) TcArgs {
  CUtensorMap k_map, v_map;          // row-gather maps of the K / V base ([L, d] bf16, box 64 x 1, 128B swizzle)
  CUtensorMap k_prev_map, k_cur_map;  // use_rows: row-gather maps of the loop's materialized rows ([n_active, d] bf16):
  CUtensorMap v_prev_map, v_cur_map;  // Khat / Vhat of the active tokens before and after the loop's residual
  CUtensorMap q_new_map, q_old_map;  // tile maps of the compact Q rows ([n_active, d] bf16, box 64 x 128); in the
                                     // indexed form q_old_map is a row-gather map of the Q store ([L, d], box 64 x 1)
  const __nv_bfloat16* o_prev;       // compact rows; in the indexed form the O stores [L, d] (may be the same)
  __nv_bfloat16* o_out;
  const __nv_bfloat16* bg_in;        // ECON: the rows' background B [L, d] by position (read instead of o_prev)
  __nv_bfloat16* bg_out;             // recomputing launch: receives B = o_prev - old term [L, d] by position, or null
  float* mass;                       // [H, L] by position: read by an ECON launch, written with bg_out otherwise
  const __nv_bfloat16* q_new;        // indexed form only: compact new Q rows, copied into q_store at the end
  __nv_bfloat16* q_store;            // indexed form only: Q store [L, d] that receives them, or null
  const int32_t* active_idx;
  int n_active;
  DevSide k, v;
  int n_old;
  int use_rows;                      // columns active in this loop are gathered from the materialized rows
  int n_full;                        // CTAs 0 .. n_full-1 take one problem each; the rest are pairs sharing one
  int32_t* part_cnt;                 // [kMaxSplit] arrival counters of the pairs (zero between launches)
  float* part_acc;                   // [pairs][2][kPartFloats] partial results
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
  uint64_t patched[kSlots];  // patch -> QK issuers: residual-carrying columns of the slot are rewritten (dirty chunks only)
  uint64_t done[kSlots];     // the two PV issuers -> TMA: the MMAs that read the slot have finished (a term's PV of a chunk
                             // is issued after its softmax, hence after its QK^T of the chunk has completed)
  uint64_t q_full;           // TMA -> QK issuers: the Q tiles of the current row tile have arrived
  uint64_t s_full[2][2];     // QK issuer -> softmax (per term, per S buffer): S of the chunk is in tensor memory
  uint64_t p_full[2][2];     // softmax -> PV issuer (per term, per buffer): P of the chunk is in tensor memory
  uint64_t p_free[2][2];     // PV issuer -> QK issuer: the PV MMAs that read the buffer's P have finished
  uint64_t acc_done;         // PV issuers -> softmax: all accumulation of the tile finished
  uint32_t tmem_base;
  int abort_flag;
  int q_lo, q_hi, i_last;    // block's slot range in active_idx, position of its last active row
  int n_plain, n_patch;      // columns without / with a payload in the current loop
  int merge_role;            // split problems: 0 = this CTA finished first (the other one merges), 1 = it merges,
                             // 2 = it should have merged but gave up waiting for the other's partial result
  int warp_cnt[kWarps][2];
  int chunk_last[kMaxChunks];       // largest column position of the chunk, INT32_MAX if the chunk is padded
  uint32_t chunk_mask[kMaxChunks];  // OR of the stream masks of the chunk's columns (0: plain gather only)
  float mass[kM];            // ECON: row sums of stream 0
  float ell[kM];
  float ref[kM];
  float ref0[kM];            // ECON: running references of stream 0
};

constexpr size_t kTcSmemBytes = 1024 /* alignment slack */ + 2 * kQTileBytes + kSlots * kSlotBytes + sizeof(TcSmemCtl) +
                                2 * kMaxCols * sizeof(int32_t);

// ECON: the old term is not recomputed (see the head of this file); the two pipelines are two streams of the new term.
template <int BITS, bool INDEXED, bool ECON>
__global__ void __launch_bounds__(kThreads, 1) loop_attn_tc_kernel(const __grid_constant__ TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_old_tile = smem;
  uint8_t* q_new_tile = smem + kQTileBytes;
  uint8_t* ring = smem + 2 * kQTileBytes;
  TcSmemCtl& ctl = *reinterpret_cast<TcSmemCtl*>(ring + kSlots * kSlotBytes);
  int32_t* ord_col = reinterpret_cast<int32_t*>(&ctl + 1);               // [kMaxCols] column positions, partitioned
  uint32_t* ord_mask = reinterpret_cast<uint32_t*>(ord_col + kMaxCols);  // bit s: payload in stream s

  fl_grid_wait();      // nothing below runs ahead of the previous kernel of the stream
  fl_grid_release();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // problem (query block b, head h) of this CTA, and for the pairs at the end of the grid which half of it
  int item = blockIdx.x, part = 0, pair = -1;
  const int n_items = a.nb * a.H;
  if (item >= a.n_full) {
    pair = (item - a.n_full) >> 1;
    part = (item - a.n_full) & 1;
    item = n_items - 1 - pair;          // the pairs walk the end of the item list backwards
  }
  // Item order: every chunk of the problems of the first query block (one per head) needs the causal mask, which
  // makes them ~20% slower than the others. With pairs they come last in the list, where they are the first to be
  // split over two CTAs (as whole problems in the early waves they delay their SMs for the rest of the launch);
  // without pairs they come first, the longest jobs before the others.
  int b, h;
  const bool has_pairs = a.n_full < n_items;
  const int first_block_at = has_pairs ? n_items - a.H : 0;     // where the H first-block problems sit in the list
  if (a.nb == 1) { b = 0; h = item; }
  else if (item >= first_block_at && item < first_block_at + a.H) { b = 0; h = item - first_block_at; }
  else {
    const int idx = has_pairs ? item : item - a.H;
    h = idx / (a.nb - 1);
    b = 1 + idx % (a.nb - 1);
  }
  const size_t prob = (size_t)h * a.nb + b;
  const int32_t* cols = a.col_idx + prob * a.c;
  const int cnt = min(__ldg(a.col_cnt + prob), kMaxCols);

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) {
      tc::mbar_init(&ctl.landed[s], kTmaWarps);
      tc::mbar_init(&ctl.patched[s], kTmaWarps);
      tc::mbar_init(&ctl.done[s], ECON ? 1 : 2);   // ECON: a slot is read by one stream only
    }
    tc::mbar_init(&ctl.q_full, 1);
    for (int t = 0; t < 2; ++t) {
      for (int pb = 0; pb < 2; ++pb) {
        tc::mbar_init(&ctl.s_full[t][pb], 1);
        tc::mbar_init(&ctl.p_full[t][pb], 4);
        tc::mbar_init(&ctl.p_free[t][pb], 1);
      }
    }
    tc::mbar_init(&ctl.acc_done, 2);
    ctl.abort_flag = 0;
    tc::fence_barrier_init();
  }
  // ---- prologue (rolled loops throughout: code that runs once per CTA is paid for in instruction fetches) ----
  // The raw column list, its stream rows and stream masks are staged in the still idle ring.
  int32_t* raw_col = reinterpret_cast<int32_t*>(ring);                     // [kMaxCols]
  uint32_t* raw_mask = reinterpret_cast<uint32_t*>(raw_col + kMaxCols);    // [kMaxCols]
  int32_t* raw_slot = reinterpret_cast<int32_t*>(raw_mask + kMaxCols);     // [kMaxCols]: row in the loop's own stream
  const int c_cap = min(a.c, kMaxCols);
  if (warp >= kColWarps) {
    // warps 14 and 15 search the block's rows in the ascending active list meanwhile
    const int target = warp == kColWarps ? b * a.q_block : min(a.L, (b + 1) * a.q_block);
    int below;
    const int r = lower_bound_warp(a.active_idx, a.n_active, target, lane, &below);
    if (lane == 0) {
      if (warp == kColWarps) ctl.q_lo = r;
      else { ctl.q_hi = r; ctl.i_last = r > 0 ? below : -1; }
    }
  } else {
    // The whole row of the column table is read without waiting for its count (entries past the count are -1),
    // and the thread that read a column goes on to look it up in the slot map of every residual stream: three
    // columns per thread and up to four streams at a time are in flight, two dependent rounds in all.
    constexpr int kBatch = 3, kStride = kColWarps * 32;
#pragma unroll 1
    for (int u0 = tid; u0 < c_cap; u0 += kBatch * kStride) {
      int j[kBatch], sl_new[kBatch];
      uint32_t mask[kBatch];
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        j[k] = u0 + k * kStride < c_cap ? __ldg(cols + u0 + k * kStride) : -1;
        mask[k] = 0;
        sl_new[k] = -1;
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
          for (int q = 0; q < 4; ++q) {
            if (sl[k][q] >= 0) mask[k] |= 1u << (sg + q);
            if (sg + q == a.n_old) sl_new[k] = sl[k][q];
          }
      }
#pragma unroll
      for (int k = 0; k < kBatch; ++k)
        if (u0 + k * kStride < c_cap) {
          raw_col[u0 + k * kStride] = j[k];
          raw_mask[u0 + k * kStride] = mask[k];
          raw_slot[u0 + k * kStride] = sl_new[k];
        }
    }
  }
  if (warp == kIssueWarp) {
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
  {
    // causal prefix, stable partition into plain / patched columns: every warp owns a contiguous span
    const int i_last = ctl.i_last;                                   // last active row of the block
    const int span = ((cnt + kWarps - 1) / kWarps + 31) & ~31;
    const int beg = warp * span, end = min(cnt, beg + span);
    int n0 = 0, n1 = 0;                                              // plain / patched columns in this warp's span
#pragma unroll 1
    for (int base = beg; base < end; base += 32) {
      const int u = base + lane;
      const bool live = u < end && raw_col[u] <= i_last;
      const bool patched = live && ((raw_mask[u] >> a.n_old) & 1u);
      n0 += __popc(__ballot_sync(0xffffffffu, live && !patched));
      n1 += __popc(__ballot_sync(0xffffffffu, patched));
    }
    if (lane == 0) { ctl.warp_cnt[warp][0] = n0; ctl.warp_cnt[warp][1] = n1; }
    __syncthreads();
    // exclusive prefix over the warps' counts: lane w of every warp holds warp w's pair
    static_assert(kWarps <= 32, "one lane per warp");
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
      const uint32_t mask = u < end ? raw_mask[u] : 0u;
      const bool live = j <= i_last;
      const bool patched = live && ((mask >> a.n_old) & 1u);
      const uint32_t m0 = __ballot_sync(0xffffffffu, live && !patched);
      const uint32_t m1 = __ballot_sync(0xffffffffu, patched);
      if (live) {
        const int dst = patched ? tot0 + before1 + __popc(m1 & lt) : before0 + __popc(m0 & lt);
        ord_col[dst] = j;
        // a column that is gathered from the materialized rows needs its row there, not its stream mask
        ord_mask[dst] = (patched && a.use_rows) ? (uint32_t)raw_slot[u] : mask;
      }
      before0 += __popc(m0);
      before1 += __popc(m1);
    }
    __syncthreads();
  }
  const int n_plain = ctl.n_plain, n_patch = ctl.n_patch;
  const int n_chunks = (n_plain + kNC - 1) / kNC + (n_patch + kNC - 1) / kNC;
  // A pair splits its problem's chunks in the middle, unless the block has several row tiles or a single chunk: then
  // the first CTA of the pair does everything and the second nothing (both see the same numbers).
  const bool split = pair >= 0 && q_hi - q_lo <= kM && n_chunks >= 2;
  const int c_mid = (n_chunks + 1) >> 1;
  const int c_lo = (split && part == 1) ? c_mid : 0;
  const int c_hi = (pair >= 0 && part == 1 && !split) ? 0 : ((split && part == 0) ? c_mid : n_chunks);
  // per chunk: the OR of its columns' stream masks and its last column (a warp per chunk, two columns per lane)
  for (int ci = warp; ci < n_chunks; ci += kWarps) {
    const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
    uint32_t m = 0;
    if (!(ck.patch && a.use_rows)) {   // chunks gathered from the materialized rows are never rewritten
      if (lane < ck.n_valid) m |= ord_mask[ck.off + lane];
      if (lane + 32 < ck.n_valid) m |= ord_mask[ck.off + lane + 32];
    }
    m = __reduce_or_sync(0xffffffffu, m);
    if (lane == 0) {
      ctl.chunk_mask[ci] = m;
      ctl.chunk_last[ci] = ck.n_valid == kNC ? ord_col[ck.off + kNC - 1] : INT32_MAX;
    }
  }
  __syncthreads();
  int g = 0;    // chunks issued so far (all tiles): S / P buffer = g & 1, one phase of its barriers per use
  int g1 = 0;   // ECON: the same count for stream 1 (g counts stream 0): a stream takes every other chunk
  int fill = 0; // ring slots filled so far: slot = fill % kSlots, phase = (fill / kSlots) & 1
  uint32_t dirty_par_cta = 0;  // per-slot phase parity of the patched[] barriers (they only see dirty chunks)

  for (int s0 = q_lo, tile = 0; s0 < q_hi && !(pair >= 0 && part == 1 && !split); s0 += kM, ++tile) {
  const int n_rows = min(kM, q_hi - s0);
  const int g0 = g, g0_1 = g1, fill0 = fill;
  const uint32_t dirty_par0 = dirty_par_cta;
  if (warp == kTmaWarp) {
    // Q tiles of this row tile: two 64-element slabs each; rows past the compact list read as zero, rows of the
    // next block (past n_rows) are computed and dropped
    if (lane == 0) {
      tc::mbar_arrive_expect_tx(&ctl.q_full, ECON ? kQTileBytes : 2 * kQTileBytes);
      tc::tma_tile2d(q_new_tile, &a.q_new_map, &ctl.q_full, h * kDH, s0);
      tc::tma_tile2d(q_new_tile + kM * 128, &a.q_new_map, &ctl.q_full, h * kDH + 64, s0);
      if (!INDEXED && !ECON) {
        tc::tma_tile2d(q_old_tile, &a.q_old_map, &ctl.q_full, h * kDH, s0);
        tc::tma_tile2d(q_old_tile + kM * 128, &a.q_old_map, &ctl.q_full, h * kDH + 64, s0);
      }
    }
    if (INDEXED && !ECON) {
      // the previous loop's Q rows come from the store: four-row gathers by position, one group of rows per lane
      __syncwarp();
      int y[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = lane * 4 + i;
        y[i] = r < n_rows ? __ldg(a.active_idx + s0 + r) : a.L;   // row L is outside the tensor: reads as zero
      }
      tc::tma_gather4(q_old_tile + lane * 512, &a.q_old_map, &ctl.q_full, h * kDH, y[0], y[1], y[2], y[3]);
      tc::tma_gather4(q_old_tile + kM * 128 + lane * 512, &a.q_old_map, &ctl.q_full, h * kDH + 64, y[0], y[1], y[2], y[3]);
    }
  }

  if (warp >= kTmaWarp) {
    // ========================================== TMA + patch ==========================================
    // In-order fills of the ring; the lookahead is whatever the four slots allow. The 64 four-row gathers
    // of a slot (K: 2 slabs x 16 groups, V: the same) are dealt round robin to the six warps, one per lane;
    // every warp announces its own share of the bytes on the slot's barrier. Chunks whose columns carry
    // residual payloads are then rewritten in place by the same warps (6 columns at a time, lanes 0-15 the K
    // row, lanes 16-31 the V row).
    const int tw = warp - kTmaWarp;
    // gather `req` of a slot: tile (K, V), 64-element slab, group of four columns
    const int req = lane * kTmaWarps + tw;
    const int my_reqs = (kSlotGathers - 1 - tw) / kTmaWarps + 1;      // requests of this warp (lanes 0 .. my_reqs - 1)
    const int is_v = (req >> 5) & 1, slab = (req >> 4) & 1, grp = req & 15;
    const void* map = is_v ? static_cast<const void*>(&a.v_map) : static_cast<const void*>(&a.k_map);
    const int half = lane >> 4, ch = lane & 15;
    const DevSide& side = half ? a.v : a.k;
    const int elem = h * kDH + ch * 8;
    const __nv_bfloat16* base_rows = static_cast<const __nv_bfloat16*>(side.base) + elem;
    const uint32_t ch_off = (ch >> 3) * (kNC * 128);
    int f = fill0;
    bool ok = true;
#pragma unroll 1
    for (int ci = c_lo; ci < c_hi && ok; ++ci) {
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      const int n_slots = (ck.patch && !ECON) ? 2 : 1;    // ECON: only the tiles after the loop's residual are needed
      const bool dirty = ctl.chunk_mask[ci] != 0;
      for (int k = 0; k < n_slots && ok; ++k)
        if (f + k >= kSlots) ok = warp_wait(&ctl.done[(f + k) % kSlots], (((f + k) / kSlots) - 1) & 1, abort_flag);
      if (!ok) break;
      if (lane == 0)
        for (int k = 0; k < n_slots; ++k) tc::mbar_arrive_expect_tx(&ctl.landed[(f + k) % kSlots], my_reqs * 512);
      __syncwarp();
      // columns that are active in this loop come from the materialized rows (old tile: before the loop's
      // residual, new tile: after it), indexed by their row in the loop's stream; all others from the base
      const bool from_rows = ck.patch && a.use_rows;
      if (req < kSlotGathers) {
        int y[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int u = grp * 4 + i;
          // a row past the end of the tensor reads as zero
          if (from_rows) y[i] = u < ck.n_valid ? (int)ord_mask[ck.off + u] : a.n_active;
          else y[i] = u < ck.n_valid ? ord_col[ck.off + u] : a.L;
        }
        for (int k = 0; k < n_slots; ++k) {
          const int slot = (f + k) % kSlots;
          const void* src = !from_rows ? map
                            : ((k == 0 && !ECON) ? (is_v ? static_cast<const void*>(&a.v_prev_map) : static_cast<const void*>(&a.k_prev_map))
                                      : (is_v ? static_cast<const void*>(&a.v_cur_map) : static_cast<const void*>(&a.k_cur_map)));
          tc::tma_gather4(ring + slot * kSlotBytes + is_v * kTileBytes + slab * (kNC * 128) + grp * 512, src,
                          &ctl.landed[slot], h * kDH + slab * 64, y[0], y[1], y[2], y[3]);
        }
      }
      if (dirty) {
        for (int k = 0; k < n_slots && ok; ++k)
          ok = warp_wait(&ctl.landed[(f + k) % kSlots], ((f + k) / kSlots) & 1, abort_flag);
        if (!ok) break;
        uint8_t* t_old = ring + (f % kSlots) * kSlotBytes + half * kTileBytes + ch_off;
        uint8_t* t_new = ring + ((f + 1) % kSlots) * kSlotBytes + half * kTileBytes + ch_off;
#pragma unroll 1
        for (int u = tw; u < ck.n_valid; u += kTmaWarps) {
          const uint32_t mask = ord_mask[ck.off + u];
          if (mask == 0) continue;
          const int j = ord_col[ck.off + u];
          const uint4 base16 = __ldg(reinterpret_cast<const uint4*>(base_rows + (size_t)j * a.d));
          uint4 v_old, v_new;
          patch_piece<BITS>(side, a.n_old, mask, j, elem, a.d, a.group, base16, v_old, v_new);
          const uint32_t off = tc::sw128_offset(u, ch & 7);
          if (ECON) {
            *reinterpret_cast<uint4*>(t_old + off) = v_new;     // the chunk's only slot holds Xhat^(r)
          } else {
            if (mask & ((1u << a.n_old) - 1u)) *reinterpret_cast<uint4*>(t_old + off) = v_old;
            if (ck.patch) *reinterpret_cast<uint4*>(t_new + off) = v_new;
          }
        }
        tc::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0)
          for (int k = 0; k < n_slots; ++k) tc::mbar_arrive(&ctl.patched[(f + k) % kSlots]);
      }
      f += n_slots;
    }
    if (INDEXED && a.q_store != nullptr && ok && !split) {
      // The Q store rows of this (row tile, head) were read by the gathers that completed q_full and belong to
      // no other CTA: the new rows take their place for the next loop.
      ok = warp_wait(&ctl.q_full, tile & 1, abort_flag);
      const int pt = tid - kTmaWarp * 32;
#pragma unroll 1
      for (int it = pt; ok && it < n_rows * 16; it += kTmaWarps * 32) {
        const int r = it >> 4, ch = it & 15;
        const int pos_r = __ldg(a.active_idx + s0 + r);
        *reinterpret_cast<uint4*>(a.q_store + (size_t)pos_r * a.d + h * kDH + ch * 8) =
            __ldg(reinterpret_cast<const uint4*>(a.q_new + (size_t)(s0 + r) * a.d + h * kDH + ch * 8));
      }
    }
  } else if (warp >= kIssueWarp) {
    // ========================================== MMA issuers ==========================================
    // One thread per term issues both kinds of MMA, in the order their operands become ready: QK^T of chunk n (its S
    // buffer is free once PV of chunk n - 2 has retired), then PV of chunk n - 1 (its P is written while QK^T of
    // chunk n executes).
    const int t = warp - kIssueWarp;      // 0: old term, 1: new term (ECON: streams 0 and 1 of the new term)
    if (lane == 0) {
      const uint32_t idesc_qk = tc::make_idesc_bf16(kM, kNC, false);
      const uint32_t idesc_pv = tc::make_idesc_bf16(kM, kDH, true);
      // Descriptors differ only in their start-address field (bits 0-13, units of 16 bytes): the low word
      // moves (no carry into the other fields: shared memory is < 256 KB), the high word stays.
      // K-major operands (Q, Khat): 32 bytes per 16-element K step inside a 64-element slab, then the next slab.
      const uint64_t q_desc = tc::make_desc_sw128(tc::smem_u32((t || ECON) ? q_new_tile : q_old_tile), 16, 1024);
      const uint64_t k_desc0 = tc::make_desc_sw128(tc::smem_u32(ring), 16, 1024);
      const uint32_t kq_hi = (uint32_t)(k_desc0 >> 32);
      const uint32_t q_lo_w = (uint32_t)q_desc, k_lo0 = (uint32_t)k_desc0;
      // MN-major Vhat: 16 key rows = two 1024-byte row groups per K step
      const uint64_t v_desc0 = tc::make_desc_sw128(tc::smem_u32(ring) + kTileBytes, kNC * 128, 1024);
      const uint32_t v_hi = (uint32_t)(v_desc0 >> 32), v_lo0 = (uint32_t)v_desc0;
      const uint32_t s_base = tmem + (t ? kSNew : kSOld);
      const uint32_t acc = tmem + (t ? kAccNew : kAccOld);
      int f = fill0;             // ring position of the chunk whose QK^T is issued next
      int pv_slot = 0;           // slots of the chunk whose PV is issued next (the previous QK^T's)
      int pv_slot1 = -1;
      uint32_t dirty_par = dirty_par0;
      // the chunks this thread issues: all of them, or (ECON) every other one starting at the stream's number
      constexpr int kStep = ECON ? 2 : 1;
      const int first = c_lo + (ECON ? t : 0);
      const int n_mine = first < c_hi ? (c_hi - first + kStep - 1) / kStep : 0;
      const int gbase = (ECON && t) ? g0_1 : g0;
#pragma unroll 1
      for (int n = 0; n <= n_mine; ++n) {
        const int ci = first + n * kStep;
        const int gc = gbase + n;
        int qk_slot = 0, qk_slot1 = -1;
        if (n < n_mine) {
          const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
          if (ECON) f = fill0 + (ci - c_lo);    // one slot per chunk, filled in chunk order
          const bool two = ck.patch && !ECON;
          const int slot0 = f % kSlots, slot1 = (f + 1) % kSlots;
          if (n == 0 && !tc::mbar_wait(&ctl.q_full, tile & 1, abort_flag)) break;
          // a term reads one slot of the chunk only (the new term of a two-slot chunk the second): it starts on it
          // without waiting for the other
          const int my_slot = (t && two) ? slot1 : slot0, my_fill = (t && two) ? f + 1 : f;
          if (!tc::mbar_wait(&ctl.landed[my_slot], (my_fill / kSlots) & 1, abort_flag)) break;
          if (ctl.chunk_mask[ci] != 0) {       // residual-carrying columns are rewritten by the patch warps
            // (ECON: the ring has an even number of slots and the streams alternate, so within a row tile a slot
            // always serves the same stream, which therefore sees every phase of the slot's barrier)
            if (!tc::mbar_wait(&ctl.patched[my_slot], (dirty_par >> my_slot) & 1, abort_flag)) break;
            dirty_par ^= 1u << slot0;
            if (two) dirty_par ^= 1u << slot1;
          }
          // the S buffer holds P of the chunk before the previous one until its PV MMAs have read it
          if (gc >= 2 && !tc::mbar_wait(&ctl.p_free[t][gc & 1], ((gc >> 1) - 1) & 1, abort_flag)) break;
          const uint32_t s_dst = s_base + (gc & 1) * kNC;
          tc::tc_fence_after();
          const uint32_t k_lo = k_lo0 + my_slot * (kSlotBytes >> 4);
#define FL_QK(KK, ACC)                                                                                       \
  tc::mma_ss_lo<ACC>(s_dst, q_lo_w + ((((KK) >> 2) * (kM * 128) + ((KK)&3) * 32) >> 4), kq_hi,               \
                     k_lo + ((((KK) >> 2) * (kNC * 128) + ((KK)&3) * 32) >> 4), kq_hi, idesc_qk)
          FL_QK(0, false); FL_QK(1, true); FL_QK(2, true); FL_QK(3, true);
          FL_QK(4, true);  FL_QK(5, true); FL_QK(6, true); FL_QK(7, true);
#undef FL_QK
          tc::mma_commit(&ctl.s_full[t][gc & 1]);
          qk_slot = slot0;
          qk_slot1 = two ? slot1 : -1;
          f += two ? 2 : 1;
        }
        if (n > 0) {
          const int gp = gc - 1, pb = gp & 1;
          if (!tc::mbar_wait(&ctl.p_full[t][pb], (gp >> 1) & 1, abort_flag)) break;
          tc::tc_fence_after();
          const uint32_t v_lo = v_lo0 + ((t && pv_slot1 >= 0) ? pv_slot1 : pv_slot) * (kSlotBytes >> 4);
          const uint32_t p_src = s_base + pb * kNC;
          const uint32_t acc0 = n > 1 ? 1u : 0u;           // the thread's first chunk of the tile overwrites the accumulator
#pragma unroll
          for (int kk = 0; kk < kNC / 16; ++kk)
            tc::mma_ts_lo(acc, p_src + kk * 8, v_lo + kk * (2048 >> 4), v_hi, idesc_pv, kk > 0 ? 1u : acc0);
          tc::mma_commit(&ctl.p_free[t][pb]);
          tc::mma_commit(&ctl.done[pv_slot]);
          if (pv_slot1 >= 0) tc::mma_commit(&ctl.done[pv_slot1]);
        }
        pv_slot = qk_slot;
        pv_slot1 = qk_slot1;
      }
      tc::mma_commit(&ctl.acc_done);
    }
    __syncwarp();
  } else {
    // ============================================ softmax ============================================
    const int grp = warp >> 2;                    // 0: old term, 1: new term (ECON: streams 0 and 1 of the new term)
    const int gt = tid & 127;                     // thread inside the term's group of four warps
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const bool row_ok = row < n_rows;
    const int pos = row_ok ? __ldg(a.active_idx + s0 + row) : -1;
    const float c2 = a.scale * kLog2e;
    const float lse2 = ((row_ok && !ECON) ? a.lse_prev[(size_t)h * a.L + pos] : 0.f) * kLog2e;
    // the epilogue reads the row's previous output (ECON: its background): have it in L2 by then (each group asks
    // for its 128-byte half)
    const __nv_bfloat16* prev_rows = ECON ? a.bg_in : a.o_prev;
    if (row_ok)
      tc::prefetch_l2(prev_rows + (INDEXED ? (size_t)pos : (size_t)(s0 + row)) * a.d + h * kDH + grp * 64);
    const uint32_t s_addr = tmem + lane_base + (grp ? kSNew : kSOld);
    float mass = 0.f, ell = 0.f, ref = -INFINITY;
    bool ok = true;
    constexpr int kStep = ECON ? 2 : 1;           // ECON: a group's stream takes every other chunk
    const int gbase = (ECON && grp) ? g0_1 : g0;
    for (int ci = c_lo + (ECON ? grp : 0), n = 0; ci < c_hi; ci += kStep, ++n) {
      const int gc = gbase + n, pb = gc & 1, n_use = gc >> 1;
      if (!warp_wait(&ctl.s_full[grp][pb], n_use & 1, abort_flag)) { ok = false; break; }
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
      // P goes over the first half of this S buffer (the QK^T issuer waited for the PV MMAs of chunk gc - 2 before it
      // overwrote the buffer): the first 32 logits are in registers before columns 0-15 are stored, the second 32
      // (columns 32-63) before columns 16-31 are
      const uint32_t sp_addr = s_addr + pb * kNC;
      // The 64 logits of the row are taken in two halves of 32 (each its own little softmax step): 64 live logits
      // plus the pipeline's state do not fit 128 registers, and what spills lands in an L1 of ~30 KB.
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
        if (ECON || grp == 1) {
          // running reference of the new term: taken from the first columns that show a finite logit and moved
          // (with a rescale of the accumulator row) only when a maximum beats it by more than the threshold
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
            // every earlier PV must have completed before the accumulator rows are rewritten (n >= 1 here: the
            // reference was set in an earlier chunk, or in this chunk's first half, whose P is not announced yet)
            if (n > 0) {
              if (!warp_wait(&ctl.p_free[grp][(gc - 1) & 1], ((gc - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
              tc::tc_fence_after();
              const uint32_t acc_col = grp ? kAccNew : kAccOld;    // the group's own accumulator
#pragma unroll 1
              for (int q4 = 0; q4 < 8; ++q4) {
                uint32_t acc[16];
                tc::tmem_ld16(tmem + lane_base + acc_col + q4 * 16, acc);
                tc::tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * factor);
                tc::tmem_st16(tmem + lane_base + acc_col + q4 * 16, acc);
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
        if (!ECON && grp == 0) mass += sum; else ell += sum;
        tc::tmem_st16(sp_addr + hf * 16, *reinterpret_cast<uint32_t(*)[16]>(&r[0]));
      }
      if (!ok) break;
      // P is announced at once: its PV MMAs free both the ring slot (for the gathers) and this S buffer (for the
      // QK^T of the chunk after the next), and both are on the critical path
      tc::tmem_wait_st();
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&ctl.p_full[grp][pb]);
    }
    // ---- epilogue ------------------------------------------------------------------------------------
    // Each group finishes 64 of the 128 head-dim columns. Its half of the O_prev tile (ECON: of the background rows) is
    // staged in shared memory with coalesced asynchronous copies, combined in place by the row-owning threads, and
    // written out coalesced again. The staging area is the first half of the group's own Q tile (the QK^T MMAs of
    // the group's term have all retired once its last S arrived); the second half takes the background rows a
    // recomputing launch leaves for later loops. In ECON both streams read the new Q tile until the very end and the
    // old one is never loaded: the groups stage in its two halves.
    uint8_t* stage = ECON ? q_old_tile + grp * (kM * 128)    // [128 rows][8 x 16 B], 16-byte chunks XOR-swizzled by row
                          : (grp ? q_new_tile : q_old_tile);
    uint8_t* stage_bg = stage + kM * 128;                    // recomputing launch with bg_out only
    const bool write_bg = !ECON && INDEXED && a.bg_out != nullptr;   // CTA-uniform
    const size_t o_col0 = (size_t)h * kDH + grp * 64;
    // a tile without a single chunk (empty column set): no issuer has waited for the Q tiles, which are still on
    // their way into the very memory the rows are staged in
    if (ok && c_hi == c_lo) ok = warp_wait(&ctl.q_full, tile & 1, abort_flag);
#pragma unroll 1
    for (int k = 0; k < 8; ++k) {
      const int idx = k * 128 + gt, rr = idx >> 3, cc = idx & 7;
      if (rr < n_rows) {
        const size_t src_row = INDEXED ? (size_t)__ldg(a.active_idx + s0 + rr) : (size_t)(s0 + rr);
        tc::cp_async16(stage + rr * 128 + ((cc ^ (rr & 7)) << 4), prev_rows + src_row * a.d + o_col0 + cc * 8);
      }
    }
    tc::cp_async_commit();
    if (ok) ok = warp_wait(&ctl.acc_done, tile & 1, abort_flag);
    tc::tc_fence_after();
    if (ECON) {
      if (grp == 0) { ctl.mass[row] = ell; ctl.ref0[row] = ref; }
      else { ctl.ell[row] = ell; ctl.ref[row] = ref; }
    } else {
      if (grp == 0) ctl.mass[row] = mass;
      else { ctl.ell[row] = ell; ctl.ref[row] = ref; }
    }
    tc::cp_async_wait<0>();
    asm volatile("bar.sync 1, 256;" ::: "memory");
    // per-row statistics. Accumulator A (tensor-memory columns 0-127) is the old term's, B (128-255) the new term's;
    // in ECON they are streams 0 and 1 of the new term, each with its own row sum and reference.
    float m_i = ECON ? (row_ok ? a.mass[(size_t)h * a.L + pos] : 0.f) : ctl.mass[row];
    float l_a = ECON ? ctl.mass[row] : 0.f, ref_a = ECON ? ctl.ref0[row] : -INFINITY;
    float l_i = ctl.ell[row], ref_i = ctl.ref[row];
    // warp-uniform: the tensor-memory reads below are collective
    const bool valid_a = ok && c_hi > c_lo;
    const bool valid_b = ok && (ECON ? c_hi > c_lo + 1 : c_hi > c_lo);
    // ---- split problems: the CTA of the pair that finishes first leaves its partial result in the workspace, the
    // other one adds it to its own (nobody waits for anybody: whoever finds the counter at 1 merges)
    const float* other = nullptr;
    float f_a = 0.f, f_b = 1.f, f_oa = 0.f, f_ob = 0.f;   // factors of accumulators A and B, own and other CTA's
    if (split) {
      // counter of the pair: each CTA adds 1 when its accumulation is complete (the one that finds 0 is first), the
      // first one adds 16 once its partial result is in the workspace; the second resets it for the next launch
      if (tid == 0) ctl.merge_role = atomicAdd(a.part_cnt + pair, 1) & 1;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (ctl.merge_role == 0) {
        float* mine = a.part_acc + ((size_t)pair * 2 + part) * kPartFloats;
#pragma unroll 1
        for (int c16 = 0; c16 < 8; ++c16) {   // accumulator A columns 0-63 of the group's half, then B: 16 at a time
          uint32_t v[16];
          const int col = (c16 >> 2) * kDH + grp * 64 + (c16 & 3) * 16;   // column of the [A | B] accumulator pair
          const bool valid = (c16 >> 2) ? valid_b : valid_a;
          if (valid) {
            tc::tmem_ld16(tmem + lane_base + kAccOld + col, v);           // kAccNew == kAccOld + kDH
            tc::tmem_wait_ld();
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) mine[(col + i) * kM + row] = valid ? __uint_as_float(v[i]) : 0.f;
        }
        if (grp == 0) {
          mine[2 * kM * kDH + row] = ECON ? (valid_a ? l_a : 0.f) : (valid_a ? m_i : 0.f);
          mine[2 * kM * kDH + 3 * kM + row] = (ECON && valid_a) ? ref_a : -INFINITY;
        } else {
          mine[2 * kM * kDH + kM + row] = valid_b ? l_i : 0.f;
          mine[2 * kM * kDH + 2 * kM + row] = valid_b ? ref_i : -INFINITY;
        }
        __threadfence();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (tid == 0) atomicAdd(a.part_cnt + pair, 16);
      } else {
        // the other CTA came first and is writing its partial result (it is resident and past its main loop: the
        // wait is short, and bounded like every other)
        if (tid == 0) {
          int seen = atomicAdd(a.part_cnt + pair, 0);
          for (int it = 0; seen < 16 && it < (1 << 16); ++it) {
            __nanosleep(100);
            seen = atomicAdd(a.part_cnt + pair, 0);
          }
          if (seen < 16) { *abort_flag = 1; ctl.merge_role = 2; }   // gave up: no output, FL_ERR_TIMEOUT
          a.part_cnt[pair] = 0;                                     // ready for the next launch either way
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (ctl.merge_role == 1) {   // CTA-uniform
          __threadfence();
          const float* theirs = a.part_acc + ((size_t)pair * 2 + (part ^ 1)) * kPartFloats;
          // the other CTA's accumulators (128 KB) come into the idle ring in one round of asynchronous copies
          static_assert(2 * kM * kDH * sizeof(float) <= (size_t)kSlots * kSlotBytes, "a partial result fits in the ring");
#pragma unroll 1
          for (int i = tid; i < 2 * kM * kDH / 4; i += 256) tc::cp_async16(ring + i * 16, theirs + i * 4);
          tc::cp_async_commit();
          other = reinterpret_cast<const float*>(ring);
          const float s0_o = __ldcg(theirs + 2 * kM * kDH + row), l_o = __ldcg(theirs + 2 * kM * kDH + kM + row);
          const float ref_o = __ldcg(theirs + 2 * kM * kDH + 2 * kM + row);
          const float ref_oa = __ldcg(theirs + 2 * kM * kDH + 3 * kM + row);
          // products and sums rounded one by one (no fused multiply-add), the two CTAs' contributions joined by one
          // commutative addition: the result must not depend on which of the two does the merging
          if (ECON) {
            const float ref_t = fmaxf(fmaxf(ref_a, ref_i), fmaxf(ref_oa, ref_o));
            f_a = ref_a > -INFINITY ? tc::ex2(ref_a - ref_t) : 0.f;
            f_b = ref_i > -INFINITY ? tc::ex2(ref_i - ref_t) : 0.f;
            f_oa = ref_oa > -INFINITY ? tc::ex2(ref_oa - ref_t) : 0.f;
            f_ob = ref_o > -INFINITY ? tc::ex2(ref_o - ref_t) : 0.f;
            l_i = __fadd_rn(__fadd_rn(__fmul_rn(l_a, f_a), __fmul_rn(l_i, f_b)),
                            __fadd_rn(__fmul_rn(s0_o, f_oa), __fmul_rn(l_o, f_ob)));
            ref_i = ref_t;
          } else {
            const float ref_t = fmaxf(ref_i, ref_o);
            f_b = ref_i > -INFINITY ? tc::ex2(ref_i - ref_t) : 0.f;
            f_ob = ref_o > -INFINITY ? tc::ex2(ref_o - ref_t) : 0.f;
            m_i = __fadd_rn(m_i, s0_o);
            l_i = __fadd_rn(__fmul_rn(l_i, f_b), __fmul_rn(l_o, f_ob));
            ref_i = ref_t;
          }
          tc::cp_async_wait<0>();
          asm volatile("bar.sync 1, 256;" ::: "memory");
        }
      }
    }
    if (ECON && other == nullptr) {   // the CTA's own two streams on a common reference
      const float ref_t = fmaxf(ref_a, ref_i);
      f_a = ref_a > -INFINITY ? tc::ex2(ref_a - ref_t) : 0.f;
      f_b = ref_i > -INFINITY ? tc::ex2(ref_i - ref_t) : 0.f;
      l_i = __fadd_rn(__fmul_rn(l_a, f_a), __fmul_rn(l_i, f_b));
      ref_i = ref_t;
    }
    const bool writer = !split || other != nullptr;       // CTA-uniform: this CTA produces the output rows
    const bool has = valid_a && ref_i > -INFINITY && (!ECON || m_i > 0.f);   // per row: T_i is not empty
    const float w = has ? m_i / l_i : 0.f;
#pragma unroll 1
    for (int c8 = 0; c8 < 8 && writer; ++c8) {   // 8 head-dim columns = one 16-byte cell of the staged row at a time
      uint32_t ao[8], an[8];
      const int col = grp * 64 + c8 * 8;
      if (valid_a) tc::tmem_ld8(tmem + lane_base + kAccOld + col, ao);
      if (valid_b) tc::tmem_ld8(tmem + lane_base + kAccNew + col, an);
      tc::tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (!valid_a) ao[i] = 0u;
        if (!valid_b) an[i] = 0u;
      }
      if (ECON) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float v = __fadd_rn(__fmul_rn(__uint_as_float(ao[i]), f_a), __fmul_rn(__uint_as_float(an[i]), f_b));
          if (other != nullptr)
            v = __fadd_rn(v, __fadd_rn(__fmul_rn(other[(col + i) * kM + row], f_oa),
                                       __fmul_rn(other[(kDH + col + i) * kM + row], f_ob)));
          an[i] = __float_as_uint(v);
        }
      } else if (other != nullptr) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          ao[i] = __float_as_uint(__fadd_rn(__uint_as_float(ao[i]), other[(col + i) * kM + row]));
          an[i] = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(an[i]), f_b),
                                            __fmul_rn(other[(kDH + col + i) * kM + row], f_ob)));
        }
      }
      uint4* cell = reinterpret_cast<uint4*>(stage + row * 128 + ((c8 ^ (row & 7)) << 4));
      uint4* cell_bg = reinterpret_cast<uint4*>(stage_bg + row * 128 + ((c8 ^ (row & 7)) << 4));
      if (has) {
        float pv[8];
        unpack8(*cell, pv);
        if (!ECON) {
          // background of the row: what stays of its previous output once the old term is taken out
#pragma unroll
          for (int i = 0; i < 8; ++i) pv[i] = pv[i] - __uint_as_float(ao[i]);
          if (write_bg) *cell_bg = pack8(pv);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) pv[i] = pv[i] + w * __uint_as_float(an[i]);
        *cell = pack8(pv);
      } else if (write_bg) {
        *cell_bg = *cell;                                   // empty T_i: the row itself is its background
      }
    }
    if (grp == 1 && row_ok && writer) {
      if (has) a.lse_out[(size_t)h * a.L + pos] = (ref_i + log2f(l_i)) * kLn2 - logf(m_i);
      else if (!ECON) a.lse_out[(size_t)h * a.L + pos] = lse2 * kLn2;
      else if (a.lse_prev != nullptr) a.lse_out[(size_t)h * a.L + pos] = a.lse_prev[(size_t)h * a.L + pos];
    }
    if (write_bg && grp == 0 && row_ok && writer) a.mass[(size_t)h * a.L + pos] = has ? m_i : 0.f;
    asm volatile("bar.sync 1, 256;" ::: "memory");
#pragma unroll 1
    for (int k = 0; k < 8 && writer; ++k) {
      const int idx = k * 128 + gt, rr = idx >> 3, cc = idx & 7;
      if (rr < n_rows) {
        const size_t dst_row = INDEXED ? (size_t)__ldg(a.active_idx + s0 + rr) : (size_t)(s0 + rr);
        *reinterpret_cast<uint4*>(a.o_out + dst_row * a.d + o_col0 + cc * 8) =
            *reinterpret_cast<const uint4*>(stage + rr * 128 + ((cc ^ (rr & 7)) << 4));
        if (write_bg)
          *reinterpret_cast<uint4*>(a.bg_out + dst_row * a.d + o_col0 + cc * 8) =
              *reinterpret_cast<const uint4*>(stage_bg + rr * 128 + ((cc ^ (rr & 7)) << 4));
      }
    }
  }
  if (INDEXED && split && a.q_store != nullptr) {   // CTA-uniform
    // Both halves of a split problem gathered the previous loop's Q rows from the store; the new rows may take their
    // place only when both are done with them, which the merging CTA knows
    __syncthreads();
    if (ctl.merge_role == 1 && !ctl.abort_flag) {
#pragma unroll 1
      for (int it = tid; it < n_rows * 16; it += kThreads) {
        const int r = it >> 4, ch = it & 15;
        const int pos_r = __ldg(a.active_idx + s0 + r);
        *reinterpret_cast<uint4*>(a.q_store + (size_t)pos_r * a.d + h * kDH + ch * 8) =
            __ldg(reinterpret_cast<const uint4*>(a.q_new + (size_t)(s0 + r) * a.d + h * kDH + ch * 8));
      }
    }
  }
  // every role is done with this tile: accumulators, Q tiles and the ring bookkeeping move on together
  if (s0 + kM < q_hi) {   // CTA-uniform: another row tile of the block follows
    if (ECON) { g += (c_hi - c_lo + 1) >> 1; g1 += (c_hi - c_lo) >> 1; }
    else g += c_hi - c_lo;
    int f = fill;
    for (int ci = c_lo; ci < c_hi; ++ci) {   // replay the tile's fills (same for every role)
      const ChunkInfo ck = chunk_info(ci, n_plain, n_patch);
      const int n_slots = (ck.patch && !ECON) ? 2 : 1;
      if (ctl.chunk_mask[ci] != 0)
        for (int k = 0; k < n_slots; ++k) dirty_par_cta ^= 1u << ((f + k) % kSlots);
      f += n_slots;
    }
    fill = f;
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
    tc::tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && ctl.abort_flag && a.status != nullptr) atomicExch(a.status, (int)FL_ERR_TIMEOUT);
}

}  // namespace

size_t fl_attn_workspace_bytes(const fl_ctx* ctx, const fl_shape* s) {
  if (s->dtype != FL_BF16 || s->head_dim != kDH) return 0;
  const int n_items = fl_n_blocks(s) * s->n_heads;
  const int rem = n_items % ctx->sm_count;
  if (rem == 0 || 2 * rem > ctx->sm_count || rem > kMaxSplit) return 0;
  return (size_t)kMaxSplit * sizeof(int32_t) + (size_t)rem * 2 * kPartFloats * sizeof(float);
}

extern "C" int fl_loop_attention_workspace_bytes(fl_ctx* ctx, const fl_shape* shape, int64_t* bytes) {
  FL_REQUIRE(ctx != nullptr && bytes != nullptr);
  const int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  *bytes = (int64_t)fl_attn_workspace_bytes(ctx, shape);
  return FL_OK;
}

extern "C" int fl_set_workspace(fl_ctx* ctx, void* workspace, int64_t bytes, void* stream) {
  FL_REQUIRE(ctx != nullptr && bytes >= 0);
  if (workspace == nullptr || bytes < (int64_t)(kMaxSplit * sizeof(int32_t))) {
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
    return workspace == nullptr ? FL_OK : FL_ERR_WORKSPACE;
  }
  FL_REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 255u) == 0);
  // the arrival counters at its head start at zero (every launch leaves them there)
  FL_CHECK_CUDA(cudaMemsetAsync(workspace, 0, kMaxSplit * sizeof(int32_t), static_cast<cudaStream_t>(stream)));
  ctx->ws = workspace;
  ctx->ws_bytes = (size_t)bytes;
  return FL_OK;
}

bool fl_loop_attn_tc_covers(const fl_ctx* ctx, const fl_shape* s, int c) {
  return s->dtype == FL_BF16 && s->head_dim == kDH && c <= kMaxCols && (size_t)ctx->max_smem_optin >= kTcSmemBytes &&
         ctx->encode_tiled != nullptr && ctx->tmaps != nullptr;
}

// Returns FL_ERR_UNSUPPORTED when the tensor path does not cover the request (caller falls back to the
// SIMT kernel, which is also CUDA). indexed != 0: q_old, o_prev and o_out are position-indexed stores [L, d] and
// q_store (may be null) receives the new Q rows. carry (indexed form only, may be null): the old-term economy's
// buffers; carry->reuse != 0 launches the ECON kernel, which reads them instead of q_old, o_prev and lse_prev.
int fl_launch_loop_attn_tc(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_old,
                           const int32_t* active_idx, int n_active, const fl_kv_store* store, const int32_t* col_idx,
                           const int32_t* col_cnt, int c, const float* lse_prev, float* lse_out, const void* o_prev,
                           void* o_out, int indexed, void* q_store, const fl_attn_carry* carry, int32_t* status,
                           cudaStream_t st) {
  if (!fl_loop_attn_tc_covers(ctx, s, c)) return FL_ERR_UNSUPPORTED;
  TcArgs a{};
  const int64_t d_row = (int64_t)s->n_heads * s->head_dim;
  if (!fl_tile_tmap(ctx, store->k_base, s->L, d_row, 1, &a.k_map) ||
      !fl_tile_tmap(ctx, store->v_base, s->L, d_row, 1, &a.v_map) ||
      !fl_tile_tmap(ctx, q_new, n_active, d_row, kM, &a.q_new_map))
    return FL_ERR_UNSUPPORTED;
  const bool econ = indexed && carry != nullptr && carry->reuse != 0;
  if (!econ && (indexed ? !fl_tile_tmap(ctx, q_old, s->L, d_row, 1, &a.q_old_map)
                        : !fl_tile_tmap(ctx, q_old, n_active, d_row, kM, &a.q_old_map)))
    return FL_ERR_UNSUPPORTED;
  if (indexed && carry != nullptr) {
    a.bg_in = econ ? static_cast<const __nv_bfloat16*>(carry->bg_store) : nullptr;
    a.bg_out = econ ? nullptr : static_cast<__nv_bfloat16*>(carry->bg_store);
    a.mass = carry->mass;
  }
  a.o_prev = static_cast<const __nv_bfloat16*>(o_prev);
  a.o_out = static_cast<__nv_bfloat16*>(o_out);
  a.q_new = static_cast<const __nv_bfloat16*>(q_new);
  a.q_store = static_cast<__nv_bfloat16*>(q_store);
  a.active_idx = active_idx; a.n_active = n_active;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.n_old = loop_r - 2;
  // the loop's materialized rows, when the caller keeps them (all four buffers)
  const fl_kv_stream& ks = store->k_res[loop_r - 2];
  const fl_kv_stream& vs = store->v_res[loop_r - 2];
  a.use_rows = ks.rows_prev != nullptr && ks.rows_cur != nullptr && vs.rows_prev != nullptr && vs.rows_cur != nullptr &&
               ks.n_rows == n_active && n_active > 0;
  if (a.use_rows && (!fl_tile_tmap(ctx, ks.rows_prev, n_active, d_row, 1, &a.k_prev_map) ||
                     !fl_tile_tmap(ctx, ks.rows_cur, n_active, d_row, 1, &a.k_cur_map) ||
                     !fl_tile_tmap(ctx, vs.rows_prev, n_active, d_row, 1, &a.v_prev_map) ||
                     !fl_tile_tmap(ctx, vs.rows_cur, n_active, d_row, 1, &a.v_cur_map)))
    return FL_ERR_UNSUPPORTED;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.lse_prev = lse_prev; a.lse_out = lse_out; a.status = status;
  a.L = s->L; a.H = s->n_heads; a.q_block = s->q_block; a.nb = fl_n_blocks(s);
  a.d = s->n_heads * s->head_dim; a.group = s->group; a.scale = s->sm_scale;
  // One CTA per (query block, head) problem; it walks the block's 128-row tiles. The problems are alike, so a grid
  // that is not a multiple of the SM count ends in a partly empty wave: when at most half of the SMs would be busy in
  // it and the caller has lent a workspace, each problem of that wave goes to a pair of CTAs (half of the chunks each).
  const int n_items = a.nb * s->n_heads;
  const int rem = n_items % ctx->sm_count;
  const size_t ws_need = (size_t)kMaxSplit * sizeof(int32_t) + (size_t)rem * 2 * kPartFloats * sizeof(float);
  const bool pairs = ctx->ws != nullptr && rem > 0 && 2 * rem <= ctx->sm_count &&
                     rem <= kMaxSplit && ctx->ws_bytes >= ws_need;
  a.n_full = pairs ? n_items - rem : n_items;
  a.part_cnt = static_cast<int32_t*>(ctx->ws);
  a.part_acc = reinterpret_cast<float*>(static_cast<uint8_t*>(ctx->ws) + kMaxSplit * sizeof(int32_t));
  const dim3 grid(a.n_full + 2 * (n_items - a.n_full));
#define FL_TC2(BITS, IDX, ECON)                                                                                  \
  do {                                                                                                           \
    auto kern = loop_attn_tc_kernel<BITS, IDX, ECON>;                                                            \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes));  \
    FL_CHECK_CUDA(fl_launch(ctx, kern, grid, dim3(kThreads), kTcSmemBytes, st, a));                             \
  } while (0)
#define FL_TC(BITS)                                   \
  do {                                                \
    if (econ) FL_TC2(BITS, true, true);               \
    else if (indexed) FL_TC2(BITS, true, false);      \
    else FL_TC2(BITS, false, false);                  \
  } while (0)
  switch (s->bits) {
    case 2: FL_TC(2); break;
    case 4: FL_TC(4); break;
    case 8: FL_TC(8); break;
    default: FL_TC(16); break;
  }
#undef FL_TC
#undef FL_TC2
  return fl_launch_status();
}
