// Pieces shared by the tensor-path attention kernels: tile geometry, bounded warp waits, the row search in the
// active list, bf16 packing, the dequantize-and-add of one 16-byte piece and the chunk layout of the partitioned
// column list.
#pragma once
#include "fl_internal.cuh"
#include "tc_ptx.cuh"

namespace fl_tc {

constexpr int kM = 128;                     // rows of a query tile
constexpr int kDH = 128;                    // head dimension of the tensor path
constexpr int kNC = 64;                     // key columns per chunk
constexpr int kTileBytes = kNC * kDH * 2;   // one K or V operand tile of a chunk: 16 KB
constexpr int kQTileBytes = kM * kDH * 2;   // 32 KB
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 60.f;   // in log2 units: rescale only when the reference falls this far behind

// Bounded wait of a fully converged warp; every lane observes the completed phase itself, so each acquires
// what the arriving threads released. Returns a warp-uniform verdict.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  bool ok = tc::mbar_try_wait(bar, parity);
  if (__all_sync(0xffffffffu, ok)) return true;
  if (!ok) ok = tc::mbar_wait(bar, parity, abort_flag);
  return __all_sync(0xffffffffu, ok);
}

// First index in the ascending array with value >= target, and through `below` the element just before it
// (INT32_MIN if there is none). All 32 lanes cooperate: 128 probes per round while the range is wide, then one
// load per lane; the active lists of the benchmark shapes (a few thousand rows) take two dependent rounds.
__device__ __forceinline__ int lower_bound_warp(const int32_t* __restrict__ arr, int n, int target, int lane, int* below) {
  int lo = 0, hi = n, prev = INT32_MIN;   // invariant: arr[lo - 1] == prev < target (or lo == 0), arr[hi] >= target (or hi == n)
  while (hi - lo > 32) {
    const int step = (hi - lo + 127) >> 7;
    int v[4];
    uint32_t less[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int idx = lo + (lane * 4 + k + 1) * step - 1;
      v[k] = idx < hi ? __ldg(arr + idx) : INT32_MAX;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) less[k] = __ballot_sync(0xffffffffu, v[k] < target);
    // probes ascend with (lane, k): the ones below the target are a prefix
    const int n_less = __popc(less[0]) + __popc(less[1]) + __popc(less[2]) + __popc(less[3]);
    if (n_less > 0) {
      const int src = (n_less - 1) >> 2, kk = (n_less - 1) & 3;
      const int cand = kk == 0 ? v[0] : (kk == 1 ? v[1] : (kk == 2 ? v[2] : v[3]));
      prev = __shfl_sync(0xffffffffu, cand, src);
    }
    const int new_lo = lo + n_less * step;
    hi = min(hi, new_lo + step - 1);
    lo = min(new_lo, hi);
  }
  const int val = lo + lane < hi ? __ldg(arr + lo + lane) : INT32_MAX;
  const int cnt = __popc(__ballot_sync(0xffffffffu, val < target));
  if (cnt > 0) prev = __shfl_sync(0xffffffffu, val, cnt - 1);
  *below = prev;
  return lo + cnt;
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
  v_old = raw;
#pragma unroll 1
  for (int s = 0; s <= n_old; ++s) {
    if (s == n_old && (mask & ((1u << n_old) - 1u))) v_old = pack8(x);
    if ((mask >> s) & 1u) apply_stream8<__nv_bfloat16, BITS>(side.s[s], j, elem, d, group, x);
  }
  v_new = ((mask >> n_old) & 1u) ? pack8(x) : v_old;
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

// INDEXED: the previous loop's Q and O rows are read from, and the new O rows written to, position-indexed
// stores (row active_idx[t] for compact row t) instead of compact buffers.

}  // namespace fl_tc
