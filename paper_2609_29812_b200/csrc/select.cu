// Stage 1 (Eq. 5: token scores and nested top-k) and the column selection of Eq. 6.
// Scoring is HBM-bound (one warp per candidate row, 16-byte loads, binary32 accumulation, warp-shuffle
// reduction). Selection is an exact radix select on the order-preserving integer image of the float
// scores, followed by an index-ordered compaction, so the result equals a full sort with the total
// order (score descending, index ascending) and comes out ascending.
#include <cstdlib>

#include "fl_internal.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// scoring
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) token_score_kernel(const T* __restrict__ h_prev, const T* __restrict__ h_cur,
                                                          const int32_t* __restrict__ cand, int n_cand, int d, float eps,
                                                          float* __restrict__ scores) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= n_cand) return;
  const size_t row = cand != nullptr ? (size_t)__ldg(cand + t) : (size_t)t;
  const T* a = h_cur + row * d;
  const T* b = h_prev + row * d;
  float num = 0.f, den = 0.f;
  int e = lane * 8;
  for (; e + 768 < d; e += 1024) {  // four chunks of each row in flight
    float x[4][8], y[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) { load8<T>(a + e + 256 * u, x[u]); load8<T>(b + e + 256 * u, y[u]); }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float df = x[u][i] - y[u][i];
        num = fmaf(df, df, num);
        den = fmaf(x[u][i], x[u][i], den);
      }
  }
  for (; e < d; e += 256) {
    float x[8], y[8];
    load8<T>(a + e, x); load8<T>(b + e, y);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float df = x[i] - y[i];
      num = fmaf(df, df, num);
      den = fmaf(x[i], x[i], den);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    num += __shfl_xor_sync(0xffffffffu, num, o);
    den += __shfl_xor_sync(0xffffffffu, den, o);
  }
  if (lane == 0) scores[t] = sqrtf(num) / (sqrtf(den) + eps);
}

// ------------------------------------------------------------------------------------------
// block-wide exact top-k, ascending output
// ------------------------------------------------------------------------------------------
constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t ordered_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger float <=> larger key
}

struct SelectSmem {
  uint32_t hist[256];
  uint32_t warp_gt[32], warp_eq[32];
  uint32_t prefix, k_rem;
};

// Selects the k (1 <= k <= n) largest of vals[0..n) with ties to the lowest index. Calls
// emit(rank, index) for every selected index, ranks ascending with the index. All threads of the
// block (kSelThreads) must call it.
template <typename Emit>
__device__ void block_topk_ascending(const float* __restrict__ vals, int n, int k, SelectSmem& sm, Emit emit) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t prefix = 0, k_rem = (uint32_t)k;
  if (k < n) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = tid; i < 256; i += kSelThreads) sm.hist[i] = 0;
      __syncthreads();
      const uint32_t hi_mask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
      for (int base = 0; base < n; base += kSelThreads) {
        const int i = base + tid;
        bool on = false;
        uint32_t digit = 0;
        if (i < n) {
          const uint32_t key = ordered_key(vals[i]);
          on = (key & hi_mask) == prefix;
          digit = (key >> shift) & 0xFFu;
        }
        // warp-aggregated histogram update: one atomic per distinct digit per warp
        const uint32_t active = __ballot_sync(0xffffffffu, on);
        if (on) {
          const uint32_t peers = __match_any_sync(active, digit);
          if ((peers & ((1u << lane) - 1)) == 0) atomicAdd(&sm.hist[digit], (uint32_t)__popc(peers));
        }
      }
      __syncthreads();
      if (warp == 0) {
        // lane owns digits [8*lane, 8*lane+8); find the digit holding the k_rem-th largest
        uint32_t local[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { local[j] = sm.hist[lane * 8 + j]; sum += local[j]; }
        // exclusive suffix sum over lanes: matching elements whose digit belongs to a higher lane
        uint32_t incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += v;
        }
        const uint32_t above = incl - sum;
        if (above < k_rem && k_rem <= above + sum) {
          uint32_t acc = above;
          for (int j = 7; j >= 0; --j) {
            if (k_rem <= acc + local[j]) {
              sm.prefix = prefix | ((uint32_t)(lane * 8 + j) << shift);
              sm.k_rem = k_rem - acc;
              break;
            }
            acc += local[j];
          }
        }
      }
      __syncthreads();
      prefix = sm.prefix;
      k_rem = sm.k_rem;
      __syncthreads();
    }
  } else {
    prefix = 0;  // every element qualifies: threshold below all keys, all "greater"
    k_rem = 0;
  }
  const uint32_t thr = prefix;
  const bool take_all = k >= n;
  // ---- index-ordered compaction: each warp owns a contiguous span ------------------------
  const int span = (((n + 31) / 32) + 31) / 32 * 32;  // per warp, multiple of 32
  const int beg = warp * span;
  const int end = min(n, beg + span);
  uint32_t gt = 0, eq = 0;
  for (int i = beg + lane; i < end; i += 32) {
    const uint32_t key = ordered_key(vals[i]);
    gt += (take_all || key > thr) ? 1u : 0u;
    eq += (!take_all && key == thr) ? 1u : 0u;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    gt += __shfl_xor_sync(0xffffffffu, gt, o);
    eq += __shfl_xor_sync(0xffffffffu, eq, o);
  }
  if (lane == 0) { sm.warp_gt[warp] = gt; sm.warp_eq[warp] = eq; }
  __syncthreads();
  uint32_t gt_before = 0, eq_before = 0;
  for (int w = 0; w < warp; ++w) { gt_before += sm.warp_gt[w]; eq_before += sm.warp_eq[w]; }
  for (int base = beg; base < end; base += 32) {
    const int i = base + lane;
    bool is_gt = false, is_eq = false;
    if (i < end) {
      const uint32_t key = ordered_key(vals[i]);
      is_gt = take_all || key > thr;
      is_eq = !take_all && key == thr;
    }
    const uint32_t m_gt = __ballot_sync(0xffffffffu, is_gt);
    const uint32_t m_eq = __ballot_sync(0xffffffffu, is_eq);
    const uint32_t lt = (1u << lane) - 1;
    const uint32_t my_gt = gt_before + __popc(m_gt & lt);
    const uint32_t my_eq = eq_before + __popc(m_eq & lt);
    if (is_gt) emit((int)(my_gt + min(my_eq, k_rem)), i);
    else if (is_eq && my_eq < k_rem) emit((int)(my_gt + my_eq), i);
    gt_before += __popc(m_gt);
    eq_before += __popc(m_eq);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads) token_select_kernel(const float* __restrict__ scores,
                                                                   const int32_t* __restrict__ cand, int n_cand, int k,
                                                                   int32_t* __restrict__ active_idx,
                                                                   int32_t* __restrict__ slot_of_pos) {
  __shared__ SelectSmem sm;
  block_topk_ascending(scores, n_cand, k, sm, [&](int rank, int i) {
    const int pos = cand != nullptr ? __ldg(cand + i) : i;
    active_idx[rank] = pos;
    slot_of_pos[pos] = rank;
  });
}

// ------------------------------------------------------------------------------------------
// The same selection with the keys staged in shared memory (problems of up to kSelCap candidates): the
// scores are read from global memory once; the radix passes run on shared memory and, as soon as the bin
// that holds the k-th largest key is small, on a compacted list of that bin's keys only.
// ------------------------------------------------------------------------------------------
constexpr int kSelCap = 49152;    // 192 KB of keys
constexpr int kSelSmall = 2048;

struct SelectSmem2 {
  uint32_t hist12[4096];
  uint32_t warp_tot[32];
  uint32_t hist[256];
  uint32_t warp_gt[32], warp_eq[32];
  uint32_t prefix, k_rem, bin_cnt, n_small;
  uint32_t small[kSelSmall];
};

// Adds the warp's keys that are `on` to the histogram: lanes that share the digit of the first matching lane
// are counted with one atomic (scores cluster in a few exponent bins, runs of equal scores are common), the
// rest add themselves.
__device__ __forceinline__ void hist_add(uint32_t* hist, bool on, uint32_t digit, int lane) {
  const uint32_t active = __ballot_sync(0xffffffffu, on);
  if (active == 0) return;
  const int leader = __ffs(active) - 1;
  const uint32_t d0 = __shfl_sync(0xffffffffu, digit, leader);
  const uint32_t same = __ballot_sync(0xffffffffu, on && digit == d0);
  if (lane == leader) atomicAdd(&hist[d0], (uint32_t)__popc(same));
  else if (on && digit != d0) atomicAdd(&hist[digit], 1u);
}

// one radix pass (`bits` <= 8 bits at `shift`) over list[0..m4*4): histogram of the keys that match `prefix`
// above the digit. Four keys per thread and step: the four dependent chains (load, vote, atomic) overlap.
__device__ __forceinline__ void radix_hist_pass(const uint32_t* list, int m4, int shift, int bits, uint32_t prefix,
                                                uint32_t* hist) {
  const int tid = threadIdx.x, lane = tid & 31;
  const uint32_t hi_mask = shift + bits >= 32 ? 0u : (0xFFFFFFFFu << (shift + bits));
  const uint32_t dmask = (1u << bits) - 1u;
  const uint4* l4 = reinterpret_cast<const uint4*>(list);
  for (int base = 0; base < m4; base += kSelThreads) {
    const int i = base + tid;
    const bool in = i < m4;
    const uint4 kv = in ? l4[i] : make_uint4(0, 0, 0, 0);
    hist_add(hist, in && (kv.x & hi_mask) == prefix, (kv.x >> shift) & dmask, lane);
    hist_add(hist, in && (kv.y & hi_mask) == prefix, (kv.y >> shift) & dmask, lane);
    hist_add(hist, in && (kv.z & hi_mask) == prefix, (kv.z >> shift) & dmask, lane);
    hist_add(hist, in && (kv.w & hi_mask) == prefix, (kv.w >> shift) & dmask, lane);
  }
}

// First level: 12-bit digit (sign, exponent, three mantissa bits) counted while the keys are staged. A warp whose
// 32 keys share the digit adds them with one atomic; otherwise every lane adds itself (a handful of lanes per bin).
__device__ __forceinline__ void hist12_add(uint32_t* hist12, uint32_t key, int lane) {
  const uint32_t d = key >> 20;
  int all_same;
  __match_all_sync(0xffffffffu, d, &all_same);
  if (all_same) { if (lane == 0) atomicAdd(&hist12[d], 32u); }
  else atomicAdd(&hist12[d], 1u);
}

__global__ void __launch_bounds__(kSelThreads, 1) column_select_smem_kernel(const float* __restrict__ col_scores,
                                                                            const int32_t* __restrict__ cand_cols,
                                                                            const int32_t* __restrict__ cand_cnt, int stride,
                                                                            int c, int L, int q_block, int nb, int vec_ok,
                                                                            int32_t* __restrict__ col_idx,
                                                                            int32_t* __restrict__ col_cnt) {
  extern __shared__ __align__(16) uint32_t keys[];   // [n rounded up to 4], padded with key 0 (below every real key)
  __shared__ SelectSmem2 sm;
  fl_grid_wait();
  fl_grid_release();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // later blocks have more candidates (causal prefix): they are dispatched first, the short ones fill the tail
  const int h = blockIdx.x, b = gridDim.y - 1 - blockIdx.y;
  const size_t prob = (size_t)h * nb + b;
  const float* vals = col_scores + prob * stride;
  const int32_t* cols = cand_cols != nullptr ? cand_cols + prob * stride : nullptr;
  int n = cand_cols != nullptr ? __ldg(cand_cnt + prob) : min(L, (b + 1) * q_block);
  n = max(0, min(n, stride));
  const int k = min(c, n);
  int32_t* out = col_idx + prob * c;
  for (int i = k + tid; i < c; i += kSelThreads) out[i] = -1;
  if (tid == 0) col_cnt[prob] = k;
  if (k == 0) return;
  const int n4 = (n + 3) >> 2;
  // ---- stage the order-preserving keys, counting their 12-bit digits on the way -----------------------------
  for (int i = tid; i < 4096; i += kSelThreads) sm.hist12[i] = 0;
  __syncthreads();
  {
    const float4* v4 = reinterpret_cast<const float4*>(vals);
    uint4* k4 = reinterpret_cast<uint4*>(keys);
    // four steps' loads are issued before the first is consumed: the staging is bound by memory latency otherwise
    // (whole warps run every step: padding keys are 0, bin 0)
    for (int base0 = 0; base0 < n4; base0 += 4 * kSelThreads) {
      float4 v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = base0 + q * kSelThreads + tid;
        v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < n4) {
          if (vec_ok && i * 4 + 3 < n) {
            v[q] = __ldg(v4 + i);
          } else {
            if (i * 4 + 0 < n) v[q].x = __ldg(vals + i * 4 + 0);
            if (i * 4 + 1 < n) v[q].y = __ldg(vals + i * 4 + 1);
            if (i * 4 + 2 < n) v[q].z = __ldg(vals + i * 4 + 2);
            if (i * 4 + 3 < n) v[q].w = __ldg(vals + i * 4 + 3);
          }
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = base0 + q * kSelThreads + tid;
        if (base0 + q * kSelThreads >= n4) break;   // CTA-uniform
        uint4 kv = make_uint4(0, 0, 0, 0);
        if (i < n4) {
          if (i * 4 + 0 < n) kv.x = ordered_key(v[q].x);
          if (i * 4 + 1 < n) kv.y = ordered_key(v[q].y);
          if (i * 4 + 2 < n) kv.z = ordered_key(v[q].z);
          if (i * 4 + 3 < n) kv.w = ordered_key(v[q].w);
          k4[i] = kv;
        }
        hist12_add(sm.hist12, kv.x, lane);
        hist12_add(sm.hist12, kv.y, lane);
        hist12_add(sm.hist12, kv.z, lane);
        hist12_add(sm.hist12, kv.w, lane);
      }
    }
  }
  __syncthreads();
  uint32_t prefix = 0, k_rem = 0;
  const bool take_all = k >= n;
  if (!take_all) {
    // ---- first level: the 12-bit bin that holds the k-th largest key (thread t owns bins 4t .. 4t+3) -------
    {
      uint32_t loc[4], sum = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) { loc[j] = sm.hist12[tid * 4 + j]; sum += loc[j]; }
      uint32_t incl = sum;                       // inclusive suffix sum over the warp (higher lanes = larger keys)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
      }
      if (lane == 0) sm.warp_tot[warp] = incl;
      __syncthreads();
      uint32_t above = incl - sum;               // keys in bins above this thread's
      for (int w2 = warp + 1; w2 < 32; ++w2) above += sm.warp_tot[w2];
      if (above < (uint32_t)k && (uint32_t)k <= above + sum) {
        uint32_t acc = above;
        for (int j = 3; j >= 0; --j) {
          if ((uint32_t)k <= acc + loc[j]) {
            sm.prefix = (uint32_t)(tid * 4 + j) << 20;
            sm.k_rem = (uint32_t)k - acc;
            sm.bin_cnt = loc[j];
            break;
          }
          acc += loc[j];
        }
      }
      if (tid == 0) sm.n_small = 0;
      __syncthreads();
      prefix = sm.prefix;
      k_rem = sm.k_rem;
    }
    const uint32_t* list = keys;
    int m4 = n4;
    int fixed = 12;                              // leading bits of the threshold found so far
    for (int pass = 0; pass < 4; ++pass) {
      // pass 0 only tries the compaction; passes 1-3 resolve 8, 8 and 4 more bits
      if (pass > 0) {
        const int bits = pass == 3 ? 4 : 8;
        const int shift = 32 - fixed - bits;
        for (int i = tid; i < 256; i += kSelThreads) sm.hist[i] = 0;
        __syncthreads();
        radix_hist_pass(list, m4, shift, bits, prefix, sm.hist);
        __syncthreads();
        if (warp == 0) {
          // lane owns digits [8*lane, 8*lane+8); find the digit holding the k_rem-th largest
          uint32_t local[8], sum = 0;
#pragma unroll
          for (int j = 0; j < 8; ++j) { local[j] = sm.hist[lane * 8 + j]; sum += local[j]; }
          uint32_t incl = sum;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
            if (lane + o < 32) incl += v;
          }
          const uint32_t above = incl - sum;
          if (above < k_rem && k_rem <= above + sum) {
            uint32_t acc = above;
            for (int j = 7; j >= 0; --j) {
              if (k_rem <= acc + local[j]) {
                sm.prefix = prefix | ((uint32_t)(lane * 8 + j) << shift);
                sm.k_rem = k_rem - acc;
                sm.bin_cnt = local[j];
                break;
              }
              acc += local[j];
            }
          }
          if (lane == 0) sm.n_small = 0;
        }
        __syncthreads();
        prefix = sm.prefix;
        k_rem = sm.k_rem;
        fixed += bits;
      }
      const uint32_t bin_cnt = sm.bin_cnt;
      if (fixed < 32 && list == keys && bin_cnt <= (uint32_t)(kSelSmall - 4)) {
        // the k-th largest key lies in a small bin: finish on that bin's keys alone
        const uint32_t hi_mask = 0xFFFFFFFFu << (32 - fixed);
        const int n_pad = n4 * 4;
        for (int base = warp * 128; base < n_pad; base += kSelThreads * 4) {   // 128 keys per warp and step
          uint32_t kk[4], m[4];
          uint32_t total = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int i = base + j * 32 + lane;
            kk[j] = i < n_pad ? keys[i] : 0u;
            m[j] = __ballot_sync(0xffffffffu, i < n_pad && (kk[j] & hi_mask) == prefix);
            total += __popc(m[j]);
          }
          if (total == 0) continue;
          uint32_t off = 0;
          if (lane == 0) off = atomicAdd(&sm.n_small, total);
          off = __shfl_sync(0xffffffffu, off, 0);
          const uint32_t lt = (1u << lane) - 1;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if ((m[j] >> lane) & 1u) sm.small[off + __popc(m[j] & lt)] = kk[j];
            off += __popc(m[j]);
          }
        }
        __syncthreads();
        // pad the list to a multiple of four with keys that cannot match the prefix of any later pass
        if (tid < 4) {
          const uint32_t m = sm.n_small;
          if (m + tid < ((m + 3) & ~3u)) sm.small[m + tid] = ~prefix;
        }
        list = sm.small;
        m4 = (int)((bin_cnt + 3) >> 2);
      }
      __syncthreads();
    }
  }
  const uint32_t thr = prefix;
  // ---- index-ordered compaction from the staged keys: each warp owns a contiguous span, walked 128 keys at a
  // time (lane l holds keys l, 32 + l, 64 + l, 96 + l of the step: votes give every key its place in index order)
  const int span = ((n + 31) / 32 + 127) / 128 * 128;
  const int beg = warp * span, end = min(n, beg + span);
  uint32_t gt = 0, eq = 0;
  for (int i = beg + lane; i < end; i += 32) {
    const uint32_t key = keys[i];
    gt += (take_all || key > thr) ? 1u : 0u;
    eq += (!take_all && key == thr) ? 1u : 0u;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    gt += __shfl_xor_sync(0xffffffffu, gt, o);
    eq += __shfl_xor_sync(0xffffffffu, eq, o);
  }
  if (lane == 0) { sm.warp_gt[warp] = gt; sm.warp_eq[warp] = eq; }
  __syncthreads();
  uint32_t gt_before = 0, eq_before = 0;
  for (int w = 0; w < warp; ++w) { gt_before += sm.warp_gt[w]; eq_before += sm.warp_eq[w]; }
  const uint32_t lt = (1u << lane) - 1;
  for (int base = beg; base < end; base += 128) {
    uint32_t kk[4], mg[4];
    bool any_eq_lane = false;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = base + j * 32 + lane;
      kk[j] = i < end ? keys[i] : 0u;
      mg[j] = __ballot_sync(0xffffffffu, i < end && (take_all || kk[j] > thr));
      any_eq_lane |= i < end && !take_all && kk[j] == thr;
    }
    if (!__any_sync(0xffffffffu, any_eq_lane)) {
      // no key of the step ties with the threshold: the selected ones are the greater ones, in index order
      uint32_t off = gt_before + min(eq_before, k_rem);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if ((mg[j] >> lane) & 1u) {
          const int i = base + j * 32 + lane;
          out[off + __popc(mg[j] & lt)] = cols != nullptr ? __ldg(cols + i) : i;
        }
        off += __popc(mg[j]);
      }
      gt_before += __popc(mg[0]) + __popc(mg[1]) + __popc(mg[2]) + __popc(mg[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int i = base + j * 32 + lane;
        const bool is_gt = (mg[j] >> lane) & 1u;
        const bool is_eq = i < end && !take_all && kk[j] == thr;
        const uint32_t me = __ballot_sync(0xffffffffu, is_eq);
        const uint32_t my_gt = gt_before + __popc(mg[j] & lt), my_eq = eq_before + __popc(me & lt);
        int rank = -1;
        if (is_gt) rank = (int)(my_gt + min(my_eq, k_rem));
        else if (is_eq && my_eq < k_rem) rank = (int)(my_gt + my_eq);
        if (rank >= 0) out[rank] = cols != nullptr ? __ldg(cols + i) : i;
        gt_before += __popc(mg[j]);
        eq_before += __popc(me);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Selection by a sampled pre-threshold (the common case: k much smaller than n, few exact ties at the boundary).
// A regular sample of the keys gives a value that, with a margin of several standard deviations, lies below the
// k-th largest key and above all but a few thousand keys. One coalesced pass over the scores collects every key at
// or above it (key and position) in shared memory; the exact k-th largest and the tie break by position are then
// found inside that short list, the winners are marked in a bit map over the positions, and the bit map is read
// out in position order. Every decision is exact: the list is a superset of the top k whenever it holds at least k
// keys, and whenever it does not (or is too long, or too many keys tie with the threshold) the CTA falls back to
// the radix select over all keys.
// ------------------------------------------------------------------------------------------
constexpr int kCandCap = 6144;         // keys the candidate list can hold
constexpr int kSample = 1024;          // one sampled key per thread
constexpr int kTieCap = 1024;          // ties with the threshold that are ranked by position here
constexpr int kBitmapWords = 8192;     // positions a problem may have: 32 * kBitmapWords

struct SampledSmem {
  SelectSmem generic;                  // fallback: radix select over all keys
  uint32_t hist[256];
  uint32_t prefix, rank, n_eq;
  uint32_t n_cand, n_tie;
  uint32_t warp_sum[32];
  int32_t tie_idx[kTieCap];
};

// `rank`-th largest (1-based) of the keys the threads hold (KPT per thread, `valid` marks the real ones), by four
// 8-bit radix passes with warp-aggregated shared-memory histograms. Returns the key; *rank_in_eq = how many of the
// keys equal to it belong to the `rank` largest, *n_eq = how many keys equal it. Only the first kpt_used slots of a
// thread are looked at (the same number in every thread). All kSelThreads threads call it.
template <int KPT>
__device__ uint32_t block_kth_largest(const uint32_t (&key)[KPT], const bool (&valid)[KPT], int kpt_used, uint32_t rank,
                                      SampledSmem& sm, uint32_t* rank_in_eq, uint32_t* n_eq) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t prefix = 0;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += kSelThreads) sm.hist[i] = 0;
    __syncthreads();
    const uint32_t hi_mask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
#pragma unroll
    for (int q = 0; q < KPT; ++q) {
      if (q >= kpt_used) break;               // CTA-uniform: the slots beyond it hold no key in any thread
      const bool on = valid[q] && (key[q] & hi_mask) == prefix;
      const uint32_t digit = (key[q] >> shift) & 0xFFu;
      const uint32_t active = __ballot_sync(0xffffffffu, on);
      if (on) {
        const uint32_t peers = __match_any_sync(active, digit);
        if ((peers & ((1u << lane) - 1)) == 0) atomicAdd(&sm.hist[digit], (uint32_t)__popc(peers));
      }
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t local[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { local[j] = sm.hist[lane * 8 + j]; sum += local[j]; }
      uint32_t incl = sum;                    // inclusive suffix sum over the lanes (higher lanes = larger digits)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
      }
      const uint32_t above = incl - sum;
      if (above < rank && rank <= above + sum) {
        uint32_t acc = above;
        for (int j = 7; j >= 0; --j) {
          if (rank <= acc + local[j]) {
            sm.prefix = prefix | ((uint32_t)(lane * 8 + j) << shift);
            sm.rank = rank - acc;
            sm.n_eq = local[j];
            break;
          }
          acc += local[j];
        }
      }
    }
    __syncthreads();
    prefix = sm.prefix;
    rank = sm.rank;
  }
  *rank_in_eq = rank;
  *n_eq = sm.n_eq;
  __syncthreads();
  return prefix;
}

__global__ void __launch_bounds__(kSelThreads, 2) column_select_sampled_kernel(const float* __restrict__ col_scores,
                                                                               const int32_t* __restrict__ cand_cols,
                                                                               const int32_t* __restrict__ cand_cnt,
                                                                               int stride, int c, int L, int q_block, int nb,
                                                                               int vec_ok, int32_t* __restrict__ col_idx,
                                                                               int32_t* __restrict__ col_cnt) {
  // dynamic shared memory: the candidate list (keys, positions), then one bit per position of the problem
  extern __shared__ __align__(16) uint32_t dyn_smem[];
  uint32_t* cand_key = dyn_smem;
  int32_t* cand_idx = reinterpret_cast<int32_t*>(dyn_smem + kCandCap);
  uint32_t* bitmap = dyn_smem + 2 * kCandCap;
  __shared__ SampledSmem sm;
  fl_grid_wait();
  fl_grid_release();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // later blocks have more candidates (causal prefix): they are dispatched first, the short ones fill the tail
  const int h = blockIdx.x, b = gridDim.y - 1 - blockIdx.y;
  const size_t prob = (size_t)h * nb + b;
  const float* vals = col_scores + prob * stride;
  const int32_t* cols = cand_cols != nullptr ? cand_cols + prob * stride : nullptr;
  int n = cand_cols != nullptr ? __ldg(cand_cnt + prob) : min(L, (b + 1) * q_block);
  n = max(0, min(n, stride));
  const int k = min(c, n);
  int32_t* out = col_idx + prob * c;
  for (int i = k + tid; i < c; i += kSelThreads) out[i] = -1;
  if (tid == 0) col_cnt[prob] = k;
  if (k == 0) return;
  if (k >= n) {   // everything is selected
    for (int i = tid; i < n; i += kSelThreads) out[i] = cols != nullptr ? __ldg(cols + i) : i;
    return;
  }
  // ---- a value below the k-th largest key: from a regular sample when the problem is too long to list whole ----
  uint32_t thr_lo = 0;                                  // n <= kCandCap: every key is a candidate
  if (n > kCandCap) {
    const uint32_t skey[1] = {ordered_key(__ldg(vals + (size_t)tid * n / kSample))};
    const bool sval[1] = {true};
    // aim at population rank k + k/2 + 256: the count of keys above the sample's r-th largest has mean r n/m and
    // standard deviation ~sqrt(r) n/m; the margin is several of those for the sizes this is used at, and a miss
    // only costs the fallback
    const uint64_t target = (uint64_t)k + (uint64_t)k / 2 + 256;
    uint32_t r_s = (uint32_t)((target * kSample + n - 1) / n);
    r_s = min(max(r_s, 1u), (uint32_t)kSample);
    uint32_t dummy0, dummy1;
    thr_lo = block_kth_largest<1>(skey, sval, 1, r_s, sm, &dummy0, &dummy1);
  }
  if (tid == 0) { sm.n_cand = 0; sm.n_tie = 0; }
  const int n_words = (n + 31) >> 5;
  for (int i = tid; i < n_words; i += kSelThreads) bitmap[i] = 0u;
  __syncthreads();
  // ---- one pass over the scores: keys at or above the pre-threshold go to the list (any order) ---------------
  {
    const float4* v4 = reinterpret_cast<const float4*>(vals);
    const int n4 = (n + 3) >> 2;
    for (int base = 0; base < n4; base += kSelThreads) {
      const int i = base + tid;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i < n4) {
        if (vec_ok && i * 4 + 3 < n) v = __ldg(v4 + i);
        else {
          if (i * 4 + 0 < n) v.x = __ldg(vals + i * 4 + 0);
          if (i * 4 + 1 < n) v.y = __ldg(vals + i * 4 + 1);
          if (i * 4 + 2 < n) v.z = __ldg(vals + i * 4 + 2);
          if (i * 4 + 3 < n) v.w = __ldg(vals + i * 4 + 3);
        }
      }
      const uint32_t kk[4] = {ordered_key(v.x), ordered_key(v.y), ordered_key(v.z), ordered_key(v.w)};
      bool on[4];
      int mine = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) { on[e] = i < n4 && i * 4 + e < n && kk[e] >= thr_lo; mine += on[e] ? 1 : 0; }
      // one atomic per warp and step: lanes take consecutive places behind it
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const int total = __shfl_sync(0xffffffffu, incl, 31);
      if (total == 0) continue;
      uint32_t at = 0;
      if (lane == 31) at = atomicAdd(&sm.n_cand, (uint32_t)total);
      at = __shfl_sync(0xffffffffu, at, 31) + (uint32_t)(incl - mine);
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (on[e]) {
          if (at < (uint32_t)kCandCap) { cand_key[at] = kk[e]; cand_idx[at] = i * 4 + e; }
          ++at;
        }
    }
  }
  __syncthreads();
  const uint32_t n_cand = sm.n_cand;
  bool fallback = n_cand < (uint32_t)k || n_cand > (uint32_t)kCandCap;    // CTA-uniform
  uint32_t thr = 0, take_eq = 0;
  if (!fallback) {
    // ---- the exact k-th largest inside the list ---------------------------------------------------------------
    constexpr int KPT = kCandCap / kSelThreads;
    uint32_t key[KPT];
    bool valid[KPT];
#pragma unroll
    for (int q = 0; q < KPT; ++q) {
      const uint32_t u = (uint32_t)(q * kSelThreads + tid);
      valid[q] = u < n_cand;
      key[q] = valid[q] ? cand_key[u] : 0u;
    }
    uint32_t n_eq;
    const int kpt_used = (int)((n_cand + kSelThreads - 1) / kSelThreads);
    thr = block_kth_largest<KPT>(key, valid, kpt_used, (uint32_t)k, sm, &take_eq, &n_eq);
    // ties with the threshold: all of them, or the take_eq lowest positions
    const bool rank_ties = take_eq < n_eq;
    if (rank_ties && n_eq > (uint32_t)kTieCap) fallback = true;            // CTA-uniform (n_eq is)
    if (!fallback) {
#pragma unroll
      for (int q = 0; q < KPT; ++q) {
        if (q >= kpt_used) break;
        if (!valid[q]) continue;
        const int idx = cand_idx[q * kSelThreads + tid];
        if (key[q] > thr || (key[q] == thr && !rank_ties)) atomicOr(&bitmap[idx >> 5], 1u << (idx & 31));
        else if (key[q] == thr) sm.tie_idx[atomicAdd(&sm.n_tie, 1u)] = idx;
      }
      __syncthreads();
      if (rank_ties) {
        // a tie is taken when fewer than take_eq ties lie at lower positions
        for (uint32_t t = tid; t < n_eq; t += kSelThreads) {
          const int mine = sm.tie_idx[t];
          uint32_t lower = 0;
          for (uint32_t u = 0; u < n_eq; ++u) lower += sm.tie_idx[u] < mine ? 1u : 0u;
          if (lower < take_eq) atomicOr(&bitmap[mine >> 5], 1u << (mine & 31));
        }
      }
      __syncthreads();
      // ---- read the bit map out in position order: every thread owns a run of words ----------------------------
      const int per = (n_words + kSelThreads - 1) / kSelThreads;
      const int w0 = tid * per, w1 = min(n_words, w0 + per);
      uint32_t cnt = 0;
      for (int w = w0; w < w1; ++w) cnt += __popc(bitmap[w]);
      uint32_t incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) sm.warp_sum[warp] = incl;
      __syncthreads();
      uint32_t before = incl - cnt;
      for (int w = 0; w < warp; ++w) before += sm.warp_sum[w];
      for (int w = w0; w < w1; ++w) {
        uint32_t bits = bitmap[w];
        while (bits) {
          const int bit = __ffs(bits) - 1;
          bits &= bits - 1;
          const int i = w * 32 + bit;
          out[before++] = cols != nullptr ? __ldg(cols + i) : i;
        }
      }
      return;
    }
  }
  // ---- fallback: the radix select over all keys (exact for every input) -------------------------------------
  block_topk_ascending(vals, n, k, sm.generic, [&](int rank, int i) { out[rank] = cols != nullptr ? __ldg(cols + i) : i; });
}

// one block per (head, query block)
__global__ void __launch_bounds__(kSelThreads) column_select_kernel(const float* __restrict__ col_scores,
                                                                    const int32_t* __restrict__ cand_cols,
                                                                    const int32_t* __restrict__ cand_cnt, int stride,
                                                                    int c, int L, int q_block, int nb,
                                                                    int32_t* __restrict__ col_idx,
                                                                    int32_t* __restrict__ col_cnt) {
  __shared__ SelectSmem sm;
  // later blocks have more candidates (causal prefix): they are dispatched first, the short ones fill the tail
  const int h = blockIdx.x, b = gridDim.y - 1 - blockIdx.y;
  const size_t prob = (size_t)h * nb + b;
  const float* vals = col_scores + prob * stride;
  const int32_t* cols = cand_cols != nullptr ? cand_cols + prob * stride : nullptr;
  int n = cand_cols != nullptr ? __ldg(cand_cnt + prob) : min(L, (b + 1) * q_block);
  n = max(0, min(n, stride));
  const int k = min(c, n);
  int32_t* out = col_idx + prob * c;
  for (int i = k + threadIdx.x; i < c; i += kSelThreads) out[i] = -1;
  if (threadIdx.x == 0) col_cnt[prob] = k;
  if (k == 0) return;
  block_topk_ascending(vals, n, k, sm, [&](int rank, int i) { out[rank] = cols != nullptr ? __ldg(cols + i) : i; });
}

}  // namespace

extern "C" int fl_select_tokens(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* h_prev, const void* h_cur,
                                const int32_t* cand, int32_t n_cand, int32_t k, float* scores, int32_t* active_idx,
                                int32_t* slot_of_pos, int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(loop_r >= 2);
  FL_REQUIRE(h_prev != nullptr && h_cur != nullptr && scores != nullptr && active_idx != nullptr &&
             slot_of_pos != nullptr);
  FL_REQUIRE(fl_aligned16(h_prev) && fl_aligned16(h_cur));
  FL_REQUIRE(k >= 1 && n_cand >= 1 && n_cand <= shape->L);
  FL_REQUIRE(cand != nullptr || n_cand == shape->L);
  const int d = shape->n_heads * shape->head_dim;
  if (d % 256 != 0) return FL_ERR_UNSUPPORTED;
  {
    const fl_idx_check ck = {cand, n_cand, 0, nullptr, 0, shape->L - 1, 1};
    rc = fl_debug_check(ctx, &ck, 1, status, stream);
    if (rc != FL_OK) return rc;
    rc = fl_debug_check_finite(ctx, h_prev, (int64_t)shape->L * d, shape->dtype, status, stream);
    if (rc != FL_OK) return rc;
    rc = fl_debug_check_finite(ctx, h_cur, (int64_t)shape->L * d, shape->dtype, status, stream);
    if (rc != FL_OK) return rc;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int warps = 8;
  const int grid = (n_cand + warps - 1) / warps;
  if (shape->dtype == FL_F32)
    token_score_kernel<float><<<grid, warps * 32, 0, st>>>(static_cast<const float*>(h_prev),
                                                           static_cast<const float*>(h_cur), cand, n_cand, d,
                                                           shape->eps, scores);
  else
    token_score_kernel<__nv_bfloat16><<<grid, warps * 32, 0, st>>>(static_cast<const __nv_bfloat16*>(h_prev),
                                                                   static_cast<const __nv_bfloat16*>(h_cur), cand,
                                                                   n_cand, d, shape->eps, scores);
  rc = fl_launch_status();
  if (rc != FL_OK) return rc;
  FL_CHECK_CUDA(cudaMemsetAsync(slot_of_pos, 0xFF, sizeof(int32_t) * (size_t)shape->L, st));
  const int k_eff = k < n_cand ? k : n_cand;
  token_select_kernel<<<1, kSelThreads, 0, st>>>(scores, cand, n_cand, k_eff, active_idx, slot_of_pos);
  return fl_launch_status();
}

extern "C" int fl_select_columns(fl_ctx* ctx, const fl_shape* shape, const float* col_scores, const int32_t* cand_cols,
                                 const int32_t* cand_cnt, int32_t n_cand, int32_t c, int32_t* col_idx, int32_t* col_cnt,
                                 int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(col_scores != nullptr && col_idx != nullptr && col_cnt != nullptr);
  FL_REQUIRE(c >= 1 && n_cand >= 1);
  if (cand_cols == nullptr) FL_REQUIRE(n_cand == shape->L);
  else FL_REQUIRE(cand_cnt != nullptr);
  const int nb = fl_n_blocks(shape);
  FL_REQUIRE(nb <= 65535);
  {
    const fl_idx_check ck = {cand_cols, (int64_t)shape->n_heads * nb * n_cand, n_cand, cand_cnt, 0, shape->L - 1, 0};
    rc = fl_debug_check(ctx, &ck, 1, status, stream);
    if (rc != FL_OK) return rc;
  }
  dim3 grid(shape->n_heads, nb);
  const size_t key_bytes = sizeof(uint32_t) * (((size_t)n_cand + 3) & ~(size_t)3);
  const int vec_ok = (fl_aligned16(col_scores) && n_cand % 4 == 0) ? 1 : 0;
  const char* staged = std::getenv("FL_SELECT_STAGED");
  if (n_cand <= 32 * kBitmapWords && !(staged != nullptr && staged[0] == '1')) {
    // sampled pre-threshold, candidate list, bit map over the positions (exact; falls back inside the kernel)
    const size_t dyn_bytes = sizeof(uint32_t) * (2 * (size_t)kCandCap + ((size_t)n_cand + 31) / 32);
    FL_CHECK_CUDA(cudaFuncSetAttribute(column_select_sampled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)dyn_bytes));
    FL_CHECK_CUDA(fl_launch(ctx, column_select_sampled_kernel, grid, dim3(kSelThreads), dyn_bytes,
                            static_cast<cudaStream_t>(stream), col_scores, cand_cols, cand_cnt, n_cand, c, shape->L,
                            shape->q_block, nb, vec_ok, col_idx, col_cnt));
  } else if (n_cand <= kSelCap && key_bytes + 32768 <= (size_t)ctx->max_smem_optin) {
    // keys staged in shared memory: the scores are read from global memory once
    FL_CHECK_CUDA(cudaFuncSetAttribute(column_select_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)key_bytes));
    FL_CHECK_CUDA(fl_launch(ctx, column_select_smem_kernel, grid, dim3(kSelThreads), key_bytes,
                            static_cast<cudaStream_t>(stream), col_scores, cand_cols, cand_cnt, n_cand, c, shape->L,
                            shape->q_block, nb, vec_ok, col_idx, col_cnt));
  } else {
    column_select_kernel<<<grid, kSelThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        col_scores, cand_cols, cand_cnt, n_cand, c, shape->L, shape->q_block, nb, col_idx, col_cnt);
  }
  return fl_launch_status();
}
