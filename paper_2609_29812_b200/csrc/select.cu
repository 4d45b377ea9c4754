// Stage 1 (Eq. 5: token scores and nested top-k) and the column selection of Eq. 6.
// Scoring is HBM-bound (one warp per candidate row, 16-byte loads, binary32 accumulation, warp-shuffle
// reduction). Selection is an exact radix select on the order-preserving integer image of the float
// scores, followed by an index-ordered compaction, so the result equals a full sort with the total
// order (score descending, index ascending) and comes out ascending.
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

// one block per (head, query block)
__global__ void __launch_bounds__(kSelThreads) column_select_kernel(const float* __restrict__ col_scores,
                                                                    const int32_t* __restrict__ cand_cols,
                                                                    const int32_t* __restrict__ cand_cnt, int stride,
                                                                    int c, int L, int q_block, int nb,
                                                                    int32_t* __restrict__ col_idx,
                                                                    int32_t* __restrict__ col_cnt) {
  __shared__ SelectSmem sm;
  const int b = blockIdx.x, h = blockIdx.y;
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
  (void)status;
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
  (void)status;
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(col_scores != nullptr && col_idx != nullptr && col_cnt != nullptr);
  FL_REQUIRE(c >= 1 && n_cand >= 1);
  if (cand_cols == nullptr) FL_REQUIRE(n_cand == shape->L);
  else FL_REQUIRE(cand_cnt != nullptr);
  const int nb = fl_n_blocks(shape);
  FL_REQUIRE(nb <= 65535 * 1024 && shape->n_heads <= 65535);
  dim3 grid(nb, shape->n_heads);
  column_select_kernel<<<grid, kSelThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      col_scores, cand_cols, cand_cnt, n_cand, c, shape->L, shape->q_block, nb, col_idx, col_cnt);
  return fl_launch_status();
}
