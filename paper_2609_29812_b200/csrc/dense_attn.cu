// Dense source loop (Eq. 2, causal) and the column statistics loop 2 starts from (Eq. 6 with m_C = 1):
// binary32 SIMT kernels. Also hosts the generic "column sums of exp(s - lse)" kernel that the sparse
// loop uses to prepare a pruned selection for loop r+1.
#include "attn_simt.cuh"

namespace {

template <typename T, int DH>
__global__ void __launch_bounds__(kAttnThreads) dense_attn_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                                  const T* __restrict__ v, T* __restrict__ o,
                                                                  float* __restrict__ lse, int L, int H, float scale) {
  extern __shared__ __align__(16) float smem[];
  float* k_tile = smem;                                         // [32][DH+1]
  float* v_tile = k_tile + kChunk * (DH + 1);                   // [32][DH]
  float4* q4 = reinterpret_cast<float4*>(v_tile + kChunk * DH); // [warps][DH]
  float4* p4 = q4 + kAttnWarps * DH;                            // [warps][32]
  const int tile = gridDim.x - 1 - blockIdx.x;  // longest rows first
  const int h = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = H * DH;
  const int i0 = tile * kQTile;
  const int iw = i0 + warp * kQW;  // first query of this warp

  for (int x = lane; x < DH; x += 32) {
    float qv[kQW];
#pragma unroll
    for (int qi = 0; qi < kQW; ++qi)
      qv[qi] = (iw + qi < L) ? to_float<T>(q[(size_t)(iw + qi) * d + h * DH + x]) : 0.f;
    q4[warp * DH + x] = make_float4(qv[0], qv[1], qv[2], qv[3]);
  }
  float m_run[kQW], l_run[kQW], acc[kQW][DH / 32];
#pragma unroll
  for (int qi = 0; qi < kQW; ++qi) {
    m_run[qi] = -INFINITY;
    l_run[qi] = 0.f;
#pragma unroll
    for (int t = 0; t < DH / 32; ++t) acc[qi][t] = 0.f;
  }
  const int i_last = min(L, i0 + kQTile) - 1;
  for (int j0 = 0; j0 <= i_last; j0 += kChunk) {
    __syncthreads();
    for (int it = threadIdx.x; it < kChunk * DH / 8; it += kAttnThreads) {
      const int u = it / (DH / 8), e = (it % (DH / 8)) * 8;
      const int j = j0 + u;
      float kv[8], vv[8];
      if (j < L) {
        load8<T>(k + (size_t)j * d + h * DH + e, kv);
        load8<T>(v + (size_t)j * d + h * DH + e, vv);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) kv[i] = vv[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        k_tile[u * (DH + 1) + e + i] = kv[i];
        v_tile[u * DH + e + i] = vv[i];
      }
    }
    __syncthreads();
    if (j0 > iw + kQW - 1) continue;  // chunk lies above the diagonal for all of this warp's rows
    float s[kQW], p[kQW];
    warp_qk<DH>(q4 + warp * DH, k_tile, lane, s);
    const int j = j0 + lane;
#pragma unroll
    for (int qi = 0; qi < kQW; ++qi) {
      const int i = iw + qi;
      const bool valid = (i < L) && (j <= i);
      const float sv = valid ? s[qi] * scale : -INFINITY;
      const float m_new = fmaxf(m_run[qi], warp_max(sv));
      float corr = 1.f;
      p[qi] = 0.f;
      if (m_new > -INFINITY) {
        corr = expf(m_run[qi] - m_new);
        p[qi] = valid ? expf(sv - m_new) : 0.f;
      }
      l_run[qi] = l_run[qi] * corr + warp_sum(p[qi]);
#pragma unroll
      for (int t = 0; t < DH / 32; ++t) acc[qi][t] *= corr;
      m_run[qi] = m_new;
    }
    p4[warp * kChunk + lane] = make_float4(p[0], p[1], p[2], p[3]);
    __syncwarp();
    warp_pv<DH>(p4 + warp * kChunk, v_tile, lane, acc);
    __syncwarp();
  }
#pragma unroll
  for (int qi = 0; qi < kQW; ++qi) {
    const int i = iw + qi;
    if (i >= L) continue;
    const float inv = 1.f / l_run[qi];
#pragma unroll
    for (int t = 0; t < DH / 32; ++t)
      o[(size_t)i * d + h * DH + lane + 32 * t] = from_float<T>(acc[qi][t] * inv);
    if (lse != nullptr && lane == 0) lse[(size_t)h * L + i] = m_run[qi] + logf(l_run[qi]);
  }
}

// ----------------------------------------------------------------------------------------------
// out[h, b, u] = sum over the block's query rows i >= column(u) of exp(scale q_i . Khat_column - lse[h, i]),
// i.e. the block column scores of Eq. 6 (probabilities already carry the mass through lse).
// Dense form : queries are all rows of the block, columns are 0 .. block end, K is the base.
// Sparse form: queries are the block's active rows (compact q), columns are col_idx[h,b,:], K is
//              rebuilt from the first n_use streams.
// One lane owns one column and adds its queries in ascending order: deterministic, no atomics.
// ----------------------------------------------------------------------------------------------
struct ColScoreArgs {
  const void* q;
  const int32_t* active_idx;
  int n_active;
  DevSide kside;
  int n_use;
  const int32_t* col_idx;
  const int32_t* col_cnt;
  int c;
  const float* lse;
  float* out;
  int L, H, q_block, nb, d, group;
  float scale;
};

constexpr int kCsQBatch = 32;

template <typename T, int DH, int BITS, bool SPARSE>
__global__ void __launch_bounds__(kAttnThreads) colscore_kernel(const __grid_constant__ ColScoreArgs a) {
  extern __shared__ __align__(16) float smem[];
  float4* q4 = reinterpret_cast<float4*>(smem);                   // [8 groups][DH]
  float* lse_s = smem + (kCsQBatch / kQW) * DH * 4;               // [32]
  int* pos_s = reinterpret_cast<int*>(lse_s + kCsQBatch);         // [32]
  float* tiles = reinterpret_cast<float*>(pos_s + kCsQBatch);     // [warps][32][DH+1]
  const int b = blockIdx.y, h = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t prob = (size_t)h * a.nb + b;
  const int blk_lo = b * a.q_block, blk_hi = min(a.L, (b + 1) * a.q_block);
  const int n_cols = SPARSE ? __ldg(a.col_cnt + prob) : blk_hi;
  const int u_cta = blockIdx.x * (kAttnWarps * kChunk);
  if (u_cta >= n_cols) return;
  const int32_t* cols = SPARSE ? a.col_idx + prob * a.c : nullptr;

  // query range of the block
  int q_lo, q_hi;
  if (SPARSE) {
    int lo = 0, hi = a.n_active;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(a.active_idx + mid) < blk_lo) lo = mid + 1; else hi = mid; }
    q_lo = lo; hi = a.n_active;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(a.active_idx + mid) < blk_hi) lo = mid + 1; else hi = mid; }
    q_hi = lo;
  } else {
    q_lo = blk_lo; q_hi = blk_hi;
  }

  // stage this warp's 32 key columns
  float* my_tile = tiles + warp * kChunk * (DH + 1);
  const int u_warp = u_cta + warp * kChunk;
  for (int it = lane; it < kChunk * DH / 8; it += 32) {
    const int u = it / (DH / 8), e = (it % (DH / 8)) * 8;
    const int uu = u_warp + u;
    float kv[8];
    if (uu < n_cols) {
      const int j = SPARSE ? __ldg(cols + uu) : uu;
      recon8<T, BITS>(a.kside, a.n_use, j, h * DH + e, a.d, a.group, kv);
#pragma unroll
      for (int i = 0; i < 8; ++i) kv[i] = to_float<T>(from_float<T>(kv[i]));  // storage precision, as in attention
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) kv[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) my_tile[u * (DH + 1) + e + i] = kv[i];
  }
  const int my_u = u_warp + lane;
  const int my_j = my_u < n_cols ? (SPARSE ? __ldg(cols + my_u) : my_u) : INT32_MAX;
  const int warp_min_j = __shfl_sync(0xffffffffu, my_j, 0);
  float total = 0.f;

  for (int qb = q_lo; qb < q_hi; qb += kCsQBatch) {
    __syncthreads();
    for (int it = threadIdx.x; it < kCsQBatch * DH / 8; it += kAttnThreads) {
      const int qq = it / (DH / 8), e = (it % (DH / 8)) * 8;
      const int qs = qb + qq;  // slot (sparse) or row (dense)
      float qv[8];
      if (qs < q_hi) load8<T>(static_cast<const T*>(a.q) + (size_t)qs * a.d + h * DH + e, qv);
      else {
#pragma unroll
        for (int i = 0; i < 8; ++i) qv[i] = 0.f;
      }
      float* dst = reinterpret_cast<float*>(q4 + (qq / kQW) * DH + e) + (qq % kQW);
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[4 * i] = qv[i];
    }
    if (threadIdx.x < kCsQBatch) {
      const int qs = qb + threadIdx.x;
      int pos = -1;
      if (qs < q_hi) pos = SPARSE ? __ldg(a.active_idx + qs) : qs;
      pos_s[threadIdx.x] = pos;
      lse_s[threadIdx.x] = pos >= 0 ? a.lse[(size_t)h * a.L + pos] : 0.f;
    }
    __syncthreads();
    if (u_warp >= n_cols) continue;
#pragma unroll 1
    for (int g = 0; g < kCsQBatch / kQW; ++g) {
      const int last_pos = max(max(pos_s[g * kQW], pos_s[g * kQW + 1]), max(pos_s[g * kQW + 2], pos_s[g * kQW + 3]));
      if (last_pos < warp_min_j) continue;  // all four rows precede every column of this warp
      float s[kQW];
      warp_qk<DH>(q4 + g * DH, my_tile, lane, s);
#pragma unroll
      for (int qi = 0; qi < kQW; ++qi) {
        const int pos = pos_s[g * kQW + qi];
        if (pos >= 0 && my_j <= pos) total += expf(s[qi] * a.scale - lse_s[g * kQW + qi]);
      }
    }
  }
  if (my_u < n_cols) a.out[prob * (SPARSE ? a.c : a.L) + my_u] = total;
}

template <int DH>
constexpr size_t dense_smem() { return sizeof(float) * (kChunk * (DH + 1) + kChunk * DH + kAttnWarps * DH * 4 + kAttnWarps * kChunk * 4); }
template <int DH>
constexpr size_t colscore_smem() {
  return sizeof(float) * ((kCsQBatch / kQW) * DH * 4 + 2 * kCsQBatch + kAttnWarps * kChunk * (DH + 1));
}

template <typename T, int DH>
int launch_dense(const fl_shape* s, const void* q, const void* k, const void* v, void* o, float* lse, float* col_scores,
                 cudaStream_t st) {
  const int tiles = (s->L + kQTile - 1) / kQTile;
  auto kern = dense_attn_kernel<T, DH>;
  FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dense_smem<DH>()));
  kern<<<dim3(tiles, s->n_heads), kAttnThreads, dense_smem<DH>(), st>>>(
      static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<T*>(o), lse, s->L,
      s->n_heads, s->sm_scale);
  int rc = fl_launch_status();
  if (rc != FL_OK || col_scores == nullptr) return rc;
  ColScoreArgs a{};
  a.q = q; a.active_idx = nullptr; a.n_active = 0;
  a.kside.base = k; a.n_use = 0;
  a.col_idx = nullptr; a.col_cnt = nullptr; a.c = 0;
  a.lse = lse; a.out = col_scores;
  a.L = s->L; a.H = s->n_heads; a.q_block = s->q_block; a.nb = fl_n_blocks(s); a.d = s->n_heads * DH;
  a.group = s->group; a.scale = s->sm_scale;
  auto ck = colscore_kernel<T, DH, 16, false>;
  FL_CHECK_CUDA(cudaFuncSetAttribute(ck, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)colscore_smem<DH>()));
  const int col_groups = (s->L + kAttnWarps * kChunk - 1) / (kAttnWarps * kChunk);
  ck<<<dim3(col_groups, a.nb, s->n_heads), kAttnThreads, colscore_smem<DH>(), st>>>(a);
  return fl_launch_status();
}

}  // namespace

// Used by the sparse loop to emit next-loop column scores (defined here to share the kernel).
int fl_launch_sparse_colscore(const fl_shape* s, const void* q_new, const int32_t* active_idx, int n_active,
                              const DevSide& kside, int n_use, const int32_t* col_idx, const int32_t* col_cnt, int c,
                              const float* lse, float* out, cudaStream_t st) {
  ColScoreArgs a{};
  a.q = q_new; a.active_idx = active_idx; a.n_active = n_active;
  a.kside = kside; a.n_use = n_use;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.lse = lse; a.out = out;
  a.L = s->L; a.H = s->n_heads; a.q_block = s->q_block; a.nb = fl_n_blocks(s); a.d = s->n_heads * s->head_dim;
  a.group = s->group; a.scale = s->sm_scale;
  const int col_groups = (c + kAttnWarps * kChunk - 1) / (kAttnWarps * kChunk);
  const dim3 grid(col_groups, a.nb, s->n_heads);
#define FL_CS_LAUNCH(T, DH, BITS)                                                                                  \
  do {                                                                                                             \
    auto ck = colscore_kernel<T, DH, BITS, true>;                                                                  \
    FL_CHECK_CUDA(cudaFuncSetAttribute(ck, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)colscore_smem<DH>())); \
    ck<<<grid, kAttnThreads, colscore_smem<DH>(), st>>>(a);                                                        \
  } while (0)
#define FL_CS_BITS(T, DH)                          \
  switch (s->bits) {                               \
    case 2: FL_CS_LAUNCH(T, DH, 2); break;         \
    case 4: FL_CS_LAUNCH(T, DH, 4); break;         \
    case 8: FL_CS_LAUNCH(T, DH, 8); break;         \
    default: FL_CS_LAUNCH(T, DH, 16); break;       \
  }
  if (s->dtype == FL_F32) {
    if (s->head_dim == 64) { FL_CS_BITS(float, 64) } else { FL_CS_BITS(float, 128) }
  } else {
    if (s->head_dim == 64) { FL_CS_BITS(__nv_bfloat16, 64) } else { FL_CS_BITS(__nv_bfloat16, 128) }
  }
#undef FL_CS_BITS
#undef FL_CS_LAUNCH
  return fl_launch_status();
}

int fl_launch_dense_tc(fl_ctx* ctx, const fl_shape* s, const void* q, const void* k, const void* v, void* o, float* lse,
                       float* col_scores, int32_t* status, cudaStream_t st);

extern "C" int fl_dense_loop_attention(fl_ctx* ctx, const fl_shape* shape, const void* q, const void* k, const void* v,
                                       void* o, float* lse, float* col_scores, int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(q != nullptr && k != nullptr && v != nullptr && o != nullptr);
  FL_REQUIRE(fl_aligned16(q) && fl_aligned16(k) && fl_aligned16(v) && fl_aligned16(o));
  FL_REQUIRE(col_scores == nullptr || lse != nullptr);
  FL_REQUIRE(shape->n_heads <= 65535 && fl_n_blocks(shape) <= 65535);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // tensor path (bf16 storage, head dimension 128); everything else runs on the binary32 kernels below
  rc = fl_launch_dense_tc(ctx, shape, q, k, v, o, lse, col_scores, status, st);
  if (rc != FL_ERR_UNSUPPORTED) return rc;
  if (shape->dtype == FL_F32)
    return shape->head_dim == 64 ? launch_dense<float, 64>(shape, q, k, v, o, lse, col_scores, st)
                                 : launch_dense<float, 128>(shape, q, k, v, o, lse, col_scores, st);
  return shape->head_dim == 64 ? launch_dense<__nv_bfloat16, 64>(shape, q, k, v, o, lse, col_scores, st)
                               : launch_dense<__nv_bfloat16, 128>(shape, q, k, v, o, lse, col_scores, st);
}
