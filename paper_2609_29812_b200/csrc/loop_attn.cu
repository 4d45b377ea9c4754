// Stages 2 + 4: attention replacement of Eq. 7 over K/V rebuilt inside the kernel from the packed
// base + residual streams (Eq. 8). This file holds the binary32 SIMT kernel (every storage type and
// head dimension) and the entry point, which dispatches to the tensor-core kernel when it applies.
#include "attn_simt.cuh"

int fl_launch_sparse_colscore(const fl_shape* s, const void* q_new, const int32_t* active_idx, int n_active,
                              const DevSide& kside, int n_use, const int32_t* col_idx, const int32_t* col_cnt, int c,
                              const float* lse, float* out, cudaStream_t st);

int fl_launch_sparse_colsum_tc(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const int32_t* active_idx,
                               int n_active, const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt,
                               int c, const float* lse, float* out, int32_t* status, cudaStream_t st);

// next-loop column scores: tensor path when it covers the request, the binary32 kernel otherwise
static int fl_next_col_scores(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const int32_t* active_idx,
                              int n_active, const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt,
                              int c, const float* lse, float* out, int32_t* status, cudaStream_t st);

int fl_launch_loop_attn_tc(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_old,
                           const int32_t* active_idx, int n_active, const fl_kv_store* store, const int32_t* col_idx,
                           const int32_t* col_cnt, int c, const float* lse_prev, float* lse_out, const void* o_prev,
                           void* o_out, int indexed, void* q_store, const fl_attn_carry* carry, int32_t* status,
                           cudaStream_t st);

// the same call as one or two single-term launches (needs the loop's materialized rows and the carried buffers)
int fl_launch_loop_attn_stream(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const void* q_store_in,
                               void* q_store_out, const int32_t* active_idx, int n_active, const fl_kv_store* store,
                               const int32_t* col_idx, const int32_t* col_cnt, int c, const float* lse_in,
                               float* lse_out, const void* o_store_in, void* o_store_out, const fl_attn_carry* carry,
                               int32_t* status, cudaStream_t st);

// whether the tensor-path kernel has a build for this request (storage type, head dimension, column budget, shared memory)
bool fl_loop_attn_tc_covers(const fl_ctx* ctx, const fl_shape* s, int c);

namespace {

struct LoopAttnArgs {
  const void* q_new;
  const void* q_old;
  const void* o_prev;
  void* o_out;
  const int32_t* active_idx;
  int n_active;
  DevSide k, v;
  int n_old;  // streams contained in Xhat^(r-1); Xhat^(r) adds stream index n_old
  const int32_t* col_idx;
  const int32_t* col_cnt;
  int c;
  const float* lse_prev;
  float* lse_out;
  int L, H, q_block, nb, d, group;
  float scale;
};

template <int DH>
constexpr size_t loop_smem() {
  return sizeof(float) * (2 * kChunk * (DH + 1) + 2 * kChunk * DH + 2 * kAttnWarps * DH * 4 + 2 * kAttnWarps * kChunk * 4);
}

template <typename T, int DH, int BITS>
__global__ void __launch_bounds__(kAttnThreads) loop_attn_kernel(const __grid_constant__ LoopAttnArgs a) {
  extern __shared__ __align__(16) float smem[];
  float* k_old = smem;                                   // [32][DH+1]
  float* k_new = k_old + kChunk * (DH + 1);
  float* v_old = k_new + kChunk * (DH + 1);              // [32][DH]
  float* v_new = v_old + kChunk * DH;
  float4* qn4 = reinterpret_cast<float4*>(v_new + kChunk * DH);  // [warps][DH]
  float4* qo4 = qn4 + kAttnWarps * DH;
  float4* pn4 = qo4 + kAttnWarps * DH;                   // [warps][32]
  float4* po4 = pn4 + kAttnWarps * kChunk;

  const int b = blockIdx.y, h = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t prob = (size_t)h * a.nb + b;
  const int blk_lo = b * a.q_block, blk_hi = min(a.L, (b + 1) * a.q_block);
  int lo = 0, hi = a.n_active;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(a.active_idx + mid) < blk_lo) lo = mid + 1; else hi = mid; }
  const int q_lo = lo; hi = a.n_active;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (__ldg(a.active_idx + mid) < blk_hi) lo = mid + 1; else hi = mid; }
  const int q_hi = lo;
  const int s0 = q_lo + blockIdx.x * kQTile;
  if (s0 >= q_hi) return;
  const int s_end = min(q_hi, s0 + kQTile);
  const int i_max = __ldg(a.active_idx + s_end - 1);
  const int cnt = __ldg(a.col_cnt + prob);
  const int32_t* cols = a.col_idx + prob * a.c;

  // this warp's four query rows
  int slot[kQW], pos[kQW];
  float lse_i[kQW];
#pragma unroll
  for (int qi = 0; qi < kQW; ++qi) {
    slot[qi] = s0 + warp * kQW + qi;
    pos[qi] = slot[qi] < s_end ? __ldg(a.active_idx + slot[qi]) : -1;
    lse_i[qi] = pos[qi] >= 0 ? a.lse_prev[(size_t)h * a.L + pos[qi]] : 0.f;
  }
  const T* qn = static_cast<const T*>(a.q_new);
  const T* qo = static_cast<const T*>(a.q_old);
  for (int x = lane; x < DH; x += 32) {
    float vn[kQW], vo[kQW];
#pragma unroll
    for (int qi = 0; qi < kQW; ++qi) {
      const size_t off = (size_t)slot[qi] * a.d + h * DH + x;
      vn[qi] = pos[qi] >= 0 ? to_float<T>(qn[off]) : 0.f;
      vo[qi] = pos[qi] >= 0 ? to_float<T>(qo[off]) : 0.f;
    }
    qn4[warp * DH + x] = make_float4(vn[0], vn[1], vn[2], vn[3]);
    qo4[warp * DH + x] = make_float4(vo[0], vo[1], vo[2], vo[3]);
  }
  float m_run[kQW], l_run[kQW], mass[kQW], acc_n[kQW][DH / 32], acc_o[kQW][DH / 32];
#pragma unroll
  for (int qi = 0; qi < kQW; ++qi) {
    m_run[qi] = -INFINITY; l_run[qi] = 0.f; mass[qi] = 0.f;
#pragma unroll
    for (int t = 0; t < DH / 32; ++t) acc_n[qi][t] = acc_o[qi][t] = 0.f;
  }

  for (int u0 = 0; u0 < cnt; u0 += kChunk) {
    if (__ldg(cols + u0) > i_max) break;  // columns ascend: nothing causal is left for this tile
    __syncthreads();
    // gather + dequantize-and-add: rebuild Khat/Vhat of loops r-1 and r for 32 selected columns
    for (int it = threadIdx.x; it < 2 * kChunk * DH / 8; it += kAttnThreads) {
      const int is_v = it / (kChunk * DH / 8);
      const int rem = it % (kChunk * DH / 8);
      const int u = rem / (DH / 8), e = (rem % (DH / 8)) * 8;
      const int j = (u0 + u < cnt) ? __ldg(cols + u0 + u) : -1;
      float xo[8], xn[8];
      if (j >= 0) {
        const DevSide& side = is_v ? a.v : a.k;
        recon8<T, BITS>(side, a.n_old, j, h * DH + e, a.d, a.group, xo);
#pragma unroll
        for (int i = 0; i < 8; ++i) xn[i] = xo[i];
        apply_stream8<T, BITS>(side.s[a.n_old], j, h * DH + e, a.d, a.group, xn);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) xo[i] = xn[i] = 0.f;
      }
      // attention consumes the reconstructed rows in storage precision (a bf16 KV cache for bf16 storage)
#pragma unroll
      for (int i = 0; i < 8; ++i) { xo[i] = to_float<T>(from_float<T>(xo[i])); xn[i] = to_float<T>(from_float<T>(xn[i])); }
      if (is_v) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { v_old[u * DH + e + i] = xo[i]; v_new[u * DH + e + i] = xn[i]; }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) { k_old[u * (DH + 1) + e + i] = xo[i]; k_new[u * (DH + 1) + e + i] = xn[i]; }
      }
    }
    __syncthreads();
    const int j = (u0 + lane < cnt) ? __ldg(cols + u0 + lane) : INT32_MAX;
    float so[kQW], sn[kQW], pn[kQW], po[kQW];
    warp_qk<DH>(qo4 + warp * DH, k_old, lane, so);
    warp_qk<DH>(qn4 + warp * DH, k_new, lane, sn);
#pragma unroll
    for (int qi = 0; qi < kQW; ++qi) {
      const bool valid = pos[qi] >= 0 && j <= pos[qi];
      po[qi] = valid ? expf(so[qi] * a.scale - lse_i[qi]) : 0.f;
      mass[qi] += po[qi];
      const float sv = valid ? sn[qi] * a.scale : -INFINITY;
      const float m_new = fmaxf(m_run[qi], warp_max(sv));
      float corr = 1.f;
      pn[qi] = 0.f;
      if (m_new > -INFINITY) {
        corr = expf(m_run[qi] - m_new);
        pn[qi] = valid ? expf(sv - m_new) : 0.f;
      }
      l_run[qi] = l_run[qi] * corr + warp_sum(pn[qi]);
#pragma unroll
      for (int t = 0; t < DH / 32; ++t) acc_n[qi][t] *= corr;
      m_run[qi] = m_new;
    }
    pn4[warp * kChunk + lane] = make_float4(pn[0], pn[1], pn[2], pn[3]);
    po4[warp * kChunk + lane] = make_float4(po[0], po[1], po[2], po[3]);
    __syncwarp();
    warp_pv<DH>(po4 + warp * kChunk, v_old, lane, acc_o);
    warp_pv<DH>(pn4 + warp * kChunk, v_new, lane, acc_n);
    __syncwarp();
  }

  const T* op = static_cast<const T*>(a.o_prev);
  T* oo = static_cast<T*>(a.o_out);
#pragma unroll
  for (int qi = 0; qi < kQW; ++qi) {
    if (pos[qi] < 0) continue;
    const float m_i = warp_sum(mass[qi]);
    const size_t off = (size_t)slot[qi] * a.d + h * DH;
    if (m_run[qi] > -INFINITY) {  // T_i not empty
      const float w = m_i / l_run[qi];
#pragma unroll
      for (int t = 0; t < DH / 32; ++t) {
        const float prev = to_float<T>(op[off + lane + 32 * t]);
        oo[off + lane + 32 * t] = from_float<T>(prev - acc_o[qi][t] + w * acc_n[qi][t]);
      }
      if (lane == 0) a.lse_out[(size_t)h * a.L + pos[qi]] = m_run[qi] + logf(l_run[qi]) - logf(m_i);
    } else {
      if (oo != op) {
#pragma unroll
        for (int t = 0; t < DH / 32; ++t) oo[off + lane + 32 * t] = op[off + lane + 32 * t];
      }
      if (lane == 0) a.lse_out[(size_t)h * a.L + pos[qi]] = lse_i[qi];
    }
  }
}

template <typename T, int DH>
int launch_loop(const fl_shape* s, const LoopAttnArgs& a, int max_tiles, cudaStream_t st) {
  const dim3 grid(max_tiles, a.nb, s->n_heads);
#define FL_LA(BITS)                                                                                               \
  do {                                                                                                            \
    auto kern = loop_attn_kernel<T, DH, BITS>;                                                                    \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)loop_smem<DH>())); \
    kern<<<grid, kAttnThreads, loop_smem<DH>(), st>>>(a);                                                         \
  } while (0)
  switch (s->bits) {
    case 2: FL_LA(2); break;
    case 4: FL_LA(4); break;
    case 8: FL_LA(8); break;
    default: FL_LA(16); break;
  }
#undef FL_LA
  return fl_launch_status();
}

}  // namespace

extern "C" int fl_loop_attention(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new, const void* q_old,
                                 const int32_t* active_idx, int32_t n_active, const fl_kv_store* store,
                                 const int32_t* col_idx, const int32_t* col_cnt, int32_t c, const float* lse_prev,
                                 float* lse_out, const void* o_prev, void* o_out, float* col_scores_next,
                                 int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(loop_r >= 2 && loop_r <= FL_MAX_LOOPS + 1);
  FL_REQUIRE(n_active >= 0 && n_active <= shape->L && c >= 1);
  rc = fl_check_store(shape, store, loop_r - 1);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(col_idx != nullptr && col_cnt != nullptr && lse_prev != nullptr && lse_out != nullptr);
  FL_REQUIRE(shape->n_heads <= 65535 && fl_n_blocks(shape) <= 65535);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n_active == 0) {
    if (col_scores_next != nullptr)
      FL_CHECK_CUDA(cudaMemsetAsync(col_scores_next, 0,
                                    sizeof(float) * (size_t)shape->n_heads * fl_n_blocks(shape) * c, st));
    return FL_OK;
  }
  FL_REQUIRE(q_new != nullptr && q_old != nullptr && o_prev != nullptr && o_out != nullptr && active_idx != nullptr);
  FL_REQUIRE(fl_aligned16(q_new) && fl_aligned16(q_old) && fl_aligned16(o_prev) && fl_aligned16(o_out));
  rc = fl_debug_check_attn(ctx, shape, loop_r - 1, active_idx, n_active, store, col_idx, col_cnt, c,
                           (int64_t)shape->n_heads * fl_n_blocks(shape), status, stream);
  if (rc != FL_OK) return rc;

  DevSide kside;
  fl_dev_side(store, true, &kside);
  if (!ctx->force_simt) {
    // tensor path (bf16 storage, head_dim 128); anything else runs on the binary32 SIMT kernel below
    rc = fl_launch_loop_attn_tc(ctx, shape, loop_r, q_new, q_old, active_idx, n_active, store, col_idx, col_cnt, c,
                                lse_prev, lse_out, o_prev, o_out, 0, nullptr, nullptr, status, st);
    if (rc == FL_OK) {
      if (col_scores_next == nullptr) return FL_OK;
      return fl_next_col_scores(ctx, shape, loop_r, q_new, active_idx, n_active, store, col_idx, col_cnt, c, lse_out,
                                col_scores_next, status, st);
    }
    if (rc != FL_ERR_UNSUPPORTED) return rc;
  }
  LoopAttnArgs a{};
  a.q_new = q_new; a.q_old = q_old; a.o_prev = o_prev; a.o_out = o_out;
  a.active_idx = active_idx; a.n_active = n_active;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.n_old = loop_r - 2;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.lse_prev = lse_prev; a.lse_out = lse_out;
  a.L = shape->L; a.H = shape->n_heads; a.q_block = shape->q_block; a.nb = fl_n_blocks(shape);
  a.d = shape->n_heads * shape->head_dim; a.group = shape->group; a.scale = shape->sm_scale;
  const int per_block = shape->q_block < n_active ? shape->q_block : n_active;
  const int max_tiles = (per_block + kQTile - 1) / kQTile;
  if (shape->dtype == FL_F32)
    rc = shape->head_dim == 64 ? launch_loop<float, 64>(shape, a, max_tiles, st)
                               : launch_loop<float, 128>(shape, a, max_tiles, st);
  else
    rc = shape->head_dim == 64 ? launch_loop<__nv_bfloat16, 64>(shape, a, max_tiles, st)
                               : launch_loop<__nv_bfloat16, 128>(shape, a, max_tiles, st);
  if (rc != FL_OK || col_scores_next == nullptr) return rc;
  // column scores that prepare a pruned selection for loop r+1 (Eq. 6 with a sparse source loop)
  return fl_next_col_scores(ctx, shape, loop_r, q_new, active_idx, n_active, store, col_idx, col_cnt, c, lse_out,
                            col_scores_next, status, st);
}

// Host-side checks of the position-indexed form, shared with the entry point that brings its own scratch.
// Returns FL_OK with *launch = 1 when a kernel is to be launched, FL_OK with *launch = 0 when the call has nothing
// to compute (no active rows), or the error every caller reports before anything is enqueued.
int fl_attn_indexed_check(const fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                          const void* q_store_in, const void* q_store_out, const int32_t* active_idx, int32_t n_active,
                          const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt, int32_t c,
                          const float* lse_in, const float* lse_out, const void* o_store_in, const void* o_store_out,
                          const fl_attn_carry* carry, int* launch) {
  *launch = 0;
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(loop_r >= 2 && loop_r <= FL_MAX_LOOPS + 1);
  FL_REQUIRE(n_active >= 0 && n_active <= shape->L && c >= 1);
  rc = fl_check_store(shape, store, loop_r - 1);
  if (rc != FL_OK) return rc;
  // a call that reuses the carried old term reads neither the previous loop's Q and O rows nor its log-normalisers
  const bool reuse = carry != nullptr && carry->reuse != 0;
  FL_REQUIRE(col_idx != nullptr && col_cnt != nullptr && lse_out != nullptr && (reuse || lse_in != nullptr));
  FL_REQUIRE(shape->n_heads <= 65535 && fl_n_blocks(shape) <= 65535);
  if (carry != nullptr) {
    FL_REQUIRE(carry->bg_store != nullptr && carry->mass != nullptr && fl_aligned16(carry->bg_store));
    FL_REQUIRE(carry->bg_store != o_store_out && carry->bg_store != o_store_in);
  }
  if (n_active == 0) return FL_OK;
  FL_REQUIRE(q_new != nullptr && o_store_out != nullptr && active_idx != nullptr);
  FL_REQUIRE(reuse || (q_store_in != nullptr && o_store_in != nullptr));
  FL_REQUIRE(fl_aligned16(q_new) && fl_aligned16(q_store_in) && fl_aligned16(q_store_out) &&
             fl_aligned16(o_store_in) && fl_aligned16(o_store_out));
  if (ctx->force_simt) return FL_ERR_UNSUPPORTED;
  if (!fl_loop_attn_tc_covers(ctx, shape, c)) return FL_ERR_UNSUPPORTED;
  *launch = 1;
  return FL_OK;
}

extern "C" int fl_loop_attention_indexed_carry(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                                               const void* q_store_in, void* q_store_out, const int32_t* active_idx,
                                               int32_t n_active, const fl_kv_store* store, const int32_t* col_idx,
                                               const int32_t* col_cnt, int32_t c, const float* lse_in, float* lse_out,
                                               const void* o_store_in, void* o_store_out, const fl_attn_carry* carry,
                                               float* col_scores_next, int32_t* status, void* stream) {
  int launch = 0;
  int rc = fl_attn_indexed_check(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active, store,
                                 col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out, carry, &launch);
  if (rc != FL_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!launch) {
    if (col_scores_next != nullptr)
      FL_CHECK_CUDA(cudaMemsetAsync(col_scores_next, 0,
                                    sizeof(float) * (size_t)shape->n_heads * fl_n_blocks(shape) * c, st));
    return FL_OK;
  }
  rc = fl_debug_check_attn(ctx, shape, loop_r - 1, active_idx, n_active, store, col_idx, col_cnt, c,
                           (int64_t)shape->n_heads * fl_n_blocks(shape), status, stream);
  if (rc != FL_OK) return rc;
  // With the carried buffers and the loop's materialized rows a call that reuses the old term runs the single-term
  // kernel (new term only, two CTAs per SM). A recomputing call stays on the fused kernel, whose two terms share the
  // gathered tiles of every column without a payload in this loop (the gathers are what bounds these kernels);
  // FL_TWO_PASS=1 at fl_create sends it through the single-term kernel twice instead (old-term pass, new-term pass).
  rc = FL_ERR_UNSUPPORTED;
  if (carry != nullptr && !ctx->fused_attn && (carry->reuse != 0 || ctx->two_pass))
    rc = fl_launch_loop_attn_stream(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active, store,
                                    col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out, carry, status, st);
  if (rc == FL_ERR_UNSUPPORTED)
    rc = fl_launch_loop_attn_tc(ctx, shape, loop_r, q_new, q_store_in, active_idx, n_active, store, col_idx, col_cnt,
                                c, lse_in, lse_out, o_store_in, o_store_out, 1, q_store_out, carry, status, st);
  if (rc != FL_OK || col_scores_next == nullptr) return rc;
  return fl_next_col_scores(ctx, shape, loop_r, q_new, active_idx, n_active, store, col_idx, col_cnt, c, lse_out,
                            col_scores_next, status, st);
}

extern "C" int fl_loop_attention_indexed(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                                         const void* q_store_in, void* q_store_out, const int32_t* active_idx,
                                         int32_t n_active, const fl_kv_store* store, const int32_t* col_idx,
                                         const int32_t* col_cnt, int32_t c, const float* lse_in, float* lse_out,
                                         const void* o_store_in, void* o_store_out, float* col_scores_next,
                                         int32_t* status, void* stream) {
  return fl_loop_attention_indexed_carry(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active,
                                         store, col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out, nullptr,
                                         col_scores_next, status, stream);
}

static int fl_next_col_scores(fl_ctx* ctx, const fl_shape* s, int loop_r, const void* q_new, const int32_t* active_idx,
                              int n_active, const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt,
                              int c, const float* lse, float* out, int32_t* status, cudaStream_t st) {
  const int rc = fl_launch_sparse_colsum_tc(ctx, s, loop_r, q_new, active_idx, n_active, store, col_idx, col_cnt, c, lse,
                                            out, status, st);
  if (rc != FL_ERR_UNSUPPORTED) return rc;
  DevSide kside;
  fl_dev_side(store, true, &kside);
  return fl_launch_sparse_colscore(s, q_new, active_idx, n_active, kside, loop_r - 1, col_idx, col_cnt, c, lse, out, st);
}
