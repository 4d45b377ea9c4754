// Sparse decode attention (Appendix D.2 as written, for decode positions; Appendix G, the item on sparse decode
// kernels): loop r >= 2 of a batch of single-token queries over the prompt's store. Every (query, head) has its own
// selected column subset and cached mass; nothing is shared between queries, so the work is a gather of the selected
// K/V rows, rebuilt on the way from the base and the residual streams (Eq. 8 chain, dequantize-and-add in
// registers), two dot products and two weighted sums per column: bound by the bytes of the selected rows.
// One CTA per (query, head); a group of dh/8 lanes owns a column at a time (16-byte loads, 8 elements per lane).
#include "attn_simt.cuh"

namespace {

constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;

struct DecodeArgs {
  const void* q_new;     // [B, H, dh]
  const void* q_old;
  const void* o_prev;
  void* o_out;
  DevSide k, v;
  int n_old;             // streams contained in Xhat^(r-1); Xhat^(r) adds stream index n_old
  const int32_t* col_idx;   // [B, H, c]
  const int32_t* col_cnt;   // [B, H]
  int c;
  const float* lse_prev;    // [B, H]
  float* lse_out;           // [B, H]
  float* p_new_out;         // [B, H, c] or null
  int H, d, group;
  float scale;
};

template <int DH>
constexpr size_t decode_smem(int c) {
  constexpr int groups = kDecWarps * (32 / (DH / 8));
  return sizeof(float) * ((size_t)2 * groups * DH + 3 * groups + (size_t)c);
}

// Merge of the CTA's column groups, in a fixed order, and the outputs of one (query, head).
template <typename T, int DH, int G>
__device__ __forceinline__ void decode_merge(const DecodeArgs& a, size_t qh, int cnt, int g, int ch, float lse_p, float mass,
                                             float m_run, float l_run, const float (&acc_o)[8], const float (&acc_n)[8],
                                             float* acc_o_s, float* acc_n_s, float* stat_s, const float* logit_s) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    acc_o_s[g * DH + ch * 8 + i] = acc_o[i];
    acc_n_s[g * DH + ch * 8 + i] = acc_n[i];
  }
  if (ch == 0) { stat_s[g] = mass; stat_s[G + g] = m_run; stat_s[2 * G + g] = l_run; }
  __syncthreads();
  float m_tot = -INFINITY, mass_tot = 0.f;
  for (int gg = 0; gg < G; ++gg) { m_tot = fmaxf(m_tot, stat_s[G + gg]); mass_tot += stat_s[gg]; }
  float l_tot = 0.f;
  for (int gg = 0; gg < G; ++gg)
    l_tot += stat_s[G + gg] > -INFINITY ? stat_s[2 * G + gg] * expf(stat_s[G + gg] - m_tot) : 0.f;
  const bool has = cnt > 0 && m_tot > -INFINITY && mass_tot > 0.f;
  const float w = has ? mass_tot / l_tot : 0.f;
  const T* op = static_cast<const T*>(a.o_prev) + qh * DH;
  T* oo = static_cast<T*>(a.o_out) + qh * DH;
  for (int x = threadIdx.x; x < DH; x += kDecThreads) {
    float so = 0.f, sn = 0.f;
    for (int gg = 0; gg < G; ++gg) {
      so += acc_o_s[gg * DH + x];
      if (stat_s[G + gg] > -INFINITY) sn += acc_n_s[gg * DH + x] * expf(stat_s[G + gg] - m_tot);
    }
    const float prev = to_float<T>(op[x]);
    oo[x] = has ? from_float<T>(prev - so + w * sn) : op[x];
  }
  if (threadIdx.x == 0) a.lse_out[qh] = has ? m_tot + logf(l_tot) - logf(mass_tot) : lse_p;
  if (a.p_new_out != nullptr) {
    float* po = a.p_new_out + qh * a.c;
    for (int u = threadIdx.x; u < a.c; u += kDecThreads) po[u] = (has && u < cnt) ? w * expf(logit_s[u] - m_tot) : 0.f;
  }
}

template <typename T, int DH, int BITS>
__global__ void __launch_bounds__(kDecThreads) decode_attn_kernel(const __grid_constant__ DecodeArgs a) {
  constexpr int LPC = DH / 8;                    // lanes per column
  constexpr int CPW = 32 / LPC;                  // columns a warp handles at a time
  constexpr int G = kDecWarps * CPW;             // column groups of the CTA
  extern __shared__ __align__(16) float smem[];
  float* acc_o_s = smem;                         // [G][DH]
  float* acc_n_s = acc_o_s + G * DH;             // [G][DH]
  float* stat_s = acc_n_s + G * DH;              // [3][G]: mass, running maximum, running sum
  float* logit_s = stat_s + 3 * G;               // [c] scaled new logits (for the probabilities that go out)
  fl_grid_wait();
  fl_grid_release();
  const int t = blockIdx.x, h = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPC, ch = lane % LPC;   // column group inside the warp, 16-byte piece of the row
  const int g = warp * CPW + sub;
  const size_t qh = (size_t)t * a.H + h;
  const int cnt = min(__ldg(a.col_cnt + qh), a.c);
  const int32_t* cols = a.col_idx + qh * a.c;
  const int elem = h * DH + ch * 8;
  float qo[8], qn[8];
  load8<T>(static_cast<const T*>(a.q_old) + qh * DH + ch * 8, qo);
  load8<T>(static_cast<const T*>(a.q_new) + qh * DH + ch * 8, qn);
  const float lse_p = a.lse_prev[qh];
  float mass = 0.f, m_run = -INFINITY, l_run = 0.f, acc_o[8], acc_n[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc_o[i] = acc_n[i] = 0.f;

  for (int u0 = 0; u0 < cnt; u0 += G) {
    const int u = u0 + g;
    const bool on = u < cnt;
    const int j = on ? __ldg(cols + u) : 0;
    float ko[8], kn[8], vo[8], vn[8];
    if (on) {
      recon8<T, BITS>(a.k, a.n_old, j, elem, a.d, a.group, ko);
      recon8<T, BITS>(a.v, a.n_old, j, elem, a.d, a.group, vo);
#pragma unroll
      for (int i = 0; i < 8; ++i) { kn[i] = ko[i]; vn[i] = vo[i]; }
      apply_stream8<T, BITS>(a.k.s[a.n_old], j, elem, a.d, a.group, kn);
      apply_stream8<T, BITS>(a.v.s[a.n_old], j, elem, a.d, a.group, vn);
      // attention consumes the reconstructed rows in storage precision (a bf16 KV cache for bf16 storage)
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        ko[i] = to_float<T>(from_float<T>(ko[i])); kn[i] = to_float<T>(from_float<T>(kn[i]));
        vo[i] = to_float<T>(from_float<T>(vo[i])); vn[i] = to_float<T>(from_float<T>(vn[i]));
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) ko[i] = kn[i] = vo[i] = vn[i] = 0.f;
    }
    float so = 0.f, sn = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) { so = fmaf(qo[i], ko[i], so); sn = fmaf(qn[i], kn[i], sn); }
#pragma unroll
    for (int o = 1; o < LPC; o <<= 1) {
      so += __shfl_xor_sync(0xffffffffu, so, o);
      sn += __shfl_xor_sync(0xffffffffu, sn, o);
    }
    if (on) {
      const float po = expf(so * a.scale - lse_p);
      mass += po;
      const float sv = sn * a.scale;
      if (ch == 0) logit_s[u] = sv;
      const float m_new = fmaxf(m_run, sv);
      const float corr = expf(m_run - m_new);          // 0 on the first column (m_run = -inf)
      const float pn = expf(sv - m_new);
      l_run = l_run * corr + pn;
      m_run = m_new;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        acc_o[i] = fmaf(po, vo[i], acc_o[i]);
        acc_n[i] = fmaf(pn, vn[i], acc_n[i] * corr);
      }
    }
  }
  decode_merge<T, DH, G>(a, qh, cnt, g, ch, lse_p, mass, m_run, l_run, acc_o, acc_n, acc_o_s, acc_n_s, stat_s, logit_s);
}

// The same for bf16 storage, head dimension 128 and at most four residual streams (NS = loop_r - 1), with the
// dependent lookups taken out of the main loop: the column list and, per stream, the slot of every selected column
// are staged in shared memory first (two rounds of independent loads for the whole problem), so that an iteration's
// loads (base rows and payloads of two columns per lane group) depend on nothing but shared memory and the hardware
// keeps several iterations' bytes in flight. Without this every iteration is three dependent trips to memory.
template <int BITS, int NS>
__global__ void __launch_bounds__(kDecThreads) decode_attn_staged_kernel(const __grid_constant__ DecodeArgs a) {
  using T = __nv_bfloat16;
  constexpr int DH = 128, LPC = 16, CPW = 2, G = kDecWarps * CPW, UN = 2;
  extern __shared__ __align__(16) float smem[];
  float* acc_o_s = smem;
  float* acc_n_s = acc_o_s + G * DH;
  float* stat_s = acc_n_s + G * DH;
  float* logit_s = stat_s + 3 * G;
  int32_t* col_s = reinterpret_cast<int32_t*>(logit_s + a.c);          // [c]
  int32_t* slot_s = col_s + a.c;                                       // [NS][c]
  fl_grid_wait();
  fl_grid_release();
  const int t = blockIdx.x, h = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPC, ch = lane % LPC;
  const int g = warp * CPW + sub;
  const size_t qh = (size_t)t * a.H + h;
  const int cnt = min(__ldg(a.col_cnt + qh), a.c);
  const int32_t* cols = a.col_idx + qh * a.c;
  for (int u = threadIdx.x; u < cnt; u += kDecThreads) {
    const int j = __ldg(cols + u);
    col_s[u] = j;
#pragma unroll
    for (int s_ = 0; s_ < NS; ++s_) slot_s[s_ * a.c + u] = __ldg(a.k.s[s_].slot + j);
  }
  const int elem = h * DH + ch * 8;
  float qo[8], qn[8];
  load8<T>(static_cast<const T*>(a.q_old) + qh * DH + ch * 8, qo);
  load8<T>(static_cast<const T*>(a.q_new) + qh * DH + ch * 8, qn);
  const float lse_p = a.lse_prev[qh];
  float mass = 0.f, m_run = -INFINITY, l_run = 0.f, acc_o[8], acc_n[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc_o[i] = acc_n[i] = 0.f;
  __syncthreads();
  const T* kb = static_cast<const T*>(a.k.base) + elem;
  const T* vb = static_cast<const T*>(a.v.base) + elem;
  for (int u0 = 0; u0 < cnt; u0 += G * UN) {
    // every load of the two columns first
    uint4 rk[UN], rv[UN];
    Payload8<T, BITS> pk[UN][NS], pv[UN][NS];
    int sl[UN][NS];
    bool on[UN];
#pragma unroll
    for (int q = 0; q < UN; ++q) {
      const int u = u0 + q * G + g;
      on[q] = u < cnt;
      const int j = on[q] ? col_s[u] : 0;
      rk[q] = on[q] ? __ldg(reinterpret_cast<const uint4*>(kb + (size_t)j * a.d)) : make_uint4(0, 0, 0, 0);
      rv[q] = on[q] ? __ldg(reinterpret_cast<const uint4*>(vb + (size_t)j * a.d)) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int s_ = 0; s_ < NS; ++s_) {
        sl[q][s_] = on[q] ? slot_s[s_ * a.c + u] : -1;
        if (sl[q][s_] >= 0) {
          payload_load<T, BITS>(a.k.s[s_], sl[q][s_], elem, a.d, a.group, pk[q][s_]);
          payload_load<T, BITS>(a.v.s[s_], sl[q][s_], elem, a.d, a.group, pv[q][s_]);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < UN; ++q) {
      float ko[8], kn[8], vo[8], vn[8];
      {
        const __nv_bfloat162* hk = reinterpret_cast<const __nv_bfloat162*>(&rk[q]);
        const __nv_bfloat162* hv = reinterpret_cast<const __nv_bfloat162*>(&rv[q]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 fk = __bfloat1622float2(hk[i]), fv = __bfloat1622float2(hv[i]);
          kn[2 * i] = fk.x; kn[2 * i + 1] = fk.y;
          vn[2 * i] = fv.x; vn[2 * i + 1] = fv.y;
        }
      }
      // Eq. 8 chain in loop order; the state before the loop's own stream is Xhat^(r-1)
#pragma unroll
      for (int s_ = 0; s_ < NS; ++s_) {
        if (s_ == NS - 1) {
#pragma unroll
          for (int i = 0; i < 8; ++i) { ko[i] = kn[i]; vo[i] = vn[i]; }
        }
        if (sl[q][s_] >= 0) {
          payload_apply<T, BITS>(pk[q][s_], kn);
          payload_apply<T, BITS>(pv[q][s_], vn);
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        ko[i] = to_float<T>(from_float<T>(ko[i])); kn[i] = to_float<T>(from_float<T>(kn[i]));
        vo[i] = to_float<T>(from_float<T>(vo[i])); vn[i] = to_float<T>(from_float<T>(vn[i]));
      }
      float so = 0.f, sn = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) { so = fmaf(qo[i], ko[i], so); sn = fmaf(qn[i], kn[i], sn); }
#pragma unroll
      for (int o = 1; o < LPC; o <<= 1) {
        so += __shfl_xor_sync(0xffffffffu, so, o);
        sn += __shfl_xor_sync(0xffffffffu, sn, o);
      }
      if (on[q]) {
        const int u = u0 + q * G + g;
        const float po = expf(so * a.scale - lse_p);
        mass += po;
        const float sv = sn * a.scale;
        if (ch == 0) logit_s[u] = sv;
        const float m_new = fmaxf(m_run, sv);
        const float corr = expf(m_run - m_new);
        const float pn = expf(sv - m_new);
        l_run = l_run * corr + pn;
        m_run = m_new;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          acc_o[i] = fmaf(po, vo[i], acc_o[i]);
          acc_n[i] = fmaf(pn, vn[i], acc_n[i] * corr);
        }
      }
    }
  }
  decode_merge<T, DH, G>(a, qh, cnt, g, ch, lse_p, mass, m_run, l_run, acc_o, acc_n, acc_o_s, acc_n_s, stat_s, logit_s);
}

template <int BITS>
int launch_decode_staged(const fl_ctx* ctx, const DecodeArgs& a, int n_streams, dim3 grid, size_t smem, cudaStream_t st) {
#define FL_DECS(NS)                                                                                       \
  do {                                                                                                    \
    auto kern = decode_attn_staged_kernel<BITS, NS>;                                                      \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));    \
    FL_CHECK_CUDA(fl_launch(ctx, kern, grid, dim3(kDecThreads), smem, st, a));                            \
  } while (0)
  switch (n_streams) {
    case 1: FL_DECS(1); break;
    case 2: FL_DECS(2); break;
    case 3: FL_DECS(3); break;
    default: FL_DECS(4); break;
  }
#undef FL_DECS
  return fl_launch_status();
}

template <typename T, int DH>
int launch_decode(const fl_ctx* ctx, const fl_shape* s, const DecodeArgs& a, int n_queries, cudaStream_t st) {
  const dim3 grid(n_queries, s->n_heads);
  if (sizeof(T) == 2 && DH == 128 && a.n_old + 1 <= 4) {
    const size_t staged = decode_smem<128>(a.c) + sizeof(int32_t) * (size_t)a.c * (a.n_old + 2);
    if (staged <= (size_t)ctx->max_smem_optin) {
      switch (s->bits) {
        case 2: return launch_decode_staged<2>(ctx, a, a.n_old + 1, grid, staged, st);
        case 4: return launch_decode_staged<4>(ctx, a, a.n_old + 1, grid, staged, st);
        case 8: return launch_decode_staged<8>(ctx, a, a.n_old + 1, grid, staged, st);
        default: return launch_decode_staged<16>(ctx, a, a.n_old + 1, grid, staged, st);
      }
    }
  }
  const size_t smem = decode_smem<DH>(a.c);
#define FL_DEC(BITS)                                                                                      \
  do {                                                                                                    \
    auto kern = decode_attn_kernel<T, DH, BITS>;                                                          \
    FL_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));    \
    FL_CHECK_CUDA(fl_launch(ctx, kern, grid, dim3(kDecThreads), smem, st, a));                            \
  } while (0)
  switch (s->bits) {
    case 2: FL_DEC(2); break;
    case 4: FL_DEC(4); break;
    case 8: FL_DEC(8); break;
    default: FL_DEC(16); break;
  }
#undef FL_DEC
  return fl_launch_status();
}

}  // namespace

extern "C" int fl_decode_attention(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new, const void* q_old,
                                   int32_t n_queries, const fl_kv_store* store, const int32_t* col_idx,
                                   const int32_t* col_cnt, int32_t c, const float* lse_prev, float* lse_out,
                                   const void* o_prev, void* o_out, float* p_new_out, int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(loop_r >= 2 && loop_r <= FL_MAX_LOOPS + 1);
  FL_REQUIRE(n_queries >= 0 && c >= 1);
  rc = fl_check_store(shape, store, loop_r - 1);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(col_idx != nullptr && col_cnt != nullptr && lse_prev != nullptr && lse_out != nullptr);
  FL_REQUIRE(n_queries <= 65535 * 32 && shape->n_heads <= 65535);
  if (n_queries == 0) return FL_OK;
  FL_REQUIRE(q_new != nullptr && q_old != nullptr && o_prev != nullptr && o_out != nullptr);
  FL_REQUIRE(fl_aligned16(q_new) && fl_aligned16(q_old) && fl_aligned16(o_prev) && fl_aligned16(o_out));
  const size_t smem = shape->head_dim == 64 ? decode_smem<64>(c) : decode_smem<128>(c);
  if (smem > (size_t)ctx->max_smem_optin) return FL_ERR_UNSUPPORTED;
  rc = fl_debug_check_attn(ctx, shape, loop_r - 1, nullptr, 0, store, col_idx, col_cnt, c,
                           (int64_t)n_queries * shape->n_heads, status, stream);
  if (rc != FL_OK) return rc;
  DecodeArgs a{};
  a.q_new = q_new; a.q_old = q_old; a.o_prev = o_prev; a.o_out = o_out;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.n_old = loop_r - 2;
  a.col_idx = col_idx; a.col_cnt = col_cnt; a.c = c;
  a.lse_prev = lse_prev; a.lse_out = lse_out; a.p_new_out = p_new_out;
  a.H = shape->n_heads; a.d = shape->n_heads * shape->head_dim; a.group = shape->group; a.scale = shape->sm_scale;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (shape->dtype == FL_F32)
    return shape->head_dim == 64 ? launch_decode<float, 64>(ctx, shape, a, n_queries, st)
                                 : launch_decode<float, 128>(ctx, shape, a, n_queries, st);
  return shape->head_dim == 64 ? launch_decode<__nv_bfloat16, 64>(ctx, shape, a, n_queries, st)
                               : launch_decode<__nv_bfloat16, 128>(ctx, shape, a, n_queries, st);
}
