// Quantized loop-1 base (Appendix E, "Quantization Setting"): the same asymmetric min/max quantizer as the residual
// streams, with the keys grouped per channel (a group = `group` consecutive positions of one channel) and the values
// per token (a group = `group` consecutive channels of one position); the most recent `tail` positions stay in the
// storage type. fl_quant_kv_base packs a layer's K and V once, after its dense loop; fl_dequant_kv_base rebuilds the
// rows the sparse loops read (code * scale + offset with one binary32 rounding, then one rounding to the storage
// type), so that the cache at rest is the packed form and the bf16 rows are a transient working copy of one layer.
// HBM-bound kernels, 16-byte accesses, bit-exact arithmetic (binary32, directed fp16 roundings of the metadata).
#include "fl_internal.cuh"

namespace {

struct BaseArgs {
  const void* k; const void* v;        // quantize: inputs [L, d]; dequantize: unused
  void* k_out; void* v_out;            // dequantize: outputs [L, d]; quantize: unused
  const void* k_tail; const void* v_tail;   // dequantize: rows Lq .. L-1 in the storage type
  int L;
  uint8_t* k_codes; __half* k_scale; __half* k_zero;
  uint8_t* v_codes; __half* v_scale; __half* v_zero;
  const uint32_t* row_mask;            // dequantize: bit t of word [h][t / 32] set = rebuild row t of head h; null = all rows
  int Lq, d, group, dh, mask_words;
};

template <int BITS>
__device__ __forceinline__ void store_codes8(uint8_t* row, int elem, const float (&q)[8]) {
  uint32_t c[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) c[i] = (uint32_t)q[i];
  if (BITS == 8) {
    *reinterpret_cast<uint2*>(row + elem) = make_uint2(c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24),
                                                       c[4] | (c[5] << 8) | (c[6] << 16) | (c[7] << 24));
  } else if (BITS == 4) {
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) w |= c[i] << (4 * i);
    *reinterpret_cast<uint32_t*>(row + elem / 2) = w;
  } else {
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) w |= c[i] << (2 * i);
    *reinterpret_cast<uint16_t*>(row + elem / 4) = (uint16_t)w;
  }
}

// scale and offset of one group from its minimum and maximum: offset rounded down, scale rounded up (fp16)
template <int BITS>
__device__ __forceinline__ void group_meta(float mn, float mx, __half& zh, __half& sh) {
  zh = __float2half_rd(mn);
  const float range = __fsub_rn(mx, __half2float(zh));
  sh = range == 0.f ? __float2half_rn(0.f) : __float2half_ru(__fdiv_rn(range, (float)((1 << BITS) - 1)));
}

template <int BITS>
__device__ __forceinline__ float code_of(float x, float zf, float sf) {
  if (sf == 0.f) return 0.f;
  const float q = rintf(__fdiv_rn(__fsub_rn(x, zf), sf));          // round half to even
  return fminf(fmaxf(q, 0.f), (float)((1 << BITS) - 1));
}

// Keys: one CTA per group of `group` consecutive positions, one thread per 8 channels. Two passes over the
// group's rows (the second finds them in L2): minimum and maximum per channel, then the codes.
template <typename T, int BITS>
__global__ void __launch_bounds__(256) base_quant_k_kernel(const __grid_constant__ BaseArgs a) {
  const int g = blockIdx.x;
  const int t0 = g * a.group, t1 = min(a.Lq, t0 + a.group);
  const T* k = static_cast<const T*>(a.k);
  for (int elem = (blockIdx.y * blockDim.x + threadIdx.x) * 8; elem < a.d; elem += gridDim.y * blockDim.x * 8) {
    float mn[8], mx[8], x[8];
    load8<T>(k + (size_t)t0 * a.d + elem, mn);
#pragma unroll
    for (int i = 0; i < 8; ++i) mx[i] = mn[i];
    for (int t = t0 + 1; t < t1; ++t) {
      load8<T>(k + (size_t)t * a.d + elem, x);
#pragma unroll
      for (int i = 0; i < 8; ++i) { mn[i] = fminf(mn[i], x[i]); mx[i] = fmaxf(mx[i], x[i]); }
    }
    __align__(16) __half zh[8];
    __align__(16) __half sh[8];
    float zf[8], sf[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      group_meta<BITS>(mn[i], mx[i], zh[i], sh[i]);
      zf[i] = __half2float(zh[i]);
      sf[i] = __half2float(sh[i]);
    }
    *reinterpret_cast<uint4*>(a.k_zero + (size_t)g * a.d + elem) = *reinterpret_cast<const uint4*>(zh);
    *reinterpret_cast<uint4*>(a.k_scale + (size_t)g * a.d + elem) = *reinterpret_cast<const uint4*>(sh);
    for (int t = t0; t < t1; ++t) {
      load8<T>(k + (size_t)t * a.d + elem, x);
      float q[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) q[i] = code_of<BITS>(x[i], zf[i], sf[i]);
      store_codes8<BITS>(a.k_codes + (size_t)t * (a.d * BITS / 8), elem, q);
    }
  }
}

// Values: one thread per 8 consecutive channels of a position; the group's minimum and maximum by shuffles over
// the group / 8 lanes that share it. blockDim.x * 8 divides d or is a multiple of it in whole rows (host).
template <typename T, int BITS>
__global__ void __launch_bounds__(256) base_quant_v_kernel(const __grid_constant__ BaseArgs a) {
  const int per_row = a.d >> 3;
  const int lanes_per_group = a.group >> 3;
  const int64_t total = (int64_t)a.Lq * per_row;      // a multiple of 32: d % 256 == 0
  const T* v = static_cast<const T*>(a.v);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / per_row), elem = (int)(i - (int64_t)t * per_row) * 8;
    float x[8];
    load8<T>(v + (size_t)t * a.d + elem, x);
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int u = 1; u < 8; ++u) { mn = fminf(mn, x[u]); mx = fmaxf(mx, x[u]); }
    for (int o = 1; o < lanes_per_group; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    __half zh, sh;
    group_meta<BITS>(mn, mx, zh, sh);
    const float zf = __half2float(zh), sf = __half2float(sh);
    float q[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) q[u] = code_of<BITS>(x[u], zf, sf);
    store_codes8<BITS>(a.v_codes + (size_t)t * (a.d * BITS / 8), elem, q);
    if (((elem >> 3) & (lanes_per_group - 1)) == 0) {
      const int gs = 31 - __clz(a.group);
      const size_t gi = (size_t)t * (a.d >> gs) + (elem >> gs);
      a.v_scale[gi] = sh;
      a.v_zero[gi] = zh;
    }
  }
}

// Rebuild rows [0, Lq) of K and V in the storage type: blockIdx.y = 0 keys (metadata per token group and channel),
// 1 values (metadata per token and channel group). One thread per 8 channels of a position, four positions per
// thread and pass so that their loads are in flight together. With a row mask only the (head, position) pairs whose
// bit is set are rebuilt; everything else of the output is left as it is.
template <typename T, int BITS>
__global__ void __launch_bounds__(256) base_dequant_kernel(const __grid_constant__ BaseArgs a) {
  fl_grid_wait();
  fl_grid_release();
  const bool is_v = blockIdx.y != 0;
  const int per_row = a.d >> 3;
  const int gs = 31 - __clz(a.group);
  const uint8_t* codes = is_v ? a.v_codes : a.k_codes;
  const __half* scale = is_v ? a.v_scale : a.k_scale;
  const __half* zero = is_v ? a.v_zero : a.k_zero;
  T* out = static_cast<T*>(is_v ? a.v_out : a.k_out);
  constexpr int U = 4;      // rows whose loads are in flight together
  // the unquantized tail rows, copied as they are (always: they are few)
  {
    const T* tail = static_cast<const T*>(is_v ? a.v_tail : a.k_tail);
    const int n_vec = (a.L - a.Lq) * per_row * (int)(sizeof(T) * 8 / 16);
    const uint4* src = reinterpret_cast<const uint4*>(tail);
    uint4* dst = reinterpret_cast<uint4*>(out + (size_t)a.Lq * a.d);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += gridDim.x * blockDim.x) dst[i] = __ldg(src + i);
  }
  // A CTA owns a run of consecutive rows and its threads the same 8 channels of each. Per batch of four rows a thread
  // makes two trips to memory: its head's mask bits (two words), then the codes (and the values' metadata) of every
  // wanted row at once. The keys' scales and offsets (per channel and token group) are read and converted once per
  // token group, not once per row. The code becomes a float by arithmetic (2^23 + c is exact), not by a conversion:
  // conversions run on a narrow pipe.
  const int rows_per_cta = (a.Lq + gridDim.x - 1) / gridDim.x;
  const int r_lo = blockIdx.x * rows_per_cta, r_hi = min(a.Lq, r_lo + rows_per_cta);
  for (int v0 = threadIdx.x; v0 < per_row; v0 += blockDim.x) {
    const int elem = v0 * 8;
    const int head = elem / a.dh;
    int tg_cached = -1;
    float ksc[8], kzr[8];
    for (int t0 = r_lo; t0 < r_hi; t0 += U) {
      uint32_t want = (1u << U) - 1u;                          // bit u: row t0 + u is rebuilt
      if (a.row_mask != nullptr) {
        const uint32_t* mrow = a.row_mask + (size_t)head * a.mask_words;
        const int w = t0 >> 5;
        const uint32_t lo = __ldg(mrow + w), hi = w + 1 < a.mask_words ? __ldg(mrow + w + 1) : 0u;
        want = __funnelshift_r(lo, hi, t0 & 31) & ((1u << U) - 1u);
      }
      if (r_hi - t0 < U) want &= (1u << (r_hi - t0)) - 1u;
      if (want == 0u) continue;
      uint32_t raw[U][BITS == 8 ? 2 : 1];
      __half vsh[U], vzh[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (!((want >> u) & 1u)) continue;
        const int t = t0 + u;
        const uint8_t* row = codes + (size_t)t * (a.d * BITS / 8);
        if (BITS == 8) {
          const uint2 r2 = __ldg(reinterpret_cast<const uint2*>(row + elem));
          raw[u][0] = r2.x; raw[u][BITS == 8 ? 1 : 0] = r2.y;
        } else if (BITS == 4) {
          raw[u][0] = __ldg(reinterpret_cast<const uint32_t*>(row + elem / 2));
        } else {
          raw[u][0] = __ldg(reinterpret_cast<const uint16_t*>(row + elem / 4));
        }
        if (is_v) {
          const size_t gi = (size_t)t * (a.d >> gs) + (elem >> gs);
          vsh[u] = __ldg(scale + gi);
          vzh[u] = __ldg(zero + gi);
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (!((want >> u) & 1u)) continue;
        const int t = t0 + u;
        float x[8];
        if (!is_v) {
          if ((t >> gs) != tg_cached) {      // the same for every thread of the CTA
            tg_cached = t >> gs;
            const size_t mi = (size_t)tg_cached * a.d + elem;
            const uint4 sraw = __ldg(reinterpret_cast<const uint4*>(scale + mi));
            const uint4 zraw = __ldg(reinterpret_cast<const uint4*>(zero + mi));
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              ksc[e] = __half2float(reinterpret_cast<const __half*>(&sraw)[e]);
              kzr[e] = __half2float(reinterpret_cast<const __half*>(&zraw)[e]);
            }
          }
        }
        const float vsc = is_v ? __half2float(vsh[u]) : 0.f, vzr = is_v ? __half2float(vzh[u]) : 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          uint32_t c;
          if (BITS == 8) c = (raw[u][BITS == 8 ? (e >> 2) : 0] >> (8 * (e & 3))) & 0xFFu;
          else if (BITS == 4) c = (raw[u][0] >> (4 * e)) & 0xFu;
          else c = (raw[u][0] >> (2 * e)) & 0x3u;
          const float cf = __fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.f);
          x[e] = is_v ? __fmaf_rn(cf, vsc, vzr) : __fmaf_rn(cf, ksc[e], kzr[e]);
        }
        store8<T>(out + (size_t)t * a.d + elem, x);
      }
    }
  }
}

// Marks the base rows a layer's sparse loops read: for every head the columns of its blocks' lists (attention) and
// the active positions (the residual chain of the quantizer starts from their base rows). Bits are only ever set.
__global__ void __launch_bounds__(256) mark_base_rows_kernel(const int32_t* __restrict__ col_idx,
                                                             const int32_t* __restrict__ col_cnt, int c, int nb, int H,
                                                             const int32_t* __restrict__ active_idx, int n_active,
                                                             uint32_t* __restrict__ mask, int mask_words) {
  fl_grid_wait();
  fl_grid_release();
  const int64_t n_col = (int64_t)H * nb * c, total = n_col + (int64_t)H * n_active;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int h, t;
    if (i < n_col) {
      const int64_t list = i / c;
      if ((int)(i - list * c) >= __ldg(col_cnt + list)) continue;
      h = (int)(list / nb);
      t = __ldg(col_idx + i);
    } else {
      const int64_t k = i - n_col;
      h = (int)(k / n_active);
      t = __ldg(active_idx + (k - (int64_t)h * n_active));
    }
    atomicOr(mask + (size_t)h * mask_words + (t >> 5), 1u << (t & 31));
  }
}

int check_base(const fl_ctx* ctx, const fl_shape* s, const fl_kv_base_q* q) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(s);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(q != nullptr && q->tail >= 0);
  FL_REQUIRE(q->group == 32 || q->group == 64 || q->group == 128);
  const int d = s->n_heads * s->head_dim;
  if (s->bits == 16 || d % 256 != 0 || d % q->group != 0) return FL_ERR_UNSUPPORTED;
  const int Lq = s->L > q->tail ? s->L - q->tail : 0;
  if (Lq > 0) {
    FL_REQUIRE(q->k_codes != nullptr && q->k_scale != nullptr && q->k_zero != nullptr && q->v_codes != nullptr &&
               q->v_scale != nullptr && q->v_zero != nullptr);
    FL_REQUIRE(fl_aligned16(q->k_codes) && fl_aligned16(q->k_scale) && fl_aligned16(q->k_zero) &&
               fl_aligned16(q->v_codes) && fl_aligned16(q->v_scale) && fl_aligned16(q->v_zero));
  }
  if (Lq < s->L) FL_REQUIRE(q->k_tail != nullptr && q->v_tail != nullptr && fl_aligned16(q->k_tail) && fl_aligned16(q->v_tail));
  return FL_OK;
}

BaseArgs base_args(const fl_shape* s, const fl_kv_base_q* q) {
  BaseArgs a{};
  a.k_codes = static_cast<uint8_t*>(q->k_codes); a.k_scale = reinterpret_cast<__half*>(q->k_scale);
  a.k_zero = reinterpret_cast<__half*>(q->k_zero);
  a.v_codes = static_cast<uint8_t*>(q->v_codes); a.v_scale = reinterpret_cast<__half*>(q->v_scale);
  a.v_zero = reinterpret_cast<__half*>(q->v_zero);
  a.Lq = s->L > q->tail ? s->L - q->tail : 0;
  a.d = s->n_heads * s->head_dim;
  a.group = q->group;
  a.dh = s->head_dim;
  a.L = s->L;
  a.k_tail = q->k_tail;
  a.v_tail = q->v_tail;
  a.mask_words = (s->L + 31) / 32;
  a.row_mask = nullptr;
  return a;
}

template <typename T>
int launch_quant_base(fl_ctx* ctx, const fl_shape* s, const BaseArgs& a, cudaStream_t st) {
  const int n_tg = (a.Lq + a.group - 1) / a.group;
  const dim3 kgrid(n_tg, (a.d / 8 + 255) / 256);
  const int kthreads = a.d / 8 < 256 ? a.d / 8 : 256;
  int64_t vb = ((int64_t)a.Lq * (a.d / 8) + 255) / 256;
  const int vgrid = (int)(vb > (int64_t)ctx->sm_count * 16 ? (int64_t)ctx->sm_count * 16 : vb);
#define FL_BASEQ(BITS)                                                          \
  do {                                                                          \
    base_quant_k_kernel<T, BITS><<<kgrid, kthreads, 0, st>>>(a);                \
    base_quant_v_kernel<T, BITS><<<vgrid, 256, 0, st>>>(a);                     \
  } while (0)
  if (s->bits == 8) FL_BASEQ(8); else if (s->bits == 4) FL_BASEQ(4); else FL_BASEQ(2);
#undef FL_BASEQ
  return fl_launch_status();
}

template <typename T>
int launch_dequant_base(fl_ctx* ctx, const fl_shape* s, const BaseArgs& a, cudaStream_t st) {
  int64_t b = a.L;     // one CTA per row, up to 16 CTAs per SM and side; each then walks several rows
  const dim3 grid((unsigned)(b > (int64_t)ctx->sm_count * 16 ? (int64_t)ctx->sm_count * 16 : b), 2);
  if (s->bits == 8) FL_CHECK_CUDA(fl_launch(ctx, base_dequant_kernel<T, 8>, grid, dim3(256), 0, st, a));
  else if (s->bits == 4) FL_CHECK_CUDA(fl_launch(ctx, base_dequant_kernel<T, 4>, grid, dim3(256), 0, st, a));
  else FL_CHECK_CUDA(fl_launch(ctx, base_dequant_kernel<T, 2>, grid, dim3(256), 0, st, a));
  return fl_launch_status();
}

}  // namespace

extern "C" int fl_quant_kv_base(fl_ctx* ctx, const fl_shape* shape, const void* k, const void* v,
                                const fl_kv_base_q* base, int32_t* status, void* stream) {
  (void)status;
  int rc = check_base(ctx, shape, base);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(k != nullptr && v != nullptr && fl_aligned16(k) && fl_aligned16(v));
  BaseArgs a = base_args(shape, base);
  a.k = k; a.v = v;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t row_bytes = (size_t)a.d * fl_elem_bytes(shape);
  if (a.Lq < shape->L) {
    const size_t n = (size_t)(shape->L - a.Lq) * row_bytes;
    FL_CHECK_CUDA(cudaMemcpyAsync(base->k_tail, static_cast<const char*>(k) + (size_t)a.Lq * row_bytes, n,
                                  cudaMemcpyDeviceToDevice, st));
    FL_CHECK_CUDA(cudaMemcpyAsync(base->v_tail, static_cast<const char*>(v) + (size_t)a.Lq * row_bytes, n,
                                  cudaMemcpyDeviceToDevice, st));
  }
  if (a.Lq == 0) return FL_OK;
  return shape->dtype == FL_F32 ? launch_quant_base<float>(ctx, shape, a, st)
                                : launch_quant_base<__nv_bfloat16>(ctx, shape, a, st);
}

extern "C" int fl_dequant_kv_base(fl_ctx* ctx, const fl_shape* shape, const fl_kv_base_q* base,
                                  const uint32_t* row_mask, void* k_out, void* v_out, int32_t* status, void* stream) {
  (void)status;
  int rc = check_base(ctx, shape, base);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(k_out != nullptr && v_out != nullptr && fl_aligned16(k_out) && fl_aligned16(v_out));
  BaseArgs a = base_args(shape, base);
  a.k_out = k_out; a.v_out = v_out;
  a.row_mask = row_mask;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return shape->dtype == FL_F32 ? launch_dequant_base<float>(ctx, shape, a, st)
                                : launch_dequant_base<__nv_bfloat16>(ctx, shape, a, st);
}

extern "C" int fl_kv_base_q_bytes(const fl_shape* shape, int32_t group, int32_t tail, int64_t* bytes) {
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  if (bytes == nullptr || tail < 0 || (group != 32 && group != 64 && group != 128)) return FL_ERR_INVALID_ARG;
  const int64_t d = (int64_t)shape->n_heads * shape->head_dim;
  if (shape->bits == 16 || d % group != 0) return FL_ERR_UNSUPPORTED;
  const int64_t Lq = shape->L > tail ? shape->L - tail : 0;
  const int64_t n_tg = (Lq + group - 1) / group;
  *bytes = 2 * Lq * (d * shape->bits / 8) + 2 * 2 * n_tg * d + 2 * 2 * Lq * (d / group) +
           2 * (shape->L - Lq) * d * fl_elem_bytes(shape);
  return FL_OK;
}

extern "C" int fl_mark_base_rows(fl_ctx* ctx, const fl_shape* shape, const int32_t* col_idx, const int32_t* col_cnt,
                                 int32_t c, const int32_t* active_idx, int32_t n_active, uint32_t* row_mask,
                                 int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(row_mask != nullptr && c >= 1 && n_active >= 0 && n_active <= shape->L);
  FL_REQUIRE(col_idx != nullptr && col_cnt != nullptr && (n_active == 0 || active_idx != nullptr));
  const int nb = fl_n_blocks(shape), H = shape->n_heads;
  {
    const fl_idx_check ck[2] = {{active_idx, n_active, 0, nullptr, 0, shape->L - 1, 1},
                                {col_idx, (int64_t)H * nb * c, c, col_cnt, 0, shape->L - 1, 1}};
    rc = fl_debug_check(ctx, ck, 2, status, stream);
    if (rc != FL_OK) return rc;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int mask_words = (shape->L + 31) / 32;
  FL_CHECK_CUDA(cudaMemsetAsync(row_mask, 0, sizeof(uint32_t) * (size_t)H * mask_words, st));
  const int64_t total = (int64_t)H * nb * c + (int64_t)H * n_active;
  int64_t blocks = (total + 255) / 256;
  if (blocks > (int64_t)ctx->sm_count * 8) blocks = (int64_t)ctx->sm_count * 8;
  FL_CHECK_CUDA(fl_launch(ctx, mark_base_rows_kernel, dim3((unsigned)blocks), dim3(256), 0, st, col_idx, col_cnt, c, nb, H,
                          active_idx, n_active, row_mask, mask_words));
  return fl_launch_status();
}
