// Stage 3: residual quantization of the active rows' K and V (Eq. 8 with the asymmetric group-wise
// min/max quantizer of Appendix E). Each thread owns 8 consecutive elements (one 16-byte load in bf16), group
// min/max by sub-warp shuffles, codes packed and stored coalesced. Two kernels share the codec (encode8): a software
// pipeline over strided rows for the common shapes (bf16 rows of up to 2048 elements, at most three earlier
// streams), which keeps the next rows' operands in flight, and a plain one-CTA-per-row kernel for everything else.
// Both also leave, when the caller lends the buffers, the reconstructed rows before and after the loop's residual
// as bf16 for the attention call of the same loop.
#include "fl_internal.cuh"

namespace {

struct QuantArgs {
  DevSide k, v;                 // base + earlier streams (read), in loop order
  const void* k_new;            // [n, H, dh]
  const void* v_new;
  const int32_t* active_idx;    // [n]
  uint8_t* k_codes; __half* k_scale; __half* k_zero;   // stream being written
  uint8_t* v_codes; __half* v_scale; __half* v_zero;
  void* k_rows_prev; void* k_rows_cur;   // optional [n, H, dh] storage type: Xhat^(r-1) / Xhat^(r) of the active rows
  void* v_rows_prev; void* v_rows_cur;
  int n_prev;                   // residual streams already in the chain (loop_r - 2)
  int d, group;
};

// Everything after the operands of 8 consecutive elements of active row t are in registers: xn = the new row,
// xh = Xhat^(r-1) (base plus the earlier streams). Writes the codes, the group's scale and offset, and the
// materialized rows when the caller wants them.
template <typename T, int BITS>
__device__ __forceinline__ void encode8(const QuantArgs& a, bool is_v, int t, int elem, int lanes_per_group,
                                        float (&xn)[8], float (&xh)[8]) {
  uint8_t* codes = is_v ? a.v_codes : a.k_codes;
  __half* scale = is_v ? a.v_scale : a.k_scale;
  __half* zero = is_v ? a.v_zero : a.k_zero;
  T* rows_prev = static_cast<T*>(is_v ? a.v_rows_prev : a.k_rows_prev);   // null: not wanted
  T* rows_cur = static_cast<T*>(is_v ? a.v_rows_cur : a.k_rows_cur);
  if (rows_prev != nullptr) store8<T>(rows_prev + (size_t)t * a.d + elem, xh);
  if constexpr (BITS == 16) {  // codec off: the stream keeps the row itself
    store8<T>(reinterpret_cast<T*>(codes) + (size_t)t * a.d + elem, xn);
    if (rows_cur != nullptr) store8<T>(rows_cur + (size_t)t * a.d + elem, xn);
  } else {
    float dl[8];
    float mn, mx;
  #pragma unroll
    for (int i = 0; i < 8; ++i) dl[i] = __fsub_rn(xn[i], xh[i]);
    mn = mx = dl[0];
  #pragma unroll
    for (int i = 1; i < 8; ++i) { mn = fminf(mn, dl[i]); mx = fmaxf(mx, dl[i]); }
    // every lane of the warp is here: the host only launches row widths for which all threads of the
    // block run the same number of iterations (d % 256 == 0, and d % 2048 == 0 beyond 2048)
    for (int o = 1; o < lanes_per_group; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const __half zh = __float2half_rd(mn);
    const float zf = __half2float(zh);
    const float range = __fsub_rn(mx, zf);
    const float qmax = (float)((1 << BITS) - 1);
    const __half sh = range == 0.f ? __float2half_rn(0.f) : __float2half_ru(__fdiv_rn(range, qmax));
    const float sf = __half2float(sh);
    // Codes: round-half-even of the binary32 quotient (delta - zero) / scale. The quotient is first formed with
    // one reciprocal per group; that estimate is within a few ulp of the correctly rounded quotient (<= 5e-5
    // absolute for codes up to 255), so its rounding to an integer is the same unless it lies within 1e-4 of a
    // half-integer. Only then (a few percent of the warps) the true divisions are redone.
    float q[8];
    bool ambiguous = false;
    if (sf != 0.f) {
      const float inv = __frcp_rn(sf);
  #pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float est = __fmul_rn(__fsub_rn(dl[i], zf), inv);
        q[i] = __fsub_rn(__fadd_rn(est, 12582912.f), 12582912.f);   // round-half-even for |est| < 2^22
        ambiguous |= 0.5f - fabsf(est - q[i]) < 1e-4f;
      }
      if (__any_sync(__activemask(), ambiguous)) {
  #pragma unroll
        for (int i = 0; i < 8; ++i) q[i] = rintf(__fdiv_rn(__fsub_rn(dl[i], zf), sf));
      }
    } else {
  #pragma unroll
      for (int i = 0; i < 8; ++i) q[i] = 0.f;
    }
    if (rows_cur != nullptr) {
      // the reconstruction every later reader of this stream forms: Xhat + (code * scale + zero), Eq. 8
  #pragma unroll
      for (int i = 0; i < 8; ++i) xh[i] = __fadd_rn(xh[i], __fmaf_rn(q[i], sf, zf));
      store8<T>(rows_cur + (size_t)t * a.d + elem, xh);
    }
    // The quotients are integers in [0, qmax] already: delta >= zero (the offset was rounded down) and
    // (max - zero) / scale <= qmax (the scale was rounded up), so the oracle's clamp never acts. Four codes at a
    // time are packed with exact binary32 arithmetic (sum of code * 2^(BITS*i) < 2^24 for BITS <= 4, two codes
    // for 8 bits), and the integer is read from the low mantissa bits of (value + 2^23).
    uint32_t packed_lo, packed_hi = 0;
    if constexpr (BITS == 8) {
      uint32_t w[4];
  #pragma unroll
      for (int i = 0; i < 4; ++i)
        w[i] = __float_as_uint(__fadd_rn(__fmaf_rn(q[2 * i + 1], 256.f, q[2 * i]), 8388608.f)) & 0xFFFFu;
      packed_lo = w[0] | (w[1] << 16);
      packed_hi = w[2] | (w[3] << 16);
    } else {
      const float r1 = (float)(1 << BITS), r2 = r1 * r1, r3 = r2 * r1;
      const float lo = __fmaf_rn(q[3], r3, __fmaf_rn(q[2], r2, __fmaf_rn(q[1], r1, q[0])));
      const float hi = __fmaf_rn(q[7], r3, __fmaf_rn(q[6], r2, __fmaf_rn(q[5], r1, q[4])));
      const uint32_t half_mask = (1u << (4 * BITS)) - 1u;
      packed_lo = (__float_as_uint(__fadd_rn(lo, 8388608.f)) & half_mask) |
                  ((__float_as_uint(__fadd_rn(hi, 8388608.f)) & half_mask) << (4 * BITS));
    }
    uint8_t* row = codes + (size_t)t * (a.d * BITS / 8);
    if (BITS == 8) *reinterpret_cast<uint2*>(row + elem) = make_uint2(packed_lo, packed_hi);
    else if (BITS == 4) *reinterpret_cast<uint32_t*>(row + elem / 2) = packed_lo;
    else *reinterpret_cast<uint16_t*>(row + elem / 4) = (uint16_t)packed_lo;
    if (((elem >> 3) & (lanes_per_group - 1)) == 0) {
      const int gs = 31 - __clz(a.group);   // power of two
      const size_t gi = (size_t)t * (a.d >> gs) + (elem >> gs);
      scale[gi] = sh;
      zero[gi] = zh;
    }
  }
}

template <typename T, int BITS>
__global__ void __launch_bounds__(256) quant_residual_kernel(const __grid_constant__ QuantArgs a) {
  fl_grid_wait();
  fl_grid_release();
  const int t = blockIdx.x;                 // active row
  const bool is_v = blockIdx.y != 0;
  const DevSide& side = is_v ? a.v : a.k;
  const T* x_new = static_cast<const T*>(is_v ? a.v_new : a.k_new) + (size_t)t * a.d;
  const int pos = __ldg(a.active_idx + t);
  const int lanes_per_group = a.group >> 3;  // 1, 2, 4, 8 or 16

  for (int elem = threadIdx.x * 8; elem < a.d; elem += blockDim.x * 8) {
    // The new row, the base row and every earlier stream's slot lookup are independent loads; the payloads of
    // four streams at a time follow as a second round (Eq. 8 chain applied in loop order afterwards).
    float xn[8], xh[8];
    load8<T>(x_new + elem, xn);
    load8<T>(static_cast<const T*>(side.base) + (size_t)pos * a.d + elem, xh);
    for (int sg = 0; sg < a.n_prev; sg += 4) {
      int sl[4];
      Payload8<T, BITS> pl[4];
#pragma unroll
      for (int si = 0; si < 4; ++si) sl[si] = sg + si < a.n_prev ? __ldg(side.s[sg + si].slot + pos) : -1;
#pragma unroll
      for (int si = 0; si < 4; ++si)
        if (sl[si] >= 0) payload_load<T, BITS>(side.s[sg + si], sl[si], elem, a.d, a.group, pl[si]);
#pragma unroll
      for (int si = 0; si < 4; ++si)
        if (sl[si] >= 0) payload_apply<T, BITS>(pl[si], xh);
    }
    encode8<T, BITS>(a, is_v, t, elem, lanes_per_group, xn, xh);
  }
}

// The same for bf16 rows of at most 2048 elements and NP <= 3 earlier streams, as a software pipeline: a CTA walks a
// strided set of rows, and while it encodes one row the operands of its next row (new row, base row, the earlier
// streams' payloads), the stream rows of the one after and the position of the third are in flight. One row per
// short-lived CTA leaves every CTA two or three dependent round trips to memory with nothing to do in between.
template <int BITS, int NP>
__global__ void __launch_bounds__(256, 4) quant_residual_pipelined_kernel(const __grid_constant__ QuantArgs a, int n) {
  using T = __nv_bfloat16;
  fl_grid_wait();
  fl_grid_release();
  const bool is_v = blockIdx.y != 0;
  const DevSide& side = is_v ? a.v : a.k;
  const int elem = threadIdx.x * 8, G = gridDim.x;
  const int lanes_per_group = a.group >> 3;
  const T* x_new = static_cast<const T*>(is_v ? a.v_new : a.k_new) + elem;
  const T* base = static_cast<const T*>(side.base) + elem;
  int t = blockIdx.x;
  if (t >= n) return;
  // fill the pipeline: positions of three rows, stream rows of two, operands of one
  int pos = __ldg(a.active_idx + t);
  int pos1 = t + G < n ? __ldg(a.active_idx + t + G) : 0;
  int pos2 = t + 2 * G < n ? __ldg(a.active_idx + t + 2 * G) : 0;
  uint4 rx = __ldg(reinterpret_cast<const uint4*>(x_new + (size_t)t * a.d));
  uint4 rh = __ldg(reinterpret_cast<const uint4*>(base + (size_t)pos * a.d));
  int sl[NP > 0 ? NP : 1], sl1[NP > 0 ? NP : 1];
  Payload8<T, BITS> pl[NP > 0 ? NP : 1];
#pragma unroll
  for (int s = 0; s < NP; ++s) {
    sl[s] = __ldg(side.s[s].slot + pos);
    sl1[s] = t + G < n ? __ldg(side.s[s].slot + pos1) : -1;
  }
#pragma unroll
  for (int s = 0; s < NP; ++s)
    if (sl[s] >= 0) payload_load<T, BITS>(side.s[s], sl[s], elem, a.d, a.group, pl[s]);
  for (;;) {
    const int t1 = t + G;
    const bool has1 = t1 < n;
    uint4 rx1 = rx, rh1 = rh;
    Payload8<T, BITS> pl1[NP > 0 ? NP : 1];
    int sl2[NP > 0 ? NP : 1];
    int pos3 = 0;
    if (has1) {
      rx1 = __ldg(reinterpret_cast<const uint4*>(x_new + (size_t)t1 * a.d));
      rh1 = __ldg(reinterpret_cast<const uint4*>(base + (size_t)pos1 * a.d));
#pragma unroll
      for (int s = 0; s < NP; ++s) {
        if (sl1[s] >= 0) payload_load<T, BITS>(side.s[s], sl1[s], elem, a.d, a.group, pl1[s]);
        sl2[s] = t + 2 * G < n ? __ldg(side.s[s].slot + pos2) : -1;
      }
      if (t + 3 * G < n) pos3 = __ldg(a.active_idx + t + 3 * G);
    }
    // row t: Xhat^(r-1) = base plus the earlier streams in loop order, then the codec
    float xn[8], xh[8];
    {
      const __nv_bfloat162* hx = reinterpret_cast<const __nv_bfloat162*>(&rx);
      const __nv_bfloat162* hh = reinterpret_cast<const __nv_bfloat162*>(&rh);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 fx = __bfloat1622float2(hx[i]), fh = __bfloat1622float2(hh[i]);
        xn[2 * i] = fx.x; xn[2 * i + 1] = fx.y;
        xh[2 * i] = fh.x; xh[2 * i + 1] = fh.y;
      }
    }
#pragma unroll
    for (int s = 0; s < NP; ++s)
      if (sl[s] >= 0) payload_apply<T, BITS>(pl[s], xh);
    // the common group of 128 elements gets its own copy of the codec, with the sub-warp reduction unrolled
    if (lanes_per_group == 16) encode8<T, BITS>(a, is_v, t, elem, 16, xn, xh);
    else encode8<T, BITS>(a, is_v, t, elem, lanes_per_group, xn, xh);
    if (!has1) break;
    t = t1;
    rx = rx1; rh = rh1;
    pos1 = pos2; pos2 = pos3;
#pragma unroll
    for (int s = 0; s < NP; ++s) { sl[s] = sl1[s]; sl1[s] = sl2[s]; pl[s] = pl1[s]; }
  }
}

// ------------------------------------------------------------------------------------------------------------
// The same pipeline with SIXTEEN consecutive elements per thread (two 16-byte loads per operand): the per-thread
// work that does not depend on the element count (addresses, slot lookups, metadata, the sub-warp reduction, the
// pipeline's bookkeeping) is paid once per 16 elements, and a group of 128 spans 8 lanes (three shuffle rounds).
// bf16 rows whose width is a multiple of 512 (whole warps per row), groups of at least 16, at most three earlier
// streams. Arithmetic identical to encode8, element by element.
// ------------------------------------------------------------------------------------------------------------
template <int BITS>
struct Pay16 {
  uint4 raw;      // BITS 8: 16 bytes; 4: x, y; 2: x
  __half sc, zr;
};
template <int BITS>
__device__ __forceinline__ void pay16_load(const DevStream& st, int slot, int elem, int d, int group, Pay16<BITS>& p) {
  const uint8_t* row = st.codes + (size_t)slot * (d * BITS / 8);
  if (BITS == 8) {
    p.raw = __ldg(reinterpret_cast<const uint4*>(row + elem));
  } else if (BITS == 4) {
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(row + elem / 2));
    p.raw.x = t.x; p.raw.y = t.y;
  } else {
    p.raw.x = __ldg(reinterpret_cast<const uint32_t*>(row + elem / 4));
  }
  const int gs = 31 - __clz(group);
  const size_t gi = (size_t)slot * (d >> gs) + (elem >> gs);
  p.sc = __ldg(st.scale + gi);
  p.zr = __ldg(st.zero + gi);
}
template <int BITS>
__device__ __forceinline__ void pay16_apply(const Pay16<BITS>& p, float (&x)[16]) {
  const float sc = __half2float(p.sc), zr = __half2float(p.zr);
  const uint32_t w[4] = {p.raw.x, p.raw.y, p.raw.z, p.raw.w};
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    uint32_t c;
    if (BITS == 8) c = (w[i >> 2] >> (8 * (i & 3))) & 0xFFu;
    else if (BITS == 4) c = (w[i >> 3] >> (4 * (i & 7))) & 0xFu;
    else c = (w[0] >> (2 * i)) & 0x3u;
    const float cf = __fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.f);   // exact: 2^23 + c
    x[i] = __fadd_rn(x[i], __fmaf_rn(cf, sc, zr));
  }
}
__device__ __forceinline__ void unpack16(const uint4& lo, const uint4& hi, float (&x)[16]) {
  const __nv_bfloat162* a = reinterpret_cast<const __nv_bfloat162*>(&lo);
  const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&hi);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 fa = __bfloat1622float2(a[i]), fb = __bfloat1622float2(b[i]);
    x[2 * i] = fa.x; x[2 * i + 1] = fa.y;
    x[8 + 2 * i] = fb.x; x[8 + 2 * i + 1] = fb.y;
  }
}
__device__ __forceinline__ void store16(__nv_bfloat16* p, const float (&x)[16]) {
  uint4 lo, hi;
  __nv_bfloat162* a = reinterpret_cast<__nv_bfloat162*>(&lo);
  __nv_bfloat162* b = reinterpret_cast<__nv_bfloat162*>(&hi);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    b[i] = __floats2bfloat162_rn(x[8 + 2 * i], x[8 + 2 * i + 1]);
  }
  reinterpret_cast<uint4*>(p)[0] = lo;
  reinterpret_cast<uint4*>(p)[1] = hi;
}

template <int BITS>
__device__ __forceinline__ void encode16(const QuantArgs& a, bool is_v, int t, int elem, int lanes_per_group,
                                         float (&xn)[16], float (&xh)[16]) {
  using T = __nv_bfloat16;
  uint8_t* codes = is_v ? a.v_codes : a.k_codes;
  __half* scale = is_v ? a.v_scale : a.k_scale;
  __half* zero = is_v ? a.v_zero : a.k_zero;
  T* rows_prev = static_cast<T*>(is_v ? a.v_rows_prev : a.k_rows_prev);
  T* rows_cur = static_cast<T*>(is_v ? a.v_rows_cur : a.k_rows_cur);
  const size_t row_off = (size_t)t * a.d + elem;
  if (rows_prev != nullptr) store16(rows_prev + row_off, xh);
  float dl[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) dl[i] = __fsub_rn(xn[i], xh[i]);
  float mn = dl[0], mx = dl[0];
#pragma unroll
  for (int i = 1; i < 16; ++i) { mn = fminf(mn, dl[i]); mx = fmaxf(mx, dl[i]); }
  for (int o = 1; o < lanes_per_group; o <<= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  const __half zh = __float2half_rd(mn);
  const float zf = __half2float(zh);
  const float range = __fsub_rn(mx, zf);
  const float qmax = (float)((1 << BITS) - 1);
  const __half sh = range == 0.f ? __float2half_rn(0.f) : __float2half_ru(__fdiv_rn(range, qmax));
  const float sf = __half2float(sh);
  float q[16];
  if (sf != 0.f) {
    // reciprocal estimate of the quotient, exact divisions only where its rounding could differ (see encode8)
    const float inv = __frcp_rn(sf);
    bool ambiguous = false;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float est = __fmul_rn(__fsub_rn(dl[i], zf), inv);
      q[i] = __fsub_rn(__fadd_rn(est, 12582912.f), 12582912.f);
      ambiguous |= 0.5f - fabsf(est - q[i]) < 1e-4f;
    }
    if (__any_sync(__activemask(), ambiguous)) {
#pragma unroll
      for (int i = 0; i < 16; ++i) q[i] = rintf(__fdiv_rn(__fsub_rn(dl[i], zf), sf));
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) q[i] = 0.f;
  }
  if (rows_cur != nullptr) {
#pragma unroll
    for (int i = 0; i < 16; ++i) xh[i] = __fadd_rn(xh[i], __fmaf_rn(q[i], sf, zf));
    store16(rows_cur + row_off, xh);
  }
  // packing by exact binary32 arithmetic (sums below 2^24), the integer read from the low mantissa bits of value + 2^23
  uint8_t* row = codes + (size_t)t * (a.d * BITS / 8);
  if constexpr (BITS == 8) {
    uint32_t w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      w[i] = __float_as_uint(__fadd_rn(__fmaf_rn(q[2 * i + 1], 256.f, q[2 * i]), 8388608.f)) & 0xFFFFu;
    *reinterpret_cast<uint4*>(row + elem) = make_uint4(w[0] | (w[1] << 16), w[2] | (w[3] << 16), w[4] | (w[5] << 16),
                                                       w[6] | (w[7] << 16));
  } else {
    const float r1 = (float)(1 << BITS), r2 = r1 * r1, r3 = r2 * r1;
    const uint32_t quad_mask = (1u << (4 * BITS)) - 1u;
    uint32_t quad[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float v = __fmaf_rn(q[4 * j + 3], r3, __fmaf_rn(q[4 * j + 2], r2, __fmaf_rn(q[4 * j + 1], r1, q[4 * j])));
      quad[j] = __float_as_uint(__fadd_rn(v, 8388608.f)) & quad_mask;
    }
    if (BITS == 4)
      *reinterpret_cast<uint2*>(row + elem / 2) = make_uint2(quad[0] | (quad[1] << 16), quad[2] | (quad[3] << 16));
    else
      *reinterpret_cast<uint32_t*>(row + elem / 4) = quad[0] | (quad[1] << 8) | (quad[2] << 16) | (quad[3] << 24);
  }
  if (((elem >> 4) & (lanes_per_group - 1)) == 0) {
    const int gs = 31 - __clz(a.group);
    const size_t gi = (size_t)t * (a.d >> gs) + (elem >> gs);
    scale[gi] = sh;
    zero[gi] = zh;
  }
}

template <int BITS, int NP>
__global__ void __launch_bounds__(256) quant_residual_wide_kernel(const __grid_constant__ QuantArgs a, int n) {
  using T = __nv_bfloat16;
  fl_grid_wait();
  fl_grid_release();
  const bool is_v = blockIdx.y != 0;
  const DevSide& side = is_v ? a.v : a.k;
  const int elem = threadIdx.x * 16, G = gridDim.x;
  const int lanes_per_group = a.group >> 4;
  const T* x_new = static_cast<const T*>(is_v ? a.v_new : a.k_new) + elem;
  const T* base = static_cast<const T*>(side.base) + elem;
  int t = blockIdx.x;
  if (t >= n) return;
  constexpr int NPA = NP > 0 ? NP : 1;
  int pos = __ldg(a.active_idx + t);
  int pos1 = t + G < n ? __ldg(a.active_idx + t + G) : 0;
  int pos2 = t + 2 * G < n ? __ldg(a.active_idx + t + 2 * G) : 0;
  const uint4* px = reinterpret_cast<const uint4*>(x_new + (size_t)t * a.d);
  const uint4* ph = reinterpret_cast<const uint4*>(base + (size_t)pos * a.d);
  uint4 rx0 = __ldg(px), rx1 = __ldg(px + 1), rh0 = __ldg(ph), rh1 = __ldg(ph + 1);
  int sl[NPA], sl_n[NPA];
  Pay16<BITS> pl[NPA];
#pragma unroll
  for (int s = 0; s < NP; ++s) {
    sl[s] = __ldg(side.s[s].slot + pos);
    sl_n[s] = t + G < n ? __ldg(side.s[s].slot + pos1) : -1;
  }
#pragma unroll
  for (int s = 0; s < NP; ++s)
    if (sl[s] >= 0) pay16_load<BITS>(side.s[s], sl[s], elem, a.d, a.group, pl[s]);
  for (;;) {
    const int t1 = t + G;
    const bool has1 = t1 < n;
    uint4 nx0 = rx0, nx1 = rx1, nh0 = rh0, nh1 = rh1;
    Pay16<BITS> pl_n[NPA];
    int sl_nn[NPA];
    int pos3 = 0;
    if (has1) {
      const uint4* qx = reinterpret_cast<const uint4*>(x_new + (size_t)t1 * a.d);
      const uint4* qh = reinterpret_cast<const uint4*>(base + (size_t)pos1 * a.d);
      nx0 = __ldg(qx); nx1 = __ldg(qx + 1); nh0 = __ldg(qh); nh1 = __ldg(qh + 1);
#pragma unroll
      for (int s = 0; s < NP; ++s) {
        if (sl_n[s] >= 0) pay16_load<BITS>(side.s[s], sl_n[s], elem, a.d, a.group, pl_n[s]);
        sl_nn[s] = t + 2 * G < n ? __ldg(side.s[s].slot + pos2) : -1;
      }
      if (t + 3 * G < n) pos3 = __ldg(a.active_idx + t + 3 * G);
    }
    float xn[16], xh[16];
    unpack16(rx0, rx1, xn);
    unpack16(rh0, rh1, xh);
#pragma unroll
    for (int s = 0; s < NP; ++s)
      if (sl[s] >= 0) pay16_apply<BITS>(pl[s], xh);
    if (lanes_per_group == 8) encode16<BITS>(a, is_v, t, elem, 8, xn, xh);
    else encode16<BITS>(a, is_v, t, elem, lanes_per_group, xn, xh);
    if (!has1) break;
    t = t1;
    rx0 = nx0; rx1 = nx1; rh0 = nh0; rh1 = nh1;
    pos1 = pos2; pos2 = pos3;
#pragma unroll
    for (int s = 0; s < NP; ++s) { sl[s] = sl_n[s]; sl_n[s] = sl_nn[s]; pl[s] = pl_n[s]; }
  }
}

template <int BITS, int NP>
int launch_quant_wide_np(const fl_ctx* ctx, const QuantArgs& a, int n_active, cudaStream_t st) {
  auto kern = quant_residual_wide_kernel<BITS, NP>;
  const int threads = a.d / 16;
  int per_sm = 0;
  FL_CHECK_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, 0));
  if (per_sm < 1) per_sm = 1;
  const int resident = ctx->sm_count * per_sm / 2;
  const int gx = n_active < resident ? n_active : (resident < 1 ? 1 : resident);
  FL_CHECK_CUDA(fl_launch(ctx, kern, dim3(gx, 2), dim3(threads), 0, st, a, n_active));
  return fl_launch_status();
}

template <int BITS>
int launch_quant_wide(const fl_ctx* ctx, const QuantArgs& a, int n_active, cudaStream_t st) {
  switch (a.n_prev) {
    case 0: return launch_quant_wide_np<BITS, 0>(ctx, a, n_active, st);
    case 1: return launch_quant_wide_np<BITS, 1>(ctx, a, n_active, st);
    case 2: return launch_quant_wide_np<BITS, 2>(ctx, a, n_active, st);
    default: return launch_quant_wide_np<BITS, 3>(ctx, a, n_active, st);
  }
}

template <int BITS, int NP>
int launch_quant_pipelined_np(const fl_ctx* ctx, const QuantArgs& a, int n_active, cudaStream_t st) {
  auto kern = quant_residual_pipelined_kernel<BITS, NP>;
  const int threads = a.d / 8;
  int per_sm = 0;   // as many CTAs as are resident at once: every one of them keeps a row in flight
  FL_CHECK_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, 0));
  if (per_sm < 1) per_sm = 1;
  const int resident = ctx->sm_count * per_sm / 2;   // the grid has two CTAs (K, V) per row slot
  const int gx = n_active < resident ? n_active : (resident < 1 ? 1 : resident);
  FL_CHECK_CUDA(fl_launch(ctx, kern, dim3(gx, 2), dim3(threads), 0, st, a, n_active));
  return fl_launch_status();
}

template <int BITS>
int launch_quant_pipelined(const fl_ctx* ctx, const QuantArgs& a, int n_active, cudaStream_t st) {
  switch (a.n_prev) {
    case 0: return launch_quant_pipelined_np<BITS, 0>(ctx, a, n_active, st);
    case 1: return launch_quant_pipelined_np<BITS, 1>(ctx, a, n_active, st);
    case 2: return launch_quant_pipelined_np<BITS, 2>(ctx, a, n_active, st);
    default: return launch_quant_pipelined_np<BITS, 3>(ctx, a, n_active, st);
  }
}

template <typename T>
int launch_quant(const fl_ctx* ctx, const fl_shape* s, const QuantArgs& a, int n_active, cudaStream_t st) {
  if (sizeof(T) == 2 && a.d % 512 == 0 && a.d <= 4096 && a.n_prev <= 3 && s->bits != 16 && a.group >= 16 &&
      !ctx->quant_narrow) {
    switch (s->bits) {
      case 2: return launch_quant_wide<2>(ctx, a, n_active, st);
      case 4: return launch_quant_wide<4>(ctx, a, n_active, st);
      default: return launch_quant_wide<8>(ctx, a, n_active, st);
    }
  }
  if (sizeof(T) == 2 && a.d <= 2048 && a.n_prev <= 3 && s->bits != 16) {
    switch (s->bits) {
      case 2: return launch_quant_pipelined<2>(ctx, a, n_active, st);
      case 4: return launch_quant_pipelined<4>(ctx, a, n_active, st);
      default: return launch_quant_pipelined<8>(ctx, a, n_active, st);
    }
  }
  const int threads = a.d / 8 < 256 ? a.d / 8 : 256;
  dim3 grid(n_active, 2);
  switch (s->bits) {
    case 2: FL_CHECK_CUDA(fl_launch(ctx, quant_residual_kernel<T, 2>, grid, dim3(threads), 0, st, a)); break;
    case 4: FL_CHECK_CUDA(fl_launch(ctx, quant_residual_kernel<T, 4>, grid, dim3(threads), 0, st, a)); break;
    case 8: FL_CHECK_CUDA(fl_launch(ctx, quant_residual_kernel<T, 8>, grid, dim3(threads), 0, st, a)); break;
    default: FL_CHECK_CUDA(fl_launch(ctx, quant_residual_kernel<T, 16>, grid, dim3(threads), 0, st, a)); break;
  }
  return fl_launch_status();
}

}  // namespace

extern "C" int fl_quant_kv_residual(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* k_new,
                                    const void* v_new, const int32_t* active_idx, int32_t n_active,
                                    const fl_kv_store* store, int32_t* status, void* stream) {
  FL_REQUIRE(ctx != nullptr);
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(loop_r >= 2 && loop_r <= FL_MAX_LOOPS + 1);
  FL_REQUIRE(n_active >= 0 && n_active <= shape->L);
  rc = fl_check_store(shape, store, loop_r - 1);
  if (rc != FL_OK) return rc;
  const fl_kv_stream& ks = store->k_res[loop_r - 2];
  const fl_kv_stream& vs = store->v_res[loop_r - 2];
  FL_REQUIRE(ks.n_rows == n_active && vs.n_rows == n_active);
  if (n_active == 0) return FL_OK;
  FL_REQUIRE(k_new != nullptr && v_new != nullptr && active_idx != nullptr);
  FL_REQUIRE(fl_aligned16(k_new) && fl_aligned16(v_new));
  const int d = shape->n_heads * shape->head_dim;
  // whole warps must enter or leave the element loop together (sub-warp shuffles inside)
  if (d % 256 != 0 || (d > 2048 && d % 2048 != 0)) return FL_ERR_UNSUPPORTED;
  {
    fl_idx_check ck[1 + 2 * FL_MAX_LOOPS];
    int n = 0;
    ck[n++] = {active_idx, n_active, 0, nullptr, 0, shape->L - 1, 1};
    for (int i = 0; i < loop_r - 2; ++i) {   // the earlier streams' slot maps: the chain is rebuilt through them
      ck[n++] = {store->k_res[i].slot_of_pos, shape->L, 0, nullptr, -1, store->k_res[i].n_rows - 1, 0};
      ck[n++] = {store->v_res[i].slot_of_pos, shape->L, 0, nullptr, -1, store->v_res[i].n_rows - 1, 0};
    }
    rc = fl_debug_check(ctx, ck, n, status, stream);
    if (rc != FL_OK) return rc;
  }

  QuantArgs a;
  fl_dev_side(store, true, &a.k);
  fl_dev_side(store, false, &a.v);
  a.k_new = k_new; a.v_new = v_new; a.active_idx = active_idx;
  a.k_codes = static_cast<uint8_t*>(ks.codes); a.k_scale = reinterpret_cast<__half*>(ks.scale);
  a.k_zero = reinterpret_cast<__half*>(ks.zero);
  a.v_codes = static_cast<uint8_t*>(vs.codes); a.v_scale = reinterpret_cast<__half*>(vs.scale);
  a.v_zero = reinterpret_cast<__half*>(vs.zero);
  const bool rows = shape->dtype == FL_BF16;   // each buffer is written when it is there (rows_cur may come alone)
  a.k_rows_prev = rows ? ks.rows_prev : nullptr; a.k_rows_cur = rows ? ks.rows_cur : nullptr;
  a.v_rows_prev = rows ? vs.rows_prev : nullptr; a.v_rows_cur = rows ? vs.rows_cur : nullptr;
  a.n_prev = loop_r - 2; a.d = d; a.group = shape->group;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return shape->dtype == FL_F32 ? launch_quant<float>(ctx, shape, a, n_active, st)
                                : launch_quant<__nv_bfloat16>(ctx, shape, a, n_active, st);
}
