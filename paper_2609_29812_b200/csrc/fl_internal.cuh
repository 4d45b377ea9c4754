// Internal declarations shared by the kernels of libflashloop (never installed).
#pragma once
#include <cuda.h>   // CUtensorMap and the tensor-map enums only; the driver is reached through the runtime
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flashloop.h"

struct fl_ctx {
  int device;
  int sm_count;
  int max_smem_optin;
  int force_simt;  // environment FL_FORCE_SIMT=1 at fl_create: keep attention on the binary32 SIMT kernels
  int fused_attn;  // environment FL_FUSED_ATTN=1 at fl_create: calls with a carried old term keep the fused kernel
  int two_pass;    // environment FL_TWO_PASS=1 at fl_create: recomputing calls with carried buffers run as two launches
  int quant_narrow;  // environment FL_QUANT_NARROW=1 at fl_create: the quantizer keeps 8 elements per thread
  void* encode_tiled;       // cuTensorMapEncodeTiled, resolved through cudaGetDriverEntryPoint (may be null)
  struct fl_tmap_cache* tmaps;  // tensor maps, keyed by (base pointer, rows, row elements, box rows)
  int pdl;                  // launch the hot-path kernels with programmatic stream serialization (FL_NO_PDL=1: off)
  void* ws;                 // caller's workspace (fl_set_workspace), or null
  size_t ws_bytes;
  void* dbg_flag;           // checked build only: device word of the index validator (allocated on first use)
};

// Index validation of the checked build (debug_bounds.cu; an empty stub otherwise). One entry per array:
// values a[0..n) must lie in [lo, hi]; with seg > 0 the array is a sequence of segments of seg entries, of which
// only the first cnt[segment] count (cnt null: all of them; a count outside [0, seg] is itself a violation);
// ascending: strictly increasing inside a segment (the whole array when seg = 0).
struct fl_idx_check {
  const int32_t* a;
  int64_t n;
  int64_t seg;
  const int32_t* cnt;
  int32_t lo, hi;
  int ascending;
};
// Returns FL_OK, or FL_ERR_INVALID_ARG (also written to *status, if given) when an index is out of range; the caller
// must then launch nothing. Synchronises the stream in the checked build.
int fl_debug_check(fl_ctx* ctx, const fl_idx_check* checks, int n_checks, int32_t* status, void* stream);
int fl_debug_init(fl_ctx* ctx);   // allocates the validator's device word (checked build); FL_OK or FL_ERR_CUDA
// n values of the storage type `dtype` must be finite; same contract as fl_debug_check.
int fl_debug_check_finite(fl_ctx* ctx, const void* x, int64_t n, int dtype, int32_t* status, void* stream);
// The index inputs of an attention call: the active list, the column lists with their counts (n_segments lists of c
// entries) and the slot maps of the first n_streams residual streams.
int fl_debug_check_attn(fl_ctx* ctx, const fl_shape* s, int n_streams, const int32_t* active_idx, int32_t n_active,
                        const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt, int32_t c,
                        int64_t n_segments, int32_t* status, void* stream);

// Layout of the loop-attention workspace: kFlMaxSplit int32 arrival counters, then per split problem two partial
// results of kFlPartFloats binary32 values (both 128 x 128 accumulators and four statistics per row).
constexpr int kFlPartFloats = 2 * 128 * 128 + 4 * 128;
constexpr int kFlMaxSplit = 256;

// Bytes of workspace with which the loop-attention launch can split the problems of its last wave (0: never useful).
size_t fl_attn_workspace_bytes(const fl_ctx* ctx, const fl_shape* s);

// Tensor map of a row-major bf16 matrix [rows, row_elems] for TMA: box = 64 elements x box_rows rows,
// 128-byte swizzle, out-of-range rows read as zero. box_rows = 1 is the map for row gathers (tile::gather4),
// box_rows = 128 loads one slab of a compact Q tile. Cached per context.
// Returns false if tensor maps are not available (caller falls back to a non-TMA kernel).
bool fl_tile_tmap(fl_ctx* ctx, const void* base, int64_t rows, int64_t row_elems, int box_rows, CUtensorMap* out);

#define FL_CHECK_CUDA(expr)                    \
  do {                                         \
    cudaError_t e__ = (expr);                  \
    if (e__ != cudaSuccess) return FL_ERR_CUDA; \
  } while (0)

#define FL_REQUIRE(cond)                     \
  do {                                       \
    if (!(cond)) return FL_ERR_INVALID_ARG;  \
  } while (0)

static inline bool fl_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Host-side checks every entry point shares. Returns FL_OK, FL_ERR_INVALID_ARG or FL_ERR_UNSUPPORTED.
int fl_check_shape(const fl_shape* s);
int fl_check_store(const fl_shape* s, const fl_kv_store* st, int n_streams_needed);
int fl_launch_status();  // maps cudaGetLastError() to a status

static inline int fl_elem_bytes(const fl_shape* s) { return s->dtype == FL_F32 ? 4 : 2; }
static inline int fl_n_blocks(const fl_shape* s) { return (s->L + s->q_block - 1) / s->q_block; }

// ---------------------------------------------------------------------------------------------
// Device view of one side (K or V) of a store: base rows and the residual streams in loop order.
// ---------------------------------------------------------------------------------------------
struct DevStream {
  const uint8_t* codes;
  const __half* scale;
  const __half* zero;
  const int32_t* slot;
};
struct DevSide {
  const void* base;
  DevStream s[FL_MAX_LOOPS];
};

static inline void fl_dev_side(const fl_kv_store* st, bool is_k, DevSide* out) {
  out->base = is_k ? st->k_base : st->v_base;
  for (int i = 0; i < FL_MAX_LOOPS; ++i) {
    const fl_kv_stream& s = is_k ? st->k_res[i] : st->v_res[i];
    out->s[i].codes = static_cast<const uint8_t*>(s.codes);
    out->s[i].scale = reinterpret_cast<const __half*>(s.scale);
    out->s[i].zero = reinterpret_cast<const __half*>(s.zero);
    out->s[i].slot = s.slot_of_pos;
  }
}

#ifdef __CUDACC__
// ---- programmatic dependent launch ---------------------------------------------------------------------------
// The kernels of the step are launched with programmatic stream serialization: the next kernel of the stream may be
// scheduled, and run up to its fl_grid_wait(), while this one is still running. Rules every such kernel keeps:
// fl_grid_wait() (= the previous kernel of the stream has completed and its writes are visible) comes before the
// first access to anything an earlier kernel may still read or write, and fl_grid_release() (the next kernel may be
// scheduled) comes after it, so that whatever runs ahead of a wait sees everything up to two kernels back.
// Launched without the attribute both are no-ops.
__device__ __forceinline__ void fl_grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void fl_grid_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t fl_launch(const fl_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                             cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (ctx != nullptr && ctx->pdl) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- 8-element vector access in storage type ---------------------------------------------------
template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 raw = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 f = __bfloat1622float2(h[i]);
    v[2 * i] = f.x;
    v[2 * i + 1] = f.y;
  }
}
template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&v)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <typename T>
__device__ __forceinline__ void store8(T* p, const float (&v)[8]);
template <>
__device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 raw;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
  *reinterpret_cast<uint4*>(p) = raw;
}
template <>
__device__ __forceinline__ void store8<float>(float* p, const float (&v)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}

// Extract the 8 codes of one lane (8 consecutive elements) from the packed stream row.
// `off8` is the element offset inside the row (multiple of 8).
template <int BITS>
__device__ __forceinline__ void load_codes8(const uint8_t* row_codes, int off8, uint32_t (&c)[8]) {
  if (BITS == 8) {
    uint2 raw = *reinterpret_cast<const uint2*>(row_codes + off8);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      c[i] = (raw.x >> (8 * i)) & 0xFFu;
      c[4 + i] = (raw.y >> (8 * i)) & 0xFFu;
    }
  } else if (BITS == 4) {
    uint32_t raw = *reinterpret_cast<const uint32_t*>(row_codes + off8 / 2);
#pragma unroll
    for (int i = 0; i < 8; ++i) c[i] = (raw >> (4 * i)) & 0xFu;
  } else {  // 2 bits
    uint32_t raw = *reinterpret_cast<const uint16_t*>(row_codes + off8 / 4);
#pragma unroll
    for (int i = 0; i < 8; ++i) c[i] = (raw >> (2 * i)) & 0x3u;
  }
}

// Add one residual stream's contribution to 8 consecutive elements of position `pos` (Eq. 8):
// x <- x + D(code) in binary32 (or x <- stored row when the codec is off). Returns false when the
// position carries no payload in this stream. `elem` = h*dh + e0 is the element offset inside a row of
// d elements (multiple of 8).
template <typename T, int BITS>
__device__ __forceinline__ bool apply_stream8(const DevStream& st, int pos, int elem, int d, int group,
                                              float (&x)[8]) {
  const int slot = __ldg(st.slot + pos);
  if (slot < 0) return false;
  if (BITS == 16) {
    load8<T>(reinterpret_cast<const T*>(st.codes) + (size_t)slot * d + elem, x);
  } else {
    uint32_t c[8];
    load_codes8<BITS>(st.codes + (size_t)slot * (d * BITS / 8), elem, c);
    const int gs = 31 - __clz(group);   // the group is a power of two: shifts instead of runtime divisions
    const size_t gi = (size_t)slot * (d >> gs) + (elem >> gs);
    const float sc = __half2float(st.scale[gi]);
    const float zr = __half2float(st.zero[gi]);
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = __fadd_rn(x[i], __fmaf_rn((float)c[i], sc, zr));
  }
  return true;
}

// One stream's payload for 8 consecutive elements, fetched ahead of its use so that the loads of several
// streams (and columns) are in flight together; applying it is the arithmetic of apply_stream8.
template <typename T, int BITS>
struct Payload8 {
  uint4 raw;      // BITS 16: the stored row piece (first 16 bytes); 8: x,y; 4 and 2: x
  uint4 raw_hi;   // BITS 16 with binary32 storage: the second 16 bytes
  __half sc, zr;  // kept as loaded: converting here would make the load round wait for its own data
};
template <typename T, int BITS>
__device__ __forceinline__ void payload_load(const DevStream& st, int slot, int elem, int d, int group,
                                             Payload8<T, BITS>& p) {
  if (BITS == 16) {
    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(st.codes) + (size_t)slot * d + elem);
    p.raw = __ldg(src);
    if (sizeof(T) == 4) p.raw_hi = __ldg(src + 1);
  } else {
    const uint8_t* row = st.codes + (size_t)slot * (d * BITS / 8);
    if (BITS == 8) {
      const uint2 t = __ldg(reinterpret_cast<const uint2*>(row + elem));
      p.raw.x = t.x; p.raw.y = t.y;
    } else if (BITS == 4) {
      p.raw.x = __ldg(reinterpret_cast<const uint32_t*>(row + elem / 2));
    } else {
      p.raw.x = __ldg(reinterpret_cast<const uint16_t*>(row + elem / 4));
    }
    const int gs = 31 - __clz(group);   // the group is a power of two: shifts instead of runtime divisions
    const size_t gi = (size_t)slot * (d >> gs) + (elem >> gs);
    p.sc = __ldg(st.scale + gi);
    p.zr = __ldg(st.zero + gi);
  }
}
template <typename T, int BITS>
__device__ __forceinline__ void payload_apply(const Payload8<T, BITS>& p, float (&x)[8]) {
  if (BITS == 16) {
    if (sizeof(T) == 4) {
      x[0] = __uint_as_float(p.raw.x); x[1] = __uint_as_float(p.raw.y);
      x[2] = __uint_as_float(p.raw.z); x[3] = __uint_as_float(p.raw.w);
      x[4] = __uint_as_float(p.raw_hi.x); x[5] = __uint_as_float(p.raw_hi.y);
      x[6] = __uint_as_float(p.raw_hi.z); x[7] = __uint_as_float(p.raw_hi.w);
    } else {
      const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&p.raw);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(hp[i]);
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
      }
    }
  } else {
    const float sc = __half2float(p.sc), zr = __half2float(p.zr);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t c;
      if (BITS == 8) c = ((i < 4 ? p.raw.x : p.raw.y) >> (8 * (i & 3))) & 0xFFu;
      else if (BITS == 4) c = (p.raw.x >> (4 * i)) & 0xFu;
      else c = (p.raw.x >> (2 * i)) & 0x3u;
      // code -> float without the conversion unit: 2^23 + c is exact in binary32
      const float cf = __fsub_rn(__uint_as_float(0x4B000000u | c), 8388608.f);
      x[i] = __fadd_rn(x[i], __fmaf_rn(cf, sc, zr));
    }
  }
}

// Reconstruct 8 consecutive elements of Xhat after the first n_use residual streams
// (Eq. 8 chain in binary32, loop order): x = ((base + D_2) + D_3) + ...
template <typename T, int BITS>
__device__ __forceinline__ void recon8(const DevSide& side, int n_use, int pos, int elem, int d, int group,
                                       float (&x)[8]) {
  load8<T>(static_cast<const T*>(side.base) + (size_t)pos * d + elem, x);
  for (int s = 0; s < n_use; ++s) apply_stream8<T, BITS>(side.s[s], pos, elem, d, group, x);
}
#endif  // __CUDACC__
