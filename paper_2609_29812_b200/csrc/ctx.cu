// Context, status strings, shared host-side validation and the KV-cache accounting call.
#include <cstdlib>
#include <cstring>
#include <new>
#include <unordered_map>

#include "fl_internal.cuh"

// Tensor maps are encoded once per (base pointer, rows, row elements, box rows) and kept in a hash table: a step of
// the 48-layer benchmark uses a few hundred of them and looks four up per attention call.
struct fl_tmap_key {
  const void* base;
  int64_t rows, row_elems;
  int box_rows;
  bool operator==(const fl_tmap_key& o) const {
    return base == o.base && rows == o.rows && row_elems == o.row_elems && box_rows == o.box_rows;
  }
};
struct fl_tmap_key_hash {
  size_t operator()(const fl_tmap_key& k) const {
    uint64_t x = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
    x ^= (uint64_t)k.rows * 0xC2B2AE3D27D4EB4Full + (uint64_t)k.row_elems * 0x165667B19E3779F9ull + (uint64_t)k.box_rows;
    return (size_t)(x ^ (x >> 29));
  }
};
struct fl_tmap_cache {
  std::unordered_map<fl_tmap_key, CUtensorMap, fl_tmap_key_hash> maps;
};

typedef CUresult (*fl_encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                       const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                       CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool fl_tile_tmap(fl_ctx* ctx, const void* base, int64_t rows, int64_t row_elems, int box_rows, CUtensorMap* out) {
  if (ctx->encode_tiled == nullptr || ctx->tmaps == nullptr) return false;
  if (rows < 1 || box_rows < 1 || box_rows > 256 || !fl_aligned16(base) || (row_elems * 2) % 16 != 0) return false;
  const fl_tmap_key key{base, rows, row_elems, box_rows};
  auto it = ctx->tmaps->maps.find(key);
  if (it != ctx->tmaps->maps.end()) { *out = it->second; return true; }
  CUtensorMap map;
  const cuuint64_t gdim[2] = {(cuuint64_t)row_elems, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)row_elems * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult rc = reinterpret_cast<fl_encode_tiled_fn>(ctx->encode_tiled)(
      &map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) return false;
  constexpr size_t kMaxEntries = 8192;   // a map describes memory the caller may free and reuse: start over when full
  if (ctx->tmaps->maps.size() >= kMaxEntries) ctx->tmaps->maps.clear();
  ctx->tmaps->maps.emplace(key, map);
  *out = map;
  return true;
}

extern "C" int fl_version(void) { return 100; }

extern "C" const char* fl_status_string(int status) {
  switch (status) {
    case FL_OK: return "ok";
    case FL_ERR_INVALID_ARG: return "invalid argument";
    case FL_ERR_UNSUPPORTED: return "unsupported configuration";
    case FL_ERR_WORKSPACE: return "problem exceeds the context workspace";
    case FL_ERR_CUDA: return "CUDA runtime error";
    case FL_ERR_TIMEOUT: return "bounded device wait ran out";
    default: return "unknown status";
  }
}

extern "C" int fl_create(fl_ctx** out, int device) {
  if (out == nullptr) return FL_ERR_INVALID_ARG;
  *out = nullptr;
  int n_dev = 0;
  FL_CHECK_CUDA(cudaGetDeviceCount(&n_dev));
  if (device < 0 || device >= n_dev) return FL_ERR_INVALID_ARG;
  FL_CHECK_CUDA(cudaSetDevice(device));
  fl_ctx* c = new (std::nothrow) fl_ctx();
  if (c == nullptr) return FL_ERR_CUDA;
  c->device = device;
  {
    const char* no_pdl = std::getenv("FL_NO_PDL");
    c->pdl = (no_pdl != nullptr && no_pdl[0] == '1') ? 0 : 1;
  }
  if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) {
    delete c;
    return FL_ERR_CUDA;
  }
  const char* env = std::getenv("FL_FORCE_SIMT");
  c->force_simt = (env != nullptr && env[0] == '1') ? 1 : 0;
  const char* fused = std::getenv("FL_FUSED_ATTN");
  c->fused_attn = (fused != nullptr && fused[0] == '1') ? 1 : 0;
  const char* two_pass = std::getenv("FL_TWO_PASS");
  c->two_pass = (two_pass != nullptr && two_pass[0] == '1') ? 1 : 0;
  const char* qn = std::getenv("FL_QUANT_NARROW");
  c->quant_narrow = (qn != nullptr && qn[0] == '1') ? 1 : 0;
  c->dbg_flag = nullptr;
  c->encode_tiled = nullptr;
  {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      c->encode_tiled = fn;
    (void)cudaGetLastError();
  }
  c->tmaps = new (std::nothrow) fl_tmap_cache();
  if (c->tmaps == nullptr) {
    delete c;
    return FL_ERR_CUDA;
  }
  if (fl_debug_init(c) != FL_OK) {
    delete c->tmaps;
    delete c;
    return FL_ERR_CUDA;
  }
  *out = c;
  return FL_OK;
}

extern "C" int fl_destroy(fl_ctx* ctx) {
  if (ctx == nullptr) return FL_ERR_INVALID_ARG;
  if (ctx->dbg_flag != nullptr) (void)cudaFree(ctx->dbg_flag);
  delete ctx->tmaps;
  delete ctx;
  return FL_OK;
}

int fl_launch_status() { return cudaGetLastError() == cudaSuccess ? FL_OK : FL_ERR_CUDA; }

int fl_check_shape(const fl_shape* s) {
  if (s == nullptr) return FL_ERR_INVALID_ARG;
  if (s->L < 1 || s->n_heads < 1 || s->q_block < 1) return FL_ERR_INVALID_ARG;
  if (s->dtype != FL_BF16 && s->dtype != FL_F32) return FL_ERR_INVALID_ARG;
  if (s->bits != 2 && s->bits != 4 && s->bits != 8 && s->bits != 16) return FL_ERR_INVALID_ARG;
  if (s->head_dim < 1) return FL_ERR_INVALID_ARG;
  if (s->group != 8 && s->group != 16 && s->group != 32 && s->group != 64 && s->group != 128)
    return FL_ERR_INVALID_ARG;
  if (s->head_dim % s->group != 0) return FL_ERR_INVALID_ARG;
  if (!(s->eps >= 0.f) || !(s->sm_scale > 0.f)) return FL_ERR_INVALID_ARG;
  if (s->head_dim != 64 && s->head_dim != 128) return FL_ERR_UNSUPPORTED;
  if ((int64_t)s->L * s->n_heads * s->head_dim > (int64_t(1) << 40)) return FL_ERR_INVALID_ARG;
  return FL_OK;
}

// The first n_streams_needed streams must be complete.
int fl_check_store(const fl_shape* s, const fl_kv_store* st, int n_streams_needed) {
  if (st == nullptr) return FL_ERR_INVALID_ARG;
  if (st->k_base == nullptr || st->v_base == nullptr) return FL_ERR_INVALID_ARG;
  if (!fl_aligned16(st->k_base) || !fl_aligned16(st->v_base)) return FL_ERR_INVALID_ARG;
  if (n_streams_needed < 0 || n_streams_needed > FL_MAX_LOOPS) return FL_ERR_INVALID_ARG;
  if (st->n_streams < n_streams_needed || st->n_streams > FL_MAX_LOOPS) return FL_ERR_INVALID_ARG;
  for (int i = 0; i < n_streams_needed; ++i) {
    for (int side = 0; side < 2; ++side) {
      const fl_kv_stream& r = side == 0 ? st->k_res[i] : st->v_res[i];
      if (r.n_rows < 0 || r.n_rows > s->L) return FL_ERR_INVALID_ARG;
      if (r.slot_of_pos == nullptr) return FL_ERR_INVALID_ARG;
      if (r.rows_prev != nullptr && r.rows_cur == nullptr) return FL_ERR_INVALID_ARG;   // rows_cur alone is fine
      if (!fl_aligned16(r.rows_prev) || !fl_aligned16(r.rows_cur)) return FL_ERR_INVALID_ARG;
      if (r.n_rows > 0) {
        if (r.codes == nullptr || !fl_aligned16(r.codes)) return FL_ERR_INVALID_ARG;
        if (s->bits != 16) {
          if (r.scale == nullptr || r.zero == nullptr) return FL_ERR_INVALID_ARG;
          if (!fl_aligned16(r.scale) || !fl_aligned16(r.zero)) return FL_ERR_INVALID_ARG;
        }
      }
    }
    if (st->k_res[i].n_rows != st->v_res[i].n_rows) return FL_ERR_INVALID_ARG;
    if ((st->k_res[i].rows_prev == nullptr) != (st->v_res[i].rows_prev == nullptr)) return FL_ERR_INVALID_ARG;
    if ((st->k_res[i].rows_cur == nullptr) != (st->v_res[i].rows_cur == nullptr)) return FL_ERR_INVALID_ARG;
  }
  return FL_OK;
}

extern "C" int fl_kv_store_bytes(const fl_shape* shape, const fl_kv_store* store, int n_loops, int share_layers,
                                 int64_t* flashloop_bytes, int64_t* dense_bytes) {
  int rc = fl_check_shape(shape);
  if (rc != FL_OK) return rc;
  if (store == nullptr || flashloop_bytes == nullptr || dense_bytes == nullptr) return FL_ERR_INVALID_ARG;
  if (n_loops < 1 || n_loops > FL_MAX_LOOPS + 1 || share_layers < 1) return FL_ERR_INVALID_ARG;
  if (store->n_streams < n_loops - 1) return FL_ERR_INVALID_ARG;
  const int64_t d = (int64_t)shape->n_heads * shape->head_dim;
  const int64_t e = fl_elem_bytes(shape);
  const int64_t row_payload =
      shape->bits == 16 ? 2 * d * e : 2 * (d * shape->bits / 8 + 2 * 2 * (d / shape->group));
  int64_t total = 2 * (int64_t)shape->L * d * e;  // loop-1 base, K and V
  for (int i = 0; i < n_loops - 1; ++i) {
    const int64_t n = store->k_res[i].n_rows;
    total += n * row_payload;
    total += (4 * ((int64_t)shape->L + n) + share_layers - 1) / share_layers;  // slot map + index list
  }
  *flashloop_bytes = total;
  *dense_bytes = (int64_t)n_loops * 2 * shape->L * d * e;
  return FL_OK;
}
