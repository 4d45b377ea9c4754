// Index validation for the checked build (-DFL_DEBUG_BOUNDS; libflashloop_debug.so). Every entry point hands the index
// arrays it is about to trust (row lists, column lists and their counts, slot maps) to fl_debug_check() before it
// launches anything, and fl_select_tokens its two hidden-state matrices to fl_debug_check_finite(). In the checked build a small kernel reads each array (and nothing the indices point to), the host
// waits for its verdict, and on a violation the call returns FL_ERR_INVALID_ARG with that code also written to the
// caller's status word: no kernel that would follow a bad index is launched, and nothing traps. The wait makes the
// checked build unusable inside a stream capture and slow; it is for tests and debugging on small shapes.
// In the normal build the function is an empty stub.
#include "fl_internal.cuh"

#ifdef FL_DEBUG_BOUNDS

namespace {

// One violation is enough: the flag is set, never cleared, by any thread that sees one.
__global__ void __launch_bounds__(256) check_indices_kernel(fl_idx_check c, int* flag) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < c.n; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t seg = c.seg > 0 ? i / c.seg : 0, k = c.seg > 0 ? i - seg * c.seg : i;
    if (c.cnt != nullptr) {
      const int32_t m = c.cnt[seg];
      if (m < 0 || m > c.seg) { atomicExch(flag, 1); continue; }     // the count itself is out of range
      if (k >= m) continue;                                          // beyond the segment's valid entries
    }
    const int32_t v = c.a[i];
    bool bad = v < c.lo || v > c.hi;
    if (c.ascending && k > 0 && !bad) bad = c.a[i - 1] >= v;
    if (bad) atomicExch(flag, 1);
  }
}

// Inputs that must be finite (the token scores divide by a norm): bf16 or binary32 values, 8 per thread and step.
template <typename T>
__global__ void __launch_bounds__(256) check_finite_kernel(const T* __restrict__ x, int64_t n, int* flag) {
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    float v;
    if (sizeof(T) == 2) v = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[i]);
    else v = reinterpret_cast<const float*>(x)[i];
    bad |= !(fabsf(v) <= 3.4028234e38f);      // false for NaN and for infinities
  }
  if (bad) atomicExch(flag, 1);
}

}  // namespace

int fl_debug_check_finite(fl_ctx* ctx, const void* x, int64_t n, int dtype, int32_t* status, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (ctx->dbg_flag == nullptr) return FL_ERR_CUDA;
  int* flag = static_cast<int*>(ctx->dbg_flag);
  FL_CHECK_CUDA(cudaMemsetAsync(flag, 0, sizeof(int), st));
  int64_t blocks = (n + 255) / 256;
  if (blocks > 8192) blocks = 8192;
  if (n > 0 && x != nullptr) {
    if (dtype == FL_F32) check_finite_kernel<float><<<(int)blocks, 256, 0, st>>>(static_cast<const float*>(x), n, flag);
    else check_finite_kernel<__nv_bfloat16><<<(int)blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), n, flag);
  }
  int host_flag = 0;
  FL_CHECK_CUDA(cudaMemcpyAsync(&host_flag, flag, sizeof(int), cudaMemcpyDeviceToHost, st));
  FL_CHECK_CUDA(cudaStreamSynchronize(st));
  if (host_flag == 0) return FL_OK;
  if (status != nullptr) {
    const int32_t code = FL_ERR_INVALID_ARG;
    FL_CHECK_CUDA(cudaMemcpyAsync(status, &code, sizeof(code), cudaMemcpyHostToDevice, st));
    FL_CHECK_CUDA(cudaStreamSynchronize(st));
  }
  return FL_ERR_INVALID_ARG;
}

int fl_debug_init(fl_ctx* ctx) {
  FL_CHECK_CUDA(cudaMalloc(&ctx->dbg_flag, sizeof(int)));
  return FL_OK;
}

int fl_debug_check(fl_ctx* ctx, const fl_idx_check* checks, int n_checks, int32_t* status, void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (ctx->dbg_flag == nullptr) return FL_ERR_CUDA;
  int* flag = static_cast<int*>(ctx->dbg_flag);
  FL_CHECK_CUDA(cudaMemsetAsync(flag, 0, sizeof(int), st));
  for (int i = 0; i < n_checks; ++i) {
    const fl_idx_check& c = checks[i];
    if (c.a == nullptr || c.n <= 0) continue;
    int64_t blocks = (c.n + 255) / 256;
    if (blocks > 4096) blocks = 4096;
    check_indices_kernel<<<(int)blocks, 256, 0, st>>>(c, flag);
  }
  int host_flag = 0;
  FL_CHECK_CUDA(cudaMemcpyAsync(&host_flag, flag, sizeof(int), cudaMemcpyDeviceToHost, st));
  FL_CHECK_CUDA(cudaStreamSynchronize(st));
  if (host_flag == 0) return FL_OK;
  if (status != nullptr) {
    const int32_t code = FL_ERR_INVALID_ARG;
    FL_CHECK_CUDA(cudaMemcpyAsync(status, &code, sizeof(code), cudaMemcpyHostToDevice, st));
    FL_CHECK_CUDA(cudaStreamSynchronize(st));
  }
  return FL_ERR_INVALID_ARG;
}

int fl_debug_check_attn(fl_ctx* ctx, const fl_shape* s, int n_streams, const int32_t* active_idx, int32_t n_active,
                        const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt, int32_t c,
                        int64_t n_segments, int32_t* status, void* stream) {
  fl_idx_check ck[2 + 2 * FL_MAX_LOOPS];
  int n = 0;
  ck[n++] = {active_idx, n_active, 0, nullptr, 0, s->L - 1, 1};
  ck[n++] = {col_idx, n_segments * c, c, col_cnt, 0, s->L - 1, 1};
  for (int i = 0; i < n_streams; ++i) {
    ck[n++] = {store->k_res[i].slot_of_pos, s->L, 0, nullptr, -1, store->k_res[i].n_rows - 1, 0};
    ck[n++] = {store->v_res[i].slot_of_pos, s->L, 0, nullptr, -1, store->v_res[i].n_rows - 1, 0};
  }
  return fl_debug_check(ctx, ck, n, status, stream);
}

extern "C" int fl_debug_bounds_enabled(void) { return 1; }

#else

int fl_debug_check_attn(fl_ctx*, const fl_shape*, int, const int32_t*, int32_t, const fl_kv_store*, const int32_t*,
                        const int32_t*, int32_t, int64_t, int32_t*, void*) {
  return FL_OK;
}

int fl_debug_check(fl_ctx*, const fl_idx_check*, int, int32_t*, void*) { return FL_OK; }
int fl_debug_init(fl_ctx*) { return FL_OK; }
int fl_debug_check_finite(fl_ctx*, const void*, int64_t, int, int32_t*, void*) { return FL_OK; }

extern "C" int fl_debug_bounds_enabled(void) { return 0; }

#endif
