// fl_loop_attention_indexed_static: the position-indexed loop attention with the workspace of its last-wave split
// taken from a fixed array in device memory instead of a buffer of the caller. Nothing here corresponds to anything in
// the paper: it is a convenience for callers that cannot hand over device memory.
#include "fl_internal.cuh"

int fl_attn_indexed_check(const fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                          const void* q_store_in, const void* q_store_out, const int32_t* active_idx, int32_t n_active,
                          const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt, int32_t c,
                          const float* lse_in, const float* lse_out, const void* o_store_in, const void* o_store_out,
                          const fl_attn_carry* carry, int* launch);

namespace {

constexpr int kStaticPairs = 74;   // problems of a last wave that can be split: half of the 148 SMs of a B200
constexpr size_t kStaticBytes =
    (size_t)kFlMaxSplit * sizeof(int32_t) + (size_t)kStaticPairs * 2 * kFlPartFloats * sizeof(float);

// The scratch itself: part of the library's device image (no allocation call ever made for it). Every device that
// loads the library holds its own copy of these 19.7 MB until the process exits, whether this entry point is used
// or not.
static __device__ __align__(256) unsigned char g_attn_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];   // device address of g_attn_scratch, looked up once per device

}  // namespace

extern "C" int fl_loop_attention_indexed_static(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                                                const void* q_store_in, void* q_store_out, const int32_t* active_idx,
                                                int32_t n_active, const fl_kv_store* store, const int32_t* col_idx,
                                                const int32_t* col_cnt, int32_t c, const float* lse_in, float* lse_out,
                                                const void* o_store_in, void* o_store_out, float* col_scores_next,
                                                int32_t* status, void* stream) {
  // the same host checks as the workspace form, before anything is enqueued
  int launch = 0;
  const int rc = fl_attn_indexed_check(ctx, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active, store,
                                       col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out, nullptr, &launch);
  if (rc != FL_OK) return rc;
  FL_REQUIRE(ctx->device >= 0 && ctx->device < kMaxDevices);
  // the split this shape would use must fit the fixed array: no silent fall-back to something else
  const size_t need = fl_attn_workspace_bytes(ctx, shape);
  if (need > kStaticBytes) return FL_ERR_WORKSPACE;
  fl_ctx with_scratch = *ctx;   // differs from the caller's context only in its workspace (owns nothing)
  with_scratch.ws = nullptr;
  with_scratch.ws_bytes = 0;
  if (launch && need > 0) {
    // The symbol's address is the CURRENT device's copy of the array: it is looked up, and cached, only while the
    // context's device is the current one. A caller on another device gets an error and nothing is cached.
    int current = -1;
    FL_CHECK_CUDA(cudaGetDevice(&current));
    if (current != ctx->device) return FL_ERR_CUDA;
    if (g_scratch_addr[ctx->device] == nullptr) {
      void* addr = nullptr;
      FL_CHECK_CUDA(cudaGetSymbolAddress(&addr, g_attn_scratch));
      if (addr == nullptr) return FL_ERR_CUDA;
      g_scratch_addr[ctx->device] = addr;
    }
    void* scratch = g_scratch_addr[ctx->device];
    // the arrival counters at the head of the scratch must be zero when the kernel starts (an earlier call that
    // ended in an error may have left them otherwise)
    FL_CHECK_CUDA(cudaMemsetAsync(scratch, 0, (size_t)kFlMaxSplit * sizeof(int32_t), static_cast<cudaStream_t>(stream)));
    with_scratch.ws = scratch;
    with_scratch.ws_bytes = kStaticBytes;
  }
  return fl_loop_attention_indexed(&with_scratch, shape, loop_r, q_new, q_store_in, q_store_out, active_idx, n_active,
                                   store, col_idx, col_cnt, c, lse_in, lse_out, o_store_in, o_store_out,
                                   col_scores_next, status, stream);
}
