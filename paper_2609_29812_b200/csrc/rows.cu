// Active-row gather / scatter (Appendix G: only the selected token rows are processed; inactive rows
// keep their hidden states and KV entries). HBM-bound copies with 16-byte accesses.
#include "fl_internal.cuh"

namespace {

// One warp per piece of at most 128 vectors (2 KB) of a row: a lane has its (up to) four 16-byte loads in flight at
// once, and a row of several KB is spread over several warps, so that the launch is two dependent rounds deep (index,
// then data) however wide the rows are.
template <bool GATHER>
__global__ void __launch_bounds__(256) rows_copy_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ idx,
                                                        int n, int vec_per_row, int pieces, uint4* __restrict__ dst) {
  fl_grid_wait();
  fl_grid_release();
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t n_work = (int64_t)n * pieces;
  for (int64_t wi = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); wi < n_work;
       wi += (int64_t)gridDim.x * warps_per_block) {
    const int t = (int)(wi / pieces), piece = (int)(wi - (int64_t)t * pieces);
    const int64_t row = __ldg(idx + t);
    const uint4* s = src + (GATHER ? row : (int64_t)t) * vec_per_row;
    uint4* d = dst + (GATHER ? (int64_t)t : row) * vec_per_row;
    const int v0 = piece * 128 + lane, v_end = min(vec_per_row, (piece + 1) * 128);
    uint4 r[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (v0 + 32 * k < v_end) r[k] = __ldg(s + v0 + 32 * k);
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (v0 + 32 * k < v_end) d[v0 + 32 * k] = r[k];
  }
}

int rows_copy(bool gather, fl_ctx* ctx, const void* src, const int32_t* idx, int32_t n, int64_t row_bytes, void* dst,
              void* stream) {
  FL_REQUIRE(ctx != nullptr);
  FL_REQUIRE(n >= 0);
  FL_REQUIRE(row_bytes > 0 && row_bytes % 16 == 0 && row_bytes / 16 <= INT32_MAX);
  if (n == 0) return FL_OK;
  FL_REQUIRE(src != nullptr && dst != nullptr && idx != nullptr);
  FL_REQUIRE(fl_aligned16(src) && fl_aligned16(dst));
  {
    // the row count of the indexed matrix is not part of this call: only sign and order can be checked
    const fl_idx_check ck = {idx, n, 0, nullptr, 0, INT32_MAX, 1};
    const int rc = fl_debug_check(ctx, &ck, 1, nullptr, stream);
    if (rc != FL_OK) return rc;
  }
  const int warps = 8;
  const int vec_per_row = (int)(row_bytes / 16);
  const int pieces = (vec_per_row + 127) / 128;
  int64_t grid64 = ((int64_t)n * pieces + warps - 1) / warps;
  const int64_t max_grid = (int64_t)ctx->sm_count * 32;
  const int grid = (int)(grid64 > max_grid ? max_grid : grid64);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (gather)
    FL_CHECK_CUDA(fl_launch(ctx, rows_copy_kernel<true>, dim3(grid), dim3(warps * 32), 0, st,
                            static_cast<const uint4*>(src), idx, n, vec_per_row, pieces, static_cast<uint4*>(dst)));
  else
    FL_CHECK_CUDA(fl_launch(ctx, rows_copy_kernel<false>, dim3(grid), dim3(warps * 32), 0, st,
                            static_cast<const uint4*>(src), idx, n, vec_per_row, pieces, static_cast<uint4*>(dst)));
  return fl_launch_status();
}

}  // namespace

extern "C" int fl_gather_rows(fl_ctx* ctx, const void* src, const int32_t* idx, int32_t n, int64_t row_bytes, void* dst,
                              void* stream) {
  return rows_copy(true, ctx, src, idx, n, row_bytes, dst, stream);
}

extern "C" int fl_scatter_update(fl_ctx* ctx, const void* src, const int32_t* idx, int32_t n, int64_t row_bytes,
                                 void* dst, void* stream) {
  return rows_copy(false, ctx, src, idx, n, row_bytes, dst, stream);
}
