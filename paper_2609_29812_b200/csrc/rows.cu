// Active-row gather / scatter (Appendix G: only the selected token rows are processed; inactive rows
// keep their hidden states and KV entries). HBM-bound copies: one warp per row, 16-byte accesses.
#include "fl_internal.cuh"

namespace {

template <bool GATHER>
__global__ void __launch_bounds__(256) rows_copy_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ idx,
                                                        int n, int vec_per_row, uint4* __restrict__ dst) {
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  for (int t = blockIdx.x * warps_per_block + (threadIdx.x >> 5); t < n; t += gridDim.x * warps_per_block) {
    const int64_t row = __ldg(idx + t);
    const uint4* s = src + (GATHER ? row : (int64_t)t) * vec_per_row;
    uint4* d = dst + (GATHER ? (int64_t)t : row) * vec_per_row;
    int v = lane;
    // four independent 16-byte loads in flight per lane before the stores
    for (; v + 96 < vec_per_row; v += 128) {
      uint4 a = __ldg(s + v), b = __ldg(s + v + 32), c = __ldg(s + v + 64), e = __ldg(s + v + 96);
      d[v] = a; d[v + 32] = b; d[v + 64] = c; d[v + 96] = e;
    }
    for (; v < vec_per_row; v += 32) d[v] = __ldg(s + v);
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
  const int warps = 8;
  int grid = (n + warps - 1) / warps;
  const int max_grid = ctx->sm_count * 16;
  if (grid > max_grid) grid = max_grid;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (gather)
    rows_copy_kernel<true><<<grid, warps * 32, 0, st>>>(static_cast<const uint4*>(src), idx, n, (int)(row_bytes / 16),
                                                        static_cast<uint4*>(dst));
  else
    rows_copy_kernel<false><<<grid, warps * 32, 0, st>>>(static_cast<const uint4*>(src), idx, n,
                                                         (int)(row_bytes / 16), static_cast<uint4*>(dst));
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
