// Hit rate of a selection (Sec. 3, Eq. 3-7): how many of the attention features of a generated
// query that exceed a threshold lie at positions the vote selected.  Pure counting: integer
// results, exact.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/snapkv.h"

namespace snapkv {
namespace {

constexpr int HIT_THREADS = 256;
constexpr int HIT_CHUNK = HIT_THREADS * 16;   // positions per block

// blockIdx.y = head (row); blockIdx.x = chunk of HIT_CHUNK positions and, with the same
// stride, of selected indices.  Per row two integer counters, added with atomics (integer
// sums do not depend on the order): out[2*row] = selected positions above the threshold
// (sum of O, Eq. 6), out[2*row + 1] = positions above the threshold (sum of M_threshold_cur).
__global__ void __launch_bounds__(HIT_THREADS)
hit_count_kernel(const float* __restrict__ a_cur, const int32_t* __restrict__ idx, int n, int k,
                 float theta, int32_t* __restrict__ out) {
  const int row = blockIdx.y;
  const float* arow = a_cur + static_cast<size_t>(row) * n;
  const int32_t* irow = idx + static_cast<size_t>(row) * k;
  const int c0 = blockIdx.x * HIT_CHUNK;
  int important = 0, hits = 0;
#pragma unroll 4
  for (int j = c0 + threadIdx.x; j < min(c0 + HIT_CHUNK, n); j += HIT_THREADS)
    important += __ldg(arow + j) > theta;
  for (int t = c0 + threadIdx.x; t < min(c0 + HIT_CHUNK, k); t += HIT_THREADS) {
    const int p = __ldg(irow + t);
    if (p >= 0 && p < n) hits += __ldg(arow + p) > theta;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    important += __shfl_xor_sync(0xffffffffu, important, o);
    hits += __shfl_xor_sync(0xffffffffu, hits, o);
  }
  __shared__ int s_imp[HIT_THREADS / 32], s_hit[HIT_THREADS / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { s_imp[warp] = important; s_hit[warp] = hits; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int ti = 0, th = 0;
    for (int w = 0; w < HIT_THREADS / 32; ++w) { ti += s_imp[w]; th += s_hit[w]; }
    if (th) atomicAdd(out + 2 * row, th);
    if (ti) atomicAdd(out + 2 * row + 1, ti);
  }
}

}  // namespace
}  // namespace snapkv

extern "C" snapkv_status_t snapkv_hit_counts(const float* a_cur, const int32_t* idx, int rows, int n,
                                             int k, float theta, int32_t* out_counts, void* stream) {
  using namespace snapkv;
  if (rows < 1 || n < 1 || k < 1 || k > n || !a_cur || !idx || !out_counts)
    return SNAPKV_ERR_INVALID_ARG;
  if (rows > 65535) return SNAPKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(a_cur) & 3) || (reinterpret_cast<uintptr_t>(idx) & 3) ||
      (reinterpret_cast<uintptr_t>(out_counts) & 3))
    return SNAPKV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(out_counts, 0, sizeof(int32_t) * 2 * static_cast<size_t>(rows), s) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  const dim3 grid((n + HIT_CHUNK - 1) / HIT_CHUNK, rows);
  hit_count_kernel<<<grid, HIT_THREADS, 0, s>>>(a_cur, idx, n, k, theta, out_counts);
  return cudaGetLastError() == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}
