// Analysis utility: per-token divergence of two KV caches (Sec. 3.2, the MSE_token equation),
//   out[r] = ||K_a[r] - K_b[r]||^2 + ||V_a[r] - V_b[r]||^2   for every row r (one token of one head),
// which the paper uses to show where the prompt's information concentrates (the cache of the guided
// branch against that of the native branch).  Pure streaming: 1 KB read and 4 bytes written per row,
// 3 flops per 4 bytes, so the kernel is built to keep HBM busy: a row is read by 8 lanes with 128-bit
// loads (32 bytes per lane and tensor), a warp takes 4 rows at a time and two such groups per
// iteration, which puts 16 independent 16-byte loads in flight per lane; 3 shuffles finish a row.
#include "ssd_internal.cuh"

namespace ssd {
namespace {

constexpr int kMseThreads = 256;
constexpr int kMseRowsPerWarpIter = 8;    // two groups of four rows

__device__ __forceinline__ float sq_diff8(const uint4& a, const uint4& b) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float d0 = __uint_as_float(aw[i] << 16) - __uint_as_float(bw[i] << 16);
    const float d1 = __uint_as_float(aw[i] & 0xffff0000u) - __uint_as_float(bw[i] & 0xffff0000u);
    s = fmaf(d0, d0, s);
    s = fmaf(d1, d1, s);
  }
  return s;
}

__global__ void __launch_bounds__(kMseThreads) ssd_kv_token_mse_kernel(const uint4* __restrict__ ka, const uint4* __restrict__ va,
                                                                       const uint4* __restrict__ kb, const uint4* __restrict__ vb,
                                                                       long long n_rows, float* __restrict__ out) {
  const int lane = threadIdx.x & 31, grp = lane >> 3, l8 = lane & 7;
  const long long warp = ((long long)blockIdx.x * kMseThreads + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * kMseThreads) >> 5;
  for (long long r0 = warp * kMseRowsPerWarpIter; r0 < n_rows; r0 += n_warps * kMseRowsPerWarpIter) {
    uint4 x[2][8];
    bool ok[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const long long r = r0 + 4 * u + grp;
      ok[u] = r < n_rows;
      if (ok[u]) {
        const size_t o = (size_t)r * 16 + l8;            // a row is 16 uint4; this lane takes uint4 l8 and l8 + 8
        x[u][0] = ka[o]; x[u][1] = ka[o + 8];
        x[u][2] = kb[o]; x[u][3] = kb[o + 8];
        x[u][4] = va[o]; x[u][5] = va[o + 8];
        x[u][6] = vb[o]; x[u][7] = vb[o + 8];
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      float s = 0.f;
      if (ok[u]) s = (sq_diff8(x[u][0], x[u][2]) + sq_diff8(x[u][1], x[u][3])) + (sq_diff8(x[u][4], x[u][6]) + sq_diff8(x[u][5], x[u][7]));
      s += __shfl_xor_sync(0xffffffffu, s, 4);
      s += __shfl_xor_sync(0xffffffffu, s, 2);
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      if (ok[u] && l8 == 0) out[r0 + 4 * u + grp] = s;
    }
  }
}

}  // namespace
}  // namespace ssd

using namespace ssd;

extern "C" int ssd_kv_token_mse(const void* k_a, const void* v_a, const void* k_b, const void* v_b, int64_t n_rows,
                                float* mse_out, void* stream) {
  if (!k_a || !v_a || !k_b || !v_b || !mse_out || n_rows < 0 || n_rows > (int64_t)1 << 40) return SSD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_a) | reinterpret_cast<uintptr_t>(v_a) | reinterpret_cast<uintptr_t>(k_b) |
       reinterpret_cast<uintptr_t>(v_b)) % 16 != 0 || reinterpret_cast<uintptr_t>(mse_out) % 4 != 0)
    return SSD_ERR_INVALID_ARG;
  if (n_rows == 0) return SSD_OK;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return SSD_ERR_CUDA;
  }
  // eight resident blocks per SM; never more warps than there are groups of rows
  const long long groups = (n_rows + kMseRowsPerWarpIter - 1) / kMseRowsPerWarpIter;
  long long blocks = (groups * 32 + kMseThreads - 1) / kMseThreads;
  if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
  ssd_kv_token_mse_kernel<<<(unsigned)blocks, kMseThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(k_a), static_cast<const uint4*>(v_a), static_cast<const uint4*>(k_b),
      static_cast<const uint4*>(v_b), (long long)n_rows, mse_out);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? SSD_OK : SSD_ERR_CUDA;
}
