// fw_cov_block_static: first-block mean and covariance of a block of patch rows
// for callers that can neither allocate device memory nor hand the library a
// workspace.  The split partial sums live in a fixed array that is part of the
// library image, so the call needs nothing but its inputs and outputs.
//
// Who needs this: code that runs where device allocation is off limits, e.g. a
// gradient hook called by a training framework whose caching allocator owns
// all device memory (a raw cudaMalloc there synchronises the whole device and
// can fail although the framework still has free blocks), or a monitoring
// callback that must not disturb the allocator's state between iterations.
//
// Cost of the convenience: every GPU that loads the library carries the
// scratch array (kScratchFloats * 4 bytes = 8 MiB) until the process exits, M
// is limited to FW_STATIC_MAX_M, and all calls share the one array.
#include <cstdio>

#include "fw_internal.h"

namespace {

constexpr int kMaxM = FW_STATIC_MAX_M;                 // 256
constexpr size_t kScratchFloats = (size_t)2 << 20;     // 2 Mi floats = 8 MiB
constexpr int kMaxSplits = 64;
constexpr int kMaxDevices = 64;

// Scratch for the split partial sums.  In host code this name is only a
// stand-in for the symbol: its device address is obtained once per device with
// cudaGetSymbolAddress (below) and passed to the kernels as an ordinary pointer.
static __device__ __align__(256) float g_static_scratch[kScratchFloats];

float* g_scratch_ptr[kMaxDevices] = {nullptr};

// Partial column sums: grid (ceil(M/32), splits), block (32, 8).
__global__ void static_colsum_kernel(const float* __restrict__ X, int64_t rows, int64_t ldx, int M, int splits,
                                     float* __restrict__ part /* splits x M */) {
  const int col = blockIdx.x * 32 + threadIdx.x;
  const int64_t per = (rows + splits - 1) / splits;
  const int64_t r0 = blockIdx.y * per;
  int64_t r1 = r0 + per;
  if (r1 > rows) r1 = rows;
  float acc = 0.f;
  if (col < M)
    for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) acc += X[r * ldx + col];
  __shared__ float sm[8][33];
  sm[threadIdx.y][threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.y == 0 && col < M) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += sm[i][threadIdx.x];
    part[(int64_t)blockIdx.y * M + col] = s;
  }
}

// mu = (sum of the partial column sums) / rows     (Eq. 4)
__global__ void static_mean_kernel(const float* __restrict__ part, int splits, int M, float inv_rows,
                                   float* __restrict__ mu) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= M) return;
  float s = 0.f;
  for (int k = 0; k < splits; ++k) s += part[(int64_t)k * M + m];
  mu[m] = s * inv_rows;
}

// Partial centred Gram: each CTA owns a 32x32 tile of the upper triangle and one
// row split; grid (tiles, tiles, splits), block (32, 8), 4 outputs per thread.
__global__ void static_gram_kernel(const float* __restrict__ X, const float* __restrict__ mu, int64_t rows,
                                   int64_t ldx, int M, int splits, float* __restrict__ part /* splits x M x M */) {
  const int bi = blockIdx.y, bj = blockIdx.x;
  if (bj < bi) return;
  const int64_t per = (rows + splits - 1) / splits;
  const int64_t r0 = blockIdx.z * per;
  int64_t r1 = r0 + per;
  if (r1 > rows) r1 = rows;
  __shared__ float As[32][33], Bs[32][33];
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  const int ci = bi * 32 + threadIdx.x, cj = bj * 32 + threadIdx.x;
  const float mi = ci < M ? mu[ci] : 0.f, mj = cj < M ? mu[cj] : 0.f;
  for (int64_t rb = r0; rb < r1; rb += 32) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int rr = threadIdx.y + 8 * q;
      const int64_t r = rb + rr;
      const bool in = r < r1;
      As[rr][threadIdx.x] = (in && ci < M) ? X[r * ldx + ci] - mi : 0.f;
      Bs[rr][threadIdx.x] = (in && cj < M) ? X[r * ldx + cj] - mj : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < 32; ++k) {
      const float b = Bs[k][threadIdx.x];
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[q] = fmaf(As[k][threadIdx.y + 8 * q], b, acc[q]);
    }
    __syncthreads();
  }
  float* P = part + (int64_t)blockIdx.z * M * M;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int i = bi * 32 + threadIdx.y + 8 * q, j = bj * 32 + threadIdx.x;
    if (i < M && j < M) P[(int64_t)i * M + j] = acc[q];
  }
}

// Phix = (sum of the partial Grams) / rows, mirrored to the lower triangle   (Eq. 5)
__global__ void static_reduce_kernel(const float* __restrict__ part, int splits, int M, float inv_rows,
                                     float* __restrict__ Phix) {
  const int j = blockIdx.x * 32 + threadIdx.x;
  const int i = blockIdx.y * 8 + threadIdx.y;
  if (i >= M || j >= M || (j >> 5) < (i >> 5)) return;      // tiles of the upper triangle only
  float s = 0.f;
  for (int k = 0; k < splits; ++k) s += part[(int64_t)k * M * M + (int64_t)i * M + j];
  s *= inv_rows;
  if (j >= i) {
    Phix[(int64_t)i * M + j] = s;
    Phix[(int64_t)j * M + i] = s;
  }
}

}  // namespace

extern "C" fw_status fw_cov_block_static(const float* X, int64_t rows, int64_t ldx, int32_t M, float* mu_out,
                                         float* phix_out, void* cuda_stream) {
  if (!X || !mu_out || !phix_out) return FW_ERR_INVALID_ARG;
  if (M < 1 || rows < 1 || ldx < M) return FW_ERR_SHAPE;
  if (M > kMaxM) {
    fprintf(stderr, "[fw] fw_cov_block_static: M = %d exceeds the static scratch limit FW_STATIC_MAX_M = %d\n",
            (int)M, kMaxM);
    return FW_ERR_SHAPE;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return FW_ERR_CUDA;
  }
  if (!g_scratch_ptr[dev]) {
    // one-time set-up on this device: resolve the device address of the scratch symbol
    float* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      fprintf(stderr, "[fw] fw_cov_block_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      cudaGetLastError();
      return FW_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  float* scratch = g_scratch_ptr[dev];
  cudaStream_t s = (cudaStream_t)cuda_stream;
  // as many row splits as the scratch array holds (every slot used is fully overwritten,
  // so nothing has to start at zero)
  int64_t splits = (int64_t)(kScratchFloats / ((size_t)M * M));
  if (splits > kMaxSplits) splits = kMaxSplits;
  const int64_t by_rows = (rows + 63) / 64;
  if (splits > by_rows) splits = by_rows;
  if (splits < 1) splits = 1;
  const int sp = (int)splits;
  const float inv_rows = 1.0f / (float)rows;
  const int t = (M + 31) / 32;
  {
    fw::ProfScope ps(FW_PROF_MISC, s);
    static_colsum_kernel<<<dim3(t, sp), dim3(32, 8), 0, s>>>(X, rows, ldx, M, sp, scratch);
  }
  {
    fw::ProfScope ps(FW_PROF_MISC, s);
    static_mean_kernel<<<(M + 127) / 128, 128, 0, s>>>(scratch, sp, M, inv_rows, mu_out);
  }
  {
    fw::ProfScope ps(FW_PROF_MISC, s);
    static_gram_kernel<<<dim3(t, t, sp), dim3(32, 8), 0, s>>>(X, mu_out, rows, ldx, M, sp, scratch);
  }
  {
    fw::ProfScope ps(FW_PROF_MISC, s);
    static_reduce_kernel<<<dim3(t, (M + 7) / 8), dim3(32, 8), 0, s>>>(scratch, sp, M, inv_rows, phix_out);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    fprintf(stderr, "[fw] fw_cov_block_static: launch failed: %s\n", cudaGetErrorString(e));
    return FW_ERR_CUDA;
  }
  return FW_OK;
}
