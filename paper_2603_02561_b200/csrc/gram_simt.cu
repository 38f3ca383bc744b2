// Streaming Gram pass, FFMA version: P[b,s] = sum_{n in slice s} h_n h_n^T.
// Used for fp32 storage (bf16 products would break the 1e-4 tolerance of that mode),
// for d = 32 and for N < 128 (shapes the tensor-core kernel does not take);
// G_b = H_b^T H_b is the matrix whose eigenvectors are V of Eq. 9.
#include "solar_internal.cuh"

namespace solar {

template <typename T, int D>
__global__ void __launch_bounds__(256)
gram_simt_kernel(const T* __restrict__ H, float* __restrict__ gpart, int* __restrict__ status,
                 int N, int chunk_rows, int splits) {
  constexpr int TR = 32;      // rows staged per step
  constexpr int R = D / 16;   // each thread owns an R x R register tile of G
  __shared__ float tile[TR][D];

  const int b = blockIdx.y, s = blockIdx.x;
  const int row0 = s * chunk_rows;
  const int row1 = min(N, row0 + chunk_rows);
  const T* Hb = H + (size_t)b * N * D;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

  float acc[R][R];
#pragma unroll
  for (int i = 0; i < R; ++i)
#pragma unroll
    for (int j = 0; j < R; ++j) acc[i][j] = 0.f;

  constexpr int VE = Vec16<T>::kElems;
  constexpr int VPR = D / VE;
  for (int base = row0; base < row1; base += TR) {
    for (int v = threadIdx.x; v < TR * VPR; v += 256) {
      const int rr = v / VPR, cc = (v % VPR) * VE;
      float tmp[VE];
      if (base + rr < row1) {
        Vec16<T>::load(Hb + (size_t)(base + rr) * D + cc, tmp);
      } else {
#pragma unroll
        for (int e = 0; e < VE; ++e) tmp[e] = 0.f;   // zero rows add nothing to a Gram
      }
#pragma unroll
      for (int e = 0; e < VE; ++e) tile[rr][cc + e] = tmp[e];
    }
    __syncthreads();
#pragma unroll 4
    for (int k = 0; k < TR; ++k) {
      float a[R], c[R];
#pragma unroll
      for (int i = 0; i < R; ++i) a[i] = tile[k][ty + 16 * i];
#pragma unroll
      for (int j = 0; j < R; ++j) c[j] = tile[k][tx + 16 * j];
#pragma unroll
      for (int i = 0; i < R; ++i)
#pragma unroll
        for (int j = 0; j < R; ++j) acc[i][j] = fmaf(a[i], c[j], acc[i][j]);
    }
    __syncthreads();
  }

  float* out = gpart + ((size_t)b * splits + s) * D * D;
#pragma unroll
  for (int i = 0; i < R; ++i)
#pragma unroll
    for (int j = 0; j < R; ++j) out[(ty + 16 * i) * D + tx + 16 * j] = acc[i][j];
  if (threadIdx.x == 0) status[b * splits + s] = kGramStatusOk;   // this kernel has no waits to lose
}

template <typename T>
static cudaError_t launch_t(int B, int N, int d, const void* H, float* gpart, int* status,
                            const GramPlan& plan, cudaStream_t st) {
  const dim3 grid(plan.splits, B), block(256);
  const int chunk_rows = plan.chunk_tiles * kGramTileRows;
  const T* h = static_cast<const T*>(H);
  switch (d) {
    case 32: gram_simt_kernel<T, 32><<<grid, block, 0, st>>>(h, gpart, status, N, chunk_rows, plan.splits); break;
    case 64: gram_simt_kernel<T, 64><<<grid, block, 0, st>>>(h, gpart, status, N, chunk_rows, plan.splits); break;
    case 128: gram_simt_kernel<T, 128><<<grid, block, 0, st>>>(h, gpart, status, N, chunk_rows, plan.splits); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_gram_simt(int B, int N, int d, solar_dtype_t dt, const void* H, float* gpart,
                             int* status, const GramPlan& plan, cudaStream_t st) {
  return dt == SOLAR_BF16 ? launch_t<__nv_bfloat16>(B, N, d, H, gpart, status, plan, st)
                          : launch_t<float>(B, N, d, H, gpart, status, plan, st);
}

}  // namespace solar
